// Parent array -> packed ancestor bitmasks and depths (Sec. 2, the mask(A) equation, plus the self bit).
//
// One CTA per request.  Rows live in shared memory and are completed by pointer jumping on bitsets:
// every node keeps a pointer `anc` (initially its parent) and a row that covers the node and all its
// ancestors below `anc`; one round does  row[i] |= row[anc[i]],  dist[i] += dist[anc[i]],
// anc[i] = anc[anc[i]],  which doubles the covered path, so ceil(log2(depth + 1)) rounds finish the
// tree.  OR-ing a row that another thread is extending in the same round is harmless: every bit a
// row ever holds is an ancestor-or-self of its node, hence an ancestor of the reader too.
// A parent index outside {-1} U [0, i) makes that node a root and reports DYSPEC_ERR_BAD_TREE.
#include "common.cuh"

namespace dyspec {

__global__ void __launch_bounds__(1024, 1)
build_tree_mask_kernel(const int32_t* __restrict__ parents, const ReqInfo* __restrict__ reqs, int single_n,
                       uint32_t* __restrict__ bits, int32_t* __restrict__ depths, int W, int32_t* status) {
  extern __shared__ __align__(16) uint8_t mask_smem[];
  trigger_dependents();   // the attention kernel may start streaming K/V now; it waits for us before it reads the mask
  int node0 = 0, n = single_n;
  if (reqs != nullptr) {
    node0 = reqs[blockIdx.x].node0;
    n = reqs[blockIdx.x].n_nodes;
  }
  if (n <= 0) return;
  const int W4 = W >> 2;
  uint4* rows = reinterpret_cast<uint4*>(mask_smem);                       // [n][W4]
  int* s_anc = reinterpret_cast<int*>(mask_smem + size_t(n) * W * 4);      // [n]
  int* s_dist = s_anc + n;                                                 // [n]
  const int tid = threadIdx.x, nthr = blockDim.x;
  bool bad = false;

  for (int i = tid; i < n; i += nthr) {
    int parent = parents[node0 + i];
    if (parent < -1 || parent >= i) {
      parent = -1;
      bad = true;
    }
    s_anc[i] = parent;
    s_dist[i] = parent >= 0 ? 1 : 0;
  }
  for (int idx = tid; idx < n * W4; idx += nthr) {
    const int i = idx / W4, w4 = idx - i * W4;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if ((i >> 7) == w4) {
      const uint32_t bit = 1u << (i & 31);
      const int k = (i >> 5) & 3;
      if (k == 0) v.x = bit; else if (k == 1) v.y = bit; else if (k == 2) v.z = bit; else v.w = bit;
    }
    rows[idx] = v;
  }
  __syncthreads();

  // blockDim.x >= n (the launcher sizes the block from the largest tree): one node per thread.
  for (int round = 0; round < 11; ++round) {     // 2^10 >= DYSPEC_MAX_NODES
    int a = -1, next = -1, add = 0;
    if (tid < n) {
      a = s_anc[tid];
      if (a >= 0) { next = s_anc[a]; add = s_dist[a]; }
    }
    if (!__syncthreads_or(a >= 0)) break;        // all pointers of this round are read before any moves
    for (int idx = tid; idx < n * W4; idx += nthr) {
      const int i = idx / W4, w4 = idx - i * W4;
      const int ai = s_anc[i];                   // still this round's pointer: rewritten after the next barrier
      if (ai >= 0) {
        const uint4 x = rows[idx], y = rows[ai * W4 + w4];
        rows[idx] = make_uint4(x.x | y.x, x.y | y.y, x.z | y.z, x.w | y.w);
      }
    }
    __syncthreads();
    if (a >= 0) {
      s_anc[tid] = next;
      s_dist[tid] += add;
    }
    __syncthreads();
  }

  // Launched with programmatic dependent launch: everything above only read `parents` and worked in
  // shared memory, so it may overlap the tail of the kernel before it in the stream.  The outputs may
  // still be in use by that kernel (the mask of the previous call): wait for it before writing.
  grid_dependency_wait();
  if (bad && status) atomicCAS(status, 0, DYSPEC_ERR_BAD_TREE);
  for (int i = tid; i < n; i += nthr)
    if (depths) depths[node0 + i] = s_dist[i];
  uint4* out = reinterpret_cast<uint4*>(bits) + size_t(node0) * W4;
  for (int idx = tid; idx < n * W4; idx += nthr) out[idx] = rows[idx];
}

cudaError_t launch_build_tree_mask(const int32_t* parents, const ReqInfo* reqs, int n_req, int single_n, int max_n,
                                   uint32_t* bits, int32_t* depths, int W, int32_t* status, cudaStream_t stream) {
  if (n_req <= 0 || max_n <= 0) return cudaSuccess;
  const size_t smem = size_t(max_n) * W * 4 + size_t(max_n) * 8;
  static size_t attr_smem = 48 * 1024;
  if (smem > attr_smem) {
    cudaError_t e = cudaFuncSetAttribute(build_tree_mask_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    attr_smem = smem;
  }
  int threads = ((max_n + 31) / 32) * 32;
  if (threads < 256) threads = 256;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(n_req));
  cfg.blockDim = dim3(unsigned(threads));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, build_tree_mask_kernel, parents, reqs, single_n, bits, depths, W, status);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dyspec
