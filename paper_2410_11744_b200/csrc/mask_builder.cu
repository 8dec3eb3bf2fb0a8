// Parent array -> packed ancestor bitmasks and depths (Sec. 2, the mask(A) equation, plus the self bit).
//
// One CTA per (request, column chunk).  Rows live in shared memory and are completed by pointer
// jumping on bitsets: every node keeps a pointer `anc` (initially its parent) and a row that covers
// the node and all its ancestors below `anc`; one round does  row[i] |= row[anc[i]],
// dist[i] += dist[anc[i]],  anc[i] = anc[anc[i]],  which doubles the covered path, so
// ceil(log2(depth + 1)) rounds finish the tree.  OR-ing a row that another thread is extending in
// the same round is harmless: every bit a row ever holds is an ancestor-or-self of its node, hence
// an ancestor of the reader too.
// Trees of up to 1024 nodes use one chunk (all W words of a row).  Larger trees are cut into chunks
// of 16 words (512 columns) so that the rows still fit in shared memory: chunk c holds columns
// [512 c, 512 c + 512) of the rows i >= 512 c (lower rows have no bit there: ancestors have smaller
// indices) and stops following a pointer once it drops below 512 c.  Chunk 0 also writes the depths.
// Optionally the kernel emits, per node, which 64-key tiles of the tree its row touches
// (bit t of node_tiles[i] = row i has a visible key in columns [64 t, 64 t + 64)); the attention
// kernel ORs these over a query tile and skips key tiles no row of it can see (App. C).
// A parent index outside {-1} U [0, i) makes that node a root and reports DYSPEC_ERR_BAD_TREE.
#include "common.cuh"

namespace dyspec {

// The work of one CTA: request (node0, n), column chunk blockIdx.y.
__device__ __forceinline__ void build_tree_mask_body(const int32_t* __restrict__ parents, int node0, int n,
                                                     uint32_t* __restrict__ bits, int32_t* __restrict__ depths,
                                                     uint32_t* __restrict__ node_tiles, int W, int CW, int32_t* status) {
  extern __shared__ __align__(16) uint8_t mask_smem[];
  trigger_dependents();   // the attention kernel may start streaming K/V now; it waits for us before it reads the mask
  if (n <= 0) return;
  const int chunk = blockIdx.y;
  const int W4 = W >> 2, CW4 = min(CW, W - chunk * CW) >> 2;               // 16-byte groups per row: all, this chunk's
  const int col4 = chunk * (CW >> 2);                                      // first 16-byte group of the chunk
  const int row0 = min(n, chunk * CW * 32);                                // rows below have no bit in these columns
  const int nr = n - row0;
  uint4* rows = reinterpret_cast<uint4*>(mask_smem);                       // [nr][CW4]
  int* s_anc = reinterpret_cast<int*>(mask_smem + size_t(nr) * CW4 * 16);  // [n]
  int* s_dist = s_anc + n;                                                 // [n]
  uint32_t* s_occ = reinterpret_cast<uint32_t*>(s_dist + n);               // [n]
  const int tid = threadIdx.x, nthr = blockDim.x;
  bool bad = false;

  for (int i = tid; i < n; i += nthr) {
    int parent = parents[node0 + i];
    if (parent < -1 || parent >= i) {
      parent = -1;
      bad = true;
    }
    s_anc[i] = parent >= row0 ? parent : -1;        // chunk 0: row0 = 0, the plain parent
    s_dist[i] = parent >= 0 ? 1 : 0;
    s_occ[i] = 0u;
  }
  for (int idx = tid; idx < nr * CW4; idx += nthr) {
    const int r = idx / CW4, w4 = idx - r * CW4;
    const int i = row0 + r;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if ((i >> 7) == col4 + w4) {
      const uint32_t bit = 1u << (i & 31);
      const int k = (i >> 5) & 3;
      if (k == 0) v.x = bit; else if (k == 1) v.y = bit; else if (k == 2) v.z = bit; else v.w = bit;
    }
    rows[idx] = v;
  }
  __syncthreads();

  // Up to two nodes per thread (n <= 2048, 1024 threads when n > 1024).
  for (int round = 0; round < 12; ++round) {     // 2^11 >= DYSPEC_MAX_NODES
    int a[2] = {-1, -1}, next[2] = {-1, -1}, add[2] = {0, 0};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int i = tid + k * nthr;
      if (i < n) {
        a[k] = s_anc[i];
        if (a[k] >= 0) { next[k] = s_anc[a[k]]; add[k] = s_dist[a[k]]; }
      }
    }
    if (!__syncthreads_or(a[0] >= 0 || a[1] >= 0)) break;   // all pointers of this round are read before any moves
    for (int idx = tid; idx < nr * CW4; idx += nthr) {
      const int r = idx / CW4, w4 = idx - r * CW4;
      const int ai = s_anc[row0 + r];            // still this round's pointer: rewritten after the next barrier
      if (ai >= 0) {
        const uint4 x = rows[idx], y = rows[(ai - row0) * CW4 + w4];
        rows[idx] = make_uint4(x.x | y.x, x.y | y.y, x.z | y.z, x.w | y.w);
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int i = tid + k * nthr;
      if (i < n && a[k] >= 0) {
        s_anc[i] = next[k];
        s_dist[i] += add[k];
      }
    }
    __syncthreads();
  }

  // Launched with programmatic dependent launch: everything above only read `parents` and worked in
  // shared memory, so it may overlap the tail of the kernel before it in the stream.  The outputs may
  // still be in use by that kernel (the mask of the previous call): wait for it before writing.
  grid_dependency_wait();
  if (bad && status) atomicCAS(status, 0, DYSPEC_ERR_BAD_TREE);
  if (chunk == 0 && depths)
    for (int i = tid; i < n; i += nthr) depths[node0 + i] = s_dist[i];
  uint4* out = reinterpret_cast<uint4*>(bits) + size_t(node0) * W4 + col4;
  for (int idx = tid; idx < row0 * CW4; idx += nthr) {           // rows above the chunk: all zero here
    const int r = idx / CW4, w4 = idx - r * CW4;
    out[size_t(r) * W4 + w4] = make_uint4(0u, 0u, 0u, 0u);
  }
  for (int idx = tid; idx < nr * CW4; idx += nthr) {
    const int r = idx / CW4, w4 = idx - r * CW4;
    const uint4 x = rows[idx];
    out[size_t(row0 + r) * W4 + w4] = x;
    if (node_tiles) {
      const uint32_t t = ((x.x | x.y) ? 1u : 0u) | ((x.z | x.w) ? 2u : 0u);
      if (t) atomicOr(&s_occ[row0 + r], t << (2 * (col4 + w4)));
    }
  }
  if (node_tiles) {
    __syncthreads();
    if (gridDim.y == 1) {
      for (int i = tid; i < n; i += nthr) node_tiles[node0 + i] = s_occ[i];
    } else {
      // a chunk of 16 words is 8 tiles: byte `chunk` of the node's word; the last chunk clears the bytes above it
      uint8_t* o8 = reinterpret_cast<uint8_t*>(node_tiles + node0);
      for (int i = tid; i < n; i += nthr) {
        o8[4 * i + chunk] = uint8_t(s_occ[i] >> (8 * chunk));
        if (chunk == int(gridDim.y) - 1)
          for (int b = chunk + 1; b < 4; ++b) o8[4 * i + b] = 0;
      }
    }
  }
}

// Request list in a plan's device table (or one request given by its size).
__global__ void __launch_bounds__(1024, 1)
build_tree_mask_kernel(const int32_t* __restrict__ parents, const ReqInfo* __restrict__ reqs, int single_n,
                       uint32_t* __restrict__ bits, int32_t* __restrict__ depths, uint32_t* __restrict__ node_tiles,
                       int W, int CW, int32_t* status) {
  int node0 = 0, n = single_n;
  if (reqs != nullptr) {
    node0 = reqs[blockIdx.x].node0;
    n = reqs[blockIdx.x].n_nodes;
  }
  build_tree_mask_body(parents, node0, n, bits, depths, node_tiles, W, CW, status);
}

// Request list passed by value (kernel parameter space): a ragged batch without a plan, one launch for
// up to kMaskBatchMax requests, one status word per request.
__global__ void __launch_bounds__(1024, 1)
build_tree_mask_batch_kernel(const int32_t* __restrict__ parents, const __grid_constant__ MaskBatch batch,
                             uint32_t* __restrict__ bits, int32_t* __restrict__ depths, int W, int CW, int32_t* status) {
  const int node0 = batch.node0[blockIdx.x], n = batch.node0[blockIdx.x + 1] - node0;
  build_tree_mask_body(parents, node0, n, bits, depths, nullptr, W, CW, status ? status + batch.first_req + blockIdx.x : nullptr);
}

namespace {
struct MaskLaunch { int CW, n_chunks, threads; size_t smem; };
MaskLaunch mask_launch_shape(int max_n, int W) {
  MaskLaunch m;
  m.CW = W <= 32 ? W : 16;                 // words per column chunk
  m.n_chunks = (W + m.CW - 1) / m.CW;
  m.smem = size_t(max_n) * m.CW * 4 + size_t(max_n) * 12;
  m.threads = ((max_n + 31) / 32) * 32;
  if (m.threads < 256) m.threads = 256;
  if (m.threads > 1024) m.threads = 1024;
  return m;
}
}  // namespace

cudaError_t launch_build_tree_mask_batch(const int32_t* parents, const MaskBatch& batch, int n_req, int max_n, uint32_t* bits,
                                         int32_t* depths, int W, int32_t* status, cudaStream_t stream) {
  if (n_req <= 0 || max_n <= 0) return cudaSuccess;
  const MaskLaunch m = mask_launch_shape(max_n, W);
  static DynSmemGrant grant;
  if (cudaError_t e = grant.ensure(build_tree_mask_batch_kernel, m.smem); e != cudaSuccess) return e;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(n_req), unsigned(m.n_chunks));
  cfg.blockDim = dim3(unsigned(m.threads));
  cfg.dynamicSmemBytes = m.smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, build_tree_mask_batch_kernel, parents, batch, bits, depths, W, m.CW, status);
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_build_tree_mask(const int32_t* parents, const ReqInfo* reqs, int n_req, int single_n, int max_n,
                                   uint32_t* bits, int32_t* depths, uint32_t* node_tiles, int W, int32_t* status,
                                   cudaStream_t stream) {
  if (n_req <= 0 || max_n <= 0) return cudaSuccess;
  const MaskLaunch ml = mask_launch_shape(max_n, W);
  const int CW = ml.CW, n_chunks = ml.n_chunks, threads = ml.threads;
  const size_t smem = ml.smem;
  static DynSmemGrant grant;
  if (cudaError_t e = grant.ensure(build_tree_mask_kernel, smem); e != cudaSuccess) return e;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(n_req), unsigned(n_chunks));
  cfg.blockDim = dim3(unsigned(threads));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, build_tree_mask_kernel, parents, reqs, single_n, bits, depths, node_tiles, W,
                                     CW, status);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dyspec
