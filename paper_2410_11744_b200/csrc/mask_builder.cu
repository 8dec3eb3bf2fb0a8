// Parent array -> packed ancestor bitmasks and depths (Sec. 2, the mask(A) equation, plus the self bit).
//
// One CTA per request, one thread per node.  Depths come from pointer jumping (log2(n) rounds on
// (ancestor, distance) pairs in shared memory); rows are then filled level by level with the
// recurrence  row[i] = row[parent[i]] | (1 << i),  a level being complete before the next one reads
// it.  A parent index outside {-1} U [0, i) makes that node a root and reports DYSPEC_ERR_BAD_TREE.
#include "common.cuh"

namespace dyspec {

__global__ void __launch_bounds__(1024, 1)
build_tree_mask_kernel(const int32_t* __restrict__ parents, const ReqInfo* __restrict__ reqs, int single_n,
                       uint32_t* __restrict__ bits, int32_t* __restrict__ depths, int W, int32_t* status) {
  __shared__ int s_anc[DYSPEC_MAX_NODES];
  __shared__ int s_dist[DYSPEC_MAX_NODES];
  __shared__ int s_max_depth;

  int node0 = 0, n = single_n;
  if (reqs != nullptr) {
    node0 = reqs[blockIdx.x].node0;
    n = reqs[blockIdx.x].n_nodes;
  }
  if (n <= 0) return;
  const int i = threadIdx.x;
  const bool live = i < n;

  int parent = -1;
  if (live) {
    parent = parents[node0 + i];
    if (parent < -1 || parent >= i) {
      parent = -1;
      if (status) atomicCAS(status, 0, DYSPEC_ERR_BAD_TREE);
    }
    s_anc[i] = parent;
    s_dist[i] = parent >= 0 ? 1 : 0;
  }
  if (i == 0) s_max_depth = 0;
  __syncthreads();

  // Pointer jumping: after round k, s_anc[i] is the 2^k-th ancestor (or -1) and s_dist[i] the
  // number of links covered so far.
  for (int span = 1; span < n; span <<= 1) {
    int a = -1, add = 0, next = -1;
    if (live) {
      a = s_anc[i];
      if (a >= 0) {
        add = s_dist[a];
        next = s_anc[a];
      }
    }
    __syncthreads();
    if (live && a >= 0) {
      s_dist[i] += add;
      s_anc[i] = next;
    }
    __syncthreads();
  }
  int depth = 0;
  if (live) {
    depth = s_dist[i];
    if (depths) depths[node0 + i] = depth;
    atomicMax(&s_max_depth, depth);
  }
  __syncthreads();
  const int max_depth = s_max_depth;

  // Level-synchronous fill.  Rows are written straight to global memory; a child reads its parent's
  // finished row back through L2 (written by this same CTA one barrier earlier).
  const int W4 = W >> 2;
  uint4* rows = reinterpret_cast<uint4*>(bits) + static_cast<size_t>(node0) * W4;
  for (int level = 0; level <= max_depth; ++level) {
    if (live && depth == level) {
      const int self_word = i >> 5;
      const uint32_t self_bit = 1u << (i & 31);
      for (int w4 = 0; w4 < W4; ++w4) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (parent >= 0) v = __ldcg(rows + static_cast<size_t>(parent) * W4 + w4);
        if ((self_word >> 2) == w4) {
          const int k = self_word & 3;
          if (k == 0) v.x |= self_bit;
          else if (k == 1) v.y |= self_bit;
          else if (k == 2) v.z |= self_bit;
          else v.w |= self_bit;
        }
        __stcg(rows + static_cast<size_t>(i) * W4 + w4, v);
      }
    }
    __syncthreads();
  }
}

cudaError_t launch_build_tree_mask(const int32_t* parents, const ReqInfo* reqs, int n_req, int single_n,
                                   uint32_t* bits, int32_t* depths, int W, int32_t* status, cudaStream_t stream) {
  if (n_req <= 0) return cudaSuccess;
  build_tree_mask_kernel<<<n_req, 1024, 0, stream>>>(parents, reqs, single_n, bits, depths, W, status);
  return cudaGetLastError();
}

}  // namespace dyspec
