// Keeping the accepted path in the KV cache after verification: for each request, the tree rows of the
// accepted nodes a_0 < a_1 < ... move to the rows right after the prefix (row L + i <- row L + a_i), in
// place, for K and V, and the prefix length grows by their number.  With keep_root the walk's start node
// (tree row 0: the last decoded token, whose K/V this step computed) is kept in front of them: it is in
// place already, the accepted nodes follow it (row L + 1 + i <- row L + a_i).
//
// a_i >= i (>= i + 1 with keep_root: the accepted nodes are proper descendants of node 0), so a
// destination never lies behind its own source, but it can be an EARLIER step's
// source (path 1, 2, 3: slot 1 receives node 2 after it has given node 1 away).  A thread owns fixed
// 16-byte columns of a row and walks the steps in order, so for any byte the read of step i precedes
// the write of step i + 1 in program order, and no two threads ever touch the same byte: no barriers.
// grid = (requests, column chunks, 2 for K / V); the copy is a few hundred KB at most, i.e. bound by
// launch latency.
#include "common.cuh"

namespace dyspec {

__global__ void __launch_bounds__(256)
compact_kv_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache, const int64_t* __restrict__ kv_row_offset,
                  const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ accepted_nodes,
                  const int32_t* __restrict__ n_accepted, int max_out, int row_vecs, int keep_root,
                  int32_t* __restrict__ new_prefix_len) {
  const int r = blockIdx.x;
  uint4* cache = blockIdx.z == 0 ? k_cache : v_cache;
  const int L = prefix_len[r];
  const int64_t base = (kv_row_offset[r] + L) * int64_t(row_vecs);
  const int n = min(n_accepted[r], max_out);
  const int32_t* acc = accepted_nodes + size_t(r) * max_out;
  const int col = blockIdx.y * blockDim.x + threadIdx.x;
  int kept = (keep_root && n > 0) ? 1 : 0;          // the root's row is where it belongs already
  for (int i = 0; i < n; ++i) {
    const int a = acc[i];
    if (a < 0 || a >= DYSPEC_MAX_NODES) continue;   // an emitted token without a tree node (or not a node index at all)
    if (col < row_vecs && a != kept) cache[base + int64_t(kept) * row_vecs + col] = cache[base + int64_t(a) * row_vecs + col];
    ++kept;
  }
  if (new_prefix_len && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) new_prefix_len[r] = L + kept;
}

// Paged cache: the accepted nodes' rows leave the request's tree rows (tree_row_offset[r] + a_i) for the
// pages of the prefix: token L + i lies in page (L + i) / page_size of the request, at row (L + i) %
// page_size of it.  With the tree rows outside the prefix pages source and destination never overlap.
// With tree_row_offset == nullptr the tree rows are tokens L .. of the paged sequence themselves (node a
// = token L + a): an in-place move again, safe for the reason given above (a thread walks the steps in
// order over its own columns; the accepted nodes increase along their path).
__global__ void __launch_bounds__(256)
compact_kv_paged_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache, const int64_t* __restrict__ tree_row_offset,
                        const int32_t* __restrict__ page_table, int pages_per_req, int page_shift,
                        const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ accepted_nodes,
                        const int32_t* __restrict__ n_accepted, int max_out, int row_vecs, int keep_root,
                        int32_t* __restrict__ new_prefix_len, int32_t* __restrict__ status) {
  const int r = blockIdx.x;
  uint4* cache = blockIdx.z == 0 ? k_cache : v_cache;
  const int L = prefix_len[r];
  const bool in_pages = tree_row_offset == nullptr;
  const int64_t src0 = in_pages ? 0 : tree_row_offset[r];
  const int n = min(n_accepted[r], max_out);
  const int32_t* acc = accepted_nodes + size_t(r) * max_out;
  const int32_t* pages = page_table + size_t(r) * pages_per_req;
  const int col = blockIdx.y * blockDim.x + threadIdx.x;
  int kept = 0;
  const int first = (keep_root && n > 0) ? -1 : 0;  // step -1 moves the root's row (tree row 0) to token L
  for (int i = first; i < n; ++i) {
    const int a = i < 0 ? 0 : acc[i];
    if (a < 0 || a >= DYSPEC_MAX_NODES) continue;   // an emitted token without a tree node (or not a node index at all)
    const int t = L + kept;
    const int pi = t >> page_shift;
    const int page = pi < pages_per_req ? pages[pi] : -1;
    if (page < 0) {                            // no page for this token: report it, keep what fits
      if (status && col == 0 && blockIdx.z == 0) atomicCAS(status, 0, DYSPEC_ERR_INVALID_ARG);
      break;
    }
    int64_t src = src0 + a;
    if (in_pages) {
      const int ts = L + a, ps = ts >> page_shift;
      const int spage = ps < pages_per_req ? pages[ps] : -1;
      if (spage < 0) {                         // the node's row has no page: nothing to move from
        if (status && col == 0 && blockIdx.z == 0) atomicCAS(status, 0, DYSPEC_ERR_INVALID_ARG);
        break;
      }
      src = (int64_t(spage) << page_shift) + (ts & ((1 << page_shift) - 1));
    }
    if (col < row_vecs) {
      const int64_t dst = (int64_t(page) << page_shift) + (t & ((1 << page_shift) - 1));
      if (dst != src) cache[dst * row_vecs + col] = cache[src * int64_t(row_vecs) + col];
    }
    ++kept;
  }
  if (new_prefix_len && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) new_prefix_len[r] = L + kept;
}

cudaError_t launch_compact_kv_paged(void* k_cache, void* v_cache, const int64_t* tree_row_offset, const int32_t* page_table,
                                    int pages_per_req, int page_shift, const int32_t* prefix_len,
                                    const int32_t* accepted_nodes, const int32_t* n_accepted, int n_req, int max_out,
                                    int row_bytes, int keep_root, int32_t* new_prefix_len, int32_t* status,
                                    cudaStream_t stream) {
  if (n_req <= 0) return cudaSuccess;
  const int row_vecs = row_bytes / 16;
  const dim3 grid(unsigned(n_req), unsigned((row_vecs + 255) / 256), 2u);
  compact_kv_paged_kernel<<<grid, 256, 0, stream>>>(static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache),
                                                    tree_row_offset, page_table, pages_per_req, page_shift, prefix_len,
                                                    accepted_nodes, n_accepted, max_out, row_vecs, keep_root, new_prefix_len, status);
  return cudaGetLastError();
}

cudaError_t launch_compact_kv(void* k_cache, void* v_cache, const int64_t* kv_row_offset, const int32_t* prefix_len,
                              const int32_t* accepted_nodes, const int32_t* n_accepted, int n_req, int max_out,
                              int row_bytes, int keep_root, int32_t* new_prefix_len, cudaStream_t stream) {
  if (n_req <= 0) return cudaSuccess;
  const int row_vecs = row_bytes / 16;
  const dim3 grid(unsigned(n_req), unsigned((row_vecs + 255) / 256), 2u);
  compact_kv_kernel<<<grid, 256, 0, stream>>>(static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), kv_row_offset,
                                              prefix_len, accepted_nodes, n_accepted, max_out, row_vecs, keep_root, new_prefix_len);
  return cudaGetLastError();
}

}  // namespace dyspec
