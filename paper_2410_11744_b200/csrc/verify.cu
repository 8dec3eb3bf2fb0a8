// Verification of a draft token tree against the target model (Algorithm 3: multi-branch rejection
// sampling along the tree), on the device, so that the step after the tree attention needs no host
// round trip.
//
// One CTA of 1024 threads per request walks the tree from node 0.  As long as the FIRST branch of the
// current node is accepted the walk needs two numbers per node, Target(node, y) and Draft(node, y), not the
// rows: one warp does it alone (first child by ballots over the parent array in shared memory, two scalar
// loads, the test), about a microsecond per node, while the other warps wait at a block barrier.  Only at
// a first rejection -- or where a token has to be drawn -- the whole block takes the node over, from
// its first branch again (the test is repeated with the same numbers, so the decision is the same):
// it loads the target row
// into registers (the residual R; thread t owns the float4 chunks t, t + 1024, ... of the vocabulary)
// and the draft row D into shared memory in the same interleaved order (coalesced global loads,
// conflict-free shared accesses).  Both carry a scalar scale instead of being renormalised in place:
//   reject y:  R <- max(R sR - D sD, 0), sR <- 1 / sum(R);  D[y] <- 0, sD <- sD / (1 - D[y] sD)
// so a rejection costs one pass over the registers plus one block reduction.  "D is all zero" is an
// exact test on the count of non-zero draft entries.  The final token is drawn from R by inverse CDF in
// token order: row totals (4096 tokens per row) by one block reduction, then one block scan inside
// the row that holds the crossing.  The random numbers are inputs (one acceptance number per node, one
// sampling number per node), so the caller's generator decides reproducibility.
//
// The branches of a node are its children in increasing index; they are gathered per visited node with
// warp ballots (no precomputed child lists).
#include "vocab_ops.cuh"

namespace dyspec {

__global__ void __launch_bounds__(kVThreads, 1)
verify_tree_kernel(const int32_t* __restrict__ parents, const int32_t* __restrict__ tokens,
                   const float* __restrict__ draft_probs, const float* __restrict__ target_probs,
                   const float* __restrict__ accept_u, const float* __restrict__ sample_u,
                   const int32_t* __restrict__ node_offsets, int max_nodes, int vocab, int bonus_at_leaf,
                   int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_nodes, int32_t* __restrict__ out_count,
                   int max_out, int32_t* status) {
  extern __shared__ __align__(16) uint8_t vsm[];
  float4* s_d = reinterpret_cast<float4*>(vsm);                                   // draft row, [chunk][thread]
  int32_t* s_par = reinterpret_cast<int32_t*>(vsm + size_t(kMaxChunks) * kVThreads * 16);   // [n] parents of the request
  int32_t* s_tok = s_par + max_nodes;                                             // [n] tokens of the nodes
  float* s_acc = reinterpret_cast<float*>(s_tok + max_nodes);                     // [n] acceptance numbers
  __shared__ int s_walk[3];                                                       // fast path -> block: node, tokens emitted, what next
  // small scalars
  __shared__ VocabScratch s_vs;
  __shared__ int s_cnt[64];
  __shared__ int s_nchild;
  __shared__ float s_ry, s_dy;
  __shared__ int16_t s_child[2048];

  const int r = blockIdx.x;
  const int node0 = node_offsets[r], n = node_offsets[r + 1] - node0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_vec = vocab >> 2;                                  // float4 chunks in a row
  const int n_chunks = (n_vec + kVThreads - 1) / kVThreads;      // per thread, <= kMaxChunks
  int n_out = 0;
  if (n <= 0 || n > max_nodes) {            // max_nodes sized the shared arrays: a larger request is refused
    if (tid == 0) {
      out_count[r] = 0;
      if (n > max_nodes && status) atomicCAS(status, 0, DYSPEC_ERR_INVALID_ARG);
    }
    return;
  }
  bool bad = false;
  for (int i = tid; i < n; i += kVThreads) {
    int p_ = parents[node0 + i];
    if (p_ < -1 || p_ >= i) { p_ = -1; bad = true; }
    s_par[i] = p_;
    s_tok[i] = tokens[node0 + i];
    s_acc[i] = accept_u[node0 + i];
  }
  if (bad && status) atomicCAS(status, 0, DYSPEC_ERR_BAD_TREE);
  __syncthreads();

  int cur = 0;
  for (int step = 0; step <= n; ++step) {                        // at most n moves; bounded in any case
    // ---- fast path: warp 0 follows first branches for as long as they are accepted
    if (warp == 0) {
      int what = 0;                                              // 1: the block must take over at `cur`; 2: a leaf
      for (int hop = 0; hop <= n; ++hop) {
        int first = 0x7fffffff;
        for (int c0 = 0; c0 < n && first == 0x7fffffff; c0 += 32) {
          const int i = c0 + lane;
          const uint32_t m = __ballot_sync(0xffffffffu, i > 0 && i < n && s_par[i] == cur);
          if (m) first = c0 + __ffs(m) - 1;
        }
        if (first == 0x7fffffff) { what = 2; break; }
        const int y = s_tok[first];
        if (y < 0 || y >= vocab) { what = 1; break; }            // not a token: the block path reports it
        float ry = 0.f, dy = 0.f;
        if (lane == 0) ry = __ldg(target_probs + size_t(node0 + cur) * vocab + y);
        if (lane == 1) dy = __ldg(draft_probs + size_t(node0 + cur) * vocab + y);
        ry = __shfl_sync(0xffffffffu, ry, 0);
        dy = __shfl_sync(0xffffffffu, dy, 1);
        const float ratio = dy > 0.f ? ry / dy : (ry > 0.f ? INFINITY : 0.f);
        if (!(s_acc[first] <= ratio)) { what = 1; break; }
        if (lane == 0 && n_out < max_out) { out_tokens[size_t(r) * max_out + n_out] = y; out_nodes[size_t(r) * max_out + n_out] = first; }
        ++n_out;
        cur = first;
      }
      if (lane == 0) { s_walk[0] = cur; s_walk[1] = n_out; s_walk[2] = what; }
    }
    __syncthreads();
    cur = s_walk[0];
    n_out = s_walk[1];
    if (s_walk[2] == 2 && !bonus_at_leaf) break;                 // as printed: the loop runs while there are branches
    // ---- the block takes the node over: branches of `cur`, in index order
    if (tid < 64) s_cnt[tid] = 0;
    __syncthreads();
    for (int c0 = warp * 32; c0 < n; c0 += kVThreads) {          // chunk of 32 nodes per warp per round
      const int i = c0 + lane;
      const bool is = i > 0 && i < n && s_par[i] == cur;
      const uint32_t m = __ballot_sync(0xffffffffu, is);
      if (lane == 0) s_cnt[c0 >> 5] = __popc(m);
    }
    __syncthreads();
    if (warp == 0) {                                             // exclusive scan of the <= 64 chunk counts
      const int a = s_cnt[lane], b = s_cnt[lane + 32];
      int xa = a, xb = b;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int ta = __shfl_up_sync(0xffffffffu, xa, o), tb = __shfl_up_sync(0xffffffffu, xb, o);
        if (lane >= o) { xa += ta; xb += tb; }
      }
      const int tot_a = __shfl_sync(0xffffffffu, xa, 31);
      s_cnt[lane] = xa - a;
      s_cnt[lane + 32] = tot_a + xb - b;
      if (lane == 31) s_nchild = tot_a + xb;
    }
    __syncthreads();
    for (int c0 = warp * 32; c0 < n; c0 += kVThreads) {
      const int i = c0 + lane;
      const bool is = i > 0 && i < n && s_par[i] == cur;
      const uint32_t m = __ballot_sync(0xffffffffu, is);
      if (is) s_child[s_cnt[c0 >> 5] + __popc(m & ((1u << lane) - 1u))] = int16_t(i);
    }
    __syncthreads();
    const int n_child = s_nchild;
    if (n_child == 0 && !bonus_at_leaf) break;                   // as printed: the loop runs while there are branches

    // ---- R <- Target(cur, .) in registers, D <- Draft(cur, .) in shared memory
    float4 R[kMaxChunks];
    const float4* t_row = reinterpret_cast<const float4*>(target_probs + size_t(node0 + cur) * vocab);
    const float4* d_row = reinterpret_cast<const float4*>(draft_probs + size_t(node0 + cur) * vocab);
    float nnz_f = 0.f;
#pragma unroll
    for (int k = 0; k < kMaxChunks; ++k) {
      const int v4 = k * kVThreads + tid;
      R[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      float4 d = make_float4(0.f, 0.f, 0.f, 0.f);
      if (k < n_chunks && v4 < n_vec) {
        R[k] = __ldg(t_row + v4);
        if (n_child > 0) {
          d = __ldg(d_row + v4);
          nnz_f += (d.x > 0.f) + (d.y > 0.f) + (d.z > 0.f) + (d.w > 0.f);
        }
      }
      if (n_child > 0) s_d[k * kVThreads + tid] = d;          // the ragged tail of the last chunk must read as zero
    }
    float sR = 1.f, sD = 1.f;
    int nnz = n_child > 0 ? int(block_sum(nnz_f, s_vs) + 0.5f) : 0;
    bool moved = false;
    for (int b = 0; b < n_child; ++b) {
      const int child = s_child[b];
      int y = s_tok[child];
      if (y < 0 || y >= vocab) {                                 // not a token: report it, carry on with a legal index
        if (tid == 0 && status) atomicCAS(status, 0, DYSPEC_ERR_INVALID_ARG);
        y = min(max(y, 0), vocab - 1);
      }
      const float c = s_acc[child];
      // the owner of token y publishes R[y] and D[y]
      const int y4 = y >> 2, yk = y4 / kVThreads, yt = y4 - yk * kVThreads, ye = y & 3;
      if (tid == yt) {
        float4 rv = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < kMaxChunks; ++k)
          if (k == yk) rv = R[k];
        const float4 dv = s_d[yk * kVThreads + yt];
        s_ry = (ye == 0 ? rv.x : ye == 1 ? rv.y : ye == 2 ? rv.z : rv.w) * sR;
        s_dy = (ye == 0 ? dv.x : ye == 1 ? dv.y : ye == 2 ? dv.z : dv.w) * sD;
      }
      __syncthreads();
      const float ry = s_ry, dy = s_dy;
      const float ratio = dy > 0.f ? ry / dy : (ry > 0.f ? INFINITY : 0.f);
      if (c <= ratio) {
        if (tid == 0 && n_out < max_out) { out_tokens[size_t(r) * max_out + n_out] = y; out_nodes[size_t(r) * max_out + n_out] = child; }
        ++n_out;
        cur = child;
        moved = true;
        break;
      }
      // ---- rejected: R <- norm(max(R - D, 0)); D[y] <- 0; stop if D is all zero; D <- norm(D)
      float part = 0.f;
#pragma unroll
      for (int k = 0; k < kMaxChunks; ++k) {
        if (k < n_chunks) {
          const float4 d = s_d[k * kVThreads + tid];
          R[k].x = fmaxf(R[k].x * sR - d.x * sD, 0.f);
          R[k].y = fmaxf(R[k].y * sR - d.y * sD, 0.f);
          R[k].z = fmaxf(R[k].z * sR - d.z * sD, 0.f);
          R[k].w = fmaxf(R[k].w * sR - d.w * sD, 0.f);
          part += (R[k].x + R[k].y) + (R[k].z + R[k].w);
        }
      }
      const float tot = block_sum(part, s_vs);                  // (its barriers also order the reads of s_d above)
      sR = tot > 0.f ? 1.f / tot : 1.f;
      if (tid == yt) {
        float* dv = reinterpret_cast<float*>(&s_d[yk * kVThreads + yt]);
        dv[ye] = 0.f;
      }
      if (dy > 0.f) --nnz;
      if (nnz <= 0) break;
      sD = sD / (1.f - dy);
      __syncthreads();
    }
    if (moved) continue;

    // ---- no branch accepted (or a leaf with the bonus token): draw the token from R by inverse CDF
    {
      float part = 0.f;
#pragma unroll
      for (int k = 0; k < kMaxChunks; ++k) part += (R[k].x + R[k].y) + (R[k].z + R[k].w);
      const float left = block_sum(part, s_vs);
      if (!(left > 0.f)) load_row(R, target_probs + size_t(node0 + cur) * vocab, vocab);    // nothing left: fall back to Target
      double total;
      const int y = sample_inverse_cdf(R, vocab, sample_u[node0 + cur], total, s_vs);
      if (tid == 0 && n_out < max_out) { out_tokens[size_t(r) * max_out + n_out] = y; out_nodes[size_t(r) * max_out + n_out] = -1; }
      ++n_out;
    }
    break;
  }
  if (tid == 0) out_count[r] = min(n_out, max_out);
}

cudaError_t launch_verify_tree(const int32_t* parents, const int32_t* tokens, const float* draft_probs,
                               const float* target_probs, const float* accept_u, const float* sample_u,
                               const int32_t* node_offsets, int n_req, int max_nodes, int vocab, int bonus_at_leaf,
                               int32_t* out_tokens, int32_t* out_nodes, int32_t* out_count, int max_out, int32_t* status,
                               cudaStream_t stream) {
  if (n_req <= 0) return cudaSuccess;
  const size_t smem = size_t(kMaxChunks) * kVThreads * 16 + size_t(max_nodes) * 12;
  static DynSmemGrant grant;
  if (cudaError_t e = grant.ensure(verify_tree_kernel, smem); e != cudaSuccess) return e;
  verify_tree_kernel<<<n_req, kVThreads, smem, stream>>>(parents, tokens, draft_probs, target_probs, accept_u, sample_u,
                                                         node_offsets, max_nodes, vocab, bonus_at_leaf, out_tokens, out_nodes,
                                                         out_count, max_out, status);
  return cudaGetLastError();
}

}  // namespace dyspec
