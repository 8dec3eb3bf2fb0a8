// Construction of the draft token tree on the device (Sec. 4.1-4.3, Algorithm 1; App. B, Algorithm 2).
//
// The draft model is a table lookup: the distribution that follows a tree position is row
// f(row of the parent, token) of `draft_table`, and the uniform number of the j-th sampling at a
// position is entry g(row, j) of `uniforms` (vocab_ops.cuh).  One CTA of 1024 threads per request.
//
// A "slot" (v, position, attempt) is the next sampling at a position, v its estimated acceptance rate.
//   greedy (Algorithm 1):   take the slot with the largest v (ties: pushed first), draw a token from
//     the position's residual distribution (the row with the tokens of the position's existing
//     children zeroed, renormalised), create the node, push (v (1 - r), position, attempt + 1) and
//     (v r, new node, 0), r = the drawn token's residual probability; m times.  The heap of the paper
//     is an array scanned by the whole block (<= 4096 slots: one pass).
//   threshold (Algorithm 2): layer by layer, each position keeps drawing while v >= t.
// The residual lives in registers (thread t owns float4 chunks t, t + 1024, ...); a draw is an
// inverse-CDF search in token order (row totals, then one block scan).  The tokens a position has
// already used are struck out in constant time whatever their number: every thread looks at one or two
// nodes of the tree, and where a node is a child of the position it sets the token's bit in the word of
// the thread that owns the token (32 tokens per thread, one shared-memory word each); after a barrier a
// thread zeroes what its word marks.  (Walking the position's child list instead costs a dependent
// shared-memory hop per earlier sibling in all 32 warps: quadratic in the width of a position, and
// language-model rows give the root hundreds of children.)
#include "vocab_ops.cuh"

namespace dyspec {

namespace {

struct TreeOut {
  int32_t* parents;
  int32_t* tokens;
  float* values;
  float* child_values;
  int32_t* rows;
};

__device__ __forceinline__ void write_node(const TreeOut& o, size_t base, int k, int parent, int token, float v, float cv,
                                           int row) {
  o.parents[base + k] = parent;
  o.tokens[base + k] = token;
  o.values[base + k] = v;
  o.child_values[base + k] = cv;
  o.rows[base + k] = row;
}

}  // namespace

__global__ void __launch_bounds__(kVThreads, 1)
build_tree_greedy_kernel(const float* __restrict__ draft_table, int n_rows, int vocab, const float* __restrict__ uniforms,
                         int n_uniforms, const int32_t* __restrict__ root_row, int m, TreeOut out,
                         int32_t* __restrict__ n_nodes_out) {
  extern __shared__ __align__(16) uint8_t csm[];
  // slots: value, position, attempt; per node: row id, token, the position it was drawn at
  const int max_slots = 2 * m + 2;
  double* s_v = reinterpret_cast<double*>(csm);                     // [max_slots]   (-1 = taken); fp64 like the draws
  int16_t* s_pos = reinterpret_cast<int16_t*>(s_v + max_slots);     // [max_slots]
  int16_t* s_att = s_pos + max_slots;                               // [max_slots]
  int32_t* s_row = reinterpret_cast<int32_t*>(s_att + max_slots + (max_slots & 1));   // [m + 1]
  int32_t* s_tok = s_row + (m + 1);                                 // [m + 1]
  int16_t* s_ppos = reinterpret_cast<int16_t*>(s_tok + (m + 1));    // [m + 1] the position (parent) a node was drawn at
  __shared__ uint32_t s_kill[kVThreads];                            // bit 4 k + e of word t: element e of thread t's chunk k is used up
  __shared__ VocabScratch s_vs;
  __shared__ double s_bv[33];
  __shared__ int s_bi[33];

  const int r = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t base = size_t(r) * (m + 1);
  if (tid == 0) {
    s_row[0] = ((root_row[r] % n_rows) + n_rows) % n_rows;        // non-negative remainder: any int32 maps to a row
    s_tok[0] = 0;
    s_ppos[0] = -1;
    s_v[0] = 1.0; s_pos[0] = 0; s_att[0] = 0;
    write_node(out, base, 0, -1, 0, 1.f, 1.f, s_row[0]);
  }
  __syncthreads();
  int n_slots = 1, n_created = 0;

  for (int step = 0; step < m; ++step) {
    // ---- the slot with the largest value (ties: lowest index = pushed first)
    double bv = -1.0;
    int bi = 0x7fffffff;
    for (int i = tid; i < n_slots; i += kVThreads) {
      const double v_ = s_v[i];
      if (v_ > bv) { bv = v_; bi = i; }                          // i increases: the first of equal values is kept
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double tv = __shfl_xor_sync(0xffffffffu, bv, o);
      const int ti = __shfl_xor_sync(0xffffffffu, bi, o);
      if (tv > bv || (tv == bv && ti < bi)) { bv = tv; bi = ti; }
    }
    __syncthreads();
    if (lane == 0) { s_bv[warp] = bv; s_bi[warp] = bi; }
    __syncthreads();
    if (warp == 0) {
      double v_ = s_bv[lane];
      int i_ = s_bi[lane];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double tv = __shfl_xor_sync(0xffffffffu, v_, o);
        const int ti = __shfl_xor_sync(0xffffffffu, i_, o);
        if (tv > v_ || (tv == v_ && ti < i_)) { v_ = tv; i_ = ti; }
      }
      if (lane == 0) { s_bv[32] = v_; s_bi[32] = i_; }
    }
    __syncthreads();
    if (s_bv[32] < 0.0) break;                                   // no live slot (cannot happen before m nodes exist)
    const int slot = s_bi[32];
    const double v = s_v[slot];
    const int pos = s_pos[slot], attempt = s_att[slot];
    const int prow = s_row[pos];
    __syncthreads();
    if (tid == 0) s_v[slot] = -1.0;

    // ---- residual of the position: its row with the tokens of its existing children zeroed
    float4 R[kMaxChunks];
    load_row(R, draft_table + size_t(prow) * vocab, vocab);
    if (attempt > 0) {                                           // (a first sampling has nothing to strike out)
      s_kill[tid] = 0u;
      __syncthreads();
      for (int c = 1 + tid; c <= n_created; c += kVThreads)
        if (s_ppos[c] == pos) {
          const int yc = s_tok[c], y4 = yc >> 2;
          atomicOr(&s_kill[y4 % kVThreads], 1u << ((y4 / kVThreads) * 4 + (yc & 3)));
        }
      __syncthreads();
      const uint32_t kill = s_kill[tid];
      if (kill) {
#pragma unroll
        for (int k = 0; k < kMaxChunks; ++k) {
          if ((kill >> (4 * k)) & 1u) R[k].x = 0.f;
          if ((kill >> (4 * k + 1)) & 1u) R[k].y = 0.f;
          if ((kill >> (4 * k + 2)) & 1u) R[k].z = 0.f;
          if ((kill >> (4 * k + 3)) & 1u) R[k].w = 0.f;
        }
      }
    }
    double total;
    const float u = uniforms[draft_uniform_index(uint32_t(prow), uint32_t(attempt), uint32_t(n_uniforms))];
    const int y = sample_inverse_cdf(R, vocab, u, total, s_vs);
    const float py = take_element(R, y, false, s_vs);
    const double rr = total > 0.0 ? double(py) / total : 0.0;

    // ---- the new node and the two slots it opens
    const int k = ++n_created;
    if (tid == 0) {
      const int krow = int(draft_row_of_child(uint32_t(prow), uint32_t(y), uint32_t(n_rows)));
      s_row[k] = krow;
      s_tok[k] = y;
      s_ppos[k] = int16_t(pos);
      write_node(out, base, k, pos, y, float(v), float(v * rr), krow);
      int ns = n_slots;
      if (1.0 - rr > 0.0) { s_v[ns] = v * (1.0 - rr); s_pos[ns] = int16_t(pos); s_att[ns] = int16_t(attempt + 1); ++ns; }
      s_v[ns] = v * rr; s_pos[ns] = int16_t(k); s_att[ns] = 0;
    }
    n_slots += (1.0 - rr > 0.0) ? 2 : 1;
    __syncthreads();
  }
  if (tid == 0) n_nodes_out[r] = n_created + 1;
}

__global__ void __launch_bounds__(kVThreads, 1)
build_tree_threshold_kernel(const float* __restrict__ draft_table, int n_rows, int vocab, const float* __restrict__ uniforms,
                            int n_uniforms, const int32_t* __restrict__ root_row, float threshold, int max_nodes,
                            TreeOut out, int32_t* __restrict__ n_nodes_out) {
  extern __shared__ __align__(16) uint8_t csm[];
  int32_t* s_row = reinterpret_cast<int32_t*>(csm);                 // [max_nodes + 1]
  double* s_cv = reinterpret_cast<double*>(csm + ((size_t(max_nodes + 1) * 4 + 7) & ~size_t(7)));   // [max_nodes + 1] value of the first sampling under a node
  __shared__ VocabScratch s_vs;

  const int r = blockIdx.x, tid = threadIdx.x;
  const size_t base = size_t(r) * (max_nodes + 1);
  if (tid == 0) {
    s_row[0] = ((root_row[r] % n_rows) + n_rows) % n_rows;        // non-negative remainder: any int32 maps to a row
    s_cv[0] = 1.0;
    write_node(out, base, 0, -1, 0, 1.f, 1.f, s_row[0]);
  }
  __syncthreads();
  int n_created = 0;
  int layer_begin = 0, layer_end = 1;                               // nodes [layer_begin, layer_end) are the current leaves
  while (layer_begin < layer_end && n_created < max_nodes) {
    for (int node = layer_begin; node < layer_end && n_created < max_nodes; ++node) {
      double v = s_cv[node];
      if (!(v >= double(threshold))) continue;
      const int prow = s_row[node];
      float4 R[kMaxChunks];
      load_row(R, draft_table + size_t(prow) * vocab, vocab);
      int attempt = 0;
      while (v >= double(threshold) && n_created < max_nodes) {
        double total;
        const float u = uniforms[draft_uniform_index(uint32_t(prow), uint32_t(attempt), uint32_t(n_uniforms))];
        const int y = sample_inverse_cdf(R, vocab, u, total, s_vs);
        const float py = take_element(R, y, true, s_vs);            // drawn tokens leave the residual
        const double rr = total > 0.0 ? double(py) / total : 0.0;
        const int k = ++n_created;
        if (tid == 0) {
          const int krow = int(draft_row_of_child(uint32_t(prow), uint32_t(y), uint32_t(n_rows)));
          s_row[k] = krow;
          s_cv[k] = v * rr;
          write_node(out, base, k, node, y, float(v), float(v * rr), krow);
        }
        v = v * (1.0 - rr);
        ++attempt;
        if (!(1.0 - rr > 0.0)) break;
      }
    }
    __syncthreads();
    layer_begin = layer_end;
    layer_end = n_created + 1;
  }
  if (tid == 0) n_nodes_out[r] = n_created + 1;
}

size_t build_tree_greedy_smem(int m) {
  const size_t max_slots = 2 * size_t(m) + 2;          // value (8 bytes) + position and attempt (2 + 2) per slot
  return 12 * max_slots + 10 * size_t(m + 1) + 64;     // row and token (4 + 4) + the 2-byte position per node
}

cudaError_t launch_build_tree_greedy(const float* draft_table, int n_rows, int vocab, const float* uniforms, int n_uniforms,
                                     const int32_t* root_row, int n_req, int m, int32_t* parents, int32_t* tokens,
                                     float* values, float* child_values, int32_t* rows, int32_t* n_nodes,
                                     cudaStream_t stream) {
  if (n_req <= 0) return cudaSuccess;
  const size_t smem = build_tree_greedy_smem(m);
  static DynSmemGrant grant;
  if (cudaError_t e = grant.ensure(build_tree_greedy_kernel, smem); e != cudaSuccess) return e;
  TreeOut out{parents, tokens, values, child_values, rows};
  build_tree_greedy_kernel<<<n_req, kVThreads, smem, stream>>>(draft_table, n_rows, vocab, uniforms, n_uniforms, root_row, m,
                                                               out, n_nodes);
  return cudaGetLastError();
}

cudaError_t launch_build_tree_threshold(const float* draft_table, int n_rows, int vocab, const float* uniforms,
                                        int n_uniforms, const int32_t* root_row, int n_req, float threshold, int max_nodes,
                                        int32_t* parents, int32_t* tokens, float* values, float* child_values, int32_t* rows,
                                        int32_t* n_nodes, cudaStream_t stream) {
  if (n_req <= 0) return cudaSuccess;
  const size_t smem = size_t(max_nodes + 1) * 12 + 16;
  TreeOut out{parents, tokens, values, child_values, rows};
  build_tree_threshold_kernel<<<n_req, kVThreads, smem, stream>>>(draft_table, n_rows, vocab, uniforms, n_uniforms, root_row,
                                                                  threshold, max_nodes, out, n_nodes);
  return cudaGetLastError();
}

}  // namespace dyspec
