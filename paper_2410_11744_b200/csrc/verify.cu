// Verification of a draft token tree against the target model (Algorithm 3: multi-branch rejection
// sampling along the tree), on the device, so that the step after the tree attention needs no host
// round trip.
//
// One CTA of 1024 threads per request walks the tree from node 0.  At a node it loads the target row
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
#include "common.cuh"

namespace dyspec {

namespace {

constexpr int kVThreads = 1024;
constexpr int kMaxChunks = 8;                 // float4 chunks per thread: vocabulary <= 8 * 1024 * 4 = 32768

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block; every thread gets the result.  `scratch` holds 33 floats.
__device__ __forceinline__ float block_sum(float v, float* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();                            // scratch may still be read from the previous use
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float t = scratch[lane];
    t = warp_sum(t);
    if (lane == 0) scratch[32] = t;
  }
  __syncthreads();
  return scratch[32];
}

}  // namespace

__global__ void __launch_bounds__(kVThreads, 1)
verify_tree_kernel(const int32_t* __restrict__ parents, const int32_t* __restrict__ tokens,
                   const float* __restrict__ draft_probs, const float* __restrict__ target_probs,
                   const float* __restrict__ accept_u, const float* __restrict__ sample_u,
                   const int32_t* __restrict__ node_offsets, int vocab, int bonus_at_leaf,
                   int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_nodes, int32_t* __restrict__ out_count,
                   int max_out, int32_t* status) {
  extern __shared__ __align__(16) uint8_t vsm[];
  float4* s_d = reinterpret_cast<float4*>(vsm);                                   // draft row, [chunk][thread]
  int32_t* s_par = reinterpret_cast<int32_t*>(vsm + size_t(kMaxChunks) * kVThreads * 16);   // [n] parents of the request
  // small scalars
  __shared__ float s_red[33];
  __shared__ float s_rows[kMaxChunks][32];
  __shared__ float s_rowtot[kMaxChunks];
  __shared__ int s_cnt[64];
  __shared__ int s_nchild, s_pick;
  __shared__ float s_ry, s_dy;
  __shared__ int16_t s_child[2048];

  const int r = blockIdx.x;
  const int node0 = node_offsets[r], n = node_offsets[r + 1] - node0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_vec = vocab >> 2;                                  // float4 chunks in a row
  const int n_chunks = (n_vec + kVThreads - 1) / kVThreads;      // per thread, <= kMaxChunks
  int n_out = 0;
  if (n <= 0) {
    if (tid == 0) out_count[r] = 0;
    return;
  }
  bool bad = false;
  for (int i = tid; i < n; i += kVThreads) {
    int p_ = parents[node0 + i];
    if (p_ < -1 || p_ >= i) { p_ = -1; bad = true; }
    s_par[i] = p_;
  }
  if (bad && status) atomicCAS(status, 0, DYSPEC_ERR_BAD_TREE);
  __syncthreads();

  int cur = 0;
  for (int step = 0; step <= n; ++step) {                        // at most n moves; bounded in any case
    // ---- branches of `cur`, in index order
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
      if (k < n_chunks && v4 < n_vec) {
        R[k] = __ldg(t_row + v4);
        if (n_child > 0) {
          const float4 d = __ldg(d_row + v4);
          s_d[k * kVThreads + tid] = d;
          nnz_f += (d.x > 0.f) + (d.y > 0.f) + (d.z > 0.f) + (d.w > 0.f);
        }
      }
    }
    float sR = 1.f, sD = 1.f;
    int nnz = n_child > 0 ? int(block_sum(nnz_f, s_red) + 0.5f) : 0;
    bool moved = false;
    for (int b = 0; b < n_child; ++b) {
      const int child = s_child[b];
      int y = tokens[node0 + child];
      if (y < 0 || y >= vocab) {                                 // not a token: report it, carry on with a legal index
        if (tid == 0 && status) atomicCAS(status, 0, DYSPEC_ERR_INVALID_ARG);
        y = min(max(y, 0), vocab - 1);
      }
      const float c = accept_u[node0 + child];
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
      const float tot = block_sum(part, s_red);                  // (its barriers also order the reads of s_d above)
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
      float rowp[kMaxChunks];
      float part = 0.f;
#pragma unroll
      for (int k = 0; k < kMaxChunks; ++k) {
        rowp[k] = (R[k].x + R[k].y) + (R[k].z + R[k].w);
        part += rowp[k];
      }
      float total = block_sum(part, s_red);
      if (!(total > 0.f)) {                                      // nothing left (Draft covers Target): fall back to Target
#pragma unroll
        for (int k = 0; k < kMaxChunks; ++k) {
          const int v4 = k * kVThreads + tid;
          R[k] = (k < n_chunks && v4 < n_vec) ? __ldg(t_row + v4) : make_float4(0.f, 0.f, 0.f, 0.f);
          rowp[k] = (R[k].x + R[k].y) + (R[k].z + R[k].w);
        }
        part = 0.f;
#pragma unroll
        for (int k = 0; k < kMaxChunks; ++k) part += rowp[k];
        total = block_sum(part, s_red);
      }
      const float target = sample_u[node0 + cur] * total;
      // row totals: row k = tokens [4096 k, 4096 k + 4096)
#pragma unroll
      for (int k = 0; k < kMaxChunks; ++k) {
        const float w_ = warp_sum(rowp[k]);
        if (lane == 0) s_rows[k][warp] = w_;
      }
      __syncthreads();
      if (warp < kMaxChunks) {
        const float w_ = warp_sum(s_rows[warp][lane]);
        if (lane == 0) s_rowtot[warp] = w_;
      }
      if (tid == 0) s_pick = 0x7fffffff;
      __syncthreads();
      // the row that holds the crossing, and the mass before it
      int krow = n_chunks - 1;
      float before = 0.f;
      {
        float acc = 0.f;
        bool found = false;
#pragma unroll
        for (int k = 0; k < kMaxChunks; ++k) {
          if (k < n_chunks && !found) {
            if (acc + s_rowtot[k] > target) { krow = k; before = acc; found = true; }
            else acc += s_rowtot[k];
          }
        }
        if (!found) before = acc - s_rowtot[n_chunks - 1];
      }
      // exclusive scan, inside that row, of the threads' 4-token sums
      float mine = 0.f;
      float4 rv = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int k = 0; k < kMaxChunks; ++k)
        if (k == krow) { mine = rowp[k]; rv = R[k]; }
      float incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      __syncthreads();
      if (lane == 31) s_red[warp] = incl;
      __syncthreads();
      if (warp == 0) {
        const float w_ = s_red[lane];
        float x = w_;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float t = __shfl_up_sync(0xffffffffu, x, o);
          if (lane >= o) x += t;
        }
        s_red[lane] = x - w_;                                    // mass of the warps before this one
      }
      __syncthreads();
      float cum = before + s_red[warp] + (incl - mine);          // mass before this thread's 4 tokens
      const int v0 = (krow * kVThreads + tid) * 4;
      int pick = 0x7fffffff;
      const float e4[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        cum += e4[e];
        if (pick == 0x7fffffff && v0 + e < vocab && cum > target) pick = v0 + e;
      }
      if (pick != 0x7fffffff) atomicMin(&s_pick, pick);
      __syncthreads();
      const int y = min(s_pick, vocab - 1);
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
  const size_t smem = size_t(kMaxChunks) * kVThreads * 16 + size_t(max_nodes) * 4;
  static size_t attr_smem = 48 * 1024;
  if (smem > attr_smem) {
    cudaError_t e = cudaFuncSetAttribute(verify_tree_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    attr_smem = smem;
  }
  verify_tree_kernel<<<n_req, kVThreads, smem, stream>>>(parents, tokens, draft_probs, target_probs, accept_u, sample_u,
                                                         node_offsets, vocab, bonus_at_leaf, out_tokens, out_nodes,
                                                         out_count, max_out, status);
  return cudaGetLastError();
}

}  // namespace dyspec
