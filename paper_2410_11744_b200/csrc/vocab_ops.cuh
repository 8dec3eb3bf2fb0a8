// Block-wide operations on one vocabulary-sized probability row held in registers, shared by the tree
// verification and tree construction kernels.  A block has 1024 threads; thread t owns the float4
// chunks t, t + 1024, ... of the row ("row k" of the layout = tokens [4096 k, 4096 k + 4096)), so
// global loads are coalesced.  Vocabulary <= 8 * 1024 * 4 = 32768.
#pragma once

#include "common.cuh"

namespace dyspec {

constexpr int kVThreads = 1024;
constexpr int kMaxChunks = 8;

struct VocabScratch {          // shared memory used by the helpers below
  double rows[kMaxChunks][32];
  double rowtot[kMaxChunks];
  double scan[32];
  float red[33];
  int pick;
  float pub[2];
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block; every thread gets the result.
__device__ __forceinline__ float block_sum(float v, VocabScratch& s) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();                            // s.red may still be read from the previous use
  if (lane == 0) s.red[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float t = s.red[lane];
    t = warp_sum(t);
    if (lane == 0) s.red[32] = t;
  }
  __syncthreads();
  return s.red[32];
}

__device__ __forceinline__ void load_row(float4 (&R)[kMaxChunks], const float* row, int vocab) {
  const int n_vec = vocab >> 2;
#pragma unroll
  for (int k = 0; k < kMaxChunks; ++k) {
    const int v4 = k * kVThreads + int(threadIdx.x);
    R[k] = v4 < n_vec ? __ldg(reinterpret_cast<const float4*>(row) + v4) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

// Element `token` of the row: its owner reads (and optionally zeroes) it and publishes it; every
// thread gets the value.  Contains block barriers.
__device__ __forceinline__ float take_element(float4 (&R)[kMaxChunks], int token, bool zero_it, VocabScratch& s) {
  const int y4 = token >> 2, yk = y4 / kVThreads, yt = y4 - yk * kVThreads, ye = token & 3;
  if (int(threadIdx.x) == yt) {
    float val = 0.f;
#pragma unroll
    for (int k = 0; k < kMaxChunks; ++k) {
      if (k == yk) {
        val = ye == 0 ? R[k].x : ye == 1 ? R[k].y : ye == 2 ? R[k].z : R[k].w;
        if (zero_it) {
          if (ye == 0) R[k].x = 0.f; else if (ye == 1) R[k].y = 0.f; else if (ye == 2) R[k].z = 0.f; else R[k].w = 0.f;
        }
      }
    }
    s.pub[0] = val;
  }
  __syncthreads();
  const float v = s.pub[0];
  __syncthreads();
  return v;
}

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Inverse-CDF draw in token order: the first token v with cumsum(R)[v] > u * sum(R) (the last token if
// rounding leaves none).  Row totals come from one reduction, then one block scan inside the row that
// holds the crossing.  The sums are carried in fp64: tokens of a 32000-word vocabulary have CDF
// intervals of ~1e-5 and less, which fp32 prefix sums (error ~1e-6 of the total) would not resolve
// reproducibly; fp64 runs at half the fp32 rate on this part and the draw is a few dozen adds per
// thread.  Returns the token; `total` receives sum(R).  Contains block barriers.
__device__ __forceinline__ int sample_inverse_cdf(const float4 (&R)[kMaxChunks], int vocab, float u, double& total,
                                                  VocabScratch& s) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_chunks = ((vocab >> 2) + kVThreads - 1) / kVThreads;
#pragma unroll
  for (int k = 0; k < kMaxChunks; ++k) {
    const double w_ = warp_sum_d((double(R[k].x) + double(R[k].y)) + (double(R[k].z) + double(R[k].w)));
    if (lane == 0) s.rows[k][warp] = w_;
  }
  __syncthreads();
  if (warp < kMaxChunks) {
    const double w_ = warp_sum_d(s.rows[warp][lane]);
    if (lane == 0) s.rowtot[warp] = w_;
  }
  if (tid == 0) s.pick = 0x7fffffff;
  __syncthreads();
  double tot = 0.0;
#pragma unroll
  for (int k = 0; k < kMaxChunks; ++k) tot += s.rowtot[k];
  total = tot;
  const double target = double(u) * tot;
  int krow = n_chunks - 1;
  double before = 0.0;
  {
    double acc = 0.0;
    bool found = false;
#pragma unroll
    for (int k = 0; k < kMaxChunks; ++k) {
      if (k < n_chunks && !found) {
        if (acc + s.rowtot[k] > target) { krow = k; before = acc; found = true; }
        else acc += s.rowtot[k];
      }
    }
    if (!found) before = acc - s.rowtot[n_chunks - 1];
  }
  double mine = 0.0;
  float4 rv = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int k = 0; k < kMaxChunks; ++k)
    if (k == krow) rv = R[k];
  mine = (double(rv.x) + double(rv.y)) + (double(rv.z) + double(rv.w));
  double incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();
  if (lane == 31) s.scan[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const double w_ = s.scan[lane];
    double x = w_;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += t;
    }
    s.scan[lane] = x - w_;                                     // mass of the warps before this one
  }
  __syncthreads();
  double cum = before + s.scan[warp] + (incl - mine);          // mass before this thread's 4 tokens
  const int v0 = (krow * kVThreads + tid) * 4;
  int pick = 0x7fffffff;
  const float e4[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    cum += double(e4[e]);
    if (pick == 0x7fffffff && v0 + e < vocab && cum > target) pick = v0 + e;
  }
  if (pick != 0x7fffffff) atomicMin(&s.pick, pick);
  __syncthreads();
  const int y = min(s.pick, vocab - 1);
  __syncthreads();
  return y;
}

// The table-lookup draft model of the construction kernels (the same integer functions as the oracle's).
__host__ __device__ __forceinline__ uint32_t draft_row_of_child(uint32_t parent_row, uint32_t token, uint32_t n_rows) {
  return (parent_row * 2654435761u + (token + 1u) * 40503u) % n_rows;
}
__host__ __device__ __forceinline__ uint32_t draft_uniform_index(uint32_t row, uint32_t attempt, uint32_t n_uniforms) {
  return (row * 7919u + attempt * 104729u + 17u) % n_uniforms;
}

}  // namespace dyspec
