// Tree-verify attention, warp-level tile regime (Sec. 2 "Tree Attention"; App. C: prefix keys are in the mask).
//
// Used when the packed query tile (tree nodes x GQA group) is small, so the work is bound by
// streaming K/V from HBM rather than by the tensor pipe.  One CTA per SM = 4 compute warps (16 query rows
// each, BM = 64) + 1 producer warp.  The producer streams 64-key K and V tiles through TMA into a
// 128-byte-swizzled shared-memory ring guarded by mbarriers; compute warps run QK^T and PV with
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate), an fp32 online softmax in the exp2 domain, and apply
// the ancestor bitmask on tree tiles.  A CTA walks its list of work items; an item either writes
// final bf16 rows or an fp32 partial (O, m, l) for the split-KV combine kernel.  In cluster mode
// (uniform small batches) the splits of a query tile are the CTAs of one thread-block cluster and
// are merged on chip through distributed shared memory instead.
#include "common.cuh"

namespace dyspec {

namespace {

constexpr int BM = 64;       // packed query rows per tile
constexpr int BN = 64;       // keys per tile
constexpr int kComputeWarps = 4;
constexpr int kThreads = (kComputeWarps + 1) * 32;

template <int D>
struct SmemLayout {
  static constexpr int kStages = (D == 128) ? 6 : 8;     // one CTA per SM: keep ~190 KB of K/V loads in flight
  static constexpr int kHalves = D / 64;                 // 64-element (128-byte) column panels per row
  static constexpr int kPanelBytes = BN * 128;           // one panel of a K or V tile: 64 rows x 128 B
  static constexpr int kTileBytes = kPanelBytes * kHalves;
  static constexpr int kQBytes = BM * 128 * kHalves;
  static constexpr int kStageBytes = 2 * kTileBytes;     // K then V
  static constexpr int kBarOffset = kQBytes + kStages * kStageBytes;
  static constexpr int kTotal = kBarOffset + 256;
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of row `row` inside a tile stored as 64-column
// panels with the 128-byte TMA swizzle (chunk index XOR row mod 8 inside each 128-byte row).
__device__ __forceinline__ uint32_t swz(int row, int chunk, int panel_bytes) {
  return static_cast<uint32_t>((chunk >> 3) * panel_bytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

}  // namespace

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_mma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  using L = SmemLayout<D>;
  constexpr int kStages = L::kStages;
  constexpr int KS = D / 16;        // k-steps of QK^T
  constexpr int DT = D / 8;         // 8-wide output column tiles
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // The swizzle pattern is a function of the shared-memory address: keep tile bases 1024-byte aligned.
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t s_q = smem_u32(smem);
  const uint32_t s_kv = s_q + L::kQBytes;
  const uint32_t s_bar = s_q + L::kBarOffset;
  // barriers: full[kStages], empty[kStages], q_full, q_empty
  const uint32_t bar_full = s_bar, bar_empty = s_bar + 8 * kStages;
  const uint32_t bar_qfull = s_bar + 16 * kStages, bar_qempty = bar_qfull + 8;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kBarOffset + 16 * kStages + 16);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // trace: the last 2048 entries of the buffer hold 8 wall-clock stamps for each of the first 256 CTAs
  auto stamp = [&](int k) {
    if (p.trace != nullptr && blockIdx.x < 256 && p.trace_capacity > 4096)
      p.trace[p.trace_capacity - 2048 + 8 * blockIdx.x + k] = global_timer_ns();
  };
  if (threadIdx.x == 0) stamp(0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, kComputeWarps);
    }
    mbar_init(bar_qfull, 1);
    mbar_init(bar_qempty, kComputeWarps);
    *abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();

  const WorkItem* my_items = p.items + size_t(blockIdx.x) * p.items_stride;
  const int item_begin = 0;
  const int item_end = my_items[0].n_in_cta;
  const int g = p.group_size;

  trigger_dependents();     // the combine kernel may be scheduled; it waits for this grid before reading partials
  if (warp == kComputeWarps) {
    // ------------------------------------------------------------------ producer warp (one lane issues)
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      uint32_t it = 0;       // running key-tile counter of this CTA (ring position)
      uint32_t qit = 0;      // running item counter (Q buffer phase)
      for (int w = item_begin; w < item_end; ++w, ++qit) {
        const WorkItem item = my_items[w];
        const WorkItem& rq = item;
        // Q tile: box (64 cols, g heads, BM/g nodes) per panel; rows land node-major, head-minor.
        mbar_wait(bar_qempty, (qit & 1) ^ 1, abort_flag, p.status);
        mbar_expect_tx(bar_qfull, L::kQBytes);
        for (int h = 0; h < L::kHalves; ++h)
          tma_load_3d(s_q + h * (BM * 128), &map_q, bar_qfull, h * 64, item.kv_head * g,
                      rq.node0 + (item.row0 >> p.log2_g));
        const int n_prefix_tiles = (rq.prefix_len + BN - 1) / BN;
        for (int t = item.tile_begin; t < item.tile_end; ++t, ++it) {
          const int stage = it % kStages;
          const uint32_t ph = (it / kStages) & 1;
          mbar_wait(bar_empty + 8 * stage, ph ^ 1, abort_flag, p.status);
          const int64_t row = rq.kv_row0 + (t < n_prefix_tiles ? int64_t(t) * BN
                                                               : int64_t(rq.prefix_len) + int64_t(t - n_prefix_tiles) * BN);
          const uint32_t dst = s_kv + stage * L::kStageBytes;
          mbar_expect_tx(bar_full + 8 * stage, L::kStageBytes);
          for (int h = 0; h < L::kHalves; ++h) {
            tma_load_3d(dst + h * L::kPanelBytes, &map_k, bar_full + 8 * stage, h * 64, item.kv_head, int(row));
            tma_load_3d(dst + L::kTileBytes + h * L::kPanelBytes, &map_v, bar_full + 8 * stage, h * 64, item.kv_head, int(row));
          }
        }
      }
    }
    if (p.cluster_size > 1) {        // every thread of the cluster takes part in the two cluster barriers
      cluster_sync_all();
      cluster_sync_all();
    }
    return;
  }

  // -------------------------------------------------------------------- compute warps
  // Everything read so far (work items, Q/K/V through TMA) is input that no kernel of this stream
  // writes.  The mask, the partials and the output are: wait for the preceding kernels here, while
  // the producer warp keeps streaming K/V.
  grid_dependency_wait();
  const int gid = lane >> 2;      // row within an 8-row slab
  const int tig = lane & 3;       // column pair within an 8-column tile
  const int wrow = warp * 16;
  uint32_t it = 0, qit = 0;

  for (int w = item_begin; w < item_end; ++w, ++qit) {
    const WorkItem item = my_items[w];
    const WorkItem& rq = item;
    const int n_prefix_tiles = (rq.prefix_len + BN - 1) / BN;
    const int n_rows = rq.n_nodes * g;                     // packed rows of this (request, kv head)
    const int row_lo = item.row0 + wrow + gid;             // the two packed rows this thread owns
    const int row_hi = row_lo + 8;
    const int node_lo = row_lo >> p.log2_g, node_hi = row_hi >> p.log2_g;
    const bool ok_lo = row_lo < n_rows, ok_hi = row_hi < n_rows;

    // Q fragments, kept in registers for the whole item.
    uint32_t qf[KS][4];
    if (threadIdx.x == 0 && w == item_begin) stamp(1);
    mbar_wait(bar_qfull, qit & 1, abort_flag, p.status);
    if (threadIdx.x == 0 && w == item_begin) stamp(2);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int row = wrow + (lane & 15);
      const int chunk = ks * 2 + (lane >> 4);
      ldmatrix_x4(s_q + swz(row, chunk, BM * 128), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_qempty);

    float o[DT][4];
#pragma unroll
    for (int j = 0; j < DT; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    for (int t = item.tile_begin; t < item.tile_end; ++t, ++it) {
      const int stage = it % kStages;
      const uint32_t ph = (it / kStages) & 1;
      const uint32_t s_k = s_kv + stage * L::kStageBytes;
      const uint32_t s_v = s_k + L::kTileBytes;
      mbar_wait(bar_full + 8 * stage, ph, abort_flag, p.status);
      if (threadIdx.x == 0 && w == item_begin && t == item.tile_begin) stamp(3);
      if (threadIdx.x == 0 && w == item_begin && t == item.tile_end - 1) stamp(4);

      // ---- S = Q K^T (16 x 64 per warp)
      float s[BN / 8][4];
#pragma unroll
      for (int j = 0; j < BN / 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
        for (int jp = 0; jp < BN / 16; ++jp) {
          const int mi = lane >> 3;
          const int row = jp * 16 + (lane & 7) + ((mi >> 1) << 3);
          const int chunk = ks * 2 + (mi & 1);
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(s_k + swz(row, chunk, L::kPanelBytes), b0, b1, b2, b3);
          mma_bf16(s[2 * jp], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b0, b1);
          mma_bf16(s[2 * jp + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b2, b3);
        }
      }

      // ---- visibility of the 64 key columns for this thread's two rows
      uint64_t vis_lo, vis_hi;
      int own;                          // leading rows of this K/V tile that belong to the request
      if (t < n_prefix_tiles) {
        const int valid = min(BN, rq.prefix_len - t * BN);
        own = min(BN, rq.prefix_len + rq.n_nodes - t * BN);
        const uint64_t m = valid >= 64 ? ~0ull : ((1ull << valid) - 1ull);
        vis_lo = vis_hi = m;
      } else {
        const int u = t - n_prefix_tiles;
        own = min(BN, rq.n_nodes - u * BN);
        vis_lo = vis_hi = 0ull;
        if (ok_lo) {
          const uint2 wv = __ldg(reinterpret_cast<const uint2*>(p.bits + size_t(rq.node0 + node_lo) * p.words_per_row) + u);
          vis_lo = (uint64_t(wv.y) << 32) | wv.x;
        }
        if (ok_hi) {
          const uint2 wv = __ldg(reinterpret_cast<const uint2*>(p.bits + size_t(rq.node0 + node_hi) * p.words_per_row) + u);
          vis_hi = (uint64_t(wv.y) << 32) | wv.x;
        }
      }

      // ---- online softmax (exp2 domain)
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int j = 0; j < BN / 8; ++j) {
        const int c = j * 8 + tig * 2;
        s[j][0] = ((vis_lo >> c) & 1ull) ? s[j][0] * p.scale_log2e : -INFINITY;
        s[j][1] = ((vis_lo >> (c + 1)) & 1ull) ? s[j][1] * p.scale_log2e : -INFINITY;
        s[j][2] = ((vis_hi >> c) & 1ull) ? s[j][2] * p.scale_log2e : -INFINITY;
        s[j][3] = ((vis_hi >> (c + 1)) & 1ull) ? s[j][3] * p.scale_log2e : -INFINITY;
        mx_lo = fmaxf(mx_lo, fmaxf(s[j][0], s[j][1]));
        mx_hi = fmaxf(mx_hi, fmaxf(s[j][2], s[j][3]));
      }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      // A row that has seen no visible key yet keeps m = -inf; use 0 as the reference so that
      // exp2(-inf - 0) = 0 and no inf - inf appears.
      const float ref_lo = mn_lo == -INFINITY ? 0.f : mn_lo;
      const float ref_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
      const float a_lo = fast_exp2(m_lo - ref_lo), a_hi = fast_exp2(m_hi - ref_hi);
      m_lo = mn_lo; m_hi = mn_hi;
      float sum_lo = 0.f, sum_hi = 0.f;
      uint32_t pf[BN / 8][2];
#pragma unroll
      for (int j = 0; j < BN / 8; ++j) {
        const float p0 = fast_exp2(s[j][0] - ref_lo), p1 = fast_exp2(s[j][1] - ref_lo);
        const float p2 = fast_exp2(s[j][2] - ref_hi), p3 = fast_exp2(s[j][3] - ref_hi);
        sum_lo += p0 + p1;
        sum_hi += p2 + p3;
        pf[j][0] = pack_bf16x2(p0, p1);
        pf[j][1] = pack_bf16x2(p2, p3);
      }
      l_lo = l_lo * a_lo + sum_lo;
      l_hi = l_hi * a_hi + sum_hi;
#pragma unroll
      for (int j = 0; j < DT; ++j) { o[j][0] *= a_lo; o[j][1] *= a_lo; o[j][2] *= a_hi; o[j][3] *= a_hi; }

      // ---- V rows past the end of the request are not ours (another request's rows, or memory the
      //      caller never wrote): zero them so that 0 * garbage cannot produce NaN (their probabilities
      //      are exactly 0).  Every compute warp writes the same zeros before its own reads.
      if (own < BN) {
        for (int idx = lane; idx < (BN - own) * (D / 8); idx += 32) {
          const int row = own + idx / (D / 8), chunk = idx % (D / 8);
          asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(s_v + swz(row, chunk, L::kPanelBytes)), "r"(0u) : "memory");
        }
        fence_proxy_async();   // order these generic-proxy writes before the next TMA write to this stage
        __syncwarp();
      }

      // ---- O += P V
#pragma unroll
      for (int kk = 0; kk < BN / 16; ++kk) {
#pragma unroll
        for (int jd = 0; jd < DT / 2; ++jd) {
          const int mi = lane >> 3;
          const int row = kk * 16 + (lane & 7) + ((mi & 1) << 3);
          const int chunk = jd * 2 + (mi >> 1);
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(s_v + swz(row, chunk, L::kPanelBytes), b0, b1, b2, b3);
          mma_bf16(o[2 * jd], pf[2 * kk][0], pf[2 * kk][1], pf[2 * kk + 1][0], pf[2 * kk + 1][1], b0, b1);
          mma_bf16(o[2 * jd + 1], pf[2 * kk][0], pf[2 * kk][1], pf[2 * kk + 1][0], pf[2 * kk + 1][1], b2, b3);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * stage);
    }

    // ---- epilogue
    if (threadIdx.x == 0 && w == item_begin) stamp(5);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    if (p.cluster_size > 1) {
      // ---- split-KV combine inside a thread-block cluster: the CTAs of a cluster hold the splits of
      // one query tile.  Each parks its partial (O, m, l) in its own shared memory (the K/V ring is
      // idle by now: a CTA owns exactly one item in this mode), the cluster synchronises, and CTA k
      // merges rows [k * BM / C, (k + 1) * BM / C) of all C partials through distributed shared memory.
      const int C = p.cluster_size;                       // 2, 4 or 8
      const int log2c = C == 2 ? 1 : (C == 4 ? 2 : 3);
      asm volatile("bar.sync 1, %0;" ::"n"(kComputeWarps * 32) : "memory");     // all warps are done with the ring
      float* sc_o = reinterpret_cast<float*>(smem + L::kQBytes);                 // [BM][D]
      float* sc_m = sc_o + BM * D;                                               // [BM]
      float* sc_l = sc_m + BM;                                                   // [BM]
      {
        const int r_lo = wrow + gid, r_hi = r_lo + 8;
#pragma unroll
        for (int j = 0; j < DT; ++j) {
          const int c = j * 8 + tig * 2;
          *reinterpret_cast<float2*>(sc_o + r_lo * D + c) = make_float2(o[j][0], o[j][1]);
          *reinterpret_cast<float2*>(sc_o + r_hi * D + c) = make_float2(o[j][2], o[j][3]);
        }
        if (tig == 0) { sc_m[r_lo] = m_lo; sc_l[r_lo] = l_lo; sc_m[r_hi] = m_hi; sc_l[r_hi] = l_hi; }
      }
      cluster_sync_all();
      // A warp merges BM / C / 4 rows from C sources: always 16 (row, source) pairs.  All their loads
      // are issued before the first use, so the merge costs about two remote-load latencies in all.
      const int rank = int(cluster_ctarank());
      const int row_base = rank * (BM >> log2c) + warp * ((BM >> log2c) / kComputeWarps);
      const uint32_t a_o = smem_u32(sc_o), a_m = smem_u32(sc_m), a_l = smem_u32(sc_l);
      constexpr int V = D / 32;
      float mm[16], ll[16];
      float vv[16][V];
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const int r = row_base + (q >> log2c);
        const uint32_t src = uint32_t(q & (C - 1));
        mm[q] = ld_dsmem_f32(map_to_cta(a_m + 4u * uint32_t(r), src));
        ll[q] = ld_dsmem_f32(map_to_cta(a_l + 4u * uint32_t(r), src));
        const uint32_t av = map_to_cta(a_o + 4u * uint32_t(r * D + lane * V), src);
        if constexpr (V == 4) {
          const float4 v = ld_dsmem_f32x4(av);
          vv[q][0] = v.x; vv[q][1] = v.y; vv[q][2] = v.z; vv[q][3] = v.w;
        } else {
          const float2 v = ld_dsmem_f32x2(av);
          vv[q][0] = v.x; vv[q][1] = v.y;
        }
      }
      // reduce groups of C consecutive pairs (one row each)
#pragma unroll
      for (int q0 = 0; q0 < 16; q0 += 2) {
        if ((q0 & (C - 1)) != 0) continue;     // q0 starts a row only when it is a multiple of C
        const int r = row_base + (q0 >> log2c);
        const int row = item.row0 + r;
        float m = -INFINITY;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          if (c < C && q0 + c < 16) m = fmaxf(m, mm[q0 + c]);
        const float ref = m == -INFINITY ? 0.f : m;
        float acc[V];
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = 0.f;
        float lsum = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c < C && q0 + c < 16) {
            const float wgt = fast_exp2(mm[q0 + c] - ref);
            lsum += wgt * ll[q0 + c];
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] += wgt * vv[q0 + c][k];
          }
        }
        if (row < n_rows) {
          const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
          const int node = row >> p.log2_g;
          const int head = item.kv_head * g + (row & (g - 1));
          __nv_bfloat16* out = p.out + (size_t(rq.node0 + node) * p.n_q_heads + head) * D;
          if constexpr (V == 4) {
            uint2 o2;
            o2.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
            o2.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
            *reinterpret_cast<uint2*>(out + lane * 4) = o2;
          } else {
            *reinterpret_cast<uint32_t*>(out + lane * 2) = pack_bf16x2(acc[0] * inv, acc[1] * inv);
          }
        }
      }
      cluster_sync_all();                                 // nobody leaves while a peer still reads its shared memory
    } else if (item.slot < 0) {
      const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
      const int head_lo = item.kv_head * g + (row_lo & (g - 1)), head_hi = item.kv_head * g + (row_hi & (g - 1));
      __nv_bfloat16* out_lo = p.out + (size_t(rq.node0 + node_lo) * p.n_q_heads + head_lo) * D;
      __nv_bfloat16* out_hi = p.out + (size_t(rq.node0 + node_hi) * p.n_q_heads + head_hi) * D;
#pragma unroll
      for (int j = 0; j < DT; ++j) {
        const int c = j * 8 + tig * 2;
        if (ok_lo) *reinterpret_cast<uint32_t*>(out_lo + c) = pack_bf16x2(o[j][0] * inv_lo, o[j][1] * inv_lo);
        if (ok_hi) *reinterpret_cast<uint32_t*>(out_hi + c) = pack_bf16x2(o[j][2] * inv_hi, o[j][3] * inv_hi);
      }
    } else {
      // partial slot: O [BM][D] fp32, then m [BM], then l [BM]
      float* slot = p.partial + size_t(item.slot) * p.slot_floats;
      const int r_lo = wrow + gid, r_hi = r_lo + 8;
#pragma unroll
      for (int j = 0; j < DT; ++j) {
        const int c = j * 8 + tig * 2;
        if (ok_lo) *reinterpret_cast<float2*>(slot + r_lo * D + c) = make_float2(o[j][0], o[j][1]);
        if (ok_hi) *reinterpret_cast<float2*>(slot + r_hi * D + c) = make_float2(o[j][2], o[j][3]);
      }
      if (tig == 0) {
        if (ok_lo) { slot[BM * D + r_lo] = m_lo; slot[BM * D + BM + r_lo] = l_lo; }
        if (ok_hi) { slot[BM * D + r_hi] = m_hi; slot[BM * D + BM + r_hi] = l_hi; }
      }
    }
    if (threadIdx.x == 0 && w == item_begin) stamp(6);
  }
  if (threadIdx.x == 0) stamp(7);
}

size_t attn_mma_smem_bytes(int head_dim) {
  return (head_dim == 128 ? SmemLayout<128>::kTotal : SmemLayout<64>::kTotal) + 1024;
}
int attn_mma_threads() { return kThreads; }

cudaError_t launch_attn_mma(int head_dim, int n_ctas, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                            const AttnParams& p, cudaStream_t stream) {
  const size_t smem = attn_mma_smem_bytes(head_dim);
  static bool attr_set[2] = {false, false};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = unsigned(p.cluster_size > 1 ? p.cluster_size : 1);
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(n_ctas));
  cfg.blockDim = dim3(unsigned(kThreads));
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = p.cluster_size > 1 ? 2 : 1;
  cudaError_t e = cudaSuccess;
  if (head_dim == 128) {
    if (!attr_set[0]) {
      cudaError_t e = cudaFuncSetAttribute(tree_attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
      if (e != cudaSuccess) return e;
      attr_set[0] = true;
    }
    cfg.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&cfg, tree_attn_mma_kernel<128>, mq, mk, mv, p);
  } else {
    if (!attr_set[1]) {
      cudaError_t e = cudaFuncSetAttribute(tree_attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
      if (e != cudaSuccess) return e;
      attr_set[1] = true;
    }
    cfg.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&cfg, tree_attn_mma_kernel<64>, mq, mk, mv, p);
  }
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dyspec
