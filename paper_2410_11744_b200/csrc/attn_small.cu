// Tree-verify attention, small-tile regime (Sec. 2 "Tree Attention"; App. C: prefix keys are in the mask).
//
// Used when the packed query tile (tree nodes x GQA group) is small, so the work is bound by
// streaming K/V from HBM rather than by the tensor pipe.  One CTA per SM, BM = 64 query rows:
//   warp 8     producer: streams 64-key K and V tiles through TMA into a 128-byte-swizzled
//              shared-memory ring guarded by mbarriers;
//   warp 9     issues S = Q K^T on the tensor cores (tcgen05.mma, M = 64, N = 64, both operands from
//              shared memory) as soon as a tile's K has landed and one of four score buffers in tensor
//              memory is free, so the scores run ahead of the softmax;
//   warp 10    issues O += P V on the tensor cores (M = 64, one product per 64-column panel of V) when a
//              warp set has put the tile's probabilities into shared memory (over the K tile, which the
//              score product has finished with), into that set's accumulator in tensor memory; the
//              commit behind it frees the ring stage;
//   warps 0-7  two sets of four compute warps (16 query rows per warp).  The sets take alternate key
//              tiles: a warp reads its 16 x 64 scores with tcgen05.ld (with M = 64 accumulator row r
//              lives in lane 32 (r / 16) + r % 16, and the 16x256b shape gives lane (gid, tig) the column
//              pairs 8 j + 2 tig of rows gid and gid + 8), applies the ancestor bitmask on tree tiles and runs the fp32
//              online softmax in the exp2 domain against a LAZY reference: the accumulator is rescaled
//              (tcgen05.ld / st) only when a row maximum has grown by more than 2^8.  The per-tile code
//              is a chain of dependent instructions, so one warp per scheduler leaves the SM mostly
//              idle; two interleaved tiles per scheduler double the rate.  At the end of an item the
//              sets exchange (m, l) through shared memory, each reads one half of the columns of both
//              accumulators, folds them and finishes that half.
// A CTA walks its list of work items; an item either writes final bf16 rows or an fp32 partial
// (O, m, l) for the split-KV combine kernel.  In cluster mode (uniform small batches) the splits of
// a query tile are the CTAs of one thread-block cluster and are merged on chip through distributed
// shared memory instead.
#include "common.cuh"

namespace dyspec {

namespace {

constexpr int BM = 64;       // packed query rows per tile
constexpr int BN = 64;       // keys per tile
constexpr int kComputeWarps = 4;                            // per warp set: 16 query rows each
constexpr int kSets = 2;                                    // two sets take alternate key tiles
constexpr int kProducerWarp = kSets * kComputeWarps;        // TMA
constexpr int kMmaWarp = kProducerWarp + 1;                 // tcgen05.mma issuer for S = Q K^T
constexpr int kPvWarp = kProducerWarp + 2;                  // tcgen05.mma issuer for O += P V
constexpr int kThreads = (kSets * kComputeWarps + 3) * 32;
constexpr int kBarExchFull = 2, kBarExchFree = 3;     // named barriers between the two warp sets

template <int D>
struct SmemLayout {
  static constexpr int kStages = (D == 128) ? 6 : 8;     // one CTA per SM: keep ~190 KB of K/V loads in flight
  static constexpr int kHalves = D / 64;                 // 64-element (128-byte) column panels per row
  static constexpr int kPanelBytes = BN * 128;           // one panel of a K or V tile: 64 rows x 128 B
  static constexpr int kTileBytes = kPanelBytes * kHalves;
  static constexpr int kQBytes = BM * 128 * kHalves;
  static constexpr int kStageBytes = 2 * kTileBytes;     // K then V
  static constexpr int kBarOffset = kQBytes + kStages * kStageBytes;
  static constexpr int kExchMlOffset = kBarOffset + 512;  // set 1 -> set 0: (m, l) of every thread's two rows
  static constexpr int kTotal = kExchMlOffset + kSets * kComputeWarps * 32 * 16;
  static constexpr int kTmemCols = 512;                  // one 64-column score buffer per ring stage (power of two)
};

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of row `row` inside a tile stored as 64-column
// panels with the 128-byte TMA swizzle (chunk index XOR row mod 8 inside each 128-byte row).
__device__ __forceinline__ uint32_t swz(int row, int chunk, int panel_bytes) {
  return static_cast<uint32_t>((chunk >> 3) * panel_bytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// ---- tcgen05 pieces for S = Q K^T (M = 64 query rows, N = 64 keys, fp32 scores in tensor memory)
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Both operands from shared memory; descriptors as (low word, constant high word).
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc) : "memory");
}
// Shared-memory matrix descriptor of a K-major operand stored as 128-byte rows with the 128-byte swizzle
// (8-row groups 1024 bytes apart): low word = address >> 4 | (16 >> 4) << 16; high word = 1024 >> 4 |
// version 1 | swizzle mode 2.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr) { return ((saddr & 0x3ffffu) >> 4) | (1u << 16); }   // 14-bit address field (a CTA in a cluster has address bits above it)
// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, both operands K-major, M = 64, N = 64.
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(BN >> 3) << 17) | (uint32_t(BM >> 4) << 24);
// With M = 64 the accumulator row r lives in TMEM lane 32 (r / 16) + r % 16, so warp w reads rows
// 16 w .. 16 w + 15 from its own lane quarter, and the 16x256b load shape hands them out in 16 x 8
// fragments: registers 4j .. 4j+3 of lane (gid = lane / 4, tig = lane % 4) are (row gid, columns
// 8j + 2 tig, +1) and (row gid + 8, same columns).
__device__ __forceinline__ void tmem_ld_scores(uint32_t taddr, float (&s)[BN / 8][4]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int j = 0; j < BN / 8; ++j) {
    s[j][0] = __uint_as_float(r[4 * j]); s[j][1] = __uint_as_float(r[4 * j + 1]);
    s[j][2] = __uint_as_float(r[4 * j + 2]); s[j][3] = __uint_as_float(r[4 * j + 3]);
  }
}

// O += P V on the tensor cores as well: M = 64 rows, K = 64 keys in four 16-key steps, one product per
// 64-column panel of V (N = 64).  P is a K-major operand (64 rows x 64 keys of bf16 = one 128-byte row each,
// same layout as a Q or K panel); a V panel is an MN-major operand (keys x 64 columns, columns contiguous):
// 8-key groups 1024 bytes apart.  (One N = D product whose operand hops from panel to panel through the
// descriptor's leading-dimension offset gave wrong upper columns in every CTA but the first of a cluster;
// per-panel products do not depend on that field.)
template <int D>
__host__ __device__ constexpr uint32_t idesc_pv() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (uint32_t(64 >> 3) << 17) | (uint32_t(BM >> 4) << 24);   // N = 64 per panel
}
constexpr int kSBufs = 4;                 // score buffers in tensor memory (64 columns each)
constexpr float kRescaleThreshold = 8.f;  // log2 units: O is rescaled only when a row maximum grows by more

// NJ 8-column groups of this warp's 16 accumulator rows (see tmem_ld_scores for the register layout)
template <int NJ>
__device__ __forceinline__ void tmem_ld_rows(uint32_t taddr, float (&v)[NJ][4]) {
  static_assert(NJ == 8, "64 columns at a time");
  tmem_ld_scores(taddr, v);
}
template <int NJ>
__device__ __forceinline__ void tmem_st_rows(uint32_t taddr, const float (&v)[NJ][4]) {
  static_assert(NJ == 8, "64 columns at a time");
  uint32_t r[32];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    r[4 * j] = __float_as_uint(v[j][0]); r[4 * j + 1] = __float_as_uint(v[j][1]);
    r[4 * j + 2] = __float_as_uint(v[j][2]); r[4 * j + 3] = __float_as_uint(v[j][3]);
  }
  asm volatile(
      "tcgen05.st.sync.aligned.16x256b.x8.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

}  // namespace

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_small_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const AttnParams p,
                     const __grid_constant__ FirstItems first) {
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
  // barriers: full[kStages], empty[kStages], q_full, q_empty, src[8] (one per cluster peer), s_full[kStages]
  const uint32_t bar_full = s_bar, bar_empty = s_bar + 8 * kStages;
  const uint32_t bar_qfull = s_bar + 16 * kStages, bar_qempty = bar_qfull + 8, bar_src = bar_qempty + 8;
  // ... s_full[4] / s_free[4] (score buffers), p_ready[kStages] (P of the stage's tile is in shared memory),
  // pv_done[2] (a set's last P V has completed), o_free (both output accumulators have been read out)
  const uint32_t bar_sfull = bar_src + 64, bar_sfree = bar_sfull + 8 * kSBufs, bar_pready = bar_sfree + 8 * kSBufs;
  const uint32_t bar_pvdone = bar_pready + 8 * kStages, bar_ofree = bar_pvdone + 16;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kBarOffset + 24 * kStages + 16 + 64 + 16 * kSBufs + 24);
  volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(smem + L::kBarOffset + 24 * kStages + 16 + 64 + 16 * kSBufs + 28);
  static_assert(24 * kStages + 16 + 64 + 16 * kSBufs + 32 <= 512, "barrier area");
  float4* exch_ml = reinterpret_cast<float4*>(smem + L::kExchMlOffset);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // trace: the last 2048 entries of the buffer hold 8 wall-clock stamps for each of the first 256 CTAs, all
  // taken by thread 0 for the CTA's first item: 0 entry, 3 first scores read, 5 key loop done, 1 set 1's
  // partial folded in, 6 partial parked, 2 pushes issued, 4 (owners) last fold done, 7 exit
  auto stamp = [&](int k) {
#ifdef DYSPEC_CTA_STAMPS
    if (p.trace != nullptr && blockIdx.x < 256 && p.trace_capacity > 4096)
      p.trace[p.trace_capacity - 2048 + 8 * blockIdx.x + k] = global_timer_ns();
#else
    (void)k;
#endif
  };
  if (threadIdx.x == 0) stamp(0);
  if (threadIdx.x == kProducerWarp * 32) {      // the descriptors' fetch overlaps the set-up below
    prefetch_tensormap(&map_q);
    prefetch_tensormap(&map_k);
    prefetch_tensormap(&map_v);
  }
  const WorkItem* my_items = p.items + size_t(blockIdx.x) * p.items_stride;
  // the CTA's w-th item: the first one comes with the kernel parameters, the others from global memory
  const bool first_here = blockIdx.x < kFirstItems;
  auto item_of = [&](int w) -> WorkItem { return (w == 0 && first_here) ? first.item[blockIdx.x] : my_items[w]; };
  const int item_begin = 0;
  const int item_end = first_here ? first.item[blockIdx.x].n_in_cta : my_items[0].n_in_cta;
  // Ring depth.  The last stage is where warp set 1 hands its partial output to set 0 (without clusters
  // the ring is busy with the next item's tiles by then).  In cluster mode a CTA that merges (an owner)
  // keeps the last TWO stages free for the partial rows its peers push into them, possibly while it
  // is still streaming K/V itself, and hands over through a ring stage once the ring is idle; a CTA
  // that does not merge receives nothing (it is the one with the most tiles).
  const bool merge_owner = p.cluster_size > 1 && ((uint32_t(first_here ? first.item[blockIdx.x].merge_owners : my_items[0].merge_owners) >> cluster_ctarank()) & 1u);
  const int n_stages = merge_owner ? kStages - 2 : kStages;
  // tensor memory: O of set 0, O of set 1 (D columns each), then the score buffers
  const uint32_t kOCols = D, kSCol0 = 2 * D;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);                  // the commit behind the tile's P V
      mbar_init(bar_pready + 8 * s, kComputeWarps);
    }
    for (int b = 0; b < kSBufs; ++b) {
      mbar_init(bar_sfull + 8 * b, 1);
      mbar_init(bar_sfree + 8 * b, kComputeWarps);
    }
    mbar_init(bar_pvdone, 1);
    mbar_init(bar_pvdone + 8, 1);
    mbar_init(bar_ofree, kSets * kComputeWarps);
    mbar_init(bar_qfull, 1);
    mbar_init(bar_qempty, 1);                    // arrived on by the commit behind an item's last Q K^T
    for (int k = 0; k < 8; ++k) mbar_init(bar_src + 8 * k, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_holder))), "r"(uint32_t(L::kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  if (p.cluster_size > 1) cluster_arrive();     // "my barriers exist"; peers wait for this only just before they push

  const int g = p.group_size;

  trigger_dependents();     // the combine kernel may be scheduled; it waits for this grid before reading partials
  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer warp (one lane issues)
    if (lane == 0) {
      int ring_stage = 0;    // ring position of the next key tile of this CTA
      uint32_t ring_phase = 0;
      uint32_t qit = 0;      // running item counter (Q buffer phase)
      for (int w = item_begin; w < item_end; ++w, ++qit) {
        const WorkItem item = item_of(w);
        const WorkItem& rq = item;
        // Q tile: box (64 cols, g heads, BM/g nodes) per panel; rows land node-major, head-minor.
        mbar_wait(bar_qempty, (qit & 1) ^ 1, abort_flag, p.status);
        mbar_expect_tx(bar_qfull, L::kQBytes);
        for (int h = 0; h < L::kHalves; ++h)
          tma_load_3d(s_q + h * (BM * 128), &map_q, bar_qfull, h * 64, item.kv_head * g,
                      rq.node0 + (item.row0 >> p.log2_g));
        const int n_prefix_tiles = prefix_tile_count(rq.prefix_len, BN, p.tree_in_pages);
        for (int t = item.tile_begin; t < item.tile_end; ++t) {
          const int stage = ring_stage;
          const uint32_t ph = ring_phase;
          if (++ring_stage == n_stages) { ring_stage = 0; ring_phase ^= 1u; }
          mbar_wait(bar_empty + 8 * stage, ph ^ 1, abort_flag, p.status);
          const int64_t row = kv_tile_row(p, item, t, n_prefix_tiles, BN);
          const uint32_t dst = s_kv + stage * L::kStageBytes;
          mbar_expect_tx(bar_full + 8 * stage, L::kStageBytes);
          for (int h = 0; h < L::kHalves; ++h) {
            tma_load_3d(dst + h * L::kPanelBytes, &map_k, bar_full + 8 * stage, h * 64, item.kv_head, int(row));
            tma_load_3d(dst + L::kTileBytes + h * L::kPanelBytes, &map_v, bar_full + 8 * stage, h * 64, item.kv_head, int(row));
          }
        }
      }
    }
    if (p.cluster_size > 1) cluster_wait();      // pairs with the arrive above (all threads of the cluster take part)
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ S = Q K^T on the tensor cores (one lane issues)
    // Issued as soon as a tile's K has landed and one of the four score buffers is free, i.e. the scores
    // run ahead of the softmax.  The products O += P V have an issuing warp of their own (below), so that
    // neither stream of hand-offs waits for the other.
    if (lane == 0) {
      uint32_t qit = 0;
      int n_base = 0;                      // key tiles of earlier items (ring / score-buffer position)
      const uint32_t q_lo = desc_lo(s_q);
      for (int w = item_begin; w < item_end; ++w, ++qit) {
        const WorkItem item = item_of(w);
        const int T = item.tile_end - item.tile_begin;
        mbar_wait(bar_qfull, qit & 1, abort_flag, p.status);
        for (int i = 0; i < T; ++i) {
          const int pos = n_base + i;
          const int stage = pos % n_stages;
          const uint32_t ph = uint32_t(pos / n_stages) & 1u;
          const int sb = pos & (kSBufs - 1), sb_use = pos / kSBufs;
          mbar_wait(bar_full + 8 * stage, ph, abort_flag, p.status);
          if (sb_use > 0) mbar_wait(bar_sfree + 8 * sb, uint32_t(sb_use - 1) & 1u, abort_flag, p.status);
          tc_fence_after();
          const uint32_t k_lo = desc_lo(s_kv + stage * L::kStageBytes);
#pragma unroll
          for (int ks = 0; ks < KS; ++ks) {
            const uint32_t off = uint32_t((ks >> 2) * L::kPanelBytes + (ks & 3) * 32) >> 4;   // Q and K panels have the same size
            umma_ss(tmem_base + kSCol0 + uint32_t(sb) * BN, q_lo + off, k_lo + off, kDescHi, kIdescQK, ks > 0 ? 1u : 0u);
          }
          tc_commit(bar_sfull + 8 * sb);
        }
        tc_commit(bar_qempty);                    // the Q tile may be replaced once these products are done
        n_base += T;
      }
    }
    if (p.cluster_size > 1) cluster_wait();
  } else if (warp == kPvWarp) {
    // ------------------------------------------------------------------ O += P V on the tensor cores (one lane issues)
    // When a warp set has put a tile's P into shared memory (where the K tile was), into the set's own
    // accumulator; the commit behind it frees the tile's ring stage.  An item's first products wait until
    // the previous item's outputs have been read out of the accumulators.
    if (lane == 0) {
      uint32_t qit = 0;
      int n_base = 0;
      constexpr uint32_t kIdescPV = idesc_pv<D>();
      for (int w = item_begin; w < item_end; ++w, ++qit) {
        const WorkItem item = item_of(w);
        const int T = item.tile_end - item.tile_begin;
        for (int m = 0; m < T; ++m) {
          const int pos = n_base + m;
          const int stage = pos % n_stages;
          const uint32_t ph = uint32_t(pos / n_stages) & 1u;
          const int pv_set = m & 1;
          mbar_wait(bar_pready + 8 * stage, ph, abort_flag, p.status);
          if (m < 2 && qit > 0) mbar_wait(bar_ofree, (qit - 1) & 1u, abort_flag, p.status);   // first product into this accumulator
          tc_fence_after();
          const uint32_t p_lo = desc_lo(s_kv + stage * L::kStageBytes);                        // P sits where the K tile was
          const uint32_t v_lo = desc_lo(s_kv + stage * L::kStageBytes + L::kTileBytes);
          // one product per 64-column panel of V (N = 64 each): no leading-dimension hop inside an operand
#pragma unroll
          for (int h = 0; h < L::kHalves; ++h)
#pragma unroll
            for (int kk = 0; kk < BN / 16; ++kk)
              umma_ss(tmem_base + uint32_t(pv_set) * kOCols + uint32_t(h) * 64u, p_lo + uint32_t(kk) * (32u >> 4),
                      v_lo + uint32_t(h) * (uint32_t(L::kPanelBytes) >> 4) + uint32_t(kk) * (2048u >> 4), kDescHi, kIdescPV,
                      (m >= 2 || kk > 0) ? 1u : 0u);
          tc_commit(bar_empty + 8 * stage);
          tc_commit(bar_pvdone + 8 * pv_set);
        }
        n_base += T;
      }
    }
    if (p.cluster_size > 1) cluster_wait();
  } else {
  // -------------------------------------------------------------------- compute warps
  // Work items and Q/K/V (through TMA) are inputs that no kernel launched with early start writes: the
  // prefix tiles need nothing else, so they are processed while the preceding kernels of the stream may
  // still be running.  The mask, the partials and the output do depend on them: every thread waits
  // for the preceding kernels right before it first reads mask words or writes to global memory.
  bool dep_ok = false;
  auto need_dep = [&]() {
    if (!dep_ok) {
      grid_dependency_wait();
      dep_ok = true;
    }
  };
  // "Every peer has initialised its barriers": the peers arrived right after their set-up, long before
  // the first K/V tile can be here, so waiting now costs nothing and the merge does not have to.
  if (p.cluster_size > 1) cluster_wait();
  const int gid = lane >> 2;      // row within an 8-row slab
  const int tig = lane & 3;       // column pair within an 8-column tile
  const int set = warp >> 2;      // warp set: takes the item's key tiles of this parity
  const int cw = warp & 3;        // row block inside the set
  const int wrow = cw * 16;
  const int ctid = cw * 32 + lane;   // thread index inside the set
  int n_base = 0;                 // key tiles of earlier items (ring / score-buffer position)
  int n_pv = 0;                   // P V products of this set so far (one phase of its pv_done barrier each)
  int pv_seen = 0;                // phases of that barrier this thread has seen complete
  // A parity wait only tells the barrier's current phase from the one before it, so a thread must never
  // fall two phases behind: every tile first confirms the product of the set's PREVIOUS tile (issued
  // right after this tile's scores, i.e. long done; one probe) before it lets the next one be issued.
  // Afterwards every product of this set issued so far has landed.
  auto confirm_pv_done = [&]() {
    if (pv_seen < n_pv) {
      mbar_wait(bar_pvdone + 8 * set, uint32_t(pv_seen) & 1u, abort_flag, p.status);
      ++pv_seen;
    }
    tc_fence_after();
  };
  uint32_t qit = 0;

  for (int w = item_begin; w < item_end; ++w, ++qit) {
    const WorkItem item = item_of(w);
    const WorkItem& rq = item;
    const int n_prefix_tiles = prefix_tile_count(rq.prefix_len, BN, p.tree_in_pages);
    const int n_rows = rq.n_nodes * g;                     // packed rows of this (request, kv head)
    const int row_lo = item.row0 + wrow + gid;             // the two packed rows this thread owns
    const int row_hi = row_lo + 8;
    const int node_lo = row_lo >> p.log2_g, node_hi = row_hi >> p.log2_g;
    const bool ok_lo = row_lo < n_rows, ok_hi = row_hi < n_rows;



    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;   // m: the reference the accumulator is scaled to
    const int T_item = item.tile_end - item.tile_begin;
    const uint32_t t_rows = tmem_base + (uint32_t(cw * 32) << 16);         // this warp's 16 accumulator rows
    const uint32_t t_o = t_rows + uint32_t(set) * kOCols;                    // this set's output accumulator
    bool first = true;

    for (int i = set; i < T_item; i += kSets) {
      const int t = item.tile_begin + i;
      const int pos = n_base + i;
      const int stage = pos % n_stages;
      const uint32_t ph = uint32_t(pos / n_stages) & 1u;
      const int sb = pos & (kSBufs - 1);
      const uint32_t s_k = s_kv + stage * L::kStageBytes;
      const uint32_t s_v = s_k + L::kTileBytes;
      // ---- S = Q K^T (16 x 64 per warp) from the tile's score buffer; the stage's own barrier is complete
      //      by then (the products were issued behind it), waiting on it as well makes the TMA-written V
      //      tile visible to this thread.
      // A tree tile's mask words are fetched first (after the preceding kernels are known to be done:
      // the mask builder is one of them), so that the loads are in flight during the waits below.
      // (Tree rows inside the paged sequence: the tile's 64 columns start shift = L % 64 bits before the
      //  64-bit group u of the row, so the group in front of it is fetched as well.)
      uint2 w_lo = make_uint2(0u, 0u), w_hi = make_uint2(0u, 0u);
      uint2 x_lo = make_uint2(0u, 0u), x_hi = make_uint2(0u, 0u);       // the group in front (shifted tiles only)
      const int shift = tree_tile_shift(rq.prefix_len, BN, p.tree_in_pages);
      if (t >= n_prefix_tiles) {
        need_dep();
        const int u = t - n_prefix_tiles;
        const uint2* bits_lo = reinterpret_cast<const uint2*>(p.bits + size_t(rq.node0 + node_lo) * p.words_per_row);
        const uint2* bits_hi = reinterpret_cast<const uint2*>(p.bits + size_t(rq.node0 + node_hi) * p.words_per_row);
        const bool cur = 2 * u < p.words_per_row;                        // a shifted tile may start in the row's last group
        if (ok_lo && cur) w_lo = ld_after_dependency_v2(bits_lo + u);
        if (ok_hi && cur) w_hi = ld_after_dependency_v2(bits_hi + u);
        if (shift != 0 && u > 0) {
          if (ok_lo) x_lo = ld_after_dependency_v2(bits_lo + u - 1);
          if (ok_hi) x_hi = ld_after_dependency_v2(bits_hi + u - 1);
        }
      }
      mbar_wait(bar_sfull + 8 * sb, uint32_t(pos / kSBufs) & 1u, abort_flag, p.status);
      mbar_wait(bar_full + 8 * stage, ph, abort_flag, p.status);
      tc_fence_after();
      if (threadIdx.x == 0 && w == item_begin && t == item.tile_begin) stamp(3);
      float s[BN / 8][4];
      tmem_ld_scores(t_rows + kSCol0 + uint32_t(sb) * BN, s);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_sfree + 8 * sb);        // the buffer may take the scores of a later tile

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
        own = min(BN, rq.n_nodes + shift - u * BN);
        vis_lo = (uint64_t(w_lo.y) << 32) | w_lo.x;
        vis_hi = (uint64_t(w_hi.y) << 32) | w_hi.x;
        if (shift != 0) {
          // tile column c is tree column u * 64 + c - shift: the row's bits from 64 u - shift onwards; in
          // front of the tree's column 0 (u = 0) are the prefix's last `shift` keys, visible to every row
          const uint64_t head = u > 0 ? 0ull : ((1ull << shift) - 1ull);
          vis_lo = (vis_lo << shift) | (((uint64_t(x_lo.y) << 32) | x_lo.x) >> (64 - shift)) | head;
          vis_hi = (vis_hi << shift) | (((uint64_t(x_hi.y) << 32) | x_hi.x) >> (64 - shift)) | head;
        }
      }

      // ---- online softmax (exp2 domain) against a LAZY reference: the accumulator lives in tensor memory, so
      //      it is rescaled only when some row's maximum has grown by more than 2^8 since the reference was
      //      set (probabilities then stay below 2^8, harmless in bf16 and fp32; the final normalisation
      //      uses the same reference).
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
      confirm_pv_done();
      if (first) {
        m_lo = mn_lo; m_hi = mn_hi;
      } else if (__any_sync(0xffffffffu, mn_lo > m_lo + kRescaleThreshold || mn_hi > m_hi + kRescaleThreshold)) {
        // O *= 2^(m - mn) for this warp's rows (every product of this set issued so far has landed)
        const float f_lo = fast_exp2(m_lo - (mn_lo == -INFINITY ? 0.f : mn_lo));
        const float f_hi = fast_exp2(m_hi - (mn_hi == -INFINITY ? 0.f : mn_hi));
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 64) {
          float ov[8][4];
          tmem_ld_rows<8>(t_o + uint32_t(c0), ov);
#pragma unroll
          for (int j = 0; j < 8; ++j) { ov[j][0] *= f_lo; ov[j][1] *= f_lo; ov[j][2] *= f_hi; ov[j][3] *= f_hi; }
          tmem_st_rows<8>(t_o + uint32_t(c0), ov);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        l_lo *= f_lo; l_hi *= f_hi;
        m_lo = mn_lo; m_hi = mn_hi;
      }
      // A row that has seen no visible key yet keeps m = -inf; use 0 as the reference so that
      // exp2(-inf - 0) = 0 and no inf - inf appears.
      const float ref_lo = m_lo == -INFINITY ? 0.f : m_lo;
      const float ref_hi = m_hi == -INFINITY ? 0.f : m_hi;
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
      l_lo += sum_lo;
      l_hi += sum_hi;

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

      // ---- P (bf16) into the stage's K region, which the score product has finished reading: 64 rows of 128
      //      bytes with the same swizzle as a K panel, so that the tensor core reads it as a K-major operand
      {
        const int r_lo_ = wrow + gid, r_hi_ = r_lo_ + 8;
#pragma unroll
        for (int j = 0; j < BN / 8; ++j) {
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(s_k + uint32_t(r_lo_ * 128 + ((j ^ (r_lo_ & 7)) << 4) + tig * 4)), "r"(pf[j][0]) : "memory");
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(s_k + uint32_t(r_hi_ * 128 + ((j ^ (r_hi_ & 7)) << 4) + tig * 4)), "r"(pf[j][1]) : "memory");
        }
      }
      fence_proxy_async();        // the tensor core reads P (and the zeroed V rows) through the async proxy
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_pready + 8 * stage);
      ++n_pv;
      first = false;
    }
    n_base += T_item;

    // ---- epilogue
    if (threadIdx.x == 0 && w == item_begin) stamp(5);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

    // ---- the two warp sets took alternate tiles into accumulators of their own.  They exchange (m, l)
    //      through shared memory, then each set reads ONE half of the columns of BOTH accumulators (thread
    //      ctid of either set owns the same rows and column pairs), folds them and runs every later step
    //      (parking, storing) on that half.
    constexpr int HT = DT / 2;                    // 8-column tiles per half
    constexpr int kAll = kSets * kComputeWarps * 32;
    const int my_tiles = (T_item - set + kSets - 1) / kSets, other_tiles = (T_item - (1 - set) + kSets - 1) / kSets;
    confirm_pv_done();                            // this set's last product has landed
    tc_fence_before();
    if (w != item_begin)          // both sets have read the previous item's values
      asm volatile("bar.sync %0, %1;" ::"n"(kBarExchFree), "n"(kAll) : "memory");
    exch_ml[set * (kComputeWarps * 32) + ctid] = make_float4(m_lo, m_hi, l_lo, l_hi);
    asm volatile("bar.sync %0, %1;" ::"n"(kBarExchFull), "n"(kAll) : "memory");   // also: the other set's products have landed
    tc_fence_after();
    const int cbase = set * (D / 2);              // first column of this set's half
    float o[HT][4];
    {
      const float4 ml = exch_ml[(1 - set) * (kComputeWarps * 32) + ctid];
      const float mn_lo = fmaxf(m_lo, ml.x), mn_hi = fmaxf(m_hi, ml.y);
      const float ref_lo = mn_lo == -INFINITY ? 0.f : mn_lo, ref_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
      const float ka_lo = fast_exp2(m_lo - ref_lo), kb_lo = fast_exp2(ml.x - ref_lo);
      const float ka_hi = fast_exp2(m_hi - ref_hi), kb_hi = fast_exp2(ml.y - ref_hi);
      static_assert(HT == 8 || HT == 4, "half of the columns: 64 or 32");
      float mine[8][4], theirs[8][4];
      // (D = 64: a half is 32 columns; the loads fetch 64 and the upper 32 are ignored -- they belong to the
      //  neighbouring buffer, which is mapped, so this is safe)
      if (my_tiles > 0) tmem_ld_rows<8>(t_rows + uint32_t(set) * kOCols + uint32_t(cbase), mine);
      if (other_tiles > 0) tmem_ld_rows<8>(t_rows + uint32_t(1 - set) * kOCols + uint32_t(cbase), theirs);
#pragma unroll
      for (int j = 0; j < HT; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float a_ = my_tiles > 0 ? mine[j][e] * (e < 2 ? ka_lo : ka_hi) : 0.f;
          const float b_ = other_tiles > 0 ? theirs[j][e] * (e < 2 ? kb_lo : kb_hi) : 0.f;
          o[j][e] = a_ + b_;
        }
      }
      l_lo = l_lo * ka_lo + ml.z * kb_lo; l_hi = l_hi * ka_hi + ml.w * kb_hi;
      m_lo = mn_lo; m_hi = mn_hi;
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_ofree);        // the accumulators may take the next item's products
    if (threadIdx.x == 0 && w == item_begin) stamp(1);
    if (p.cluster_size > 1) {
      // ---- split-KV combine inside a thread-block cluster: the CTAs of a cluster hold the splits of
      // one query tile (a CTA owns exactly one item in this mode).  The scheduler names the owners
      // (item.merge_owners): n_own of the C CTAs, each responsible for R = BM / n_own rows.  Every
      // CTA parks its partial (O, m, l) in its own shared memory (the K/V ring is idle by now),
      // grouped by owner, and PUSHES each group into its owner's receive buffer with one asynchronous
      // shared-to-shared bulk copy that signals a barrier of the owner.  An owner folds the groups
      // into its own, one source at a time as they arrive (owners first, then the CTAs with the
      // larger pieces), with loops kept rolled: this code runs once per CTA, so its cost is mostly
      // instruction fetch, and only the fold of the last arrival is on the critical path.  No remote
      // loads; the only cluster barrier is split around the whole kernel body.
      const int C = p.cluster_size;                       // 2, 4 or 8
      const uint32_t owners = uint32_t(item.merge_owners);
      const int n_own = __popc(owners);                   // 1, 2, 4 or 8
      const int log2r = 6 - (31 - __clz(n_own));
      const int R = 1 << log2r;                           // rows per owner
      const int chunk_floats = R * (D + 2);               // R rows of O, then R maxima, then R sums
      const uint32_t chunk_bytes = uint32_t(chunk_floats) * 4u;
      const int rank = int(cluster_ctarank());
      const bool own = (owners >> rank) & 1u;
      const int my_oi = __popc(owners & ((1u << rank) - 1u));                                        // which group is mine
      float* send = reinterpret_cast<float*>(smem + L::kQBytes);                                    // [n_own][chunk]
      float* recv = reinterpret_cast<float*>(smem + L::kQBytes + (kStages - 2) * L::kStageBytes);   // [C - 1][chunk]
      if (own && threadIdx.x == 0)
        for (int s_ = 0; s_ < C; ++s_)
          if (s_ != rank) mbar_expect_tx(bar_src + 8 * s_, chunk_bytes);
      // (every warp is done with the ring: all of them met at the hand-over barrier)
      {
        // columns are XOR-swizzled by the row so that the 8 rows a warp stores at once hit different banks
        const int r_lo = wrow + gid, r_hi = r_lo + 8;
        float* c_lo = send + (r_lo >> log2r) * chunk_floats;
        float* c_hi = send + (r_hi >> log2r) * chunk_floats;
        const int rr_lo = r_lo & (R - 1), rr_hi = r_hi & (R - 1);
#pragma unroll
        for (int j = 0; j < HT; ++j) {
          const int c = cbase + j * 8 + tig * 2;
          *reinterpret_cast<float2*>(c_lo + rr_lo * D + (c ^ ((rr_lo & 7) << 3))) = make_float2(o[j][0], o[j][1]);
          *reinterpret_cast<float2*>(c_hi + rr_hi * D + (c ^ ((rr_hi & 7) << 3))) = make_float2(o[j][2], o[j][3]);
        }
        if (tig == 0 && set == 0) {
          c_lo[R * D + rr_lo] = m_lo; c_lo[R * D + R + rr_lo] = l_lo;
          c_hi[R * D + rr_hi] = m_hi; c_hi[R * D + R + rr_hi] = l_hi;
        }
      }
      if (threadIdx.x == 0) stamp(6);
      fence_proxy_async();                                 // the bulk copies below read what was just stored
      asm volatile("bar.sync 1, %0;" ::"n"(kSets * kComputeWarps * 32) : "memory");
      // one copy per (owner, quarter of the group): four lanes of warp 0 per owner, so that the copies overlap
      const int tgt = lane & 7, piece = lane >> 3;
      const bool pusher = warp == 0 && tgt < C && tgt != rank && ((owners >> tgt) & 1u);
      if (pusher) {
        const uint32_t slot = uint32_t(rank < tgt ? rank : rank - 1);           // where owner `tgt` keeps source `rank`
        const uint32_t oi = uint32_t(__popc(owners & ((1u << tgt) - 1u)));      // the group that owner is responsible for
        const uint32_t part = chunk_bytes >> 2, at = uint32_t(piece) * part;    // a multiple of 16 bytes for every R and D
        dsmem_push(map_to_cta(smem_u32(recv) + slot * chunk_bytes + at, uint32_t(tgt)),
                   smem_u32(send) + oi * chunk_bytes + at, part, map_to_cta(bar_src + 8 * rank, uint32_t(tgt)));
      }
      if (threadIdx.x == 0) stamp(2);
      if (own) {
        need_dep();                                        // the merged rows go to global memory
        float* acc_o = send + my_oi * chunk_floats;        // the running merge lives in this CTA's own group
        float* acc_m = acc_o + R * D;
        float* acc_l = acc_m + R;
        const int tid = threadIdx.x;                       // compute warps (both sets) are threads 0 .. 255
        const int n_vec = (R * D) >> 2;                    // float4 elements of a group
        constexpr int kB = 4;
        // Sources in the order they are expected: the other owners (small pieces), then the rest.  The
        // LAST source is folded, normalised and stored to global memory in one pass (no write-back of
        // the merged rows, no barriers behind it): it is the only fold on the critical path.
        uint32_t pool_a = owners & ~(1u << rank), pool_b = ((1u << C) - 1u) & ~owners;
#pragma unroll 1
        for (int k_src = 0; k_src < C - 1; ++k_src) {
          int s_;
          if (pool_a) { s_ = __ffs(pool_a) - 1; pool_a &= pool_a - 1u; }
          else { s_ = __ffs(pool_b) - 1; pool_b &= pool_b - 1u; }
          const bool last = k_src == C - 2;
          mbar_wait(bar_src + 8 * s_, 0, abort_flag, p.status);
          const float* src_o = recv + (s_ < rank ? s_ : s_ - 1) * chunk_floats;
          const float* src_m = src_o + R * D;
          const float* src_l = src_m + R;
          // batches of kB independent elements per thread: all loads first, then the math, then the
          // stores (a rolled element-by-element loop is a chain of shared-memory latencies)
#pragma unroll 1
          for (int base = tid; base < n_vec; base += kB * kSets * kComputeWarps * 32) {
            float4 a[kB], b_[kB];
            float ma[kB], ms[kB], la[kB], ls[kB];
#pragma unroll
            for (int k = 0; k < kB; ++k) {
              const int idx = min(base + k * kSets * kComputeWarps * 32, n_vec - 1);
              const int rr = idx / (D / 4);
              ma[k] = acc_m[rr]; ms[k] = src_m[rr];
              la[k] = acc_l[rr]; ls[k] = src_l[rr];
              a[k] = reinterpret_cast<const float4*>(acc_o)[idx];
              b_[k] = reinterpret_cast<const float4*>(src_o)[idx];
            }
#pragma unroll
            for (int k = 0; k < kB; ++k) {
              const float mn = fmaxf(ma[k], ms[k]);
              const float ref = mn == -INFINITY ? 0.f : mn;
              const float keep = fast_exp2(ma[k] - ref), wgt = fast_exp2(ms[k] - ref);
              a[k].x = a[k].x * keep + b_[k].x * wgt; a[k].y = a[k].y * keep + b_[k].y * wgt;
              a[k].z = a[k].z * keep + b_[k].z * wgt; a[k].w = a[k].w * keep + b_[k].w * wgt;
              la[k] = la[k] * keep + ls[k] * wgt;
            }
            if (!last) {
#pragma unroll
              for (int k = 0; k < kB; ++k) {
                const int idx = base + k * kSets * kComputeWarps * 32;
                if (idx < n_vec) reinterpret_cast<float4*>(acc_o)[idx] = a[k];
              }
            } else {
              // normalise and write the rows (element idx sits at swizzled column c of row rr)
#pragma unroll
              for (int k = 0; k < kB; ++k) {
                const int idx = base + k * kSets * kComputeWarps * 32;
                const int rr = idx / (D / 4);
                const int c = ((idx - rr * (D / 4)) * 4) ^ ((rr & 7) << 3);
                const int row = item.row0 + my_oi * R + rr;
                if (idx < n_vec && row < n_rows) {
                  const float inv = la[k] > 0.f ? 1.f / la[k] : 0.f;
                  const int node = row >> p.log2_g;
                  const int head = item.kv_head * g + (row & (g - 1));
                  uint2 o2;
                  o2.x = pack_bf16x2(a[k].x * inv, a[k].y * inv);
                  o2.y = pack_bf16x2(a[k].z * inv, a[k].w * inv);
                  *reinterpret_cast<uint2*>(p.out + (size_t(rq.node0 + node) * p.n_q_heads + head) * D + c) = o2;
                }
              }
            }
          }
          if (!last) {
            asm volatile("bar.sync 1, %0;" ::"n"(kSets * kComputeWarps * 32) : "memory");   // every row's old maximum has been used
            if (tid < R) {
              const float ma = acc_m[tid], ms = src_m[tid];
              const float mn = fmaxf(ma, ms);
              const float ref = mn == -INFINITY ? 0.f : mn;
              acc_l[tid] = acc_l[tid] * fast_exp2(ma - ref) + src_l[tid] * fast_exp2(ms - ref);
              acc_m[tid] = mn;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kSets * kComputeWarps * 32) : "memory");
          }
        }
        if (threadIdx.x == 0) stamp(4);
      }
      if (pusher) dsmem_push_wait_source_read();          // the parked rows must outlive the copies that read them
    } else if (item.slot < 0) {
      need_dep();
      const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
      const int head_lo = item.kv_head * g + (row_lo & (g - 1)), head_hi = item.kv_head * g + (row_hi & (g - 1));
      __nv_bfloat16* out_lo = p.out + (size_t(rq.node0 + node_lo) * p.n_q_heads + head_lo) * D;
      __nv_bfloat16* out_hi = p.out + (size_t(rq.node0 + node_hi) * p.n_q_heads + head_hi) * D;
#pragma unroll
      for (int j = 0; j < HT; ++j) {
        const int c = cbase + j * 8 + tig * 2;
        if (ok_lo) *reinterpret_cast<uint32_t*>(out_lo + c) = pack_bf16x2(o[j][0] * inv_lo, o[j][1] * inv_lo);
        if (ok_hi) *reinterpret_cast<uint32_t*>(out_hi + c) = pack_bf16x2(o[j][2] * inv_hi, o[j][3] * inv_hi);
      }
    } else {
      // partial slot: O [BM][D] fp32, then m [BM], then l [BM]
      need_dep();                                          // (the previous launch's combine may still be reading the slots)
      float* slot = p.partial + size_t(item.slot) * p.slot_floats;
      const int r_lo = wrow + gid, r_hi = r_lo + 8;
#pragma unroll
      for (int j = 0; j < HT; ++j) {
        const int c = cbase + j * 8 + tig * 2;
        if (ok_lo) *reinterpret_cast<float2*>(slot + r_lo * D + c) = make_float2(o[j][0], o[j][1]);
        if (ok_hi) *reinterpret_cast<float2*>(slot + r_hi * D + c) = make_float2(o[j][2], o[j][3]);
      }
      if (tig == 0 && set == 0) {
        if (ok_lo) { slot[BM * D + r_lo] = m_lo; slot[BM * D + BM + r_lo] = l_lo; }
        if (ok_hi) { slot[BM * D + r_hi] = m_hi; slot[BM * D + BM + r_hi] = l_hi; }
      }
    }
  }
  if (threadIdx.x == 0) stamp(7);
  }  // compute warps

  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(L::kTmemCols)) : "memory");
  }
}

size_t attn_small_smem_bytes(int head_dim) {
  return (head_dim == 128 ? SmemLayout<128>::kTotal : SmemLayout<64>::kTotal) + 1024;
}
int attn_small_threads() { return kThreads; }

// How many clusters of `cluster_size` CTAs of this kernel the current device can hold at once (the SMs of a
// cluster come from one GPC, so fewer than SMs / cluster_size); -1 when that cannot be asked (no device).
// Asked once per (device, head dimension, cluster size).
int attn_small_max_clusters(int head_dim, int cluster_size) {
  static std::atomic<int> cache[DynSmemGrant::kDevices][2][4];
  static std::atomic<bool> init{false};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= DynSmemGrant::kDevices) { cudaGetLastError(); return -1; }
  if (!init.exchange(true))
    for (auto& d : cache) for (auto& h : d) for (auto& c : h) c.store(-2);
  const int hi = head_dim == 128 ? 0 : 1, ci = cluster_size == 8 ? 3 : cluster_size == 4 ? 2 : cluster_size == 2 ? 1 : 0;
  const int have = cache[dev][hi][ci].load();
  if (have != -2) return have;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = unsigned(cluster_size);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(cluster_size));
  cfg.blockDim = dim3(unsigned(kThreads));
  cfg.dynamicSmemBytes = attn_small_smem_bytes(head_dim);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  static DynSmemGrant grant[2];
  cudaError_t e;
  if (head_dim == 128) {
    e = grant[0].ensure(tree_attn_small_kernel<128>, cfg.dynamicSmemBytes);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, tree_attn_small_kernel<128>, &cfg);
  } else {
    e = grant[1].ensure(tree_attn_small_kernel<64>, cfg.dynamicSmemBytes);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, tree_attn_small_kernel<64>, &cfg);
  }
  if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
  cache[dev][hi][ci].store(n);
  return n;
}

cudaError_t launch_attn_small(int head_dim, int n_ctas, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                            const AttnParams& p, const WorkItem* host_items, cudaStream_t stream) {
  // host_items: the host copy of p.items (same stride); each CTA's first item travels as a kernel parameter
  FirstItems first;
  for (int c = 0; c < kFirstItems; ++c)
    first.item[c] = c < n_ctas ? host_items[size_t(c) * p.items_stride] : WorkItem{};
  const size_t smem = attn_small_smem_bytes(head_dim);
  static DynSmemGrant grant[2];
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
    if (cudaError_t ge = grant[0].ensure(tree_attn_small_kernel<128>, smem); ge != cudaSuccess) return ge;
    cfg.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&cfg, tree_attn_small_kernel<128>, mq, mk, mv, p, first);
  } else {
    if (cudaError_t ge = grant[1].ensure(tree_attn_small_kernel<64>, smem); ge != cudaSuccess) return ge;
    cfg.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&cfg, tree_attn_small_kernel<64>, mq, mk, mv, p, first);
  }
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dyspec
