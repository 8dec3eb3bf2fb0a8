// Tree-verify attention, tensor-core regime (Sec. 2 "Tree Attention"; App. C: prefix keys are in the mask).
//
// Used when tree nodes x GQA group fill 128-row tiles, i.e. when QK^T and PV are real dense
// contractions.  One CTA per SM, 12 warps:
//   warp 0        TMA producer: Q tile (2 x 128 packed rows) once per work item, then K and V tiles
//                 (128 keys) into a 5-slot shared-memory ring, 128-byte swizzled, mbarrier-guarded.
//   warps 1, 3    tcgen05.mma issuers, one per query half (one lane each).  S = Q K^T: both operands
//                 from shared memory, accumulator in TMEM.  O += P V: P from TMEM (bf16, written by the
//                 softmax warps), V from shared memory as an MN-major operand.  Issuing a tcgen05.mma
//                 holds the thread until the pipe has taken it, so with one issuer the pipe idles
//                 during every barrier probe and commit; with two, one warp's hand-offs overlap the
//                 other's batch.
//   warp 2        allocates / frees the 512 TMEM columns: one S buffer (128 fp32 columns) that the halves
//                 use in turn, P_A and P_B (64 columns of bf16 pairs each), O_A, O_B (128 each).
//   warps 4-7     softmax of query half A: one thread per row, S read with tcgen05.ld (after which the
//                 buffer is handed to the other half), fp32 online softmax in the exp2 domain, ancestor
//                 bitmask on tree tiles, P written with tcgen05.st.  The running output lives in TMEM and
//                 is rescaled only when the row maximum grows by more than 2^8 (the final normalisation
//                 uses the same reference).
//   warps 8-11    the same for query half B.  The two halves alternate on the tensor pipe, so one
//                 half's softmax overlaps the other half's MMAs, and each K/V tile is loaded once
//                 for 256 query rows.
// An item whose group was cut along the keys writes an fp32 partial (O, m, l); after all of its items a CTA
// merges, for each of its split items, a share of the group's rows (no combine launch; see the end of the
// softmax branch).
// Plans with few long groups of equal length run one thread-block cluster per group instead: the cluster's
// hardware barrier stands in for the arrival counters, fences and polling (the partials still travel
// through L2: moving them between the CTAs' shared memories was measured and is no quicker).
// Every wait on a flag or an mbarrier is bounded (see mbar_wait); every TMA load goes to this CTA alone, also
// when the kernel is launched in clusters (the cluster is used for its hardware barrier only).
#include "common.cuh"
#include <type_traits>

namespace dyspec {

namespace {

constexpr int BMH = 128;          // rows of one UMMA tile (one query half)
constexpr int BN = 128;           // keys per tile
constexpr int kThreads = 384;
constexpr int kSlots = 5;
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

template <int D>
struct TcLayout {
  static constexpr int kPanels = D / 64;
  static constexpr int kPanelBytes = 128 * 128;               // 128 rows x 128 bytes
  static constexpr int kTileBytes = kPanels * kPanelBytes;    // one K tile, V tile or query half
  static constexpr int kQBytes = 2 * kTileBytes;
  static constexpr int kRingOffset = kQBytes;
  static constexpr int kBarOffset = kRingOffset + kSlots * kTileBytes;
  static constexpr int kItemRingOffset = kBarOffset + 512;   // queue plans: the CTA's next work items, 8 entries of 64 bytes
  static constexpr int kTotal = kItemRingOffset + 512;
  // Cluster plans (C CTAs per group): CTA k of a cluster merges rows [256 k / C, 256 (k + 1) / C) of the group.
  // When its products are done a CTA keeps its own share of its partial in shared memory, over the (idle) Q
  // tile: the rows (D + 4 floats each: the padding keeps 16-byte row accesses of a warp off each other's
  // banks), then their maxima, then their sums.  The other shares go to their owners' slots in the workspace.
  static constexpr int kParkRow = D + 4;
  static constexpr int kParkRowBytes = kParkRow * 4 + 8;       // a row and its two scalars
  static constexpr int kSpillRowBytes = D * 4 + 8;             // the same in the workspace: rows of D floats (whole 32-byte sectors)
  static_assert(BMH * kParkRowBytes <= kBarOffset, "a share of 128 rows fits in front of the barriers");
};

// Trace tags (see dyspec_set_trace): tag = role << 14 | event << 10 | key-tile index j.
// role 0 = MMA issuer, 1 = softmax half A (row 0), 2 = softmax half B (row 0).
// MMA events: 1 / 3 P ready seen (half A / B), 5 / 6 PV issued, 2 / 4 next QK issued.  Softmax events: 1 S ready seen, 2 S row loaded,
// 3 maximum known, 4 P stored (before wait::st), 5 P published, 6 last PV seen, 7 epilogue done.
// MMA event 9 = role start, 7 = end-of-tile commits issued, 8 = V slot seen.
#define DYSPEC_TAG(role, event, j) ((uint32_t(role) << 14) | (uint32_t(event) << 10) | (uint32_t(j) & 1023u))

// barrier indices (8 bytes each)
enum { B_QFULL = 0, B_QFREE = 1, B_SLOT_FULL = 2, B_SLOT_EMPTY = B_SLOT_FULL + kSlots,
       B_SREADY = B_SLOT_EMPTY + kSlots, B_PREADY = B_SREADY + 2, B_ODONE = B_PREADY + 2, B_OFREE = B_ODONE + 2,
       B_PVDONE = B_OFREE + 2, B_QFULLB = B_PVDONE + 2, B_COUNT = B_QFULLB + 1 };

// Hardware named barriers for thread-to-thread hand-offs inside the CTA (P ready: 128 softmax threads
// -> the MMA-issuing warp): an order of magnitude quicker to notice than an mbarrier in shared memory
// (tens of cycles against 180-300), which is what the issuing warp's time goes into.  mbarriers stay
// where an asynchronous unit signals (TMA bytes, tcgen05.commit).  The arriving side never runs a
// phase ahead: it cannot produce P(j+1) before the issuing warp, having consumed P(j), has issued the
// scores it is computed from.  Every participant reaches its arrive / sync unconditionally (bounded
// mbarrier waits that run out just fall through), so these cannot wait for ever.
__device__ __forceinline__ void named_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void named_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
constexpr int kBarPReady = 1;               // named barriers 1, 2: P of half A, B is in TMEM
constexpr int kPReadyCount = BMH + 32;      // a half's softmax threads + the issuing warp
constexpr int kBarPartial = 3;              // named barriers 3, 4: a half's partial rows are written (its 128 threads)
constexpr int kBarMerge = 5;                // all 256 softmax threads, around the split-KV merge

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// tcgen05.mma with the descriptors given as (low word, constant high word): the issuing thread
// spends one integer add per instruction instead of rebuilding 64-bit descriptors.
__device__ __forceinline__ void umma_ss_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                             uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
      "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_ts_lohi(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                             uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");
}
// Descriptor words: low = address >> 4 | (leading byte offset >> 4) << 16; high = stride byte offset >> 4 |
// version 1 (bit 46) | 128-byte swizzle (bits 61-63).
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes) { return (sbo_bytes >> 4) | (1u << 14) | (2u << 29); }
// (The address field is 14 bits: an address in the shared window of a CTA that runs in a cluster has bits
//  above them, which must not leak into the leading-offset field.)
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) { return ((saddr & 0x3ffffu) >> 4) | ((lbo_bytes >> 4) << 16); }

// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, A K-major, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(b_mn_major) << 16) | (uint32_t(n >> 3) << 17) | (uint32_t(128 >> 4) << 24);
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// 256-bit global stores (sm_100): one full 32-byte sector per lane and instruction, which matters when
// every lane of a warp writes to a different row.
__device__ __forceinline__ void st_global_v8(void* ptr, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"l"(ptr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Packed fp32 pairs (sm_100: one instruction works on two floats held in a 64-bit register pair)
// and the three-input maximum: the softmax threads are bound by instruction issue, and these halve
// the count of the scale, sum and max instructions.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3_f32(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Which key tiles of an item's range are processed.  The prefix tiles always are; of the tree tiles
// only those that some row of the query tile can see (App. C: empty blocks of the tree mask are
// skipped), when the caller passed the per-node tile sets; all of them otherwise.  Every role of the
// CTA derives the same walk from the same inputs.
struct TileWalk {
  int P;            // prefix tiles in the range: tiles tile_begin .. tile_begin + P - 1
  int T;            // tiles processed in all
  uint32_t need;    // tree tiles processed: bit u = tree columns [u * BN, (u + 1) * BN)
  uint32_t first;   // those of them that are processed first (see walk_first); 0 = plain ascending order
};
__device__ __forceinline__ TileWalk walk_dense(const WorkItem& item, int n_prefix_tiles) {
  TileWalk wk;
  wk.P = max(0, min(item.tile_end, n_prefix_tiles) - item.tile_begin);
  const int u0 = max(item.tile_begin, n_prefix_tiles) - n_prefix_tiles, u1 = item.tile_end - n_prefix_tiles;
  wk.need = u1 > u0 ? (((1u << u1) - 1u) & ~((1u << u0) - 1u)) : 0u;
  wk.T = wk.P + __popc(wk.need);
  wk.first = 0u;
  return wk;
}
// Next tree tile of a walk: the `first` ones in ascending order, then the others in ascending order.
__device__ __forceinline__ int pop_tree_tile(uint32_t& rem, uint32_t first) {
  const uint32_t a = rem & first;
  const int u = __ffs(a ? a : rem) - 1;
  rem &= ~(1u << u);
  return u;
}
// The tree tiles that hold the query tile's own columns: every row sees its own key, so these are needed
// whatever the tile sets say, and a walk that may skip tiles runs them before it has to read the sets
// (i.e. before it has to wait for the mask kernel, or for whatever precedes the call in the stream).
__device__ __forceinline__ uint32_t walk_first(const AttnParams& p, const WorkItem& item, const TileWalk& dense) {
  const int node_lo = item.row0 >> p.log2_g;
  const int node_hi = min(item.n_nodes, ((item.row0 + 2 * BMH - 1) >> p.log2_g) + 1);   // one past the tile's last node
  const int u_lo = node_lo / BN, u_hi = (node_hi - 1) / BN;
  return dense.need & ((2u << u_hi) - 1u) & ~((1u << u_lo) - 1u);
}
// Can the tile sets shorten this walk at all?  Only tiles other than the query tile's own can be skipped, and
// the tile with the root never is; reading the sets costs a round trip to global memory in every role, after
// waiting for the mask kernel.  With fewer than three candidates that has not paid (512-token random trees:
// 16.0 us with the sets read against 14.6 without).
__device__ __forceinline__ bool walk_may_skip(const AttnParams& p, const WorkItem& item, const TileWalk& dense) {
  return p.node_tiles != nullptr && __popc(dense.need & ~walk_first(p, item, dense)) > 2;
}
// Whole warp.  The mask kernel must have completed (grid_dependency_wait) before this reads node_tiles.
__device__ __forceinline__ TileWalk walk_sparse(const AttnParams& p, const WorkItem& item, int n_prefix_tiles, int lane) {
  TileWalk wk = walk_dense(item, n_prefix_tiles);
  if (!walk_may_skip(p, item, wk)) return wk;
  const int node_lo = item.row0 >> p.log2_g;
  const int node_hi = min(item.n_nodes, ((item.row0 + 2 * BMH - 1) >> p.log2_g) + 1);
  uint32_t occ = 0u;
  for (int node = node_lo + lane; node < node_hi; node += 32) occ |= ld_after_dependency_u32(p.node_tiles + item.node0 + node);
  occ = __reduce_or_sync(0xffffffffu, occ);
  // node_tiles counts 64-column tiles; a key tile here is BN = 128 columns: OR the bit pairs together
  uint32_t x = (occ | (occ >> 1)) & 0x55555555u;
  x = (x | (x >> 1)) & 0x33333333u;
  x = (x | (x >> 2)) & 0x0f0f0f0fu;
  x = (x | (x >> 4)) & 0x00ff00ffu;
  x = (x | (x >> 8)) & 0x0000ffffu;
  const uint32_t lowest = wk.need & (0u - wk.need);
  wk.first = walk_first(p, item, wk);
  wk.need = (wk.need & x) | wk.first;
  if (wk.P == 0 && wk.need == 0u) wk.need = lowest;    // an item always runs at least one (fully masked) tile
  wk.T = wk.P + __popc(wk.need);
  return wk;
}

}  // namespace

// kDyn: the CTAs take their items from the shared queue (AttnParams::queue) instead of fixed lists.  A
// template parameter, not a run-time flag: the softmax threads sit right at the register limit and the
// fixed-list kernel should compile exactly as it would without the queue.
// kInPages: the tree rows are part of the paged sequence (AttnParams::tree_in_pages): key tiles follow the
// sequence and a row's mask slice is shifted.  A template parameter for the same reason (the shift code as
// a run-time branch cost the ordinary layouts 2 % on the ragged batch of 8).
template <int D, bool kDyn, bool kInPages>
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const AttnParams p,
                    const __grid_constant__ FirstItems first) {
  using L = TcLayout<D>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t s_q = smem_u32(smem);
  const uint32_t s_ring = s_q + L::kRingOffset;
  const uint32_t s_bar = s_q + L::kBarOffset;
  auto bar = [&](int i) { return s_bar + 8u * uint32_t(i); };
  volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(smem + L::kBarOffset + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kBarOffset + 8 * B_COUNT + 8);
  // "S read out" counters, one per half: its four softmax warps each add 1 after loading a score tile.
  // A monotonic counter, not a phase barrier: the waiting issuer may not have looked at this half's
  // counter for many uses (items with one half in between), which a parity wait would misread.
  const uint32_t s_free_ctr = s_bar + 8u * uint32_t(B_COUNT) + 16u;
  // Shared work queue (see AttnParams::queue): the producer warp takes the CTA's next item and passes
  // its index on to the other roles through an 8-entry ring (a full barrier per entry; the roles are
  // never more than two items apart, since there is one Q buffer, so entries need no "empty" barrier).
  const uint32_t q_full = s_bar + 8u * uint32_t(B_COUNT) + 32u;
  volatile int32_t* q_idx = reinterpret_cast<volatile int32_t*>(smem + L::kBarOffset + 8 * B_COUNT + 96);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(bar(B_QFULL), 1);
    mbar_init(bar(B_QFULLB), 1);
    mbar_init(bar(B_QFREE), 2);
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(bar(B_SLOT_FULL + s), 1);
      mbar_init(bar(B_SLOT_EMPTY + s), 2);
    }
    for (int h = 0; h < 2; ++h) {
      mbar_init(bar(B_SREADY + h), 1);
      mbar_init(bar(B_PREADY + h), BMH);
      mbar_init(bar(B_ODONE + h), 1);
      mbar_init(bar(B_OFREE + h), BMH);
      mbar_init(bar(B_PVDONE + h), 1);
    }
    for (int e = 0; e < 8; ++e) mbar_init(q_full + 8u * uint32_t(e), 1);
    *abort_flag = 0;
    *reinterpret_cast<volatile uint32_t*>(smem + L::kBarOffset + 8 * B_COUNT + 16) = 0u;
    *reinterpret_cast<volatile uint32_t*>(smem + L::kBarOffset + 8 * B_COUNT + 20) = 0u;
    fence_barrier_init();
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_holder))), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  // Fixed lists: CTA c's items are my_items[0 .. item_end).  Queue: my_items is the whole queue, the
  // CTA's k-th item is my_items[index], the index -1 ends the CTA's work.
  // Every CTA's first item also travels with the kernel parameters: its first loads then do not wait for
  // a read of the work list from global memory (about a microsecond when the list is not in L2).
  const WorkItem* my_items = p.items + (kDyn ? size_t(0) : size_t(blockIdx.x) * p.items_stride);
  const bool first_here = blockIdx.x < kFirstItems;
  const int item_end = kDyn ? 0x7fffffff : (first_here ? first.item[blockIdx.x].n_in_cta : my_items[0].n_in_cta);
  // Queue plans: the producer warp, which runs ahead of the other roles, also copies each item it takes into
  // a ring in shared memory, so that the issuing and softmax warps do not pay a global-memory round trip
  // (about a microsecond, on their critical path) at every item boundary.
  uint4* q_item = reinterpret_cast<uint4*>(smem + L::kItemRingOffset);
  auto item_of = [&](int w, int at) -> WorkItem {
    if (w == 0 && first_here) return first.item[blockIdx.x];
    if constexpr (kDyn) {
      if (w > 0) {
        union { WorkItem it; uint4 v[4]; } u;
#pragma unroll
        for (int i = 0; i < 4; ++i) u.v[i] = q_item[((w - 1) & 7) * 4 + i];
        return u.it;
      }
    }
    return my_items[at];
  };
  // for the producer warp (all lanes call it): takes the next item off the queue and publishes it
  auto take_index = [&](int k) -> int {
    if (k == 0) return int(blockIdx.x);
    int idx = 0;
    if (lane == 0) {
      // The queue words were cleared by the last CTA of the previous launch that used this plan; that
      // launch is complete once the kernels this one depends on are.
      if (k == 1) grid_dependency_wait();
      const int t = atomicAdd(p.queue, 1) + int(gridDim.x);
      idx = t < p.n_items_total ? t : -1;
      q_idx[(k - 1) & 7] = idx;
      if (idx >= 0) {
        const uint4* src = reinterpret_cast<const uint4*>(p.items + idx);
#pragma unroll
        for (int i = 0; i < 4; ++i) q_item[((k - 1) & 7) * 4 + i] = __ldg(src + i);
      }
      mbar_arrive(q_full + 8u * uint32_t((k - 1) & 7));      // (release: the entry is written)
      if (idx < 0 && atomicAdd(p.queue + 1, 1) == int(gridDim.x) - 1) {   // every CTA has drained the queue
        p.queue[0] = 0;
        p.queue[1] = 0;
      }
    }
    __syncwarp();                                            // the other lanes of the producer read the entry too
    return __shfl_sync(0xffffffffu, idx, 0);
  };
  // for every other role
  auto next_index = [&](int k) -> int {
    if (k == 0) return int(blockIdx.x);
    // a wait that ran out (the CTA is in its error state) ends the CTA's work: never index with a stale entry
    if (!mbar_wait(q_full + 8u * uint32_t((k - 1) & 7), uint32_t((k - 1) >> 3) & 1u, abort_flag, p.status)) return -1;
    const int idx = q_idx[(k - 1) & 7];
    return idx < p.n_items_total ? idx : -1;
  };
  const int g = p.group_size;
  // Cluster plans: where packed row pr of the parked partial lies (share pr / rows, rows = 256 / C), in bytes
  // from the start of shared memory: the row itself, and its maximum (its sum is 4 * rows bytes further).
  // Cluster plans: share d of this CTA's partial (the rows CTA d of the cluster merges) stays in shared memory
  // when d is this CTA, else it goes to slot (rank - d) mod C - 1 of CTA d's C - 1 slots in the workspace
  // (p.partial), from where d reads it through L2.
  const int park_log2rows = 8 - (p.cluster_size >= 8 ? 3 : p.cluster_size >= 4 ? 2 : 1);
  const uint32_t cl_rank = p.cluster_size > 1 ? cluster_ctarank() : 0u;
  // Writes packed row pr (D fp32 values as bit patterns), its maximum and its sum where they belong.  Rows in the
  // workspace are D floats apart and written with 32-byte stores: whole sectors, which L2 takes without
  // first fetching them from memory.
  auto park_row = [&](int pr, const uint32_t* vals, float m_row, float l_row) {
    const int rows = 1 << park_log2rows, d = pr >> park_log2rows, lr = pr & (rows - 1);
    const int src_no = (int(cl_rank) - d) & (p.cluster_size - 1);
    if (src_no > 0) {
      uint8_t* base = reinterpret_cast<uint8_t*>(p.partial) +
                      (size_t(blockIdx.x - cl_rank + uint32_t(d)) * size_t(p.cluster_size - 1) + size_t(src_no - 1)) * size_t(rows * L::kSpillRowBytes);
      float* row_at = reinterpret_cast<float*>(base) + lr * D;
#pragma unroll
      for (int i = 0; i < D / 8; ++i) st_global_v8(row_at + 8 * i, vals + 8 * i);
      float* max_at = reinterpret_cast<float*>(base) + rows * D + lr;
      max_at[0] = m_row;
      max_at[rows] = l_row;
    } else {
      const uint32_t base = s_q;                           // (ld.shared / st.shared by 32-bit address: the compiler cannot tell that `smem` is shared)
      const uint32_t row_at = base + uint32_t(lr * (L::kParkRow * 4));
#pragma unroll
      for (int i = 0; i < D / 4; ++i) st_shared_v4(row_at + 16u * uint32_t(i), vals[4 * i], vals[4 * i + 1], vals[4 * i + 2], vals[4 * i + 3]);
      const uint32_t max_at = base + uint32_t(rows * (L::kParkRow * 4) + 4 * lr);
      st_shared_f32(max_at, m_row);
      st_shared_f32(max_at + uint32_t(4 * rows), l_row);
    }
  };

  // Register budget: the softmax threads hold a whole S row; the control warps need few registers.
  trigger_dependents();     // the next kernel of the stream may be scheduled; it waits for this grid before it touches what this one writes
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // The whole warp walks the loop (the tile walk is a warp-wide computation); one lane issues.
    {
      const bool elected = lane == 0;
      if (elected) {
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
      }
      uint32_t sc = 0, qit = 0;
      for (int w = 0; w < item_end; ++w, ++qit) {
        int item_at = w;
        if constexpr (kDyn) {
          item_at = take_index(w);
          if (item_at < 0) break;
        }
        const WorkItem item = item_of(w, item_at);
        const WorkItem& rq = item;
        const int nh = (rq.n_nodes * g - item.row0 > BMH) ? 2 : 1;
        mbar_wait(bar(B_QFREE), (qit & 1) ^ 1, abort_flag, p.status);
        // Half A's rows first, then (below) the first K tile, then half B's rows: the item's first score
        // product needs only the first two, and at a launch's start every CTA is waiting for exactly that.
        auto load_q_half = [&](int h, int b) {
          if (elected) {
            mbar_expect_tx(bar(b), L::kTileBytes);
            for (int pn = 0; pn < L::kPanels; ++pn)
              tma_load_3d(s_q + h * L::kTileBytes + pn * L::kPanelBytes, &map_q, bar(b), pn * 64, item.kv_head * g,
                          rq.node0 + ((item.row0 + h * BMH) >> p.log2_g));
          }
        };
        load_q_half(0, B_QFULL);
        const int n_prefix_tiles = prefix_tile_count(rq.prefix_len, BN, kInPages ? 1 : 0);
        // Prefix tiles stream at once; the set of tree tiles may depend on the mask kernel's output,
        // so it is settled (after waiting for that kernel) only when the walk reaches the tree.
        TileWalk wk = walk_dense(item, n_prefix_tiles);
        bool exact = !walk_may_skip(p, item, wk);
        if (!exact) wk.first = walk_first(p, item, wk);
        uint32_t rem = wk.need;
        for (int j = 0;; ++j) {
          if (!exact && j >= wk.P + __popc(wk.first)) {
            grid_dependency_wait();
            wk = walk_sparse(p, item, n_prefix_tiles, lane);
            rem = wk.need & ~wk.first;                   // (the first ones are behind us)
            exact = true;
          }
          if (j >= wk.T) break;
          int t = item.tile_begin + j;
          if (j >= wk.P) t = n_prefix_tiles + pop_tree_tile(rem, wk.first);
          const int64_t row = kv_tile_row(p, item, t, n_prefix_tiles, BN);
          for (int kv = 0; kv < 2; ++kv, ++sc) {
            const int slot = sc % kSlots;
            const uint32_t ph = (sc / kSlots) & 1;
            mbar_wait(bar(B_SLOT_EMPTY + slot), ph ^ 1, abort_flag, p.status);
            if (elected) {
              mbar_expect_tx(bar(B_SLOT_FULL + slot), L::kTileBytes);
              for (int pn = 0; pn < L::kPanels; ++pn)
                tma_load_3d(s_ring + slot * L::kTileBytes + pn * L::kPanelBytes, kv == 0 ? &map_k : &map_v,
                            bar(B_SLOT_FULL + slot), pn * 64, item.kv_head, int(row));
            }
            if (j == 0 && kv == 0 && nh == 2) load_q_half(1, B_QFULLB);
          }
        }
      }
    }
  } else if (warp == 1 || warp == 3) {
    // ------------------------------------------------------------------ MMA issuers: warp 1 for query half A, warp 3 for B
    // Issuing a tcgen05.mma holds the thread until the tensor pipe has taken it, so nothing queues up
    // behind a batch and the pipe idles while its issuer probes barriers, commits or waits.  With one
    // issuer per half, one warp's hand-offs overlap the other's batch.  The halves share the S buffer
    // and the K/V slots: S is handed from use to use in the fixed order A(0) B(0) A(1) B(1) ... (an
    // item with one half: A only) through the "S read out" barrier of the half that used it last, and a
    // slot or the Q tile is released by two commits (both from warp 1 when the item has no half B).
    // The whole warp walks the loop; only the elected lane issues the tcgen05 instructions.
    {
      const int h = warp == 1 ? 0 : 1;
      const bool elected = lane == 0;
      TraceCursor tc_cur = trace_open(p, 0, 3);
      if (!elected || h != 0) tc_cur.at = nullptr;
      trace_event(tc_cur, DYSPEC_TAG(0, 9, 0));
      constexpr uint32_t idesc_qk = make_idesc(BN, 0);
      constexpr uint32_t idesc_pv = make_idesc(D, 1);
      constexpr uint32_t kHiK = desc_hi(1024);            // K-major operands (Q, K): 8-row groups 1024 B apart
      constexpr uint32_t kHiV = desc_hi(1024);            // MN-major operand (V): 8-key groups 1024 B apart
      const uint32_t q_lo0 = desc_lo(s_q, 16) + uint32_t(h) * (L::kTileBytes >> 4);
      const uint32_t ring_k_lo0 = desc_lo(s_ring, 16);
      const uint32_t ring_v_lo0 = desc_lo(s_ring, L::kPanelBytes);   // leading offset = next 64-column panel
      auto issue_qk = [=](uint32_t slot) {
        const uint32_t b_lo = ring_k_lo0 + slot * (L::kTileBytes >> 4);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (uint32_t(ks >> 2) * L::kPanelBytes + uint32_t(ks & 3) * 32u) >> 4;
          if (elected) umma_ss_lohi(tmem_base, q_lo0 + off, kHiK, b_lo + off, kHiK, idesc_qk, ks > 0 ? 1u : 0u);
        }
        if (elected) tc_commit(s_bar + 8u * uint32_t(B_SREADY + h));
      };
      auto issue_pv = [=](uint32_t slot, bool accumulate) {
        const uint32_t b_lo = ring_v_lo0 + slot * (L::kTileBytes >> 4);
        const uint32_t d_tmem = tmem_base + 256u + uint32_t(h) * 128u;
        const uint32_t a_tmem = tmem_base + 128u + uint32_t(h) * 64u;
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk)
          if (elected) umma_ts_lohi(d_tmem, a_tmem + uint32_t(kk) * 8u, b_lo + uint32_t(kk) * (2048u >> 4), kHiV, idesc_pv,
                       (accumulate || kk > 0) ? 1u : 0u);
      };
      uint32_t sc = 0, qit = 0;
      uint32_t n_use[2] = {0, 0};           // S uses (QK^T products) issued so far by half A / B, both counted by both warps
      int last_user = -1;                   // which half used the S buffer last (-1: nobody yet)
      uint32_t n_it = 0;                    // items this half took part in (O-free phase)
      // Before S use: the half that used the buffer last must have read its scores out.
      auto wait_s_free = [&]() {
        if (last_user >= 0) {
          counter_wait(s_free_ctr + 4u * uint32_t(last_user), 4u * n_use[last_user], abort_flag, p.status);
          tc_fence_after();
        }
      };
      for (int w = 0; w < item_end; ++w, ++qit) {
        int item_at = w;
        if constexpr (kDyn) {
          item_at = next_index(w);
          if (item_at < 0) break;
        }
        const WorkItem item = item_of(w, item_at);
        const WorkItem& rq = item;
        const bool two = rq.n_nodes * g - item.row0 > BMH;        // both query halves live
        const int n_prefix_tiles = prefix_tile_count(rq.prefix_len, BN, kInPages ? 1 : 0);
        TileWalk wk = walk_dense(item, n_prefix_tiles);
        bool exact = !walk_may_skip(p, item, wk);
        int T = exact ? wk.T : 0x7fffffff;
        const int n_sure = exact ? 0 : wk.P + __popc(walk_first(p, item, wk));   // tiles that run whatever the tile sets say
        auto settle = [&](int j) {
          if (!exact && j + 2 >= n_sure) {
            grid_dependency_wait();
            wk = walk_sparse(p, item, n_prefix_tiles, lane);
            T = wk.T;
            exact = true;
          }
        };
        settle(-1);
        // S uses of this item, in order: tile 0: A (B), tile 1: A (B), ...  Each warp issues its own and
        // only counts the other's.
        auto release = [&](int b) {                               // one of the two commits that free a slot / the Q tile
          if (elected) tc_commit(bar(b));
          if (!two && elected) tc_commit(bar(b));                 // no half B in this item: warp 1 gives both
        };
        const bool mine = h == 0 || two;
        if (mine) mbar_wait(bar(h == 0 ? B_QFULL : B_QFULLB), (h == 0 ? qit : n_it) & 1, abort_flag, p.status);
        {
          const uint32_t kslot = sc % kSlots, kph = (sc / kSlots) & 1;
          ++sc;
          if (mine) {
            mbar_wait(bar(B_SLOT_FULL + kslot), kph, abort_flag, p.status);
            tc_fence_after();
          }
          // use A(0)
          if (h == 0) { wait_s_free(); issue_qk(kslot); }
          ++n_use[0]; last_user = 0;
          if (two) {                                              // use B(0)
            if (h == 1) { wait_s_free(); issue_qk(kslot); }
            ++n_use[1]; last_user = 1;
          }
          if (mine) {
            release(B_SLOT_EMPTY + kslot);
            if (T == 1) release(B_QFREE);                         // Q is reusable once the item's last QK^T has run
          }
        }
        for (int j = 0;; ++j) {
          settle(j);
          if (j >= T) break;
          const uint32_t vslot = sc % kSlots, vph = (sc / kSlots) & 1;
          ++sc;
          const bool more = j + 1 < T;
          const uint32_t kslot = sc % kSlots, kph = (sc / kSlots) & 1;
          if (more) ++sc;
          if (mine) {
            const uint32_t got = __reduce_and_sync(0xffffffffu,
                mbar_test_wait3(bar(B_SLOT_FULL + vslot), vph, bar(B_SLOT_FULL + (more ? kslot : vslot)), more ? kph : vph,
                                bar(B_SLOT_FULL + vslot), vph));
            if (!(got & 1u)) mbar_wait(bar(B_SLOT_FULL + vslot), vph, abort_flag, p.status);
            if (more && !(got & 2u)) mbar_wait(bar(B_SLOT_FULL + kslot), kph, abort_flag, p.status);
            if (j == 0) mbar_wait(bar(B_OFREE + h), (n_it & 1) ^ 1, abort_flag, p.status);
          }
          // S = Q K(j+1)^T as soon as the S buffer has been read out: issued BEFORE this tile's PV, it does
          // not depend on P, so the tensor work is off the softmax threads' chain.
          if (more) {
            if (h == 0) { wait_s_free(); issue_qk(kslot); }
            ++n_use[0]; last_user = 0;
            if (two) {
              if (h == 1) { wait_s_free(); issue_qk(kslot); }
              ++n_use[1]; last_user = 1;
            }
          }
          if (mine) {
            trace_event(tc_cur, DYSPEC_TAG(0, 2, j));
            named_sync(kBarPReady + h, kPReadyCount);
            tc_fence_after();
            trace_event(tc_cur, DYSPEC_TAG(0, 1, j));
            issue_pv(vslot, j > 0);
            if (elected) tc_commit(bar((more ? B_PVDONE : B_ODONE) + h));
            trace_event(tc_cur, DYSPEC_TAG(0, 5, j));
            release(B_SLOT_EMPTY + vslot);
            if (more) release(B_SLOT_EMPTY + kslot);
            if (j + 2 == T) release(B_QFREE);
            trace_event(tc_cur, DYSPEC_TAG(0, 7, j));
          }
        }
        if (mine) ++n_it;
      }
    }
  }
  // cluster plans: "every CTA has written its partial" (the softmax threads arrive once theirs is out; the
  // hardware barrier counts every thread of the cluster, these warps included)
  if (p.cluster_size > 1) {
    __syncwarp();
    cluster_arrive();
    cluster_wait();
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    // ------------------------------------------------------------------ softmax + epilogue warps
    // Q/K/V and the work items are inputs no kernel launched with early start writes, and full prefix
    // tiles need nothing else: they are processed while the preceding kernels of the stream may still be
    // running.  The mask, the tile sets, the partials and the output do depend on those kernels: the
    // thread waits for them right before it first touches any of these.
    bool dep_ok = false;
    auto need_dep = [&]() {
      if (!dep_ok) {
        grid_dependency_wait();
        dep_ok = true;
      }
    };
    const int h = (warp - 4) >> 2;                       // query half
    const int r = ((warp & 3) << 5) + lane;              // row of the half == TMEM lane
    const uint32_t lane_sel = uint32_t((warp & 3) << 5) << 16;
    const uint32_t t_s = tmem_base + lane_sel;                                  // scores (one buffer, the halves take turns)
    const uint32_t t_p = tmem_base + 128u + uint32_t(h) * 64u + lane_sel;       // this half's probabilities (bf16 pairs)
    const uint32_t t_o = tmem_base + 256u + uint32_t(h) * 128u + lane_sel;
    TraceCursor tc_cur = trace_open(p, 1 + h, 3);
    // wall-clock stamps of every CTA (last 2048 entries of the trace buffer, 8 per CTA, first 256 CTAs), by
    // row 0 of half A: 0 start, 1 first scores seen, 2 / 4 last PV of item 0 / 1 seen, 3 / 5 epilogue of item 0 / 1
    // done, 6 first split-KV merge may start (all partials of its group have arrived), 7 exit
    auto stamp = [&](int k) {
#ifdef DYSPEC_CTA_STAMPS
      if (p.trace != nullptr && h == 0 && r == 0 && blockIdx.x < 256 && p.trace_capacity > 4096)
        p.trace[p.trace_capacity - 2048 + 8 * blockIdx.x + k] = global_timer_ns();
#else
      (void)k;
#endif
    };
    stamp(0);
    uint32_t n_s = 0, n_o = 0;                           // S-ready / O-done phases seen by this half
    uint32_t n_pv = 0;                                   // PV-done phases seen by this half
    uint32_t sc = 0;                                     // ring position (to find V slots)

    for (int w = 0; w < item_end; ++w) {
      int item_at = w;
      if constexpr (kDyn) {
        item_at = next_index(w);
        if (item_at < 0) break;
      }
      const WorkItem item = item_of(w, item_at);
      const WorkItem& rq = item;
      const int n_rows = rq.n_nodes * g;
      const int nh = (n_rows - item.row0 > BMH) ? 2 : 1;
      const int n_prefix_tiles = prefix_tile_count(rq.prefix_len, BN, kInPages ? 1 : 0);
      if (walk_may_skip(p, item, walk_dense(item, n_prefix_tiles))) need_dep();   // the tile walk reads the per-node tile sets
      const TileWalk wk = walk_sparse(p, item, n_prefix_tiles, lane);
      const int T = wk.T;
      if (h >= nh) {
        sc += 2u * uint32_t(T);
        if (item.slot >= 0 && p.merge_in_kernel) {         // this half has no rows: nothing to write, but the group counts halves
          need_dep();
          if (r == 0) red_release_gpu_add(p.counters + 2 * item.group, 1);
        }
        if (p.cluster_size > 1) {                          // cluster plan: the peers read this half's rows all the same
          named_sync(kBarMerge, 2 * BMH);                  // (the other half's products no longer read the Q tile and the ring)
          const int pr = h * BMH + r;
          need_dep();                                      // (shares go to the workspace)
          uint32_t zeros[D];
#pragma unroll
          for (int i = 0; i < D; ++i) zeros[i] = 0u;
          park_row(pr, zeros, -INFINITY, 0.f);
        }
        continue;
      }
      uint32_t rem = wk.need;
      const int row = item.row0 + h * BMH + r;
      const bool ok = row < n_rows;
      const int node = row >> p.log2_g;
      const uint4* mask_row = reinterpret_cast<const uint4*>(p.bits + size_t(rq.node0 + (ok ? node : 0)) * p.words_per_row);

      float m_used = -INFINITY, l = 0.f;
      for (int j = 0; j < T; ++j) {
        int t = item.tile_begin + j;
        if (j >= wk.P) t = n_prefix_tiles + pop_tree_tile(rem, wk.first);
        const uint32_t vslot = sc + 1u;
        sc += 2u;
        // visibility of the 128 key columns of this tile for this row
        uint32_t vis[4];
        int own;
        bool all_visible = false;                 // CTA-uniform: a full prefix tile needs no mask at all
        if (t < n_prefix_tiles) {
          const int valid = min(BN, rq.prefix_len - t * BN);
          all_visible = valid == BN;
          own = min(BN, rq.prefix_len + rq.n_nodes - t * BN);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int rem = valid - 32 * q4;
            vis[q4] = rem >= 32 ? 0xffffffffu : (rem <= 0 ? 0u : ((1u << rem) - 1u));
          }
        } else {
          const int u = t - n_prefix_tiles;
          const int shift = tree_tile_shift(rq.prefix_len, BN, kInPages ? 1 : 0);
          own = min(BN, rq.n_nodes + shift - u * BN);
          uint4 mv = make_uint4(0u, 0u, 0u, 0u);
          need_dep();
          if (ok && (!kInPages || 4 * u < p.words_per_row)) mv = ld_after_dependency_v4(mask_row + u);   // (a shifted tile may start past the row's last group)
          vis[0] = mv.x; vis[1] = mv.y; vis[2] = mv.z; vis[3] = mv.w;
          if (kInPages && shift != 0) {
            // Tree rows inside the paged sequence: tile column c is tree column u * 128 + c - shift, i.e. the
            // 128 bits that start `shift` bits before group u of the row; in front of the tree's column 0
            // (u = 0) are the prefix's last `shift` keys, visible to every row.
            uint4 pv = make_uint4(0u, 0u, 0u, 0u);
            if (ok && u > 0) pv = ld_after_dependency_v4(mask_row + u - 1);
            const int o = BN - shift, ws = o >> 5, bs = o & 31;          // window = bits o .. o + 127 of (pv, mv)
            const uint32_t x[8] = {pv.x, pv.y, pv.z, pv.w, mv.x, mv.y, mv.z, mv.w};
            uint32_t a[5];
#pragma unroll
            for (int q4 = 0; q4 < 5; ++q4) a[q4] = ws == 0 ? x[q4] : ws == 1 ? x[q4 + 1] : ws == 2 ? x[q4 + 2] : x[q4 + 3];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const int head = u > 0 ? 0 : shift - 32 * q4;
              vis[q4] = __funnelshift_r(a[q4], a[q4 + 1], bs) | (head >= 32 ? 0xffffffffu : (head <= 0 ? 0u : ((1u << head) - 1u)));
            }
          }
        }

        mbar_wait(bar(B_SREADY + h), n_s & 1, abort_flag, p.status);
        if (n_s == 0) stamp(1);
        ++n_s;
        tc_fence_after();
        if (r == 0) trace_event(tc_cur, DYSPEC_TAG(1 + h, 1, j));

        // the whole S row (128 fp32) in registers: four loads in flight, one wait
        uint32_t sv[BN];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(t_s + uint32_t(c) * 32u, sv + 32 * c);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) red_release_shared_add(s_free_ctr + 4u * uint32_t(h), 1u);   // this warp's rows are in registers: 4 of these and S may be overwritten
        if (r == 0) trace_event(tc_cur, DYSPEC_TAG(1 + h, 2, j));
        if (!all_visible) {
#pragma unroll
          for (int i = 0; i < BN; ++i)
            if (!((vis[i >> 5] >> (i & 31)) & 1u)) sv[i] = 0xff800000u;   // -inf
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < BN; i += 8) {
          mx4[0] = max3_f32(mx4[0], __uint_as_float(sv[i]), __uint_as_float(sv[i + 1]));
          mx4[1] = max3_f32(mx4[1], __uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3]));
          mx4[2] = max3_f32(mx4[2], __uint_as_float(sv[i + 4]), __uint_as_float(sv[i + 5]));
          mx4[3] = max3_f32(mx4[3], __uint_as_float(sv[i + 6]), __uint_as_float(sv[i + 7]));
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2e;   // scale > 0
        const float m_new = fmaxf(m_used, mx);
        if (r == 0) trace_event(tc_cur, DYSPEC_TAG(1 + h, 3, j));
        if (j > 0) {
          // P(j-1) is still being read, and O still being written, until PV(j-1) has completed
          mbar_wait(bar(B_PVDONE + h), n_pv & 1, abort_flag, p.status);
          ++n_pv;
          tc_fence_after();
        }
        if (j == 0) {
          m_used = m_new;
        } else if (__any_sync(0xffffffffu, m_new > m_used + kRescaleThreshold)) {
          // rescale the running output of this warp's 32 rows: O *= 2^(m_used - m_new)
          const float f = fast_exp2(m_used - (m_new == -INFINITY ? 0.f : m_new));
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t v[32];
            tmem_ld32(t_o + uint32_t(c) * 32u, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * f);
            tmem_st32(t_o + uint32_t(c) * 32u, v);
          }
          l *= f;
          m_used = m_new;
        }
        const float neg_ref = m_used == -INFINITY ? 0.f : -m_used;

        // P = 2^(s * scale - ref) as bf16 pairs, written over the first 64 S columns (masked: 2^-inf = 0)
        const uint64_t scale2 = pack_f32x2(p.scale_log2e, p.scale_log2e), ref2 = pack_f32x2(neg_ref, neg_ref);
        uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint64_t x = fma_f32x2(pack_f32x2(__uint_as_float(sv[32 * c + 2 * i]), __uint_as_float(sv[32 * c + 2 * i + 1])),
                                         scale2, ref2);
            float x0, x1;
            unpack_f32x2(x, x0, x1);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
            pk[i] = pack_bf16x2(p0, p1);
          }
          tmem_st16(t_p + uint32_t(c) * 16u, pk);
        }
        {
          float a0, a1, b0, b1;
          unpack_f32x2(sum2[0], a0, a1);
          unpack_f32x2(sum2[1], b0, b1);
          l += (a0 + a1) + (b0 + b1);
        }
        if (r == 0) trace_event(tc_cur, DYSPEC_TAG(1 + h, 4, j));

        // V rows past the end of the request are not ours: zero them (their probabilities are 0, but
        // 0 * garbage could be NaN).  Half A's warps do it, before P is published to the MMA warp.
        if (own < BN && h == 0) {
          mbar_wait(bar(B_SLOT_FULL + vslot % kSlots), (vslot / kSlots) & 1, abort_flag, p.status);
          uint8_t* v_tile = smem + L::kRingOffset + (vslot % kSlots) * L::kTileBytes;
          for (int idx = r; idx < (BN - own) * 8 * L::kPanels; idx += BMH) {
            const int pn = idx / ((BN - own) * 8), rem = idx % ((BN - own) * 8);
            *reinterpret_cast<uint4*>(v_tile + pn * L::kPanelBytes + (own + rem / 8) * 128 + (rem % 8) * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();
        }
        tmem_wait_st();
        tc_fence_before();
        named_arrive(kBarPReady + h, kPReadyCount);
        if (r == 0) trace_event(tc_cur, DYSPEC_TAG(1 + h, 5, j));
      }

      // ---- epilogue: wait for the last PV, read O, normalise (or emit the partial)
      mbar_wait(bar(B_ODONE + h), n_o & 1, abort_flag, p.status);
      ++n_o;
      if (w < (kDyn ? 1 : 2)) stamp(2 + 2 * w);
      if (r == 0) trace_event(tc_cur, DYSPEC_TAG(1 + h, 6, 0));
      tc_fence_after();
      need_dep();                                          // global writes from here on
      const int head = item.kv_head * g + (row & (g - 1));
      // The CTA's LAST item (fixed lists) leaves through shared memory: this half's region of the Q tile is
      // dead by now (only this half's score products read it, and they have all completed), so the rows
      // are parked there, 16-byte chunks XOR-swizzled by the row, and copied out with whole rows per warp
      // instruction instead of one 32-byte piece of 32 different rows.
      bool staged = false;
      if constexpr (!kDyn) staged = w == item_end - 1;
      constexpr int RB = 2 * D;                            // bytes of a row in the staging region (128 rows of them = one Q half)
      constexpr int CH = RB / 16;                          // 16-byte chunks per row
      uint8_t* stage = smem + h * L::kTileBytes;
      auto stage_at = [&](int srow, int ch) -> uint4* {
        return reinterpret_cast<uint4*>(stage + (ch >> 3) * L::kPanelBytes + srow * 128 + (((ch & 7) ^ (srow & 7)) << 4));
      };
      if (p.cluster_size > 1) {
        // Cluster plan: the item is one piece of its group's keys, the other pieces are with the other CTAs
        // of the cluster.  The row's unnormalised output, maximum and sum are parked in this CTA's shared
        // memory, where the peers fetch them (see the merge behind the item loop).
        uint32_t ov[D];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) tmem_ld32(t_o + uint32_t(c) * 32u, ov + 32 * c);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar(B_OFREE + h));
        named_sync(kBarMerge, 2 * BMH);                    // both halves' products are done: Q tile and ring are idle
        const int pr = h * BMH + r;
        park_row(pr, ov, m_used, l);                       // shared memory, or the owner's slot in the workspace
      } else if (item.slot < 0 && staged) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        uint32_t ov[D];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) tmem_ld32(t_o + uint32_t(c) * 32u, ov + 32 * c);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar(B_OFREE + h));
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) {                  // bf16 row: D / 2 words = CH chunks
          uint4 v;
          v.x = pack_bf16x2(__uint_as_float(ov[8 * ch + 0]) * inv, __uint_as_float(ov[8 * ch + 1]) * inv);
          v.y = pack_bf16x2(__uint_as_float(ov[8 * ch + 2]) * inv, __uint_as_float(ov[8 * ch + 3]) * inv);
          v.z = pack_bf16x2(__uint_as_float(ov[8 * ch + 4]) * inv, __uint_as_float(ov[8 * ch + 5]) * inv);
          v.w = pack_bf16x2(__uint_as_float(ov[8 * ch + 6]) * inv, __uint_as_float(ov[8 * ch + 7]) * inv);
          *stage_at(r, ch) = v;
        }
        named_sync(kBarPartial + h, BMH);
#pragma unroll 4
        for (int id = r; id < BMH * CH; id += BMH) {
          const int srow = id / CH, ch = id % CH;
          const int grow = item.row0 + h * BMH + srow;
          if (grow < n_rows) {
            __nv_bfloat16* dst = p.out + (size_t(rq.node0 + (grow >> p.log2_g)) * p.n_q_heads + item.kv_head * g + (grow & (g - 1))) * D;
            *reinterpret_cast<uint4*>(dst + ch * 8) = *stage_at(srow, ch);
          }
        }
      } else if (item.slot < 0) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        __nv_bfloat16* out = p.out + (size_t(rq.node0 + node) * p.n_q_heads + head) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(t_o + uint32_t(c) * 32u, v);
          tmem_wait_ld();
          if (c == D / 32 - 1) { tc_fence_before(); mbar_arrive(bar(B_OFREE + h)); }
          if (ok) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
              pk[i] = pack_bf16x2(__uint_as_float(v[2 * i]) * inv, __uint_as_float(v[2 * i + 1]) * inv);
            st_global_v8(out + c * 32, pk);
            st_global_v8(out + c * 32 + 16, pk + 8);
          }
        }
      } else {
        // partial slot: O [256][D] fp32, then m [256], then l [256]
        float* slot = p.partial + size_t(item.slot) * p.slot_floats;
        const int pr = h * BMH + r;
        uint32_t ov[D];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) tmem_ld32(t_o + uint32_t(c) * 32u, ov + 32 * c);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar(B_OFREE + h));
        if (staged) {
          // an fp32 row is twice the staging row: two passes of D / 2 columns
#pragma unroll
          for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
            for (int ch = 0; ch < CH; ++ch)
              *stage_at(r, ch) = make_uint4(ov[pass * (D / 2) + 4 * ch], ov[pass * (D / 2) + 4 * ch + 1],
                                            ov[pass * (D / 2) + 4 * ch + 2], ov[pass * (D / 2) + 4 * ch + 3]);
            named_sync(kBarPartial + h, BMH);
#pragma unroll 4
            for (int id = r; id < BMH * CH; id += BMH) {
              const int srow = id / CH, ch = id % CH;
              if (item.row0 + h * BMH + srow < n_rows)
                *reinterpret_cast<uint4*>(slot + (h * BMH + srow) * D + pass * (D / 2) + 4 * ch) = *stage_at(srow, ch);
            }
            if (pass == 0) named_sync(kBarPartial + h, BMH);   // all of pass 0 is read before the region is written again
          }
        } else if (ok) {   // the workspace is 256-byte aligned and slots / rows are multiples of 32 bytes
#pragma unroll
          for (int i = 0; i < D / 8; ++i) st_global_v8(slot + pr * D + i * 8, ov + 8 * i);
        }
        if (ok) {
          slot[2 * BMH * D + pr] = m_used;
          slot[2 * BMH * D + 2 * BMH + pr] = l;
        }
        if (p.merge_in_kernel) {
          // the group's items merge the rows themselves once every half of every item has arrived
          named_sync(kBarPartial + h, BMH);             // the half's rows are written (CTA scope) ...
          if (r == 0) {
            __threadfence();                            // ... one cumulative fence makes them visible GPU-wide
            red_release_gpu_add(p.counters + 2 * item.group, 1);
          }
        }
      }
      if (r == 0) trace_event(tc_cur, DYSPEC_TAG(1 + h, 7, 0));
      if (w < (kDyn ? 1 : 2)) stamp(3 + 2 * w);
#ifdef DYSPEC_CTA_STAMPS
      // developer statistics for the queue plans (which stamp item 0 only): slot 4 = items, slot 5 = key tiles of this CTA
      if (kDyn && p.trace != nullptr && h == 0 && r == 0 && blockIdx.x < 256 && p.trace_capacity > 4096) {
        p.trace[p.trace_capacity - 2048 + 8 * blockIdx.x + 4] = (unsigned long long)(w + 1);
        p.trace[p.trace_capacity - 2048 + 8 * blockIdx.x + 5] += (unsigned long long)T;
      }
#endif
    }
    // ---- split-KV merge (no combine launch): every item of a split group merges a share of the group's
    // rows once all of the group's partials are in the workspace.  Done after ALL of the CTA's items, so
    // that no CTA waits for a partial while it still owes one (arrivals never depend on a wait).  All CTAs
    // of the launch are resident (one wave), so the waits end; they are bounded all the same.
    if constexpr (!kDyn) {
      if (p.merge_in_kernel) {
        const int tid = h * BMH + r;                     // 0 .. 255
        const int mw = tid >> 5;                         // merge warp 0 .. 7
        for (int w = 0; w < item_end; ++w) {
          const WorkItem item = item_of(w, w);
          if (item.slot < 0) continue;
          int32_t* ctr = p.counters + 2 * item.group;
          const int ns = item.n_splits;
          if (tid == 0) {
            const uint64_t t0 = global_timer_ns();
            uint32_t spins = 0;
            while (ld_acquire_gpu(ctr) < 2 * ns) {
              if ((++spins & 0x3f) == 0 && (*abort_flag || global_timer_ns() - t0 > kWaitLimitNs)) {
                *abort_flag = 1;
                if (p.status) atomicCAS(p.status, 0, DYSPEC_ERR_TIMEOUT);
                break;
              }
            }
          }
          named_sync(kBarMerge, 2 * BMH);
          stamp(6);
          const int n_rows = item.n_nodes * g;
          const int share = ((2 * BMH + ns - 1) / ns + 7) & ~7;                 // rows per item, a multiple of the 8 merge warps
          const int s_idx = item.slot - item.slot0;
          const int row_lo = s_idx * share, row_hi = min(2 * BMH, row_lo + share);
          const float* base = p.partial + size_t(item.slot0) * p.slot_floats;
          const float* base_m = base + 2 * BMH * D;                             // a slot: O [256][D], m [256], l [256]
          constexpr int V = D / 32;                                             // floats per lane
          constexpr int KR = 4, KS = 4;                                         // rows per warp and pass; partials in flight per row
          // A pass: KR rows per warp.  Lane 8 k + u fetches (m, l) of row k from partials u, u + 8, ...; every lane
          // fetches its V columns of KS partial rows per row at a time, so a pass is one or two round trips
          // to L2 whatever the number of splits (a loop that uses each value as it arrives is a chain of them).
          for (int pr0 = row_lo + KR * mw; pr0 < row_hi; pr0 += 8 * KR) {
            const int lk = lane >> 3, lu = lane & 7;
            const int lrow = min(pr0 + lk, 2 * BMH - 1);
            if (ns <= 8) {
              // Up to eight splits (the usual case): the row's scalars AND the first four partial rows are
              // requested together, before anything is used: one round trip for up to four splits, two beyond.
              float mv = -INFINITY, lv = 0.f;
              if (lu < ns) {
                const float* sl = base_m + size_t(lu) * p.slot_floats;
                mv = ld_cg_f32(sl + lrow);
                lv = ld_cg_f32(sl + 2 * BMH + lrow);
              }
              float acc[KR][V];
#pragma unroll
              for (int k = 0; k < KR; ++k)
#pragma unroll
                for (int e = 0; e < V; ++e) acc[k][e] = 0.f;
              float f_l = 0.f, lsum = 0.f;
#pragma unroll
              for (int s1 = 0; s1 < 8; s1 += KS) {
                if (s1 >= ns) break;
                float vv[KR][KS][V];
#pragma unroll
                for (int k = 0; k < KR; ++k)
#pragma unroll
                  for (int u = 0; u < KS; ++u) {
                    const int pr = min(pr0 + k, 2 * BMH - 1);
                    const float* sl = base + size_t(min(s1 + u, ns - 1)) * p.slot_floats + pr * D;
                    if constexpr (V == 4) {
                      const float4 x = ld_cg_f32x4(sl + lane * 4);
                      vv[k][u][0] = x.x; vv[k][u][1] = x.y; vv[k][u][2] = x.z; vv[k][u][3] = x.w;
                    } else {
                      const float2 x = ld_cg_f32x2(sl + lane * 2);
                      vv[k][u][0] = x.x; vv[k][u][1] = x.y;
                    }
                  }
                if (s1 == 0) {                                 // the row's reference and this lane's weight
                  float m_r = mv;
                  m_r = fmaxf(m_r, __shfl_xor_sync(0xffffffffu, m_r, 1));
                  m_r = fmaxf(m_r, __shfl_xor_sync(0xffffffffu, m_r, 2));
                  m_r = fmaxf(m_r, __shfl_xor_sync(0xffffffffu, m_r, 4));
                  f_l = lu < ns ? fast_exp2(mv - (m_r == -INFINITY ? 0.f : m_r)) : 0.f;
                  lsum = f_l * lv;
                  lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
                  lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
                  lsum += __shfl_xor_sync(0xffffffffu, lsum, 4);
                }
#pragma unroll
                for (int k = 0; k < KR; ++k)
#pragma unroll
                  for (int u = 0; u < KS; ++u) {
                    const float f = __shfl_sync(0xffffffffu, f_l, 8 * k + s1 + u);     // 0 for a split that does not exist
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[k][e] += f * vv[k][u][e];
                  }
              }
#pragma unroll
              for (int k = 0; k < KR; ++k) {
                const float lk_sum = __shfl_sync(0xffffffffu, lsum, 8 * k);
                const int pr = pr0 + k, row = item.row0 + pr;
                if (pr < row_hi && row < n_rows) {
                  const float inv = lk_sum > 0.f ? 1.f / lk_sum : 0.f;
                  __nv_bfloat16* out = p.out + (size_t(item.node0 + (row >> p.log2_g)) * p.n_q_heads + item.kv_head * g + (row & (g - 1))) * D;
                  if constexpr (V == 4) {
                    uint2 o;
                    o.x = pack_bf16x2(acc[k][0] * inv, acc[k][1] * inv);
                    o.y = pack_bf16x2(acc[k][2] * inv, acc[k][3] * inv);
                    *reinterpret_cast<uint2*>(out + lane * 4) = o;
                  } else {
                    *reinterpret_cast<uint32_t*>(out + lane * 2) = pack_bf16x2(acc[k][0] * inv, acc[k][1] * inv);
                  }
                }
              }
              continue;
            }
            float m_l = -INFINITY;
            for (int s_ = lu; s_ < ns; s_ += 8) m_l = fmaxf(m_l, ld_cg_f32(base_m + size_t(s_) * p.slot_floats + lrow));
            m_l = fmaxf(m_l, __shfl_xor_sync(0xffffffffu, m_l, 1));
            m_l = fmaxf(m_l, __shfl_xor_sync(0xffffffffu, m_l, 2));
            m_l = fmaxf(m_l, __shfl_xor_sync(0xffffffffu, m_l, 4));
            const float ref_l = m_l == -INFINITY ? 0.f : m_l;                   // the row's reference, known to its 8 lanes
            float acc[KR][V], lsum = 0.f;
#pragma unroll
            for (int k = 0; k < KR; ++k)
#pragma unroll
              for (int e = 0; e < V; ++e) acc[k][e] = 0.f;
            for (int s0 = 0; s0 < ns; s0 += 8) {
              // weights of partials s0 .. s0 + 7 for this lane's row
              float f_l = 0.f;
              if (s0 + lu < ns) {
                const float* sl = base_m + size_t(s0 + lu) * p.slot_floats;
                const float mv = ld_cg_f32(sl + lrow), lv = ld_cg_f32(sl + 2 * BMH + lrow);
                f_l = fast_exp2(mv - ref_l);
                lsum += f_l * lv;
              }
              for (int s1 = s0; s1 < min(ns, s0 + 8); s1 += KS) {
                float vv[KR][KS][V];
#pragma unroll
                for (int k = 0; k < KR; ++k)
#pragma unroll
                  for (int u = 0; u < KS; ++u) {
                    const int pr = min(pr0 + k, 2 * BMH - 1);
                    const float* sl = base + size_t(min(s1 + u, ns - 1)) * p.slot_floats + pr * D;
                    if constexpr (V == 4) {
                      const float4 x = ld_cg_f32x4(sl + lane * 4);
                      vv[k][u][0] = x.x; vv[k][u][1] = x.y; vv[k][u][2] = x.z; vv[k][u][3] = x.w;
                    } else {
                      const float2 x = ld_cg_f32x2(sl + lane * 2);
                      vv[k][u][0] = x.x; vv[k][u][1] = x.y;
                    }
                  }
#pragma unroll
                for (int k = 0; k < KR; ++k)
#pragma unroll
                  for (int u = 0; u < KS; ++u) {
                    float f = __shfl_sync(0xffffffffu, f_l, 8 * k + ((s1 - s0 + u) & 7));
                    if (s1 + u >= ns) f = 0.f;
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[k][e] += f * vv[k][u][e];
                  }
              }
            }
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 4);
#pragma unroll
            for (int k = 0; k < KR; ++k) {
              const float lk_sum = __shfl_sync(0xffffffffu, lsum, 8 * k);
              const int pr = pr0 + k, row = item.row0 + pr;
              if (pr < row_hi && row < n_rows) {
                const float inv = lk_sum > 0.f ? 1.f / lk_sum : 0.f;
                const int node = row >> p.log2_g;
                const int head = item.kv_head * g + (row & (g - 1));
                __nv_bfloat16* out = p.out + (size_t(item.node0 + node) * p.n_q_heads + head) * D;
                if constexpr (V == 4) {
                  uint2 o;
                  o.x = pack_bf16x2(acc[k][0] * inv, acc[k][1] * inv);
                  o.y = pack_bf16x2(acc[k][2] * inv, acc[k][3] * inv);
                  *reinterpret_cast<uint2*>(out + lane * 4) = o;
                } else {
                  *reinterpret_cast<uint32_t*>(out + lane * 2) = pack_bf16x2(acc[k][0] * inv, acc[k][1] * inv);
                }
              }
            }
          }
          // the group's last merger leaves the counter pair at zero for the next launch
          if (tid == 0 && atomicAdd(ctr + 1, 1) == ns - 1) {
            ctr[0] = 0;
            ctr[1] = 0;
          }
        }
      }
    }
    // ---- split-KV merge of a cluster plan: the CTAs of a cluster hold the pieces of one (request, kv head,
    // query tile) group, one item each, and CTA k merges rows [k * 256 / C, (k + 1) * 256 / C) of the C
    // partials.  Every CTA has kept its own share of those rows in shared memory and written its shares of the
    // peers' rows to their slots in the workspace; the cluster barrier (release / acquire) makes all of it
    // visible, so there are no arrival counters, no fences and no polling, and the slowest CTA of the cluster
    // is the only thing anybody waits for.  The peers' shares come back through L2: shared-to-shared copies
    // between the CTAs (bulk pushes, or loads of a peer's shared memory) were built and measured first and
    // were no quicker -- a CTA moves about 27 GB/s that way, and loads with one row per lane far less.
    if constexpr (!kDyn) {
      if (p.cluster_size > 1) {
        const int tid = h * BMH + r;
        const uint32_t rank = cl_rank;
        __syncwarp();
        cluster_arrive_release();                          // this thread's parked and spilled values are written
        cluster_wait();
        stamp(6);
        const WorkItem item = item_of(0, 0);
        const int n_rows = item.n_nodes * g;
        need_dep();                                        // global writes below
        auto merge = [&](auto c_tag) {
          constexpr int C = decltype(c_tag)::value;
          constexpr int kRows = 2 * BMH / C;               // rows per CTA
          constexpr int V = D / 32;                        // floats per lane: a warp reads one whole row per load
          constexpr int KR = 4;                            // rows per warp and pass
          constexpr int NR = C - 1;                        // sources in the workspace (source 0 is this CTA's own share)
          constexpr int kSpill = kRows * L::kSpillRowBytes;   // bytes of a share in the workspace
          const int mw = tid >> 5, lk = lane >> 3, lu = lane & 7;
          const float* spilled = reinterpret_cast<const float*>(reinterpret_cast<const uint8_t*>(p.partial) +
                                                               size_t(blockIdx.x) * size_t(NR) * size_t(kSpill));
          // This code runs once per CTA, so the loop over the passes stays rolled.  A pass: KR rows per warp; lane
          // 8 k + u holds (m, l) of row k from source u; every lane its V columns of the KR rows from all C
          // sources, all requested before anything is used, the workspace's one pass ahead.
          constexpr int kPasses = kRows / (8 * KR);
          static_assert(kRows % (8 * KR) == 0, "whole passes");
          float nvv[KR][NR][V], nmv = -INFINITY, nlv = 0.f;           // the next pass's values from the workspace
          auto fetch_spilled = [&](int r0) {
            nmv = -INFINITY;
            nlv = 0.f;
            if (lu > 0 && lu < C) {
              const float* sc_ = spilled + (lu - 1) * (kSpill / 4) + kRows * D + r0 + lk;
              nmv = ld_cg_f32(sc_);
              nlv = ld_cg_f32(sc_ + kRows);
            }
#pragma unroll
            for (int k = 0; k < KR; ++k)
#pragma unroll
              for (int q = 0; q < NR; ++q) {
                const float* at = spilled + q * (kSpill / 4) + (r0 + k) * D + lane * V;
                if constexpr (V == 4) {
                  const float4 x = ld_cg_f32x4(at);
                  nvv[k][q][0] = x.x; nvv[k][q][1] = x.y; nvv[k][q][2] = x.z; nvv[k][q][3] = x.w;
                } else {
                  const float2 x = ld_cg_f32x2(at);
                  nvv[k][q][0] = x.x; nvv[k][q][1] = x.y;
                }
              }
          };
          fetch_spilled(KR * mw);
#pragma unroll 1
          for (int ps = 0; ps < kPasses; ++ps) {
            const int r0 = KR * mw + ps * 8 * KR;
            float mv = nmv, lv = nlv;
            float vv[KR][C][V];
#pragma unroll
            for (int k = 0; k < KR; ++k)
#pragma unroll
              for (int q = 0; q < NR; ++q)
#pragma unroll
                for (int e = 0; e < V; ++e) vv[k][1 + q][e] = nvv[k][q][e];
            if (ps + 1 < kPasses) fetch_spilled(r0 + 8 * KR);
            if (lu == 0) {                                 // this CTA's own share: shared memory
              const uint32_t at = s_q + uint32_t(kRows * (L::kParkRow * 4) + 4 * (r0 + lk));
              mv = ld_shared_f32(at);
              lv = ld_shared_f32(at + uint32_t(4 * kRows));
            }
#pragma unroll
            for (int k = 0; k < KR; ++k) {
              const uint32_t src = s_q + uint32_t((r0 + k) * (L::kParkRow * 4) + lane * (4 * V));
              if constexpr (V == 4) {
                const float4 x = ld_shared_f32x4(src);
                vv[k][0][0] = x.x; vv[k][0][1] = x.y; vv[k][0][2] = x.z; vv[k][0][3] = x.w;
              } else {
                const float2 x = ld_shared_f32x2(src);
                vv[k][0][0] = x.x; vv[k][0][1] = x.y;
              }
            }
            float m_r = mv;
            m_r = fmaxf(m_r, __shfl_xor_sync(0xffffffffu, m_r, 1));
            m_r = fmaxf(m_r, __shfl_xor_sync(0xffffffffu, m_r, 2));
            m_r = fmaxf(m_r, __shfl_xor_sync(0xffffffffu, m_r, 4));
            const float f_l = lu < C ? fast_exp2(mv - (m_r == -INFINITY ? 0.f : m_r)) : 0.f;
            float lsum = f_l * lv;
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 4);
#pragma unroll
            for (int k = 0; k < KR; ++k) {
              float acc[V];
#pragma unroll
              for (int e = 0; e < V; ++e) acc[e] = 0.f;
#pragma unroll
              for (int s_ = 0; s_ < C; ++s_) {
                const float f = __shfl_sync(0xffffffffu, f_l, 8 * k + s_);
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] += f * vv[k][s_][e];
              }
              const float lk_sum = __shfl_sync(0xffffffffu, lsum, 8 * k);
              const int row = item.row0 + int(rank) * kRows + r0 + k;
              if (row < n_rows) {
                const float inv = lk_sum > 0.f ? 1.f / lk_sum : 0.f;
                __nv_bfloat16* out = p.out + (size_t(item.node0 + (row >> p.log2_g)) * p.n_q_heads + item.kv_head * g + (row & (g - 1))) * D;
                if constexpr (V == 4) {
                  uint2 o;
                  o.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
                  o.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
                  *reinterpret_cast<uint2*>(out + lane * 4) = o;
                } else {
                  *reinterpret_cast<uint32_t*>(out + lane * 2) = pack_bf16x2(acc[0] * inv, acc[1] * inv);
                }
              }
            }
          }
        };
        if (p.cluster_size == 2) merge(std::integral_constant<int, 2>{});
        else if (p.cluster_size == 4) merge(std::integral_constant<int, 4>{});
        else merge(std::integral_constant<int, 8>{});
      }
    }
    stamp(7);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

namespace {
template <int D, bool kDyn, bool kInPages>
cudaError_t launch_one(cudaLaunchConfig_t& cfg, size_t smem, const CUtensorMap& mq, const CUtensorMap& mk,
                       const CUtensorMap& mv, const AttnParams& p, const FirstItems& first) {
  static DynSmemGrant grant;           // one per instantiation
  if (cudaError_t e = grant.ensure(tree_attn_tc_kernel<D, kDyn, kInPages>, smem); e != cudaSuccess) return e;
  cfg.dynamicSmemBytes = smem;
  return cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<D, kDyn, kInPages>, mq, mk, mv, p, first);
}
}  // namespace

// Workspace bytes per CTA of a cluster plan: its peers' shares of the rows it merges.
size_t attn_tc_cluster_workspace_per_cta(int head_dim, int cluster_size) {
  if (cluster_size < 2) return 0;
  const int row_bytes = head_dim == 128 ? TcLayout<128>::kSpillRowBytes : TcLayout<64>::kSpillRowBytes;
  return size_t(cluster_size - 1) * size_t(2 * BMH / cluster_size) * size_t(row_bytes);
}

// How many clusters of `cluster_size` CTAs of this kernel the current device can hold at once (0: such a
// cluster cannot be launched at all, e.g. on a reduced share of the SMs); -1 when that cannot be asked
// (no device).  Asked once per (device, head dimension, cluster size).
int attn_tc_max_clusters(int head_dim, int cluster_size) {
  static std::atomic<int> cache[DynSmemGrant::kDevices][2][4];
  static std::atomic<bool> init{false};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= DynSmemGrant::kDevices) { cudaGetLastError(); return -1; }
  if (!init.exchange(true))
    for (auto& d : cache) for (auto& h : d) for (auto& c : h) c.store(-2);
  const int hi = head_dim == 128 ? 0 : 1, ci = cluster_size == 8 ? 3 : cluster_size == 4 ? 2 : cluster_size == 2 ? 1 : 0;
  int have = cache[dev][hi][ci].load();
  if (have != -2 && have != -3) return have;           // (-3: another thread is filling the table; ask again below, harmless)
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = unsigned(cluster_size);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(cluster_size));
  cfg.blockDim = dim3(unsigned(kThreads));
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  cudaError_t e;
  if (head_dim == 128) {
    cfg.dynamicSmemBytes = TcLayout<128>::kTotal + 1024;
    static DynSmemGrant grant;
    e = grant.ensure(tree_attn_tc_kernel<128, false, false>, cfg.dynamicSmemBytes);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, tree_attn_tc_kernel<128, false, false>, &cfg);
  } else {
    cfg.dynamicSmemBytes = 120 * 1024;
    static DynSmemGrant grant;
    e = grant.ensure(tree_attn_tc_kernel<64, false, false>, cfg.dynamicSmemBytes);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, tree_attn_tc_kernel<64, false, false>, &cfg);
  }
  if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
  cache[dev][hi][ci].store(n);
  return n;
}

cudaError_t launch_attn_tc(int head_dim, int n_ctas, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                           const AttnParams& p, const WorkItem* host_items, cudaStream_t stream) {
  // host_items: the host copy of p.items (same layout); each CTA's first item travels as a kernel parameter
  FirstItems first;
  const size_t stride = p.queue != nullptr ? 1 : size_t(p.items_stride);
  for (int c = 0; c < kFirstItems; ++c) first.item[c] = c < n_ctas ? host_items[size_t(c) * stride] : WorkItem{};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;      // cluster plans: one cluster per split group
  attr[1].val.clusterDim.x = unsigned(p.cluster_size > 1 ? p.cluster_size : 1);
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(n_ctas));
  cfg.blockDim = dim3(unsigned(kThreads));
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = p.cluster_size > 1 ? 2 : 1;
  const bool dyn = p.queue != nullptr;
  cudaError_t le = cudaSuccess;
  if (head_dim == 128) {
    const size_t smem = TcLayout<128>::kTotal + 1024;
    if (p.tree_in_pages)
      le = dyn ? launch_one<128, true, true>(cfg, smem, mq, mk, mv, p, first) : launch_one<128, false, true>(cfg, smem, mq, mk, mv, p, first);
    else
      le = dyn ? launch_one<128, true, false>(cfg, smem, mq, mk, mv, p, first) : launch_one<128, false, false>(cfg, smem, mq, mk, mv, p, first);
  } else {
    // padded past half of an SM's shared memory: one CTA per SM, since each CTA takes all 512 TMEM columns
    const size_t smem = 120 * 1024;
    static_assert(TcLayout<64>::kTotal + 1024 <= 120 * 1024, "smem layout");
    if (p.tree_in_pages)
      le = dyn ? launch_one<64, true, true>(cfg, smem, mq, mk, mv, p, first) : launch_one<64, false, true>(cfg, smem, mq, mk, mv, p, first);
    else
      le = dyn ? launch_one<64, true, false>(cfg, smem, mq, mk, mv, p, first) : launch_one<64, false, false>(cfg, smem, mq, mk, mv, p, first);
  }
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace dyspec
