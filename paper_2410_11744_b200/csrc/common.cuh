// Shared device/host declarations of the tree-verify attention library (internal; not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <atomic>

#include "../../include/dyspec.h"

namespace dyspec {

constexpr int kDefaultSMs = 148;        // B200: 2 dies x 74 SMs (the scheduler asks the device; this is the fallback)
constexpr float kLog2e = 1.4426950408889634f;

// One verification request, device-side view.
struct ReqInfo {
  int64_t kv_row0;     // row of the request's token 0 in k_cache / v_cache
  int32_t prefix_len;  // L_r
  int32_t n_nodes;     // n_r
  int32_t node0;       // first query / output / mask row of the request
  int32_t pad;
};

// One unit of scheduled work: a tile of packed query rows of one (request, kv head) against a
// contiguous range of that group's key tiles.  Packed row p of a (request, kv head) pair is
// node p / g, query head kv_head * g + p % g.  Key tiles of a group: first the prefix tiles
// (tile t covers prefix keys [t*BN, min(L, (t+1)*BN))), then the tree tiles (tile u covers tree
// columns [u*BN, (u+1)*BN)).  The request's shape is repeated inside the item and CTA c's items sit
// at a fixed stride (items[c * stride + k], k < items[c * stride].n_in_cta), so a CTA reaches its
// work with one dependent global load instead of three.
struct WorkItem {
  int64_t kv_row0;     // row of the request's token 0 in k_cache / v_cache
  int32_t prefix_len;  // L_r
  int32_t n_nodes;     // n_r
  int32_t node0;       // first query / output / mask row of the request
  int32_t kv_head;
  int32_t row0;        // first packed row of the query tile (multiple of BM)
  int32_t tile_begin;  // key-tile range [tile_begin, tile_end) of the group's tile list
  int32_t tile_end;
  int32_t slot;        // index of the fp32 partial slot to write, or -1: write the final bf16 rows
  int32_t group;       // split-group id (arrival counter index) when slot >= 0
  int32_t n_splits;    // number of items the group was cut into
  int32_t slot0;       // first partial slot of the group (slots slot0 .. slot0 + n_splits - 1)
  int32_t n_in_cta;    // in the first item of a CTA: how many items the CTA owns
  int32_t req;         // request index
  int32_t merge_owners;  // cluster mode: bit k set = CTA k of the cluster merges a share of the rows (see attn_small.cu)
};
static_assert(sizeof(WorkItem) == 64, "WorkItem is one 64-byte record");

// The first work item of every CTA, passed to the small-tile kernel by value (kernel parameter space):
// a CTA then knows its first item without a global-memory round trip in front of its first loads.
constexpr int kFirstItems = 148;
struct FirstItems { WorkItem item[kFirstItems]; };

// Request list of a ragged mask-builder call without a plan, passed by value: request k of the launch
// owns nodes node0[k] .. node0[k + 1] - 1; first_req = index of the launch's first request in the batch
// (its status word).
constexpr int kMaskBatchMax = 768;
struct MaskBatch {
  int32_t node0[kMaskBatchMax + 1];
  int32_t first_req;
};

// A split query-tile group, for the combine step.
struct GroupInfo {
  int32_t req;
  int32_t kv_head;
  int32_t row0;
  int32_t slot0;       // first partial slot; the group's slots are slot0 .. slot0 + n_splits - 1
  int32_t n_splits;
  int32_t pad[3];
};

// Parameters common to the attention kernels.
struct AttnParams {
  const ReqInfo* reqs;
  const WorkItem* items;           // [n_ctas * items_stride]
  const GroupInfo* groups;         // split groups only
  const uint32_t* bits;            // ancestor bitmasks [sum n][W]
  const uint32_t* node_tiles;      // optional [sum n]: bit t = the node's row touches tree columns [64 t, 64 t + 64)
  __nv_bfloat16* out;              // [sum n][H_q][D]
  float* partial;                  // split-KV partials: slot s at partial + s * slot_floats
  int32_t* counters;               // two words per split group, in the caller's workspace, zero between calls:
                                   // [2 g] = halves of the group's items whose partial is written, [2 g + 1] = items that have merged their share
  int32_t merge_in_kernel;         // tensor-core regime: the items of a split group merge the group's rows themselves (no combine launch)
  int32_t* status;                 // may be null
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t group_size;              // g
  int32_t log2_g;
  int32_t words_per_row;           // W
  int32_t slot_floats;             // BM * (D + 2)
  float scale_log2e;               // scale * log2(e)
  int32_t items_stride;            // items per CTA slot in `items`
  int32_t cluster_size;            // > 1: one cluster per split group; partials are merged through distributed shared memory
  unsigned long long* trace;       // optional event trace (null in normal use): [0] = count, then entries
  int32_t trace_capacity;
  // Paged cache (null page_table = contiguous layout): prefix token t of request r lies at cache row
  // (page_table[r * pages_per_req + (t >> page_shift)] << page_shift) + (t & (page_size - 1)); the
  // request's tree rows start at its kv_row0.  The page size is a multiple of every key-tile size,
  // so a prefix tile never straddles two pages.
  const int32_t* page_table;
  int32_t pages_per_req;
  int32_t page_shift;
  // Paged cache with the tree rows INSIDE the paged sequence (node j = token L + j): key tiles then follow
  // the sequence, not the tree: the first L / BN tiles are full prefix tiles, tile L / BN + u covers tokens
  // [(L / BN + u) BN, ...), i.e. tree columns u BN - L % BN onwards (its leading L % BN keys, for u = 0, are
  // the prefix's last ones), and a row's mask slice for the tile is its bit row shifted by L % BN.
  int32_t tree_in_pages;
  // Shared work queue (null = every CTA has a fixed list): `items` then holds all n_items_total items in
  // queue order, CTA c starts with item c and takes further ones with an atomic add on queue[0];
  // queue[1] counts the CTAs that found the queue empty, and the last of them clears both words.
  int32_t* queue;
  int32_t n_items_total;
};

// Dynamic shared memory above 48 KB has to be granted per (kernel, device).  One of these per kernel
// remembers what each device of the process has been granted so far; safe to call from several
// host threads (the worst case is a repeated, idempotent grant).
struct DynSmemGrant {
  static constexpr int kDevices = 64;
  std::atomic<size_t> granted[kDevices];
  template <typename Kernel>
  cudaError_t ensure(Kernel kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return cudaSuccess;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool cached = dev >= 0 && dev < kDevices;
    if (cached && granted[dev].load(std::memory_order_acquire) >= bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes));
    if (e != cudaSuccess) return e;
    if (cached) granted[dev].store(bytes, std::memory_order_release);
    return cudaSuccess;
  }
};

// Key tiles of a (request, query tile) group, host and device: the tiles in front of the first one that
// needs the mask, and how far the tree's column 0 sits inside that one (0 unless the tree rows are
// part of the paged sequence).
__host__ __device__ inline int prefix_tile_count(int prefix_len, int bn, int tree_in_pages) {
  return tree_in_pages ? prefix_len / bn : (prefix_len + bn - 1) / bn;
}
__host__ __device__ inline int tree_tile_shift(int prefix_len, int bn, int tree_in_pages) {
  return tree_in_pages ? prefix_len % bn : 0;
}

#ifdef __CUDACC__
// First cache row of key tile t of a work item's group (tiles of BN keys: prefix tiles, then tree tiles).
__device__ __forceinline__ int64_t kv_tile_row(const AttnParams& p, const WorkItem& it, int t, int n_prefix_tiles, int BN) {
  if (t >= n_prefix_tiles && !p.tree_in_pages)
    return it.kv_row0 + (p.page_table ? 0 : int64_t(it.prefix_len)) + int64_t(t - n_prefix_tiles) * BN;
  const int64_t s = int64_t(t) * BN;
  if (!p.page_table) return it.kv_row0 + s;
  const int32_t page = __ldg(p.page_table + int64_t(it.req) * p.pages_per_req + (s >> p.page_shift));
  return (int64_t(page) << p.page_shift) + (s & ((int64_t(1) << p.page_shift) - 1));
}

// ------------------------------------------------------------------------------------------------
// PTX helpers (sm_100a).  Every wait is bounded: when it runs out the kernel records
// DYSPEC_ERR_TIMEOUT and carries on without waiting any more, so it always terminates.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// Non-blocking probe.  A try_wait that does not succeed at once suspends the thread for a
// hardware-defined time slice and is slow to notice the completion (~700 cycles measured on B200);
// polling with test_wait sees it within one probe latency (~180 cycles).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// Three probes whose round trips overlap: the answers come back together, about one probe latency
// after the first was issued (three mbar_test_wait calls in a row would take three latencies, since
// each consumes its predicate before the next is issued).  Bit k of the result = barrier k's phase done.
__device__ __forceinline__ uint32_t mbar_test_wait3(uint32_t bar0, uint32_t parity0, uint32_t bar1, uint32_t parity1,
                                                    uint32_t bar2, uint32_t parity2) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p0, p1, p2;\n\t.reg .u32 r0, r1, r2;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p0, [%1], %2;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p1, [%3], %4;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p2, [%5], %6;\n\t"
      "selp.u32 r0, 1, 0, p0;\n\tselp.u32 r1, 2, 0, p1;\n\tselp.u32 r2, 4, 0, p2;\n\t"
      "or.b32 r0, r0, r1;\n\tor.b32 %0, r0, r2;\n\t}"
      : "=r"(done)
      : "r"(bar0), "r"(parity0), "r"(bar1), "r"(parity1), "r"(bar2), "r"(parity2)
      : "memory");
  return done;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

constexpr uint64_t kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // 1 s per wait, then give up

// Bounded mbarrier wait.  `abort_flag` lives in shared memory: once any wait of the CTA ran out,
// later waits return at once.  Returns false when the wait did not complete.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  // fast path: spin on the non-blocking probe (lowest hand-off latency); ordinary waits end here
#pragma unroll 1
  for (int i = 0; i < 256; ++i)
    if (mbar_test_wait(bar, parity)) return true;
  if (*abort_flag) return false;
  const uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0xff) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        if (status) atomicCAS(status, 0, DYSPEC_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Bounded wait on a monotonically increasing shared-memory counter (release/acquire at CTA scope):
// a much shorter hand-off than an mbarrier when the waiter only needs "at least `target` arrivals".
__device__ __forceinline__ uint32_t ld_acquire_shared(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_shared_add(uint32_t addr, uint32_t v) {
  asm volatile("red.release.cta.shared::cta.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ bool counter_wait(uint32_t addr, uint32_t target, volatile int* abort_flag, int32_t* status) {
#pragma unroll 1
  for (int i = 0; i < 64; ++i)
    if (int32_t(ld_acquire_shared(addr) - target) >= 0) return true;
  if (*abort_flag) return false;
  const uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  while (int32_t(ld_acquire_shared(addr) - target) < 0) {
    if ((++spins & 0x3ff) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        if (status) atomicCAS(status, 0, DYSPEC_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// start while its predecessor in the stream is still running; it must call grid_dependency_wait()
// before it reads anything the predecessor writes or writes anything the predecessor (or earlier
// kernels) may still read.  The predecessor lets dependents start early with trigger_dependents().
// Loads of data that a preceding kernel of the stream wrote (mask words, tile sets), for use after
// grid_dependency_wait(): ordinary coherent loads that the compiler may not move (a read-only __ldg
// could legally be hoisted above the wait and would then see the buffer's old contents).
__device__ __forceinline__ uint4 ld_after_dependency_v4(const void* ptr) {
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr) : "memory");
  return v;
}
__device__ __forceinline__ uint2 ld_after_dependency_v2(const void* ptr) {
  uint2 v;
  asm volatile("ld.global.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(ptr) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ld_after_dependency_u32(const void* ptr) {
  uint32_t v;
  asm volatile("ld.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}
// Cross-CTA hand-off through global memory (split-KV merge inside the attention kernel).
__device__ __forceinline__ void red_release_gpu_add(int32_t* addr, int32_t v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ int32_t ld_acquire_gpu(const int32_t* addr) {
  int32_t v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
  return v;
}
// Data another SM wrote during this launch: read from L2 (this SM's L1 may hold a stale line).
__device__ __forceinline__ float4 ld_cg_f32x4(const float* ptr) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_cg_f32x2(const float* ptr) {
  float2 v;
  asm volatile("ld.global.cg.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(ptr) : "memory");
  return v;
}
__device__ __forceinline__ float ld_cg_f32(const float* ptr) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(ptr) : "memory");
  return v;
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void trigger_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Thread-block cluster helpers (distributed shared memory; every copy has exactly one destination CTA).
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of the cluster barrier, for a hand-shake whose latency should stay hidden: every
// thread arrives early and waits only when it needs the peers to have arrived.
// (relaxed: what the peers must see -- the initialised mbarriers -- was published by fence.mbarrier_init)
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// Asynchronous copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) from this CTA's
// shared memory into a peer CTA's; the peer's mbarrier receives the byte count when the data has
// landed.  dst and bar are shared::cluster addresses (see map_to_cta).  One destination CTA.
__device__ __forceinline__ void dsmem_push(uint32_t dst_cluster_addr, uint32_t src_local_addr, uint32_t bytes,
                                           uint32_t bar_cluster_addr) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_cluster_addr), "r"(src_local_addr), "r"(bytes), "r"(bar_cluster_addr) : "memory");
}
// Until this returns, the source of this thread's dsmem_push calls must stay intact.
__device__ __forceinline__ void dsmem_push_wait_source_read() {
  asm volatile("cp.async.bulk.commit_group;\n\tcp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(cta_rank));
  return r;
}
// Loads and stores of this CTA's own shared memory by 32-bit shared-window address.
__device__ __forceinline__ float ld_shared_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_shared_f32x2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_shared_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_shared_f32(uint32_t addr, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ float ld_dsmem_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_dsmem_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_dsmem_f32x2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}

// TMA: 3-D tiled load global -> shared, completion on an mbarrier (destination: this CTA only).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Optional in-kernel event trace (CTA 0 only; libraries built with -DDYSPEC_TRACE).  Each traced thread owns one region of the buffer
// (region = role) and keeps its own cursor in a register, so an event costs one plain store:
// entry = tag << 44 | low 44 bits of the SM clock.
struct TraceCursor {
  unsigned long long* at;
  unsigned long long* end;
};
__device__ __forceinline__ TraceCursor trace_open(const AttnParams& p, int role, int n_roles) {
  TraceCursor c{nullptr, nullptr};
  if (p.trace != nullptr && blockIdx.x == 0) {
    const int per = (p.trace_capacity > 4096 ? p.trace_capacity - 2048 : p.trace_capacity) / n_roles;
    c.at = p.trace + size_t(role) * per;
    c.end = c.at + per;
  }
  return c;
}
__device__ __forceinline__ void trace_event(TraceCursor& c, uint32_t tag) {
#ifdef DYSPEC_TRACE
  if (c.at != nullptr && c.at < c.end)
    *c.at++ = ((unsigned long long)tag << 44) | ((unsigned long long)clock64() & ((1ull << 44) - 1));
#else
  // Compiled out of the ordinary library: even the never-taken checks (a handful per key tile in the MMA-
  // issuing and softmax loops) cost the tensor-core kernel 8 - 10 % (config 4: 38.0 -> 35.0 us).
  (void)c; (void)tag;
#endif
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
#endif  // __CUDACC__

}  // namespace dyspec
