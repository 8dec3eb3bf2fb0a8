// C ABI of the tree-verify attention library: argument checks, the host-side ragged scheduler
// (plan), TMA tensor-map encoding and kernel launches.  See include/dyspec.h for the contract.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <tuple>
#include <vector>

#include "common.cuh"

namespace dyspec {
// kernels (defined in the other translation units)
cudaError_t launch_build_tree_mask(const int32_t* parents, const ReqInfo* reqs, int n_req, int single_n, int max_n,
                                   uint32_t* bits, int32_t* depths, uint32_t* node_tiles, int W, int32_t* status,
                                   cudaStream_t stream);
cudaError_t launch_build_tree_mask_batch(const int32_t* parents, const MaskBatch& batch, int n_req, int max_n, uint32_t* bits,
                                         int32_t* depths, int W, int32_t* status, cudaStream_t stream);
cudaError_t launch_dfs_reorder(const int32_t* parents, const ReqInfo* reqs, int n_req, int single_n, int max_n,
                               int32_t* order, int32_t* new_of_old, int32_t* new_parents, int32_t* status,
                               cudaStream_t stream);
cudaError_t launch_mask_block_count(const uint32_t* bits, int n, int W, int block, unsigned long long* count,
                                    cudaStream_t stream);
cudaError_t launch_verify_tree(const int32_t* parents, const int32_t* tokens, const float* draft_probs,
                               const float* target_probs, const float* accept_u, const float* sample_u,
                               const int32_t* node_offsets, int n_req, int max_nodes, int vocab, int bonus_at_leaf,
                               int32_t* out_tokens, int32_t* out_nodes, int32_t* out_count, int max_out, int32_t* status,
                               cudaStream_t stream);
cudaError_t launch_build_tree_greedy(const float* draft_table, int n_rows, int vocab, const float* uniforms, int n_uniforms,
                                     const int32_t* root_row, int n_req, int m, int32_t* parents, int32_t* tokens,
                                     float* values, float* child_values, int32_t* rows, int32_t* n_nodes,
                                     cudaStream_t stream);
cudaError_t launch_build_tree_threshold(const float* draft_table, int n_rows, int vocab, const float* uniforms,
                                        int n_uniforms, const int32_t* root_row, int n_req, float threshold, int max_nodes,
                                        int32_t* parents, int32_t* tokens, float* values, float* child_values, int32_t* rows,
                                        int32_t* n_nodes, cudaStream_t stream);
cudaError_t launch_compact_kv_paged(void* k_cache, void* v_cache, const int64_t* tree_row_offset, const int32_t* page_table,
                                    int pages_per_req, int page_shift, const int32_t* prefix_len,
                                    const int32_t* accepted_nodes, const int32_t* n_accepted, int n_req, int max_out,
                                    int row_bytes, int keep_root, int32_t* new_prefix_len, int32_t* status,
                                    cudaStream_t stream);
cudaError_t launch_compact_kv(void* k_cache, void* v_cache, const int64_t* kv_row_offset, const int32_t* prefix_len,
                              const int32_t* accepted_nodes, const int32_t* n_accepted, int n_req, int max_out,
                              int row_bytes, int keep_root, int32_t* new_prefix_len, cudaStream_t stream);
cudaError_t launch_attn_small(int head_dim, int n_ctas, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                            const AttnParams& p, const WorkItem* host_items, cudaStream_t stream);
cudaError_t launch_combine(int head_dim, int bm, int n_split_groups, const AttnParams& p, cudaStream_t stream);
int attn_tc_max_clusters(int head_dim, int cluster_size);
int attn_small_max_clusters(int head_dim, int cluster_size);
size_t attn_tc_cluster_workspace_per_cta(int head_dim, int cluster_size);
cudaError_t launch_attn_tc(int head_dim, int n_ctas, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                           const AttnParams& p, const WorkItem* host_items, cudaStream_t stream);
}  // namespace dyspec

using namespace dyspec;

namespace {

// Testing knobs and the developer trace (dyspec_set_tuning, dyspec_set_trace).  Process-wide, but never
// read while they change: every reader takes a copy under the mutex, and a plan keeps the copy it was
// created with, so concurrent plan creation and attention calls stay well defined.
struct Tuning {
  int force_regime = -1;
  int force_ctas = 0;
  int item_cost = 0;       // scheduler experiment knob (0 = default)
  int combine_mode = 2;    // 0 separate combine kernel; 2 merge on chip (clusters) / in the attention kernel when the plan
                           // allows; 1 as 2 but the tensor-core regime never uses clusters (merge through the workspace)
  int whole_groups = 0;    // 0: the scheduler's cost model chooses; 1: never deal whole groups; 2: always
  unsigned long long* trace = nullptr;   // device buffer for the optional kernel event trace
  int trace_capacity = 0;
};
Tuning g_tuning;
std::mutex g_tuning_mutex;
Tuning current_tuning() {
  std::lock_guard<std::mutex> lock(g_tuning_mutex);
  return g_tuning;
}

// SMs of the current device (the scheduler balances over them); B200's count where no device can be asked
// (the host-only dry run on a machine without a GPU).
int device_sm_count() {
  static std::mutex m;
  static int cached[64] = {};
  int dev = -1, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) { cudaGetLastError(); return kDefaultSMs; }
  std::lock_guard<std::mutex> lock(m);
  if (dev < 64 && cached[dev] > 0) return cached[dev];
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { cudaGetLastError(); return kDefaultSMs; }
  if (dev < 64) cached[dev] = n;
  return n;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

// bf16 tensor [rows][heads][D] viewed as (D, heads, rows); box = (64, box_heads, box_rows), 128-byte swizzle.
bool encode_map(CUtensorMap* map, const void* base, int64_t rows, int heads, int D, int box_heads, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (rows <= 0) rows = 1;
  const cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(heads), cuuint64_t(rows)};
  const cuuint64_t strides[2] = {cuuint64_t(D) * 2, cuuint64_t(heads) * D * 2};
  const cuuint32_t box[3] = {64u, cuuint32_t(box_heads), cuuint32_t(box_rows)};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// DYSPEC_ERR_CUDA, with the runtime's own message on stderr when DYSPEC_DEBUG is set in the environment.
int cuda_failed(cudaError_t e, const char* where) {
  if (std::getenv("DYSPEC_DEBUG")) std::fprintf(stderr, "dyspec: %s: %s\n", where, cudaGetErrorString(e));
  return DYSPEC_ERR_CUDA;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Small host tables -> device memory, stream-ordered, WITHOUT a host pointer that has to outlive the
// call: the bytes travel in the kernel's parameter space (copied when the launch is enqueued), one
// launch per 3584-byte piece.  A cudaMemcpyAsync from pageable memory would stage through the driver
// (and may synchronise the stream); this needs neither pinned memory nor a staging buffer.
struct TablePiece { uint4 v[224]; };
__global__ void __launch_bounds__(224) write_table_kernel(uint4* dst, const __grid_constant__ TablePiece piece, int n_vec) {
  if (int(threadIdx.x) < n_vec) dst[threadIdx.x] = piece.v[threadIdx.x];
}
// dst: 16-byte aligned device memory with room for `bytes` rounded up to 16.
cudaError_t write_table(void* dst, const void* src, size_t bytes, cudaStream_t stream) {
  const unsigned char* from = static_cast<const unsigned char*>(src);
  unsigned char* to = static_cast<unsigned char*>(dst);
  while (bytes > 0) {
    TablePiece piece;
    const size_t take = std::min(bytes, sizeof(piece.v));
    memset(&piece, 0, sizeof(piece));
    memcpy(piece.v, from, take);
    write_table_kernel<<<1, 224, 0, stream>>>(reinterpret_cast<uint4*>(to), piece, int((take + 15) / 16));
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
    from += take; to += take; bytes -= take;
  }
  return cudaSuccess;
}

}  // namespace

struct dyspec_plan {
  int hq = 0, hkv = 0, d = 0, g = 1, log2g = 0, W = 0;
  float scale = 0.f;
  int n_req = 0;
  int64_t kv_total_rows = 0;
  int page_size = 0;                    // > 0: paged cache (prefix through a page table, kv_row0 = first tree row)
  bool tree_in_pages = false;           // paged cache whose tree rows are tokens L .. L + n - 1 of the paged sequence
  int64_t total_nodes = 0;
  int max_nodes = 0;
  int regime = 0, bm = 64, bn = 64;
  int n_sms = kDefaultSMs;              // SMs the scheduler balances over (those of the device current at creation)
  Tuning tune;                          // the testing knobs as they were when the plan was created
  std::vector<ReqInfo> reqs;
  std::vector<WorkItem> items;          // compact list, CTA by CTA
  std::vector<WorkItem> items_strided;  // device layout: CTA c's items at [c * items_stride, ...)
  int items_stride = 1;
  int cluster = 1;                      // > 1: one thread-block cluster of this size per split group
  std::vector<int32_t> cta_begin;
  std::vector<GroupInfo> split_groups;
  int n_ctas = 0, n_slots = 0, max_splits = 1;
  int64_t total_tiles = 0, n_groups = 0;
  // device copies (one allocation)
  void* d_blob = nullptr;
  int device = -1;                      // the device the copies live on (the one current at creation)
  ReqInfo* d_reqs = nullptr;
  WorkItem* d_items = nullptr;
  GroupInfo* d_groups = nullptr;
  int32_t* d_counters = nullptr;
  bool dynamic = false;                 // whole groups taken from a shared queue (longest first) instead of fixed lists
  bool allow_queue = true;              // false: fixed lists only (callers that cannot provide zeroed queue words)
  size_t queue_offset = 0;              // dynamic plans: byte offset of the two queue words inside the caller's workspace
  size_t counters_offset = 0;           // plans with split groups: byte offset of the groups' counter pairs in the workspace
  bool merge_in_kernel = false;         // tensor-core regime: split groups are merged by their own items, no combine launch
  int cluster_fit[9] = {-1, -1, -1, -1, -1, -1, -1, -1, -1};   // clusters of C CTAs of the regime's kernel the device holds at once (-1: not known)
  std::vector<WorkItem> items_queue;    // dynamic plans: all items in queue order
  size_t workspace_bytes = 0;
};

namespace {

// Host scheduler: cut the (request, kv head, query tile) groups' key-tile lists into work items
// and deal them to CTAs so that every CTA gets about the same number of key tiles (plus a fixed
// per-item cost for the Q load and the epilogue).  A group that ends up in several items is a
// split-KV group: its items write fp32 partials that the combine step merges.
void schedule(dyspec_plan& pl) {
  const int bm = pl.bm, bn = pl.bn, g = pl.g;
  const int nodes_per_tile = bm / g;
  struct Group { int req, kvh, row0, tiles; };
  std::vector<Group> groups;
  int64_t total_tiles = 0;
  for (int r = 0; r < pl.n_req; ++r) {
    const ReqInfo& rq = pl.reqs[r];
    if (rq.n_nodes == 0) continue;
    // (tree rows inside the paged sequence: the tiles follow the sequence, and the tree's column 0 sits
    //  L % bn keys inside the first tile that needs the mask)
    const int prefix_tiles = prefix_tile_count(rq.prefix_len, bn, pl.tree_in_pages);
    const int shift = tree_tile_shift(rq.prefix_len, bn, pl.tree_in_pages);
    const int q_tiles = (rq.n_nodes + nodes_per_tile - 1) / nodes_per_tile;
    for (int kvh = 0; kvh < pl.hkv; ++kvh)
      for (int qt = 0; qt < q_tiles; ++qt) {
        // parents[i] < i: a node only sees tree columns <= its own index, so tree tiles past the
        // tile's last node are never needed.
        const int last_node = std::min(rq.n_nodes, (qt + 1) * nodes_per_tile);
        const int tiles = prefix_tiles + (shift + last_node + bn - 1) / bn;
        groups.push_back({r, kvh, qt * bm, tiles});
        total_tiles += tiles;
      }
  }
  pl.total_tiles = total_tiles;
  pl.n_groups = int64_t(groups.size());
  pl.items.clear();
  pl.cta_begin.clear();
  pl.split_groups.clear();
  pl.n_slots = 0;
  pl.max_splits = 1;
  pl.items_strided.clear();
  pl.items_stride = 1;
  pl.dynamic = false;
  pl.items_queue.clear();
  if (groups.empty()) { pl.n_ctas = 0; pl.cta_begin.push_back(0); return; }

  // Cluster mode (warp-level regime): when every group can be cut into the same number C of pieces
  // and all pieces fit in one wave, launch one cluster of C CTAs per group; the pieces are merged
  // through distributed shared memory instead of a round trip through global memory.
  pl.cluster = 1;
  const Tuning& tn = pl.tune;
  const int kNumSMs = pl.n_sms;
  if (pl.regime == 0 && tn.combine_mode == 2 && tn.force_ctas <= 0) {
    int max_tiles = 0;
    for (const Group& gr : groups) max_tiles = std::max(max_tiles, gr.tiles);
    const double mean_tiles = double(total_tiles) / double(groups.size());
    for (int C : {8, 4, 2}) {
      if (int64_t(groups.size()) * C > kNumSMs) continue;
      if (pl.cluster_fit[C] >= 0 && int64_t(groups.size()) > pl.cluster_fit[C]) continue;   // all clusters at once, or none
      if (mean_tiles / C < 2.0 || double(max_tiles) > 1.3 * mean_tiles) continue;
      bool ok = true;
      for (const Group& gr : groups) ok = ok && gr.tiles >= C;
      if (!ok) continue;
      pl.cluster = C;
      break;
    }
  }
  if (pl.cluster > 1) {
    const int C = pl.cluster;
    pl.cta_begin.push_back(0);
    for (size_t gi = 0; gi < groups.size(); ++gi) {
      const Group& gr = groups[gi];
      const ReqInfo& rq = pl.reqs[size_t(gr.req)];
      // Who merges: with equal pieces every CTA takes BM / C rows.  With unequal pieces the CTAs with
      // the larger pieces finish last; they only hand their partial rows over, and the C / 2 CTAs with
      // the smallest pieces (lowest ranks on ties) share the rows, so the merge work is done -- all
      // but folding in the last arrival -- before the slowest CTA gets there.
      int owners = (1 << C) - 1;
      {
        int lo = gr.tiles, hi = 0;
        for (int c = 0; c < C; ++c) {
          const int sz = int(int64_t(gr.tiles) * (c + 1) / C) - int(int64_t(gr.tiles) * c / C);
          lo = std::min(lo, sz); hi = std::max(hi, sz);
        }
        if (hi != lo) {
          owners = 0;
          int taken = 0;
          for (int want = lo; want <= hi && taken < C / 2; ++want)
            for (int c = 0; c < C && taken < C / 2; ++c) {
              const int sz = int(int64_t(gr.tiles) * (c + 1) / C) - int(int64_t(gr.tiles) * c / C);
              if (sz == want) { owners |= 1 << c; ++taken; }
            }
        }
      }
      for (int c = 0; c < C; ++c) {
        WorkItem it{};
        it.kv_row0 = rq.kv_row0; it.prefix_len = rq.prefix_len; it.n_nodes = rq.n_nodes; it.node0 = rq.node0;
        it.req = gr.req; it.kv_head = gr.kvh; it.row0 = gr.row0;
        it.tile_begin = int(int64_t(gr.tiles) * c / C);
        it.tile_end = int(int64_t(gr.tiles) * (c + 1) / C);
        it.slot = -1; it.slot0 = -1; it.group = int(gi); it.n_splits = C; it.n_in_cta = 1;
        it.merge_owners = owners;
        pl.items.push_back(it);
        pl.cta_begin.push_back(int32_t(pl.items.size()));
      }
    }
    pl.max_splits = C;
    pl.n_ctas = int(pl.items.size());
    pl.items_stride = 1;
    pl.items_strided = pl.items;
    return;
  }

  const int ctas_per_sm = 1;   // one wave: every CTA is resident from the start and owns its SM's load queue
  int max_ctas = tn.force_ctas > 0 ? tn.force_ctas : kNumSMs * ctas_per_sm;
  // fixed per-item overhead (Q load, pipeline fill, epilogue), in key tiles: measured ~1 tile of 64 keys in
  // regime 0 and ~3 tiles of 128 keys in regime 1
  const int item_cost = tn.item_cost > 0 ? tn.item_cost : (pl.regime == 0 ? 1 : 3);
  const int min_tiles = pl.regime == 0 ? 2 : 2;          // smallest piece worth a split
  const int64_t total_cost = total_tiles + int64_t(groups.size()) * item_cost;
  int64_t target = (total_cost + max_ctas - 1) / max_ctas;
  if (target < item_cost + min_tiles) target = item_cost + min_tiles;

  // Deal the tiles out with a per-CTA budget of `target`; a budget that leaves a CTA too little
  // room for a useful piece moves on to the next CTA, so the count can overshoot: grow the budget
  // until the work fits in max_ctas (one wave).
  for (int attempt = 0; attempt < 64; ++attempt) {
  pl.items.clear();
  pl.cta_begin.clear();
  pl.split_groups.clear();
  pl.n_slots = 0;
  pl.max_splits = 1;
  int64_t used = 0;
  pl.cta_begin.push_back(0);
  for (size_t gi = 0; gi < groups.size(); ++gi) {
    const Group& gr = groups[gi];
    const size_t first_item = pl.items.size();
    int begin = 0;
    while (begin < gr.tiles) {
      int64_t room = target - used;
      if (room < item_cost + min_tiles && used > 0) {
        pl.cta_begin.push_back(int32_t(pl.items.size()));
        used = 0;
        room = target;
      }
      int take = int(std::min<int64_t>(gr.tiles - begin, room - item_cost));
      const int rem = gr.tiles - begin - take;
      if (rem > 0 && rem < min_tiles) take = gr.tiles - begin;
      WorkItem it{};
      const ReqInfo& rq = pl.reqs[size_t(gr.req)];
      it.kv_row0 = rq.kv_row0; it.prefix_len = rq.prefix_len; it.n_nodes = rq.n_nodes; it.node0 = rq.node0;
      it.slot0 = -1; it.n_in_cta = 0;
      it.req = gr.req; it.kv_head = gr.kvh; it.row0 = gr.row0;
      it.tile_begin = begin; it.tile_end = begin + take;
      it.slot = -1; it.group = int(gi); it.n_splits = 1;
      pl.items.push_back(it);
      used += take + item_cost;
      begin += take;
    }
    const int n_splits = int(pl.items.size() - first_item);
    if (n_splits > 1) {
      GroupInfo info{};
      info.req = gr.req; info.kv_head = gr.kvh; info.row0 = gr.row0;
      info.slot0 = pl.n_slots; info.n_splits = n_splits;
      for (int s = 0; s < n_splits; ++s) {
        pl.items[first_item + s].slot = pl.n_slots + s;
        pl.items[first_item + s].slot0 = pl.n_slots;
        pl.items[first_item + s].n_splits = n_splits;
        pl.items[first_item + s].group = int(pl.split_groups.size());
      }
      pl.n_slots += n_splits;
      pl.max_splits = std::max(pl.max_splits, n_splits);
      pl.split_groups.push_back(info);
    }
  }
  pl.cta_begin.push_back(int32_t(pl.items.size()));
  pl.n_ctas = int(pl.cta_begin.size()) - 1;
  if (pl.n_ctas <= max_ctas) break;
  target += std::max<int64_t>(1, target / 64);
  }
  // The alternative without any split: whole groups dealt to the CTAs, largest first, each to the CTA
  // with the least work so far.  No partials and no combine launch, but the longest group bounds the
  // makespan.  Costs in key tiles: every item item_cost; an item that writes a partial one more tile
  // (fp32 rows instead of bf16); the combine launch behind the main kernel three (regime 1: 128-key
  // tiles of ~2 us) or four (regime 0) -- measured on the Llama2-70B shape, where the budgeted plan
  // (136 CTAs, 32 split groups) took 53.5 us and whole groups on 128 CTAs 48.1 us.
  if (tn.whole_groups != 1 && (tn.force_ctas <= 0 || tn.whole_groups == 2)) {
    // (tensor-core regime with the merge inside the kernel: no combine launch; writing the fp32 partial,
    //  publishing it and merging a share of the rows cost a split item about four tiles: 7 us measured)
    const bool in_kernel = pl.regime == 1 && tn.combine_mode != 0;
    const int partial_cost = in_kernel ? 4 : 1, combine_cost = in_kernel ? 0 : (pl.regime == 0 ? 4 : 3);
    int64_t cost_split = 0;
    for (int c = 0; c < pl.n_ctas; ++c) {
      int64_t load = 0;
      for (int k = pl.cta_begin[size_t(c)]; k < pl.cta_begin[size_t(c) + 1]; ++k) {
        const WorkItem& it = pl.items[size_t(k)];
        load += (it.tile_end - it.tile_begin) + item_cost + (it.slot >= 0 ? partial_cost : 0);
      }
      cost_split = std::max(cost_split, load);
    }
    if (!pl.split_groups.empty()) cost_split += combine_cost;
    const int n_bins = int(std::min<int64_t>(int64_t(groups.size()), max_ctas));
    std::vector<size_t> order(groups.size());
    for (size_t i = 0; i < order.size(); ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](size_t a, size_t b) { return groups[a].tiles > groups[b].tiles; });
    std::vector<int64_t> load(size_t(n_bins), 0);
    std::vector<std::vector<size_t>> bins{size_t(n_bins)};
    for (size_t gi : order) {
      size_t best = 0;
      for (size_t b = 1; b < load.size(); ++b)
        if (load[b] < load[best]) best = b;
      load[best] += groups[gi].tiles + item_cost;
      bins[best].push_back(gi);
    }
    const int64_t cost_whole = *std::max_element(load.begin(), load.end());
    if (!pl.split_groups.empty() && (cost_whole <= cost_split || tn.whole_groups == 2)) {
      pl.items.clear();
      pl.cta_begin.clear();
      pl.split_groups.clear();
      pl.n_slots = 0;
      pl.max_splits = 1;
      pl.cta_begin.push_back(0);
      for (const std::vector<size_t>& bin : bins) {
        for (size_t gi : bin) {
          const Group& gr = groups[gi];
          const ReqInfo& rq = pl.reqs[size_t(gr.req)];
          WorkItem it{};
          it.kv_row0 = rq.kv_row0; it.prefix_len = rq.prefix_len; it.n_nodes = rq.n_nodes; it.node0 = rq.node0;
          it.slot0 = -1; it.n_in_cta = 0;
          it.req = gr.req; it.kv_head = gr.kvh; it.row0 = gr.row0;
          it.tile_begin = 0; it.tile_end = gr.tiles;
          it.slot = -1; it.group = int(gi); it.n_splits = 1;
          pl.items.push_back(it);
        }
        pl.cta_begin.push_back(int32_t(pl.items.size()));
      }
      pl.n_ctas = n_bins;
      // More groups than CTAs (tensor-core regime): the fixed lists above are only the nominal plan.
      // On the device the CTAs take the groups from one queue, longest first (CTA c starts with the
      // c-th longest), so that what the cost model cannot see -- tree tiles skipped by the tile sets,
      // cache misses of one request's long prefix -- does not leave some CTAs working while others idle.
      if (pl.allow_queue && pl.regime == 1 && int64_t(groups.size()) > n_bins) {
        pl.dynamic = true;
        for (size_t gi : order) {
          const Group& gr = groups[gi];
          const ReqInfo& rq = pl.reqs[size_t(gr.req)];
          WorkItem it{};
          it.kv_row0 = rq.kv_row0; it.prefix_len = rq.prefix_len; it.n_nodes = rq.n_nodes; it.node0 = rq.node0;
          it.slot0 = -1; it.n_in_cta = 1;
          it.req = gr.req; it.kv_head = gr.kvh; it.row0 = gr.row0;
          it.tile_begin = 0; it.tile_end = gr.tiles;
          it.slot = -1; it.group = int(gi); it.n_splits = 1;
          pl.items_queue.push_back(it);
        }
      }
    }
  }

  // Few long groups (tensor-core regime, merge inside the kernel): cut every group into pieces of equal
  // length, ONE piece per CTA, as many pieces as there are SMs to take them.  Against the budgeted plan
  // this avoids CTAs with two split items (each pays the start-up and the partial epilogue again: on the
  // Llama2-7B shape with a 4096-key prefix those CTAs finished 8 us after the others).
  if (pl.regime == 1 && tn.combine_mode != 0 && tn.force_ctas <= 0 && tn.whole_groups != 2 && !pl.dynamic &&
      int64_t(groups.size()) * 2 <= max_ctas) {
    const int item_cost_ = item_cost, partial_cost = 4;
    int64_t cost_now = 0;
    for (int c = 0; c < pl.n_ctas; ++c) {
      int64_t load = 0;
      for (int k = pl.cta_begin[size_t(c)]; k < pl.cta_begin[size_t(c) + 1]; ++k) {
        const WorkItem& it = pl.items[size_t(k)];
        load += (it.tile_end - it.tile_begin) + item_cost_ + (it.slot >= 0 ? partial_cost : 0);
      }
      cost_now = std::max(cost_now, load);
    }
    std::vector<int> pieces(groups.size(), std::max(1, int(max_ctas / int64_t(groups.size()))));
    int used_ctas = 0;
    for (size_t gi = 0; gi < groups.size(); ++gi) {
      pieces[gi] = std::min(pieces[gi], std::max(1, groups[gi].tiles / 2));     // a piece has at least two tiles
      used_ctas += pieces[gi];
    }
    auto piece_len = [&](size_t gi) { return (groups[gi].tiles + pieces[gi] - 1) / pieces[gi]; };
    while (used_ctas < max_ctas) {            // the spare CTAs go to the groups whose pieces are longest
      size_t best = 0;
      for (size_t gi = 1; gi < groups.size(); ++gi)
        if (piece_len(gi) > piece_len(best)) best = gi;
      if (pieces[best] + 1 > groups[best].tiles / 2) break;
      ++pieces[best];
      ++used_ctas;
    }
    int64_t cost_even = 0;
    for (size_t gi = 0; gi < groups.size(); ++gi)
      cost_even = std::max<int64_t>(cost_even, piece_len(gi) + item_cost_ + (pieces[gi] > 1 ? partial_cost : 0));
    if (cost_even < cost_now) {
      pl.items.clear();
      pl.cta_begin.clear();
      pl.split_groups.clear();
      pl.n_slots = 0;
      pl.max_splits = 1;
      pl.cta_begin.push_back(0);
      for (size_t gi = 0; gi < groups.size(); ++gi) {
        const Group& gr = groups[gi];
        const ReqInfo& rq = pl.reqs[size_t(gr.req)];
        const int C = pieces[gi];
        for (int c = 0; c < C; ++c) {
          WorkItem it{};
          it.kv_row0 = rq.kv_row0; it.prefix_len = rq.prefix_len; it.n_nodes = rq.n_nodes; it.node0 = rq.node0;
          it.req = gr.req; it.kv_head = gr.kvh; it.row0 = gr.row0;
          it.tile_begin = int(int64_t(gr.tiles) * c / C);
          it.tile_end = int(int64_t(gr.tiles) * (c + 1) / C);
          it.n_in_cta = 0;
          if (C > 1) {
            it.slot = pl.n_slots + c; it.slot0 = pl.n_slots; it.n_splits = C; it.group = int(pl.split_groups.size());
          } else {
            it.slot = -1; it.slot0 = -1; it.n_splits = 1; it.group = int(gi);
          }
          pl.items.push_back(it);
          pl.cta_begin.push_back(int32_t(pl.items.size()));
        }
        if (C > 1) {
          GroupInfo info{};
          info.req = gr.req; info.kv_head = gr.kvh; info.row0 = gr.row0; info.slot0 = pl.n_slots; info.n_splits = C;
          pl.n_slots += C;
          pl.max_splits = std::max(pl.max_splits, C);
          pl.split_groups.push_back(info);
        }
      }
      pl.n_ctas = int(pl.items.size());
    }
    // The same idea with one thread-block cluster per group (C pieces each, C the same for all groups): the
    // pieces' partials then stay in shared memory (each CTA fetches its share of the rows from its peers),
    // which costs a piece about one tile instead of four (the fp32 partials of all CTAs at once go through
    // L2 at its bandwidth, twice).  Needs groups of similar length and at least two tiles per piece.
    if (tn.combine_mode == 2) {
      int max_tiles = 0, min_tiles_g = INT32_MAX;
      for (const Group& gr : groups) { max_tiles = std::max(max_tiles, gr.tiles); min_tiles_g = std::min(min_tiles_g, gr.tiles); }
      int64_t cost_plan = 0;                             // of the plan chosen so far
      for (int c = 0; c < pl.n_ctas; ++c) {
        int64_t load = 0;
        for (int k = pl.cta_begin[size_t(c)]; k < pl.cta_begin[size_t(c) + 1]; ++k) {
          const WorkItem& it = pl.items[size_t(k)];
          load += (it.tile_end - it.tile_begin) + item_cost_ + (it.slot >= 0 ? partial_cost : 0);
        }
        cost_plan = std::max(cost_plan, load);
      }
      int best_c = 0;
      int64_t best_cost = cost_plan;
      for (int C : {8, 4, 2}) {
        if (int64_t(groups.size()) * C > max_ctas || min_tiles_g < 2 * C) continue;
        // all clusters at once (the SMs of a cluster come from one GPC, so fewer fit than SMs / C): the ones
        // left over would run as a second wave
        if (pl.cluster_fit[C] >= 0 && int64_t(groups.size()) > pl.cluster_fit[C]) continue;
        const int64_t cost = (max_tiles + C - 1) / C + item_cost_ + 1;
        if (cost < best_cost) { best_cost = cost; best_c = C; }
      }
      if (best_c > 0) {
        const int C = best_c;
        pl.cluster = C;
        pl.items.clear();
        pl.cta_begin.clear();
        pl.split_groups.clear();
        pl.n_slots = 0;
        pl.cta_begin.push_back(0);
        for (size_t gi = 0; gi < groups.size(); ++gi) {
          const Group& gr = groups[gi];
          const ReqInfo& rq = pl.reqs[size_t(gr.req)];
          for (int c = 0; c < C; ++c) {
            WorkItem it{};
            it.kv_row0 = rq.kv_row0; it.prefix_len = rq.prefix_len; it.n_nodes = rq.n_nodes; it.node0 = rq.node0;
            it.req = gr.req; it.kv_head = gr.kvh; it.row0 = gr.row0;
            it.tile_begin = int(int64_t(gr.tiles) * c / C);
            it.tile_end = int(int64_t(gr.tiles) * (c + 1) / C);
            it.slot = -1; it.slot0 = -1; it.group = int(gi); it.n_splits = C; it.n_in_cta = 1;
            pl.items.push_back(it);
            pl.cta_begin.push_back(int32_t(pl.items.size()));
          }
        }
        pl.max_splits = C;
        pl.n_ctas = int(pl.items.size());
      }
    }
  }

  if (pl.dynamic) {                     // device layout: the queue itself
    pl.items_stride = 1;
    pl.items_strided = pl.items_queue;
    return;
  }
  // Order of a CTA's items.  Items are independent, and a kernel waits for the preceding kernels of the
  // stream only in front of an item's first tree tile or, for a piece without tree tiles, in front of its
  // partial write.  So the items that can run longest without that wait go first: in a chain of calls a
  // CTA then starts on work that does not depend on the previous call while that call is still draining.
  {
    const int bn = pl.bn;
    auto ungated_tiles = [&](const WorkItem& it) {
      const int npt = prefix_tile_count(it.prefix_len, bn, pl.tree_in_pages);
      const int prefix_part = std::max(0, std::min(int(it.tile_end), npt) - int(it.tile_begin));
      return it.tile_end > npt ? prefix_part : int(it.tile_end - it.tile_begin);
    };
    for (int c = 0; c < pl.n_ctas; ++c)
      std::stable_sort(pl.items.begin() + pl.cta_begin[size_t(c)], pl.items.begin() + pl.cta_begin[size_t(c) + 1],
                       [&](const WorkItem& a, const WorkItem& b) { return ungated_tiles(a) > ungated_tiles(b); });
  }
  // device layout: fixed stride per CTA, count in the CTA's first item
  pl.items_stride = 1;
  for (int c = 0; c < pl.n_ctas; ++c) pl.items_stride = std::max(pl.items_stride, pl.cta_begin[size_t(c) + 1] - pl.cta_begin[size_t(c)]);
  pl.items_strided.assign(size_t(pl.n_ctas) * size_t(pl.items_stride), WorkItem{});
  for (int c = 0; c < pl.n_ctas; ++c) {
    const int b = pl.cta_begin[size_t(c)], e = pl.cta_begin[size_t(c) + 1];
    for (int k = b; k < e; ++k) pl.items_strided[size_t(c) * size_t(pl.items_stride) + size_t(k - b)] = pl.items[size_t(k)];
    pl.items_strided[size_t(c) * size_t(pl.items_stride)].n_in_cta = e - b;
  }
}

int upload(dyspec_plan& pl) {
  auto pad = [](size_t x) { return (x + 255) & ~size_t(255); };
  const size_t b_reqs = pad(std::max<size_t>(1, pl.reqs.size()) * sizeof(ReqInfo));
  const size_t b_items = pad(std::max<size_t>(1, pl.items_strided.size()) * sizeof(WorkItem));
  const size_t b_groups = pad(std::max<size_t>(1, pl.split_groups.size()) * sizeof(GroupInfo));
  const size_t b_counters = pad(std::max<size_t>(1, pl.split_groups.size()) * sizeof(int32_t));
  const size_t total = b_reqs + b_items + b_groups + b_counters;
  std::vector<uint8_t> host(total, 0);
  size_t off = 0;
  if (!pl.reqs.empty()) memcpy(host.data() + off, pl.reqs.data(), pl.reqs.size() * sizeof(ReqInfo));
  const size_t o_reqs = off; off += b_reqs;
  if (!pl.items_strided.empty()) memcpy(host.data() + off, pl.items_strided.data(), pl.items_strided.size() * sizeof(WorkItem));
  const size_t o_items = off; off += b_items;
  if (!pl.split_groups.empty()) memcpy(host.data() + off, pl.split_groups.data(), pl.split_groups.size() * sizeof(GroupInfo));
  const size_t o_groups = off; off += b_groups;
  const size_t o_counters = off;
  if (cudaGetDevice(&pl.device) != cudaSuccess) return DYSPEC_ERR_CUDA;
  if (cudaMalloc(&pl.d_blob, total) != cudaSuccess) { pl.d_blob = nullptr; return DYSPEC_ERR_CUDA; }
  if (cudaMemcpy(pl.d_blob, host.data(), total, cudaMemcpyHostToDevice) != cudaSuccess) return DYSPEC_ERR_CUDA;
  uint8_t* base = static_cast<uint8_t*>(pl.d_blob);
  pl.d_reqs = reinterpret_cast<ReqInfo*>(base + o_reqs);
  pl.d_items = reinterpret_cast<WorkItem*>(base + o_items);
  pl.d_groups = reinterpret_cast<GroupInfo*>(base + o_groups);
  pl.d_counters = reinterpret_cast<int32_t*>(base + o_counters);
  return DYSPEC_OK;
}

}  // namespace

extern "C" {

const char* dyspec_error_string(int code) {
  switch (code) {
    case DYSPEC_OK: return "ok";
    case DYSPEC_ERR_INVALID_ARG: return "invalid argument";
    case DYSPEC_ERR_UNSUPPORTED: return "unsupported shape";
    case DYSPEC_ERR_WORKSPACE: return "workspace too small or misaligned";
    case DYSPEC_ERR_CUDA: return "CUDA call failed";
    case DYSPEC_ERR_BAD_TREE: return "parent index outside {-1} U [0, i)";
    case DYSPEC_ERR_TIMEOUT: return "bounded in-kernel wait ran out";
    default: return "unknown error code";
  }
}

int dyspec_version(void) { return 100; }

int dyspec_words_per_row(int max_nodes) {
  if (max_nodes < 0 || max_nodes > DYSPEC_MAX_NODES) return DYSPEC_ERR_INVALID_ARG;
  if (max_nodes == 0) return 4;
  return 4 * ((max_nodes + 127) / 128);
}

int dyspec_set_tuning(int force_regime, int force_ctas, int combine_mode) {
  if (combine_mode < 0) return DYSPEC_ERR_INVALID_ARG;
  const int whole = combine_mode >> 4;
  combine_mode &= 15;
  if (force_regime < -1 || force_regime > 1 || combine_mode > 2 || whole > 2) return DYSPEC_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_tuning_mutex);
  g_tuning.whole_groups = whole;
  g_tuning.force_regime = force_regime;
  g_tuning.force_ctas = force_ctas >= 0 ? force_ctas : 0;
  g_tuning.item_cost = force_ctas < 0 ? -force_ctas : 0;   // negative values select the per-item cost instead (experiments)
  g_tuning.combine_mode = combine_mode;
  return DYSPEC_OK;
}

int dyspec_set_trace(void* trace_buffer, int capacity_entries) {
  if (capacity_entries < 0 || (trace_buffer == nullptr) != (capacity_entries == 0)) return DYSPEC_ERR_INVALID_ARG;
#if !defined(DYSPEC_TRACE) && !defined(DYSPEC_CTA_STAMPS)
  if (trace_buffer != nullptr) return DYSPEC_ERR_UNSUPPORTED;      // the hooks are compiled out of this build
#endif
  std::lock_guard<std::mutex> lock(g_tuning_mutex);
  g_tuning.trace = static_cast<unsigned long long*>(trace_buffer);
  g_tuning.trace_capacity = capacity_entries;
  return DYSPEC_OK;
}

static int build_tree_mask_checked(const int32_t* parents, int n_nodes, uint32_t* ancestor_bits, int32_t* depths,
                                   uint32_t* node_tiles, int words_per_row, int32_t* status, dyspec_stream_t stream) {
  if (n_nodes < 0 || words_per_row <= 0 || (words_per_row & 3)) return DYSPEC_ERR_INVALID_ARG;
  if (n_nodes > DYSPEC_MAX_NODES || words_per_row > DYSPEC_MAX_NODES / 32) return DYSPEC_ERR_UNSUPPORTED;
  if (32 * words_per_row < n_nodes) return DYSPEC_ERR_INVALID_ARG;
  if (n_nodes == 0) return DYSPEC_OK;
  if (!parents || !ancestor_bits) return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(ancestor_bits, 16) || !aligned(parents, 4) || !aligned(node_tiles, 4)) return DYSPEC_ERR_INVALID_ARG;
  cudaError_t e = launch_build_tree_mask(parents, nullptr, 1, n_nodes, n_nodes, ancestor_bits, depths, node_tiles,
                                         words_per_row, status, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : DYSPEC_ERR_CUDA;
}

int dyspec_build_tree_mask(const int32_t* parents, int n_nodes, uint32_t* ancestor_bits, int32_t* depths,
                           int words_per_row, int32_t* status, dyspec_stream_t stream) {
  return build_tree_mask_checked(parents, n_nodes, ancestor_bits, depths, nullptr, words_per_row, status, stream);
}

int dyspec_build_tree_mask_batched(const int32_t* parents, const int32_t* node_offsets_host, int n_req,
                                   uint32_t* ancestor_bits, int32_t* depths, int words_per_row, int32_t* status,
                                   dyspec_stream_t stream) {
  if (n_req < 0 || (n_req > 0 && !node_offsets_host)) return DYSPEC_ERR_INVALID_ARG;
  for (int r = 0; r < n_req; ++r)
    if (node_offsets_host[r] < 0 || node_offsets_host[r + 1] < node_offsets_host[r]) return DYSPEC_ERR_INVALID_ARG;
  if (n_req == 0 || node_offsets_host[n_req] == 0) return DYSPEC_OK;
  if (words_per_row <= 0 || (words_per_row & 3)) return DYSPEC_ERR_INVALID_ARG;
  if (words_per_row > DYSPEC_MAX_NODES / 32) return DYSPEC_ERR_UNSUPPORTED;
  int max_n = 0;
  for (int r = 0; r < n_req; ++r) max_n = std::max(max_n, node_offsets_host[r + 1] - node_offsets_host[r]);
  if (max_n > DYSPEC_MAX_NODES) return DYSPEC_ERR_UNSUPPORTED;
  if (32 * words_per_row < max_n) return DYSPEC_ERR_INVALID_ARG;
  if (!parents || !ancestor_bits || !aligned(ancestor_bits, 16) || !aligned(parents, 4)) return DYSPEC_ERR_INVALID_ARG;
  // Without a plan there is no device copy of the request list: it travels with the launch, in the
  // kernel's parameter space.  One launch takes up to kMaskBatchMax requests.
  for (int r0 = 0; r0 < n_req; r0 += kMaskBatchMax) {
    const int cnt = std::min(kMaskBatchMax, n_req - r0);
    MaskBatch batch;
    memset(&batch, 0, sizeof(batch));
    int piece_max = 0;
    for (int k = 0; k <= cnt; ++k) batch.node0[k] = node_offsets_host[r0 + k];
    for (int k = 0; k < cnt; ++k) piece_max = std::max(piece_max, batch.node0[k + 1] - batch.node0[k]);
    batch.first_req = r0;
    cudaError_t e = launch_build_tree_mask_batch(parents, batch, cnt, piece_max, ancestor_bits, depths, words_per_row, status,
                                                 reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_failed(e, "batched mask launch");
  }
  return DYSPEC_OK;
}

int dyspec_build_tree_mask_tiles(const int32_t* parents, int n_nodes, uint32_t* ancestor_bits, int32_t* depths,
                                 uint32_t* node_tiles, int words_per_row, int32_t* status, dyspec_stream_t stream) {
  if (n_nodes > 0 && !node_tiles) return DYSPEC_ERR_INVALID_ARG;
  return build_tree_mask_checked(parents, n_nodes, ancestor_bits, depths, node_tiles, words_per_row, status, stream);
}

int dyspec_dfs_reorder(const int32_t* parents, int n_nodes, int32_t* order, int32_t* new_of_old, int32_t* new_parents,
                       int32_t* status, dyspec_stream_t stream) {
  if (n_nodes < 0) return DYSPEC_ERR_INVALID_ARG;
  if (n_nodes > DYSPEC_MAX_NODES) return DYSPEC_ERR_UNSUPPORTED;
  if (n_nodes == 0) return DYSPEC_OK;
  if (!parents || !aligned(parents, 4) || !aligned(order, 4) || !aligned(new_of_old, 4) || !aligned(new_parents, 4))
    return DYSPEC_ERR_INVALID_ARG;
  if (new_parents == parents) return DYSPEC_ERR_INVALID_ARG;      // not in place: other requests' CTAs may still read
  cudaError_t e = launch_dfs_reorder(parents, nullptr, 1, n_nodes, n_nodes, order, new_of_old, new_parents, status,
                                     reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : DYSPEC_ERR_CUDA;
}

int dyspec_mask_block_count(const uint32_t* ancestor_bits, int n_nodes, int words_per_row, int block, uint64_t* count,
                            dyspec_stream_t stream) {
  if (n_nodes < 0 || words_per_row <= 0 || (words_per_row & 3) || 32 * words_per_row < n_nodes) return DYSPEC_ERR_INVALID_ARG;
  if (!(block == 32 || block == 64 || block == 128)) return DYSPEC_ERR_UNSUPPORTED;
  if (n_nodes > DYSPEC_MAX_NODES) return DYSPEC_ERR_UNSUPPORTED;
  if (!count || !aligned(count, 8) || (n_nodes > 0 && (!ancestor_bits || !aligned(ancestor_bits, 16)))) return DYSPEC_ERR_INVALID_ARG;
  cudaError_t e = launch_mask_block_count(ancestor_bits, n_nodes, words_per_row, block,
                                          reinterpret_cast<unsigned long long*>(count), reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : DYSPEC_ERR_CUDA;
}

int dyspec_verify_tree(const int32_t* parents, const int32_t* tokens, const float* draft_probs, const float* target_probs,
                       const float* accept_u, const float* sample_u, const int32_t* node_offsets, int n_req,
                       int max_nodes, int vocab, int bonus_at_leaf, int32_t* accepted_tokens, int32_t* accepted_nodes,
                       int32_t* n_accepted, int max_out, int32_t* status, dyspec_stream_t stream) {
  if (n_req < 0 || max_nodes < 0 || vocab <= 0 || (vocab & 3) || max_out <= 0) return DYSPEC_ERR_INVALID_ARG;
  if (max_nodes > DYSPEC_MAX_NODES || vocab > DYSPEC_MAX_VOCAB) return DYSPEC_ERR_UNSUPPORTED;
  if (n_req == 0) return DYSPEC_OK;
  if (!parents || !tokens || !draft_probs || !target_probs || !accept_u || !sample_u || !node_offsets ||
      !accepted_tokens || !accepted_nodes || !n_accepted)
    return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(draft_probs, 16) || !aligned(target_probs, 16)) return DYSPEC_ERR_INVALID_ARG;
  cudaError_t e = launch_verify_tree(parents, tokens, draft_probs, target_probs, accept_u, sample_u, node_offsets, n_req,
                                     max_nodes, vocab, bonus_at_leaf, accepted_tokens, accepted_nodes, n_accepted, max_out,
                                     status, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : cuda_failed(e, "verify launch");
}

static int check_tree_build_args(const float* draft_table, int n_rows, int vocab, const float* uniforms, int n_uniforms,
                                 const int32_t* root_row, int n_req, int nodes, const void* parents, const void* tokens,
                                 const void* values, const void* child_values, const void* rows, const void* n_nodes) {
  if (n_rows <= 0 || vocab <= 0 || (vocab & 3) || n_uniforms <= 0 || n_req < 0 || nodes < 0) return DYSPEC_ERR_INVALID_ARG;
  if (vocab > DYSPEC_MAX_VOCAB || nodes > DYSPEC_MAX_NODES - 1) return DYSPEC_ERR_UNSUPPORTED;
  if (n_req == 0) return DYSPEC_OK;
  if (!draft_table || !uniforms || !root_row || !parents || !tokens || !values || !child_values || !rows || !n_nodes)
    return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(draft_table, 16)) return DYSPEC_ERR_INVALID_ARG;
  return DYSPEC_OK;
}

int dyspec_build_tree_greedy(const float* draft_table, int n_rows, int vocab, const float* uniforms, int n_uniforms,
                             const int32_t* root_row, int n_req, int m, int32_t* parents, int32_t* tokens, float* values,
                             float* child_values, int32_t* rows, int32_t* n_nodes, dyspec_stream_t stream) {
  const int rc = check_tree_build_args(draft_table, n_rows, vocab, uniforms, n_uniforms, root_row, n_req, m, parents, tokens,
                                       values, child_values, rows, n_nodes);
  if (rc != DYSPEC_OK || n_req == 0) return rc;
  cudaError_t e = launch_build_tree_greedy(draft_table, n_rows, vocab, uniforms, n_uniforms, root_row, n_req, m, parents,
                                           tokens, values, child_values, rows, n_nodes, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : cuda_failed(e, "greedy tree launch");
}

int dyspec_build_tree_threshold(const float* draft_table, int n_rows, int vocab, const float* uniforms, int n_uniforms,
                                const int32_t* root_row, int n_req, float threshold, int max_nodes, int32_t* parents,
                                int32_t* tokens, float* values, float* child_values, int32_t* rows, int32_t* n_nodes,
                                dyspec_stream_t stream) {
  const int rc = check_tree_build_args(draft_table, n_rows, vocab, uniforms, n_uniforms, root_row, n_req, max_nodes, parents,
                                       tokens, values, child_values, rows, n_nodes);
  if (rc != DYSPEC_OK || n_req == 0) return rc;
  if (!(threshold > 0.f)) return DYSPEC_ERR_INVALID_ARG;
  cudaError_t e = launch_build_tree_threshold(draft_table, n_rows, vocab, uniforms, n_uniforms, root_row, n_req, threshold,
                                              max_nodes, parents, tokens, values, child_values, rows, n_nodes,
                                              reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : cuda_failed(e, "threshold tree launch");
}

int dyspec_compact_kv(void* k_cache, void* v_cache, const int64_t* kv_row_offset, const int32_t* prefix_len,
                      const int32_t* accepted_nodes, const int32_t* n_accepted, int n_req, int max_out, int n_kv_heads,
                      int head_dim, int keep_root, int32_t* new_prefix_len, dyspec_stream_t stream) {
  if (n_req < 0 || max_out <= 0 || n_kv_heads <= 0 || head_dim <= 0) return DYSPEC_ERR_INVALID_ARG;
  const int64_t row_bytes = int64_t(n_kv_heads) * head_dim * 2;
  if (row_bytes % 16 != 0 || row_bytes > (1 << 24)) return DYSPEC_ERR_UNSUPPORTED;
  if (n_req == 0) return DYSPEC_OK;
  if (!k_cache || !v_cache || !kv_row_offset || !prefix_len || !accepted_nodes || !n_accepted) return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(k_cache, 16) || !aligned(v_cache, 16)) return DYSPEC_ERR_INVALID_ARG;
  cudaError_t e = launch_compact_kv(k_cache, v_cache, kv_row_offset, prefix_len, accepted_nodes, n_accepted, n_req, max_out,
                                    int(row_bytes), keep_root != 0, new_prefix_len, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : cuda_failed(e, "compact launch");
}

int dyspec_compact_kv_paged(void* k_cache, void* v_cache, const int64_t* tree_row_offset, const int32_t* page_table,
                            int pages_per_req, int page_size, const int32_t* prefix_len, const int32_t* accepted_nodes,
                            const int32_t* n_accepted, int n_req, int max_out, int n_kv_heads, int head_dim,
                            int keep_root, int32_t* new_prefix_len, int32_t* status, dyspec_stream_t stream) {
  if (n_req < 0 || max_out <= 0 || n_kv_heads <= 0 || head_dim <= 0 || pages_per_req <= 0) return DYSPEC_ERR_INVALID_ARG;
  if (page_size <= 0 || (page_size & (page_size - 1))) return DYSPEC_ERR_INVALID_ARG;
  const int64_t row_bytes = int64_t(n_kv_heads) * head_dim * 2;
  if (row_bytes % 16 != 0 || row_bytes > (1 << 24)) return DYSPEC_ERR_UNSUPPORTED;
  if (n_req == 0) return DYSPEC_OK;
  if (!k_cache || !v_cache || !page_table || !prefix_len || !accepted_nodes || !n_accepted)   // (tree_row_offset may be NULL)
    return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(k_cache, 16) || !aligned(v_cache, 16)) return DYSPEC_ERR_INVALID_ARG;
  int shift = 0;
  while ((1 << shift) < page_size) ++shift;
  cudaError_t e = launch_compact_kv_paged(k_cache, v_cache, tree_row_offset, page_table, pages_per_req, shift, prefix_len,
                                          accepted_nodes, n_accepted, n_req, max_out, int(row_bytes), keep_root != 0, new_prefix_len,
                                          status, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : cuda_failed(e, "paged compact launch");
}

// Validates the arguments and runs the scheduler; no CUDA call.
static int make_host_plan(dyspec_plan** out, int n_q_heads, int n_kv_heads, int head_dim, int n_req,
                          const int32_t* prefix_len, const int32_t* n_nodes, const int64_t* kv_row_offset,
                          int64_t kv_total_rows, int words_per_row, float scale, int page_size = 0,
                          bool allow_queue = true, bool tree_in_pages = false) {
  *out = nullptr;
  if (n_q_heads <= 0 || n_kv_heads <= 0 || n_req < 0 || kv_total_rows < 0) return DYSPEC_ERR_INVALID_ARG;
  if (page_size < 0 || (page_size & (page_size - 1))) return DYSPEC_ERR_INVALID_ARG;
  if (page_size != 0 && (page_size < 128 || page_size > (1 << 20))) return DYSPEC_ERR_UNSUPPORTED;
  if (n_req > 0 && (!prefix_len || !n_nodes || !kv_row_offset)) return DYSPEC_ERR_INVALID_ARG;
  if (words_per_row <= 0 || (words_per_row & 3)) return DYSPEC_ERR_INVALID_ARG;
  if (words_per_row > DYSPEC_MAX_NODES / 32) return DYSPEC_ERR_UNSUPPORTED;
  if (n_q_heads % n_kv_heads != 0) return DYSPEC_ERR_UNSUPPORTED;
  const int g = n_q_heads / n_kv_heads;
  if (!(g == 1 || g == 2 || g == 4 || g == 8)) return DYSPEC_ERR_UNSUPPORTED;
  if (!(head_dim == 64 || head_dim == 128)) return DYSPEC_ERR_UNSUPPORTED;
  if (kv_total_rows >= (int64_t(1) << 31)) return DYSPEC_ERR_UNSUPPORTED;
  dyspec_plan* pl = new (std::nothrow) dyspec_plan();
  if (!pl) return DYSPEC_ERR_CUDA;
  pl->hq = n_q_heads; pl->hkv = n_kv_heads; pl->d = head_dim; pl->g = g;
  pl->log2g = g == 1 ? 0 : g == 2 ? 1 : g == 4 ? 2 : 3;
  pl->W = words_per_row;
  pl->scale = scale > 0.f ? scale : 1.0f / std::sqrt(float(head_dim));
  pl->n_req = n_req;
  pl->kv_total_rows = kv_total_rows;
  pl->page_size = page_size;
  pl->tree_in_pages = tree_in_pages && page_size != 0;
  pl->allow_queue = allow_queue;
  int64_t node0 = 0;
  int max_rows = 0;
  for (int r = 0; r < n_req; ++r) {
    if (prefix_len[r] < 0 || n_nodes[r] < 0 || kv_row_offset[r] < 0) { delete pl; return DYSPEC_ERR_INVALID_ARG; }
    if (n_nodes[r] > DYSPEC_MAX_NODES) { delete pl; return DYSPEC_ERR_UNSUPPORTED; }
    if (32 * words_per_row < n_nodes[r]) { delete pl; return DYSPEC_ERR_INVALID_ARG; }
    if (!pl->tree_in_pages && kv_row_offset[r] + (page_size ? 0 : prefix_len[r]) + n_nodes[r] > kv_total_rows) { delete pl; return DYSPEC_ERR_INVALID_ARG; }
    ReqInfo rq{};
    rq.kv_row0 = kv_row_offset[r]; rq.prefix_len = prefix_len[r]; rq.n_nodes = n_nodes[r]; rq.node0 = int32_t(node0);
    pl->reqs.push_back(rq);
    node0 += n_nodes[r];
    max_rows = std::max(max_rows, n_nodes[r] * g);
    pl->max_nodes = std::max(pl->max_nodes, int(n_nodes[r]));
  }
  if (node0 >= (int64_t(1) << 31)) { delete pl; return DYSPEC_ERR_UNSUPPORTED; }
  pl->total_nodes = node0;
  // Regime: tcgen05 tiles (2 x 128 packed rows per item) when some request has more packed rows
  // (nodes x group) than one warp-level tile holds, else warp-level tiles (64 packed rows).
  pl->tune = current_tuning();
  pl->n_sms = device_sm_count();
  pl->regime = pl->tune.force_regime >= 0 ? pl->tune.force_regime : (max_rows > 64 ? 1 : 0);
  pl->bm = pl->regime == 0 ? 64 : 256;    // packed query rows per work item (regime 1: two 128-row halves)
  pl->bn = pl->regime == 0 ? 64 : 128;    // keys per tile
  if (pl->tune.combine_mode == 2)
    for (int C : {2, 4, 8})
      pl->cluster_fit[C] = pl->regime == 1 ? attn_tc_max_clusters(pl->d, C) : attn_small_max_clusters(pl->d, C);
  schedule(*pl);
  // A cluster plan of the tensor-core regime needs C CTAs of 1 CTA / SM side by side: where the device cannot
  // hold even one such cluster (a reduced share of its SMs), plan again without clusters.
  // (The same when the device cannot hold all of the plan's clusters at once -- the SMs of a cluster have to
  //  come from one GPC -- since the clusters left over would run as a second wave.)
  if (pl->regime == 1 && pl->cluster > 1) {
    const int fit = attn_tc_max_clusters(pl->d, pl->cluster);
    if (fit >= 0 && fit < pl->n_ctas / pl->cluster) {
      pl->tune.combine_mode = 1;
      schedule(*pl);
    }
  }
  pl->workspace_bytes = size_t(pl->n_slots) * size_t(pl->bm) * (pl->d + 2) * sizeof(float);
  if (pl->regime == 1 && pl->cluster > 1)   // cluster plan: the shares a CTA's peers cannot push into its shared memory
    pl->workspace_bytes = size_t(pl->n_ctas) * attn_tc_cluster_workspace_per_cta(pl->d, pl->cluster);
  if (!pl->split_groups.empty()) {      // the groups' counter pairs follow the partials
    pl->counters_offset = (pl->workspace_bytes + 255) & ~size_t(255);
    pl->workspace_bytes = pl->counters_offset + ((pl->split_groups.size() * 2 * sizeof(int32_t) + 255) & ~size_t(255));
    // (the items of a group wait for each other inside the kernel: only when every CTA of the launch is
    //  resident at once, i.e. one CTA per SM and no more CTAs than SMs; a forced larger grid keeps the combine launch)
    pl->merge_in_kernel = pl->regime == 1 && pl->tune.combine_mode != 0 && pl->n_ctas <= pl->n_sms;
  }
  if (pl->dynamic) {                    // the queue words follow the partials (there are none in such a plan today)
    pl->queue_offset = (pl->workspace_bytes + 255) & ~size_t(255);
    pl->workspace_bytes = pl->queue_offset + 256;
  }
  *out = pl;
  return DYSPEC_OK;
}

int dyspec_plan_create(dyspec_plan_t** plan, int n_q_heads, int n_kv_heads, int head_dim, int n_req,
                       const int32_t* prefix_len, const int32_t* n_nodes, const int64_t* kv_row_offset,
                       int64_t kv_total_rows, int words_per_row, float scale) {
  if (!plan) return DYSPEC_ERR_INVALID_ARG;
  dyspec_plan* pl = nullptr;
  int rc = make_host_plan(&pl, n_q_heads, n_kv_heads, head_dim, n_req, prefix_len, n_nodes, kv_row_offset,
                          kv_total_rows, words_per_row, scale);
  *plan = nullptr;
  if (rc != DYSPEC_OK) return rc;
  rc = upload(*pl);
  if (rc != DYSPEC_OK) { dyspec_plan_destroy(pl); return rc; }
  *plan = pl;
  return DYSPEC_OK;
}

int dyspec_plan_create_paged(dyspec_plan_t** plan, int n_q_heads, int n_kv_heads, int head_dim, int n_req,
                             const int32_t* prefix_len, const int32_t* n_nodes, const int64_t* tree_row_offset,
                             int64_t kv_total_rows, int page_size, int words_per_row, float scale) {
  if (!plan) return DYSPEC_ERR_INVALID_ARG;
  *plan = nullptr;
  if (page_size <= 0) return DYSPEC_ERR_INVALID_ARG;
  dyspec_plan* pl = nullptr;
  // no tree rows of their own: node j of request r is token L_r + j of its paged sequence
  const bool in_pages = tree_row_offset == nullptr;
  const std::vector<int64_t> zeros(size_t(std::max(n_req, 1)), 0);
  int rc = make_host_plan(&pl, n_q_heads, n_kv_heads, head_dim, n_req, prefix_len, n_nodes,
                          in_pages ? zeros.data() : tree_row_offset, kv_total_rows, words_per_row, scale, page_size, true, in_pages);
  if (rc != DYSPEC_OK) return rc;
  rc = upload(*pl);
  if (rc != DYSPEC_OK) { dyspec_plan_destroy(pl); return rc; }
  *plan = pl;
  return DYSPEC_OK;
}

int dyspec_schedule_dry_run(int n_q_heads, int n_kv_heads, int head_dim, int n_req, const int32_t* prefix_len,
                            const int32_t* n_nodes, int words_per_row, int32_t* items_out, int max_items,
                            int32_t* cta_begin_out, int max_ctas, int64_t* info_out) {
  std::vector<int64_t> off(size_t(std::max(n_req, 1)), 0);
  int64_t rows = 0;
  for (int r = 0; r < n_req && prefix_len && n_nodes; ++r) {
    off[size_t(r)] = rows;
    rows += int64_t(std::max(prefix_len[r], 0)) + std::max(n_nodes[r], 0);
  }
  dyspec_plan* pl = nullptr;
  const int rc = make_host_plan(&pl, n_q_heads, n_kv_heads, head_dim, n_req, prefix_len, n_nodes, off.data(), rows,
                                words_per_row, 0.f);
  if (rc != DYSPEC_OK) return rc;
  const int n_items = int(pl->items.size());
  if (items_out)
    for (int i = 0; i < n_items && i < max_items; ++i) {
      const WorkItem& it = pl->items[size_t(i)];
      const int32_t rec[8] = {it.req, it.kv_head, it.row0, it.tile_begin, it.tile_end, it.slot, it.group, it.n_splits};
      memcpy(items_out + 8 * i, rec, sizeof(rec));
    }
  if (cta_begin_out)
    for (int c = 0; c <= pl->n_ctas && c < max_ctas; ++c) cta_begin_out[c] = pl->cta_begin[size_t(c)];
  if (info_out) {
    info_out[0] = n_items; info_out[1] = pl->n_ctas; info_out[2] = pl->n_groups; info_out[3] = int64_t(pl->split_groups.size());
    info_out[4] = pl->max_splits; info_out[5] = pl->regime; info_out[6] = pl->total_tiles; info_out[7] = pl->bm;
    info_out[8] = pl->bn; info_out[9] = int64_t(pl->workspace_bytes); info_out[10] = pl->cluster;
    info_out[11] = (!pl->split_groups.empty() && !pl->merge_in_kernel) ? 1 : 0;
  }
  delete pl;
  return n_items;
}

int dyspec_plan_destroy(dyspec_plan_t* plan) {
  if (!plan) return DYSPEC_OK;
  if (plan->d_blob) cudaFree(plan->d_blob);
  delete plan;
  return DYSPEC_OK;
}

size_t dyspec_plan_workspace_bytes(const dyspec_plan_t* plan) { return plan ? plan->workspace_bytes : 0; }

int64_t dyspec_plan_info(const dyspec_plan_t* plan, int field) {
  if (!plan) return DYSPEC_ERR_INVALID_ARG;
  switch (field) {
    case 0: return int64_t(plan->items.size());
    case 1: return plan->n_ctas;
    case 2: return plan->n_groups;
    case 3: return int64_t(plan->split_groups.size());
    case 4: return plan->max_splits;
    case 5: return plan->regime;
    case 6: return plan->total_tiles;
    case 7: return plan->bm;
    case 8: return plan->cluster;
    case 9: return plan->dynamic ? 1 : 0;
    case 10: return (!plan->split_groups.empty() && !plan->merge_in_kernel) ? 1 : 0;
    default: return DYSPEC_ERR_INVALID_ARG;
  }
}

static int plan_build_tree_mask_checked(const dyspec_plan_t* plan, const int32_t* parents, uint32_t* ancestor_bits,
                                        int32_t* depths, uint32_t* node_tiles, int32_t* status, dyspec_stream_t stream) {
  if (!plan) return DYSPEC_ERR_INVALID_ARG;
  if (plan->n_req == 0 || plan->total_nodes == 0) return DYSPEC_OK;
  if (!parents || !ancestor_bits || !aligned(ancestor_bits, 16) || !aligned(node_tiles, 4)) return DYSPEC_ERR_INVALID_ARG;
  cudaError_t e = launch_build_tree_mask(parents, plan->d_reqs, plan->n_req, 0, plan->max_nodes, ancestor_bits, depths,
                                         node_tiles, plan->W, status, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : DYSPEC_ERR_CUDA;
}

int dyspec_plan_build_tree_mask(const dyspec_plan_t* plan, const int32_t* parents, uint32_t* ancestor_bits,
                                int32_t* depths, int32_t* status, dyspec_stream_t stream) {
  return plan_build_tree_mask_checked(plan, parents, ancestor_bits, depths, nullptr, status, stream);
}

int dyspec_plan_build_tree_mask_tiles(const dyspec_plan_t* plan, const int32_t* parents, uint32_t* ancestor_bits,
                                      int32_t* depths, uint32_t* node_tiles, int32_t* status, dyspec_stream_t stream) {
  if (plan && plan->total_nodes > 0 && !node_tiles) return DYSPEC_ERR_INVALID_ARG;
  return plan_build_tree_mask_checked(plan, parents, ancestor_bits, depths, node_tiles, status, stream);
}

int dyspec_plan_dfs_reorder(const dyspec_plan_t* plan, const int32_t* parents, int32_t* order, int32_t* new_of_old,
                            int32_t* new_parents, int32_t* status, dyspec_stream_t stream) {
  if (!plan) return DYSPEC_ERR_INVALID_ARG;
  if (plan->n_req == 0 || plan->total_nodes == 0) return DYSPEC_OK;
  if (!parents || !aligned(parents, 4) || !aligned(order, 4) || !aligned(new_of_old, 4) || !aligned(new_parents, 4))
    return DYSPEC_ERR_INVALID_ARG;
  if (new_parents == parents) return DYSPEC_ERR_INVALID_ARG;
  cudaError_t e = launch_dfs_reorder(parents, plan->d_reqs, plan->n_req, 0, plan->max_nodes, order, new_of_old,
                                     new_parents, status, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DYSPEC_OK : DYSPEC_ERR_CUDA;
}

int dyspec_tree_attention_ragged(const dyspec_plan_t* plan, const void* q, const void* k_cache, const void* v_cache,
                                 const uint32_t* ancestor_bits, void* out, void* workspace, size_t workspace_bytes,
                                 int32_t* status, dyspec_stream_t stream) {
  return dyspec_tree_attention_ragged_sparse(plan, q, k_cache, v_cache, ancestor_bits, nullptr, out, workspace,
                                             workspace_bytes, status, stream);
}

static int run_attention(const dyspec_plan_t* plan, const void* q, const void* k_cache, const void* v_cache,
                         const int32_t* page_table, int pages_per_req, const uint32_t* ancestor_bits,
                         const uint32_t* node_tiles, void* out, void* workspace, size_t workspace_bytes, int32_t* status,
                         dyspec_stream_t stream);

int dyspec_tree_attention_ragged_sparse(const dyspec_plan_t* plan, const void* q, const void* k_cache,
                                        const void* v_cache, const uint32_t* ancestor_bits, const uint32_t* node_tiles,
                                        void* out, void* workspace, size_t workspace_bytes, int32_t* status,
                                        dyspec_stream_t stream) {
  if (plan && plan->page_size != 0) return DYSPEC_ERR_INVALID_ARG;      // a paged plan needs its page table
  return run_attention(plan, q, k_cache, v_cache, nullptr, 0, ancestor_bits, node_tiles, out, workspace, workspace_bytes,
                       status, stream);
}

int dyspec_tree_attention_paged(const dyspec_plan_t* plan, const void* q, const void* k_cache, const void* v_cache,
                                const int32_t* page_table, int pages_per_req, const uint32_t* ancestor_bits,
                                const uint32_t* node_tiles, void* out, void* workspace, size_t workspace_bytes,
                                int32_t* status, dyspec_stream_t stream) {
  if (!plan || plan->page_size == 0) return DYSPEC_ERR_INVALID_ARG;
  if (plan->n_ctas == 0) return DYSPEC_OK;
  if (!page_table || !aligned(page_table, 4) || pages_per_req <= 0) return DYSPEC_ERR_INVALID_ARG;
  for (const ReqInfo& rq : plan->reqs)                                   // every prefix token has a table entry
    if ((int64_t(rq.prefix_len) + (plan->tree_in_pages ? rq.n_nodes : 0) + plan->page_size - 1) / plan->page_size > pages_per_req)
      return DYSPEC_ERR_INVALID_ARG;
  return run_attention(plan, q, k_cache, v_cache, page_table, pages_per_req, ancestor_bits, node_tiles, out, workspace,
                       workspace_bytes, status, stream);
}

static int run_attention(const dyspec_plan_t* plan, const void* q, const void* k_cache, const void* v_cache,
                         const int32_t* page_table, int pages_per_req, const uint32_t* ancestor_bits,
                         const uint32_t* node_tiles, void* out, void* workspace, size_t workspace_bytes, int32_t* status,
                         dyspec_stream_t stream) {
  if (!plan) return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(node_tiles, 4)) return DYSPEC_ERR_INVALID_ARG;
  if (plan->n_ctas == 0) return DYSPEC_OK;
  if (!q || !k_cache || !v_cache || !ancestor_bits || !out) return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(out, 16) || !aligned(ancestor_bits, 16))
    return DYSPEC_ERR_INVALID_ARG;
  int dev = -1;                          // the plan's tables live on the device it was created on
  if (cudaGetDevice(&dev) != cudaSuccess) return DYSPEC_ERR_CUDA;
  if (dev != plan->device) return DYSPEC_ERR_INVALID_ARG;
  if (plan->workspace_bytes > 0 && (!workspace || workspace_bytes < plan->workspace_bytes || !aligned(workspace, 256)))
    return DYSPEC_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

  CUtensorMap mq, mk, mv;
  const int bm = plan->bm, bn = plan->bn;
  const int q_box_rows = plan->regime == 0 ? 64 : 128;   // packed rows per TMA box of Q
  if (!encode_map(&mq, q, plan->total_nodes, plan->hq, plan->d, plan->g, q_box_rows / plan->g) ||
      !encode_map(&mk, k_cache, plan->kv_total_rows, plan->hkv, plan->d, 1, bn) ||
      !encode_map(&mv, v_cache, plan->kv_total_rows, plan->hkv, plan->d, 1, bn))
    return DYSPEC_ERR_CUDA;

  AttnParams p{};
  p.reqs = plan->d_reqs; p.items = plan->d_items; p.groups = plan->d_groups;
  p.bits = ancestor_bits; p.out = static_cast<__nv_bfloat16*>(out);
  p.node_tiles = plan->tree_in_pages ? nullptr : node_tiles;   // the tile sets count unshifted tree tiles
  p.partial = static_cast<float*>(workspace);
  p.counters = plan->split_groups.empty() ? nullptr
                                          : reinterpret_cast<int32_t*>(static_cast<unsigned char*>(workspace) + plan->counters_offset);
  p.merge_in_kernel = plan->merge_in_kernel ? 1 : 0;
  p.status = status;
  p.queue = plan->dynamic ? reinterpret_cast<int32_t*>(static_cast<unsigned char*>(workspace) + plan->queue_offset) : nullptr;
  p.n_items_total = int32_t(plan->items_strided.size());
  p.n_q_heads = plan->hq; p.n_kv_heads = plan->hkv; p.group_size = plan->g; p.log2_g = plan->log2g;
  p.words_per_row = plan->W; p.slot_floats = bm * (plan->d + 2);
  p.scale_log2e = plan->scale * kLog2e;
  p.items_stride = plan->items_stride;
  p.cluster_size = plan->cluster;
  {
    const Tuning now = current_tuning();
    p.trace = now.trace; p.trace_capacity = now.trace_capacity;
  }
  p.page_table = page_table; p.pages_per_req = pages_per_req;
  p.tree_in_pages = plan->tree_in_pages ? 1 : 0;
  for (p.page_shift = 0; page_table && (1 << p.page_shift) < plan->page_size; ++p.page_shift) {}

  cudaError_t e;
  if (plan->regime == 0) e = launch_attn_small(plan->d, plan->n_ctas, mq, mk, mv, p, plan->items_strided.data(), st);
  else e = launch_attn_tc(plan->d, plan->n_ctas, mq, mk, mv, p, plan->items_strided.data(), st);
  if (e != cudaSuccess) return cuda_failed(e, "attention launch");
  if (plan->merge_in_kernel) return DYSPEC_OK;
  e = launch_combine(plan->d, bm, int(plan->split_groups.size()), p, st);
  return e == cudaSuccess ? DYSPEC_OK : cuda_failed(e, "combine launch");
}

// ---- single-request convenience form -------------------------------------------------------------
//
// In a decoding loop the prefix grows and the tree changes at every step, but all layers of a step
// share one (prefix_len, n_nodes).  So the cache is small and bounded: per (device, static shape) a
// handful of slots, each a host plan plus a device table buffer that is reused when the slot is
// recycled (least recently used first), and ONE workspace sized for the worst case of that shape (a
// plan never has more than two split pieces per CTA).  A miss runs the host scheduler and sends the
// tables down the stream in kernel parameters: no allocation, no synchronisation, after the first calls.
namespace {
struct DefaultShape { int hq = 0, hkv = 0, d = 0, W = 0; float scale = 0.f; };
DefaultShape g_shape;
constexpr int kSingleSlots = 8;
struct SingleSlot {
  dyspec_plan* plan = nullptr;          // host object; its device tables live in `blob`
  int prefix_len = -1, n_nodes = -1;
  uint64_t used = 0;                    // for least-recently-used replacement
  void* blob = nullptr;
  size_t blob_bytes = 0;
};
struct ShapeCache {
  SingleSlot slot[kSingleSlots];
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  uint64_t clock = 0;
};
// keyed by device, static shape and scale (bit pattern)
std::map<std::tuple<int, int, int, int, int, uint32_t>, ShapeCache> g_cache;
std::mutex g_cache_mutex;

// Places the plan's tables in `blob` (laid out as upload() does) through the stream.
int send_tables(dyspec_plan& pl, void* blob, size_t blob_bytes, cudaStream_t st, size_t* needed) {
  auto pad = [](size_t x) { return (x + 255) & ~size_t(255); };
  const size_t b_reqs = pad(std::max<size_t>(1, pl.reqs.size()) * sizeof(ReqInfo));
  const size_t b_items = pad(std::max<size_t>(1, pl.items_strided.size()) * sizeof(WorkItem));
  const size_t b_groups = pad(std::max<size_t>(1, pl.split_groups.size()) * sizeof(GroupInfo));
  const size_t b_counters = pad(std::max<size_t>(1, pl.split_groups.size()) * sizeof(int32_t));
  *needed = b_reqs + b_items + b_groups + b_counters;
  if (!blob || blob_bytes < *needed) return DYSPEC_ERR_WORKSPACE;
  uint8_t* base = static_cast<uint8_t*>(blob);
  pl.d_reqs = reinterpret_cast<ReqInfo*>(base);
  pl.d_items = reinterpret_cast<WorkItem*>(base + b_reqs);
  pl.d_groups = reinterpret_cast<GroupInfo*>(base + b_reqs + b_items);
  pl.d_counters = reinterpret_cast<int32_t*>(base + b_reqs + b_items + b_groups);
  if (write_table(pl.d_reqs, pl.reqs.data(), pl.reqs.size() * sizeof(ReqInfo), st) != cudaSuccess ||
      write_table(pl.d_items, pl.items_strided.data(), pl.items_strided.size() * sizeof(WorkItem), st) != cudaSuccess ||
      write_table(pl.d_groups, pl.split_groups.data(), pl.split_groups.size() * sizeof(GroupInfo), st) != cudaSuccess ||
      cudaMemsetAsync(pl.d_counters, 0, b_counters, st) != cudaSuccess)
    return DYSPEC_ERR_CUDA;
  return DYSPEC_OK;
}
}  // namespace

int dyspec_set_default_shape(int n_q_heads, int n_kv_heads, int head_dim, int words_per_row, float scale) {
  if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0) return DYSPEC_ERR_INVALID_ARG;
  const int g = n_q_heads / n_kv_heads;
  if (!(g == 1 || g == 2 || g == 4 || g == 8) || !(head_dim == 64 || head_dim == 128)) return DYSPEC_ERR_UNSUPPORTED;
  if (words_per_row <= 0 || (words_per_row & 3)) return DYSPEC_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  g_shape.hq = n_q_heads; g_shape.hkv = n_kv_heads; g_shape.d = head_dim; g_shape.W = words_per_row; g_shape.scale = scale;
  return DYSPEC_OK;
}

int dyspec_release_cache(void) {
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  int dev0 = -1;
  cudaGetDevice(&dev0);
  for (auto& kv : g_cache) {
    if (cudaSetDevice(std::get<0>(kv.first)) != cudaSuccess) continue;
    for (SingleSlot& sl : kv.second.slot) {
      delete sl.plan;                    // host only: its tables are in the slot's buffer
      if (sl.blob) cudaFree(sl.blob);
    }
    if (kv.second.workspace) cudaFree(kv.second.workspace);
  }
  g_cache.clear();
  if (dev0 >= 0) cudaSetDevice(dev0);
  return DYSPEC_OK;
}

int dyspec_tree_attention(const void* q, const void* k_cache, const void* v_cache, int prefix_len,
                          const uint32_t* ancestor_bits, int n_nodes, void* out, dyspec_stream_t stream) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return DYSPEC_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  std::lock_guard<std::mutex> lock(g_cache_mutex);      // held across the launch: the slot must not be recycled under it
  if (g_shape.hq == 0) return DYSPEC_ERR_INVALID_ARG;
  if (prefix_len < 0 || n_nodes < 0) return DYSPEC_ERR_INVALID_ARG;
  uint32_t scale_bits;
  memcpy(&scale_bits, &g_shape.scale, 4);
  ShapeCache& sc = g_cache[std::make_tuple(dev, g_shape.hq, g_shape.hkv, g_shape.d, g_shape.W, scale_bits)];
  SingleSlot* hit = nullptr;
  SingleSlot* lru = &sc.slot[0];
  for (SingleSlot& sl : sc.slot) {
    if (sl.plan && sl.prefix_len == prefix_len && sl.n_nodes == n_nodes) hit = &sl;
    if (sl.used < lru->used) lru = &sl;
  }
  if (!hit) {
    const int32_t L = prefix_len, n = n_nodes;
    const int64_t off = 0;
    dyspec_plan* pl = nullptr;
    // fixed work lists only: the one workspace is shared by every plan of the shape, so there is no place
    // for a queue head that stays zero between launches of different plans
    int rc = make_host_plan(&pl, g_shape.hq, g_shape.hkv, g_shape.d, 1, &L, &n, &off, int64_t(L) + n, g_shape.W,
                            g_shape.scale, 0, false);
    if (rc != DYSPEC_OK) return rc;
    pl->device = dev;
    if (!sc.workspace) {                 // once per (device, shape): at most two split pieces per CTA, 256-row tiles
      const size_t worst = size_t(2) * size_t(pl->n_sms) * 256 * size_t(g_shape.d + 2) * sizeof(float) + 16 * size_t(pl->n_sms) + 1024;
      if (cudaMalloc(&sc.workspace, worst) != cudaSuccess) { sc.workspace = nullptr; delete pl; return DYSPEC_ERR_CUDA; }
      if (cudaMemsetAsync(sc.workspace, 0, worst, st) != cudaSuccess) { delete pl; return DYSPEC_ERR_CUDA; }
      sc.workspace_bytes = worst;
    }
    if (pl->workspace_bytes > sc.workspace_bytes) { delete pl; return DYSPEC_ERR_WORKSPACE; }   // cannot happen (see above)
    size_t needed = 0;
    rc = send_tables(*pl, lru->blob, lru->blob_bytes, st, &needed);
    if (rc == DYSPEC_ERR_WORKSPACE) {    // the slot's table buffer is too small (or not there yet): replace it
      if (lru->blob) cudaFree(lru->blob);              // (synchronises: nothing in flight reads it afterwards)
      lru->blob = nullptr;
      lru->blob_bytes = std::max<size_t>(needed, size_t(64) << 10);
      if (cudaMalloc(&lru->blob, lru->blob_bytes) != cudaSuccess) { lru->blob = nullptr; lru->blob_bytes = 0; delete pl; return DYSPEC_ERR_CUDA; }
      rc = send_tables(*pl, lru->blob, lru->blob_bytes, st, &needed);
    }
    if (rc != DYSPEC_OK) { delete pl; return rc; }
    delete lru->plan;
    lru->plan = pl; lru->prefix_len = prefix_len; lru->n_nodes = n_nodes;
    hit = lru;
  }
  hit->used = ++sc.clock;
  return dyspec_tree_attention_ragged(hit->plan, q, k_cache, v_cache, ancestor_bits, out, sc.workspace,
                                      sc.workspace_bytes, nullptr, stream);
}

}  // extern "C"

// ---- allocation-free single-request form ----------------------------------------------------------
//
// Everything the attention kernels need beyond the caller's inputs and outputs -- the scheduled work
// list and the split-KV partials -- is placed in one fixed device array that is part of the library
// image.  The array's name is only a host-side handle: kernels get the real device address, looked up
// once per device with cudaGetSymbolAddress.
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[DYSPEC_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
unsigned char* g_static_scratch_addr[kMaxDevices] = {};
std::mutex g_static_scratch_mutex;

// Device address of the scratch array on the current device (set-up on first use per device).
int static_scratch_base(unsigned char** base) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DYSPEC_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DYSPEC_ERR_CUDA;
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(ptr);
  }
  *base = g_static_scratch_addr[dev];
  return DYSPEC_OK;
}

}  // namespace

extern "C" int dyspec_tree_attention_static(const void* q, const void* k_cache, const void* v_cache, int prefix_len,
                                            const uint32_t* ancestor_bits, int n_nodes, void* out, int n_q_heads,
                                            int n_kv_heads, int head_dim, int words_per_row, float scale,
                                            int32_t* status, dyspec_stream_t stream) {
  if (prefix_len < 0 || n_nodes < 0) return DYSPEC_ERR_INVALID_ARG;
  const int32_t L = prefix_len, n = n_nodes;
  const int64_t off = 0;
  dyspec_plan* pl = nullptr;
  // fixed work lists only: the scratch array is rewritten by every call, there is no zeroed queue to share
  int rc = make_host_plan(&pl, n_q_heads, n_kv_heads, head_dim, 1, &L, &n, &off, int64_t(L) + n, words_per_row, scale,
                          0, false);
  if (rc != DYSPEC_OK) return rc;
  struct Guard { dyspec_plan* p; ~Guard() { delete p; } } guard{pl};   // host-only object: nothing to cudaFree
  if (pl->n_ctas == 0) return DYSPEC_OK;
  if (!q || !k_cache || !v_cache || !ancestor_bits || !out) return DYSPEC_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(out, 16) || !aligned(ancestor_bits, 16))
    return DYSPEC_ERR_INVALID_ARG;

  // layout inside the scratch array: [requests | work items | split groups | counters | partials]
  auto pad = [](size_t x) { return (x + 255) & ~size_t(255); };
  const size_t o_reqs = 0;
  const size_t o_items = o_reqs + pad(pl->reqs.size() * sizeof(ReqInfo));
  const size_t o_groups = o_items + pad(pl->items_strided.size() * sizeof(WorkItem));
  const size_t o_counters = o_groups + pad(std::max<size_t>(1, pl->split_groups.size()) * sizeof(GroupInfo));
  const size_t o_partial = o_counters + pad(std::max<size_t>(1, pl->split_groups.size()) * sizeof(int32_t));
  const size_t total = o_partial + pl->workspace_bytes;
  if (total > size_t(DYSPEC_STATIC_SCRATCH_BYTES)) return DYSPEC_ERR_WORKSPACE;   // batch too large for the fixed array

  unsigned char* base = nullptr;
  rc = static_scratch_base(&base);
  if (rc != DYSPEC_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

  // The array keeps whatever the previous call left: rewrite the tables, clear the counters.  The tables
  // travel in kernel parameters (write_table), so nothing on the device ever refers to this call's host memory.
  if (write_table(base + o_reqs, pl->reqs.data(), pl->reqs.size() * sizeof(ReqInfo), st) != cudaSuccess ||
      write_table(base + o_items, pl->items_strided.data(), pl->items_strided.size() * sizeof(WorkItem), st) != cudaSuccess ||
      (!pl->split_groups.empty() &&
       write_table(base + o_groups, pl->split_groups.data(), pl->split_groups.size() * sizeof(GroupInfo), st) != cudaSuccess))
    return DYSPEC_ERR_CUDA;
  // the split groups' counter pairs sit inside the workspace part, behind the partials: they must start at zero
  if (!pl->split_groups.empty() &&
      cudaMemsetAsync(base + o_partial + pl->counters_offset, 0, pl->workspace_bytes - pl->counters_offset, st) != cudaSuccess)
    return DYSPEC_ERR_CUDA;

  CUtensorMap mq, mk, mv;
  const int bm = pl->bm, bn = pl->bn;
  const int q_box_rows = pl->regime == 0 ? 64 : 128;
  if (!encode_map(&mq, q, pl->total_nodes, pl->hq, pl->d, pl->g, q_box_rows / pl->g) ||
      !encode_map(&mk, k_cache, pl->kv_total_rows, pl->hkv, pl->d, 1, bn) ||
      !encode_map(&mv, v_cache, pl->kv_total_rows, pl->hkv, pl->d, 1, bn))
    return DYSPEC_ERR_CUDA;

  AttnParams p{};
  p.reqs = reinterpret_cast<const ReqInfo*>(base + o_reqs);
  p.items = reinterpret_cast<const WorkItem*>(base + o_items);
  p.groups = reinterpret_cast<const GroupInfo*>(base + o_groups);
  p.partial = reinterpret_cast<float*>(base + o_partial);
  p.counters = pl->split_groups.empty() ? nullptr : reinterpret_cast<int32_t*>(base + o_partial + pl->counters_offset);
  p.merge_in_kernel = pl->merge_in_kernel ? 1 : 0;
  p.bits = ancestor_bits; p.out = static_cast<__nv_bfloat16*>(out); p.status = status;
  p.n_q_heads = pl->hq; p.n_kv_heads = pl->hkv; p.group_size = pl->g; p.log2_g = pl->log2g;
  p.words_per_row = pl->W; p.slot_floats = bm * (pl->d + 2);
  p.scale_log2e = pl->scale * kLog2e;
  p.items_stride = pl->items_stride;
  p.cluster_size = pl->cluster;

  cudaError_t e;
  if (pl->regime == 0) e = launch_attn_small(pl->d, pl->n_ctas, mq, mk, mv, p, pl->items_strided.data(), st);
  else e = launch_attn_tc(pl->d, pl->n_ctas, mq, mk, mv, p, pl->items_strided.data(), st);
  if (e != cudaSuccess) return DYSPEC_ERR_CUDA;
  if (pl->merge_in_kernel) return DYSPEC_OK;
  e = launch_combine(pl->d, bm, int(pl->split_groups.size()), p, st);
  return e == cudaSuccess ? DYSPEC_OK : DYSPEC_ERR_CUDA;
}
