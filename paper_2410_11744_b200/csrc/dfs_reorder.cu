// Depth-first renumbering of a token tree (App. C: DySpec orders the tree tokens by DFS, which
// approximates heavy-path order, so that the attention mask touches few b x b blocks).
//
// One CTA per request.  new index of node i = its position in the pre-order walk that visits roots
// and the children of every node in increasing old index.  No thread walks the tree: the CTA builds
// the Euler tour of the forest as a linked list (an "enter" and an "exit" element per node) and
// ranks it by pointer jumping, ceil(log2(2 n)) rounds whatever the shape of the tree.
//
//   1. previous sibling of every node, in index order.  A warp looks at 32 consecutive nodes and
//      groups equal parents with match.any; the last lane of each group records itself in a byte
//      table [parent][chunk]; the first lane of each group then finds the nearest earlier chunk
//      that holds the same parent.  Roots are the children of a virtual node n.
//   2. first child / next sibling follow from that, and with them the tour:
//        enter(i) -> enter(first child of i), or exit(i) for a leaf
//        exit(i)  -> enter(next sibling of i), or exit(parent of i), or the end of the list
//   3. list ranking with weight 1 on enter elements: S(e) = number of enter elements from e to the
//      end, so the pre-order index of node i is n - S(enter(i)).
//
// A parent outside {-1} U [0, i) makes that node a root and reports DYSPEC_ERR_BAD_TREE, as in the
// mask builder.
#include "common.cuh"

namespace dyspec {

namespace {
constexpr uint32_t kNone = 0xFFFFu;
}

__global__ void __launch_bounds__(1024, 1)
dfs_reorder_kernel(const int32_t* __restrict__ parents, const ReqInfo* __restrict__ reqs, int single_n,
                   int32_t* __restrict__ order, int32_t* __restrict__ new_of_old, int32_t* __restrict__ new_parents,
                   int32_t* status) {
  extern __shared__ __align__(16) uint8_t ro_smem[];
  // No early launch of dependents here: the kernel that follows is normally the mask builder, which
  // reads its parent array (this kernel's output) before it waits on its predecessor.  Without the
  // trigger the stream serialises the two completely.
  int node0 = 0, n = single_n;
  if (reqs != nullptr) {
    node0 = reqs[blockIdx.x].node0;
    n = reqs[blockIdx.x].n_nodes;
  }
  if (n <= 0) return;
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
  const int n_chunks = (n + 31) >> 5;
  const int row_bytes = (n_chunks + 3) & ~3;                       // table row: one byte per chunk, whole words
  // layout: parents [n] | first child [n] u16 | next sibling [n] u16 | union { table [(n+1)][row_bytes], lists 2 x [2n] u32 }
  int32_t* s_par = reinterpret_cast<int32_t*>(ro_smem);
  uint16_t* s_fc = reinterpret_cast<uint16_t*>(s_par + n);
  uint16_t* s_ns = s_fc + n;
  const size_t head = (size_t(n) * 8 + 15) & ~size_t(15);
  uint8_t* s_table = ro_smem + head;
  uint32_t* s_list_a = reinterpret_cast<uint32_t*>(ro_smem + head);
  uint32_t* s_list_b = s_list_a + 2 * n;
  bool bad = false;

  for (int i = tid; i < n; i += nthr) {
    int parent = parents[node0 + i];
    if (parent < -1 || parent >= i) {
      parent = -1;
      bad = true;
    }
    s_par[i] = parent;
    s_fc[i] = uint16_t(kNone);
    s_ns[i] = uint16_t(kNone);
  }
  {
    const int words = (n + 1) * (row_bytes >> 2);
    uint32_t* t32 = reinterpret_cast<uint32_t*>(s_table);
    for (int k = tid; k < words; k += nthr) t32[k] = 0u;
  }
  __syncthreads();

  // ---- 1a. per chunk: group equal parents; the last lane of a group enters itself in the table
  for (int c = warp; c < n_chunks; c += nwarps) {
    const int i = c * 32 + lane;
    const int key = i < n ? (s_par[i] < 0 ? n : s_par[i]) : -1 - lane;    // lanes past the end match nobody
    const uint32_t grp = __match_any_sync(0xffffffffu, key);
    if (i < n && lane == 31 - __clz(grp)) s_table[key * row_bytes + c] = uint8_t(lane + 1);
  }
  __syncthreads();
  // ---- 1b. previous sibling -> next-sibling and first-child links
  for (int c = warp; c < n_chunks; c += nwarps) {
    const int i = c * 32 + lane;
    const int key = i < n ? (s_par[i] < 0 ? n : s_par[i]) : -1 - lane;
    const uint32_t grp = __match_any_sync(0xffffffffu, key);
    if (i < n) {
      const uint32_t lower = grp & ((1u << lane) - 1u);
      int prev = -1;
      if (lower) {
        prev = c * 32 + (31 - __clz(lower));
      } else {
        const uint32_t* row = reinterpret_cast<const uint32_t*>(s_table + key * row_bytes);
        for (int wd = (c - 1) >> 2; wd >= 0 && c > 0; --wd) {
          uint32_t v = row[wd];
          const int keep = c - 4 * wd;                               // bytes of chunks < c
          if (keep < 4) v &= (1u << (8 * keep)) - 1u;
          if (v) {
            const int b = (31 - __clz(v)) >> 3;
            prev = (4 * wd + b) * 32 + int((v >> (8 * b)) & 0xFFu) - 1;
            break;
          }
        }
      }
      if (prev >= 0) s_ns[prev] = uint16_t(i);
      else if (key < n) s_fc[key] = uint16_t(i);
    }
  }
  __syncthreads();      // the table is dead from here on; its memory becomes the two lists

  // ---- 2. Euler tour: element i = enter(i), element n + i = exit(i); entry = next << 16 | weight
  for (int e = tid; e < 2 * n; e += nthr) {
    uint32_t nx, weight;
    if (e < n) {
      nx = s_fc[e] != kNone ? uint32_t(s_fc[e]) : uint32_t(n + e);
      weight = 1u;
    } else {
      const int i = e - n;
      nx = s_ns[i] != kNone ? uint32_t(s_ns[i]) : (s_par[i] >= 0 ? uint32_t(n + s_par[i]) : kNone);
      weight = 0u;
    }
    s_list_a[e] = (nx << 16) | weight;
  }
  __syncthreads();

  // ---- 3. list ranking: after round r an element points 2^r steps ahead and holds the weight of those steps
  uint32_t* cur = s_list_a;
  uint32_t* nxt = s_list_b;
  for (int span = 1; span < 2 * n; span <<= 1) {
    for (int e = tid; e < 2 * n; e += nthr) {
      const uint32_t a = cur[e];
      const uint32_t to = a >> 16;
      uint32_t r = a;
      if (to != kNone) {
        const uint32_t b = cur[to];
        r = (b & 0xFFFF0000u) | ((a & 0xFFFFu) + (b & 0xFFFFu));
      }
      nxt[e] = r;
    }
    __syncthreads();
    uint32_t* t = cur; cur = nxt; nxt = t;
  }

  grid_dependency_wait();     // outputs may still be in use by the kernel before this one in the stream
  if (bad && status) atomicCAS(status, 0, DYSPEC_ERR_BAD_TREE);
  for (int i = tid; i < n; i += nthr) {
    const int pre = n - int(cur[i] & 0xFFFFu);
    const int parent = s_par[i];
    if (new_of_old) new_of_old[node0 + i] = pre;
    if (order) order[node0 + pre] = i;
    if (new_parents) new_parents[node0 + pre] = parent >= 0 ? n - int(cur[parent] & 0xFFFFu) : -1;
  }
}

size_t dfs_reorder_smem_bytes(int max_n) {
  const size_t head = (size_t(max_n) * 8 + 15) & ~size_t(15);
  const size_t row_bytes = (((size_t(max_n) + 31) >> 5) + 3) & ~size_t(3);
  const size_t table = (size_t(max_n) + 1) * row_bytes;
  const size_t lists = size_t(max_n) * 16;
  return head + (table > lists ? table : lists);
}

cudaError_t launch_dfs_reorder(const int32_t* parents, const ReqInfo* reqs, int n_req, int single_n, int max_n,
                               int32_t* order, int32_t* new_of_old, int32_t* new_parents, int32_t* status,
                               cudaStream_t stream) {
  if (n_req <= 0 || max_n <= 0) return cudaSuccess;
  const size_t smem = dfs_reorder_smem_bytes(max_n);
  static DynSmemGrant grant;
  if (cudaError_t e = grant.ensure(dfs_reorder_kernel, smem); e != cudaSuccess) return e;
  int threads = ((max_n + 31) / 32) * 32;
  if (threads < 128) threads = 128;
  if (threads > 1024) threads = 1024;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(n_req));
  cfg.blockDim = dim3(unsigned(threads));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, dfs_reorder_kernel, parents, reqs, single_n, order, new_of_old, new_parents,
                                     status);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dyspec

// ---------------------------------------------------------------------------------------------------
// Block count of a packed tree mask (App. C.1, Table 5): the number of block x block tiles that hold
// at least one visible (query, key) pair.  One thread per tile of the lower triangle.
// ---------------------------------------------------------------------------------------------------
namespace dyspec {

__global__ void mask_block_count_kernel(const uint32_t* __restrict__ bits, int n, int W, int block,
                                        unsigned long long* __restrict__ count) {
  const int nb = (n + block - 1) / block;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  bool hit = false;
  if (idx < nb * nb) {
    const int rb = idx / nb, cb = idx - rb * nb;
    if (cb <= rb) {                       // ancestors have smaller indices: nothing above the diagonal
      const int wpb = block >> 5;         // words per block column
      uint32_t any = 0u;
      for (int r = rb * block; r < min(n, (rb + 1) * block); ++r)
        for (int w = 0; w < wpb; ++w) any |= bits[size_t(r) * W + cb * wpb + w];
      hit = any != 0u;
    }
  }
  const uint32_t votes = __ballot_sync(0xffffffffu, hit);
  if ((threadIdx.x & 31) == 0 && votes) atomicAdd(count, (unsigned long long)__popc(votes));
}

cudaError_t launch_mask_block_count(const uint32_t* bits, int n, int W, int block, unsigned long long* count,
                                    cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(count, 0, sizeof(unsigned long long), stream);
  if (e != cudaSuccess || n <= 0) return e;
  const int nb = (n + block - 1) / block;
  const int threads = 256, blocks = (nb * nb + threads - 1) / threads;
  mask_block_count_kernel<<<blocks, threads, 0, stream>>>(bits, n, W, block, count);
  return cudaGetLastError();
}

}  // namespace dyspec
