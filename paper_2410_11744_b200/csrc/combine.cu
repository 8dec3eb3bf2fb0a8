// Split-KV combine: merges the fp32 partials (O_s, m_s, l_s) that the attention kernels wrote for a
// query tile whose key range was cut into several work items, and writes the final bf16 rows:
//   m = max_s m_s,  w_s = 2^(m_s - m),  out = (sum_s w_s O_s) / (sum_s w_s l_s)
// (m_s are running maxima of scale*log2(e)*score, so the weights are powers of two of differences).
// One warp per packed query row; lanes cover the head dimension with 16- or 8-byte accesses.
#include "common.cuh"

namespace dyspec {

template <int D>
__global__ void __launch_bounds__(256)
combine_kernel(const AttnParams p, int bm) {
  // Launched early (programmatic dependent launch), and lets its own successor start early too: the next
  // call's kernels wait for this grid's completion themselves before they touch anything it reads or writes.
  trigger_dependents();
  grid_dependency_wait();   // the partials must be complete
  const int rows_per_block = 8;
  const int blocks_per_group = bm / rows_per_block;
  const GroupInfo gi = p.groups[blockIdx.x / blocks_per_group];
  const int r = (blockIdx.x % blocks_per_group) * rows_per_block + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const ReqInfo rq = p.reqs[gi.req];
  const int row = gi.row0 + r;
  if (row >= rq.n_nodes * p.group_size) return;

  const float* base = p.partial + size_t(gi.slot0) * p.slot_floats;
  float m = -INFINITY;
  for (int s = 0; s < gi.n_splits; ++s) m = fmaxf(m, base[size_t(s) * p.slot_floats + bm * D + r]);
  const float ref = m == -INFINITY ? 0.f : m;

  constexpr int V = D / 32;  // floats per lane
  float acc[V];
#pragma unroll
  for (int k = 0; k < V; ++k) acc[k] = 0.f;
  float l = 0.f;
  for (int s = 0; s < gi.n_splits; ++s) {
    const float* slot = base + size_t(s) * p.slot_floats;
    const float w = fast_exp2(slot[bm * D + r] - ref);
    l += w * slot[bm * D + bm + r];
    if constexpr (V == 4) {
      const float4 v = *reinterpret_cast<const float4*>(slot + r * D + lane * 4);
      acc[0] += w * v.x; acc[1] += w * v.y; acc[2] += w * v.z; acc[3] += w * v.w;
    } else {
      const float2 v = *reinterpret_cast<const float2*>(slot + r * D + lane * 2);
      acc[0] += w * v.x; acc[1] += w * v.y;
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  const int node = row >> p.log2_g;
  const int head = gi.kv_head * p.group_size + (row & (p.group_size - 1));
  __nv_bfloat16* out = p.out + (size_t(rq.node0 + node) * p.n_q_heads + head) * D;
  if constexpr (V == 4) {
    uint2 o;
    o.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
    o.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
    *reinterpret_cast<uint2*>(out + lane * 4) = o;
  } else {
    *reinterpret_cast<uint32_t*>(out + lane * 2) = pack_bf16x2(acc[0] * inv, acc[1] * inv);
  }
}

cudaError_t launch_combine(int head_dim, int bm, int n_split_groups, const AttnParams& p, cudaStream_t stream) {
  if (n_split_groups <= 0) return cudaSuccess;
  const int blocks = n_split_groups * (bm / 8);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(blocks));
  cfg.blockDim = dim3(256u);
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (head_dim == 128) e = cudaLaunchKernelEx(&cfg, combine_kernel<128>, p, bm);
  else e = cudaLaunchKernelEx(&cfg, combine_kernel<64>, p, bm);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dyspec
