// Expert parallelism on top of the routing plan (the paper's setting: section "Decoupling Communication
// Optimization"; appendix "Efficiency Experiment Detail").
//
// Experts are split over ranks, tokens stay where they are, and routed rows travel: rank r sends the rows of its
// tokens that chose an expert of rank p to p, p runs its experts on what it received and sends the results back.
// Because the routing is known before the step (it comes from the cache, not from the layer), every rank can work out
// all per-peer row counts from the per-rank expert histograms alone: no size exchange and no host synchronisation
// sits between the plan and the transfer.
//
// What lives here is the part around the transfer; the transfer itself is the caller's collective (NCCL all-to-all
// with the split sizes computed below) into buffers in the receiving GPU's own memory.  Nothing in this library reads
// another GPU's memory.
//   grouter_ep_relabel_host   renumbers the experts so that every rank owns a contiguous range (then the rows for
//                             one peer are a contiguous range of the sender's expert-ordered rows: no extra gather)
//   grouter_ep_layout_host    send / receive counts and offsets per peer, and the (source rank, local expert) segments
//                             of the rows a rank receives
//   grouter_ep_expand_ids     local expert id of every received row (one id per row): the receiving rank plans and
//                             runs its experts on the received rows as a k = 1 problem with unit gates
//   grouter_ep_dispatch_rows  rows[slot_to_row[s], :] = (gate_s) * src[token of s, :]     sender, before the transfer
//   grouter_ep_combine_rows   out[t, :] = sum_j (gate) * rows[slot_to_row[t*k+j], :],     sender, after the return
//                             dgates[t, j] = <dY[t, :], rows[slot_to_row[t*k+j], :]>
// Forward:  dispatch X (no gates) -> transfer -> experts (unit gates) -> transfer back -> combine with the gates (Eq. 1).
// Backward: dispatch dY with the gates -> transfer -> experts' backward -> transfer back -> combine without gates = dX;
//           dgates from the forward's returned rows and dY.
#include "common.cuh"

namespace grouter {

constexpr int EP_THREADS = 256;
constexpr int EP_WARPS = EP_THREADS / 32;

__device__ __forceinline__ uint4 ep_ld_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void ep_unpack8(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
__device__ __forceinline__ uint4 ep_pack8(const float (&f)[8]) {
  uint4 v;
  __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return v;
}
__device__ __forceinline__ float ep_gate(const void* gates, int gate_is_f32, size_t slot) {
  if (gate_is_f32) return __ldg(reinterpret_cast<const float*>(gates) + slot);
  return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(gates)[slot]);
}

// One warp per token, 16-byte accesses: the token's row is read once and written (scaled by the slot's gate when gates
// are given) to the k rows its slots own in the expert-ordered, unpadded row buffer.
__global__ void __launch_bounds__(EP_THREADS) ep_dispatch_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ rows,
                                                                      const int32_t* __restrict__ slot_to_row, const void* __restrict__ gates,
                                                                      int gate_is_f32, int T, int k, int d) {
  const int lane = threadIdx.x & 31;
  const int gwarp = blockIdx.x * EP_WARPS + (threadIdx.x >> 5), nwarps = gridDim.x * EP_WARPS;
  const int units = d >> 3;
  for (int t = gwarp; t < T; t += nwarps) {
    const int my_row = lane < k ? __ldg(slot_to_row + (size_t)t * k + lane) : 0;
    const float my_gate = (gates != nullptr && lane < k) ? ep_gate(gates, gate_is_f32, (size_t)t * k + lane) : 1.f;
    const char* s = reinterpret_cast<const char*>(src + (size_t)t * d);
    for (int u = lane; u < units; u += 32) {
      const uint4 v = ep_ld_v4(s + (size_t)u * 16);
      float f[8];
      if (gates != nullptr) ep_unpack8(v, f);
      for (int j = 0; j < k; ++j) {
        const int row = __shfl_sync(0xffffffffu, my_row, j);
        uint4 o = v;
        if (gates != nullptr) {
          const float g = __shfl_sync(0xffffffffu, my_gate, j);
          float h[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) h[i] = g * f[i];
          o = ep_pack8(h);
        }
        *reinterpret_cast<uint4*>(reinterpret_cast<char*>(rows + (size_t)row * d) + (size_t)u * 16) = o;
      }
    }
  }
}

// One warp per token: fp32 sum, in slot order, of the token's k returned rows (each times its gate when gates are
// given), rounded once to bf16; and / or the k inner products of the rows with dY[t, :].
__global__ void __launch_bounds__(EP_THREADS) ep_combine_rows_kernel(const __nv_bfloat16* __restrict__ rows, const int32_t* __restrict__ slot_to_row,
                                                                     const void* __restrict__ gates, int gate_is_f32,
                                                                     __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dY,
                                                                     float* __restrict__ dgates, int T, int k, int d) {
  const int lane = threadIdx.x & 31;
  const int gwarp = blockIdx.x * EP_WARPS + (threadIdx.x >> 5), nwarps = gridDim.x * EP_WARPS;
  const int units = d >> 3;
  for (int t = gwarp; t < T; t += nwarps) {
    const int my_row = lane < k ? __ldg(slot_to_row + (size_t)t * k + lane) : 0;
    const float my_gate = (gates != nullptr && lane < k) ? ep_gate(gates, gate_is_f32, (size_t)t * k + lane) : 1.f;
    float my_dot = 0.f;       // lane j ends up with <dY[t], row of slot j>
    for (int u = lane; u < units + lane; u += 32) {      // every lane runs the same number of rounds (shuffles inside)
      const bool have = u < units;
      float acc[8], dy[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = dy[i] = 0.f;
      if (have && dY != nullptr) ep_unpack8(ep_ld_v4(reinterpret_cast<const char*>(dY + (size_t)t * d) + (size_t)u * 16), dy);
      for (int j = 0; j < k; ++j) {
        const int row = __shfl_sync(0xffffffffu, my_row, j);
        const float g = __shfl_sync(0xffffffffu, my_gate, j);
        float f[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = 0.f;
        if (have) ep_unpack8(ep_ld_v4(reinterpret_cast<const char*>(rows + (size_t)row * d) + (size_t)u * 16), f);
        float part = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          acc[i] += g * f[i];
          part += dy[i] * f[i];
        }
        if (dgates != nullptr) {
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
          if (lane == j) my_dot += part;
        }
      }
      if (have && out != nullptr) *reinterpret_cast<uint4*>(reinterpret_cast<char*>(out + (size_t)t * d) + (size_t)u * 16) = ep_pack8(acc);
    }
    if (dgates != nullptr && lane < k) dgates[(size_t)t * k + lane] = my_dot;
  }
}

// Local expert of every received row: the rows arrive as n_seg = (source ranks) x (local experts) segments, source
// rank outermost; seg_offsets is their exclusive prefix.  A row's segment is found by bisection.
__global__ void __launch_bounds__(EP_THREADS) ep_expand_ids_kernel(const int32_t* __restrict__ seg_offsets, int n_seg, int n_local,
                                                                   uint8_t* __restrict__ idx_u8, int32_t* __restrict__ idx_i32) {
  const int n_rows = __ldg(seg_offsets + n_seg);
  for (int r = blockIdx.x * EP_THREADS + threadIdx.x; r < n_rows; r += gridDim.x * EP_THREADS) {
    int lo = 0, hi = n_seg;   // invariant: seg_offsets[lo] <= r < seg_offsets[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (__ldg(seg_offsets + mid) <= r) lo = mid; else hi = mid;
    }
    const int e = lo % n_local;
    if (idx_u8) idx_u8[r] = (uint8_t)e;
    else idx_i32[r] = e;
  }
}

}  // namespace grouter

using namespace grouter;

extern "C" {

int grouter_ep_relabel_host(int32_t E, int32_t world, const int32_t* expert_rank, int32_t* relabel, int32_t* first_expert) {
  if (!expert_rank || !relabel || !first_expert || E < 1 || world < 1) return GROUTER_ERR_INVALID_ARG;
  for (int e = 0; e < E; ++e)
    if (expert_rank[e] < 0 || expert_rank[e] >= world) return GROUTER_ERR_INVALID_ARG;
  int next = 0;
  for (int r = 0; r < world; ++r) {
    first_expert[r] = next;
    for (int e = 0; e < E; ++e)
      if (expert_rank[e] == r) relabel[e] = next++;
  }
  first_expert[world] = next;
  return GROUTER_OK;
}

int grouter_ep_layout_host(int32_t world, int32_t rank, int32_t E, const int32_t* first_expert, const int32_t* counts_all,
                           int32_t* send_counts, int32_t* send_offsets, int32_t* recv_counts, int32_t* recv_offsets,
                           int32_t* recv_seg_offsets) {
  if (!first_expert || !counts_all || !send_counts || !send_offsets || !recv_counts || !recv_offsets || !recv_seg_offsets)
    return GROUTER_ERR_INVALID_ARG;
  if (world < 1 || rank < 0 || rank >= world || E < 1) return GROUTER_ERR_INVALID_ARG;
  if (first_expert[0] != 0 || first_expert[world] != E) return GROUTER_ERR_INVALID_ARG;
  for (int r = 0; r < world; ++r)
    if (first_expert[r] > first_expert[r + 1]) return GROUTER_ERR_INVALID_ARG;
  const int32_t* mine = counts_all + (size_t)rank * E;
  const int e0 = first_expert[rank], n_local = first_expert[rank + 1] - e0;
  int64_t so = 0, ro = 0;
  for (int p = 0; p < world; ++p) {
    int64_t s = 0, r = 0;
    for (int e = first_expert[p]; e < first_expert[p + 1]; ++e) s += mine[e];          // my rows for p's experts
    for (int e = 0; e < n_local; ++e) {
      const int32_t c = counts_all[(size_t)p * E + e0 + e];                              // p's rows for my experts
      if (c < 0) return GROUTER_ERR_INVALID_ARG;
      recv_seg_offsets[(size_t)p * n_local + e] = (int32_t)(ro + r);
      r += c;
    }
    if (so + s > 2147483647ll || ro + r > 2147483647ll) return GROUTER_ERR_UNSUPPORTED;
    send_counts[p] = (int32_t)s;
    send_offsets[p] = (int32_t)so;
    recv_counts[p] = (int32_t)r;
    recv_offsets[p] = (int32_t)ro;
    so += s;
    ro += r;
  }
  send_offsets[world] = (int32_t)so;
  recv_offsets[world] = (int32_t)ro;
  recv_seg_offsets[(size_t)world * n_local] = (int32_t)ro;
  return GROUTER_OK;
}

int grouter_ep_expand_ids(const int32_t* seg_offsets, int32_t n_seg, int32_t n_local, int32_t n_rows, int32_t idx_dtype, void* idx_out,
                          void* stream) {
  if (!seg_offsets || !idx_out || n_seg < 1 || n_local < 1 || n_seg % n_local || n_rows < 0) return GROUTER_ERR_INVALID_ARG;
  if (idx_dtype != GROUTER_IDX_U8 && idx_dtype != GROUTER_IDX_I32) return GROUTER_ERR_INVALID_ARG;
  if (idx_dtype == GROUTER_IDX_U8 && n_local > 256) return GROUTER_ERR_UNSUPPORTED;
  if (n_rows == 0) return GROUTER_OK;
  int grid = (n_rows + EP_THREADS - 1) / EP_THREADS;
  if (grid > 1184) grid = 1184;
  ep_expand_ids_kernel<<<grid, EP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      seg_offsets, n_seg, n_local, idx_dtype == GROUTER_IDX_U8 ? static_cast<uint8_t*>(idx_out) : nullptr,
      idx_dtype == GROUTER_IDX_I32 ? static_cast<int32_t*>(idx_out) : nullptr);
  return cudaGetLastError() == cudaSuccess ? GROUTER_OK : GROUTER_ERR_CUDA;
}

static int ep_grid(const grouter_ctx* ctx) {
  const int want = (ctx->T_act + EP_WARPS - 1) / EP_WARPS, cap = ctx->num_sms * 8;
  return want < cap ? (want < 1 ? 1 : want) : cap;
}

int grouter_ep_dispatch_rows(grouter_ctx* ctx, const void* src, const void* gates, void* rows, void* stream) {
  if (!ctx || !src || !rows) return GROUTER_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(rows) | reinterpret_cast<uintptr_t>(gates)) & 15u) return GROUTER_ERR_MISALIGNED;
  if (!ctx->planned) return GROUTER_ERR_INVALID_STATE;
  const grouter_dims& dm = ctx->dims;
  ep_dispatch_rows_kernel<<<ep_grid(ctx), EP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(src), static_cast<__nv_bfloat16*>(rows), ctx->pp.slot_to_row, gates,
      dm.gate_dtype == GROUTER_GATE_F32, ctx->T_act, dm.k, dm.d);
  return cudaGetLastError() == cudaSuccess ? GROUTER_OK : GROUTER_ERR_CUDA;
}

int grouter_ep_combine_rows(grouter_ctx* ctx, const void* rows, const void* gates, void* out, const void* dY, float* dgates, void* stream) {
  if (!ctx || !rows || (!out && !dgates) || (dgates && !dY)) return GROUTER_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(rows) | reinterpret_cast<uintptr_t>(gates) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(dY) |
       reinterpret_cast<uintptr_t>(dgates)) & 15u)
    return GROUTER_ERR_MISALIGNED;
  if (!ctx->planned) return GROUTER_ERR_INVALID_STATE;
  const grouter_dims& dm = ctx->dims;
  ep_combine_rows_kernel<<<ep_grid(ctx), EP_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(rows), ctx->pp.slot_to_row, gates, dm.gate_dtype == GROUTER_GATE_F32,
      static_cast<__nv_bfloat16*>(out), static_cast<const __nv_bfloat16*>(dY), dgates, ctx->T_act, dm.k, dm.d);
  return cudaGetLastError() == cudaSuccess ? GROUTER_OK : GROUTER_ERR_CUDA;
}

}  // extern "C"
