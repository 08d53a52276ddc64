// HBM-bound row movers between token order and expert-contiguous (padded) order.
//
// Both run token-major with one warp per token and 128-bit accesses, so each
// token row is read (scatter) or written (reduce) exactly once and every
// routed row is touched exactly once: (T + R) * d * 2 bytes, the algorithmic
// minimum.
//   scatter_rows: dst[prow(t*k+j), :] = src[t, :]      (gather of X / dY)
//   reduce_rows : out[t, :] = sum_j src[prow(t*k+j), :]  (Eq. 1 combine; dX)
// prow(s) = slot_to_row[s] + row_shift[e], e the expert whose segment holds the row (found by bisection of the
// offsets, which every block keeps in shared memory): the plan stores the permutation once, unpadded.
// The gate weights are already folded into the rows by the GEMM epilogues, so
// the combine is an unweighted fp32 sum in slot order (deterministic).
#include "common.cuh"

namespace grouter {

constexpr int MOVE_THREADS = 256;
constexpr int MOVE_WARPS = MOVE_THREADS / 32;
constexpr int SCATTER_SEG = 8;
constexpr int REDUCE_SEG = 8;

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_v4(void* p, const uint4& v) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

constexpr int MAX_EXPERTS = 1024;

// Offsets and row shifts into shared memory (E + 1 and E entries).
__device__ __forceinline__ void load_layout(const int32_t* __restrict__ offsets, const int32_t* __restrict__ row_shift, int E,
                                            int32_t* s_off, int32_t* s_shift) {
  for (int e = threadIdx.x; e <= E; e += blockDim.x) {
    s_off[e] = __ldg(offsets + e);
    if (e < E) s_shift[e] = __ldg(row_shift + e);
  }
  __syncthreads();
}
// Padded row of routed row `row`: its expert is the last e with offsets[e] <= row (never an expert without rows).
__device__ __forceinline__ int padded_row(int row, const int32_t* s_off, const int32_t* s_shift, int E) {
  int lo = 0, hi = E;  // invariant: s_off[lo] <= row < s_off[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s_off[mid] <= row) lo = mid; else hi = mid;
  }
  return row + s_shift[lo];
}

// The same for a row taken from the caller's slot_to_row; the checked build returns -1 (and sets the status bit) for a
// row outside [0, offsets[E]) or a padded row outside the buffers' rows_cap rows, and the movers skip such a slot.
__device__ __forceinline__ int checked_padded_row(int row, const int32_t* s_off, const int32_t* s_shift, int E, int rows_cap,
                                                  int32_t* status) {
  if (!GROUTER_CHECKED((unsigned)row < (unsigned)s_off[E], status)) return -1;
  const int prow = padded_row(row, s_off, s_shift, E);
  return GROUTER_CHECKED((unsigned)prow < (unsigned)rows_cap, status) ? prow : -1;
}

// SEG: 16-byte units each lane holds per pass; a warp moves SEG * 512 contiguous bytes of a row at a time.
template <int SEG>
__global__ void __launch_bounds__(MOVE_THREADS) scatter_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                                    const int32_t* __restrict__ slot_to_row,
                                                                    const int32_t* __restrict__ offsets,
                                                                    const int32_t* __restrict__ row_shift,
                                                                    const int32_t* __restrict__ pad_begin,
                                                                    const int32_t* __restrict__ pad_offsets, int T, int k, int d, int E,
                                                                    int rows_cap, int32_t* __restrict__ status) {
  __shared__ int32_t s_off[MAX_EXPERTS + 1], s_shift[MAX_EXPERTS];
  load_layout(offsets, row_shift, E, s_off, s_shift);
  const int lane = threadIdx.x & 31;
  const int gwarp = blockIdx.x * MOVE_WARPS + (threadIdx.x >> 5);
  const int nwarps = gridDim.x * MOVE_WARPS;
  const int units = d >> 3;  // 16-byte units per row
  for (int t = gwarp; t < T; t += nwarps) {
    const int my_prow = lane < k ? checked_padded_row(__ldg(slot_to_row + (size_t)t * k + lane), s_off, s_shift, E, rows_cap, status) : 0;
    const char* s = reinterpret_cast<const char*>(src + (size_t)t * d);
    for (int u0 = 0; u0 < units; u0 += 32 * SEG) {
      uint4 v[SEG];
#pragma unroll
      for (int i = 0; i < SEG; ++i) {
        const int u = u0 + i * 32 + lane;
        if (u < units) v[i] = ld_nc_v4(s + (size_t)u * 16);
      }
      for (int j = 0; j < k; ++j) {
        const int prow = __shfl_sync(0xffffffffu, my_prow, j);
        if (DEBUG_BOUNDS && prow < 0) continue;
        char* o = reinterpret_cast<char*>(dst + (size_t)prow * d);
#pragma unroll
        for (int i = 0; i < SEG; ++i) {
          const int u = u0 + i * 32 + lane;
          if (u < units) st_v4(o + (size_t)u * 16, v[i]);
        }
      }
    }
  }
  // zero the pad rows of every expert segment
  const uint4 z = make_uint4(0u, 0u, 0u, 0u);
  for (int e = gwarp; e < E; e += nwarps) {
    const int r0 = pad_begin[e], r1 = pad_offsets[e + 1];
    if (!GROUTER_CHECKED(r0 >= 0 && r1 <= rows_cap && r1 - r0 < ROW_TILE, status)) continue;
    for (int r = r0; r < r1; ++r) {
      char* o = reinterpret_cast<char*>(dst + (size_t)r * d);
      for (int u = lane; u < units; u += 32) st_v4(o + (size_t)u * 16, z);
    }
  }
}

__device__ __forceinline__ void acc_bf16x8(float (&a)[8], const uint4& v) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(p[i]);
    a[2 * i] += f.x;
    a[2 * i + 1] += f.y;
  }
}

// SEG: 16-byte units each lane accumulates per pass.  A warp reads SEG * 512 contiguous bytes of one routed row
// before it moves to the next row, so DRAM sees long sequential bursts instead of many interleaved short ones.
template <int SEG>
__global__ void __launch_bounds__(MOVE_THREADS) reduce_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ out,
                                                                   const int32_t* __restrict__ slot_to_row,
                                                                   const int32_t* __restrict__ offsets,
                                                                   const int32_t* __restrict__ row_shift, int T, int k, int d, int E,
                                                                   const float* __restrict__ dgate_part, int n_part, size_t part_stride,
                                                                   float* __restrict__ dgates, int32_t* __restrict__ status) {
  __shared__ int32_t s_off[MAX_EXPERTS + 1], s_shift[MAX_EXPERTS];
  load_layout(offsets, row_shift, E, s_off, s_shift);
  const int lane = threadIdx.x & 31;
  const int gwarp = blockIdx.x * MOVE_WARPS + (threadIdx.x >> 5);
  const int nwarps = gridDim.x * MOVE_WARPS;
  const int units = d >> 3;
  for (int t = gwarp; t < T; t += nwarps) {
    const int my_prow = lane < k ? checked_padded_row(__ldg(slot_to_row + (size_t)t * k + lane), s_off, s_shift, E, (int)part_stride, status) : 0;
    if (dgates != nullptr && lane < k) {
      float g = 0.f;
      for (int n = 0; n < n_part && (!DEBUG_BOUNDS || my_prow >= 0); ++n) g += dgate_part[(size_t)n * part_stride + my_prow];
      dgates[(size_t)t * k + lane] = g;
    }
    char* o = reinterpret_cast<char*>(out + (size_t)t * d);
    for (int u0 = 0; u0 < units; u0 += 32 * SEG) {
      float acc[SEG][8];
#pragma unroll
      for (int i = 0; i < SEG; ++i)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[i][c] = 0.f;
      for (int j = 0; j < k; ++j) {          // slot order: the sum is deterministic
        const int prow = __shfl_sync(0xffffffffu, my_prow, j);
        if (DEBUG_BOUNDS && prow < 0) continue;
        const char* s = reinterpret_cast<const char*>(src + (size_t)prow * d);
        uint4 v[SEG];
#pragma unroll
        for (int i = 0; i < SEG; ++i) {
          const int u = u0 + i * 32 + lane;
          if (u < units) v[i] = ld_nc_v4(s + (size_t)u * 16);
        }
#pragma unroll
        for (int i = 0; i < SEG; ++i) {
          const int u = u0 + i * 32 + lane;
          if (u < units) acc_bf16x8(acc[i], v[i]);
        }
      }
#pragma unroll
      for (int i = 0; i < SEG; ++i) {
        const int u = u0 + i * 32 + lane;
        if (u < units) {
          uint4 v;
          __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
          for (int c = 0; c < 4; ++c) p[c] = __floats2bfloat162_rn(acc[i][2 * c], acc[i][2 * c + 1]);
          st_v4(o + (size_t)u * 16, v);
        }
      }
    }
  }
}

// out = bf16(in), eight elements per thread and pass (the last step of the fused combine).
__global__ void __launch_bounds__(MOVE_THREADS) cast_rows_kernel(const float4* __restrict__ in, uint4* __restrict__ out, size_t n8) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
    const float4 a = in[2 * i], b = in[2 * i + 1];
    uint4 v;
    __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
    p[0] = __floats2bfloat162_rn(a.x, a.y);
    p[1] = __floats2bfloat162_rn(a.z, a.w);
    p[2] = __floats2bfloat162_rn(b.x, b.y);
    p[3] = __floats2bfloat162_rn(b.z, b.w);
    out[i] = v;
  }
}

cudaError_t launch_cast_rows(grouter_ctx* ctx, const float* in, __nv_bfloat16* out, size_t n, cudaStream_t st) {
  const size_t n8 = n / 8;
  size_t want = (n8 + MOVE_THREADS - 1) / MOVE_THREADS;
  const size_t cap = (size_t)ctx->num_sms * 8;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  cast_rows_kernel<<<(unsigned)want, MOVE_THREADS, 0, st>>>(reinterpret_cast<const float4*>(in), reinterpret_cast<uint4*>(out), n8);
  return cudaGetLastError();
}

__global__ void idle_kernel(unsigned long long nanoseconds) {
  unsigned long long t0, t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  do {
    __nanosleep(2000);
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  } while (t - t0 < nanoseconds);
}

cudaError_t launch_idle(int microseconds, cudaStream_t st) {
  if (microseconds > 1000000) microseconds = 1000000;
  idle_kernel<<<1, 1, 0, st>>>((unsigned long long)microseconds * 1000ull);
  return cudaGetLastError();
}

static int mover_grid(const grouter_ctx* ctx, int T) {
  const int want = (T + MOVE_WARPS - 1) / MOVE_WARPS;
  const int cap = ctx->num_sms * 8;
  return want < cap ? (want < 1 ? 1 : want) : cap;
}

cudaError_t launch_scatter_rows(grouter_ctx* ctx, const __nv_bfloat16* src, __nv_bfloat16* dst, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  scatter_rows_kernel<SCATTER_SEG><<<mover_grid(ctx, ctx->T_act), MOVE_THREADS, 0, st>>>(src, dst, ctx->pp.slot_to_row, ctx->pp.offsets, ctx->pp.row_shift,
                                                                      ctx->pp.pad_begin, ctx->pp.pad_offsets, ctx->T_act, dm.k, dm.d, dm.E_tgt, (int)ctx->R_pad_max, ctx->pp.status);
  return cudaGetLastError();
}

cudaError_t launch_reduce_rows(grouter_ctx* ctx, const __nv_bfloat16* src, __nv_bfloat16* out, const float* dgate_part, int n_part,
                               float* dgates, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  reduce_rows_kernel<REDUCE_SEG><<<mover_grid(ctx, ctx->T_act), MOVE_THREADS, 0, st>>>(src, out, ctx->pp.slot_to_row, ctx->pp.offsets, ctx->pp.row_shift, ctx->T_act, dm.k, dm.d,
                                                                     dm.E_tgt, dgate_part, n_part, (size_t)ctx->R_pad_max, dgates, ctx->pp.status);
  return cudaGetLastError();
}

}  // namespace grouter
