// Router head that writes the pre-dispatch routing cache (the step before the routing plan).
//
//   r(x) = g(TopK(s(x), k))                      Eq. 2, section "Mixture-of-Experts"
//   s(x) = W~_s^T h,   W~_s = W_s M              section "Expert Folding", Matrix Folding Implementation
//
// The fold is applied to the scores, before TopK: by linearity  h^T (W_s M) = (h^T W_s) M,  so the source scores come
// from one GEMM on the router's own bf16 score layer (the tcgen05 core, fp32 out) and every target expert's score is the
// sum of the source scores mapped to it.  That sum runs over ascending source id through a per-target list built once
// per call, so the result does not depend on thread timing.  One warp then handles one token: k rounds of a warp-wide
// arg-max (higher score first, lower id on equal scores), softmax over the kept scores or a sigmoid of each, and the
// record of the cache: k uint8 ids and k bfloat16 coefficients (appendix "Efficiency Experiment Detail").
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"

namespace grouter {

constexpr int ROUTE_THREADS = 256;
constexpr int ROUTE_WARPS = ROUTE_THREADS / 32;
constexpr int ROUTE_MAX_E = 256;              // uint8 ids
constexpr int ROUTE_PER_LANE = ROUTE_MAX_E / 32;

// Sources of every target in ascending order: grp_off[E_tgt+1], grp_src[E_src] (a stable counting sort by target,
// one block).  A fold target outside [0, E_tgt) counts as target 0 and raises STATUS_BAD_INDEX.
__global__ void __launch_bounds__(ROUTE_THREADS) route_groups_kernel(const int32_t* __restrict__ fold_map, int E_src, int E_tgt,
                                                                     int32_t* __restrict__ grp_off, int32_t* __restrict__ grp_src,
                                                                     int32_t* __restrict__ status) {
  __shared__ int32_t s_cnt[ROUTE_MAX_E + 1];
  const int tid = threadIdx.x;
  for (int j = tid; j <= E_tgt; j += ROUTE_THREADS) s_cnt[j] = 0;
  __syncthreads();
  if (tid == 0) {   // E_src is a few hundred at most: one thread keeps the order trivially stable
    for (int i = 0; i < E_src; ++i) {
      int j = fold_map ? fold_map[i] : i;
      if ((unsigned)j >= (unsigned)E_tgt) {
        atomicOr(status, STATUS_BAD_INDEX);
        j = 0;
      }
      s_cnt[j + 1] += 1;
    }
    for (int j = 0; j < E_tgt; ++j) s_cnt[j + 1] += s_cnt[j];
    for (int j = 0; j <= E_tgt; ++j) grp_off[j] = s_cnt[j];
    for (int i = 0; i < E_src; ++i) {
      int j = fold_map ? fold_map[i] : i;
      if ((unsigned)j >= (unsigned)E_tgt) j = 0;
      grp_src[s_cnt[j]++] = i;
    }
  }
}

__global__ void __launch_bounds__(ROUTE_THREADS) route_topk_kernel(const float* __restrict__ S_src, const int32_t* __restrict__ grp_off,
                                                                   const int32_t* __restrict__ grp_src, int T, int E_src, int E_tgt, int k,
                                                                   int norm, uint8_t* __restrict__ idx_out,
                                                                   __nv_bfloat16* __restrict__ gates_out, float* __restrict__ scores_out) {
  __shared__ float s_src[ROUTE_WARPS][ROUTE_MAX_E * 4];   // source scores of the warp's token (E_src <= 1024)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nwarps = gridDim.x * ROUTE_WARPS;
  float* mine = s_src[warp];
  for (int t = blockIdx.x * ROUTE_WARPS + warp; t < T; t += nwarps) {
    const float* row = S_src + (size_t)t * E_src;
    for (int i = lane; i < E_src; i += 32) mine[i] = __ldcs(row + i);
    __syncwarp();
    // folded scores of targets lane, lane + 32, ...
    float v[ROUTE_PER_LANE];
#pragma unroll
    for (int q = 0; q < ROUTE_PER_LANE; ++q) {
      const int j = lane + 32 * q;
      float acc = -INFINITY;
      if (j < E_tgt) {
        if (grp_off == nullptr) {       // no fold: target j is source j
          acc = mine[j];
        } else {
          acc = 0.f;
          const int b = __ldg(grp_off + j), e = __ldg(grp_off + j + 1);
          for (int p = b; p < e; ++p) acc += mine[__ldg(grp_src + p)];
        }
        if (scores_out) scores_out[(size_t)t * E_tgt + j] = acc;
      }
      v[q] = acc;
    }
    __syncwarp();
    // k rounds of warp arg-max: higher score first, lower id on equal scores
    float my_score = 0.f;
    int my_id = 0;
    for (int r = 0; r < k; ++r) {
      float best = -INFINITY;
      int best_j = 0x7fffffff;
#pragma unroll
      for (int q = 0; q < ROUTE_PER_LANE; ++q) {
        const int j = lane + 32 * q;
        if (j < E_tgt && (v[q] > best || (v[q] == best && j < best_j))) {
          best = v[q];
          best_j = j;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oj = __shfl_xor_sync(0xffffffffu, best_j, o);
        if (ob > best || (ob == best && oj < best_j)) {
          best = ob;
          best_j = oj;
        }
      }
      if ((best_j & 31) == lane) {      // the owner retires the winner
#pragma unroll
        for (int q = 0; q < ROUTE_PER_LANE; ++q)
          if (q == (best_j >> 5)) v[q] = -INFINITY;
      }
      if (lane == r) {
        my_score = best;
        my_id = best_j;
      }
    }
    // g over the kept scores (lane r < k holds the r-th; lane 0 holds the largest)
    float coef;
    if (norm == 0) {
      const float top = __shfl_sync(0xffffffffu, my_score, 0);
      const float e = lane < k ? expf(my_score - top) : 0.f;
      float sum = e;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      coef = e / sum;
    } else {
      coef = 1.f / (1.f + expf(-my_score));
    }
    if (lane < k) {
      idx_out[(size_t)t * k + lane] = (uint8_t)my_id;
      gates_out[(size_t)t * k + lane] = __float2bfloat16_rn(coef);
    }
    __syncwarp();
  }
}

// ------------------------------------------------------------------------------------------------------------------
// One-kernel form (E_src <= 256, k <= 8): score GEMM, fold, top-k, normalisation and the cache record in one launch.
//
// A CTA owns 128 tokens.  Warp 0 streams the tokens' hidden states and the score layer through a 3-stage ring of
// 128-byte-swizzled tiles (TMA), warp 1 issues the MMAs (one CTA, M = 128, N = the source experts rounded up to 16)
// into a TMEM accumulator of up to 256 columns, and each thread of warps 2-5 then owns one token: it reads its row of
// source scores from TMEM 32 columns at a time, sums them per target expert and keeps the best eight (score, id)
// pairs in a sorted register list.  With a fold map the score layer's rows are first gathered into target order
// (route_permute_ws_kernel), so that a target's sources are neighbouring accumulator columns in ascending source id:
// the per-target sums then run over contiguous columns, in the same order as in the two-kernel form.  The fp32
// [T, E_src] score matrix never goes to memory.
// ------------------------------------------------------------------------------------------------------------------
constexpr int RF_THREADS = 192;            // warp 0 producer, warp 1 issuer, warps 2-5 one thread per token
constexpr int RF_STAGES = 3;
constexpr int RF_BM = 128, RF_BK = 64;
constexpr int RF_A_BYTES = RF_BM * RF_BK * 2;      // 16 KB
constexpr int RF_MAX_N = 256;
constexpr int RF_KEEP = 8;                 // length of the per-token best list (k <= RF_KEEP)
constexpr uint32_t RF_TMEM_COLS = 256;

// Rows of the score layer gathered into target order: W_perm[p, :] = W_s[grp_src[p], :].
__global__ void __launch_bounds__(256) route_permute_ws_kernel(const uint4* __restrict__ W_s, const int32_t* __restrict__ grp_src, int E_src,
                                                               int units, uint4* __restrict__ W_perm) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < E_src * units; i += gridDim.x * blockDim.x) {
    const int p = i / units, u = i - p * units;
    W_perm[i] = W_s[(size_t)grp_src[p] * units + u];
  }
}

struct RouteFusedParams {
  int T, d_h, E_src, E_tgt, k, norm, nb;          // nb: MMA N (E_src rounded up to a multiple of 16)
  const int32_t* grp_off;                          // [E_tgt + 1] first accumulator column of every target, or null (no fold)
  uint8_t* idx_out;
  __nv_bfloat16* gates_out;
  float* scores_out;
  int32_t* status;
  unsigned long long wait_limit_ns;
};

__global__ void __launch_bounds__(RF_THREADS) route_fused_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW,
                                                                 const RouteFusedParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const int b_bytes = p.nb * RF_BK * 2;
  const int stage_bytes = RF_A_BYTES + b_bytes;        // nb is a multiple of 16, so every tile starts on a 1024-byte boundary
  const uint32_t bar_base = smem_base + RF_STAGES * stage_bytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (RF_STAGES + s); };
  const uint32_t tfull_bar = bar_base + 8u * (2 * RF_STAGES);
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  __shared__ int32_t s_grp[RF_MAX_N + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < RF_STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(tfull_bar, 1);
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmH);
    ptx::prefetch_tensormap(&tmW);
  }
  if (p.grp_off != nullptr)
    for (int j = threadIdx.x; j <= p.E_tgt; j += RF_THREADS) s_grp[j] = __ldg(p.grp_off + j);
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&s_tmem_base), RF_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;
  const int row0 = blockIdx.x * RF_BM;
  const int nk = (p.d_h + RF_BK - 1) / RF_BK;

  if (warp == 0) {
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int ks = 0; ks < nk; ++ks) {
        if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, p.wait_limit_ns)) break;
        const uint32_t sa = smem_base + s * stage_bytes, sb = sa + RF_A_BYTES;
        ptx::mbar_arrive_expect_tx(full_bar(s), (uint32_t)(RF_A_BYTES + b_bytes));
        ptx::tma_load_2d(sa, &tmH, full_bar(s), ks * RF_BK, row0);       // box {64 k, 128 tokens}; rows beyond T read as zeros
        ptx::tma_load_2d(sb, &tmW, full_bar(s), ks * RF_BK, 0);          // box {64 k, nb experts}; rows beyond E_src read as zeros
        if (++s == RF_STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_bf16(RF_BM, p.nb, false, false);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int ks = 0; ks < nk && ok; ++ks) {
        if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, p.wait_limit_ns)) {
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        const uint32_t sa = smem_base + s * stage_bytes, sb = sa + RF_A_BYTES;
#pragma unroll
        for (int kk = 0; kk < RF_BK / 16; ++kk) {
          // K-major, 128-byte swizzle: 8-row groups 1024 B apart; 16 K-elements = 32 B further along the row
          const uint64_t da = ptx::make_smem_desc_sw128(sa + kk * 32, 16, 1024);
          const uint64_t db = ptx::make_smem_desc_sw128(sb + kk * 32, 16, 1024);
          ptx::umma_bf16(tmem_base, da, db, idesc, (ks | kk) != 0 ? 1u : 0u);
        }
        ptx::umma_commit(empty_bar(s));
        if (++s == RF_STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
      if (ok) ptx::umma_commit(tfull_bar);
    }
    __syncwarp();
  } else {
    // ===================== one thread per token =====================
    const int quad = warp & 3;                       // the TMEM lane quadrant this warp may read
    const int t = row0 + quad * 32 + lane;
    const bool have = t < p.T;
    if (ptx::mbar_wait_bounded(tfull_bar, 0u, abort_flag, p.wait_limit_ns)) {
      ptx::tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
      float bv[RF_KEEP];
      int bi[RF_KEEP];
#pragma unroll
      for (int q = 0; q < RF_KEEP; ++q) {
        bv[q] = -INFINITY;
        bi[q] = 0x7fffffff;
      }
      // a candidate arrives with an id larger than every id seen so far: on equal scores the earlier one stays ahead
      auto offer = [&](float v, int j) {
        if (v > bv[RF_KEEP - 1]) {
#pragma unroll
          for (int q = RF_KEEP - 1; q >= 0; --q) {
            const bool shift = q > 0 && v > bv[q > 0 ? q - 1 : 0];
            const bool here = !shift && v > bv[q];
            const float nv = shift ? bv[q > 0 ? q - 1 : 0] : (here ? v : bv[q]);
            const int ni = shift ? bi[q > 0 ? q - 1 : 0] : (here ? j : bi[q]);
            bv[q] = nv;
            bi[q] = ni;
          }
        }
      };
      const bool folded = p.grp_off != nullptr;
      int j = 0;                    // current target
      int next_edge = folded ? s_grp[1] : 1;
      float acc = 0.f;
      float* srow = (p.scores_out != nullptr && have) ? p.scores_out + (size_t)t * p.E_tgt : nullptr;
      for (int c0 = 0; c0 < p.nb; c0 += 32) {        // nb is a multiple of 16: the last chunk may be half used
        uint32_t r[32];
        if (c0 + 32 <= p.nb) {
          ptx::tmem_ld32(t_row + c0, r);
        } else {
          uint32_t h[16];
          ptx::tmem_ld16(t_row + c0, h);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            r[i] = h[i];
            r[16 + i] = 0u;
          }
        }
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int c = c0 + i;
          if (c < p.E_src) {                          // uniform over the warp
            if (!folded) {
              const float v = __uint_as_float(r[i]);
              if (srow) srow[c] = v;
              offer(v, c);
            } else {
              while (c >= next_edge && j < p.E_tgt) {   // targets whose columns are complete (also targets without sources)
                if (srow) srow[j] = acc;
                offer(acc, j);
                acc = 0.f;
                ++j;
                next_edge = s_grp[min(j + 1, p.E_tgt)];
              }
              acc += __uint_as_float(r[i]);
            }
          }
        }
      }
      if (folded) {
        while (j < p.E_tgt) {
          if (srow) srow[j] = acc;
          offer(acc, j);
          acc = 0.f;
          ++j;
        }
      }
      // g over the kept scores: softmax over the k kept, or a sigmoid of each
      float coef[RF_KEEP];
      if (p.norm == 0) {
        float sum = 0.f;
#pragma unroll
        for (int q = 0; q < RF_KEEP; ++q) {
          coef[q] = q < p.k ? expf(bv[q] - bv[0]) : 0.f;
          sum += coef[q];
        }
#pragma unroll
        for (int q = 0; q < RF_KEEP; ++q) coef[q] = coef[q] / sum;
      } else {
#pragma unroll
        for (int q = 0; q < RF_KEEP; ++q) coef[q] = 1.f / (1.f + expf(-bv[q]));
      }
      if (have) {
        if (p.k == RF_KEEP) {
          uint32_t lo = 0u, hi = 0u;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            lo |= (uint32_t)(bi[q] & 0xff) << (8 * q);
            hi |= (uint32_t)(bi[4 + q] & 0xff) << (8 * q);
          }
          *reinterpret_cast<uint2*>(p.idx_out + (size_t)t * RF_KEEP) = make_uint2(lo, hi);
          uint4 g;
          __nv_bfloat162* gp = reinterpret_cast<__nv_bfloat162*>(&g);
#pragma unroll
          for (int q = 0; q < 4; ++q) gp[q] = __floats2bfloat162_rn(coef[2 * q], coef[2 * q + 1]);
          *reinterpret_cast<uint4*>(p.gates_out + (size_t)t * RF_KEEP) = g;
        } else {
#pragma unroll
          for (int q = 0; q < RF_KEEP; ++q)
            if (q < p.k) {
              p.idx_out[(size_t)t * p.k + q] = (uint8_t)bi[q];
              p.gates_out[(size_t)t * p.k + q] = __float2bfloat16_rn(coef[q]);
            }
        }
      }
    }
    ptx::tc_fence_before();
  }

  // ---- teardown ----
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
    const uint64_t t0 = ptx::globaltimer_ns();      // copies still in flight towards this CTA's shared memory may land
    while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, RF_TMEM_COLS);
  }
}

namespace {
inline size_t align_up256(size_t v) { return (v + 255) / 256 * 256; }
struct RouteWs {
  size_t scores, grp_off, grp_src, w_perm, bytes;
};
// d_h_max: the permuted copy of the score layer (fold map, one-kernel form) is laid out for rows of up to 4096 elements
constexpr int ROUTE_WPERM_COLS = 4096;
RouteWs route_ws(int T, int E_src, int E_tgt) {
  RouteWs w{};
  size_t off = 0;
  w.w_perm = off; off += align_up256(E_src <= RF_MAX_N ? (size_t)E_src * ROUTE_WPERM_COLS * 2 : 0);
  w.scores = off; off += align_up256((size_t)T * E_src * 4);
  w.grp_off = off; off += align_up256((size_t)(E_tgt + 1) * 4);
  w.grp_src = off; off += align_up256((size_t)E_src * 4);
  w.bytes = off;
  return w;
}
int check_route(int T, int d_h, int E_src, int E_tgt, int k, int norm) {
  if (T < 1 || d_h < 1 || E_src < 1 || E_tgt < 1 || k < 1) return GROUTER_ERR_INVALID_ARG;
  if (norm != GROUTER_NORM_SOFTMAX && norm != GROUTER_NORM_SIGMOID) return GROUTER_ERR_INVALID_ARG;
  if (T % 8 || d_h % 8 || E_src % 8) return GROUTER_ERR_UNSUPPORTED;        // the score GEMM works in units of 8
  if (E_tgt > ROUTE_MAX_E || E_src > 4 * ROUTE_MAX_E || k > 32 || k > E_tgt) return GROUTER_ERR_UNSUPPORTED;
  return GROUTER_OK;
}
}  // namespace
}  // namespace grouter

extern "C" {

size_t grouter_route_workspace_bytes(int32_t T, int32_t E_src, int32_t E_tgt) {
  if (T < 1 || E_src < 1 || E_tgt < 1) return 0;
  return grouter::route_ws(T, E_src, E_tgt).bytes;
}

int grouter_route(const void* H, const void* W_s, const int32_t* fold_map, int32_t T, int32_t d_h, int32_t E_src, int32_t E_tgt,
                  int32_t k, int32_t norm, void* idx_out, void* gates_out, float* scores_out, void* workspace, int32_t* status,
                  void* stream) {
  using namespace grouter;
  if (!H || !W_s || !idx_out || !gates_out || !workspace || !status) return GROUTER_ERR_INVALID_ARG;
  const int rc = check_route(T, d_h, E_src, E_tgt, k, norm);
  if (rc != GROUTER_OK) return rc;
  if (!fold_map && E_src != E_tgt) return GROUTER_ERR_INVALID_ARG;
  auto mis = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; };
  if (mis(H, 16) || mis(W_s, 16) || mis(workspace, 256) || mis(gates_out, 2) || mis(status, 4) || (fold_map && mis(fold_map, 4)) ||
      (scores_out && mis(scores_out, 4)))
    return GROUTER_ERR_MISALIGNED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const RouteWs w = route_ws(T, E_src, E_tgt);
  char* base = static_cast<char*>(workspace);
  float* S_src = reinterpret_cast<float*>(base + w.scores);
  int32_t* grp_off = reinterpret_cast<int32_t*>(base + w.grp_off);
  int32_t* grp_src = reinterpret_cast<int32_t*>(base + w.grp_src);
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (E_src <= RF_MAX_N && k <= RF_KEEP && d_h <= ROUTE_WPERM_COLS) {
    // ---- one-kernel form ----
    const void* W_use = W_s;
    RouteFusedParams fp{};
    if (fold_map) {
      route_groups_kernel<<<1, ROUTE_THREADS, 0, st>>>(fold_map, E_src, E_tgt, grp_off, grp_src, status);
      if (cudaGetLastError() != cudaSuccess) return GROUTER_ERR_CUDA;
      uint4* W_perm = reinterpret_cast<uint4*>(base + w.w_perm);
      const int units = d_h / 8;
      route_permute_ws_kernel<<<(E_src * units + 255) / 256, 256, 0, st>>>(static_cast<const uint4*>(W_s), grp_src, E_src, units, W_perm);
      if (cudaGetLastError() != cudaSuccess) return GROUTER_ERR_CUDA;
      W_use = W_perm;
      fp.grp_off = grp_off;
    }
    fp.T = T; fp.d_h = d_h; fp.E_src = E_src; fp.E_tgt = E_tgt; fp.k = k; fp.norm = norm;
    fp.nb = (E_src + 15) / 16 * 16;
    fp.idx_out = static_cast<uint8_t*>(idx_out);
    fp.gates_out = static_cast<__nv_bfloat16*>(gates_out);
    fp.scores_out = scores_out;
    fp.status = status;
    fp.wait_limit_ns = DEFAULT_WAIT_LIMIT_NS;
    CUtensorMap tmH, tmW;
    if (!make_bf16_tile_map(&tmH, H, (uint64_t)T, (uint64_t)d_h, RF_BM) || !make_bf16_tile_map(&tmW, W_use, (uint64_t)E_src, (uint64_t)d_h, (uint32_t)fp.nb))
      return GROUTER_ERR_CUDA;
    const int smem = RF_STAGES * (RF_A_BYTES + fp.nb * RF_BK * 2) + 1024 + 64;       // two CTAs per SM up to 128 source experts
    static bool configured[64] = {};
    if (dev < 0 || dev >= 64 || !configured[dev]) {
      const int smem_max = RF_STAGES * (RF_A_BYTES + RF_MAX_N * RF_BK * 2) + 1024 + 64;
      if (cudaFuncSetAttribute(route_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess) return GROUTER_ERR_CUDA;
      if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    route_fused_kernel<<<(T + RF_BM - 1) / RF_BM, RF_THREADS, smem, st>>>(tmH, tmW, fp);
    return cudaGetLastError() == cudaSuccess ? GROUTER_OK : GROUTER_ERR_CUDA;
  }
  // ---- two-kernel form: source scores [T, d_h] x [E_src, d_h]^T on the tensor cores, fp32 out ----
  if (launch_dense_gemm(H, 0, W_s, 0, S_src, T, E_src, d_h, status, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (fold_map) {
    route_groups_kernel<<<1, ROUTE_THREADS, 0, st>>>(fold_map, E_src, E_tgt, grp_off, grp_src, status);
    if (cudaGetLastError() != cudaSuccess) return GROUTER_ERR_CUDA;
  } else {
    grp_off = nullptr;
  }
  int grid = (T + ROUTE_WARPS - 1) / ROUTE_WARPS;
  if (grid > sms * 8) grid = sms * 8;
  route_topk_kernel<<<grid, ROUTE_THREADS, 0, st>>>(S_src, grp_off, grp_src, T, E_src, E_tgt, k, norm, static_cast<uint8_t*>(idx_out),
                                                    static_cast<__nv_bfloat16*>(gates_out), scores_out);
  if (cudaGetLastError() != cudaSuccess) return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}

}  // extern "C"
