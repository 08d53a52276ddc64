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

namespace {
inline size_t align_up256(size_t v) { return (v + 255) / 256 * 256; }
struct RouteWs {
  size_t scores, grp_off, grp_src, bytes;
};
RouteWs route_ws(int T, int E_src, int E_tgt) {
  RouteWs w{};
  size_t off = 0;
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
  // source scores: [T, d_h] x [E_src, d_h]^T on the tensor cores, fp32 out
  if (launch_dense_gemm(H, 0, W_s, 0, S_src, T, E_src, d_h, status, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (fold_map) {
    route_groups_kernel<<<1, ROUTE_THREADS, 0, st>>>(fold_map, E_src, E_tgt, grp_off, grp_src, status);
    if (cudaGetLastError() != cudaSuccess) return GROUTER_ERR_CUDA;
  } else {
    grp_off = nullptr;
  }
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int grid = (T + ROUTE_WARPS - 1) / ROUTE_WARPS;
  if (grid > sms * 8) grid = sms * 8;
  route_topk_kernel<<<grid, ROUTE_THREADS, 0, st>>>(S_src, grp_off, grp_src, T, E_src, E_tgt, k, norm, static_cast<uint8_t*>(idx_out),
                                                    static_cast<__nv_bfloat16*>(gates_out), scores_out);
  if (cudaGetLastError() != cudaSuccess) return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}

}  // extern "C"
