// Grouped bf16 GEMMs of the routed expert layer on the sm_100a tensor cores.
//
// One persistent, warp-specialised kernel template serves all seven products:
//   UP        [G|U] = Xp  * W_gu[e]^T   epilogue: H' = g * silu(G) * U          (Eq. 1, expert FFN)
//   DOWN      O'    = H'  * W_d[e]^T
//   DH        dA    = dYp * W_d[e]      epilogue: d-gate partials, dG, dU       (SwiGLU backward)
//   DX        dXp   = [dG|dU] * W_gu[e]
//   WGRAD_D   dW_d[e]  = dYp_e^T * H'_e     (contraction over the expert's rows)
//   WGRAD_GU  dW_gu[e] = [dG|dU]_e^T * Xp_e
//   DENSE     C = A * B on plain matrices (component check)
//
// Tile: 128 x 256 x 64 per CTA, one CTA per SM.  Warp 0 issues TMA tile loads
// (128-byte swizzle) into a 4-stage shared-memory ring; warp 1 issues
// tcgen05.mma (M=128, N=256, K=16) into one of two 256-column TMEM
// accumulators; warps 2-9 drain the other accumulator with tcgen05.ld and run
// the fused epilogue, so the epilogue of tile i overlaps the main loop of tile
// i+1.  Operands may be K-major (rows of the stored matrix run along K) or
// MN-major (rows run along M/N); both are described to the MMA by
// shared-memory descriptors, so no operand is ever transposed in memory.
//
// Every mbarrier wait is bounded; on give-up the CTA raises an abort flag, ORs
// STATUS_TIMEOUT into the status word, leaves its loops, frees TMEM and exits.
#include "common.cuh"
#include "ptx.cuh"

namespace grouter {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;            // 16 KB
constexpr int B_BYTES = BN * BK * 2;            // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;  // 48 KB
constexpr int ATOM_BYTES = 64 * BK * 2;         // one 64x64 bf16 box = 8 KB
constexpr int EPI_WARPS = 8;                    // two warps per TMEM lane quadrant, each takes half of the columns
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;
constexpr int GEMM_SMEM = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
constexpr uint32_t TMEM_COLS = 512;

struct GemmParams {
  // schedule
  const int32_t* n_m_tiles;    // device scalar: 128-row tiles in use (row-parallel modes)
  const int32_t* tile_expert;  // device [tiles]
  const int32_t* pad_offsets;  // device [E+1]
  int32_t E, d, F;
  int32_t M, N, K;             // DENSE: problem; WGRAD: per-expert output M x N
  int32_t tiles_m, tiles_n;    // output tiles per problem (tiles_m unused by row-parallel modes)
  int64_t R_pad_max;
  // epilogue
  const int32_t* prow_to_slot;
  const void* gates;
  int32_t gate_is_f32;
  __nv_bfloat16* out_b0;       // UP: G      DOWN/DX: O / dXp     DH: dGU
  __nv_bfloat16* out_b1;       // UP: U
  __nv_bfloat16* out_b2;       // UP: H'
  const __nv_bfloat16* in_G;   // DH
  const __nv_bfloat16* in_U;   // DH
  float* out_f;                // WGRAD / DENSE: C ; DH: dgate_part
  int32_t* status;
};

struct Tile {
  int a_x, a_y;   // TMA coordinates of the A tile at k-step 0
  int b_x, b_y, b_y2;
  int num_k;
  int row0, col0; // output origin (row within the output matrix of this problem)
  int e;
  int m_valid, n_valid;
};

template <int MODE>
__device__ __forceinline__ int total_tiles(const GemmParams& p) {
  if (MODE == MODE_WGRAD_D || MODE == MODE_WGRAD_GU) return p.E * p.tiles_m * p.tiles_n;
  if (MODE == MODE_DENSE) return p.tiles_m * p.tiles_n;
  return __ldg(p.n_m_tiles) * p.tiles_n;
}

template <int MODE>
__device__ __forceinline__ Tile decode_tile(const GemmParams& p, int t) {
  Tile ti;
  if (MODE == MODE_UP || MODE == MODE_DOWN || MODE == MODE_DH || MODE == MODE_DX) {
    const int mt = t / p.tiles_n, nt = t - mt * p.tiles_n;
    ti.e = __ldg(p.tile_expert + mt);
    ti.row0 = mt * BM;
    ti.m_valid = BM;
    ti.a_x = 0;
    ti.a_y = ti.row0;
    if (MODE == MODE_UP) {          // B = W_gu as [E*2F, d], K-major; 128 gate rows + 128 up rows
      ti.col0 = nt * 128;
      ti.n_valid = min(128, p.F - ti.col0);
      ti.b_x = 0;
      ti.b_y = ti.e * 2 * p.F + ti.col0;
      ti.b_y2 = ti.b_y + p.F;
      ti.num_k = (p.d + BK - 1) / BK;
    } else if (MODE == MODE_DOWN) { // B = W_d as [E*d, F], K-major
      ti.col0 = nt * BN;
      ti.n_valid = min(BN, p.d - ti.col0);
      ti.b_x = 0;
      ti.b_y = ti.e * p.d + ti.col0;
      ti.b_y2 = ti.b_y + 128;
      ti.num_k = (p.F + BK - 1) / BK;
    } else if (MODE == MODE_DH) {   // B = W_d as [E*d, F], MN-major (N = F contiguous), K = d
      ti.col0 = nt * BN;
      ti.n_valid = min(BN, p.F - ti.col0);
      ti.b_x = ti.col0;
      ti.b_y = ti.e * p.d;
      ti.b_y2 = 0;
      ti.num_k = (p.d + BK - 1) / BK;
    } else {                        // DX: B = W_gu as [E*2F, d], MN-major (N = d contiguous), K = 2F
      ti.col0 = nt * BN;
      ti.n_valid = min(BN, p.d - ti.col0);
      ti.b_x = ti.col0;
      ti.b_y = ti.e * 2 * p.F;
      ti.b_y2 = 0;
      ti.num_k = (2 * p.F + BK - 1) / BK;
    }
  } else if (MODE == MODE_WGRAD_D || MODE == MODE_WGRAD_GU) {
    const int per = p.tiles_m * p.tiles_n;
    ti.e = t / per;
    const int r = t - ti.e * per;
    const int mt = r / p.tiles_n, nt = r - mt * p.tiles_n;
    const int k0 = __ldg(p.pad_offsets + ti.e), k1 = __ldg(p.pad_offsets + ti.e + 1);
    ti.row0 = mt * BM;
    ti.col0 = nt * BN;
    ti.m_valid = min(BM, p.M - ti.row0);
    ti.n_valid = min(BN, p.N - ti.col0);
    ti.a_x = ti.row0;   // both operands MN-major: x runs along M/N, y along the expert's rows
    ti.a_y = k0;
    ti.b_x = ti.col0;
    ti.b_y = k0;
    ti.b_y2 = 0;
    ti.num_k = (k1 - k0) / BK;
  } else {  // DENSE
    const int mt = t / p.tiles_n, nt = t - mt * p.tiles_n;
    ti.e = 0;
    ti.row0 = mt * BM;
    ti.col0 = nt * BN;
    ti.m_valid = min(BM, p.M - ti.row0);
    ti.n_valid = min(BN, p.N - ti.col0);
    ti.a_x = ti.row0;  // interpreted per operand major below
    ti.a_y = ti.row0;
    ti.b_x = ti.col0;
    ti.b_y = ti.col0;
    ti.b_y2 = ti.col0 + 128;
    ti.num_k = (p.K + BK - 1) / BK;
  }
  return ti;
}

__device__ __forceinline__ float gate_of_row(const GemmParams& p, int prow) {
  const int slot = __ldg(p.prow_to_slot + prow);
  if (slot < 0) return 0.f;
  if (p.gate_is_f32) return __ldg(reinterpret_cast<const float*>(p.gates) + slot);
  return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.gates)[slot]);
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// Stores 32 consecutive bf16 of one row (fp32 in v), 16 bytes at a time, columns >= n_left masked off.
__device__ __forceinline__ void store_row32_bf16(__nv_bfloat16* dst, const float (&v)[32], int n_left) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (q * 8 < n_left) {
      uint4 o;
      o.x = pack_bf16(v[q * 8 + 0], v[q * 8 + 1]);
      o.y = pack_bf16(v[q * 8 + 2], v[q * 8 + 3]);
      o.z = pack_bf16(v[q * 8 + 4], v[q * 8 + 5]);
      o.w = pack_bf16(v[q * 8 + 6], v[q * 8 + 7]);
      *reinterpret_cast<uint4*>(dst + q * 8) = o;
    }
  }
}

template <int MODE, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
  // barriers (8 bytes each): full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), EPI_WARPS);
    }
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&s_tmem_base), TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;

  const int n_tiles = total_tiles<MODE>(p);

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        const Tile ti = decode_tile<MODE>(p, t);
        for (int ks = 0; ks < ti.num_k; ++ks) {
          if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag)) break;
          const uint32_t sa = smem_base + s * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          const uint32_t fb = full_bar(s);
          ptx::mbar_arrive_expect_tx(fb, STAGE_BYTES);
          const int k0 = ks * BK;
          if (!A_MN) {
            ptx::tma_load_2d(sa, &tmA, fb, k0, ti.a_y);                       // box {64 k, 128 rows}
          } else {
            ptx::tma_load_2d(sa, &tmA, fb, ti.a_x, (MODE == MODE_DENSE ? 0 : ti.a_y) + k0);              // box {64 m, 64 k}
            ptx::tma_load_2d(sa + ATOM_BYTES, &tmA, fb, ti.a_x + 64, (MODE == MODE_DENSE ? 0 : ti.a_y) + k0);
          }
          if (!B_MN) {
            ptx::tma_load_2d(sb, &tmB, fb, k0, ti.b_y);                       // 2 x box {64 k, 128 rows}
            ptx::tma_load_2d(sb + B_BYTES / 2, &tmB, fb, k0, ti.b_y2);
          } else {
            const int by = (MODE == MODE_DENSE ? 0 : ti.b_y) + k0;
#pragma unroll
            for (int i = 0; i < 4; ++i) ptx::tma_load_2d(sb + i * ATOM_BYTES, &tmB, fb, ti.b_x + 64 * i, by);  // box {64 n, 64 k}
          }
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(BM, BN, A_MN, B_MN);
      // K-major: 8-row groups are 1024 B apart (SBO); 16 K-elements = 32 B further along the row.
      // MN-major: 64-wide MN atoms are one 8 KB box apart (LBO), 8-k groups 1024 B apart (SBO);
      //           16 K-elements = 16 rows of 128 B = 2048 B further.
      constexpr uint32_t a_lbo = A_MN ? ATOM_BYTES : 16, a_sbo = 1024, a_kadv = A_MN ? 2048 : 32;
      constexpr uint32_t b_lbo = B_MN ? ATOM_BYTES : 16, b_sbo = 1024, b_kadv = B_MN ? 2048 : 32;
      int s = 0, acc = 0;
      uint32_t ph = 0, acc_ph = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        const Tile ti = decode_tile<MODE>(p, t);
        if (!ptx::mbar_wait_bounded(tempty_bar(acc), acc_ph ^ 1u, abort_flag)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        bool ok = true;
        for (int ks = 0; ks < ti.num_k; ++ks) {
          if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag)) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + s * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            const uint64_t da = ptx::make_smem_desc_sw128(sa + kk * a_kadv, a_lbo, a_sbo);
            const uint64_t db = ptx::make_smem_desc_sw128(sb + kk * b_kadv, b_lbo, b_sbo);
            ptx::umma_bf16(d_tmem, da, db, idesc, (ks | kk) != 0 ? 1u : 0u);
          }
          ptx::umma_commit(empty_bar(s));  // stage reusable once these MMAs have read it
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (!ok) break;
        if (ti.num_k > 0) ptx::umma_commit(tfull_bar(acc));
        else ptx::mbar_arrive(tfull_bar(acc));
        if (++acc == 2) {
          acc = 0;
          acc_ph ^= 1u;
        }
      }
    }
    __syncwarp();
  } else {
    // ===================== epilogue (warps 2..9) =====================
    const int quad = warp & 3;            // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;     // which half of the tile's columns this warp drains
    const int r = quad * 32 + lane;       // row of the tile owned by this thread
    int acc = 0;
    uint32_t acc_ph = 0;
    for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
      const Tile ti = decode_tile<MODE>(p, t);
      if (!ptx::mbar_wait_bounded(tfull_bar(acc), acc_ph, abort_flag)) break;
      ptx::tc_fence_after();
      const uint32_t t_row = tmem_base + (uint32_t)acc * BN + ((uint32_t)(quad * 32) << 16);
      const bool have_acc = ti.num_k > 0;

      if (MODE == MODE_UP) {
        const size_t prow = (size_t)ti.row0 + r;
        const float g = gate_of_row(p, (int)prow);
        const size_t o = prow * p.F + ti.col0;
        for (int c = half * 2; c < half * 2 + 2; ++c) {
          const int n_left = ti.n_valid - c * 32;
          if (n_left <= 0) break;
          uint32_t rg[32], ru[32];
          ptx::tmem_ld32(t_row + c * 32, rg);
          ptx::tmem_ld32(t_row + 128 + c * 32, ru);
          ptx::tmem_ld_wait();
          float vg[32], vu[32], vh[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            vg[i] = __uint_as_float(rg[i]);
            vu[i] = __uint_as_float(ru[i]);
            const float sg = __fdividef(1.f, 1.f + __expf(-vg[i]));
            vh[i] = g * vg[i] * sg * vu[i];
          }
          store_row32_bf16(p.out_b0 + o + c * 32, vg, n_left);
          store_row32_bf16(p.out_b1 + o + c * 32, vu, n_left);
          store_row32_bf16(p.out_b2 + o + c * 32, vh, n_left);
        }
      } else if (MODE == MODE_DOWN || MODE == MODE_DX) {
        const size_t prow = (size_t)ti.row0 + r;
        const size_t o = prow * p.d + ti.col0;
        for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
          const int n_left = ti.n_valid - c * 32;
          if (n_left <= 0) break;
          uint32_t ra[32];
          ptx::tmem_ld32(t_row + c * 32, ra);
          ptx::tmem_ld_wait();
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(ra[i]);
          store_row32_bf16(p.out_b0 + o + c * 32, v, n_left);
        }
      } else if (MODE == MODE_DH) {
        const size_t prow = (size_t)ti.row0 + r;
        const float g = gate_of_row(p, (int)prow);
        const size_t gi = prow * p.F + ti.col0;
        const size_t oi = prow * 2 * (size_t)p.F + ti.col0;
        float dgate = 0.f;
        for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
          const int n_left = ti.n_valid - c * 32;
          if (n_left <= 0) break;
          // saved pre-activations of this chunk: issue the loads before waiting on TMEM
          uint4 g4[4], u4[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (q * 8 < n_left) {
              g4[q] = *reinterpret_cast<const uint4*>(p.in_G + gi + c * 32 + q * 8);
              u4[q] = *reinterpret_cast<const uint4*>(p.in_U + gi + c * 32 + q * 8);
            }
          }
          uint32_t ra[32];
          ptx::tmem_ld32(t_row + c * 32, ra);
          ptx::tmem_ld_wait();
          float vdg[32], vdu[32];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (q * 8 < n_left) {
              float fg[8], fu[8];
              unpack8(g4[q], fg);
              unpack8(u4[q], fu);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float dA = __uint_as_float(ra[q * 8 + i]);
                const float sg = __fdividef(1.f, 1.f + __expf(-fg[i]));
                const float si = fg[i] * sg;            // silu(G)
                dgate += dA * si * fu[i];                // <dA, H>
                const float dH = g * dA;
                vdg[q * 8 + i] = dH * fu[i] * sg * (1.f + fg[i] * (1.f - sg));
                vdu[q * 8 + i] = dH * si;
              }
            } else {
#pragma unroll
              for (int i = 0; i < 8; ++i) vdg[q * 8 + i] = vdu[q * 8 + i] = 0.f;
            }
          }
          store_row32_bf16(p.out_b0 + oi + c * 32, vdg, n_left);
          store_row32_bf16(p.out_b0 + oi + p.F + c * 32, vdu, n_left);
        }
        const int nt = ti.col0 / BN;
        p.out_f[(size_t)(nt * 2 + half) * p.R_pad_max + prow] = dgate;
      } else {  // WGRAD_D, WGRAD_GU, DENSE: fp32 tile store
        float* C = p.out_f;
        size_t ld;
        if (MODE == MODE_DENSE) {
          ld = (size_t)p.N;
        } else {
          ld = (size_t)p.N;
          C += (size_t)ti.e * p.M * p.N;
        }
        const bool row_ok = r < ti.m_valid;
        float* crow = C + ((size_t)ti.row0 + r) * ld + ti.col0;
        for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
          const int n_left = ti.n_valid - c * 32;
          if (n_left <= 0) break;
          uint32_t ra[32];
          if (have_acc) {
            ptx::tmem_ld32(t_row + c * 32, ra);
            ptx::tmem_ld_wait();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) ra[i] = 0u;
          }
          if (row_ok) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              if (q * 4 < n_left) {
                const uint4 v = make_uint4(ra[q * 4], ra[q * 4 + 1], ra[q * 4 + 2], ra[q * 4 + 3]);
                *reinterpret_cast<uint4*>(crow + c * 32 + q * 4) = v;
              }
            }
          }
        }
      }

      // all TMEM reads of this warp are complete (wait::ld above): hand the accumulator back
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
      if (++acc == 2) {
        acc = 0;
        acc_ph ^= 1u;
      }
    }
  }

  // ---- teardown ----
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
    // give copies still in flight towards this CTA's shared memory time to land
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------
// Host side: tensor maps and launches
// ------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(ptr);
  return fn;
}

// bf16 matrix [rows, cols] row-major; box = {64 columns, box_rows rows}, 128-byte swizzle, zero fill out of bounds.
static bool make_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstr[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int MODE, bool A_MN, bool B_MN>
static cudaError_t launch_t(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p, int grid, cudaStream_t st) {
  static bool configured = false;
  auto kern = grouped_gemm_kernel<MODE, A_MN, B_MN>;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  kern<<<grid, GEMM_THREADS, GEMM_SMEM, st>>>(tmA, tmB, p);
  return cudaGetLastError();
}

static inline int cdiv(int a, int b) { return (a + b - 1) / b; }

cudaError_t launch_grouped_gemm(grouter_ctx* ctx, GemmMode mode, const Workspace& ws, const void* gates, const void* W_gu,
                                const void* W_d, float* dW_gu, float* dW_d, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  const uint64_t Rp = (uint64_t)ctx->R_pad_max;
  const int d = dm.d, F = dm.ffn, E = dm.E_tgt;
  GemmParams p{};
  p.n_m_tiles = ctx->pp.n_m_tiles;
  p.tile_expert = ctx->pp.tile_expert;
  p.pad_offsets = ctx->pp.pad_offsets;
  p.E = E;
  p.d = d;
  p.F = F;
  p.R_pad_max = ctx->R_pad_max;
  p.prow_to_slot = ctx->pp.prow_to_slot;
  p.gates = gates;
  p.gate_is_f32 = dm.gate_dtype == GROUTER_GATE_F32;
  p.status = ctx->pp.status;
  CUtensorMap tmA, tmB;
  bool ok = true;
  const int grid = ctx->num_sms;
  switch (mode) {
    case MODE_UP:
      ok = make_map(&tmA, ws.Xp, Rp, d, 128) && make_map(&tmB, W_gu, (uint64_t)E * 2 * F, d, 128);
      p.tiles_n = cdiv(F, 128);
      p.out_b0 = ws.G; p.out_b1 = ws.U; p.out_b2 = ws.Hs;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_UP, false, false>(tmA, tmB, p, grid, st);
    case MODE_DOWN:
      ok = make_map(&tmA, ws.Hs, Rp, F, 128) && make_map(&tmB, W_d, (uint64_t)E * d, F, 128);
      p.tiles_n = cdiv(d, BN);
      p.out_b0 = ws.O;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_DOWN, false, false>(tmA, tmB, p, grid, st);
    case MODE_DH:
      ok = make_map(&tmA, ws.dYp, Rp, d, 128) && make_map(&tmB, W_d, (uint64_t)E * d, F, 64);
      p.tiles_n = cdiv(F, BN);
      p.out_b0 = ws.dGU; p.in_G = ws.G; p.in_U = ws.U; p.out_f = ws.dgate_part;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_DH, false, true>(tmA, tmB, p, grid, st);
    case MODE_DX:
      ok = make_map(&tmA, ws.dGU, Rp, 2 * (uint64_t)F, 128) && make_map(&tmB, W_gu, (uint64_t)E * 2 * F, d, 64);
      p.tiles_n = cdiv(d, BN);
      p.out_b0 = ws.O;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_DX, false, true>(tmA, tmB, p, grid, st);
    case MODE_WGRAD_D:
      ok = make_map(&tmA, ws.dYp, Rp, d, 64) && make_map(&tmB, ws.Hs, Rp, F, 64);
      p.M = d; p.N = F;
      p.tiles_m = cdiv(d, BM); p.tiles_n = cdiv(F, BN);
      p.out_f = dW_d;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_WGRAD_D, true, true>(tmA, tmB, p, grid, st);
    case MODE_WGRAD_GU:
      ok = make_map(&tmA, ws.dGU, Rp, 2 * (uint64_t)F, 64) && make_map(&tmB, ws.Xp, Rp, d, 64);
      p.M = 2 * F; p.N = d;
      p.tiles_m = cdiv(2 * F, BM); p.tiles_n = cdiv(d, BN);
      p.out_f = dW_gu;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_WGRAD_GU, true, true>(tmA, tmB, p, grid, st);
    default:
      return cudaErrorInvalidValue;
  }
}

cudaError_t launch_dense_gemm(const void* A, int a_mn, const void* B, int b_mn, float* C, int M, int N, int K, int32_t* status,
                              cudaStream_t st) {
  GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  p.tiles_m = cdiv(M, BM);
  p.tiles_n = cdiv(N, BN);
  p.out_f = C;
  p.status = status;
  CUtensorMap tmA, tmB;
  const bool ok = (a_mn ? make_map(&tmA, A, K, M, 64) : make_map(&tmA, A, M, K, 128)) &&
                  (b_mn ? make_map(&tmB, B, K, N, 64) : make_map(&tmB, B, N, K, 128));
  if (!ok) return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int grid = p.tiles_m * p.tiles_n;
  if (grid > sms) grid = sms;
  if (a_mn && b_mn) return launch_t<MODE_DENSE, true, true>(tmA, tmB, p, grid, st);
  if (a_mn) return launch_t<MODE_DENSE, true, false>(tmA, tmB, p, grid, st);
  if (b_mn) return launch_t<MODE_DENSE, false, true>(tmA, tmB, p, grid, st);
  return launch_t<MODE_DENSE, false, false>(tmA, tmB, p, grid, st);
}

}  // namespace grouter
