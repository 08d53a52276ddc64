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
// Tile: 256 x 256 x 64 per CTA pair (a cluster of two CTAs on neighbouring SMs, one pair-wide tcgen05.mma with
// M = 256).  Each CTA owns 128 rows of the tile and half of B's 256 columns, so per 64-deep k-step it stages
// 16 KB of A and 16 KB of B: a third less operand traffic per FLOP than a one-CTA 128 x 256 tile and room for a
// 5-stage ring.  In every CTA warp 0 issues its TMA tile loads (128-byte swizzle; the byte counts of both CTAs
// complete on the leader CTA's barrier); warp 1 of the leader CTA issues the MMAs for the pair into one of two
// 256-column TMEM accumulators (present in both CTAs) and releases stages / publishes accumulators to both
// CTAs with multicast commits; warps 2-9 of each CTA drain the other accumulator with tcgen05.ld and run the
// fused epilogue on their CTA's 128 rows, so the epilogue of tile i overlaps the main loop of tile i+1.  bf16 outputs
// leave through swizzled shared-memory staging blocks and TMA tile stores; fp32 outputs (weight gradients) are read
// from TMEM in the MMA-fragment arrangement, where four neighbouring threads own a 32-byte run of a row, and go
// straight to global memory in full sectors: the main loop runs at the shared-memory bandwidth, so every staged
// byte the epilogue avoids is main-loop time won.
// Operands may be K-major (rows of the stored matrix run along K) or MN-major (rows run along M/N); both are
// described to the MMA by shared-memory descriptors, so no operand is ever transposed in memory.
//
// Tiles are handed out by a grid-wide counter (all products but DENSE): a pair takes the next tile of the list when it
// is ready for one, so the pairs always work on neighbouring tiles and the operand rows they share are in L2 together.
//
// Every wait (mbarriers, tile queue) is bounded; on give-up the CTA raises an abort flag, ORs STATUS_TIMEOUT into the status
// word, leaves its loops, and the pair meets at a cluster barrier before freeing TMEM and exiting.
#include "common.cuh"
#include "ptx.cuh"

namespace grouter {

constexpr int BM = 128;                         // rows of the tile owned by one CTA
constexpr int PM = 2 * BM;                      // rows of the pair's tile
constexpr int BN = 256, BK = 64;
constexpr int BNH = BN / 2;                     // B columns staged by one CTA
constexpr int STAGES = 5;
constexpr int A_BYTES = BM * BK * 2;            // 16 KB
constexpr int B_BYTES = BNH * BK * 2;           // 16 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;  // 32 KB per CTA and stage
constexpr int ATOM_BYTES = 64 * BK * 2;         // one 64x64 bf16 box = 8 KB
constexpr int EPI_WARPS = 8;                    // two warps per TMEM lane quadrant, each takes half of the columns
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;
constexpr int EPI_STAGE_BYTES = 32 * 128;       // one staging block: 32 rows x 128 bytes; two per epilogue warp
constexpr int GEMM_SMEM = STAGES * STAGE_BYTES + EPI_WARPS * 2 * EPI_STAGE_BYTES + 1024 /*align*/ + 256 /*barriers, tile queue*/;
constexpr uint32_t TMEM_COLS = 512;

struct GemmParams {
  // schedule
  const int32_t* n_pair_tiles; // device scalar: 256-row tiles in use (row-parallel modes)
  const int32_t* pair_row0;    // device [tiles] first padded row
  const int32_t* pair_expert;  // device [tiles] expert | PAIR_VALID2
  const int32_t* n_wchunks;    // device scalar: (expert, row chunk) entries (weight-gradient modes)
  const int32_t* wchunk_expert;// device [chunks] expert | WCHUNK_SPLIT
  const int32_t* wchunk_row0;  // device [chunks] first padded row
  const int32_t* wchunk_rows;  // device [chunks] rows, multiple of 64
  int32_t E, d, F, k;
  int32_t n_slots;             // routed slots of the plan in use (tokens * k)
  int32_t accumulate;          // weight-gradient modes: add every tile into the caller's gradient
  int32_t M, N, K;             // DENSE: problem; WGRAD: per-expert output M x N
  int32_t tiles_m, tiles_n;    // output tiles per problem (tiles_m unused by row-parallel modes)
  int64_t R_pad_max;
  // epilogue
  const int32_t* row_to_slot;  // the plan's inverse permutation (unpadded rows)
  const int32_t* row_shift;    // [E] padded row - row, per expert
  const int32_t* pad_begin;    // [E] first pad row of each expert's padded segment
  const void* gates;
  int32_t gate_is_f32;
  const __nv_bfloat16* in_G;   // DH
  const __nv_bfloat16* in_U;   // DH
  float* out_f;                // DH: dgate_part; weight gradients / DENSE: the fp32 output [E, M, N]; DOWN_ADD: Y accumulator [T, d]
  int32_t* status;
  unsigned int* tile_counter;  // device scalar, zero at launch (unused by DENSE, which has no context to keep one)
  unsigned long long* cycles;  // null, or GEMM_CYCLE_COUNTERS counters every issuer adds its account to
  unsigned long long wait_limit_ns;   // how long any one wait (barrier, tile queue) may last before the CTA gives up
};

struct Tile {     // one CTA's share of a pair tile
  int a_x, a_y;   // TMA coordinates of this CTA's A rows at k-step 0
  int b_x, b_y;   // ... and of this CTA's half of B
  int num_k;      // k-steps that contribute to the result
  int steps;      // k-steps that pass through the operand ring: max(num_k, 1)
  int row0, col0; // origin of this CTA's 128 x 256 output block within the output matrix of this problem
  int e;
  int m_valid, n_valid;   // m_valid <= 0: this CTA's rows are not part of the problem (it still feeds its B half)
  bool add;               // weight gradients: the tile is one of several partial sums added into a zeroed output
};

template <int MODE>
__device__ __forceinline__ int total_tiles(const GemmParams& p) {
  if (MODE == MODE_WGRAD_D || MODE == MODE_WGRAD_GU) return __ldg(p.n_wchunks) * p.tiles_m * p.tiles_n;
  if (MODE == MODE_DENSE) return p.tiles_m * p.tiles_n;
  return __ldg(p.n_pair_tiles) * p.tiles_n;
}

// Share of pair tile t that CTA `rank` (0 = leader) of the pair works on.
template <int MODE>
__device__ __forceinline__ Tile decode_tile(const GemmParams& p, int t, int rank) {
  Tile ti;
  ti.add = false;
  if (MODE == MODE_UP || MODE == MODE_DOWN || MODE == MODE_DOWN_ADD || MODE == MODE_DH || MODE == MODE_DX) {
    const int mt = t / p.tiles_n, nt = t - mt * p.tiles_n;
    const int pe = __ldg(p.pair_expert + mt);
    ti.e = pe & ~PAIR_VALID2;
    ti.row0 = __ldg(p.pair_row0 + mt) + rank * BM;
    ti.m_valid = (rank == 0 || (pe & PAIR_VALID2)) ? BM : 0;
    ti.a_x = 0;
    // a CTA without rows of its own loads its A block from beyond the last row: TMA fills zeros, which costs
    // no memory traffic and keeps the unused half of the pair's MMA quiet
    ti.a_y = ti.m_valid > 0 ? ti.row0 : (int)p.R_pad_max;
    if (MODE == MODE_UP) {          // B = W_gu as [E*2F, d], K-major; leader stages 128 gate rows, peer the 128 up rows
      ti.col0 = nt * 128;
      ti.n_valid = min(128, p.F - ti.col0);
      ti.b_x = 0;
      ti.b_y = ti.e * 2 * p.F + rank * p.F + ti.col0;
      ti.num_k = (p.d + BK - 1) / BK;
    } else if (MODE == MODE_DOWN || MODE == MODE_DOWN_ADD) { // B = W_d as [E*d, F], K-major
      ti.col0 = nt * BN;
      ti.n_valid = min(BN, p.d - ti.col0);
      ti.b_x = 0;
      ti.b_y = ti.e * p.d + ti.col0 + rank * BNH;
      ti.num_k = (p.F + BK - 1) / BK;
    } else if (MODE == MODE_DH) {   // B = W_d as [E*d, F], MN-major (N = F contiguous), K = d
      ti.col0 = nt * BN;
      ti.n_valid = min(BN, p.F - ti.col0);
      ti.b_x = ti.col0 + rank * BNH;
      ti.b_y = ti.e * p.d;
      ti.num_k = (p.d + BK - 1) / BK;
    } else {                        // DX: B = W_gu as [E*2F, d], MN-major (N = d contiguous), K = 2F
      ti.col0 = nt * BN;
      ti.n_valid = min(BN, p.d - ti.col0);
      ti.b_x = ti.col0 + rank * BNH;
      ti.b_y = ti.e * 2 * p.F;
      ti.num_k = (2 * p.F + BK - 1) / BK;
    }
  } else if (MODE == MODE_WGRAD_D || MODE == MODE_WGRAD_GU) {
    // all output tiles of one (expert, row chunk) are adjacent in the schedule: the CTA pairs in flight read the
    // same chunk of operand rows, which therefore stays in L2 however long the expert's row list is.  A chunk's
    // tiles take more than one round of the CTA pairs; the operand whose slabs the inner loop walks is fetched
    // again in every round, so the inner loop runs along the dimension with fewer tiles.
    const int per = p.tiles_m * p.tiles_n;
    const int ci = t / per;
    const int r = t - ci * per;
    int mt, nt;
    if (p.tiles_m < p.tiles_n) {
      nt = r / p.tiles_m;
      mt = r - nt * p.tiles_m;
    } else {
      mt = r / p.tiles_n;
      nt = r - mt * p.tiles_n;
    }
    const int we = __ldg(p.wchunk_expert + ci);
    ti.e = we & ~WCHUNK_SPLIT;
    ti.add = (we & WCHUNK_SPLIT) != 0 || p.accumulate != 0;
    const int k0 = __ldg(p.wchunk_row0 + ci), k1 = k0 + __ldg(p.wchunk_rows + ci);
    ti.row0 = mt * PM + rank * BM;
    ti.col0 = nt * BN;
    ti.m_valid = min(BM, p.M - ti.row0);
    ti.n_valid = min(BN, p.N - ti.col0);
    ti.a_x = ti.row0;   // both operands MN-major: x runs along M/N, y along the expert's rows
    ti.b_x = ti.col0 + rank * BNH;
    ti.num_k = (k1 - k0) / BK;
    // An expert without rows still sends one k-step through the pipeline, so that every tile is paced by the same
    // barriers: its boxes lie beyond the last row, where TMA fills zeros without touching memory, and the epilogue
    // ignores the accumulator.
    ti.a_y = ti.b_y = ti.num_k > 0 ? k0 : (int)p.R_pad_max;
  } else {  // DENSE
    const int mt = t / p.tiles_n, nt = t - mt * p.tiles_n;
    ti.e = 0;
    ti.row0 = mt * PM + rank * BM;
    ti.col0 = nt * BN;
    ti.m_valid = min(BM, p.M - ti.row0);
    ti.n_valid = min(BN, p.N - ti.col0);
    ti.a_x = ti.row0;                 // MN-major A: x; K-major A: y (set below)
    ti.a_y = ti.row0;
    ti.b_x = ti.col0 + rank * BNH;    // MN-major B: x; K-major B: y
    ti.b_y = ti.col0 + rank * BNH;
    ti.num_k = (p.K + BK - 1) / BK;
  }
  ti.steps = ti.num_k > 0 ? ti.num_k : 1;
  return ti;
}

// Gate of padded row `prow` of expert e (0 on a pad row): the slot is row_to_slot[prow - row_shift[e]].
__device__ __forceinline__ float gate_of_row(const GemmParams& p, int e, int prow) {
  if (prow >= __ldg(p.pad_begin + e)) return 0.f;
  const int slot = __ldg(p.row_to_slot + (prow - __ldg(p.row_shift + e)));
  if (!GROUTER_CHECKED((unsigned)slot < (unsigned)p.n_slots, p.status)) return 0.f;   // the caller's array, checked build only
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

template <int MODE, bool A_MN, bool B_MN, bool COUNT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmC1,
                    const __grid_constant__ CUtensorMap tmC2, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // The dynamic shared memory starts at the same offset in both CTAs of the pair, so every address derived
  // below names the same location in either CTA (the MMA descriptors and multicast commits rely on that).
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage_base = smem_base + STAGES * STAGE_BYTES;          // epilogue staging, 2 x 4 KB per warp
  const uint32_t bar_base = stage_base + EPI_WARPS * 2 * EPI_STAGE_BYTES;
  // barriers (8 bytes each): full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]; then the tile queue's slots
  //   full[s]       leader only: one arrival (leader's producer, with the byte count of BOTH CTAs' loads)
  //   empty[s]      each CTA: one arrival per round, delivered to both CTAs by the leader's multicast commit
  //   tmem_full[a]  each CTA: one arrival per tile, delivered to both CTAs by the leader's multicast commit
  //   tmem_empty[a] leader only: 2 * EPI_WARPS arrivals, one per epilogue warp of either CTA
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  // Tile queue (all modes but DENSE).  The pair takes its tiles from a grid-wide counter instead of a fixed stride: the
  // pairs then always work on neighbouring tiles of the list, whatever their individual pace, so the operand rows the
  // neighbours share are fetched from DRAM once.  The leader's producer draws the numbers (two tiles ahead, so the
  // round trip of the atomic is never waited for) and writes them into a ring of TQ 8-byte slots {sequence, tile} in
  // both CTAs; the other roles poll their CTA's copy: slot i % TQ holds the pair's i-th tile once its sequence word
  // reads i + 1.  Nobody acknowledges a slot, because nobody can fall TQ tiles behind: every tile passes at least one
  // stage through the operand ring (the producer is at most STAGES tiles ahead of the issuer), and the issuer starts a
  // tile only after every epilogue warp has finished the tile two before it, so the oldest number still unread is at
  // most STAGES + 3 tiles older than the newest one written (STAGES + 4 <= TQ slots in use).
  constexpr bool DYN = MODE != MODE_DENSE;
  constexpr int TQ = 16;
  static_assert(STAGES + 4 <= TQ && (TQ & (TQ - 1)) == 0, "tile queue too short for the operand ring");
  auto tq_slot = [&](int i) { return bar_base + 8u * (2 * STAGES + 4) + 8u * (uint32_t)(i & (TQ - 1)); };
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int rank = (int)ptx::cluster_ctarank();      // 0 = leader of the pair
  const int pair_id = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 2 * EPI_WARPS);
    }
    for (int q = 0; q < TQ; ++q) ptx::st_shared_volatile_v2(tq_slot(q), 0u, 0u);   // sequence 0: nothing published
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    ptx::prefetch_tensormap(&tmC0);
    if (MODE == MODE_UP || MODE == MODE_DH) ptx::prefetch_tensormap(&tmC1);
    if (MODE == MODE_UP) ptx::prefetch_tensormap(&tmC2);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(&s_tmem_base), TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();      // the peer's barriers are initialised and its TMEM is allocated
  ptx::tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;

  const int n_tiles = total_tiles<MODE>(p);
  // L2 residency: B (an expert's weights, or the row chunk every output tile of a weight gradient reads) is
  // reused by other CTA pairs and later tiles; the outputs are streamed out once and must not displace it.
  const uint64_t keep_a = ptx::l2_policy_evict_normal(), keep_b = ptx::l2_policy_evict_last(), stream_out = ptx::l2_policy_evict_first();
  // Reader side of the tile queue: the next tile of this pair, or a number >= n_tiles when there is none (also after
  // a timeout).
  int tq_i = 0;     // tiles this thread has taken so far
  auto next_tile = [&]() -> int {
    const uint32_t want = (uint32_t)tq_i + 1u, addr = tq_slot(tq_i);
    ++tq_i;
    uint32_t seq, v;
    ptx::ld_shared_volatile_v2(addr, seq, v);
    if (seq == want) return (int)v;
    const uint64_t t0 = ptx::globaltimer_ns();
    for (;;) {
#pragma unroll 1
      for (int i = 0; i < 128; ++i) {
        ptx::ld_shared_volatile_v2(addr, seq, v);
        if (seq == want) return (int)v;
      }
      if (*abort_flag) return 0x7fffffff;
      if (ptx::globaltimer_ns() - t0 > p.wait_limit_ns) {
        *abort_flag = 1;
        return 0x7fffffff;
      }
    }
  };

  if (warp == 0) {
    // ===================== TMA producer (both CTAs) =====================
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      // leader with a tile queue: draws tile numbers and writes them to both CTAs' rings
      int pq_i = 0;
      auto publish = [&](int v) {
        const uint32_t seq = (uint32_t)pq_i + 1u, addr = tq_slot(pq_i);
        ++pq_i;
        ptx::st_shared_volatile_v2(addr, seq, (uint32_t)v);
        ptx::st_shared_cluster_volatile_v2(ptx::map_to_cta(addr, 1), seq, (uint32_t)v);
        // every pair stops at its first number >= n_tiles, so n_tiles + n_pairs numbers are drawn in all: whoever
        // holds the last one leaves the counter at zero for the next launch
        if (v == n_tiles + n_pairs - 1) atomicExch(p.tile_counter, 0u);
      };
      const bool draws = DYN && rank == 0;
      int t = pair_id, t1 = 0x7fffffff;   // this tile and, when drawing, the one after it (already published)
      if (DYN) {
        if (draws) {
          t = (int)atomicAdd(p.tile_counter, 1u);
          if (t < n_tiles) t1 = (int)atomicAdd(p.tile_counter, 1u);
          publish(t);
          if (t < n_tiles) publish(t1);
        } else {
          t = next_tile();
        }
      }
      while (t < n_tiles && !*abort_flag) {
        int t2 = 0x7fffffff;
        if (draws && t1 < n_tiles) t2 = (int)atomicAdd(p.tile_counter, 1u);   // wanted a whole tile from now
        const Tile ti = decode_tile<MODE>(p, t, rank);
        bool ok = true;
        for (int ks = 0; ks < ti.steps; ++ks) {
          if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, p.wait_limit_ns)) {
            ok = false;
            break;
          }
          const uint32_t sa = smem_base + s * STAGE_BYTES;
          const uint32_t sb = sa + A_BYTES;
          if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(s), 2 * STAGE_BYTES);
          const uint32_t fb = ptx::map_to_cta(full_bar(s), 0);   // both CTAs' bytes complete on the leader's barrier
          const int k0 = ks * BK;
          if (!A_MN) {
            ptx::tma_load_2d_pair(sa, &tmA, fb, k0, ti.a_y, keep_a);                       // box {64 k, 128 rows}
          } else {
            const int ay = (MODE == MODE_DENSE ? 0 : ti.a_y) + k0;
            ptx::tma_load_2d_pair(sa, &tmA, fb, ti.a_x, ay, keep_a);                       // 2 x box {64 m, 64 k}
            ptx::tma_load_2d_pair(sa + ATOM_BYTES, &tmA, fb, ti.a_x + 64, ay, keep_a);
          }
          if (!B_MN) {
            ptx::tma_load_2d_pair(sb, &tmB, fb, k0, ti.b_y, keep_b);                       // box {64 k, 128 rows}
          } else {
            const int by = (MODE == MODE_DENSE ? 0 : ti.b_y) + k0;
            ptx::tma_load_2d_pair(sb, &tmB, fb, ti.b_x, by, keep_b);                       // 2 x box {64 n, 64 k}
            ptx::tma_load_2d_pair(sb + ATOM_BYTES, &tmB, fb, ti.b_x + 64, by, keep_b);
          }
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (!ok) break;
        if (!DYN) {
          t += n_pairs;
        } else if (draws) {
          if (t1 < n_tiles) publish(t2);
          t = t1;
          t1 = t2;
        } else {
          t = next_tile();
        }
      }
      // every stage release the leader has multicast to this CTA must have landed before the CTA may exit
      for (int i = 0; i < STAGES && !*abort_flag; ++i) {
        if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, p.wait_limit_ns)) break;
        if (++s == STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ===================== MMA issuer (leader CTA only) =====================
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(PM, BN, A_MN, B_MN);
      // K-major: 8-row groups are 1024 B apart (SBO); 16 K-elements = 32 B further along the row.
      // MN-major: 64-wide MN atoms are one 8 KB box apart (LBO), 8-k groups 1024 B apart (SBO);
      //           16 K-elements = 16 rows of 128 B = 2048 B further.
      constexpr uint32_t a_lbo = A_MN ? ATOM_BYTES : 16, a_sbo = 1024, a_kadv = A_MN ? 2048 : 32;
      constexpr uint32_t b_lbo = B_MN ? ATOM_BYTES : 16, b_sbo = 1024, b_kadv = B_MN ? 2048 : 32;
      constexpr uint16_t both = 3;
      // The operand descriptors are not rebuilt per MMA: only their address field (bits 0-13, address >> 4) changes, by
      // constants, and no carry can leave it (shared-memory addresses stay below 2^18).
      const uint64_t da0 = ptx::make_smem_desc_sw128(smem_base, a_lbo, a_sbo);
      const uint64_t db0 = ptx::make_smem_desc_sw128(smem_base + A_BYTES, b_lbo, b_sbo);
      const uint32_t a_hi = (uint32_t)(da0 >> 32), b_hi = (uint32_t)(db0 >> 32);
      uint32_t a_lo = (uint32_t)da0, b_lo = (uint32_t)db0;    // of the current stage
      int s = 0, acc = 0;
      uint32_t ph = 0, acc_ph = 0;
      // account of where this issuer's cycles go (measurement aid; an instantiation of its own, because clock reads in
      // this thread, two per k-step, cost 3-5 % of the kernel even when their results are not used)
      constexpr bool count = COUNT;
      long long c_acc = 0, c_full = 0, n_tiles_done = 0, n_ksteps = 0;
      const long long c_begin = count ? clock64() : 0;
      for (int t = DYN ? next_tile() : pair_id; t < n_tiles && !*abort_flag; t = DYN ? next_tile() : t + n_pairs) {
        const Tile ti = decode_tile<MODE>(p, t, 0);
        const long long c_t0 = count ? clock64() : 0;
        if (!ptx::mbar_wait_bounded(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p.wait_limit_ns)) break;
        if (count) {
          c_acc += clock64() - c_t0;
          n_tiles_done += 1;
          n_ksteps += ti.steps;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        bool ok = true;
        for (int ks = 0; ks < ti.steps; ++ks) {
          const long long c_k0 = count ? clock64() : 0;
          if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, p.wait_limit_ns)) {
            ok = false;
            break;
          }
          if (count) c_full += clock64() - c_k0;
          ptx::tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            ptx::umma_bf16_pair_split(d_tmem, a_lo + kk * (a_kadv >> 4), a_hi, b_lo + kk * (b_kadv >> 4), b_hi, idesc, (ks | kk) != 0 ? 1u : 0u);
          ptx::umma_commit_pair(empty_bar(s), both);  // stage reusable in both CTAs once these MMAs have read it
          a_lo += STAGE_BYTES >> 4;
          b_lo += STAGE_BYTES >> 4;
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
            a_lo = (uint32_t)da0;
            b_lo = (uint32_t)db0;
          }
        }
        if (!ok) break;
        ptx::umma_commit_pair(tfull_bar(acc), both);
        if (++acc == 2) {
          acc = 0;
          acc_ph ^= 1u;
        }
      }
      if (count) {
        atomicAdd(p.cycles + 0, (unsigned long long)(clock64() - c_begin));
        atomicAdd(p.cycles + 1, (unsigned long long)c_full);
        atomicAdd(p.cycles + 2, (unsigned long long)c_acc);
        atomicAdd(p.cycles + 3, (unsigned long long)n_tiles_done);
        atomicAdd(p.cycles + 4, (unsigned long long)n_ksteps);
      }
    }
    __syncwarp();
  } else {
    // ===================== epilogue (warps 2..9 of both CTAs) =====================
    // Thread (quad, lane) owns row quad*32 + lane of this CTA's 128 rows; the warp drains the 128 accumulator
    // columns of its half.  Results go through two warp-private 32-row x 128-byte staging blocks in shared
    // memory (128-byte swizzle, conflict-free) and leave as TMA tile stores: full 128-byte lines, clipped at the
    // tensor bounds, so no store is masked by hand.  Each store is its own bulk group and the blocks alternate,
    // so a block is free again once all but the newest group have been read out of shared memory.
    const int quad = warp & 3;            // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;     // which half of the tile's columns this warp drains
    const int r = quad * 32 + lane;       // row of this CTA's block owned by this thread
    const uint32_t blk_a = stage_base + (uint32_t)(warp - 2) * (2 * EPI_STAGE_BYTES);
    const uint32_t blk_b = blk_a + EPI_STAGE_BYTES;
    const uint32_t row_off = (uint32_t)lane * 128u;
    const uint32_t sw = (uint32_t)(lane & 7);
    auto stage_wait_all = [&]() {         // every store issued so far has been read out of shared memory
      if (lane == 0) ptx::bulk_wait_read0();
      __syncwarp();
    };
    auto stage_wait_older = [&]() {       // ... every store but the newest
      if (lane == 0) ptx::bulk_wait_read1();
      __syncwarp();
    };
    auto stage_put = [&](uint32_t blk, int q, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {  // 16-byte unit q of this row
      ptx::st_shared_v4(blk + row_off + (((uint32_t)q ^ sw) << 4), a, b, c, d);
    };
    auto stage_put_bf16 = [&](uint32_t blk, int q0, const float (&v)[32]) {  // 32 fp32 -> 4 units of 8 bf16
#pragma unroll
      for (int q = 0; q < 4; ++q)
        stage_put(blk, q0 + q, pack_bf16(v[q * 8 + 0], v[q * 8 + 1]), pack_bf16(v[q * 8 + 2], v[q * 8 + 3]),
                  pack_bf16(v[q * 8 + 4], v[q * 8 + 5]), pack_bf16(v[q * 8 + 6], v[q * 8 + 7]));
    };
    auto stage_send_2d = [&](uint32_t blk, const CUtensorMap* tm, int x, int y) {
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        ptx::tma_store_2d(tm, blk, x, y, stream_out);
        ptx::bulk_commit();
      }
    };
    // DH: saved pre-activations G and U of one 32-column chunk of this thread's row (zeros beyond F)
    auto load_gu = [&](const Tile& ti, int c, uint4 (&g4)[4], uint4 (&u4)[4]) {
      const int c0 = half * 128 + c * 32;
      const int n_left = ti.m_valid > 0 ? ti.n_valid - c0 : 0;
      const size_t gi = ((size_t)ti.row0 + r) * p.F + ti.col0 + c0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (q * 8 < n_left) {
          g4[q] = *reinterpret_cast<const uint4*>(p.in_G + gi + q * 8);
          u4[q] = *reinterpret_cast<const uint4*>(p.in_U + gi + q * 8);
        } else {
          g4[q] = make_uint4(0u, 0u, 0u, 0u);
          u4[q] = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    };
    const uint32_t leader_tempty[2] = {ptx::map_to_cta(tempty_bar(0), 0), ptx::map_to_cta(tempty_bar(1), 0)};
    int acc = 0;
    uint32_t acc_ph = 0;
    uint32_t flip = 0;                    // staging block the next single-block store uses (they strictly alternate)
    for (int t = DYN ? next_tile() : pair_id; t < n_tiles && !*abort_flag; t = DYN ? next_tile() : t + n_pairs) {
      const Tile ti = decode_tile<MODE>(p, t, rank);
      const bool live = ti.m_valid > 0;    // false: this CTA only lent its half of B to the pair
      uint4 g4[4], u4[4];
      if (MODE == MODE_DH) load_gu(ti, 0, g4, u4);   // in flight while the main loop of this tile finishes
      if (!ptx::mbar_wait_bounded(tfull_bar(acc), acc_ph, abort_flag, p.wait_limit_ns)) break;
      ptx::tc_fence_after();
      const uint32_t t_row = tmem_base + (uint32_t)acc * BN + ((uint32_t)(quad * 32) << 16);
      const bool have_acc = ti.num_k > 0;
      const int y0 = ti.row0 + quad * 32;  // first output row of this warp's block

      if (MODE == MODE_UP) {
        // accumulator columns 0..127 = gate, 128..255 = up, for F-columns col0..col0+127; this warp: 64 of them
        if (live && ti.n_valid - half * 64 > 0) {
          const float g = gate_of_row(p, ti.e, ti.row0 + r);
          const int x = ti.col0 + half * 64;
          uint32_t ph[32];                 // H' of the 64 columns, packed bf16 pairs
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            uint32_t rg[32], ru[32];
            ptx::tmem_ld32(t_row + half * 64 + cc * 32, rg);
            ptx::tmem_ld32(t_row + 128 + half * 64 + cc * 32, ru);
            ptx::tmem_ld_wait();
            if (cc == 0) stage_wait_all();
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint32_t wg[4], wu[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int c = q * 8 + 2 * i;
                const float g0 = __uint_as_float(rg[c]), g1 = __uint_as_float(rg[c + 1]);
                const float u0 = __uint_as_float(ru[c]), u1 = __uint_as_float(ru[c + 1]);
                const float s0 = __fdividef(1.f, 1.f + __expf(-g0)), s1 = __fdividef(1.f, 1.f + __expf(-g1));
                wg[i] = pack_bf16(g0, g1);
                wu[i] = pack_bf16(u0, u1);
                ph[cc * 16 + q * 4 + i] = pack_bf16(g * g0 * s0 * u0, g * g1 * s1 * u1);
              }
              stage_put(blk_a, cc * 4 + q, wg[0], wg[1], wg[2], wg[3]);
              stage_put(blk_b, cc * 4 + q, wu[0], wu[1], wu[2], wu[3]);
            }
          }
          stage_send_2d(blk_a, &tmC0, x, y0);
          stage_send_2d(blk_b, &tmC1, x, y0);
          stage_wait_older();              // block a has been read (the store of block b may still be reading)
#pragma unroll
          for (int q = 0; q < 8; ++q) stage_put(blk_a, q, ph[q * 4], ph[q * 4 + 1], ph[q * 4 + 2], ph[q * 4 + 3]);
          stage_send_2d(blk_a, &tmC2, x, y0);
        }
      } else if (MODE == MODE_DOWN || MODE == MODE_DX) {
#pragma unroll
        for (int blk = 0; blk < 2; ++blk) {          // two 64-column blocks per warp, one staging block each
          const int cb = half * 128 + blk * 64;
          if (live && ti.n_valid - cb > 0) {
            const uint32_t sb = flip ? blk_b : blk_a;   // not the block of the previous store
            flip ^= 1u;
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              uint32_t ra[32];
              ptx::tmem_ld32(t_row + cb + cc * 32, ra);
              ptx::tmem_ld_wait();
              if (cc == 0) stage_wait_older();
              float v[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(ra[i]);
              stage_put_bf16(sb, cc * 4, v);
            }
            stage_send_2d(sb, &tmC0, ti.col0 + cb, y0);
          }
        }
      } else if (MODE == MODE_DOWN_ADD) {
        // Combine folded into the product (Eq. 1): this thread's row belongs to one token; its gate-weighted expert
        // output is added to the token's fp32 row with 16-byte reductions.  The order in which a token's k rows arrive
        // is not fixed, so Y may differ in the last bits from run to run.
        int tok = -1;
        if (live) {
          const int prow = ti.row0 + r;
          if (prow < __ldg(p.pad_begin + ti.e)) {
            const int slot = __ldg(p.row_to_slot + (prow - __ldg(p.row_shift + ti.e)));
            if (GROUTER_CHECKED((unsigned)slot < (unsigned)p.n_slots, p.status)) tok = slot / p.k;
          }
        }
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const int c0 = half * 128 + cc * 32;
          if (live && ti.n_valid - c0 > 0) {             // warp-uniform
            uint32_t ra[32];
            ptx::tmem_ld32(t_row + c0, ra);
            ptx::tmem_ld_wait();
            if (tok >= 0) {
              float* dst = p.out_f + (size_t)tok * p.d + ti.col0 + c0;
#pragma unroll
              for (int q = 0; q < 8; ++q)
                if (c0 + 4 * q < ti.n_valid) ptx::red_add_v4_f32(dst + 4 * q, ra[4 * q], ra[4 * q + 1], ra[4 * q + 2], ra[4 * q + 3]);
            }
          }
        }
      } else if (MODE == MODE_DH) {
        const float g = live ? gate_of_row(p, ti.e, ti.row0 + r) : 0.f;
        float dgate = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {                // four 32-column chunks; chunks 2c, 2c+1 fill one pair of blocks
          const int cb = half * 128 + (c >> 1) * 64; // first column of the 64-column block
          const int c0 = half * 128 + c * 32;
          const int n_left = live ? ti.n_valid - c0 : 0;
          uint4 cg[4], cu[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            cg[q] = g4[q];
            cu[q] = u4[q];
          }
          if (c < 3) load_gu(ti, c + 1, g4, u4);     // next chunk's loads fly during this chunk's arithmetic
          if (n_left > 0) {
            uint32_t ra[32];
            ptx::tmem_ld32(t_row + c0, ra);
            ptx::tmem_ld_wait();
            if ((c & 1) == 0) stage_wait_all();
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float fg[8], fu[8], vdg[8], vdu[8];
              unpack8(cg[q], fg);
              unpack8(cu[q], fu);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float dA = (q * 8 < n_left) ? __uint_as_float(ra[q * 8 + i]) : 0.f;
                const float sg = __fdividef(1.f, 1.f + __expf(-fg[i]));
                const float si = fg[i] * sg;            // silu(G)
                dgate += dA * si * fu[i];                // <dA, H>
                const float dH = g * dA;
                vdg[i] = dH * fu[i] * sg * (1.f + fg[i] * (1.f - sg));
                vdu[i] = dH * si;
              }
              stage_put(blk_a, (c & 1) * 4 + q, pack_bf16(vdg[0], vdg[1]), pack_bf16(vdg[2], vdg[3]), pack_bf16(vdg[4], vdg[5]),
                        pack_bf16(vdg[6], vdg[7]));
              stage_put(blk_b, (c & 1) * 4 + q, pack_bf16(vdu[0], vdu[1]), pack_bf16(vdu[2], vdu[3]), pack_bf16(vdu[4], vdu[5]),
                        pack_bf16(vdu[6], vdu[7]));
            }
          }
          // after the second chunk of a block pair (or the last valid one): ship dG and dU of these 64 columns
          if ((c & 1) == 1 && live && ti.n_valid - cb > 0) {
            stage_send_2d(blk_a, &tmC0, ti.col0 + cb, y0);   // dG: columns [0,F) of [dG|dU]
            stage_send_2d(blk_b, &tmC1, ti.col0 + cb, y0);   // dU: columns [F,2F)
          }
        }
        if (live) {
          const int nt = ti.col0 / BN;
          p.out_f[(size_t)(nt * 2 + half) * p.R_pad_max + (size_t)ti.row0 + r] = dgate;
        }
      } else {  // WGRAD_D, WGRAD_GU, DENSE: fp32 tile straight from TMEM to global memory (stored, or added for a partial sum)
        if (ti.m_valid > quad * 32 && (have_acc || !ti.add)) {
#pragma unroll
          for (int rh = 0; rh < 2; ++rh) {
            const int ra_row = quad * 32 + rh * 16 + (lane >> 2), rb_row = ra_row + 8;
            float* pa = p.out_f + ((size_t)ti.e * p.M + (size_t)(ti.row0 + ra_row)) * p.N + ti.col0;
            float* pb = pa + (size_t)8 * p.N;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
              const int c0 = half * 128 + cc * 32;
              if (ti.n_valid - c0 > 0) {
                uint32_t r[16];
                if (have_acc) {
                  ptx::tmem_ld_16x256b_x4(tmem_base + (uint32_t)acc * BN + ((uint32_t)(quad * 32 + rh * 16) << 16) + c0, r);
                  ptx::tmem_ld_wait();
                } else {
#pragma unroll
                  for (int i = 0; i < 16; ++i) r[i] = 0u;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int col = c0 + 8 * j + 2 * (lane & 3);
                  if (col < ti.n_valid) {
                    if (ra_row < ti.m_valid) {
                      if (ti.add) ptx::red_add_v2_f32(pa + col, r[4 * j], r[4 * j + 1]);
                      else ptx::st_global_v2_stream(pa + col, r[4 * j], r[4 * j + 1]);
                    }
                    if (rb_row < ti.m_valid) {
                      if (ti.add) ptx::red_add_v2_f32(pb + col, r[4 * j + 2], r[4 * j + 3]);
                      else ptx::st_global_v2_stream(pb + col, r[4 * j + 2], r[4 * j + 3]);
                    }
                  }
                }
              }
            }
          }
        }
      }

      // all TMEM reads of this warp are complete (wait::ld above): hand the accumulator back
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(leader_tempty[acc]);
      if (++acc == 2) {
        acc = 0;
        acc_ph ^= 1u;
      }
    }
    if (lane == 0) ptx::bulk_wait0();   // every tile store of this warp has landed
    __syncwarp();
  }

  // ---- teardown ----
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
    // give copies and barrier arrivals still in flight towards either CTA's shared memory time to land
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();      // neither CTA leaves while the other may still touch its shared memory or TMEM
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
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

// bf16 matrix [rows, cols] with a row pitch of pitch_elems elements; box = {64 columns, box_rows rows},
// 128-byte swizzle, zero fill (loads) / clipping (stores) out of bounds.
static bool make_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint64_t pitch_elems = 0) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (pitch_elems == 0) pitch_elems = cols;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstr[1] = {pitch_elems * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_bf16_tile_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return make_map(tm, base, rows, cols, box_rows);
}

struct Maps {
  CUtensorMap A, B, C0, C1, C2;
};

template <int MODE, bool A_MN, bool B_MN, bool COUNT>
static cudaError_t launch_tc(const Maps& m, const GemmParams& p, int grid, cudaStream_t st) {
  // the opt-in to more than 48 KB of dynamic shared memory is a per-device setting: once per device and instantiation
  static bool configured[64] = {};
  auto kern = grouped_gemm_kernel<MODE, A_MN, B_MN, COUNT>;
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  kern<<<grid, GEMM_THREADS, GEMM_SMEM, st>>>(m.A, m.B, m.C0, m.C1, m.C2, p);
  return cudaGetLastError();
}

template <int MODE, bool A_MN, bool B_MN>
static cudaError_t launch_t(const Maps& m, const GemmParams& p, int grid, cudaStream_t st) {
  if constexpr (MODE != MODE_DENSE) {
    if (p.cycles != nullptr) return launch_tc<MODE, A_MN, B_MN, true>(m, p, grid, st);
  }
  return launch_tc<MODE, A_MN, B_MN, false>(m, p, grid, st);
}

static inline int cdiv(int a, int b) { return (a + b - 1) / b; }

cudaError_t launch_grouped_gemm(grouter_ctx* ctx, GemmMode mode, const Workspace& ws, const void* gates, const void* W_gu,
                                const void* W_d, float* dW_gu, float* dW_d, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  const uint64_t Rp = (uint64_t)ctx->R_pad_max;
  const int d = dm.d, F = dm.ffn, E = dm.E_tgt;
  GemmParams p{};
  p.n_pair_tiles = ctx->pp.n_pair_tiles;
  p.pair_row0 = ctx->pp.pair_row0;
  p.pair_expert = ctx->pp.pair_expert;
  p.n_wchunks = ctx->pp.n_wchunks;
  p.wchunk_expert = ctx->pp.wchunk_expert;
  p.wchunk_row0 = ctx->pp.wchunk_row0;
  p.wchunk_rows = ctx->pp.wchunk_rows;
  p.E = E;
  p.d = d;
  p.F = F;
  p.k = dm.k;
  p.n_slots = (int32_t)ctx->R_act;
  p.R_pad_max = ctx->R_pad_max;
  p.accumulate = (dm.flags & GROUTER_FLAG_ACCUMULATE_DW) ? 1 : 0;
  p.row_to_slot = ctx->pp.row_to_slot;
  p.row_shift = ctx->pp.row_shift;
  p.pad_begin = ctx->pp.pad_begin;
  p.gates = gates;
  p.gate_is_f32 = dm.gate_dtype == GROUTER_GATE_F32;
  p.status = ctx->pp.status;
  p.tile_counter = ctx->pp.tile_counter;
  p.cycles = ctx->count_cycles ? ctx->d_cycles + (int)(mode == MODE_DOWN_ADD ? MODE_DOWN : mode) * GEMM_CYCLE_COUNTERS : nullptr;
  p.wait_limit_ns = ctx->wait_limit_ns;
  Maps m;
  bool ok = true;
  const int grid = ctx->num_sms & ~1;   // whole CTA pairs, one CTA per SM
  switch (mode) {
    case MODE_UP:
      ok = make_map(&m.A, ws.Xp, Rp, d, 128) && make_map(&m.B, W_gu, (uint64_t)E * 2 * F, d, 128) && make_map(&m.C0, ws.G, Rp, F, 32) &&
           make_map(&m.C1, ws.U, Rp, F, 32) && make_map(&m.C2, ws.Hs, Rp, F, 32);
      p.tiles_n = cdiv(F, 128);
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_UP, false, false>(m, p, grid, st);
    case MODE_DOWN:
      ok = make_map(&m.A, ws.Hs, Rp, F, 128) && make_map(&m.B, W_d, (uint64_t)E * d, F, 128) && make_map(&m.C0, ws.O, Rp, d, 32);
      m.C1 = m.C2 = m.C0;
      p.tiles_n = cdiv(d, BN);
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_DOWN, false, false>(m, p, grid, st);
    case MODE_DOWN_ADD:
      ok = make_map(&m.A, ws.Hs, Rp, F, 128) && make_map(&m.B, W_d, (uint64_t)E * d, F, 128);
      m.C0 = m.C1 = m.C2 = m.A;   // results leave as reductions, without a tensor map
      p.tiles_n = cdiv(d, BN);
      p.out_f = ws.Yacc;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_DOWN_ADD, false, false>(m, p, grid, st);
    case MODE_DH:
      // [dG|dU] is one [R_pad, 2F] buffer; the stores see it as two [R_pad, F] views so that clipping stops at F
      ok = make_map(&m.A, ws.dYp, Rp, d, 128) && make_map(&m.B, W_d, (uint64_t)E * d, F, 64) &&
           make_map(&m.C0, ws.dGU, Rp, F, 32, 2 * (uint64_t)F) && make_map(&m.C1, ws.dGU + F, Rp, F, 32, 2 * (uint64_t)F);
      m.C2 = m.C0;
      p.tiles_n = cdiv(F, BN);
      p.in_G = ws.G; p.in_U = ws.U; p.out_f = ws.dgate_part;
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_DH, false, true>(m, p, grid, st);
    case MODE_DX:
      ok = make_map(&m.A, ws.dGU, Rp, 2 * (uint64_t)F, 128) && make_map(&m.B, W_gu, (uint64_t)E * 2 * F, d, 64) &&
           make_map(&m.C0, ws.O, Rp, d, 32);
      m.C1 = m.C2 = m.C0;
      p.tiles_n = cdiv(d, BN);
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_DX, false, true>(m, p, grid, st);
    case MODE_WGRAD_D:
      ok = make_map(&m.A, ws.dYp, Rp, d, 64) && make_map(&m.B, ws.Hs, Rp, F, 64);
      m.C0 = m.C1 = m.C2 = m.A;   // fp32 tiles are stored without a tensor map
      p.M = d; p.N = F; p.out_f = dW_d;
      p.tiles_m = cdiv(d, PM); p.tiles_n = cdiv(F, BN);
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_WGRAD_D, true, true>(m, p, grid, st);
    case MODE_WGRAD_GU:
      ok = make_map(&m.A, ws.dGU, Rp, 2 * (uint64_t)F, 64) && make_map(&m.B, ws.Xp, Rp, d, 64);
      m.C0 = m.C1 = m.C2 = m.A;
      p.M = 2 * F; p.N = d; p.out_f = dW_gu;
      p.tiles_m = cdiv(2 * F, PM); p.tiles_n = cdiv(d, BN);
      if (!ok) return cudaErrorInvalidValue;
      return launch_t<MODE_WGRAD_GU, true, true>(m, p, grid, st);
    default:
      return cudaErrorInvalidValue;
  }
}

// Zero-fill of the gradients that the weight-gradient GEMMs build up from several partial sums.  Every block first
// collects the experts in question (those whose first chunk carries the split flag) into shared memory, then the grid
// sweeps their gradient matrices with 16-byte stores.
__global__ void __launch_bounds__(256) zero_split_dw_kernel(const int32_t* __restrict__ n_wchunks, const int32_t* __restrict__ wchunk_expert,
                                                            const int32_t* __restrict__ wchunk_row0, const int32_t* __restrict__ pad_offsets,
                                                            float4* __restrict__ dW_gu, float4* __restrict__ dW_d, size_t gu_vec4,
                                                            size_t d_vec4) {
  constexpr int MAX_LIST = 1024;          // more split experts than this cannot exist (E_tgt <= 1024)
  __shared__ int s_list[MAX_LIST];
  __shared__ int s_wcnt[8];
  __shared__ int s_n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) s_n = 0;
  __syncthreads();
  const int n = *n_wchunks;
  // ordered compaction of the split experts, in chunk-list order
  for (int base = 0; base < n; base += 256) {
    const int ci = base + threadIdx.x;
    int e = -1;
    if (ci < n) {
      const int we = wchunk_expert[ci];
      if ((we & WCHUNK_SPLIT) && wchunk_row0[ci] == pad_offsets[we & ~WCHUNK_SPLIT]) e = we & ~WCHUNK_SPLIT;   // once per expert: at its first chunk
    }
    const unsigned m = __ballot_sync(0xffffffffu, e >= 0);
    if (lane == 0) s_wcnt[warp] = __popc(m);
    __syncthreads();
    int at = s_n + __popc(m & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) at += s_wcnt[w];
    if (e >= 0 && at < MAX_LIST) s_list[at] = e;
    __syncthreads();
    if (threadIdx.x == 0) {
      int add = 0;
      for (int w = 0; w < 8; ++w) add += s_wcnt[w];
      s_n += add;
    }
    __syncthreads();
  }
  const int n_split = min(s_n, MAX_LIST);
  const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  const size_t first = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
  for (int j = 0; j < n_split; ++j) {
    float4* gu = dW_gu + (size_t)s_list[j] * gu_vec4;
    float4* dd = dW_d + (size_t)s_list[j] * d_vec4;
    for (size_t i = first; i < gu_vec4; i += stride) gu[i] = z;
    for (size_t i = first; i < d_vec4; i += stride) dd[i] = z;
  }
}

cudaError_t launch_zero_split_dw(grouter_ctx* ctx, float* dW_gu, float* dW_d, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  const size_t per_gu = (size_t)2 * dm.ffn * dm.d / 4, per_d = (size_t)dm.d * dm.ffn / 4;   // d, ffn multiples of 8
  zero_split_dw_kernel<<<ctx->num_sms * 4, 256, 0, st>>>(ctx->pp.n_wchunks, ctx->pp.wchunk_expert, ctx->pp.wchunk_row0, ctx->pp.pad_offsets,
                                                         reinterpret_cast<float4*>(dW_gu), reinterpret_cast<float4*>(dW_d), per_gu, per_d);
  return cudaGetLastError();
}

// One CTA, one thread, one barrier that nobody ever arrives at: the bounded wait of the GEMM pipeline runs out after
// `limit_ns` and the kernel reports it the way the pipeline does (STATUS_TIMEOUT in the status word).  Nothing else is
// in flight: no copy, no TMEM, no second CTA.
__global__ void wait_selftest_kernel(unsigned long long limit_ns, int32_t* status, unsigned long long* waited_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int s_abort;
  s_abort = 0;
  const uint32_t b = ptx::smem_u32(&bar);
  ptx::mbar_init(b, 1);
  ptx::fence_mbar_init();
  const uint64_t t0 = ptx::globaltimer_ns();
  const bool arrived = ptx::mbar_wait_bounded(b, 0u, &s_abort, limit_ns);
  *waited_ns = ptx::globaltimer_ns() - t0;
  if (!arrived) atomicOr(status, STATUS_TIMEOUT);
}

cudaError_t launch_wait_selftest(grouter_ctx* ctx, unsigned long long limit_ns, unsigned long long* d_waited_ns, cudaStream_t st) {
  wait_selftest_kernel<<<1, 1, 0, st>>>(limit_ns, ctx->pp.status, d_waited_ns);
  return cudaGetLastError();
}

cudaError_t launch_dense_gemm(const void* A, int a_mn, const void* B, int b_mn, float* C, int M, int N, int K, int32_t* status,
                              cudaStream_t st) {
  GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  p.tiles_m = cdiv(M, PM);
  p.tiles_n = cdiv(N, BN);
  p.status = status;
  p.out_f = C;
  p.wait_limit_ns = DEFAULT_WAIT_LIMIT_NS;
  Maps m;
  const bool ok = (a_mn ? make_map(&m.A, A, K, M, 64) : make_map(&m.A, A, M, K, 128)) &&
                  (b_mn ? make_map(&m.B, B, K, N, 64) : make_map(&m.B, B, N, K, 128));
  if (!ok) return cudaErrorInvalidValue;
  m.C0 = m.C1 = m.C2 = m.A;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int grid = 2 * p.tiles_m * p.tiles_n;   // one CTA pair per tile, at most one CTA per SM
  if (grid > (sms & ~1)) grid = sms & ~1;
  if (a_mn && b_mn) return launch_t<MODE_DENSE, true, true>(m, p, grid, st);
  if (a_mn) return launch_t<MODE_DENSE, true, false>(m, p, grid, st);
  if (b_mn) return launch_t<MODE_DENSE, false, true>(m, p, grid, st);
  return launch_t<MODE_DENSE, false, false>(m, p, grid, st);
}

}  // namespace grouter
