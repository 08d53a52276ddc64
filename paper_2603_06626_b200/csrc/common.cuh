// Shared declarations of the CUDA path (host launchers, context, status bits).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "grouter.h"

namespace grouter {

// Sticky device status bits (ORed into ctx->d_status).
constexpr int STATUS_BAD_INDEX = 1;
constexpr int STATUS_TIMEOUT = 2;
constexpr int STATUS_BOUNDS = 4;      // checked build only

// Checked build (compiled with -DGROUTER_DEBUG_BOUNDS, as paper_2603_06626_b200.build.build(debug=True) does): an index
// that a kernel takes from data — a permutation entry, a staging position, a work-list slot — is tested before it is
// used; a value outside its array sets STATUS_BOUNDS in the status word and the access is skipped, so the kernel ends
// normally and grouter_status reports GROUTER_ERR_BOUNDS.  The release build compiles every test to `true`.
#ifdef GROUTER_DEBUG_BOUNDS
constexpr bool DEBUG_BOUNDS = true;
#define GROUTER_CHECKED(cond, status_word) ((cond) ? true : (atomicOr((status_word), ::grouter::STATUS_BOUNDS), false))
#else
constexpr bool DEBUG_BOUNDS = false;
#define GROUTER_CHECKED(cond, status_word) (true)
#endif
constexpr unsigned long long DEFAULT_WAIT_LIMIT_NS = 4000000000ull;   // bounded device-side waits give up after this long

constexpr int ROW_TILE = 128;        // rows one CTA owns in a GEMM tile; expert segments are padded to it
constexpr int PAIR_VALID2 = 1 << 30; // flag in PaddedPlan::pair_expert
// The weight-gradient GEMMs contract over an expert's rows in chunks of at most `wgrad_chunk_blocks` row tiles; an expert
// with several chunks has its gradient summed from partial tiles.  Long chunks mean few partial sums; short chunks give
// the CTA pairs enough tiles when the output matrices are small.  The context picks a power of two between these bounds.
constexpr int WGRAD_KCHUNK_MIN = 1024, WGRAD_KCHUNK_MAX = 16384;
constexpr int WGRAD_LEN_BUCKETS = 32;   // the chunk list is ordered by chunk length in this many classes
constexpr int GEMM_CYCLE_COUNTERS = 5;   // issuer cycles, cycles waiting for operands, for a free accumulator, tiles, k-steps
constexpr int WCHUNK_SPLIT = 1 << 30; // flag in PaddedPlan::wchunk_expert: the expert has several chunks
constexpr int PLAN_THREADS = 256;    // 8 warps per plan block
constexpr int PLAN_WARPS = PLAN_THREADS / 32;
// Two forms of the plan kernels.  The counted form (E_tgt <= 256 and a fold table that fits shared memory) gives every
// thread a run of `ipt` consecutive slots and a private counter per expert; the ballot form serves everything else.
constexpr int PLAN_COUNTED_MAX_E = 256;
constexpr int PLAN_COUNTED_MAX_ESRC = 4096;
constexpr int PLAN_MIN_CHUNK = 2048; // ballot form: slots per plan block (lower bound)
constexpr int PLAN_MAX_BLOCKS = 1184;// ballot form: 148 SMs x 8 resident blocks

struct PlanGeom {
  int chunk;    // slots per block, multiple of 256
  int nblk;     // blocks
  int ipt;      // counted form: consecutive slots per thread (16, 32 or 64); 0 = ballot form
};

inline PlanGeom plan_geom(int64_t R, int E_src, int E_tgt) {
  PlanGeom g;
  if (E_tgt <= PLAN_COUNTED_MAX_E && E_src <= PLAN_COUNTED_MAX_ESRC) {
    // short runs while the problem is small (more blocks in flight), long ones once every SM has several blocks anyway
    // (the per-block scan of the counters costs the same whatever the run length)
    g.ipt = R <= (1 << 20) ? 16 : R <= (1 << 22) ? 32 : 64;
    g.chunk = g.ipt * PLAN_THREADS;
  } else {
    int64_t chunk = (R + PLAN_MAX_BLOCKS - 1) / PLAN_MAX_BLOCKS;
    if (chunk < PLAN_MIN_CHUNK) chunk = PLAN_MIN_CHUNK;
    chunk = (chunk + PLAN_THREADS - 1) / PLAN_THREADS * PLAN_THREADS;
    g.ipt = 0;
    g.chunk = (int)chunk;
  }
  g.nblk = (int)((R + g.chunk - 1) / g.chunk);
  if (g.nblk < 1) g.nblk = 1;
  return g;
}

// What the context keeps of the plan: the 128-row-padded layout the GEMMs use and their work lists.  The
// permutation itself stays in the caller's arrays (row_to_slot, slot_to_row, offsets), which fwd and bwd read:
// padded row = row + row_shift[expert of the row].
struct PaddedPlan {
  int32_t* pad_offsets;   // [E_tgt+1] first padded row of each expert; [E_tgt] = rows in use
  int32_t* row_shift;     // [E_tgt]   pad_offsets[e] - offsets[e]
  int32_t* pad_begin;     // [E_tgt]   first pad row of expert e (pad_offsets[e] + counts[e])
  // Tile list of the row-parallel GEMMs.  A tile is 256 rows of one expert (two 128-row halves, one per CTA
  // of a pair); an expert with an odd number of 128-row blocks ends in a tile whose second half is unused.
  int32_t* pair_prefix;   // [E_tgt+1] exclusive prefix of 256-row tiles per expert
  int32_t* pair_row0;     // [max_m_tiles] first padded row of each 256-row tile
  int32_t* pair_expert;   // [max_m_tiles] expert of the tile; bit 30 set when the second half holds rows of that expert
  int32_t* n_pair_tiles;  // [1]
  // Work list of the weight-gradient GEMMs: one entry per (expert, chunk of rows).  An expert with several
  // chunks adds them into its pre-zeroed gradient (vector reductions to global memory); a one-chunk expert stores.
  int32_t* wchunk_expert; // [max_wchunks] expert | WCHUNK_SPLIT
  int32_t* wchunk_row0;   // [max_wchunks] first padded row of the chunk
  int32_t* wchunk_rows;   // [max_wchunks] rows in the chunk (multiple of 64; 0 for an expert without slots)
  int32_t* n_wchunks;     // [1]
  int32_t* blk_prefix;    // [E_tgt * nblk] per-block histogram, then exclusive prefix over blocks
  unsigned int* ticket;   // [1] last-block-done counter
  int wgrad_chunk_blocks;       // longest weight-gradient chunk, in row tiles
  unsigned int* tile_counter;   // [1] next tile of the running grouped GEMM; zero between launches
  int32_t* status;        // [1] sticky status bits
  int max_m_tiles, max_wchunks;   // entries the two work lists have room for
  // the caller's plan arrays of the latest grouter_plan (device pointers; valid until the caller overwrites them)
  const int32_t* offsets;      // [E_tgt+1]
  const int32_t* row_to_slot;  // [R]
  const int32_t* slot_to_row;  // [R]
};

}  // namespace grouter

struct grouter_ctx {
  grouter_dims dims;
  int device;
  int64_t R;
  // tokens the calls work on (grouter_set_active_tokens; dims.T unless set lower), their slots, and the plan blocks they take
  int32_t T_act;
  int64_t R_act;
  int nblk_act;
  int64_t R_pad_max;      // round_up(R,128) + 128*E_tgt
  int max_m_tiles;
  int max_wchunks;        // E_tgt + R_pad_max / (chunk rows) + 1
  grouter::PlanGeom geom;
  grouter::PaddedPlan pp;
  void* d_block;          // one allocation backing pp
  bool planned;
  bool forwarded;
  int num_sms;
  // copy pipeline of grouter_moe_step_host: uploads, compute and downloads of consecutive steps overlap
  cudaStream_t s_in, s_out;          // host->device and device->host copy streams
  cudaStream_t s_side;               // bandwidth-bound kernels that run beside a GEMM (see grouter_moe_bwd)
  cudaEvent_t ev_fork, ev_zero_done, ev_dx_done, ev_join, ev_plan_done, ev_dy_gathered, ev_down_done, ev_combined;
  // set by grouter_moe_step_host around its fwd / bwd calls: the step call may let work of one pass run beside the other
  bool step_combine_on_side;         // fwd: the combine goes to s_side (its completion is ev_combined)
  bool step_dy_pregathered;          // bwd: dY was gathered on s_side already (completion: ev_dy_gathered)
  bool overlap;                      // run those kernels on s_side (default) or in line
  cudaEvent_t ev_in_fwd[2], ev_in_bwd[2], ev_fwd_done[2], ev_bwd_done[2], ev_out_done[2];   // per staging set
  int64_t host_steps;                // steps submitted so far; step i uses staging set i & 1
  // optional per-kernel timing (event pool)
  cudaEvent_t* ev_start;
  cudaEvent_t* ev_stop;
  int* ev_slot;
  int ev_cap;
  int ev_used;
  int idle_gap_us;        // measurement aid: idle time inserted after every timed kernel (0 = none)
  bool count_cycles;      // measurement aid: the grouped GEMMs account for their issuers' cycles
  unsigned long long* d_cycles;   // device [6 GEMMs][GEMM_CYCLE_COUNTERS], summed over CTA pairs and launches
  unsigned long long wait_limit_ns;   // limit of every bounded device-side wait of this context's kernels
  unsigned long long* d_waited;   // device [1] scratch of grouter_wait_selftest
};

namespace grouter {

// Workspace carve-up (all offsets 256-byte aligned).
struct Workspace {
  __nv_bfloat16* Xp;    // [R_pad_max, d]   gathered tokens
  __nv_bfloat16* G;     // [R_pad_max, F]   gate pre-activation
  __nv_bfloat16* U;     // [R_pad_max, F]   up pre-activation
  __nv_bfloat16* Hs;    // [R_pad_max, F]   gate-scaled hidden state g*silu(G)*U
  __nv_bfloat16* O;     // [R_pad_max, d]   expert outputs (fwd) / dXp (bwd)
  __nv_bfloat16* dYp;   // [R_pad_max, d]   gathered upstream gradient
  __nv_bfloat16* dGU;   // [R_pad_max, 2F]  [dG | dU]
  float* dgate_part;    // [2*ceil(F/256), R_pad_max] partial row sums for d-gate
  float* Yacc;          // [T, d] fp32 sum of the routed rows (only with GROUTER_FLAG_FUSED_COMBINE)
  size_t bytes;
};
Workspace carve_workspace(const grouter_dims& dm, int64_t R_pad_max, void* base);

// ---- launchers (each returns a cudaError_t from the launch) ----
// phase 0: per-block histograms; 1: prefixes over blocks, offsets, padded layout, work lists; 2: stable permutation, tile list
constexpr int PLAN_PHASES = 3;
cudaError_t launch_plan(grouter_ctx* ctx, int phase, const void* idx, const int32_t* fold_map, int32_t* counts, int32_t* offsets,
                        int32_t* row_to_slot, int32_t* slot_to_row, cudaStream_t st);

// dst[prow,:] = src[slot/k,:] for every routed slot (prow = slot_to_row[slot] + row_shift[expert]); pad rows zero-filled.
cudaError_t launch_scatter_rows(grouter_ctx* ctx, const __nv_bfloat16* src, __nv_bfloat16* dst, cudaStream_t st);
// out[t,:] = sum_j src[prow(t*k+j),:] (fp32 sum in slot order); optionally
// dgates[t,j] = sum_n dgate_part[n][prow].
// out[i] = bf16(in[i]) for n elements (n a multiple of 8).
cudaError_t launch_cast_rows(grouter_ctx* ctx, const float* in, __nv_bfloat16* out, size_t n, cudaStream_t st);
cudaError_t launch_reduce_rows(grouter_ctx* ctx, const __nv_bfloat16* src, __nv_bfloat16* out, const float* dgate_part,
                               int n_part, float* dgates, cudaStream_t st);

// MODE_DOWN_ADD: the down product with the combine folded into its epilogue (fp32 reductions into a [T, d] accumulator).
enum GemmMode { MODE_UP = 0, MODE_DOWN = 1, MODE_DH = 2, MODE_DX = 3, MODE_WGRAD_D = 4, MODE_WGRAD_GU = 5, MODE_DENSE = 6, MODE_DOWN_ADD = 7 };

cudaError_t launch_grouped_gemm(grouter_ctx* ctx, GemmMode mode, const Workspace& ws, const void* gates, const void* W_gu,
                                const void* W_d, float* dW_gu, float* dW_d, cudaStream_t st);
// Zero-fills dW_gu[e] and dW_d[e] of every expert whose rows are split over several chunks.
cudaError_t launch_zero_split_dw(grouter_ctx* ctx, float* dW_gu, float* dW_d, cudaStream_t st);
// A kernel that only lets `microseconds` pass (one thread watching the global timer, capped at one second).
cudaError_t launch_idle(int microseconds, cudaStream_t st);
// Tensor map of a row-major bf16 matrix [rows, cols] for 128-byte-swizzled tiles of 64 columns x box_rows rows.
bool make_bf16_tile_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// Measures one bounded wait that cannot succeed (see grouter_wait_selftest).
cudaError_t launch_wait_selftest(grouter_ctx* ctx, unsigned long long limit_ns, unsigned long long* d_waited_ns, cudaStream_t st);
cudaError_t launch_dense_gemm(const void* A, int a_mn, const void* B, int b_mn, float* C, int M, int N, int K, int32_t* status,
                              cudaStream_t st);

}  // namespace grouter
