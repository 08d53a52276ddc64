// C-ABI entry points: argument checks, context, workspace carve-up and the
// launch sequence of the forward and backward passes.
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

using namespace grouter;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_dims(const grouter_dims* dm) {
  if (!dm) return GROUTER_ERR_INVALID_ARG;
  if (dm->T < 1 || dm->d < 1 || dm->ffn < 1 || dm->E_src < 1 || dm->E_tgt < 1 || dm->k < 1) return GROUTER_ERR_INVALID_ARG;
  if (dm->idx_dtype != GROUTER_IDX_U8 && dm->idx_dtype != GROUTER_IDX_I32) return GROUTER_ERR_INVALID_ARG;
  if (dm->gate_dtype != GROUTER_GATE_BF16 && dm->gate_dtype != GROUTER_GATE_F32) return GROUTER_ERR_INVALID_ARG;
  if (dm->flags & ~(GROUTER_FLAG_ACCUMULATE_DW | GROUTER_FLAG_FUSED_COMBINE)) return GROUTER_ERR_INVALID_ARG;
  if (dm->d % 8 || dm->ffn % 8) return GROUTER_ERR_UNSUPPORTED;
  if (dm->E_tgt > 1024 || dm->k > 32) return GROUTER_ERR_UNSUPPORTED;
  if (dm->idx_dtype == GROUTER_IDX_U8 && dm->E_src > 256) return GROUTER_ERR_UNSUPPORTED;
  const int64_t R = (int64_t)dm->T * dm->k;
  if (R >= (int64_t)2147483647 - (1 << 18)) return GROUTER_ERR_UNSUPPORTED;
  return GROUTER_OK;
}

inline int64_t r_pad_max(const grouter_dims& dm) {
  const int64_t R = (int64_t)dm.T * dm.k;
  return (R + ROW_TILE - 1) / ROW_TILE * ROW_TILE + (int64_t)ROW_TILE * dm.E_tgt;
}

struct Staging {  // device copies of the per-step host inputs/outputs of grouter_moe_step_host
  size_t idx, gates, X, dY, Y, dX, dgates, counts, offsets, r2s, s2r, bytes;
};
Staging staging_layout(const grouter_dims& dm) {
  Staging s{};
  const size_t R = (size_t)dm.T * dm.k, Td = (size_t)dm.T * dm.d;
  size_t off = 0;
  auto take = [&](size_t n) { size_t o = off; off += align_up(n, 256); return o; };
  s.idx = take(R * (dm.idx_dtype == GROUTER_IDX_U8 ? 1 : 4));
  s.gates = take(R * (dm.gate_dtype == GROUTER_GATE_BF16 ? 2 : 4));
  s.X = take(Td * 2);
  s.dY = take(Td * 2);
  s.Y = take(Td * 2);
  s.dX = take(Td * 2);
  s.dgates = take(R * 4);
  s.counts = take((size_t)dm.E_tgt * 4);
  s.offsets = take((size_t)(dm.E_tgt + 1) * 4);
  s.r2s = take(R * 4);
  s.s2r = take(R * 4);
  s.bytes = off;
  return s;
}

// Names of the kernel slots (grouter_timing_read's order): the NVTX range around every launch carries one of them, so a
// timeline or an `ncu --nvtx --nvtx-include` filter can address a step of the path by name.
const char* const kSlotName[GROUTER_NUM_KERNELS] = {"plan_hist", "plan_permute", "gather_X", "gemm_up_swiglu", "gemm_down", "combine_Y",
                                                   "gather_dY", "gemm_dH", "wgrad_down", "gemm_dX", "wgrad_gate_up", "reduce_dX",
                                                   "zero_split_dW", "plan_scan"};

// Brackets one kernel launch with an NVTX range (a no-op unless a tool is attached) and, while timing is enabled, with
// an event pair.
struct Timed {
  grouter_ctx* c;
  cudaStream_t st;
  int i;
  Timed(grouter_ctx* ctx, int slot, cudaStream_t s) : c(ctx), st(s), i(-1) {
    nvtxRangePushA(kSlotName[slot]);
    if (c->ev_cap > 0 && c->ev_used < c->ev_cap) {
      i = c->ev_used++;
      c->ev_slot[i] = slot;
      cudaEventRecord(c->ev_start[i], st);
    }
  }
  ~Timed() {
    nvtxRangePop();
    if (i >= 0) {
      cudaEventRecord(c->ev_stop[i], st);
      if (c->idle_gap_us > 0) launch_idle(c->idle_gap_us, st);   // the next kernel starts on a GPU that has rested
    }
  }
};

void free_events(grouter_ctx* c) {
  for (int i = 0; i < c->ev_cap; ++i) {
    cudaEventDestroy(c->ev_start[i]);
    cudaEventDestroy(c->ev_stop[i]);
  }
  delete[] c->ev_start;
  delete[] c->ev_stop;
  delete[] c->ev_slot;
  c->ev_start = c->ev_stop = nullptr;
  c->ev_slot = nullptr;
  c->ev_cap = c->ev_used = 0;
}

}  // namespace

namespace grouter {
Workspace carve_workspace(const grouter_dims& dm, int64_t Rp, void* base) {
  Workspace w{};
  char* b = static_cast<char*>(base);
  size_t off = 0;
  auto take = [&](size_t n) { size_t o = off; off += align_up(n, 256); return o; };
  const size_t rd = (size_t)Rp * dm.d * 2, rf = (size_t)Rp * dm.ffn * 2;
  const size_t oXp = take(rd), oG = take(rf), oU = take(rf), oH = take(rf), oO = take(rd), odY = take(rd), odGU = take(2 * rf);
  const size_t oPart = take((size_t)(2 * ((dm.ffn + 255) / 256)) * Rp * 4);
  const size_t oYacc = take((dm.flags & GROUTER_FLAG_FUSED_COMBINE) ? (size_t)dm.T * dm.d * 4 : 0);
  w.bytes = off;
  if (b) {
    w.Xp = reinterpret_cast<__nv_bfloat16*>(b + oXp);
    w.G = reinterpret_cast<__nv_bfloat16*>(b + oG);
    w.U = reinterpret_cast<__nv_bfloat16*>(b + oU);
    w.Hs = reinterpret_cast<__nv_bfloat16*>(b + oH);
    w.O = reinterpret_cast<__nv_bfloat16*>(b + oO);
    w.dYp = reinterpret_cast<__nv_bfloat16*>(b + odY);
    w.dGU = reinterpret_cast<__nv_bfloat16*>(b + odGU);
    w.dgate_part = reinterpret_cast<float*>(b + oPart);
    w.Yacc = (dm.flags & GROUTER_FLAG_FUSED_COMBINE) ? reinterpret_cast<float*>(b + oYacc) : nullptr;
  }
  return w;
}
}  // namespace grouter

extern "C" {

int grouter_checked_build(void) { return grouter::DEBUG_BOUNDS ? 1 : 0; }

const char* grouter_strerror(int code) {
  switch (code) {
    case GROUTER_OK: return "ok";
    case GROUTER_ERR_INVALID_ARG: return "invalid argument";
    case GROUTER_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case GROUTER_ERR_UNSUPPORTED: return "unsupported size or type";
    case GROUTER_ERR_INVALID_STATE: return "call order: plan before fwd, fwd before bwd";
    case GROUTER_ERR_CUDA: return "CUDA call failed";
    case GROUTER_ERR_BAD_INDEX: return "expert id or fold target out of range (seen on device)";
    case GROUTER_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case GROUTER_ERR_NO_DEVICE: return "no usable sm_100 CUDA device";
    case GROUTER_ERR_BOUNDS: return "checked build: a kernel met an index outside its array and skipped the access";
    default: return "unknown error";
  }
}

size_t grouter_workspace_bytes(const grouter_dims* dims) {
  if (check_dims(dims) != GROUTER_OK) return 0;
  return carve_workspace(*dims, r_pad_max(*dims), nullptr).bytes;
}

size_t grouter_host_staging_bytes(const grouter_dims* dims) {
  if (check_dims(dims) != GROUTER_OK) return 0;
  return 2 * staging_layout(*dims).bytes;   // two sets: consecutive steps are in flight together
}

int grouter_create(grouter_ctx** out, const grouter_dims* dims) {
  if (!out) return GROUTER_ERR_INVALID_ARG;
  *out = nullptr;
  const int rc = check_dims(dims);
  if (rc != GROUTER_OK) return rc;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return GROUTER_ERR_NO_DEVICE;
  int major = 0, sms = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GROUTER_ERR_NO_DEVICE;
  if (major != 10) return GROUTER_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  grouter_ctx* c = new (std::nothrow) grouter_ctx();
  if (!c) return GROUTER_ERR_INVALID_ARG;
  c->dims = *dims;
  c->device = dev;
  c->num_sms = sms;
  c->R = (int64_t)dims->T * dims->k;
  c->R_pad_max = r_pad_max(*dims);
  c->max_m_tiles = (int)(c->R_pad_max / ROW_TILE);
  {
    // Chunk length of the weight gradients: as long as possible, but short enough that the smaller of the two
    // gradients (d x ffn per expert) still yields about four tiles per CTA pair over the whole batch.
    const int64_t tiles_d = (int64_t)((dims->d + 255) / 256) * ((dims->ffn + 255) / 256);
    const int64_t want = c->R_pad_max * tiles_d / (4 * (int64_t)(sms > 1 ? sms / 2 : 1));
    int chunk = WGRAD_KCHUNK_MAX;
    while (chunk > WGRAD_KCHUNK_MIN && chunk > want) chunk >>= 1;
    c->pp.wgrad_chunk_blocks = chunk / ROW_TILE;
    c->max_wchunks = dims->E_tgt + (int)(c->R_pad_max / chunk) + 1;
  }
  c->geom = plan_geom(c->R, dims->E_src, dims->E_tgt);
  c->T_act = dims->T;
  c->R_act = c->R;
  c->nblk_act = c->geom.nblk;
  c->planned = c->forwarded = false;
  c->ev_start = c->ev_stop = nullptr;
  c->ev_slot = nullptr;
  c->ev_cap = c->ev_used = 0;
  c->host_steps = 0;
  c->idle_gap_us = 0;
  c->count_cycles = false;
  c->d_cycles = nullptr;
  c->wait_limit_ns = DEFAULT_WAIT_LIMIT_NS;
  c->d_waited = nullptr;
  c->s_in = c->s_out = c->s_side = nullptr;
  c->ev_fork = c->ev_zero_done = c->ev_dx_done = c->ev_join = c->ev_plan_done = c->ev_dy_gathered = c->ev_down_done = c->ev_combined = nullptr;
  c->step_combine_on_side = c->step_dy_pregathered = false;
  c->overlap = true;
  for (int i = 0; i < 2; ++i) c->ev_in_fwd[i] = c->ev_in_bwd[i] = c->ev_fwd_done[i] = c->ev_bwd_done[i] = c->ev_out_done[i] = nullptr;
  {
    bool ok = cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->s_side, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_zero_done, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_dx_done, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_plan_done, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_dy_gathered, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_down_done, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_combined, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaEventCreateWithFlags(&c->ev_in_fwd[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&c->ev_in_bwd[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&c->ev_fwd_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&c->ev_bwd_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&c->ev_out_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      grouter_destroy(c);
      return GROUTER_ERR_CUDA;
    }
  }
  const int E = dims->E_tgt;
  size_t off = 0;
  auto take = [&](size_t n) { size_t o = off; off += align_up(n, 256); return o; };
  const size_t o_pad = take((size_t)(E + 1) * 4), o_shift = take((size_t)E * 4), o_pb = take((size_t)E * 4), o_pp = take((size_t)(E + 1) * 4);
  const size_t o_pr = take((size_t)c->max_m_tiles * 4), o_pe = take((size_t)c->max_m_tiles * 4), o_nt = take(4);
  const size_t o_we = take((size_t)c->max_wchunks * 4), o_wr = take((size_t)c->max_wchunks * 4), o_wn = take((size_t)c->max_wchunks * 4), o_nw = take(4);
  const size_t o_bp = take((size_t)E * c->geom.nblk * 4), o_tk = take(4), o_st = take(4);
  const size_t o_cy = take(6 * GEMM_CYCLE_COUNTERS * sizeof(unsigned long long)), o_wt = take(sizeof(unsigned long long));
  if (cudaMalloc(&c->d_block, off) != cudaSuccess) {
    c->d_block = nullptr;
    grouter_destroy(c);
    return GROUTER_ERR_CUDA;
  }
  if (cudaMemset(c->d_block, 0, off) != cudaSuccess) {
    grouter_destroy(c);
    return GROUTER_ERR_CUDA;
  }
  char* b = static_cast<char*>(c->d_block);
  c->pp.pad_offsets = reinterpret_cast<int32_t*>(b + o_pad);
  c->pp.row_shift = reinterpret_cast<int32_t*>(b + o_shift);
  c->pp.pad_begin = reinterpret_cast<int32_t*>(b + o_pb);
  c->pp.pair_prefix = reinterpret_cast<int32_t*>(b + o_pp);
  c->pp.pair_row0 = reinterpret_cast<int32_t*>(b + o_pr);
  c->pp.pair_expert = reinterpret_cast<int32_t*>(b + o_pe);
  c->pp.n_pair_tiles = reinterpret_cast<int32_t*>(b + o_nt);
  c->pp.wchunk_expert = reinterpret_cast<int32_t*>(b + o_we);
  c->pp.wchunk_row0 = reinterpret_cast<int32_t*>(b + o_wr);
  c->pp.wchunk_rows = reinterpret_cast<int32_t*>(b + o_wn);
  c->pp.n_wchunks = reinterpret_cast<int32_t*>(b + o_nw);
  c->pp.blk_prefix = reinterpret_cast<int32_t*>(b + o_bp);
  c->pp.ticket = reinterpret_cast<unsigned int*>(b + o_tk);
  c->pp.tile_counter = c->pp.ticket + 4;   // same 256-byte slot
  c->pp.status = reinterpret_cast<int32_t*>(b + o_st);
  c->pp.max_m_tiles = c->max_m_tiles;
  c->pp.max_wchunks = c->max_wchunks;
  c->d_cycles = reinterpret_cast<unsigned long long*>(b + o_cy);
  c->d_waited = reinterpret_cast<unsigned long long*>(b + o_wt);
  *out = c;
  return GROUTER_OK;
}

void grouter_destroy(grouter_ctx* ctx) {
  if (!ctx) return;
  free_events(ctx);
  if (ctx->s_in) cudaStreamDestroy(ctx->s_in);
  if (ctx->s_out) cudaStreamDestroy(ctx->s_out);
  if (ctx->s_side) cudaStreamDestroy(ctx->s_side);
  for (cudaEvent_t e : {ctx->ev_fork, ctx->ev_zero_done, ctx->ev_dx_done, ctx->ev_join, ctx->ev_plan_done, ctx->ev_dy_gathered, ctx->ev_down_done, ctx->ev_combined})
    if (e) cudaEventDestroy(e);
  for (int i = 0; i < 2; ++i) {
    cudaEvent_t evs[5] = {ctx->ev_in_fwd[i], ctx->ev_in_bwd[i], ctx->ev_fwd_done[i], ctx->ev_bwd_done[i], ctx->ev_out_done[i]};
    for (cudaEvent_t e : evs)
      if (e) cudaEventDestroy(e);
  }
  if (ctx->d_block) cudaFree(ctx->d_block);
  delete ctx;
}

int grouter_plan(grouter_ctx* ctx, const void* idx, const int32_t* fold_map, int32_t* counts, int32_t* offsets,
                 int32_t* row_to_slot, int32_t* slot_to_row, void* stream) {
  if (!ctx || !idx || !counts || !offsets || !row_to_slot || !slot_to_row) return GROUTER_ERR_INVALID_ARG;
  if (!aligned16(idx) || !aligned16(counts) || !aligned16(offsets) || !aligned16(row_to_slot) || !aligned16(slot_to_row) ||
      (fold_map && !aligned16(fold_map)))
    return GROUTER_ERR_MISALIGNED;
  if (!fold_map && ctx->dims.E_src != ctx->dims.E_tgt) return GROUTER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static const int slot_of_phase[PLAN_PHASES] = {0, 13, 1};
  for (int phase = 0; phase < PLAN_PHASES; ++phase) {
    Timed tm(ctx, slot_of_phase[phase], st);
    if (launch_plan(ctx, phase, idx, fold_map, counts, offsets, row_to_slot, slot_to_row, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  // fwd and bwd read the permutation from the caller's arrays
  ctx->pp.offsets = offsets;
  ctx->pp.row_to_slot = row_to_slot;
  ctx->pp.slot_to_row = slot_to_row;
  ctx->planned = true;
  ctx->forwarded = false;
  return GROUTER_OK;
}

int grouter_moe_fwd(grouter_ctx* ctx, const void* X, const void* gates, const void* W_gu, const void* W_d, void* Y,
                    void* workspace, void* stream) {
  if (!ctx || !X || !gates || !W_gu || !W_d || !Y || !workspace) return GROUTER_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(gates) || !aligned16(W_gu) || !aligned16(W_d) || !aligned16(Y) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return GROUTER_ERR_MISALIGNED;
  if (!ctx->planned) return GROUTER_ERR_INVALID_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Workspace ws = carve_workspace(ctx->dims, ctx->R_pad_max, workspace);
  {
    Timed tm(ctx, 2, st);
    if (launch_scatter_rows(ctx, static_cast<const __nv_bfloat16*>(X), ws.Xp, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  {
    Timed tm(ctx, 3, st);
    if (launch_grouped_gemm(ctx, MODE_UP, ws, gates, W_gu, W_d, nullptr, nullptr, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  if (ctx->dims.flags & GROUTER_FLAG_FUSED_COMBINE) {
    // the down product adds every routed row into the token's fp32 row; a last pass rounds to bf16
    const size_t n = (size_t)ctx->T_act * ctx->dims.d;
    {
      Timed tm(ctx, 5, st);
      if (cudaMemsetAsync(ws.Yacc, 0, n * sizeof(float), st) != cudaSuccess) return GROUTER_ERR_CUDA;
    }
    {
      Timed tm(ctx, 4, st);
      if (launch_grouped_gemm(ctx, MODE_DOWN_ADD, ws, gates, W_gu, W_d, nullptr, nullptr, st) != cudaSuccess) return GROUTER_ERR_CUDA;
    }
    {
      Timed tm(ctx, 5, st);
      if (launch_cast_rows(ctx, ws.Yacc, static_cast<__nv_bfloat16*>(Y), n, st) != cudaSuccess) return GROUTER_ERR_CUDA;
    }
  } else {
    {
      Timed tm(ctx, 4, st);
      if (launch_grouped_gemm(ctx, MODE_DOWN, ws, gates, W_gu, W_d, nullptr, nullptr, st) != cudaSuccess) return GROUTER_ERR_CUDA;
    }
    if (ctx->step_combine_on_side) {
      // (step call only) the combine runs beside the backward pass's first kernels; whoever needs Y or overwrites the
      // expert outputs waits for ev_combined
      if (cudaEventRecord(ctx->ev_down_done, st) != cudaSuccess || cudaStreamWaitEvent(ctx->s_side, ctx->ev_down_done, 0) != cudaSuccess)
        return GROUTER_ERR_CUDA;
      {
        Timed tm(ctx, 5, ctx->s_side);
        if (launch_reduce_rows(ctx, ws.O, static_cast<__nv_bfloat16*>(Y), nullptr, 0, nullptr, ctx->s_side) != cudaSuccess) return GROUTER_ERR_CUDA;
      }
      if (cudaEventRecord(ctx->ev_combined, ctx->s_side) != cudaSuccess) return GROUTER_ERR_CUDA;
    } else {
      Timed tm(ctx, 5, st);
      if (launch_reduce_rows(ctx, ws.O, static_cast<__nv_bfloat16*>(Y), nullptr, 0, nullptr, st) != cudaSuccess) return GROUTER_ERR_CUDA;
    }
  }
  ctx->forwarded = true;
  return GROUTER_OK;
}

int grouter_moe_bwd(grouter_ctx* ctx, const void* dY, const void* X, const void* gates, const void* W_gu, const void* W_d,
                    void* dX, float* dW_gu, float* dW_d, float* dgates, void* workspace, void* stream) {
  if (!ctx || !dY || !X || !gates || !W_gu || !W_d || !dX || !dW_gu || !dW_d || !dgates || !workspace) return GROUTER_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(gates) || !aligned16(W_gu) || !aligned16(W_d) || !aligned16(dX) ||
      !aligned16(dW_gu) || !aligned16(dW_d) || !aligned16(dgates) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return GROUTER_ERR_MISALIGNED;
  if (!ctx->planned || !ctx->forwarded) return GROUTER_ERR_INVALID_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Workspace ws = carve_workspace(ctx->dims, ctx->R_pad_max, workspace);
  const int n_part = 2 * ((ctx->dims.ffn + 255) / 256);  // two column halves per 256-wide tile
  // Two bandwidth-bound kernels have no business on the GEMMs' critical path: the zero-fill of split experts' gradients
  // (needs only the plan) and the final reduction of dX (needs the dX product, not the last weight gradient).  They run
  // on a stream of the context beside the GEMMs, forked from and joined back into the caller's stream with events, so
  // the caller sees one ordered call (the pattern is capturable in a CUDA graph).
  const bool side = ctx->overlap && ctx->idle_gap_us == 0;
  cudaStream_t ss = side ? ctx->s_side : st;
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };
  if (side) {
    if (!ok(cudaEventRecord(ctx->ev_fork, st)) || !ok(cudaStreamWaitEvent(ss, ctx->ev_fork, 0))) return GROUTER_ERR_CUDA;
  }
  {
    Timed tm(ctx, 12, ss);
    // (when accumulating, the caller's gradients are the starting value of every expert's sum: nothing to zero)
    if (!(ctx->dims.flags & GROUTER_FLAG_ACCUMULATE_DW) && launch_zero_split_dw(ctx, dW_gu, dW_d, ss) != cudaSuccess)
      return GROUTER_ERR_CUDA;
  }
  if (side && !ok(cudaEventRecord(ctx->ev_zero_done, ss))) return GROUTER_ERR_CUDA;
  if (ctx->step_dy_pregathered) {
    if (!ok(cudaStreamWaitEvent(st, ctx->ev_dy_gathered, 0))) return GROUTER_ERR_CUDA;
  } else {
    Timed tm(ctx, 6, st);
    if (launch_scatter_rows(ctx, static_cast<const __nv_bfloat16*>(dY), ws.dYp, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  {
    Timed tm(ctx, 7, st);
    if (launch_grouped_gemm(ctx, MODE_DH, ws, gates, W_gu, W_d, nullptr, nullptr, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  if (side && !ok(cudaStreamWaitEvent(st, ctx->ev_zero_done, 0))) return GROUTER_ERR_CUDA;
  {
    Timed tm(ctx, 8, st);
    if (launch_grouped_gemm(ctx, MODE_WGRAD_D, ws, gates, W_gu, W_d, dW_gu, dW_d, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  if (ctx->step_combine_on_side && !ok(cudaStreamWaitEvent(st, ctx->ev_combined, 0))) return GROUTER_ERR_CUDA;   // dXp reuses the expert outputs' buffer
  {
    Timed tm(ctx, 9, st);
    if (launch_grouped_gemm(ctx, MODE_DX, ws, gates, W_gu, W_d, nullptr, nullptr, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  if (side) {
    if (!ok(cudaEventRecord(ctx->ev_dx_done, st)) || !ok(cudaStreamWaitEvent(ss, ctx->ev_dx_done, 0))) return GROUTER_ERR_CUDA;
  }
  {
    Timed tm(ctx, 11, ss);
    if (launch_reduce_rows(ctx, ws.O, static_cast<__nv_bfloat16*>(dX), ws.dgate_part, n_part, dgates, ss) != cudaSuccess)
      return GROUTER_ERR_CUDA;
  }
  if (side && !ok(cudaEventRecord(ctx->ev_join, ss))) return GROUTER_ERR_CUDA;
  {
    Timed tm(ctx, 10, st);
    if (launch_grouped_gemm(ctx, MODE_WGRAD_GU, ws, gates, W_gu, W_d, dW_gu, dW_d, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  }
  if (side && !ok(cudaStreamWaitEvent(st, ctx->ev_join, 0))) return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}

int grouter_moe_step_host(grouter_ctx* ctx, const void* idx_host, const void* gates_host, const void* X_host, const void* dY_host,
                          const int32_t* fold_map, const void* W_gu, const void* W_d, void* Y_host, void* dX_host,
                          float* dgates_host, float* dW_gu, float* dW_d, void* workspace, void* stream) {
  if (!ctx || !idx_host || !gates_host || !X_host || !dY_host || !Y_host || !dX_host || !dgates_host || !workspace)
    return GROUTER_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return GROUTER_ERR_MISALIGNED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const grouter_dims& dm = ctx->dims;
  const size_t ws_bytes = carve_workspace(dm, ctx->R_pad_max, nullptr).bytes;
  const Staging sg = staging_layout(dm);
  const int set = (int)(ctx->host_steps & 1);
  char* sb = static_cast<char*>(workspace) + ws_bytes + (size_t)set * sg.bytes;
  const size_t R = (size_t)ctx->T_act * dm.k, Td = (size_t)ctx->T_act * dm.d;     // copies move the active tokens only
  const size_t idx_b = R * (dm.idx_dtype == GROUTER_IDX_U8 ? 1 : 4), gate_b = R * (dm.gate_dtype == GROUTER_GATE_BF16 ? 2 : 4);
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };

  // uploads (copy stream): the staging set is free once the step that used it last has downloaded its results
  if (!ok(cudaStreamWaitEvent(ctx->s_in, ctx->ev_out_done[set], 0))) return GROUTER_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(sb + sg.idx, idx_host, idx_b, cudaMemcpyHostToDevice, ctx->s_in))) return GROUTER_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(sb + sg.gates, gates_host, gate_b, cudaMemcpyHostToDevice, ctx->s_in))) return GROUTER_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(sb + sg.X, X_host, Td * 2, cudaMemcpyHostToDevice, ctx->s_in))) return GROUTER_ERR_CUDA;
  if (!ok(cudaEventRecord(ctx->ev_in_fwd[set], ctx->s_in))) return GROUTER_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(sb + sg.dY, dY_host, Td * 2, cudaMemcpyHostToDevice, ctx->s_in))) return GROUTER_ERR_CUDA;   // during plan + fwd
  if (!ok(cudaEventRecord(ctx->ev_in_bwd[set], ctx->s_in))) return GROUTER_ERR_CUDA;

  // compute (caller's stream); with overlap on, dY is gathered beside the forward products and the combine runs beside the
  // backward pass's first kernels, both on the context's side stream
  if (!ok(cudaStreamWaitEvent(st, ctx->ev_in_fwd[set], 0))) return GROUTER_ERR_CUDA;
  int rc = grouter_plan(ctx, sb + sg.idx, fold_map, reinterpret_cast<int32_t*>(sb + sg.counts), reinterpret_cast<int32_t*>(sb + sg.offsets),
                        reinterpret_cast<int32_t*>(sb + sg.r2s), reinterpret_cast<int32_t*>(sb + sg.s2r), stream);
  if (rc != GROUTER_OK) return rc;
  const bool side = ctx->overlap && ctx->idle_gap_us == 0 && !(dm.flags & GROUTER_FLAG_FUSED_COMBINE);
  if (side) {
    const Workspace ws = carve_workspace(dm, ctx->R_pad_max, workspace);
    if (!ok(cudaEventRecord(ctx->ev_plan_done, st)) || !ok(cudaStreamWaitEvent(ctx->s_side, ctx->ev_plan_done, 0)) ||
        !ok(cudaStreamWaitEvent(ctx->s_side, ctx->ev_in_bwd[set], 0)))
      return GROUTER_ERR_CUDA;
    {
      Timed tm(ctx, 6, ctx->s_side);
      if (launch_scatter_rows(ctx, reinterpret_cast<const __nv_bfloat16*>(sb + sg.dY), ws.dYp, ctx->s_side) != cudaSuccess) return GROUTER_ERR_CUDA;
    }
    if (!ok(cudaEventRecord(ctx->ev_dy_gathered, ctx->s_side))) return GROUTER_ERR_CUDA;
  }
  ctx->step_combine_on_side = side;
  rc = grouter_moe_fwd(ctx, sb + sg.X, sb + sg.gates, W_gu, W_d, sb + sg.Y, workspace, stream);
  ctx->step_combine_on_side = false;
  if (rc != GROUTER_OK) return rc;
  if (!ok(cudaEventRecord(ctx->ev_fwd_done[set], side ? ctx->s_side : st))) return GROUTER_ERR_CUDA;     // Y is complete
  if (!ok(cudaStreamWaitEvent(st, ctx->ev_in_bwd[set], 0))) return GROUTER_ERR_CUDA;
  ctx->step_dy_pregathered = side;
  ctx->step_combine_on_side = side;      // bwd: the dX product waits for the combine before it reuses the buffer
  rc = grouter_moe_bwd(ctx, sb + sg.dY, sb + sg.X, sb + sg.gates, W_gu, W_d, sb + sg.dX, dW_gu, dW_d,
                       reinterpret_cast<float*>(sb + sg.dgates), workspace, stream);
  ctx->step_dy_pregathered = ctx->step_combine_on_side = false;
  if (rc != GROUTER_OK) return rc;
  if (!ok(cudaEventRecord(ctx->ev_bwd_done[set], st))) return GROUTER_ERR_CUDA;

  // downloads (copy stream): Y leaves while the backward pass runs
  if (!ok(cudaStreamWaitEvent(ctx->s_out, ctx->ev_fwd_done[set], 0))) return GROUTER_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(Y_host, sb + sg.Y, Td * 2, cudaMemcpyDeviceToHost, ctx->s_out))) return GROUTER_ERR_CUDA;
  if (!ok(cudaStreamWaitEvent(ctx->s_out, ctx->ev_bwd_done[set], 0))) return GROUTER_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(dX_host, sb + sg.dX, Td * 2, cudaMemcpyDeviceToHost, ctx->s_out))) return GROUTER_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(dgates_host, sb + sg.dgates, R * 4, cudaMemcpyDeviceToHost, ctx->s_out))) return GROUTER_ERR_CUDA;
  if (!ok(cudaEventRecord(ctx->ev_out_done[set], ctx->s_out))) return GROUTER_ERR_CUDA;
  ctx->host_steps += 1;
  return GROUTER_OK;
}

int grouter_host_wait(grouter_ctx* ctx, int32_t steps_in_flight) {
  if (!ctx || steps_in_flight < 0 || steps_in_flight > 1) return GROUTER_ERR_INVALID_ARG;
  // step i records ev_out_done[i & 1] last; waiting for it covers every earlier step as well (one download stream)
  const int64_t last_needed = ctx->host_steps - 1 - steps_in_flight;
  if (last_needed < 0) return GROUTER_OK;
  if (cudaEventSynchronize(ctx->ev_out_done[last_needed & 1]) != cudaSuccess) return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}

int grouter_status(grouter_ctx* ctx, void* stream) {
  if (!ctx) return GROUTER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t h = 0;
  if (cudaMemcpyAsync(&h, ctx->pp.status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (h != 0) {
    if (cudaMemsetAsync(ctx->pp.status, 0, 4, st) != cudaSuccess) return GROUTER_ERR_CUDA;
    if (h & STATUS_TIMEOUT) {
      // a grouped GEMM that gave up left its tile counter mid-count: the next launch must start from zero again
      if (cudaMemsetAsync(ctx->pp.tile_counter, 0, sizeof(unsigned int), st) != cudaSuccess) return GROUTER_ERR_CUDA;
      return GROUTER_ERR_TIMEOUT;
    }
    if (h & STATUS_BOUNDS) return GROUTER_ERR_BOUNDS;
    return GROUTER_ERR_BAD_INDEX;
  }
  return GROUTER_OK;
}

int grouter_timing_enable(grouter_ctx* ctx, int32_t n_records) {
  if (!ctx || n_records < 0) return GROUTER_ERR_INVALID_ARG;
  free_events(ctx);
  if (n_records == 0) return GROUTER_OK;
  ctx->ev_start = new (std::nothrow) cudaEvent_t[n_records];
  ctx->ev_stop = new (std::nothrow) cudaEvent_t[n_records];
  ctx->ev_slot = new (std::nothrow) int[n_records];
  if (!ctx->ev_start || !ctx->ev_stop || !ctx->ev_slot) return GROUTER_ERR_INVALID_ARG;
  for (int i = 0; i < n_records; ++i) {
    if (cudaEventCreate(&ctx->ev_start[i]) != cudaSuccess || cudaEventCreate(&ctx->ev_stop[i]) != cudaSuccess) {
      ctx->ev_cap = i;
      free_events(ctx);
      return GROUTER_ERR_CUDA;
    }
  }
  ctx->ev_cap = n_records;
  ctx->ev_used = 0;
  return GROUTER_OK;
}

int grouter_timing_gap(grouter_ctx* ctx, int32_t microseconds) {
  if (!ctx || microseconds < 0 || microseconds > 1000000) return GROUTER_ERR_INVALID_ARG;
  ctx->idle_gap_us = microseconds;
  return GROUTER_OK;
}

int grouter_gemm_cycles_enable(grouter_ctx* ctx, int32_t on) {
  if (!ctx) return GROUTER_ERR_INVALID_ARG;
  ctx->count_cycles = on != 0;
  return GROUTER_OK;
}

int grouter_gemm_cycles_read(grouter_ctx* ctx, void* stream, uint64_t* counters) {
  if (!ctx || !counters) return GROUTER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = 6 * GEMM_CYCLE_COUNTERS * sizeof(unsigned long long);
  if (cudaMemcpyAsync(counters, ctx->d_cycles, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (cudaMemsetAsync(ctx->d_cycles, 0, bytes, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}

int grouter_timing_read(grouter_ctx* ctx, void* stream, float* total_ms, int32_t* launches) {
  if (!ctx || !total_ms || !launches) return GROUTER_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return GROUTER_ERR_CUDA;
  for (int k = 0; k < GROUTER_NUM_KERNELS; ++k) {
    total_ms[k] = 0.f;
    launches[k] = 0;
  }
  for (int i = 0; i < ctx->ev_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->ev_start[i], ctx->ev_stop[i]) != cudaSuccess) return GROUTER_ERR_CUDA;
    total_ms[ctx->ev_slot[i]] += ms;
    launches[ctx->ev_slot[i]] += 1;
  }
  ctx->ev_used = 0;
  return GROUTER_OK;
}

int grouter_set_active_tokens(grouter_ctx* ctx, int32_t tokens) {
  if (!ctx || tokens < 1 || tokens > ctx->dims.T) return GROUTER_ERR_INVALID_ARG;
  ctx->T_act = tokens;
  ctx->R_act = (int64_t)tokens * ctx->dims.k;
  ctx->nblk_act = (int)((ctx->R_act + ctx->geom.chunk - 1) / ctx->geom.chunk);     // never more than the context was laid out for
  ctx->planned = ctx->forwarded = false;      // the previous plan covered another number of tokens
  return GROUTER_OK;
}

int grouter_set_overlap(grouter_ctx* ctx, int32_t on) {
  if (!ctx) return GROUTER_ERR_INVALID_ARG;
  ctx->overlap = on != 0;
  return GROUTER_OK;
}

int grouter_set_wait_limit(grouter_ctx* ctx, int64_t microseconds) {
  if (!ctx || microseconds < 1 || microseconds > 60000000) return GROUTER_ERR_INVALID_ARG;
  ctx->wait_limit_ns = (unsigned long long)microseconds * 1000ull;
  return GROUTER_OK;
}

int grouter_wait_selftest(grouter_ctx* ctx, int64_t limit_microseconds, int64_t* waited_microseconds, void* stream) {
  if (!ctx || !waited_microseconds || limit_microseconds < 1 || limit_microseconds > 1000000) return GROUTER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (launch_wait_selftest(ctx, (unsigned long long)limit_microseconds * 1000ull, ctx->d_waited, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  unsigned long long ns = 0;
  if (cudaMemcpyAsync(&ns, ctx->d_waited, sizeof(ns), cudaMemcpyDeviceToHost, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return GROUTER_ERR_CUDA;
  *waited_microseconds = (int64_t)(ns / 1000ull);
  return GROUTER_OK;
}

int32_t grouter_wgrad_chunk_rows(const grouter_ctx* ctx) { return ctx ? ctx->pp.wgrad_chunk_blocks * grouter::ROW_TILE : 0; }

int grouter_dense_gemm(const void* A, int a_mn_major, const void* B, int b_mn_major, float* C, int32_t M, int32_t N, int32_t K,
                       int32_t* status, void* stream) {
  if (!A || !B || !C || !status || M < 1 || N < 1 || K < 1) return GROUTER_ERR_INVALID_ARG;
  if (M % 8 || N % 8 || K % 8) return GROUTER_ERR_UNSUPPORTED;
  if (!aligned16(A) || !aligned16(B) || !aligned16(C)) return GROUTER_ERR_MISALIGNED;
  if (launch_dense_gemm(A, a_mn_major, B, b_mn_major, C, M, N, K, status, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}

}  // extern "C"
