/*
 * grouter.h — C ABI of the B200 (sm_100a) routed SwiGLU expert layer under
 * preemptive routing.
 *
 * The layer is the MoE feed-forward block of the paper's Eq. 1 (section
 * "Mixture-of-Experts"),   y = sum_i r(x)_i f_i(x),   evaluated with the
 * coefficient vector r(x) *loaded* instead of computed: a frozen router ran
 * ahead of time and cached, per token, k expert ids and k gate scores (section
 * "Decoupling Preemptive Routing"; appendix "Efficiency Experiment Detail",
 * Pre-Dispatch: uint8 ids, bfloat16 scores).  f_i is a bias-free SwiGLU FFN,
 *   f_i(x) = W_d[i] ( silu(W_g[i] x) * (W_u[i] x) ).
 *
 * Conventions for every call
 *   - All tensor arguments are DEVICE pointers unless the name ends in _host.
 *     They are caller-owned, contiguous, row-major and 16-byte aligned.
 *   - bf16 tensors are passed as `const void*` / `void*`.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work and return; they do not synchronise, and after
 *     grouter_create they do not allocate.
 *   - Return value: GROUTER_OK (0) or a negative GROUTER_ERR_* for problems the
 *     host can see.  Problems only the device can see (an expert id out of
 *     range, a bounded wait that ran out) set a sticky status word; the
 *     kernels keep every access in bounds and finish, and grouter_status()
 *     reports it.  Nothing traps.
 *   - Outputs are overwritten, never accumulated into (dW_* excepted under
 *     GROUTER_FLAG_ACCUMULATE_DW).
 *
 * Sizes: T tokens, d model width, ffn expert hidden width, k experts per token,
 * E_src ids that may appear in idx, E_tgt experts that own weights
 * (E_tgt == E_src unless a fold map is given), R = T*k routed slots,
 * slot s = t*k + j.  Required: d % 8 == 0, ffn % 8 == 0, 1 <= E_tgt <= 1024,
 * R < 2^31 - 2^18.
 */
#ifndef GROUTER_H_
#define GROUTER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  GROUTER_OK = 0,
  GROUTER_ERR_INVALID_ARG = -1,   /* NULL pointer, non-positive size, bad enum         */
  GROUTER_ERR_MISALIGNED = -2,    /* a tensor pointer is not 16-byte aligned           */
  GROUTER_ERR_UNSUPPORTED = -3,   /* d or ffn not a multiple of 8, E_tgt > 1024, ...   */
  GROUTER_ERR_INVALID_STATE = -4, /* fwd/bwd before plan, bwd before fwd               */
  GROUTER_ERR_CUDA = -5,          /* a CUDA runtime/driver call failed                 */
  GROUTER_ERR_BAD_INDEX = -6,     /* device saw an expert id or fold target out of range */
  GROUTER_ERR_TIMEOUT = -7,       /* a bounded device-side wait ran out                */
  GROUTER_ERR_NO_DEVICE = -8,     /* no usable CUDA device / not sm_100                */
  GROUTER_ERR_BOUNDS = -9         /* checked build only: a kernel met an index outside its array (see grouter_checked_build) */
};

enum { GROUTER_IDX_U8 = 0, GROUTER_IDX_I32 = 1 };
enum { GROUTER_GATE_BF16 = 0, GROUTER_GATE_F32 = 1 };
/* grouter_moe_bwd adds the weight gradients into dW_gu / dW_d instead of overwriting them (gradient accumulation
 * over micro-batches; the caller zeroes them before the first one).  Experts without slots are left untouched. */
enum { GROUTER_FLAG_ACCUMULATE_DW = 1,
       /* grouter_moe_fwd folds the combine of Eq. 1 into the down product: its epilogue adds every gate-weighted routed row
        * into an fp32 [T, d] accumulator in the workspace (16-byte reductions) and one more pass rounds it to bf16 Y; the
        * expert-ordered output rows are never written.  The order of a token's k additions is not fixed, so Y may differ
        * in its last bits from run to run (without the flag it is bit-reproducible).  The workspace grows by 4*T*d bytes. */
       GROUTER_FLAG_FUSED_COMBINE = 2 };

typedef struct grouter_ctx grouter_ctx; /* opaque */

typedef struct {
  int32_t T, d, ffn, E_src, E_tgt, k;
  int32_t idx_dtype;  /* GROUTER_IDX_U8 (the paper's cache format, E_src <= 256) or GROUTER_IDX_I32 */
  int32_t gate_dtype; /* GROUTER_GATE_BF16 (the paper's cache format) or GROUTER_GATE_F32           */
  int32_t flags;      /* 0 or an OR of GROUTER_FLAG_* */
} grouter_dims;

/* Creates a context for one layer shape on the current CUDA device.  Host call;
 * the only call that allocates: device memory for the padded layout, the tile
 * and chunk lists, per-block histograms (4 * E_tgt bytes per 4096-16384 slots)
 * and the status word.
 * Errors: INVALID_ARG, UNSUPPORTED, NO_DEVICE, CUDA. */
int grouter_create(grouter_ctx** out, const grouter_dims* dims);
void grouter_destroy(grouter_ctx* ctx);

/* Bytes of device workspace grouter_moe_fwd / grouter_moe_bwd need for `dims`.
 * The workspace carries the expert-ordered activations from fwd to the
 * matching bwd (gathered tokens, gate/up pre-activations, gated hidden state),
 * so it must not be touched in between.  Rows are padded per expert to a
 * multiple of 128, so it is sized for T*k + 128*E_tgt rows.  0 on bad dims. */
size_t grouter_workspace_bytes(const grouter_dims* dims);
/* Extra bytes grouter_moe_step_host needs after the workspace proper (two staging sets). */
size_t grouter_host_staging_bytes(const grouter_dims* dims);

/* Routing-plan build: a stable counting sort of the R slots by target expert.
 *   e_s            = fold_map ? fold_map[idx[s]] : idx[s]
 *   counts[e]      = #{ s : e_s == e }
 *   offsets[e]     = sum_{e' < e} counts[e'],   offsets[E_tgt] = R
 *   slot_to_row[s] = offsets[e_s] + #{ s' < s : e_s' == e_s }
 *   row_to_slot    = inverse permutation
 * The fold map is the compact form of the paper's binary folding matrix M
 * (section "Expert Folding", Matrix Folding): fold_map[i] = the j with M_ij = 1.
 * It is applied to the cached ids after top-k, so a token may own several rows
 * of one target expert.
 *   idx         [T,k] uint8 or int32 (dims.idx_dtype), values in [0,E_src)
 *   fold_map    [E_src] int32 in [0,E_tgt), or NULL for the identity
 *   counts      [E_tgt] int32 out          offsets     [E_tgt+1] int32 out
 *   row_to_slot [R] int32 out              slot_to_row [R] int32 out
 * fwd and bwd read offsets, row_to_slot and slot_to_row from these arrays (the
 * context keeps the pointers, the 128-row-padded layout and the GEMMs' work
 * lists): leave them in place and unchanged until the last fwd/bwd that uses
 * this plan has completed.  One plan may serve any number of fwd/bwd calls (all
 * MoE layers of a micro-batch share the same frozen router; section "Decoupled
 * Structure Extraction").
 * An id outside [0,E_src) or a fold target outside [0,E_tgt) is treated as
 * expert 0 and sets the sticky status GROUTER_ERR_BAD_INDEX. */
int grouter_plan(grouter_ctx* ctx, const void* idx, const int32_t* fold_map, int32_t* counts, int32_t* offsets,
                 int32_t* row_to_slot, int32_t* slot_to_row, void* stream);

/* Routing-plan build for callers that cannot allocate device memory (the paper has
 * no counterpart: this is a deployment aid).  grouter_plan needs a context, and
 * grouter_create takes its scratch from cudaMalloc.  A host that has given the
 * whole device to a pooling allocator, runs under a fixed memory budget, or
 * cannot afford the device-wide synchronisation of an allocation inside its loop
 * calls this instead: the scratch is a fixed array inside the library image
 * (about 0.3 MB, present on every GPU that loads the library until the process
 * exits), and the call makes no cudaMalloc/cudaFree and uses no allocating
 * library routine.
 *   Same definition and outputs as grouter_plan (counts, offsets, row_to_slot,
 *   slot_to_row; bit-identical results); sizes are passed directly.
 *   idx_dtype: GROUTER_IDX_U8 or GROUTER_IDX_I32.  fold_map: [E_src] or NULL (then E_src == E_tgt).
 *   status: optional device int32 the kernels OR status bits into (1 = an id or fold
 *           target was out of range and was treated as expert 0); cleared by the call.
 *           NULL keeps the word inside the library's scratch, where the caller cannot read it.
 * Limits: T*k <= 524288 and E_tgt <= 256; larger problems return
 * GROUTER_ERR_UNSUPPORTED ("unsupported size or type") and must use
 * grouter_create + grouter_plan.  Other errors as grouter_plan.
 * The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current); make that first call outside
 * any stream capture.  All calls on a device share the one array and it keeps the
 * previous call's contents (the call clears the words that must start at zero), so
 * two calls whose kernels may overlap on the GPU (different streams, no ordering
 * between them) race: order them on one stream or with events.  Nothing from this
 * call feeds grouter_moe_fwd/bwd, which read the plan kept by a context. */
int grouter_plan_noalloc(const void* idx, int32_t idx_dtype, const int32_t* fold_map, int32_t T, int32_t k, int32_t E_src,
                         int32_t E_tgt, int32_t* counts, int32_t* offsets, int32_t* row_to_slot, int32_t* slot_to_row,
                         int32_t* status, void* stream);

/* Router head: writes the pre-dispatch routing cache from router hidden states (the step before grouter_plan; in
 * the paper it runs once over the corpus, in the data pipeline).  Eq. 2, section "Mixture-of-Experts":
 *   r(x) = g(TopK(s(x), k)),   s(x) = W~_s^T h,   W~_s = W_s M   (section "Expert Folding", Matrix Folding)
 * with the fold applied to the scores BEFORE TopK (a token never picks one target twice), unlike the id fold of
 * grouter_plan.  g is a softmax over the k kept scores or a sigmoid of each.
 *   H         [T, d_h] bf16 router hidden states          W_s   [E_src, d_h] bf16 score layer, one row per source expert
 *   fold_map  [E_src] int32 in [0,E_tgt): the j with M_ij = 1, or NULL (E_src == E_tgt)
 *   idx_out   [T,k] uint8: kept experts, scores descending, equal scores by ascending id
 *   gates_out [T,k] bf16:  r(x) of the kept experts, round-to-nearest-even
 *   scores_out [T,E_tgt] f32 folded scores, or NULL       workspace: grouter_route_workspace_bytes(T, E_src, E_tgt) bytes, 256-aligned
 *   status    device int32 the kernels OR bits into: 1 = a fold target was out of range (counted as target 0),
 *             2 = a bounded wait in the score GEMM ran out.  The caller zeroes it.
 * Required: T, d_h, E_src multiples of 8; E_tgt <= 256 (uint8 ids); E_src <= 1024; k <= min(32, E_tgt); finite inputs.
 * Scores are accumulated in fp32; where two scores differ by less than fp32 rounding the kept set may differ from an
 * exact evaluation.  Errors: INVALID_ARG, UNSUPPORTED, MISALIGNED, CUDA. */
enum { GROUTER_NORM_SOFTMAX = 0, GROUTER_NORM_SIGMOID = 1 };
size_t grouter_route_workspace_bytes(int32_t T, int32_t E_src, int32_t E_tgt);
int grouter_route(const void* H, const void* W_s, const int32_t* fold_map, int32_t T, int32_t d_h, int32_t E_src, int32_t E_tgt,
                  int32_t k, int32_t norm, void* idx_out, void* gates_out, float* scores_out, void* workspace, int32_t* status,
                  void* stream);

/* Routing statistics of a cached routing table (inputs of the method's offline stages; see the sections "Expert
 * Folding", "Decoupling Communication Optimization", the appendices "Maximal Violation" and "Efficiency Experiment
 * Detail", Algorithm 1).  Samples are consecutive runs of seq_len tokens; S = T / seq_len.  A token's repeated id
 * counts once.
 *   idx          [T,k] uint8 or int32 (idx_dtype), values in [0,E)
 *   node_of_expert [E] int32 in [0,n_nodes), or NULL when local_tokens and best_node are NULL
 *   loads        [E] int32 out: tokens per expert L_i              max_vio [1] f32 out: (max L - mean L) / mean L
 *   coact        [E,E] int32 out: P_ij = tokens activating both i and j (diagonal: L_i)
 *   phi          [S,E] f32 out: routing affinity vectors, phi(X)_i = (1/|X|) #{t in X : expert i kept}
 *   local_tokens [S,n_nodes] int32 out or NULL: tokens of the sample with at least one kept expert on the node
 *   best_node    [S] int32 out or NULL: the node with the most local tokens (lowest-numbered among equals); needs local_tokens
 *   status       device int32, bit 1 ORed in when an id or node number is out of range (that entry is skipped); caller zeroes it
 * Required: T a multiple of seq_len, k <= 32, E <= 1024 (256 for uint8 ids), n_nodes <= 64.  All outputs are device
 * pointers and are overwritten.  Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int grouter_routing_stats(const void* idx, int32_t idx_dtype, int32_t T, int32_t k, int32_t E, int32_t seq_len,
                          const int32_t* node_of_expert, int32_t n_nodes, int32_t* loads, int32_t* coact, float* phi, float* max_vio,
                          int32_t* local_tokens, int32_t* best_node, int32_t* status, void* stream);
/* Greedy affinity folding (section "Expert Folding", Expert Folding Mapping), on the HOST: from the co-activation
 * matrix coact_host [E_src,E_src] to fold_map_host [E_src] -> [0,E_tgt).  Groups hold floor(E_src/E_tgt) experts, the
 * first E_src mod E_tgt of them one more; a group is opened by the lowest-numbered unassigned expert and grown by the
 * unassigned expert with the largest summed co-activation with its members (lower id on equal sums); target j is
 * group j.  Needs E_tgt <= E_src.  Plain host arrays; no GPU work. */
int grouter_fold_greedy_host(const int32_t* coact_host, int32_t E_src, int32_t E_tgt, int32_t* fold_map_host);

/* ---- Expert parallelism (section "Decoupling Communication Optimization"; appendix "Efficiency Experiment Detail") ----
 * Experts are split over `world` ranks; every rank keeps its own tokens, and routed rows travel to the rank that owns
 * their expert and back.  With preemptive routing all per-peer row counts follow from the per-rank expert histograms
 * (grouter_plan's `counts` of every rank, known before the step from the routing cache), so the transfer needs no
 * size exchange.  These calls do everything around the transfer; the transfer is the caller's collective (e.g. an
 * NCCL all-to-all with the split sizes below) into the receiver's own memory.
 *
 * grouter_ep_relabel_host (host): renumbers the experts so that every rank owns a contiguous range.
 *   expert_rank [E] in [0,world): owner of each expert (any assignment, e.g. the paper's expert grouping)
 *   relabel [E] out: new id of each expert (ranks ascending, old order kept within a rank); compose it with the fold
 *           map (fold_map'[i] = relabel[fold_map[i]]) and store the weights in the new order
 *   first_expert [world+1] out: rank r owns new ids first_expert[r] .. first_expert[r+1]-1
 * grouter_ep_layout_host (host): per-peer counts and offsets for rank `rank`, in rows.
 *   counts_all [world,E]: row q = `counts` of rank q's plan (new ids)
 *   send_counts/send_offsets [world]/[world+1]: the rows for peer p are rows send_offsets[p] .. of this rank's
 *           expert-ordered rows (grouter_ep_dispatch_rows writes them in exactly that order)
 *   recv_counts/recv_offsets [world]/[world+1]: rows arriving from peer q land at recv_offsets[q]
 *   recv_seg_offsets [world*n_local+1], n_local = experts of `rank`: exclusive prefix of the (source rank, local expert)
 *           segments of the received rows
 * grouter_ep_expand_ids (device): idx_out[r] = local expert (0..n_local-1) of received row r, from recv_seg_offsets on
 *   the device; the receiving rank then runs grouter_plan / fwd / bwd on the received rows as T = rows, k = 1, unit gates.
 * grouter_ep_dispatch_rows (device): rows[slot_to_row[s], :] = gate_s * src[token of s, :]  (gates NULL: plain copy).
 *   rows [T*k, d] bf16, expert-ordered and unpadded.  Forward: src = X, no gates.  Backward: src = dY with the gates.
 * grouter_ep_combine_rows (device): out[t,:] = sum_j gate * rows[slot_to_row[t*k+j], :] in fp32, slot order (gates NULL:
 *   plain sum), and/or dgates[t,j] = <dY[t,:], rows[slot_to_row[t*k+j], :]>.  out or dgates may be NULL (not both).
 *   Forward: rows = returned expert outputs, with the gates -> Y (Eq. 1).  Backward: rows = returned input gradients,
 *   no gates -> dX; dgates from the forward's returned rows and dY.
 * The two row calls need a prior grouter_plan on ctx (they read its slot_to_row) and use ctx's T, k, d, gate_dtype.
 * Errors: INVALID_ARG, MISALIGNED, INVALID_STATE, UNSUPPORTED, CUDA. */
int grouter_ep_relabel_host(int32_t E, int32_t world, const int32_t* expert_rank, int32_t* relabel, int32_t* first_expert);
int grouter_ep_layout_host(int32_t world, int32_t rank, int32_t E, const int32_t* first_expert, const int32_t* counts_all,
                           int32_t* send_counts, int32_t* send_offsets, int32_t* recv_counts, int32_t* recv_offsets,
                           int32_t* recv_seg_offsets);
int grouter_ep_expand_ids(const int32_t* seg_offsets, int32_t n_seg, int32_t n_local, int32_t n_rows, int32_t idx_dtype, void* idx_out,
                          void* stream);
int grouter_ep_dispatch_rows(grouter_ctx* ctx, const void* src, const void* gates, void* rows, void* stream);
int grouter_ep_combine_rows(grouter_ctx* ctx, const void* rows, const void* gates, void* out, const void* dY, float* dgates,
                            void* stream);

/* Forward, Eq. 1:  Y[t,:] = sum_j gates[t,j] * f_{e(t,j)}(X[t,:]).
 *   X     [T,d] bf16             gates [T,k] bf16 or f32 (dims.gate_dtype), used as given
 *   W_gu  [E_tgt, 2*ffn, d] bf16: rows 0..ffn-1 gate projection, ffn..2ffn-1 up projection
 *   W_d   [E_tgt, d, ffn] bf16   Y     [T,d] bf16 out (fp32 accumulate)
 *   workspace: grouter_workspace_bytes(dims) bytes
 * Needs a prior grouter_plan on the same ctx (else INVALID_STATE). */
int grouter_moe_fwd(grouter_ctx* ctx, const void* X, const void* gates, const void* W_gu, const void* W_d, void* Y,
                    void* workspace, void* stream);

/* Backward of grouter_moe_fwd for L with dL/dY = dY (expert gradient as in the
 * paper's appendix on joint optimisation: dL/dtheta_e = dL/dy * sum_i r_i * grad f_i).
 *   dY     [T,d] bf16                 dX     [T,d] bf16 out
 *   dW_gu  [E_tgt, 2*ffn, d] f32 out  dW_d   [E_tgt, d, ffn] f32 out
 *   dgates [T,k] f32 out: dgates[t,j] = <dY[t,:], f_{e(t,j)}(X[t,:])> (gates are leaf inputs)
 * Experts that received no slot get exact zeros in dW_* (with GROUTER_FLAG_ACCUMULATE_DW every expert's gradient is
 * added to what dW_* holds, and such experts are left as they are).  An expert with more than
 * grouter_wgrad_chunk_rows(ctx) rows is contracted in chunks of rows that are added into its gradient in no fixed order,
 * so its dW_* may differ in the last bits from run to run; everything else (Y, dX, dgates, dW_* of smaller experts) is bit-reproducible.  Uses the workspace
 * contents left by the matching grouter_moe_fwd (else INVALID_STATE). */
int grouter_moe_bwd(grouter_ctx* ctx, const void* dY, const void* X, const void* gates, const void* W_gu,
                    const void* W_d, void* dX, float* dW_gu, float* dW_d, float* dgates, void* workspace,
                    void* stream);

/* A context is laid out for dims.T tokens; this makes its later calls (plan, fwd, bwd, the step call, the
 * expert-parallel row calls) work on the first `tokens` of them only, 1 <= tokens <= dims.T: every [T, ...] argument is
 * then a [tokens, ...] array and T*k becomes tokens*k.  Host call, no allocation; a new grouter_plan is needed
 * afterwards.  For batches whose size changes from step to step, e.g. the rows an expert-parallel rank receives: one
 * context for the largest batch serves them all.  The paper has no counterpart. */
int grouter_set_active_tokens(grouter_ctx* ctx, int32_t tokens);

/* grouter_moe_bwd runs two bandwidth-bound kernels (the zero-fill of split experts' gradients, the final reduction of
 * dX) on a stream the context owns, beside the tensor-core products they do not depend on, and joins them back into
 * `stream` before it returns: to the caller the call is ordered on `stream` as ever.  on = 0 puts them back in line
 * (measurement aid; the default is on).  No counterpart in the paper. */
int grouter_set_overlap(grouter_ctx* ctx, int32_t on);

/* Longest run of an expert's rows that the weight-gradient products of grouter_moe_bwd contract in one piece (host
 * only; a power of two between 1024 and 16384 fixed at grouter_create from the dims and the device's SM count: as long
 * as possible, shorter when the per-expert gradient matrices are too small to keep every SM busy otherwise).  The
 * paper has no counterpart: it is a scheduling parameter of this implementation.  Returns 0 for a null context. */
int32_t grouter_wgrad_chunk_rows(const grouter_ctx* ctx);

/* One whole step from HOST buffers: uploads idx, gates, X, dY, runs plan, fwd and bwd on `stream`, and downloads
 * Y, dX, dgates.  Weights, weight gradients and fold_map stay on the device.  The copies run on two streams the
 * context owns, ordered against the compute with events: dY is uploaded while plan and fwd run, Y is downloaded
 * while bwd runs, and with two device staging sets the uploads of step i+1 and the downloads of step i overlap
 * the compute of their neighbours.  Pass pinned host memory, otherwise the copies serialise.
 *   workspace: grouter_workspace_bytes + grouter_host_staging_bytes (the latter holds both staging sets).
 * The call returns after enqueueing.  Host outputs of a step may be read, and its host inputs overwritten,
 * only after grouter_host_wait says the step is complete; synchronising `stream` alone is NOT enough (the
 * downloads run on the context's own stream).  Keeping one step in flight therefore needs two sets of host
 * buffers, used alternately. */
int grouter_moe_step_host(grouter_ctx* ctx, const void* idx_host, const void* gates_host, const void* X_host,
                          const void* dY_host, const int32_t* fold_map, const void* W_gu, const void* W_d,
                          void* Y_host, void* dX_host, float* dgates_host, float* dW_gu, float* dW_d,
                          void* workspace, void* stream);
/* Blocks the calling host thread until all but the `steps_in_flight` (0 or 1) most recently submitted
 * grouter_moe_step_host calls are complete: their host outputs are written and their host inputs consumed.
 * (No counterpart in the paper: host-side plumbing of the step call.) */
int grouter_host_wait(grouter_ctx* ctx, int32_t steps_in_flight);

/* Synchronises `stream` and returns the sticky device status (GROUTER_OK,
 * GROUTER_ERR_BAD_INDEX, GROUTER_ERR_TIMEOUT) or GROUTER_ERR_CUDA; clears it. */
int grouter_status(grouter_ctx* ctx, void* stream);

const char* grouter_strerror(int code);

/* Every device-side wait of this library's kernels (an operand stage, an accumulator, the next tile number) gives up
 * after a limit, 4 s by default; the CTA then sets GROUTER_ERR_TIMEOUT in the status word, waits for its own copies in
 * flight, frees its tensor memory and returns, so the context stays usable.  grouter_set_wait_limit changes the limit
 * for this context's later launches (1 .. 60,000,000 us).  The paper has no counterpart: failure handling of this
 * implementation. */
int grouter_set_wait_limit(grouter_ctx* ctx, int64_t microseconds);
/* Self-test of that mechanism without disturbing a pipeline: launches one thread that waits, with the same bounded
 * wait the GEMMs use, on a barrier nothing ever arrives at, for limit_microseconds (1 .. 1,000,000).  The wait runs
 * out, the kernel sets the timeout bit in the context's status word and returns; the call synchronises `stream` and
 * writes how long the kernel waited to *waited_microseconds (host).  grouter_status then reports
 * GROUTER_ERR_TIMEOUT once and clears it. */
int grouter_wait_selftest(grouter_ctx* ctx, int64_t limit_microseconds, int64_t* waited_microseconds, void* stream);

/* No counterpart in the paper: a development aid in place of a memory checker.  Returns 1 when the library was compiled
 * with -DGROUTER_DEBUG_BOUNDS (paper_2603_06626_b200.build.build(debug=True) -> libgrouter_debug.so), else 0.  In that
 * build the kernels test every index they take from data before they use it: the entries of the caller's
 * slot_to_row / row_to_slot that the row movers and the GEMM epilogues follow, the staging positions, piece and
 * work-list slots of the plan kernels.  A value outside its array sets a sticky status bit and the access is skipped;
 * the kernel finishes and grouter_status() returns GROUTER_ERR_BOUNDS (after GROUTER_ERR_TIMEOUT, before
 * GROUTER_ERR_BAD_INDEX, when several are set).  Results are the same as the release build's on valid inputs.  The
 * release build contains none of these tests: there a corrupted permutation array is the caller's error, as any bad
 * pointer is. */
int grouter_checked_build(void);

/* Per-kernel device timing (measurement aid; no counterpart in the paper).
 * grouter_timing_enable(ctx, n) creates n CUDA event pairs (host call, allocates;
 * n = 0 frees them and switches timing off).  While enabled, every kernel launch
 * of plan/fwd/bwd is bracketed by an event pair on the caller's stream until the
 * pool is used up.  grouter_timing_read synchronises `stream`, adds up the
 * elapsed milliseconds and launch counts per kernel slot, and empties the pool.
 * Slots: 0 plan_hist, 1 plan_permute, 2 gather_X, 3 gemm_up_swiglu, 4 gemm_down,
 * 5 combine_Y, 6 gather_dY, 7 gemm_dH, 8 wgrad_down, 9 gemm_dX, 10 wgrad_gate_up,
 * 11 reduce_dX, 12 zero_split_dW, 13 plan_scan.   total_ms, launches: HOST arrays of GROUTER_NUM_KERNELS entries. */
#define GROUTER_NUM_KERNELS 14
int grouter_timing_enable(grouter_ctx* ctx, int32_t n_records);
/* While timing is enabled, let `microseconds` (0..1000000; 0 = off, the default) of idle time pass on the stream after
 * every timed kernel, so that each kernel is measured on a GPU that is not already at its power cap: the figure to
 * hold against a burst peak, where the back-to-back figure belongs with a sustained peak. */
int grouter_timing_gap(grouter_ctx* ctx, int32_t microseconds);

/* Measurement aid with no counterpart in the paper: where the tensor-core issuers' cycles go.  While enabled (on != 0;
 * off by default), the one MMA-issuing thread of every CTA pair of every grouped GEMM of fwd/bwd adds to five device
 * counters per GEMM: [0] its SM cycles from first tile to last, [1] of these the cycles spent waiting for operand stages
 * to arrive in shared memory, [2] the cycles spent waiting for a free accumulator (epilogue behind), [3] tiles, [4] k-steps
 * (256 x 256 x 64 each; the tensor cores need 512 cycles for one).  grouter_gemm_cycles_read copies the sums since the
 * last read into counters (HOST array of 6 x 5 values, GEMMs in the order up, down, dH, dX, wgrad_down, wgrad_gate_up),
 * zeroes them and synchronises `stream`.  The accounting costs a few clock reads per k-step: leave it off when timing. */
int grouter_gemm_cycles_enable(grouter_ctx* ctx, int32_t on);
int grouter_gemm_cycles_read(grouter_ctx* ctx, void* stream, uint64_t* counters);
int grouter_timing_read(grouter_ctx* ctx, void* stream, float* total_ms, int32_t* launches);

/* Component check of the tensor-core core used by every grouped GEMM (no
 * counterpart in the paper): C[M,N] (f32) = A * B with bf16 operands.
 *   a_mn_major == 0: A stored [M,K] (K contiguous); != 0: A stored [K,M].
 *   b_mn_major == 0: B stored [N,K] (K contiguous); != 0: B stored [K,N].
 * M, N, K multiples of 8.  `status` is a device int32 the kernel ORs error bits into. */
int grouter_dense_gemm(const void* A, int a_mn_major, const void* B, int b_mn_major, float* C, int32_t M, int32_t N,
                       int32_t K, int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GROUTER_H_ */
