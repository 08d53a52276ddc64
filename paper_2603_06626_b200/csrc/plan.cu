// Routing-plan build: a stable counting sort of the R = T*k slots by target
// expert, in two launches.
//
//   plan_hist_kernel    every block histograms a contiguous chunk of slots
//                       (one private histogram per warp, built from warp
//                       ballots so no atomics are needed); the last
//                       block to finish turns the per-block histograms into
//                       exclusive prefixes over blocks, scans the expert
//                       counts into offsets, and lays out the 128-row-padded
//                       segments and the tile list the grouped GEMMs walk.
//   plan_permute_kernel every warp walks its sub-chunk in slot order; the rank
//                       of a slot among equal experts is (block prefix) +
//                       (earlier warps of the block) + (earlier lanes), which
//                       makes the permutation stable and bit-reproducible.
//
// The fold map is the compact form of the paper's binary folding matrix M
// (section "Expert Folding"): e_s = fold_map[idx_s].
#include "common.cuh"

namespace grouter {

// Target expert of a raw id: range check, fold map, range check; a bad id or fold target counts as expert 0.
__device__ __forceinline__ int fold_expert(int raw, const int32_t* __restrict__ fold_map, int E_src, int E_tgt, int32_t* status) {
  bool bad = false;
  if ((unsigned)raw >= (unsigned)E_src) {
    bad = true;
    raw = 0;
  }
  int e = fold_map ? __ldg(fold_map + raw) : raw;
  if ((unsigned)e >= (unsigned)E_tgt) {
    bad = true;
    e = 0;
  }
  if (bad) atomicOr(status, STATUS_BAD_INDEX);
  return e;
}

// Lanes of the warp that hold the same key as this lane (invalid lanes carry key -1 and match each other only).
// One ballot per key bit: constant cost, unlike match.any whose cost grows with the number of distinct keys.
__device__ __forceinline__ unsigned same_key_lanes(int key, int key_bits) {
  unsigned peers = __ballot_sync(0xffffffffu, key >= 0);
  if (key < 0) peers = ~peers;
  for (int b = 0; b < key_bits; ++b) {
    const unsigned ones = __ballot_sync(0xffffffffu, (key >> b) & 1);
    peers &= ((key >> b) & 1) ? ones : ~ones;
  }
  return peers;
}
__device__ __forceinline__ int bits_for(int n) { return n <= 1 ? 0 : 32 - __clz(n - 1); }

// Per-warp histograms of this block's chunk into hist[w*E + e] (smem, pre-zeroed).
template <typename IdxT>
__device__ __forceinline__ void warp_histogram(const IdxT* __restrict__ idx, const int32_t* __restrict__ fold_map, int R, int E_src,
                                               int E_tgt, int chunk, int32_t* hist, int32_t* status) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wlen = chunk / PLAN_WARPS;
  const int base = blockIdx.x * chunk + warp * wlen;
  int32_t* h = hist + warp * E_tgt;
  const int key_bits = bits_for(E_tgt);
  int raw_next = (base + lane < R) ? (int)idx[base + lane] : 0;   // ids are fetched one iteration ahead
  for (int i = 0; i < wlen; i += 32) {
    const int s = base + i + lane;
    const bool valid = s < R;
    const int raw = raw_next;
    if (i + 32 < wlen && s + 32 < R) raw_next = (int)idx[s + 32];
    const int e = valid ? fold_expert(raw, fold_map, E_src, E_tgt, status) : -1;
    const unsigned mask = same_key_lanes(e, key_bits);
    if (valid && lane == __ffs(mask) - 1) h[e] += __popc(mask);
    __syncwarp();
    if (base + i + 32 >= R) break;
  }
}

template <typename IdxT>
__global__ void __launch_bounds__(PLAN_THREADS) plan_hist_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ fold_map,
                                                                 int R, int E_src, int E_tgt, int chunk, int nblk, PaddedPlan pp,
                                                                 int32_t* __restrict__ counts, int32_t* __restrict__ offsets) {
  extern __shared__ int32_t sm[];  // plan_hist_smem_ints(E) ints
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < PLAN_WARPS * E_tgt; i += PLAN_THREADS) sm[i] = 0;
  __syncthreads();
  warp_histogram(idx, fold_map, R, E_src, E_tgt, chunk, sm, pp.status);
  __syncthreads();
  for (int e = tid; e < E_tgt; e += PLAN_THREADS) {
    int tot = 0;
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) tot += sm[w * E_tgt + e];
    pp.blk_prefix[e * nblk + blockIdx.x] = tot;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned t = atomicAdd(pp.ticket, 1u);
    s_last = (t == (unsigned)(nblk - 1));
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- last block: prefixes over blocks, offsets, padded layout, tile list ----
  int32_t* s_cnt = sm;                    // [E]
  int32_t* s_off = sm + E_tgt;            // [E+1]
  int32_t* s_pad = sm + 2 * E_tgt + 1;    // [E+1]
  int32_t* s_pair = sm + 3 * E_tgt + 2;   // [E+1] exclusive prefix of 256-row tiles per expert
  int32_t* s_wch = sm + 4 * E_tgt + 3;    // [E+1] exclusive prefix of weight-gradient row chunks per expert
  int32_t* s_wpos = sm + 5 * E_tgt + 4;   // [2E] list position of each expert's longer / shorter chunks, then [chunk lengths + 1]
  __syncthreads();
  // Exclusive prefix over blocks of every expert's per-block counts (row e of blk_prefix), and the expert totals.
  // Eight lanes share one expert: each sums a contiguous segment of the row with its loads batched eight deep, the
  // eight segment sums are scanned with shuffles, and a second sweep writes the running prefixes back.
  {
    const int grp = lane >> 3, gl = lane & 7;
    const int seg = (nblk + 7) >> 3;
    for (int e0 = warp * 4; e0 < E_tgt; e0 += PLAN_WARPS * 4) {
      const int e = e0 + grp;
      const bool have = e < E_tgt;
      int32_t* rowp = pp.blk_prefix + (size_t)(have ? e : 0) * nblk;
      const int b_lo = min(gl * seg, nblk), b_hi = have ? min(b_lo + seg, nblk) : b_lo;
      int sum = 0;
      for (int b = b_lo; b < b_hi; b += 8) {
        int v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (b + j < b_hi) ? __ldcg(rowp + b + j) : 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) sum += v[j];
      }
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, o, 8);
        if (gl >= o) incl += n;
      }
      int run = incl - sum;
      for (int b = b_lo; b < b_hi; b += 8) {
        int v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (b + j < b_hi) ? __ldcg(rowp + b + j) : 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (b + j < b_hi) rowp[b + j] = run;
          run += v[j];
        }
      }
      if (have && gl == 7) s_cnt[e] = incl;
    }
  }
  __syncthreads();
  if (warp == 0) {
    const int per = (E_tgt + 31) / 32;
    const int e0 = min(lane * per, E_tgt), e1 = min(e0 + per, E_tgt);
    const int chunk_blocks = pp.wgrad_chunk_blocks;
    auto chunks_of = [chunk_blocks](int blocks) { return blocks == 0 ? 1 : (blocks + chunk_blocks - 1) / chunk_blocks; };
    int sum = 0, psum = 0, tsum = 0, wsum = 0;
    for (int e = e0; e < e1; ++e) {
      const int blocks = (s_cnt[e] + ROW_TILE - 1) / ROW_TILE;
      sum += s_cnt[e];
      psum += blocks * ROW_TILE;
      tsum += (blocks + 1) >> 1;
      wsum += chunks_of(blocks);
    }
    int isum = sum, ipsum = psum, itsum = tsum, iwsum = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, isum, o);
      const int b = __shfl_up_sync(0xffffffffu, ipsum, o);
      const int c = __shfl_up_sync(0xffffffffu, itsum, o);
      const int w = __shfl_up_sync(0xffffffffu, iwsum, o);
      if (lane >= o) {
        isum += a;
        ipsum += b;
        itsum += c;
        iwsum += w;
      }
    }
    int off = isum - sum, poff = ipsum - psum, toff = itsum - tsum, woff = iwsum - wsum;
    for (int e = e0; e < e1; ++e) {
      const int blocks = (s_cnt[e] + ROW_TILE - 1) / ROW_TILE;
      s_off[e] = off;
      s_pad[e] = poff;
      s_pair[e] = toff;
      s_wch[e] = woff;
      off += s_cnt[e];
      poff += blocks * ROW_TILE;
      toff += (blocks + 1) >> 1;
      woff += chunks_of(blocks);
    }
    if (lane == 31) {
      s_off[E_tgt] = isum;
      s_pad[E_tgt] = ipsum;
      s_pair[E_tgt] = itsum;
      s_wch[E_tgt] = iwsum;
    }
  }
  __syncthreads();
  for (int e = tid; e <= E_tgt; e += PLAN_THREADS) {
    offsets[e] = s_off[e];
    pp.pad_offsets[e] = s_pad[e];
    if (e < E_tgt) {
      counts[e] = s_cnt[e];
      pp.row_shift[e] = s_pad[e] - s_off[e];
      pp.pad_begin[e] = s_pad[e] + s_cnt[e];
    }
  }
  const int n_tiles = s_pair[E_tgt];
  if (tid == 0) {
    *pp.n_pair_tiles = n_tiles;
    *pp.ticket = 0u;  // ready for the next plan
    *pp.tile_counter = 0u;  // a grouped GEMM that gave up on a timeout may have left it mid-count
  }
  // expert and first row of every 256-row tile: the last e with s_pair[e] <= t owns tile t
  for (int t = tid; t < n_tiles; t += PLAN_THREADS) {
    int lo = 0, hi = E_tgt;  // invariant: s_pair[lo] <= t < s_pair[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_pair[mid] <= t) lo = mid; else hi = mid;
    }
    const int row0 = s_pad[lo] + (t - s_pair[lo]) * 2 * ROW_TILE;
    pp.pair_row0[t] = row0;
    pp.pair_expert[t] = lo | (row0 + ROW_TILE < s_pad[lo + 1] ? PAIR_VALID2 : 0);
  }
  // Row chunks of the weight-gradient GEMMs: an expert without slots keeps one empty chunk (its gradient is zero-filled).
  // An expert's blocks are cut into n chunks of near-equal size: `rem` chunks of base + 1 blocks, then n - rem of base.
  // The list is ordered by chunk length, longest first, in WGRAD_LEN_BUCKETS classes of length (within a class by
  // expert, then by position): tiles of similar cost are neighbours, and the shortest tiles at the end even out the tail.
  if (tid == 0) *pp.n_wchunks = s_wch[E_tgt];
  {
    const int chunk_blocks = pp.wgrad_chunk_blocks;
    auto len_class = [chunk_blocks](int blocks) { return (blocks * WGRAD_LEN_BUCKETS + chunk_blocks - 1) / chunk_blocks; };   // 0 .. BUCKETS
    // chunks of every class, then the first list position of every class (descending)
    int32_t* s_len = s_wpos + 2 * E_tgt;   // [WGRAD_LEN_BUCKETS + 1]
    for (int i = tid; i <= WGRAD_LEN_BUCKETS; i += PLAN_THREADS) s_len[i] = 0;
    __syncthreads();
    for (int e = tid; e < E_tgt; e += PLAN_THREADS) {
      const int blocks = (s_pad[e + 1] - s_pad[e]) / ROW_TILE;
      const int n = s_wch[e + 1] - s_wch[e];
      const int base = blocks / n, rem = blocks - base * n;
      if (rem) atomicAdd(&s_len[len_class(base + 1)], rem);
      atomicAdd(&s_len[len_class(base)], n - rem);
    }
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int l = WGRAD_LEN_BUCKETS; l >= 0; --l) {
        const int c = s_len[l];
        s_len[l] = run;
        run += c;
      }
    }
    __syncthreads();
    // within one class: experts in ascending order, an expert's longer chunks before its shorter ones.  One warp per
    // class walks the experts 32 at a time.
    for (int l = warp; l <= WGRAD_LEN_BUCKETS; l += PLAN_WARPS) {
      int run = s_len[l];
      for (int e0 = 0; e0 < E_tgt; e0 += 32) {
        const int e = e0 + lane;
        int c0 = 0, c1 = 0;    // chunks of the expert's two lengths that fall into class l
        if (e < E_tgt) {
          const int blocks = (s_pad[e + 1] - s_pad[e]) / ROW_TILE;
          const int n = s_wch[e + 1] - s_wch[e];
          const int base = blocks / n, rem = blocks - base * n;
          if (rem && len_class(base + 1) == l) c0 = rem;
          if (len_class(base) == l) c1 = n - rem;
        }
        int incl = c0 + c1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        const int first = run + incl - (c0 + c1);
        if (c0) s_wpos[e] = first;
        if (c1) s_wpos[E_tgt + e] = first + c0;
        run += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
    __syncthreads();
  }
  for (int e = tid; e < E_tgt; e += PLAN_THREADS) {
    const int blocks = (s_pad[e + 1] - s_pad[e]) / ROW_TILE;
    const int n = s_wch[e + 1] - s_wch[e];
    const int base = blocks / n, rem = blocks - base * n;
    for (int c = 0; c < n; ++c) {
      const int i = c < rem ? s_wpos[e] + c : s_wpos[E_tgt + e] + (c - rem);
      pp.wchunk_expert[i] = e | (n > 1 ? WCHUNK_SPLIT : 0);
      pp.wchunk_row0[i] = s_pad[e] + (c * base + min(c, rem)) * ROW_TILE;
      int rows = (base + (c < rem ? 1 : 0)) * ROW_TILE;
      // the contraction runs in steps of 64 rows: when the expert's last block holds at most 64 real rows, its second
      // half is all padding (zeros) and is left out
      const int tail = s_cnt[e] & (ROW_TILE - 1);
      if (c == n - 1 && tail >= 1 && tail <= ROW_TILE / 2) rows -= ROW_TILE / 2;
      pp.wchunk_rows[i] = rows;
    }
  }
  // pad rows carry no slot
  for (int e = warp; e < E_tgt; e += PLAN_WARPS) {
    const int r0 = s_pad[e] + s_cnt[e], r1 = s_pad[e + 1];
    for (int r = r0 + lane; r < r1; r += 32) pp.prow_to_slot[r] = -1;
  }
}

template <typename IdxT>
__global__ void __launch_bounds__(PLAN_THREADS) plan_permute_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ fold_map,
                                                                    int R, int E_src, int E_tgt, int chunk, int nblk, PaddedPlan pp,
                                                                    const int32_t* __restrict__ offsets, int32_t* __restrict__ row_to_slot,
                                                                    int32_t* __restrict__ slot_to_row) {
  extern __shared__ int32_t sm[];  // PLAN_WARPS*E + E ints
  int32_t* s_shift = sm + PLAN_WARPS * E_tgt;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < PLAN_WARPS * E_tgt; i += PLAN_THREADS) sm[i] = 0;
  __syncthreads();
  warp_histogram(idx, fold_map, R, E_src, E_tgt, chunk, sm, pp.status);
  __syncthreads();
  // per-warp histogram -> first row of (block, warp, expert)
  for (int e = tid; e < E_tgt; e += PLAN_THREADS) {
    int base = offsets[e] + pp.blk_prefix[e * nblk + blockIdx.x];
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) {
      const int t = sm[w * E_tgt + e];
      sm[w * E_tgt + e] = base;
      base += t;
    }
    s_shift[e] = pp.row_shift[e];
  }
  __syncthreads();
  const int wlen = chunk / PLAN_WARPS;
  const int base = blockIdx.x * chunk + warp * wlen;
  int32_t* cur = sm + warp * E_tgt;
  const unsigned lt = (1u << lane) - 1u;
  const int key_bits = bits_for(E_tgt);
  int raw_next = (base + lane < R) ? (int)idx[base + lane] : 0;   // ids are fetched one iteration ahead
  for (int i = 0; i < wlen; i += 32) {
    const int s = base + i + lane;
    const bool valid = s < R;
    const int raw = raw_next;
    if (i + 32 < wlen && s + 32 < R) raw_next = (int)idx[s + 32];
    const int e = valid ? fold_expert(raw, fold_map, E_src, E_tgt, pp.status) : -1;
    const unsigned mask = same_key_lanes(e, key_bits);
    const int row = valid ? cur[e] + __popc(mask & lt) : 0;
    __syncwarp();
    if (valid && lane == 31 - __clz(mask)) cur[e] = row + 1;
    __syncwarp();
    if (valid) {
      const int prow = row + s_shift[e];
      slot_to_row[s] = row;
      row_to_slot[row] = s;
      pp.slot_to_prow[s] = prow;
      pp.prow_to_slot[prow] = s;
    }
    if (base + i + 32 >= R) break;
  }
}

// per-warp histograms while counting; the last block's scans and chunk ordering afterwards
static int plan_hist_smem_ints(int E) {
  const int a = PLAN_WARPS * E, b = 7 * E + 4 + WGRAD_LEN_BUCKETS + 2;
  return a > b ? a : b;
}

template <typename IdxT>
static cudaError_t launch_plan_t(grouter_ctx* ctx, int phase, const IdxT* idx, const int32_t* fold_map, int32_t* counts,
                                 int32_t* offsets, int32_t* row_to_slot, int32_t* slot_to_row, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  const int R = (int)ctx->R, E = dm.E_tgt;
  const int chunk = ctx->geom.chunk, nblk = ctx->geom.nblk;
  if (phase == 0) {
    const size_t sm1 = sizeof(int32_t) * (size_t)plan_hist_smem_ints(E);
    plan_hist_kernel<IdxT><<<nblk, PLAN_THREADS, sm1, st>>>(idx, fold_map, R, dm.E_src, E, chunk, nblk, ctx->pp, counts, offsets);
  } else {
    const size_t sm2 = sizeof(int32_t) * (size_t)(PLAN_WARPS * E + E);
    plan_permute_kernel<IdxT><<<nblk, PLAN_THREADS, sm2, st>>>(idx, fold_map, R, dm.E_src, E, chunk, nblk, ctx->pp, offsets,
                                                               row_to_slot, slot_to_row);
  }
  return cudaGetLastError();
}

// phase 0: histogram + scans (counts, offsets, padded layout); phase 1: stable permutation.
cudaError_t launch_plan(grouter_ctx* ctx, int phase, const void* idx, const int32_t* fold_map, int32_t* counts, int32_t* offsets,
                        int32_t* row_to_slot, int32_t* slot_to_row, cudaStream_t st) {
  if (ctx->dims.idx_dtype == GROUTER_IDX_U8)
    return launch_plan_t<uint8_t>(ctx, phase, (const uint8_t*)idx, fold_map, counts, offsets, row_to_slot, slot_to_row, st);
  return launch_plan_t<int32_t>(ctx, phase, (const int32_t*)idx, fold_map, counts, offsets, row_to_slot, slot_to_row, st);
}

}  // namespace grouter

// ------------------------------------------------------------------------
// grouter_plan_noalloc: the same two plan kernels, run without a context.
//
// grouter_create owns the plan's scratch (per-block histograms, the ticket of
// the last-block scan, the padded copy of the permutation) in memory it gets
// from cudaMalloc.  Some hosts cannot make that call: a process that has
// handed the whole device to a pooling allocator with a fixed reservation, a
// plug-in running under a memory budget it may not exceed, or a
// latency-critical loop that cannot take the device-wide synchronisation an
// allocation implies.  For them the scratch lives in the library image itself:
// one file-scope __device__ array that every GPU loading the library holds
// until the process exits.  Its size fixes the largest problem this entry
// point accepts.
// ------------------------------------------------------------------------
namespace grouter {
namespace {

constexpr int NOALLOC_MAX_R = 1 << 19;       // routed slots T*k
constexpr int NOALLOC_MAX_E = 256;           // target experts
constexpr int NOALLOC_MAX_ROWS = NOALLOC_MAX_R + ROW_TILE * NOALLOC_MAX_E;          // padded rows
constexpr int NOALLOC_MAX_BLOCKS = NOALLOC_MAX_R / PLAN_MIN_CHUNK;                   // plan_geom never uses more
// layout of the scratch, in 32-bit words (every part starts on a 256-byte boundary)
constexpr int NA_PAD_OFFSETS = 0;                                     // [E+1]
constexpr int NA_ROW_SHIFT = NA_PAD_OFFSETS + 320;                    // [E]
constexpr int NA_PAD_BEGIN = NA_ROW_SHIFT + 256;                      // [E]
constexpr int NA_N_TILES = NA_PAD_BEGIN + 256;                        // [1]
constexpr int NA_TICKET = NA_N_TILES + 64;                            // [1]
constexpr int NA_STATUS = NA_TICKET + 64;                             // [1] used when the caller passes no status word
constexpr int NA_PAIR_ROW0 = NA_STATUS + 64;                          // [rows/128]
constexpr int NA_PAIR_EXPERT = NA_PAIR_ROW0 + NOALLOC_MAX_ROWS / ROW_TILE;     // [rows/128]
constexpr int NOALLOC_MAX_WCHUNKS = (NOALLOC_MAX_E + NOALLOC_MAX_ROWS / WGRAD_KCHUNK_MAX + 1 + 63) / 64 * 64;
constexpr int NA_WCHUNK_EXPERT = NA_PAIR_EXPERT + NOALLOC_MAX_ROWS / ROW_TILE; // [chunks]
constexpr int NA_WCHUNK_ROW0 = NA_WCHUNK_EXPERT + NOALLOC_MAX_WCHUNKS;         // [chunks]
constexpr int NA_WCHUNK_ROWS = NA_WCHUNK_ROW0 + NOALLOC_MAX_WCHUNKS;           // [chunks]
constexpr int NA_N_WCHUNKS = NA_WCHUNK_ROWS + NOALLOC_MAX_WCHUNKS;             // [1]
constexpr int NA_SLOT_TO_PROW = NA_N_WCHUNKS + 64;                             // [R]
constexpr int NA_PROW_TO_SLOT = NA_SLOT_TO_PROW + NOALLOC_MAX_R;      // [rows]
constexpr int NA_BLK_PREFIX = NA_PROW_TO_SLOT + NOALLOC_MAX_ROWS;     // [E * blocks]
constexpr int NA_WORDS = NA_BLK_PREFIX + NOALLOC_MAX_E * NOALLOC_MAX_BLOCKS;
static_assert(NA_PAIR_ROW0 % 64 == 0 && NA_PAIR_EXPERT % 64 == 0 && NA_SLOT_TO_PROW % 64 == 0 && NA_PROW_TO_SLOT % 64 == 0 && NA_BLK_PREFIX % 64 == 0,
              "scratch parts must start on 256-byte boundaries");

// About 4.6 MB per GPU.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a
// device address and must never be handed to a kernel as one.
static __device__ __align__(256) int32_t g_plan_scratch[NA_WORDS];

constexpr int NOALLOC_MAX_DEVICES = 64;
int32_t* g_plan_scratch_addr[NOALLOC_MAX_DEVICES] = {};   // device address of the array, per device, once looked up

// Device address of this device's copy of the scratch array (looked up on the first call per device).
int32_t* plan_scratch_on_current_device(int* rc) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) {
    *rc = GROUTER_ERR_NO_DEVICE;
    return nullptr;
  }
  int32_t* p = __atomic_load_n(&g_plan_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (p == nullptr) {
    void* sym = nullptr;
    if (cudaGetSymbolAddress(&sym, g_plan_scratch) != cudaSuccess || sym == nullptr) {
      *rc = GROUTER_ERR_CUDA;
      return nullptr;
    }
    p = static_cast<int32_t*>(sym);
    __atomic_store_n(&g_plan_scratch_addr[dev], p, __ATOMIC_RELEASE);   // racing threads store the same value
  }
  *rc = GROUTER_OK;
  return p;
}

}  // namespace
}  // namespace grouter

extern "C" int grouter_plan_noalloc(const void* idx, int32_t idx_dtype, const int32_t* fold_map, int32_t T, int32_t k, int32_t E_src,
                                    int32_t E_tgt, int32_t* counts, int32_t* offsets, int32_t* row_to_slot, int32_t* slot_to_row,
                                    int32_t* status, void* stream) {
  using namespace grouter;
  if (!idx || !counts || !offsets || !row_to_slot || !slot_to_row) return GROUTER_ERR_INVALID_ARG;
  if (T < 1 || k < 1 || E_src < 1 || E_tgt < 1) return GROUTER_ERR_INVALID_ARG;
  if (idx_dtype != GROUTER_IDX_U8 && idx_dtype != GROUTER_IDX_I32) return GROUTER_ERR_INVALID_ARG;
  if (!fold_map && E_src != E_tgt) return GROUTER_ERR_INVALID_ARG;
  if (idx_dtype == GROUTER_IDX_U8 && E_src > 256) return GROUTER_ERR_UNSUPPORTED;
  // beyond the fixed scratch: the caller has to use grouter_create + grouter_plan
  if ((int64_t)T * k > NOALLOC_MAX_R || E_tgt > NOALLOC_MAX_E) return GROUTER_ERR_UNSUPPORTED;
  auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (misaligned(idx) || misaligned(counts) || misaligned(offsets) || misaligned(row_to_slot) || misaligned(slot_to_row) ||
      (fold_map && misaligned(fold_map)) || (status && (reinterpret_cast<uintptr_t>(status) & 3u)))
    return GROUTER_ERR_MISALIGNED;
  int rc = GROUTER_OK;
  int32_t* base = plan_scratch_on_current_device(&rc);
  if (!base) return rc;

  grouter_ctx c{};   // lives on the host stack for the duration of the two launches
  c.dims.T = T; c.dims.d = 8; c.dims.ffn = 8; c.dims.E_src = E_src; c.dims.E_tgt = E_tgt; c.dims.k = k;
  c.dims.idx_dtype = idx_dtype; c.dims.gate_dtype = GROUTER_GATE_BF16;
  c.R = (int64_t)T * k;
  c.geom = plan_geom(c.R);
  c.pp.pad_offsets = base + NA_PAD_OFFSETS;
  c.pp.row_shift = base + NA_ROW_SHIFT;
  c.pp.pad_begin = base + NA_PAD_BEGIN;
  c.pp.n_pair_tiles = base + NA_N_TILES;
  c.pp.ticket = reinterpret_cast<unsigned int*>(base + NA_TICKET);
  c.pp.tile_counter = c.pp.ticket + 4;
  c.pp.wgrad_chunk_blocks = WGRAD_KCHUNK_MAX / ROW_TILE;   // the chunk list is scratch here: fewest entries
  c.pp.status = status ? status : base + NA_STATUS;
  c.pp.pair_row0 = base + NA_PAIR_ROW0;
  c.pp.pair_expert = base + NA_PAIR_EXPERT;
  c.pp.wchunk_expert = base + NA_WCHUNK_EXPERT;
  c.pp.wchunk_row0 = base + NA_WCHUNK_ROW0;
  c.pp.wchunk_rows = base + NA_WCHUNK_ROWS;
  c.pp.n_wchunks = base + NA_N_WCHUNKS;
  c.pp.slot_to_prow = base + NA_SLOT_TO_PROW;
  c.pp.prow_to_slot = base + NA_PROW_TO_SLOT;
  c.pp.blk_prefix = base + NA_BLK_PREFIX;
  if (c.geom.nblk > NOALLOC_MAX_BLOCKS) return GROUTER_ERR_UNSUPPORTED;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array still holds whatever the previous call left.  The ticket must count from zero and the status
  // word must start clear; every other part is overwritten before it is read.
  if (cudaMemsetAsync(c.pp.ticket, 0, sizeof(unsigned int), st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (cudaMemsetAsync(c.pp.status, 0, sizeof(int32_t), st) != cudaSuccess) return GROUTER_ERR_CUDA;
  for (int phase = 0; phase < 2; ++phase)
    if (launch_plan(&c, phase, idx, fold_map, counts, offsets, row_to_slot, slot_to_row, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}
