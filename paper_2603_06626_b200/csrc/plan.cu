// Routing-plan build: a stable counting sort of the R = T*k slots by target
// expert, in three launches.
//
//   phase 0  per-block histograms       every block counts the experts of a contiguous chunk of slots
//   phase 1  scans and layout           one block per expert turns its row of per-block counts into exclusive
//                                       prefixes over blocks; the last block to finish scans the expert totals into
//                                       offsets, lays out the 128-row-padded segments and orders the work list of
//                                       the weight-gradient GEMMs
//   phase 2  stable permutation         rank of a slot among equal experts = (earlier blocks) + (earlier slots of
//                                       this block); also writes the tile list of the row-parallel GEMMs
//
// Phases 0 and 2 come in two forms.
//   counted (E_tgt <= 256, fold table in shared memory): a thread owns a run of 16-64 consecutive slots, fetched with
//     16-byte loads, and a private 16-bit counter per expert in shared memory (no atomics, no warp votes).  A scan over
//     the threads' counters gives every thread its first rank per expert; the thread then walks its run once more,
//     handing out ranks in slot order.  The ranks fill a shared-memory staging array ordered by (expert, rank), so
//     row_to_slot is written in contiguous runs, one per expert and chunk, in pieces of at most 128 entries shared out
//     among the warps; every slot's row is parked in shared memory on the way and slot_to_row leaves as one
//     contiguous copy.  With many chunks a block takes several in turn and fetches the next one's ids while it writes
//     the current one out.
//   ballot (any E_tgt up to 1024, any E_src): a warp walks its sub-chunk 32 slots at a time; lanes with equal keys are
//     found with one vote per key bit.
// Both are bit-reproducible: no result depends on the order in which threads or blocks run.
//
// The fold map is the compact form of the paper's binary folding matrix M
// (section "Expert Folding"): e_s = fold_map[idx_s].
#include <type_traits>
#include "common.cuh"

namespace grouter {

// Programmatic dependent launch between the plan's three kernels: a kernel lets its successor's blocks be scheduled
// early (launch_successor), and the successor does whatever needs none of the predecessor's results (clearing its
// counters, loading the fold table) before it waits for the predecessor to finish and its writes to be visible
// (wait_for_predecessor).  On a plain launch both are no-ops.
__device__ __forceinline__ void launch_successor() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ int bits_for(int n) { return n <= 1 ? 0 : 32 - __clz(n - 1); }

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// ------------------------------------------------------------------------------------------------------------------
// Counted form
// ------------------------------------------------------------------------------------------------------------------

// How raw ids become target experts.  `table` (shared memory, one 16-bit entry per source id) holds the fold target, or
// 0x8000 for a target outside [0, E_tgt); without a fold map the id is the target.
struct FoldView {
  const uint16_t* table;   // null: identity
  int E_src;
  bool plain;              // 8-bit ids, no fold map, E_src == 256: every byte is a valid target as it stands
};

__device__ __forceinline__ uint32_t fold_one(uint32_t raw, const FoldView& f, int& bad) {
  if (raw >= (uint32_t)f.E_src) {
    bad = 1;
    raw = 0;
  }
  if (f.table == nullptr) return raw;
  const uint32_t t = f.table[raw];
  if (t & 0x8000u) bad = 1;
  return t & 0xffu;
}

// Target experts of 16 slots whose 8-bit ids are in registers: v = the 16 bytes at slot s (a multiple of 16), zeros at
// or beyond R; slots at or beyond R are not checked.
__device__ __forceinline__ uint4 check_targets16(const uint4& v, int s, int R, const FoldView& f, int& bad) {
  uint32_t w[4] = {v.x, v.y, v.z, v.w};
  if (!f.plain) {
    const int n = min(16, max(0, R - s));
    // without a fold map a valid id is its own target: test four bytes at once for id >= E_src (bit 7 of a byte of
    // `over`), and take the byte-by-byte path only for a word that holds a bad id, a fold table, or the ragged end
    const uint32_t add = (uint32_t)((f.E_src <= 128 ? 128 - f.E_src : 256 - f.E_src) * 0x01010101);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (f.table == nullptr && q * 4 + 4 <= n) {
        const uint32_t t = ((w[q] & 0x7f7f7f7fu) + add) & 0x80808080u;     // low seven bits reach the bound
        const uint32_t over = f.E_src <= 128 ? (t | (w[q] & 0x80808080u)) : (t & w[q]);
        if (over == 0u) continue;
      }
      uint32_t o = 0u;
#pragma unroll
      for (int b = 0; b < 4; ++b)
        if (q * 4 + b < n) o |= fold_one((w[q] >> (8 * b)) & 0xffu, f, bad) << (8 * b);
      w[q] = o;
    }
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// Target experts of the 16 slots s .. s+15 as 16 bytes (slot s+i in byte i); slots at or beyond R read as 0 and are
// not checked.  s is a multiple of 16 and idx is 16-byte aligned, so every 16-byte load is aligned and holds at least
// one valid id: it cannot leave the page the ids end in.
template <typename IdxT>
__device__ __forceinline__ uint4 load_targets16(const IdxT* __restrict__ idx, int s, int R, const FoldView& f, int& bad) {
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  if (sizeof(IdxT) == 1) {
    const uint4 v = s < R ? ld_nc_v4(reinterpret_cast<const uint8_t*>(idx) + s) : make_uint4(0u, 0u, 0u, 0u);
    return check_targets16(v, s, R, f, bad);
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (s + 4 * q < R) {
        const uint4 v = ld_nc_v4(reinterpret_cast<const int32_t*>(idx) + s + 4 * q);
        const uint32_t r[4] = {v.x, v.y, v.z, v.w};
        uint32_t o = 0u;
#pragma unroll
        for (int b = 0; b < 4; ++b)
          if (s + 4 * q + b < R) o |= fold_one(r[b], f, bad) << (8 * b);
        w[q] = o;
      }
    }
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// Fold table into shared memory (one thread per entry, strided); returns the view the item loops use.
template <typename IdxT>
__device__ __forceinline__ FoldView make_fold_view(const int32_t* __restrict__ fold_map, int E_src, int E_tgt, uint16_t* s_fold) {
  FoldView f;
  f.E_src = E_src;
  f.table = fold_map ? s_fold : nullptr;
  f.plain = sizeof(IdxT) == 1 && fold_map == nullptr && E_src == 256;
  if (fold_map)
    for (int i = threadIdx.x; i < E_src; i += PLAN_THREADS) {
      const int t = __ldg(fold_map + i);
      s_fold[i] = (unsigned)t < (unsigned)E_tgt ? (uint16_t)t : (uint16_t)0x8000u;
    }
  return f;
}

// Private counters of the counted form.  Every thread keeps one 16-bit counter per expert in shared memory; threads t
// and t + 128 share the 32-bit word [e][t & 127] (low and high half), so the 32 lanes of a warp always touch 32
// different banks whatever their experts are, and a counter's address is e * 512 + a per-thread constant.  A thread
// reads and writes only its own halves (16-bit accesses), so nothing needs an atomic: shared-memory atomics cost about
// ten cycles per warp instruction here, conflict-free or not, which made both walks slower than plain loads and stores.
// To keep several loads in flight the walks take four slots at a time: four loads, then the ranks are corrected in
// registers for equal experts among the four, then four stores in slot order (a later store of the same counter holds
// the larger value).  No half can overflow: every value stays at or below the block's slot count (at most 16384).
constexpr int CNT_ROW_WORDS = PLAN_THREADS / 2;     // words per expert row

// (32-bit registers on both: a load zero-extends into a wider register and a store takes the low half of one, so no
// conversion instructions surround them)
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts_u16(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// Shared-memory address of this thread's counter of expert 0; the one of expert e lies e * 512 bytes further.
__device__ __forceinline__ uint32_t my_counters(const uint32_t* s_cnt) {
  return (uint32_t)__cvta_generic_to_shared(s_cnt) + 4u * (threadIdx.x & (CNT_ROW_WORDS - 1)) + (threadIdx.x >= CNT_ROW_WORDS ? 2u : 0u);
}
// Four slots (experts in the bytes of w, slot order = byte order; only the first n are real): bumps their counters and
// returns the values the counters held before each slot's own bump.
__device__ __forceinline__ void bump4(uint32_t mine, uint32_t w, int n, uint32_t (&before)[4]) {
  const uint32_t a0 = mine + ((w & 0xffu) << 9), a1 = mine + ((w & 0xff00u) << 1), a2 = mine + ((w & 0xff0000u) >> 7),
                 a3 = mine + ((w >> 24) << 9);
  uint32_t c0 = lds_u16(a0), c1 = lds_u16(a1), c2 = lds_u16(a2), c3 = lds_u16(a3);
  c1 += (a1 == a0);
  c2 += (a2 == a0) + (a2 == a1);
  c3 += (a3 == a0) + (a3 == a1) + (a3 == a2);
  before[0] = c0; before[1] = c1; before[2] = c2; before[3] = c3;
  if (n >= 4) {
    sts_u16(a0, c0 + 1u);
    sts_u16(a1, c1 + 1u);
    sts_u16(a2, c2 + 1u);
    sts_u16(a3, c3 + 1u);
  } else {
    if (n > 0) sts_u16(a0, c0 + 1u);
    if (n > 1) sts_u16(a1, c1 + 1u);
    if (n > 2) sts_u16(a2, c2 + 1u);
  }
}

// Tile list of the row-parallel GEMMs, written by the threads of phase 2 before they start on the permutation:
// expert and first padded row of every 256-row tile.  The last e with pair_prefix[e] <= t owns tile t.
// s_pp / s_po: shared-memory copies of pair_prefix and pad_offsets, E_tgt + 1 entries each.
__device__ __forceinline__ void write_tile_list(const PaddedPlan& pp, int E_tgt, int32_t* s_pp, int32_t* s_po) {
  for (int e = threadIdx.x; e <= E_tgt; e += PLAN_THREADS) {
    s_pp[e] = pp.pair_prefix[e];
    s_po[e] = pp.pad_offsets[e];
  }
  __syncthreads();
  const int n_tiles = s_pp[E_tgt];
  for (int t = blockIdx.x * PLAN_THREADS + threadIdx.x; t < n_tiles; t += gridDim.x * PLAN_THREADS) {
    int lo = 0, hi = E_tgt;  // invariant: s_pp[lo] <= t < s_pp[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_pp[mid] <= t) lo = mid; else hi = mid;
    }
    const int row0 = s_po[lo] + (t - s_pp[lo]) * 2 * ROW_TILE;
    if (!GROUTER_CHECKED(t < pp.max_m_tiles, pp.status)) continue;
    pp.pair_row0[t] = row0;
    pp.pair_expert[t] = lo | (row0 + ROW_TILE < s_po[lo + 1] ? PAIR_VALID2 : 0);
  }
}

// Phase 0, counted form: per-warp histograms with shared-memory adds (a word of four equal ids is one add of 4).
// Shared-memory atomics cost about ten cycles per warp instruction here, with or without conflicts; private counters
// as in phase 2 (no atomics, but 512 bytes of counters per expert to clear and to sum per block) were measured slower
// for this kernel, which needs nothing but the block's totals.
template <typename IdxT, int V>
__global__ void __launch_bounds__(PLAN_THREADS) plan_count_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ fold_map,
                                                                  int R, int E_src, int E_tgt, int nblk,
                                                                  int32_t* __restrict__ blk_hist, int32_t* __restrict__ status) {
  constexpr int IPT = 16 * V;
  constexpr int CHUNK = IPT * PLAN_THREADS;
  extern __shared__ __align__(16) uint32_t sm_u32[];
  uint32_t* s_hist = sm_u32;                                                       // [PLAN_WARPS][E_tgt]
  uint16_t* s_fold = reinterpret_cast<uint16_t*>(sm_u32 + PLAN_WARPS * E_tgt);     // [E_src]
  const int tid = threadIdx.x, warp = tid >> 5;
  launch_successor();
  for (int i = tid; i < PLAN_WARPS * E_tgt; i += PLAN_THREADS) s_hist[i] = 0u;
  const FoldView f = make_fold_view<IdxT>(fold_map, E_src, E_tgt, s_fold);
  __syncthreads();
  uint32_t* h = s_hist + warp * E_tgt;
  const int s0 = blockIdx.x * CHUNK + tid * IPT;
  const int n_mine = min(IPT, max(0, R - s0));
  int bad = 0;
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const uint4 ev = load_targets16<IdxT>(idx, s0 + 16 * v, R, f, bad);
    const uint32_t w[4] = {ev.x, ev.y, ev.z, ev.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int nq = n_mine - (16 * v + 4 * q);
      if (nq >= 4 && w[q] == __byte_perm(w[q], 0u, 0x0321)) {
        atomicAdd(h + (w[q] & 0xffu), 4u);
      } else {
#pragma unroll
        for (int b = 0; b < 4; ++b)
          if (b < nq) atomicAdd(h + ((w[q] >> (8 * b)) & 0xffu), 1u);
      }
    }
  }
  if (bad) atomicOr(status, STATUS_BAD_INDEX);
  __syncthreads();
  for (int e = tid; e < E_tgt; e += PLAN_THREADS) {
    uint32_t tot = 0u;
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) tot += s_hist[w * E_tgt + e];
    blk_hist[(size_t)e * nblk + blockIdx.x] = (int32_t)tot;
  }
}

constexpr int PLACE_SEG = 128;        // positions of the staging array one warp copies out at a time

// Shared-memory layout of plan_place_kernel, in bytes from the start of the dynamic block.
struct PlaceSmem {
  int cnt, stage, first, seg, fold, pp, po, bytes;
};
__host__ __device__ inline PlaceSmem place_smem(int E_src, int E_tgt, int ipt, bool with_fold) {
  PlaceSmem m;
  int off = 0;
  auto take = [&](int n) { const int o = off; off += (n + 15) / 16 * 16; return o; };
  const int cnt_bytes = E_tgt * CNT_ROW_WORDS * 4, row_bytes = ipt * PLAN_THREADS * 4;
  m.cnt = take(cnt_bytes > row_bytes ? cnt_bytes : row_bytes);   // private counters; afterwards the row of every slot of the chunk
  m.stage = take(ipt * PLAN_THREADS * 2);       // slot (as its index within the chunk) at every (expert, rank) position
  m.first = take(E_tgt * 4);                    // per expert: first staging position
  m.seg = take((ipt * PLAN_THREADS / PLACE_SEG + E_tgt) * 8);   // pieces of at most PLACE_SEG positions, none across two experts
  m.fold = take(with_fold ? E_src * 2 : 0);
  m.pp = take((E_tgt + 1) * 4);
  m.po = take((E_tgt + 1) * 4);
  m.bytes = off;
  return m;
}

// Phase 2, counted form.  A block takes chunks blockIdx.x, blockIdx.x + gridDim.x, ...; the ids and the per-expert
// prefixes of its next chunk are fetched while the current one is written out.
template <typename IdxT, int V>
__global__ void __launch_bounds__(PLAN_THREADS, 2) plan_place_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ fold_map,
                                                                     int R, int E_src, int E_tgt, int nblk, PaddedPlan pp,
                                                                     const int32_t* __restrict__ offsets, int32_t* __restrict__ row_to_slot,
                                                                     int32_t* __restrict__ slot_to_row) {
  constexpr int IPT = 16 * V;
  constexpr int CHUNK = IPT * PLAN_THREADS;
  constexpr bool BYTES = sizeof(IdxT) == 1;     // 8-bit ids are fetched ahead as they are; wider ones are folded as they are read
  static_assert(CHUNK <= 32768, "ranks within a block are kept in 16 bits, two to a word");
  extern __shared__ __align__(16) uint8_t sm_raw[];
  const PlaceSmem L = place_smem(E_src, E_tgt, IPT, fold_map != nullptr);
  uint32_t* s_cnt = reinterpret_cast<uint32_t*>(sm_raw + L.cnt);
  uint16_t* s_stage = reinterpret_cast<uint16_t*>(sm_raw + L.stage);
  int32_t* s_rows = reinterpret_cast<int32_t*>(sm_raw + L.cnt);     // the counters' space, once they are no longer needed
  int32_t* s_first = reinterpret_cast<int32_t*>(sm_raw + L.first);
  int2* s_seg = reinterpret_cast<int2*>(sm_raw + L.seg);
  uint16_t* s_fold = reinterpret_cast<uint16_t*>(sm_raw + L.fold);
  __shared__ uint32_t s_warp_sum[PLAN_WARPS];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  uint4 ev[V];
  auto fetch_ids = [&](int c) {
    if (BYTES) {
      const int s = c * CHUNK + tid * IPT;
#pragma unroll
      for (int v = 0; v < V; ++v)
        ev[v] = s + 16 * v < R ? ld_nc_v4(reinterpret_cast<const uint8_t*>(idx) + s + 16 * v) : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  // Expert tid's slots in the chunks before chunk c and up to its end, from the prefixes over blocks that phase 1 left.
  // Nothing is computed from the two values here: the loads stay in flight until the next chunk's set-up reads them.
  int before_e = 0, upto_e = 0, off_e = 0, total_e = 0;
  auto fetch_prefix = [&](int c) {
    if (tid < E_tgt) {
      const int32_t* rowp = pp.blk_prefix + (size_t)tid * nblk + c;
      before_e = __ldcg(rowp);
      upto_e = c + 1 < nblk ? __ldcg(rowp + 1) : total_e;
    }
  };

  fetch_ids(blockIdx.x);                         // in flight while the block sets itself up
  const FoldView f = make_fold_view<IdxT>(fold_map, E_src, E_tgt, s_fold);
  wait_for_predecessor();                        // everything below reads what phase 1 wrote
  if (tid < E_tgt) {
    off_e = __ldg(offsets + tid);
    total_e = __ldg(offsets + tid + 1) - off_e;
  }
  fetch_prefix(blockIdx.x);
  if (blockIdx.x * PLAN_THREADS < __ldg(pp.pair_prefix + E_tgt))
    write_tile_list(pp, E_tgt, reinterpret_cast<int32_t*>(sm_raw + L.pp), reinterpret_cast<int32_t*>(sm_raw + L.po));
  const uint32_t mine = my_counters(s_cnt);
  const uint32_t stage_addr = (uint32_t)__cvta_generic_to_shared(s_stage);

  for (int c = blockIdx.x; c < nblk; c += gridDim.x) {
    const int chunk0 = c * CHUNK;
    const int s0 = chunk0 + tid * IPT;
    const int n_mine = min(IPT, max(0, R - s0));
    {
      uint4* z = reinterpret_cast<uint4*>(s_cnt);
      for (int i = tid; i < E_tgt * CNT_ROW_WORDS / 4; i += PLAN_THREADS) z[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    // ---- per expert (E_tgt <= 256 = one per thread): exclusive scans over the experts of the slot counts (= the
    // expert's first position in the staging array) and of the piece counts, in one word; then the expert's pieces ----
    int n_seg;
    {
      const int e = tid, cnt_e = upto_e - before_e;
      const uint32_t both = (uint32_t)cnt_e | ((uint32_t)((cnt_e + PLACE_SEG - 1) / PLACE_SEG) << 16);   // sums stay below 2^16 each
      uint32_t incl = both;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (lane == 31) s_warp_sum[warp] = incl;
      __syncthreads();
      uint32_t excl = incl - both, total = 0u;
#pragma unroll
      for (int w = 0; w < PLAN_WARPS; ++w) {
        const uint32_t ws = s_warp_sum[w];
        if (w < warp) excl += ws;
        total += ws;
      }
      n_seg = (int)(total >> 16);
      if (!GROUTER_CHECKED(n_seg <= CHUNK / PLACE_SEG + E_tgt, pp.status)) n_seg = 0;
      if (e < E_tgt) {
        const int start = (int)(excl & 0xffffu), first_row = off_e + before_e;
        s_first[e] = start;
        int2* sg = s_seg + (excl >> 16);
        const bool fits = GROUTER_CHECKED(cnt_e >= 0 && start + cnt_e <= CHUNK && (int)(excl >> 16) + (cnt_e + PLACE_SEG - 1) / PLACE_SEG <= CHUNK / PLACE_SEG + E_tgt,
                                          pp.status);
        for (int i = 0; fits && i < cnt_e; i += PLACE_SEG) *sg++ = make_int2((start + i) | (min(PLACE_SEG, cnt_e - i) << 16), first_row + i);
      }
    }
    __syncthreads();

    // ---- first walk: count this thread's slots per expert (a chunk that lies wholly below R needs no per-slot bounds) ----
    const bool whole = chunk0 + CHUNK <= R;
    int bad = 0;
    auto walk1 = [&](auto whole_chunk) {
      constexpr bool WHOLE = decltype(whole_chunk)::value;
#pragma unroll
      for (int v = 0; v < V; ++v) {
        if constexpr (BYTES) ev[v] = check_targets16(ev[v], s0 + 16 * v, R, f, bad);
        else ev[v] = load_targets16<IdxT>(idx, s0 + 16 * v, R, f, bad);
        const uint32_t w[4] = {ev[v].x, ev[v].y, ev[v].z, ev[v].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t before[4];
          const int n = WHOLE ? 4 : n_mine - (16 * v + 4 * q);
          if (n > 0) bump4(mine, w[q], n, before);
        }
      }
    };
    if (whole) walk1(std::true_type{}); else walk1(std::false_type{});
    if (bad) atomicOr(pp.status, STATUS_BAD_INDEX);
    __syncthreads();

    // ---- exclusive scan over the threads, expert row by expert row (a warp keeps several rows in flight, so that their
    // shuffle chains overlap); the result starts at the expert's first staging position, so a counter then holds the
    // staging position of its thread's next slot of that expert ----
    constexpr int ROWS_AT_ONCE = 4;
    for (int e0 = warp * ROWS_AT_ONCE; e0 < E_tgt; e0 += PLAN_WARPS * ROWS_AT_ONCE) {
      uint4 a[ROWS_AT_ONCE];
      uint32_t sum[ROWS_AT_ONCE], incl[ROWS_AT_ONCE];
#pragma unroll
      for (int j = 0; j < ROWS_AT_ONCE; ++j) {
        // lane's words: threads 4*lane .. +3 (low halves) and 128 + 4*lane .. (high halves)
        a[j] = e0 + j < E_tgt ? reinterpret_cast<const uint4*>(s_cnt + (e0 + j) * CNT_ROW_WORDS)[lane] : make_uint4(0u, 0u, 0u, 0u);
        sum[j] = a[j].x + a[j].y + a[j].z + a[j].w;
        incl[j] = sum[j];
      }
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
        for (int j = 0; j < ROWS_AT_ONCE; ++j) {
          const uint32_t n = __shfl_up_sync(0xffffffffu, incl[j], o);
          if (lane >= o) incl[j] += n;
        }
      }
#pragma unroll
      for (int j = 0; j < ROWS_AT_ONCE; ++j) {
        const uint32_t total = __shfl_sync(0xffffffffu, incl[j], 31);
        if (e0 + j < E_tgt) {
          const uint32_t start = (uint32_t)s_first[e0 + j];
          // low halves count from `start`, high halves (threads 128..255) from start + (slots of threads 0..127)
          const uint32_t x0 = incl[j] - sum[j] + (start | ((start + (total & 0xffffu)) << 16));
          const uint32_t x1 = x0 + a[j].x, x2 = x1 + a[j].y, x3 = x2 + a[j].z;
          reinterpret_cast<uint4*>(s_cnt + (e0 + j) * CNT_ROW_WORDS)[lane] = make_uint4(x0, x1, x2, x3);
        }
      }
    }
    __syncthreads();

    // ---- second walk: hand out the positions in slot order ----
    auto walk2 = [&](auto whole_chunk) {
      constexpr bool WHOLE = decltype(whole_chunk)::value;
#pragma unroll
      for (int v = 0; v < V; ++v) {
        const uint32_t w[4] = {ev[v].x, ev[v].y, ev[v].z, ev[v].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int i0 = 16 * v + 4 * q;
          const int n = WHOLE ? 4 : n_mine - i0;
          if (n <= 0) continue;
          uint32_t pos[4];
          bump4(mine, w[q], n, pos);
#pragma unroll
          for (int b = 0; b < 4; ++b)
            if (b < n && GROUTER_CHECKED(pos[b] < (uint32_t)CHUNK, pp.status)) sts_u16(stage_addr + 2u * pos[b], (uint32_t)(tid * IPT + i0 + b));
        }
      }
    };
    if (whole) walk2(std::true_type{}); else walk2(std::false_type{});
    __syncthreads();

    // ---- the next chunk's ids and prefixes set out now and arrive while this chunk is written out ----
    if (c + (int)gridDim.x < nblk) {
      fetch_ids(c + gridDim.x);
      fetch_prefix(c + gridDim.x);
    }

    // ---- every expert's run of this chunk is contiguous in the staging array and in row_to_slot: the inverse
    // permutation goes out piece by piece.  A warp takes pieces warp, warp + 8, ...: every lane fetches one piece's
    // description, the warp then works through them four at a time, the staging loads of all four before any store
    // (shared-memory latency is long while the SM's other block walks its counters).  The row of every slot is parked
    // in shared memory (the counters are done with) ----
    for (int j0 = warp; j0 < n_seg; j0 += 32 * PLAN_WARPS) {
      const int jm = j0 + lane * PLAN_WARPS;
      const int2 my = jm < n_seg ? s_seg[jm] : make_int2(0, 0);        // length 0: nothing to do
      const int n_here = min(32, (n_seg - j0 + PLAN_WARPS - 1) / PLAN_WARPS);
      for (int i = 0; i < n_here; i += 4) {
        int a[4][4], n[4], row0[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int sx = __shfl_sync(0xffffffffu, my.x, (i + u) & 31), sy = __shfl_sync(0xffffffffu, my.y, (i + u) & 31);
          const uint16_t* src = s_stage + (sx & 0xffff);
          n[u] = sx >> 16;
          if (!GROUTER_CHECKED(n[u] <= PLACE_SEG && (sx & 0xffff) + n[u] <= CHUNK && sy >= 0 && sy <= R - n[u], pp.status)) n[u] = 0;
          row0[u] = sy + lane;
#pragma unroll
          for (int q = 0; q < 4; ++q) a[u][q] = lane + 32 * q < n[u] ? (int)src[lane + 32 * q] : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (lane + 32 * q < n[u] && GROUTER_CHECKED(a[u][q] < CHUNK, pp.status)) {
              row_to_slot[row0[u] + 32 * q] = chunk0 + a[u][q];
              s_rows[a[u][q]] = row0[u] + 32 * q;
            }
        }
      }
    }
    __syncthreads();

    // ---- slot_to_row: the chunk's rows, in slot order, as one contiguous copy ----
    {
      const int n_here = min(CHUNK, R - chunk0);
      int32_t* dst = slot_to_row + chunk0;     // chunk0 is a multiple of 4096: 16-byte aligned
      if (n_here == CHUNK) {
#pragma unroll
        for (int i0 = 0; i0 < CHUNK; i0 += 16 * PLAN_THREADS) {       // four 16-byte loads, then four stores
          int4 v[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<const int4*>(s_rows + i0 + 4 * (u * PLAN_THREADS + tid));
#pragma unroll
          for (int u = 0; u < 4; ++u) *reinterpret_cast<int4*>(dst + i0 + 4 * (u * PLAN_THREADS + tid)) = v[u];
        }
      } else {
        for (int i = 4 * tid; i < n_here; i += 4 * PLAN_THREADS) {
          if (i + 4 <= n_here) {
            *reinterpret_cast<int4*>(dst + i) = *reinterpret_cast<const int4*>(s_rows + i);
          } else {
            for (int j = i; j < n_here; ++j) dst[j] = s_rows[j];
          }
        }
      }
    }
    __syncthreads();      // the rows are read before the next chunk's counters take their place
  }
}

// ------------------------------------------------------------------------------------------------------------------
// Ballot form
// ------------------------------------------------------------------------------------------------------------------

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
__global__ void __launch_bounds__(PLAN_THREADS) plan_hist_ballot_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ fold_map,
                                                                        int R, int E_src, int E_tgt, int chunk, int nblk,
                                                                        int32_t* __restrict__ blk_hist, int32_t* __restrict__ status) {
  extern __shared__ int32_t sm[];  // PLAN_WARPS * E_tgt ints
  const int tid = threadIdx.x;
  launch_successor();
  for (int i = tid; i < PLAN_WARPS * E_tgt; i += PLAN_THREADS) sm[i] = 0;
  __syncthreads();
  warp_histogram(idx, fold_map, R, E_src, E_tgt, chunk, sm, status);
  __syncthreads();
  for (int e = tid; e < E_tgt; e += PLAN_THREADS) {
    int tot = 0;
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) tot += sm[w * E_tgt + e];
    blk_hist[(size_t)e * nblk + blockIdx.x] = tot;
  }
}

template <typename IdxT>
__global__ void __launch_bounds__(PLAN_THREADS) plan_permute_ballot_kernel(const IdxT* __restrict__ idx, const int32_t* __restrict__ fold_map,
                                                                           int R, int E_src, int E_tgt, int chunk, int nblk, PaddedPlan pp,
                                                                           const int32_t* __restrict__ offsets, int32_t* __restrict__ row_to_slot,
                                                                           int32_t* __restrict__ slot_to_row) {
  extern __shared__ int32_t sm[];  // PLAN_WARPS * E_tgt ints, then 2 * (E_tgt + 1) for the tile list
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  wait_for_predecessor();
  write_tile_list(pp, E_tgt, sm + PLAN_WARPS * E_tgt, sm + PLAN_WARPS * E_tgt + E_tgt + 1);
  for (int i = tid; i < PLAN_WARPS * E_tgt; i += PLAN_THREADS) sm[i] = 0;
  __syncthreads();
  warp_histogram(idx, fold_map, R, E_src, E_tgt, chunk, sm, pp.status);
  __syncthreads();
  // per-warp histogram -> first row of (block, warp, expert)
  for (int e = tid; e < E_tgt; e += PLAN_THREADS) {
    int base = offsets[e] + pp.blk_prefix[(size_t)e * nblk + blockIdx.x];
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) {
      const int t = sm[w * E_tgt + e];
      sm[w * E_tgt + e] = base;
      base += t;
    }
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
      slot_to_row[s] = row;
      row_to_slot[row] = s;
    }
    if (base + i + 32 >= R) break;
  }
}

// ------------------------------------------------------------------------------------------------------------------
// Phase 1: prefixes over blocks, expert offsets, padded layout, work list of the weight gradients
// ------------------------------------------------------------------------------------------------------------------
static int plan_scan_smem_ints(int E) { return 11 * E + 4 + 2 * (WGRAD_LEN_BUCKETS + 1); }

// Offsets, padded layout, tile prefix and the weight gradients' chunk list from the expert counts in s_cnt (= sm[0..E)).
// Runs in one block of any size (a multiple of 32 threads); sm holds plan_scan_smem_ints(E_tgt) ints.
__device__ __forceinline__ void plan_layout(int32_t* sm, int E_tgt, const PaddedPlan& pp, int32_t* __restrict__ counts,
                                            int32_t* __restrict__ offsets) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nthr = blockDim.x, nwarps = blockDim.x >> 5;
  int32_t* s_cnt = sm;                    // [E]
  int32_t* s_off = sm + E_tgt;            // [E+1]
  int32_t* s_pad = sm + 2 * E_tgt + 1;    // [E+1]
  int32_t* s_pair = sm + 3 * E_tgt + 2;   // [E+1] exclusive prefix of 256-row tiles per expert
  int32_t* s_wch = sm + 4 * E_tgt + 3;    // [E+1] exclusive prefix of weight-gradient row chunks per expert
  int32_t* s_wpos = sm + 5 * E_tgt + 4;   // [2E] list position of each expert's longer / shorter chunks; the chunk-list arrays follow
  __syncthreads();     // s_cnt is complete
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
  for (int e = tid; e <= E_tgt; e += nthr) {
    offsets[e] = s_off[e];
    pp.pad_offsets[e] = s_pad[e];
    pp.pair_prefix[e] = s_pair[e];
    if (e < E_tgt) {
      counts[e] = s_cnt[e];
      pp.row_shift[e] = s_pad[e] - s_off[e];
      pp.pad_begin[e] = s_pad[e] + s_cnt[e];
    }
  }
  if (tid == 0) {
    *pp.n_pair_tiles = s_pair[E_tgt];
    *pp.ticket = 0u;  // ready for the next plan
    *pp.tile_counter = 0u;  // a grouped GEMM that gave up on a timeout may have left it mid-count
    *pp.n_wchunks = s_wch[E_tgt];
  }
  // Row chunks of the weight-gradient GEMMs: an expert without slots keeps one empty chunk (its gradient is zero-filled).
  // An expert's blocks are cut into n chunks of near-equal size: `rem` chunks of base + 1 blocks, then n - rem of base.
  // The list is ordered by chunk length, longest first, in WGRAD_LEN_BUCKETS classes of length (within a class by
  // expert, then by position): tiles of similar cost are neighbours, and the shortest tiles at the end even out the tail.
  {
    const int chunk_blocks = pp.wgrad_chunk_blocks;
    auto len_class = [chunk_blocks](int blocks) { return (blocks * WGRAD_LEN_BUCKETS + chunk_blocks - 1) / chunk_blocks; };   // 0 .. BUCKETS
    int32_t* s_c = s_wpos + 2 * E_tgt;                   // [2E] chunks of the expert's longer / shorter length
    int32_t* s_cl = s_c + 2 * E_tgt;                     // [2E] their length classes
    int32_t* s_len = s_cl + 2 * E_tgt;                   // [BUCKETS + 1] chunks per class
    int32_t* s_start = s_len + WGRAD_LEN_BUCKETS + 1;    // [BUCKETS + 1] first list position of each class
    for (int i = tid; i <= WGRAD_LEN_BUCKETS; i += nthr) s_len[i] = 0;
    __syncthreads();
    for (int e = tid; e < E_tgt; e += nthr) {
      const int blocks = (s_pad[e + 1] - s_pad[e]) / ROW_TILE;
      const int n = s_wch[e + 1] - s_wch[e];
      const int base = blocks / n, rem = blocks - base * n;
      const int cl0 = len_class(base + 1), cl1 = len_class(base);
      s_c[e] = rem;
      s_c[E_tgt + e] = n - rem;
      s_cl[e] = cl0;
      s_cl[E_tgt + e] = cl1;
      if (rem) atomicAdd(&s_len[cl0], rem);
      atomicAdd(&s_len[cl1], n - rem);
    }
    __syncthreads();
    if (warp == 0) {   // classes in descending order: lane p holds class BUCKETS - p; class 0 comes after all of them
      static_assert(WGRAD_LEN_BUCKETS == 32, "one lane per non-zero length class");
      const int v = s_len[WGRAD_LEN_BUCKETS - lane];
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      s_start[WGRAD_LEN_BUCKETS - lane] = incl - v;
      if (lane == 31) s_start[0] = incl;
    }
    __syncthreads();
    // within one class: experts in ascending order, an expert's longer chunks before its shorter ones.  One warp per
    // (non-empty) class walks the experts 32 at a time.
    for (int l = warp; l <= WGRAD_LEN_BUCKETS; l += nwarps) {
      if (s_len[l] == 0) continue;
      int run = s_start[l];
      for (int e0 = 0; e0 < E_tgt; e0 += 32) {
        const int e = e0 + lane;
        int c0 = 0, c1 = 0;    // chunks of the expert's two lengths that fall into class l
        if (e < E_tgt) {
          if (s_cl[e] == l) c0 = s_c[e];
          if (s_cl[E_tgt + e] == l) c1 = s_c[E_tgt + e];
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
  // chunk entries: a thread per expert for the usual few chunks, the whole block for an expert cut into many
  auto write_chunk = [&](int e, int c, int n, int base, int rem) {
    const int i = c < rem ? s_wpos[e] + c : s_wpos[E_tgt + e] + (c - rem);
    if (!GROUTER_CHECKED((unsigned)i < (unsigned)pp.max_wchunks, pp.status)) return;
    pp.wchunk_expert[i] = e | (n > 1 ? WCHUNK_SPLIT : 0);
    pp.wchunk_row0[i] = s_pad[e] + (c * base + min(c, rem)) * ROW_TILE;
    int rows = (base + (c < rem ? 1 : 0)) * ROW_TILE;
    // the contraction runs in steps of 64 rows: when the expert's last block holds at most 64 real rows, its second
    // half is all padding (zeros) and is left out
    const int tail = s_cnt[e] & (ROW_TILE - 1);
    if (c == n - 1 && tail >= 1 && tail <= ROW_TILE / 2) rows -= ROW_TILE / 2;
    pp.wchunk_rows[i] = rows;
  };
  constexpr int MANY_CHUNKS = 16;
  for (int e = tid; e < E_tgt; e += nthr) {
    const int blocks = (s_pad[e + 1] - s_pad[e]) / ROW_TILE;
    const int n = s_wch[e + 1] - s_wch[e];
    if (n > MANY_CHUNKS) continue;
    const int base = blocks / n, rem = blocks - base * n;
    for (int c = 0; c < n; ++c) write_chunk(e, c, n, base, rem);
  }
  for (int e = 0; e < E_tgt; ++e) {
    const int n = s_wch[e + 1] - s_wch[e];
    if (n <= MANY_CHUNKS) continue;
    const int blocks = (s_pad[e + 1] - s_pad[e]) / ROW_TILE;
    const int base = blocks / n, rem = blocks - base * n;
    for (int c = tid; c < n; c += nthr) write_chunk(e, c, n, base, rem);
  }
}


__global__ void __launch_bounds__(PLAN_THREADS) plan_scan_kernel(int E_tgt, int nblk, PaddedPlan pp, int32_t* __restrict__ counts,
                                                                 int32_t* __restrict__ offsets) {
  extern __shared__ int32_t sm[];  // plan_scan_smem_ints(E_tgt) ints
  __shared__ int s_warp_sum[PLAN_WARPS];
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  launch_successor();
  wait_for_predecessor();

  // ---- this block's expert: exclusive prefix over blocks of its per-block counts, in place; the total is counts[e] ----
  {
    const int e = blockIdx.x;
    int32_t* rowp = pp.blk_prefix + (size_t)e * nblk;
    int carry = 0;
    for (int b0 = 0; b0 < nblk; b0 += PLAN_THREADS * 8) {
      const int b = b0 + tid * 8;
      int v[8], sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        v[j] = (b + j < nblk) ? __ldcg(rowp + b + j) : 0;
        sum += v[j];
      }
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (lane == 31) s_warp_sum[warp] = incl;
      __syncthreads();
      int before = 0, total = 0;
#pragma unroll
      for (int w = 0; w < PLAN_WARPS; ++w) {
        const int t = s_warp_sum[w];
        if (w < warp) before += t;
        total += t;
      }
      int run = carry + before + incl - sum;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (b + j < nblk) rowp[b + j] = run;
        run += v[j];
      }
      carry += total;
      __syncthreads();
    }
    if (tid == 0) counts[e] = carry;     // read back by the last block
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned t = atomicAdd(pp.ticket, 1u);
    s_last = (t == (unsigned)(E_tgt - 1));
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  for (int e = tid; e < E_tgt; e += PLAN_THREADS) sm[e] = __ldcg(counts + e);
  plan_layout(sm, E_tgt, pp, counts, offsets);
}

// ------------------------------------------------------------------------------------------------------------------
// Launch
// ------------------------------------------------------------------------------------------------------------------
// Opt-in to more than 48 KB of dynamic shared memory: a per-device, per-kernel setting, raised when a launch needs more
// than the kernel was last given on this device.  (The kernel is a template argument so that every kernel has its own
// record: kernels with equal signatures share a function-pointer type.)
template <auto Kern>
static cudaError_t allow_smem(size_t bytes) {
  static size_t granted[64] = {};
  if (bytes <= 48 * 1024) return cudaSuccess;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (dev >= 0 && dev < 64 && granted[dev] >= bytes) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && dev >= 0 && dev < 64) granted[dev] = bytes;
  return e;
}

// Launch as a programmatic dependent of the previous kernel on the stream: its blocks may be scheduled before that
// kernel has finished; the kernel itself waits (wait_for_predecessor) before it touches the predecessor's results.
template <typename... Params, typename... Args>
static cudaError_t launch_dependent(void (*kern)(Params...), int grid, int block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<Params>(args)...);
}

template <typename IdxT, int V>
static cudaError_t launch_counted(grouter_ctx* ctx, int phase, const IdxT* idx, const int32_t* fold_map, int32_t* offsets,
                                  int32_t* row_to_slot, int32_t* slot_to_row, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  const int E = dm.E_tgt, nblk = ctx->nblk_act;
  if (phase == 0) {
    const size_t sm0 = (size_t)PLAN_WARPS * E * 4 + (fold_map ? (size_t)dm.E_src * 2 : 0);
    cudaError_t e = allow_smem<plan_count_kernel<IdxT, V>>(sm0);
    if (e != cudaSuccess) return e;
    plan_count_kernel<IdxT, V><<<nblk, PLAN_THREADS, sm0, st>>>(idx, fold_map, (int)ctx->R_act, dm.E_src, E, nblk, ctx->pp.blk_prefix, ctx->pp.status);
  } else {
    const size_t sm2 = (size_t)place_smem(dm.E_src, E, 16 * V, fold_map != nullptr).bytes;
    cudaError_t e = allow_smem<plan_place_kernel<IdxT, V>>(sm2);
    if (e != cudaSuccess) return e;
    // two blocks fit an SM (one with more than 128 experts); with many chunks a block takes every grid-th one.  A context
    // that does not know the SM count (the one grouter_plan_noalloc builds: at most 128 chunks) gets a block per chunk.
    const int resident = 2 * ctx->num_sms;
    const int grid = ctx->num_sms > 0 && nblk > 4 * resident ? resident : nblk;   // few chunks per block would only unbalance the blocks
    return launch_dependent(plan_place_kernel<IdxT, V>, grid, PLAN_THREADS, sm2, st, idx, fold_map, (int)ctx->R_act, dm.E_src, E, nblk, ctx->pp,
                            (const int32_t*)offsets, row_to_slot, slot_to_row);
  }
  return cudaGetLastError();
}

template <typename IdxT>
static cudaError_t launch_plan_t(grouter_ctx* ctx, int phase, const IdxT* idx, const int32_t* fold_map, int32_t* counts,
                                 int32_t* offsets, int32_t* row_to_slot, int32_t* slot_to_row, cudaStream_t st) {
  const grouter_dims& dm = ctx->dims;
  const int R = (int)ctx->R_act, E = dm.E_tgt;
  const int chunk = ctx->geom.chunk, nblk = ctx->nblk_act;
  if (phase == 1) {
    const size_t sm1 = sizeof(int32_t) * (size_t)plan_scan_smem_ints(E);
    return launch_dependent(plan_scan_kernel, E, PLAN_THREADS, sm1, st, E, nblk, ctx->pp, counts, offsets);
  }
  switch (ctx->geom.ipt) {
    case 16: return launch_counted<IdxT, 1>(ctx, phase, idx, fold_map, offsets, row_to_slot, slot_to_row, st);
    case 32: return launch_counted<IdxT, 2>(ctx, phase, idx, fold_map, offsets, row_to_slot, slot_to_row, st);
    case 64: return launch_counted<IdxT, 4>(ctx, phase, idx, fold_map, offsets, row_to_slot, slot_to_row, st);
    default: break;
  }
  if (phase == 0) {
    const size_t sm0 = sizeof(int32_t) * (size_t)(PLAN_WARPS * E);
    plan_hist_ballot_kernel<IdxT><<<nblk, PLAN_THREADS, sm0, st>>>(idx, fold_map, R, dm.E_src, E, chunk, nblk, ctx->pp.blk_prefix, ctx->pp.status);
  } else {
    const size_t sm2 = sizeof(int32_t) * (size_t)(PLAN_WARPS * E + 2 * (E + 1));
    return launch_dependent(plan_permute_ballot_kernel<IdxT>, nblk, PLAN_THREADS, sm2, st, idx, fold_map, R, dm.E_src, E, chunk, nblk, ctx->pp,
                            (const int32_t*)offsets, row_to_slot, slot_to_row);
  }
  return cudaGetLastError();
}

cudaError_t launch_plan(grouter_ctx* ctx, int phase, const void* idx, const int32_t* fold_map, int32_t* counts, int32_t* offsets,
                        int32_t* row_to_slot, int32_t* slot_to_row, cudaStream_t st) {
  if (ctx->dims.idx_dtype == GROUTER_IDX_U8)
    return launch_plan_t<uint8_t>(ctx, phase, (const uint8_t*)idx, fold_map, counts, offsets, row_to_slot, slot_to_row, st);
  return launch_plan_t<int32_t>(ctx, phase, (const int32_t*)idx, fold_map, counts, offsets, row_to_slot, slot_to_row, st);
}

}  // namespace grouter

// ------------------------------------------------------------------------
// grouter_plan_noalloc: the same plan kernels, run without a context.
//
// grouter_create owns the plan's scratch (per-block histograms, the ticket of
// the last-block scan, the padded layout and the work lists) in memory it gets
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
constexpr int NOALLOC_MAX_BLOCKS = NOALLOC_MAX_R / PLAN_MIN_CHUNK;                   // plan_geom never uses more (either form)
static_assert(16 * PLAN_THREADS >= PLAN_MIN_CHUNK, "the counted form's smallest chunk must not be shorter than the ballot form's");
// layout of the scratch, in 32-bit words (every part starts on a 256-byte boundary)
constexpr int NA_PAD_OFFSETS = 0;                                     // [E+1]
constexpr int NA_ROW_SHIFT = NA_PAD_OFFSETS + 320;                    // [E]
constexpr int NA_PAD_BEGIN = NA_ROW_SHIFT + 256;                      // [E]
constexpr int NA_PAIR_PREFIX = NA_PAD_BEGIN + 256;                    // [E+1]
constexpr int NA_N_TILES = NA_PAIR_PREFIX + 320;                      // [1]
constexpr int NA_TICKET = NA_N_TILES + 64;                            // [1]
constexpr int NA_STATUS = NA_TICKET + 64;                             // [1] used when the caller passes no status word
constexpr int NA_PAIR_ROW0 = NA_STATUS + 64;                          // [rows/128]
constexpr int NA_PAIR_EXPERT = NA_PAIR_ROW0 + NOALLOC_MAX_ROWS / ROW_TILE;     // [rows/128]
constexpr int NOALLOC_MAX_WCHUNKS = (NOALLOC_MAX_E + NOALLOC_MAX_ROWS / WGRAD_KCHUNK_MAX + 1 + 63) / 64 * 64;
constexpr int NA_WCHUNK_EXPERT = NA_PAIR_EXPERT + NOALLOC_MAX_ROWS / ROW_TILE; // [chunks]
constexpr int NA_WCHUNK_ROW0 = NA_WCHUNK_EXPERT + NOALLOC_MAX_WCHUNKS;         // [chunks]
constexpr int NA_WCHUNK_ROWS = NA_WCHUNK_ROW0 + NOALLOC_MAX_WCHUNKS;           // [chunks]
constexpr int NA_N_WCHUNKS = NA_WCHUNK_ROWS + NOALLOC_MAX_WCHUNKS;             // [1]
constexpr int NA_BLK_PREFIX = NA_N_WCHUNKS + 64;                      // [E * blocks]
constexpr int NA_WORDS = NA_BLK_PREFIX + NOALLOC_MAX_E * NOALLOC_MAX_BLOCKS;
static_assert(NA_PAIR_ROW0 % 64 == 0 && NA_PAIR_EXPERT % 64 == 0 && NA_WCHUNK_EXPERT % 64 == 0 && NA_BLK_PREFIX % 64 == 0,
              "scratch parts must start on 256-byte boundaries");

// About 0.3 MB per GPU.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a
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

  grouter_ctx c{};   // lives on the host stack for the duration of the launches
  c.dims.T = T; c.dims.d = 8; c.dims.ffn = 8; c.dims.E_src = E_src; c.dims.E_tgt = E_tgt; c.dims.k = k;
  c.dims.idx_dtype = idx_dtype; c.dims.gate_dtype = GROUTER_GATE_BF16;
  c.R = (int64_t)T * k;
  c.geom = plan_geom(c.R, E_src, E_tgt);
  c.T_act = T;
  c.R_act = c.R;
  c.nblk_act = c.geom.nblk;
  c.pp.pad_offsets = base + NA_PAD_OFFSETS;
  c.pp.row_shift = base + NA_ROW_SHIFT;
  c.pp.pad_begin = base + NA_PAD_BEGIN;
  c.pp.pair_prefix = base + NA_PAIR_PREFIX;
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
  c.pp.blk_prefix = base + NA_BLK_PREFIX;
  c.pp.max_m_tiles = NOALLOC_MAX_ROWS / ROW_TILE;
  c.pp.max_wchunks = NOALLOC_MAX_WCHUNKS;
  if (c.geom.nblk > NOALLOC_MAX_BLOCKS) return GROUTER_ERR_UNSUPPORTED;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array still holds whatever the previous call left.  The ticket must count from zero and the status
  // word must start clear; every other part is overwritten before it is read.
  if (cudaMemsetAsync(c.pp.ticket, 0, sizeof(unsigned int), st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (cudaMemsetAsync(c.pp.status, 0, sizeof(int32_t), st) != cudaSuccess) return GROUTER_ERR_CUDA;
  for (int phase = 0; phase < PLAN_PHASES; ++phase)
    if (launch_plan(&c, phase, idx, fold_map, counts, offsets, row_to_slot, slot_to_row, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  return GROUTER_OK;
}
