// Routing statistics over a cached routing table: the inputs of the method's offline stages.
//
//   loads L_i and MaxVio_Global = (max L - mean L) / mean L            appendix "Maximal Violation"
//   co-activation matrix P = sum_t a_t a_t^T (a_t: the token's 0/1 vector)   section "Expert Folding"
//   routing affinity vectors phi(X)_i = (1/|X|) #{t in X : e_i kept}   section "Decoupling Communication Optimization"
//   |T_s(n)| and best_node of Algorithm 1 (sample placement)           appendix "Efficiency Experiment Detail"
// plus, on the host, the greedy affinity folding that turns P into the fold map (section "Expert Folding").
//
// A sample (a run of seq_len tokens) is split over several blocks.  Counts are integers built with shared-memory atomics
// and merged with global integer atomics, so every result is exact and independent of scheduling; a second small kernel
// turns the per-sample counts into phi, picks each sample's node and computes MaxVio.
#include <vector>

#include "common.cuh"

namespace grouter {

constexpr int STATS_THREADS = 256;
constexpr int STATS_MAX_K = 32;
constexpr int STATS_MAX_NODES = 64;
constexpr int STATS_SMEM_P_MAX_E = 128;     // P of the block lives in shared memory up to this many experts (64 KB)

template <typename IdxT>
__global__ void __launch_bounds__(STATS_THREADS) routing_stats_kernel(const IdxT* __restrict__ idx, int k, int E, int seq_len,
                                                                      const int32_t* __restrict__ node_of_expert, int n_nodes,
                                                                      int32_t* __restrict__ loads, int32_t* __restrict__ coact,
                                                                      int32_t* __restrict__ phi_counts, int32_t* __restrict__ local_tokens,
                                                                      int32_t* __restrict__ status, int p_in_smem, int blocks_per_sample) {
  extern __shared__ int32_t sm[];
  int32_t* s_hist = sm;                      // [E]
  int32_t* s_node = sm + E;                  // [STATS_MAX_NODES]
  int32_t* s_P = sm + E + STATS_MAX_NODES;   // [E*E] when p_in_smem
  const int tid = threadIdx.x;
  const int s = blockIdx.x / blocks_per_sample, part = blockIdx.x - s * blocks_per_sample;
  const int n_sm = E + STATS_MAX_NODES + (p_in_smem ? E * E : 0);
  for (int i = tid; i < n_sm; i += STATS_THREADS) sm[i] = 0;
  __syncthreads();
  for (int lt = part * STATS_THREADS + tid; lt < seq_len; lt += blocks_per_sample * STATS_THREADS) {
    const size_t t = (size_t)s * seq_len + lt;
    int ids[STATS_MAX_K];
    int n = 0;
    for (int j = 0; j < k; ++j) {              // the token's distinct, in-range ids
      const int e = (int)idx[t * k + j];
      if ((unsigned)e >= (unsigned)E) {
        atomicOr(status, STATUS_BAD_INDEX);
        continue;
      }
      bool seen = false;
      for (int q = 0; q < n; ++q) seen |= ids[q] == e;
      if (!seen) ids[n++] = e;
    }
    unsigned long long nodes = 0ull;
    for (int a = 0; a < n; ++a) {
      atomicAdd(&s_hist[ids[a]], 1);
      if (node_of_expert) {
        const int nd = __ldg(node_of_expert + ids[a]);
        if ((unsigned)nd < (unsigned)n_nodes) nodes |= 1ull << nd;
        else atomicOr(status, STATUS_BAD_INDEX);
      }
      for (int b = 0; b < n; ++b) {
        if (p_in_smem) atomicAdd(&s_P[ids[a] * E + ids[b]], 1);
        else atomicAdd(&coact[(size_t)ids[a] * E + ids[b]], 1);
      }
    }
    while (nodes) {                            // one count per node that holds at least one of the token's experts
      const int nd = __ffsll((long long)nodes) - 1;
      nodes &= nodes - 1;
      atomicAdd(&s_node[nd], 1);
    }
  }
  __syncthreads();
  for (int e = tid; e < E; e += STATS_THREADS) {
    const int c = s_hist[e];
    if (c) {
      atomicAdd(&phi_counts[(size_t)s * E + e], c);
      atomicAdd(&loads[e], c);
    }
  }
  if (p_in_smem)
    for (int i = tid; i < E * E; i += STATS_THREADS)
      if (s_P[i]) atomicAdd(&coact[i], s_P[i]);
  if (local_tokens)
    for (int n = tid; n < n_nodes; n += STATS_THREADS)
      if (s_node[n]) atomicAdd(&local_tokens[(size_t)s * n_nodes + n], s_node[n]);
}

// Per sample: counts -> phi (in place: the buffer holds int32 counts on entry, float quotients on exit) and the node of
// Algorithm 1 (strictly more local tokens wins, so the first maximum stays).
__global__ void __launch_bounds__(STATS_THREADS) stats_finish_kernel(float* __restrict__ phi, int E, int seq_len, int S,
                                                                     const int32_t* __restrict__ local_tokens, int n_nodes,
                                                                     int32_t* __restrict__ best_node) {
  const size_t n = (size_t)S * E;
  for (size_t i = (size_t)blockIdx.x * STATS_THREADS + threadIdx.x; i < n; i += (size_t)gridDim.x * STATS_THREADS) {
    const int c = reinterpret_cast<const int32_t*>(phi)[i];
    phi[i] = (float)c / (float)seq_len;
  }
  if (best_node)
    for (int s = blockIdx.x * STATS_THREADS + threadIdx.x; s < S; s += gridDim.x * STATS_THREADS) {
      int best = 0, most = -1;
      for (int nd = 0; nd < n_nodes; ++nd) {
        const int c = local_tokens[(size_t)s * n_nodes + nd];
        if (c > most) {
          most = c;
          best = nd;
        }
      }
      best_node[s] = best;
    }
}

__global__ void __launch_bounds__(STATS_THREADS) max_vio_kernel(const int32_t* __restrict__ loads, int E, float* __restrict__ max_vio) {
  __shared__ long long s_sum[STATS_THREADS];
  __shared__ int s_max[STATS_THREADS];
  long long sum = 0;
  int mx = 0;
  for (int e = threadIdx.x; e < E; e += STATS_THREADS) {
    sum += loads[e];
    mx = max(mx, loads[e]);
  }
  s_sum[threadIdx.x] = sum;
  s_max[threadIdx.x] = mx;
  __syncthreads();
  for (int o = STATS_THREADS / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      s_sum[threadIdx.x] += s_sum[threadIdx.x + o];
      s_max[threadIdx.x] = max(s_max[threadIdx.x], s_max[threadIdx.x + o]);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double mean = (double)s_sum[0] / (double)E;
    *max_vio = mean > 0.0 ? (float)(((double)s_max[0] - mean) / mean) : 0.f;
  }
}

}  // namespace grouter

extern "C" {

int grouter_routing_stats(const void* idx, int32_t idx_dtype, int32_t T, int32_t k, int32_t E, int32_t seq_len,
                          const int32_t* node_of_expert, int32_t n_nodes, int32_t* loads, int32_t* coact, float* phi, float* max_vio,
                          int32_t* local_tokens, int32_t* best_node, int32_t* status, void* stream) {
  using namespace grouter;
  if (!idx || !loads || !coact || !phi || !max_vio || !status) return GROUTER_ERR_INVALID_ARG;
  if (T < 1 || k < 1 || E < 1 || seq_len < 1 || T % seq_len) return GROUTER_ERR_INVALID_ARG;
  if (idx_dtype != GROUTER_IDX_U8 && idx_dtype != GROUTER_IDX_I32) return GROUTER_ERR_INVALID_ARG;
  if ((local_tokens || best_node) && (!node_of_expert || n_nodes < 1)) return GROUTER_ERR_INVALID_ARG;
  if (best_node && !local_tokens) return GROUTER_ERR_INVALID_ARG;   // the node choice is read off the local-token counts
  if (k > STATS_MAX_K || E > 1024 || (node_of_expert && n_nodes > STATS_MAX_NODES)) return GROUTER_ERR_UNSUPPORTED;
  if (idx_dtype == GROUTER_IDX_U8 && E > 256) return GROUTER_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(loads, 0, (size_t)E * 4, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (cudaMemsetAsync(coact, 0, (size_t)E * E * 4, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  const int p_in_smem = E <= STATS_SMEM_P_MAX_E;
  const size_t smem = sizeof(int32_t) * ((size_t)E + STATS_MAX_NODES + (p_in_smem ? (size_t)E * E : 0));
  const int S = T / seq_len;
  if (cudaMemsetAsync(phi, 0, (size_t)S * E * 4, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  if (local_tokens && cudaMemsetAsync(local_tokens, 0, (size_t)S * n_nodes * 4, st) != cudaSuccess) return GROUTER_ERR_CUDA;
  int bps = (seq_len + STATS_THREADS - 1) / STATS_THREADS;           // blocks per sample
  if (bps > 32) bps = 32;
  int32_t* phi_counts = reinterpret_cast<int32_t*>(phi);
  cudaError_t err;
  if (idx_dtype == GROUTER_IDX_U8) {
    auto kern = routing_stats_kernel<uint8_t>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return GROUTER_ERR_CUDA;
    kern<<<S * bps, STATS_THREADS, smem, st>>>(static_cast<const uint8_t*>(idx), k, E, seq_len, node_of_expert, n_nodes, loads, coact,
                                               phi_counts, local_tokens, status, p_in_smem, bps);
    err = cudaGetLastError();
  } else {
    auto kern = routing_stats_kernel<int32_t>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return GROUTER_ERR_CUDA;
    kern<<<S * bps, STATS_THREADS, smem, st>>>(static_cast<const int32_t*>(idx), k, E, seq_len, node_of_expert, n_nodes, loads, coact,
                                               phi_counts, local_tokens, status, p_in_smem, bps);
    err = cudaGetLastError();
  }
  if (err != cudaSuccess) return GROUTER_ERR_CUDA;
  int fin = (int)(((size_t)S * E + STATS_THREADS - 1) / STATS_THREADS);
  if (fin > 1024) fin = 1024;
  stats_finish_kernel<<<fin, STATS_THREADS, 0, st>>>(phi, E, seq_len, S, local_tokens, n_nodes, best_node);
  if (cudaGetLastError() != cudaSuccess) return GROUTER_ERR_CUDA;
  max_vio_kernel<<<1, STATS_THREADS, 0, st>>>(loads, E, max_vio);
  return cudaGetLastError() == cudaSuccess ? GROUTER_OK : GROUTER_ERR_CUDA;
}

int grouter_fold_greedy_host(const int32_t* coact_host, int32_t E_src, int32_t E_tgt, int32_t* fold_map_host) {
  if (!coact_host || !fold_map_host || E_src < 1 || E_tgt < 1) return GROUTER_ERR_INVALID_ARG;
  if (E_tgt > E_src) return GROUTER_ERR_INVALID_ARG;
  const int g_avg = E_src / E_tgt, n_extra = E_src % E_tgt;
  std::vector<char> assigned((size_t)E_src, 0);
  std::vector<long long> aff((size_t)E_src);        // summed affinity of every expert to the group being grown
  int next_seed = 0;
  for (int g = 0; g < E_tgt; ++g) {
    const int size = g_avg + (g < n_extra ? 1 : 0);
    while (assigned[next_seed]) ++next_seed;        // the lowest-numbered unassigned expert opens the group
    int last = next_seed;
    assigned[last] = 1;
    fold_map_host[last] = g;
    for (int j = 0; j < E_src; ++j) aff[j] = 0;
    for (int n = 1; n < size; ++n) {
      int best = -1;
      for (int j = 0; j < E_src; ++j) {
        if (assigned[j]) continue;
        aff[j] += coact_host[(size_t)last * E_src + j];
        if (best < 0 || aff[j] > aff[best]) best = j;   // equal sums: the lower id stays
      }
      last = best;
      assigned[last] = 1;
      fold_map_host[last] = g;
    }
  }
  return GROUTER_OK;
}

}  // extern "C"
