// Stages 2 and 3: Capacity-Aware Token Drop (Eq. 7-10, Algorithm 1) and Expanded Drop
// (Algorithm 2).  Both reduce to: per expert, list the candidate tokens in token order, find
// the C-th largest score with a shared-memory radix select over the float bit patterns
// (non-negative floats order like unsigned integers), and keep everything above it plus the
// first (C - #above) candidates equal to it, in token order.
//
// Batches below the token-parallel threshold run the cluster select of drop_cluster.cu; the
// per-expert kernel k_select of this file, which lists the candidates in scratch memory, serves
// the entry point with built-in scratch and batches no other path takes:
// one small memset (the E candidate counters) and two launches:
//   k_count_candidates  one CTA per 256 tokens: per-expert candidate counts (shared-memory
//                       histogram, then integer atomics: the totals do not depend on order), and
//                       the initial state of the outputs that k_select only touches sparsely
//                       (keep_mask = 0, slot_row = -1 for Expanded Drop).
//   k_select            one CTA per expert: prefix sums of the counts, ordered compaction,
//                       radix select, ordered placement.
#include <mutex>

#include "common.cuh"
#include "select.cuh"

namespace capmoe {

// token-parallel select (drop_parallel.cu): large batches and device-level capacity
size_t drop_parallel_ws_bytes(int64_t N, int E);
int drop_parallel_clear(void* ws_ptr, int64_t N, int E, int S, cudaStream_t st);
int drop_parallel(const float* scores, const float* topk_score, const int32_t* topk_idx, int64_t N, int E, int k,
                  int64_t C_seg, int D, int seg_m, int expanded, const int32_t* token_group, uint64_t* keep_mask,
                  int32_t* cand_out, int32_t* kept, int32_t* expert_offsets, int32_t* slot_row, void* ws_ptr,
                  size_t ws_bytes, cudaStream_t st, bool counters_cleared);

// cluster select (drop_cluster.cu): batches below the token-parallel threshold
bool drop_cluster_takes(int64_t N, int E, bool expanded);
template <bool EXPANDED>
int drop_cluster(const float* score_src, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C, int D,
                 const int32_t* token_group, const int32_t* load, uint64_t* keep_mask, int32_t* cand_out, int32_t* kept,
                 int32_t* expert_offsets, int32_t* slot_row, cudaStream_t st);

namespace {

// Batches the cluster select does not take go to the token-parallel select, whose 64-bit keys
// hold the pair's position t*E + e in 32 bits.
inline bool use_parallel(int64_t N, int E, bool expanded) {
  return !drop_cluster_takes(N, E, expanded) && (unsigned long long)N * (unsigned)E < (1ull << 32);
}

constexpr int CNT_THREADS = 256;
constexpr int TPT = 4;                               // tokens (candidates) per thread per round in k_select
constexpr int CNT_TOKENS = CNT_THREADS;              // tokens per counting CTA
constexpr int SEL_TOKENS = SEL_THREADS * TPT;        // tokens per compaction round
constexpr int E_STRIDE = 256;                        // E <= 256

struct DropWs {
  int32_t* cand;      // [E_STRIDE] candidate counts (when the caller has no array for them)
  uint32_t* key;      // [cap] score bits of each candidate, expert-major, token order inside
  int32_t* tok;       // [cap]
  int32_t* slot;      // [cap]
};

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

inline size_t ws_bytes_needed(int64_t N, int E, int k, int D, int expanded) {
  const int64_t cap = N * (int64_t)(expanded ? k + E / D : k);
  return align256(sizeof(int32_t) * E_STRIDE) + 3 * align256(sizeof(int32_t) * (size_t)cap);
}

inline DropWs carve(void* ws, int64_t N, int E, int k, int D, int expanded) {
  const int64_t cap = N * (int64_t)(expanded ? k + E / D : k);
  char* p = (char*)ws;
  DropWs w;
  w.cand = (int32_t*)p; p += align256(sizeof(int32_t) * E_STRIDE);
  w.key = (uint32_t*)p; p += align256(sizeof(int32_t) * (size_t)cap);
  w.tok = (int32_t*)p;  p += align256(sizeof(int32_t) * (size_t)cap);
  w.slot = (int32_t*)p;
  return w;
}

// Candidates per expert among this CTA's tokens: |{t : e in topk(t)}| (+ |{t : h(t) = e/m, e not
// in topk(t)}| when EXPANDED); plus the initial state of keep_mask / slot_row for these tokens.
template <bool EXPANDED>
__global__ void __launch_bounds__(CNT_THREADS)
k_count_candidates(const int32_t* __restrict__ topk_idx, int64_t N, int E, int k, int D,
                   const int32_t* __restrict__ token_group, int32_t* __restrict__ cand,
                   unsigned long long* __restrict__ keep_mask, int32_t* __restrict__ slot_row) {
  allow_next_kernel();
  wait_for_previous_kernel();
  extern __shared__ int hist[];
  for (int i = threadIdx.x; i < E; i += CNT_THREADS) hist[i] = 0;
  __syncthreads();
  const int64_t t0 = (int64_t)blockIdx.x * CNT_TOKENS;
  const int64_t t1 = min(N, t0 + CNT_TOKENS);
  const int m = EXPANDED ? E / D : 1;
  for (int64_t t = t0 + threadIdx.x; t < t1; t += CNT_THREADS) {
    const int32_t* row = topk_idx + t * k;
    for (int j = 0; j < k; ++j) atomicAdd(&hist[row[j]], 1);
    if (EXPANDED) {
      const int g = home_group(t, N, D, token_group);
      for (int i = 0; i < m; ++i) {
        const int e = g * m + i;
        bool in = false;
        for (int j = 0; j < k; ++j) in |= (row[j] == e);
        if (!in) atomicAdd(&hist[e], 1);
      }
    }
  }
  const int W = (E + 63) >> 6;
  for (int64_t i = t0 * W + threadIdx.x; i < t1 * W; i += CNT_THREADS) keep_mask[i] = 0ull;
  if (EXPANDED) {       // local-expert slots that are already top-k slots are never written again
    const int slots = k + m;
    for (int64_t i = t0 * slots + threadIdx.x; i < t1 * slots; i += CNT_THREADS) slot_row[i] = -1;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < E; i += CNT_THREADS)
    if (hist[i]) atomicAdd(&cand[i], hist[i]);
}

// One CTA per expert.
template <bool EXPANDED>
__global__ void __launch_bounds__(SEL_THREADS)
k_select(const float* __restrict__ score_src,   // topk_score [N,k] (Token Drop) or scores [N,E] (Expanded)
         const int32_t* __restrict__ topk_idx, int64_t N, int E, int k, int64_t C, int D,
         const int32_t* __restrict__ token_group, const int32_t* __restrict__ cand, DropWs ws,
         unsigned long long* __restrict__ keep_mask, int32_t* __restrict__ kept,
         int32_t* __restrict__ expert_offsets, int32_t* __restrict__ slot_row) {
  allow_next_kernel();
  wait_for_previous_kernel();
  __shared__ int hist[RADIX_BINS];
  __shared__ uint32_t scan_sh[SEL_WARPS + 1];
  __shared__ uint32_t found[3];
  const int e = blockIdx.x;
  const int tid = threadIdx.x;
  const int m = EXPANDED ? E / D : 1;
  const int slots = EXPANDED ? k + m : k;
  const int W = (E + 63) >> 6;

  // candidate totals, candidate base (prefix of cand) and row offset (prefix of min(cand, C))
  uint32_t base, off, n, total;
  {
    const uint32_t c = tid < E ? (uint32_t)cand[tid] : 0u;     // E <= 256 <= SEL_THREADS
    const uint32_t kc = c < (uint32_t)C ? c : (uint32_t)C;
    const uint32_t b = block_scan(c, scan_sh, total);
    const uint32_t o = block_scan(kc, scan_sh, total);
    if (tid == e) { found[0] = b; found[1] = o; found[2] = c; }
    __syncthreads();
    base = found[0]; off = found[1]; n = found[2];
    __syncthreads();
  }
  const uint32_t keep_n = n < (uint32_t)C ? n : (uint32_t)C;
  if (tid == 0) {
    kept[e] = (int32_t)keep_n;
    expert_offsets[e] = (int32_t)off;
    if (e == E - 1) expert_offsets[E] = (int32_t)(off + keep_n);
  }
  const bool need_select = n > keep_n;
  for (int i = tid; i < RADIX_BINS; i += SEL_THREADS) hist[i] = 0;
  __syncthreads();

  // pass 1: list this expert's candidates in token order (each thread owns TPT consecutive
  // tokens per round); first-level histogram on the way
  uint32_t* wkey = ws.key + base;
  int32_t* wtok = ws.tok + base;
  int32_t* wslot = ws.slot + base;
  uint32_t running = 0;
  for (int64_t t0 = 0; t0 < N; t0 += SEL_TOKENS) {
    // TPT sub-rounds of SEL_THREADS consecutive tokens each: all loads are issued before the
    // first scan, so their latencies overlap; the scans then run in token order.
    int slot[TPT];
    uint32_t key[TPT];
#pragma unroll
    for (int u = 0; u < TPT; ++u) {
      const int64_t t = t0 + (int64_t)u * SEL_THREADS + tid;
      slot[u] = -1;
      if (t < N) {
        const int32_t* row = topk_idx + t * k;
        for (int j = 0; j < k; ++j)
          if (row[j] == e) slot[u] = j;
        if (EXPANDED)
          if (slot[u] < 0 && home_group(t, N, D, token_group) == e / m) slot[u] = k + (e % m);
      }
    }
#pragma unroll
    for (int u = 0; u < TPT; ++u) {
      const int64_t t = t0 + (int64_t)u * SEL_THREADS + tid;
      key[u] = 0;
      if (slot[u] >= 0)
        key[u] = __float_as_uint(EXPANDED ? score_src[t * E + e] : score_src[t * k + slot[u]]);
    }
#pragma unroll
    for (int u = 0; u < TPT; ++u) {
      if (t0 + (int64_t)u * SEL_THREADS >= N) break;           // uniform across the block
      uint32_t tot;
      const uint32_t p = running + block_scan(slot[u] >= 0 ? 1u : 0u, scan_sh, tot);
      if (slot[u] >= 0) {
        wkey[p] = key[u]; wtok[p] = (int32_t)(t0 + (int64_t)u * SEL_THREADS + tid); wslot[p] = slot[u];
        if (need_select) atomicAdd(&hist[key[u] >> 21], 1);
      }
      running += tot;
    }
  }
  __syncthreads();   // list and histogram complete (block-visible: same CTA wrote them)

  if (!need_select) {
    for (uint32_t i = tid; i < n; i += SEL_THREADS) {
      const int32_t t = wtok[i];
      slot_row[(int64_t)t * slots + wslot[i]] = (int32_t)(off + i);
      atomicOr(&keep_mask[(int64_t)t * W + (e >> 6)], 1ull << (e & 63));
    }
    return;
  }

  // radix select of the C-th largest key: 11, 11, 10 bits (C == 0 keeps nothing: no threshold)
  uint32_t rank = (uint32_t)C;
  uint32_t tau = 0, need = 0;
  if (C > 0) {
    find_bin(hist, RADIX_BINS, rank, scan_sh, found);
    const uint32_t b1 = found[0]; rank = found[1];
    __syncthreads();
    for (int i = tid; i < RADIX_BINS; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    for (uint32_t i = tid; i < n; i += SEL_THREADS) {
      const uint32_t kv = wkey[i];
      if ((kv >> 21) == b1) atomicAdd(&hist[(kv >> 10) & 2047u], 1);
    }
    __syncthreads();
    find_bin(hist, RADIX_BINS, rank, scan_sh, found);
    const uint32_t b2 = found[0]; rank = found[1];
    __syncthreads();
    for (int i = tid; i < RADIX_BINS; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = (b1 << 11) | b2;
    for (uint32_t i = tid; i < n; i += SEL_THREADS) {
      const uint32_t kv = wkey[i];
      if ((kv >> 10) == prefix) atomicAdd(&hist[kv & 1023u], 1);
    }
    __syncthreads();
    find_bin(hist, 1024, rank, scan_sh, found);
    tau = (prefix << 10) | found[0];
    need = found[1];                     // how many candidates equal to tau are kept
    __syncthreads();
  }

  // ordered pass (TPT consecutive candidates per thread): keep key > tau, and the first `need`
  // with key == tau
  uint32_t run_gt = 0, run_eq = 0;
  for (uint32_t i0 = 0; i0 < n; i0 += SEL_TOKENS) {
    uint32_t kv[TPT];
    uint32_t packed = 0;
#pragma unroll
    for (int u = 0; u < TPT; ++u) {
      const uint32_t i = i0 + (uint32_t)tid * TPT + u;
      kv[u] = (i < n && C > 0) ? wkey[i] : 0u;
      if (i < n && C > 0) packed += (kv[u] > tau ? 1u : 0u) | (kv[u] == tau ? 0x10000u : 0u);
    }
    uint32_t tot;
    const uint32_t before = block_scan(packed, scan_sh, tot);   // per round <= 4096 of each: fits 16 bits
    uint32_t gt_before = run_gt + (before & 0xffffu);
    uint32_t eq_before = run_eq + (before >> 16);
#pragma unroll
    for (int u = 0; u < TPT; ++u) {
      const uint32_t i = i0 + (uint32_t)tid * TPT + u;
      if (i < n) {
        const bool gt = C > 0 && kv[u] > tau, eq = C > 0 && kv[u] == tau;
        const bool keep = gt || (eq && eq_before < need);
        const int32_t t = wtok[i];
        int32_t row = -1;
        if (keep) {
          row = (int32_t)(off + gt_before + (eq_before < need ? eq_before : need));
          atomicOr(&keep_mask[(int64_t)t * W + (e >> 6)], 1ull << (e & 63));
        }
        slot_row[(int64_t)t * slots + wslot[i]] = row;
        gt_before += gt ? 1u : 0u;
        eq_before += eq ? 1u : 0u;
      }
    }
    run_gt += tot & 0xffffu;
    run_eq += tot >> 16;
  }
}

template <bool EXPANDED>
int run_drop(const float* score_src, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C, int D,
             const int32_t* token_group, uint64_t* keep_mask, int32_t* cand_out, int32_t* kept,
             int32_t* expert_offsets, int32_t* slot_row, void* ws_ptr, size_t ws_bytes, cudaStream_t st,
             bool counters_cleared = false) {
  cudaError_t err;
  if (N == 0) {
    if ((err = cudaMemsetAsync(kept, 0, sizeof(int32_t) * E, st)) != cudaSuccess) return note_cuda(err);
    if ((err = cudaMemsetAsync(expert_offsets, 0, sizeof(int32_t) * (E + 1), st)) != cudaSuccess) return note_cuda(err);
    if (cand_out && (err = cudaMemsetAsync(cand_out, 0, sizeof(int32_t) * E, st)) != cudaSuccess) return note_cuda(err);
    return CAPMOE_OK;
  }
  if (ws_bytes < ws_bytes_needed(N, E, k, D, EXPANDED ? 1 : 0)) return CAPMOE_EWORKSPACE;
  DropWs ws = carve(ws_ptr, N, E, k, D, EXPANDED ? 1 : 0);
  int32_t* cand = cand_out ? cand_out : ws.cand;
  if (!counters_cleared && (err = cudaMemsetAsync(cand, 0, sizeof(int32_t) * E, st)) != cudaSuccess)
    return note_cuda(err);
  int rc = note_cuda(launch_chained(k_count_candidates<EXPANDED>, (unsigned)ceil_div(N, CNT_TOKENS), CNT_THREADS,
                                    sizeof(int) * E, st, topk_idx, N, E, k, D, token_group, cand,
                                    (unsigned long long*)keep_mask, slot_row));
  count_launch(1);
  if (rc != CAPMOE_OK) return rc;
  rc = note_cuda(launch_chained(k_select<EXPANDED>, (unsigned)E, SEL_THREADS, 0, st, score_src, topk_idx, N, E, k, C, D,
                                token_group, (const int32_t*)cand, ws, (unsigned long long*)keep_mask, kept,
                                expert_offsets, slot_row));
  count_launch(1);
  return rc;
}

int empty_batch(int E, int32_t* cand_out, int32_t* kept, int32_t* expert_offsets, cudaStream_t st) {
  cudaError_t err;
  if ((err = cudaMemsetAsync(kept, 0, sizeof(int32_t) * E, st)) != cudaSuccess) return note_cuda(err);
  if ((err = cudaMemsetAsync(expert_offsets, 0, sizeof(int32_t) * (E + 1), st)) != cudaSuccess) return note_cuda(err);
  if (cand_out && (err = cudaMemsetAsync(cand_out, 0, sizeof(int32_t) * E, st)) != cudaSuccess) return note_cuda(err);
  return CAPMOE_OK;
}

int validate(int64_t N, int E, int k, int64_t C) {
  if (N < 0 || E < 1 || k < 1 || k > E || C < 0 || C > N) return CAPMOE_EINVAL;
  if (E > 256 || k > 32) return CAPMOE_EUNSUPPORTED;
  return CAPMOE_OK;
}

}  // namespace
}  // namespace capmoe

using namespace capmoe;

extern "C" int capmoe_drop_workspace_bytes(int64_t N, int E, int k, int D, int expanded, size_t* bytes) {
  if (!bytes || N < 0 || E < 1 || k < 1 || k > E) return CAPMOE_EINVAL;
  if (expanded && (D < 1 || E % D != 0)) return CAPMOE_EINVAL;
  if (N * (int64_t)(expanded ? k + E / D : k) >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  const size_t a = ws_bytes_needed(N, E, k, expanded ? D : 1, expanded);
  const size_t b = drop_parallel_ws_bytes(N, E);
  *bytes = a > b ? a : b;
  return CAPMOE_OK;
}

size_t capmoe::drop_ws_required(int mode, int64_t N, int E, int k, int D) {
  if (N <= 0) return 0;
  const bool device_level = mode >= 3, expanded = mode == 2 || mode == 4;
  const bool parallel = device_level || use_parallel(N, E, expanded);
  return parallel ? drop_parallel_ws_bytes(N, E) : ws_bytes_needed(N, E, k, D, expanded ? 1 : 0);
}

int capmoe::drop_clear_counters(int mode, int64_t N, int E, int k, int D, int32_t* cand, void* ws, size_t ws_bytes,
                                cudaStream_t st) {
  if (N <= 0 || !ws) return CAPMOE_OK;                        // the stage handles (and checks) these itself
  const bool device_level = mode >= 3, expanded = mode == 2 || mode == 4;
  const bool parallel = device_level || use_parallel(N, E, expanded);
  if (parallel) {
    if (ws_bytes < drop_parallel_ws_bytes(N, E)) return CAPMOE_EWORKSPACE;
    return drop_parallel_clear(ws, N, E, device_level ? D : E, st);
  }
  if (ws_bytes < ws_bytes_needed(N, E, k, D, expanded ? 1 : 0)) return CAPMOE_EWORKSPACE;
  if (drop_cluster_takes(N, E, expanded)) return CAPMOE_OK;  // the cluster select starts from nothing
  int32_t* c = (expanded && cand) ? cand : carve(ws, N, E, k, D, expanded ? 1 : 0).cand;
  return note_cuda(cudaMemsetAsync(c, 0, sizeof(int32_t) * E, st));
}

int capmoe::token_drop_impl(const float* topk_score, const int32_t* topk_idx, int64_t N, int E, int k,
                                 int64_t C, uint64_t* keep_mask, int32_t* kept, int32_t* expert_offsets,
                                 int32_t* slot_row, void* ws, size_t ws_bytes, void* stream, bool counters_cleared,
                                 bool* defer_mask, const int32_t* load) {
  const bool may_defer = defer_mask && *defer_mask;
  if (defer_mask) *defer_mask = false;
  int rc = validate(N, E, k, C);
  if (rc != CAPMOE_OK) return rc;
  if (!kept || !expert_offsets) return CAPMOE_EINVAL;
  if (N > 0 && (!topk_score || !topk_idx || !keep_mask || !slot_row || !ws)) return CAPMOE_EINVAL;
  if (N * (int64_t)k >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return empty_batch(E, nullptr, kept, expert_offsets, as_stream(stream));
  if (use_parallel(N, E, false))
    return drop_parallel(nullptr, topk_score, topk_idx, N, E, k, C, 1, 1, 0, nullptr, keep_mask, nullptr, kept,
                         expert_offsets, slot_row, ws, ws_bytes, as_stream(stream), counters_cleared);
  if (ws_bytes < ws_bytes_needed(N, E, k, 1, 0)) return CAPMOE_EWORKSPACE;
  if (drop_cluster_takes(N, E, false)) {
    if (may_defer) *defer_mask = true;
    return drop_cluster<false>(topk_score, topk_idx, N, E, k, C, 1, nullptr, load, may_defer ? nullptr : keep_mask, nullptr,
                               kept, expert_offsets, slot_row, as_stream(stream));
  }
  return run_drop<false>(topk_score, topk_idx, N, E, k, C, 1, nullptr, keep_mask, nullptr, kept,
                         expert_offsets, slot_row, ws, ws_bytes, as_stream(stream), counters_cleared);
}

int capmoe::expanded_drop_impl(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k,
                                    int64_t C, int D, const int32_t* token_group, uint64_t* keep_mask,
                                    int32_t* cand, int32_t* kept, int32_t* expert_offsets, int32_t* slot_row,
                                    void* ws, size_t ws_bytes, void* stream, bool counters_cleared, bool* defer_mask,
                                    const int32_t* load) {
  const bool may_defer = defer_mask && *defer_mask;
  if (defer_mask) *defer_mask = false;
  int rc = validate(N, E, k, C);
  if (rc != CAPMOE_OK) return rc;
  if (D < 1 || E % D != 0) return CAPMOE_EINVAL;
  if (!kept || !expert_offsets || !cand) return CAPMOE_EINVAL;
  if (N > 0 && (!scores || !topk_idx || !keep_mask || !slot_row || !ws)) return CAPMOE_EINVAL;
  if (N * (int64_t)(k + E / D) >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return empty_batch(E, cand, kept, expert_offsets, as_stream(stream));
  if (use_parallel(N, E, true))
    return drop_parallel(scores, nullptr, topk_idx, N, E, k, C, D, 1, 1, token_group, keep_mask, cand, kept,
                         expert_offsets, slot_row, ws, ws_bytes, as_stream(stream), counters_cleared);
  if (ws_bytes < ws_bytes_needed(N, E, k, D, 1)) return CAPMOE_EWORKSPACE;
  if (drop_cluster_takes(N, E, true)) {
    if (may_defer) *defer_mask = true;
    return drop_cluster<true>(scores, topk_idx, N, E, k, C, D, token_group, load, may_defer ? nullptr : keep_mask, cand, kept,
                              expert_offsets, slot_row, as_stream(stream));
  }
  return run_drop<true>(scores, topk_idx, N, E, k, C, D, token_group, keep_mask, cand, kept, expert_offsets,
                        slot_row, ws, ws_bytes, as_stream(stream), counters_cleared);
}

int capmoe::device_drop_impl(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k,
                                  int64_t C_dev, int D, int expanded, const int32_t* token_group,
                                  uint64_t* keep_mask, int32_t* cand, int32_t* kept, int32_t* expert_offsets,
                                  int32_t* slot_row, void* ws, size_t ws_bytes, void* stream, bool counters_cleared) {
  if (N < 0 || E < 1 || k < 1 || k > E || D < 1 || E % D != 0 || C_dev < 0) return CAPMOE_EINVAL;
  if (C_dev > N * (int64_t)(E / D)) return CAPMOE_EINVAL;
  if (E > 256 || k > 32) return CAPMOE_EUNSUPPORTED;
  if (!kept || !expert_offsets || !cand) return CAPMOE_EINVAL;
  if (N > 0 && (!scores || !topk_idx || !keep_mask || !slot_row || !ws)) return CAPMOE_EINVAL;
  if (N * (int64_t)(k + E / D) >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  cudaStream_t st = as_stream(stream);
  if (N == 0) {
    cudaError_t err;
    if ((err = cudaMemsetAsync(kept, 0, sizeof(int32_t) * E, st)) != cudaSuccess) return note_cuda(err);
    if ((err = cudaMemsetAsync(expert_offsets, 0, sizeof(int32_t) * (E + 1), st)) != cudaSuccess) return note_cuda(err);
    if ((err = cudaMemsetAsync(cand, 0, sizeof(int32_t) * E, st)) != cudaSuccess) return note_cuda(err);
    return CAPMOE_OK;
  }
  return drop_parallel(scores, nullptr, topk_idx, N, E, k, C_dev, D, E / D, expanded ? 1 : 0, token_group, keep_mask,
                       cand, kept, expert_offsets, slot_row, ws, ws_bytes, st, counters_cleared);
}

// ---------------------------------------------------------------------------------------------
// Token Drop for callers that cannot provide scratch memory (see capmoe_token_drop_static in the
// header).  The scratch lives in a fixed array in device memory that belongs to the library.
namespace capmoe {
namespace {

constexpr int64_t STATIC_MAX_PAIRS = CAPMOE_STATIC_DROP_MAX_PAIRS;
// same layout as carve(): the candidate counters, then three int32 lists of STATIC_MAX_PAIRS entries
constexpr size_t STATIC_WS_BYTES = sizeof(int32_t) * E_STRIDE + 3 * sizeof(int32_t) * (size_t)STATIC_MAX_PAIRS;
static_assert((sizeof(int32_t) * (size_t)STATIC_MAX_PAIRS) % 256 == 0, "lists must stay 256-byte aligned");

static __device__ __align__(256) unsigned char g_static_drop_ws[STATIC_WS_BYTES];

constexpr int MAX_DEVICES = 64;
static void* g_static_ws_addr[MAX_DEVICES];      // device address of the array, per device ordinal
static bool g_static_ws_ready[MAX_DEVICES];
static std::mutex g_static_ws_mutex;

// In host code `g_static_drop_ws` is only a handle; the address a kernel can use has to be asked
// for, once per device, while that device is current.
int static_ws_for_current_device(void** out) {
  int dev = -1;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return note_cuda(err);
  if (dev < 0 || dev >= MAX_DEVICES) return CAPMOE_EUNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_ws_mutex);
  if (!g_static_ws_ready[dev]) {
    void* p = nullptr;
    err = cudaGetSymbolAddress(&p, g_static_drop_ws);
    if (err != cudaSuccess) return note_cuda(err);
    if (!p) return note_cuda(cudaErrorInvalidSymbol);
    g_static_ws_addr[dev] = p;
    g_static_ws_ready[dev] = true;
  }
  *out = g_static_ws_addr[dev];
  return CAPMOE_OK;
}

}  // namespace
}  // namespace capmoe

extern "C" int capmoe_token_drop_static(const float* topk_score, const int32_t* topk_idx, int64_t N, int E,
                                        int k, int64_t C, uint64_t* keep_mask, int32_t* kept,
                                        int32_t* expert_offsets, int32_t* slot_row, void* stream) {
  int rc = validate(N, E, k, C);
  if (rc != CAPMOE_OK) return rc;
  if (!kept || !expert_offsets) return CAPMOE_EINVAL;
  if (N > 0 && (!topk_score || !topk_idx || !keep_mask || !slot_row)) return CAPMOE_EINVAL;
  if (N * (int64_t)k > STATIC_MAX_PAIRS) return CAPMOE_EWORKSPACE;   // beyond the built-in scratch
  void* ws = nullptr;
  rc = static_ws_for_current_device(&ws);
  if (rc != CAPMOE_OK) return rc;
  // run_drop zeroes the candidate counters itself (the only part that has to start at zero); the
  // three lists are fully rewritten before they are read, so nothing else of the previous call's
  // contents matters.
  return run_drop<false>(topk_score, topk_idx, N, E, k, C, 1, nullptr, keep_mask, nullptr, kept,
                         expert_offsets, slot_row, ws, STATIC_WS_BYTES, as_stream(stream));
}

// ---------------------------------------------------------------------------------------------
// Drop metrics: 32-bit keys for the select (the paper's "Score", "Order", "Reverse Order",
// "Random").  The drop entry points compare their score input by bit pattern, so a key array
// passed in place of the scores selects by that metric.
namespace capmoe {
namespace {

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void __launch_bounds__(256)
k_drop_keys(int metric, unsigned long long seed, const float* __restrict__ scores, const int32_t* __restrict__ idx,
            int64_t total, int cols, int E, uint32_t* __restrict__ keys) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= total) return;
  const int64_t t = i / cols;
  const int c = (int)(i - t * cols);
  const int e = idx ? idx[i] : c;
  uint32_t key;
  if (metric == CAPMOE_METRIC_SCORE) key = __float_as_uint(scores[i]);
  else if (metric == CAPMOE_METRIC_ORDER) key = 0x3f800000u;              // all equal: earlier tokens first
  else if (metric == CAPMOE_METRIC_REVERSE_ORDER) key = (uint32_t)t;      // later tokens first
  else
    key = (uint32_t)(mix64(seed + 0x9E3779B97F4A7C15ull *
                                      ((unsigned long long)t * (unsigned)E + (unsigned)e + 1ull)) >> 32);
  keys[i] = key;
}

}  // namespace
}  // namespace capmoe

extern "C" int capmoe_drop_keys(int metric, uint64_t seed, const float* scores, const int32_t* idx, int64_t N,
                                int cols, int E, uint32_t* keys, void* stream) {
  if (metric < CAPMOE_METRIC_SCORE || metric > CAPMOE_METRIC_RANDOM) return CAPMOE_EINVAL;
  if (N < 0 || cols < 1 || E < 1 || (!idx && cols != E)) return CAPMOE_EINVAL;
  if (N == 0) return CAPMOE_OK;
  if (!keys || (metric == CAPMOE_METRIC_SCORE && !scores)) return CAPMOE_EINVAL;
  const int64_t total = N * cols;
  if (total >= ((int64_t)1 << 38)) return CAPMOE_EUNSUPPORTED;
  k_drop_keys<<<(unsigned)ceil_div(total, 256), 256, 0, as_stream(stream)>>>(
      metric, (unsigned long long)seed, scores, idx, total, cols, E, keys);
  return check_launch();
}

extern "C" int capmoe_token_drop(const float* topk_score, const int32_t* topk_idx, int64_t N, int E, int k,
                                 int64_t C, uint64_t* keep_mask, int32_t* kept, int32_t* expert_offsets,
                                 int32_t* slot_row, void* ws, size_t ws_bytes, void* stream) {
  return token_drop_impl(topk_score, topk_idx, N, E, k, C, keep_mask, kept, expert_offsets, slot_row, ws, ws_bytes,
                         stream, false, nullptr, nullptr);
}

extern "C" int capmoe_expanded_drop(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k,
                                    int64_t C, int D, const int32_t* token_group, uint64_t* keep_mask,
                                    int32_t* cand, int32_t* kept, int32_t* expert_offsets, int32_t* slot_row,
                                    void* ws, size_t ws_bytes, void* stream) {
  return expanded_drop_impl(scores, topk_idx, N, E, k, C, D, token_group, keep_mask, cand, kept, expert_offsets,
                            slot_row, ws, ws_bytes, stream, false, nullptr, nullptr);
}

extern "C" int capmoe_device_drop(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k,
                                  int64_t C_dev, int D, int expanded, const int32_t* token_group,
                                  uint64_t* keep_mask, int32_t* cand, int32_t* kept, int32_t* expert_offsets,
                                  int32_t* slot_row, void* ws, size_t ws_bytes, void* stream) {
  return device_drop_impl(scores, topk_idx, N, E, k, C_dev, D, expanded, token_group, keep_mask, cand, kept,
                          expert_offsets, slot_row, ws, ws_bytes, stream, false);
}
