// Per-expert capacity select for batches below the token-parallel threshold (stages 2 and 3:
// Token Drop, Eq. 7-10 / Algorithm 1; Expanded Drop, Algorithm 2), built for latency: one launch
// that counts, selects and places, no scratch memory, no memset, no pass over global memory after
// the first.
//
// An expert is served by a thread-block cluster of R CTAs (R = 1, 2, 4 or 8, chosen so that the
// E*R CTAs about fill the GPU).  CTA r of the cluster owns the r-th contiguous block of tokens, warp
// w of it 32*TPT consecutive ones, and lane l of the warp tokens l, l+32, ... of those: for a fixed u
// the lanes of a warp hold 32 consecutive tokens, so their loads and stores share cache lines, and
// token order is (rank, warp, u, lane) order.  A thread
// reads the top-k lists of its tokens once and keeps, for each token that is a candidate of the
// expert, the candidate's slot and key (the score's bit pattern: non-negative floats order like
// unsigned integers) in registers for the rest of the kernel:
//   1. Counts: the top-k lists also give the candidates of EVERY expert among this CTA's tokens
//      (shared-memory histogram); the CTAs of the cluster read each other's histograms through
//      distributed shared memory, so every cluster knows cand[e'] for all experts, hence
//      kept[e'] = min(cand[e'], C) and the row offset of its own segment, without waiting for any
//      other cluster.  A caller that has the router's load histogram passes it in and the count of
//      the top-k part is skipped.
//   2. The three radix levels (11, 11, 10 bits) of the C-th largest key: every CTA adds its
//      candidates' digits to a histogram in the cluster leader's shared memory (one atomic per
//      distinct digit per warp), the leader finds the bin and tells the others (two cluster barriers
//      per level).  A level whose bin is kept as a whole ends the search, which for tie-free scores
//      usually happens after the second.  Skipped when the expert is not over capacity.
//   3. Ranks: candidates above the threshold, and the first `need` equal to it, are kept; their
//      rows follow from one block scan in token order plus the totals of the lower-ranked CTAs
//      (exchanged through every CTA's shared memory, one more cluster barrier).
// Every slot_row entry is written exactly once, by the cluster of the slot's expert; positions never
// come from atomics.  The keep mask is derived from slot_row afterwards (k_mask_from_rows, or the
// permute kernel of a whole-layer forward), so nothing has to start at zero.
#include <cooperative_groups.h>

#include "common.cuh"
#include "select.cuh"

namespace cg = cooperative_groups;

namespace capmoe {
namespace {

constexpr int MAX_R = 8;             // portable cluster size limit
constexpr int MAX_E = 256;

// Exclusive prefix sum over the block with one barrier: warp scans, the 32 warp totals through
// shared memory, and every warp scans those itself.  wt: 32 words that nobody else touches
// until the next barrier after the call.  total = sum over the block.
__device__ __forceinline__ uint32_t block_scan1(uint32_t v, uint32_t* wt, uint32_t& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) wt[wid] = incl;
  __syncthreads();
  const uint32_t w = wt[lane];                          // SEL_WARPS == 32
  uint32_t wi = w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
    if (lane >= o) wi += n;
  }
  total = __shfl_sync(0xffffffffu, wi, 31);
  const uint32_t warp_before = __shfl_sync(0xffffffffu, wi - w, wid);
  return warp_before + incl - v;
}

// The same for TPT values per thread whose order is (warp, u, lane): ex[u] = sum of all values that
// come before this thread's u-th one.
template <int TPT>
__device__ __forceinline__ void block_scan_tokens(const uint32_t (&p)[TPT], uint32_t (&ex)[TPT], uint32_t* wt,
                                                  uint32_t& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  uint32_t run = 0;                                    // the warp's values of the lower u (warp-uniform)
#pragma unroll
  for (int u = 0; u < TPT; ++u) {
    uint32_t incl = p[u];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    ex[u] = run + incl - p[u];
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 31) wt[wid] = run;
  __syncthreads();
  const uint32_t w = wt[lane];                          // SEL_WARPS == 32
  uint32_t wi = w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
    if (lane >= o) wi += n;
  }
  total = __shfl_sync(0xffffffffu, wi, 31);
  const uint32_t warp_before = __shfl_sync(0xffffffffu, wi - w, wid);
#pragma unroll
  for (int u = 0; u < TPT; ++u) ex[u] += warp_before;
}

template <bool EXPANDED, int TPT>
__global__ void __launch_bounds__(SEL_THREADS)
k_select_cluster(const float* __restrict__ score_src,   // topk_score [N,k] (Token Drop) or scores [N,E] (Expanded)
                 const int32_t* __restrict__ topk_idx, int64_t N, int E, int k, int64_t C, int D,
                 const int32_t* __restrict__ token_group, const int32_t* __restrict__ load /* [E] or NULL */, int R,
                 int64_t T /* tokens per CTA */, int32_t* __restrict__ cand_out /* [E] or NULL */, int32_t* __restrict__ kept,
                 int32_t* __restrict__ expert_offsets, int32_t* __restrict__ slot_row) {
  allow_next_kernel();
  wait_for_previous_kernel();
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ int hist[3][RADIX_BINS];               // the leader's copies are the cluster's histograms
  __shared__ int cnt[MAX_E];                        // tokens of this CTA whose top-k holds expert e'
  __shared__ int dupc[MAX_E];                       // ... and whose home device is that of e' (Expanded Drop)
  __shared__ int homec[MAX_E];                      // tokens of this CTA per home device (explicit token_group only)
  __shared__ uint32_t wt[5][SEL_WARPS];             // warp totals of the five block scans
  __shared__ uint32_t found[4][3];
  __shared__ uint32_t totals[MAX_R];                // per CTA of the cluster: kept-above | equal << 16
  const int tid = threadIdx.x, lane = tid & 31;
  const int rank = R > 1 ? (int)cluster.block_rank() : 0;
  const int e = blockIdx.x / R;
  const int m = EXPANDED ? E / D : 1;
  const int slots = EXPANDED ? k + m : k;
  const bool count_homes = EXPANDED && token_group != nullptr;

  for (int i = tid; i < 3 * RADIX_BINS; i += SEL_THREADS) (&hist[0][0])[i] = 0;
  if (tid < MAX_E) { cnt[tid] = 0; dupc[tid] = 0; homec[tid] = 0; }
  __syncthreads();

  // This thread's tokens (see the head of the file).  Sixteen top-k entries (JJ of every token) are
  // requested before the first is used, so that the loads of a thread overlap; each entry is counted
  // for its expert and compared with this cluster's expert.
  const int64_t hi = min(N, (int64_t)(rank + 1) * T);
  const int64_t tok0 = (int64_t)rank * T + (int64_t)(tid >> 5) * (32 * TPT) + lane;   // token of u: tok0 + 32 u
  int slot[TPT], home_lo[TPT];                      // home_lo: first expert of the token's home device
  uint32_t key[TPT];
  bool dup[TPT];                                    // Expanded Drop: home-device expert that is already a top-k slot
  {
    int g = 0;
#pragma unroll
    for (int u = 0; u < TPT; ++u) {
      const int64_t t = tok0 + 32 * u;
      slot[u] = -1; dup[u] = false; home_lo[u] = -m;   // (-m for a token past the end: matches no expert)
      if (EXPANDED && t < hi) {
        if (token_group) g = token_group[t];
        else if (u == 0) g = (int)((t * (int64_t)D) / N);
        else while ((int64_t)(g + 1) * N <= t * (int64_t)D) ++g;        // floor(t * D / N), from the previous token's
        home_lo[u] = g * m;
        if (count_homes) atomicAdd(&homec[g], 1);
      }
    }
  }
  // A token's k entries are contiguous and the lanes of a warp hold consecutive tokens; with k a
  // multiple of 4 (or 2) the entries are fetched four (two) at a time.  (With TPT consecutive tokens
  // per thread and scalar loads this loop took 7 of the kernel's 18 us at 64 experts and k = 8, 19 of
  // 42 us at 16384 tokens with k = 6: every load instruction touched up to 32 cache lines.)
  constexpr int JJ = TPT <= 2 ? 8 : 16 / TPT;
  const uintptr_t idx_addr = reinterpret_cast<uintptr_t>(topk_idx);
  const int vec = (k & 3) == 0 && JJ >= 4 && (idx_addr & 15) == 0 ? 4 : (k & 1) == 0 && (idx_addr & 7) == 0 ? 2 : 1;
  for (int j0 = 0; j0 < k; j0 += JJ) {
    int32_t v[TPT][JJ];
    if (vec == 4) {
      if constexpr (JJ >= 4) {
#pragma unroll
        for (int u = 0; u < TPT; ++u)
#pragma unroll
          for (int jj = 0; jj < JJ; jj += 4) {
            int4 q = make_int4(-1, -1, -1, -1);
            if (tok0 + 32 * u < hi && j0 + jj < k) q = *reinterpret_cast<const int4*>(topk_idx + (tok0 + 32 * u) * k + j0 + jj);
            v[u][jj] = q.x; v[u][jj + 1] = q.y; v[u][jj + 2] = q.z; v[u][jj + 3] = q.w;
          }
      }
    } else if (vec == 2) {
#pragma unroll
      for (int u = 0; u < TPT; ++u)
#pragma unroll
        for (int jj = 0; jj < JJ; jj += 2) {
          int2 q = make_int2(-1, -1);
          if (tok0 + 32 * u < hi && j0 + jj < k) q = *reinterpret_cast<const int2*>(topk_idx + (tok0 + 32 * u) * k + j0 + jj);
          v[u][jj] = q.x; v[u][jj + 1] = q.y;
        }
    } else {
#pragma unroll
      for (int u = 0; u < TPT; ++u)
#pragma unroll
        for (int jj = 0; jj < JJ; ++jj)
          v[u][jj] = (tok0 + 32 * u < hi && j0 + jj < k) ? topk_idx[(tok0 + 32 * u) * k + j0 + jj] : -1;
    }
#pragma unroll
    for (int u = 0; u < TPT; ++u)
#pragma unroll
      for (int jj = 0; jj < JJ; ++jj) {
        const int ev = v[u][jj];
        if (ev >= 0) {
          if (!load) atomicAdd(&cnt[ev], 1);          // (aggregating these per warp with match.any measured slower)
          if (EXPANDED && (unsigned)(ev - home_lo[u]) < (unsigned)m) atomicAdd(&dupc[ev], 1);
          if (ev == e) slot[u] = j0 + jj;
        }
      }
  }
  if (EXPANDED) {
#pragma unroll
    for (int u = 0; u < TPT; ++u)
      if (home_lo[u] == e - e % m) {
        if (slot[u] < 0) slot[u] = k + (e % m);
        else dup[u] = true;
      }
  }
#pragma unroll
  for (int u = 0; u < TPT; ++u) {
    const int64_t t = tok0 + 32 * u;
    key[u] = 0;
    if (slot[u] >= 0) key[u] = __float_as_uint(EXPANDED ? score_src[t * E + e] : score_src[t * k + slot[u]]);
  }
  if (R > 1) cluster.sync(); else __syncthreads();  // every CTA of the cluster runs and has counted its tokens

  // candidates of every expert over all N tokens; this expert's total and its segment's row offset
  uint32_t off, n;
  {
    uint32_t c_mine = 0;                            // thread e' < E: cand[e']
    if (tid < E) {
      int c = load ? load[tid] : 0, dd = 0, hh = 0;
      for (int q = 0; q < R; ++q) {
        if (!load) c += R > 1 ? *cluster.map_shared_rank(&cnt[tid], q) : cnt[tid];
        if (EXPANDED) dd += R > 1 ? *cluster.map_shared_rank(&dupc[tid], q) : dupc[tid];
        if (count_homes) hh += R > 1 ? *cluster.map_shared_rank(&homec[tid / m], q) : homec[tid / m];
      }
      if (EXPANDED) {
        if (!count_homes) {                         // contiguous blocks: tokens t with floor(t*D/N) == g
          const int64_t g = tid / m;
          hh = (int)((((g + 1) * N + D - 1) / D) - ((g * N + D - 1) / D));
        }
        c += hh - dd;                               // home-device tokens that do not already hold e' in their top-k
      }
      c_mine = (uint32_t)c;
    }
    const uint32_t kc = c_mine < (uint32_t)C ? c_mine : (uint32_t)C;
    uint32_t total;
    const uint32_t o = block_scan1(kc, wt[0], total);
    if (tid == e) { found[0][0] = o; found[0][1] = c_mine; }
    __syncthreads();
    off = found[0][0]; n = found[0][1];
  }
  const uint32_t keep_n = n < (uint32_t)C ? n : (uint32_t)C;
  if (rank == 0 && tid == 0) {
    kept[e] = (int32_t)keep_n;
    expert_offsets[e] = (int32_t)off;
    if (e == E - 1) expert_offsets[E] = (int32_t)(off + keep_n);
    if (cand_out) cand_out[e] = (int32_t)n;
  }
  const bool select = n > keep_n && C > 0;          // over capacity: a threshold has to be found
  const bool keep_all = n <= keep_n;                // (C == 0 with candidates: keep none)

  uint32_t tau = 0, need = 0;
  if (select) {
    // One radix level: digits of the candidates that match the prefix so far go to the leader's
    // histogram (one atomic per distinct digit per warp); the leader finds the bin that holds the
    // rank-th largest key (thread i sums bins 2i and 2i+1 counted from the top, a block scan locates
    // the pair) and tells every CTA: (bin, rank inside the bin, keys in the bin).
    auto level = [&](int lv, uint32_t prefix_shift, uint32_t prefix, uint32_t digit_shift, uint32_t digit_mask,
                     int nbins, uint32_t rank_left, uint32_t& bin, uint32_t& rank_in_bin, uint32_t& in_bin) {
      int* lead = R > 1 ? cluster.map_shared_rank(&hist[lv][0], 0) : &hist[lv][0];
#pragma unroll
      for (int u = 0; u < TPT; ++u) {
        const bool in = slot[u] >= 0 && (prefix_shift >= 32u || (key[u] >> prefix_shift) == prefix);
        const uint32_t digit = in ? ((key[u] >> digit_shift) & digit_mask) : 0xffffffffu;
        const unsigned same = __match_any_sync(0xffffffffu, digit);
        if (in && lane == __ffs(same) - 1) atomicAdd(&lead[digit], __popc(same));
      }
      if (R > 1) cluster.sync(); else __syncthreads();
      if (rank == 0) {
        const int p0 = 2 * tid, p1 = p0 + 1;
        const uint32_t h0 = p0 < nbins ? (uint32_t)hist[lv][nbins - 1 - p0] : 0u;
        const uint32_t h1 = p1 < nbins ? (uint32_t)hist[lv][nbins - 1 - p1] : 0u;
        uint32_t total;
        const uint32_t before = block_scan1(h0 + h1, wt[1 + lv], total);
        uint32_t b = 0xffffffffu, r = 0, c = 0;
        if (before < rank_left && rank_left <= before + h0) { b = (uint32_t)(nbins - 1 - p0); r = rank_left - before; c = h0; }
        else if (before + h0 < rank_left && rank_left <= before + h0 + h1) {
          b = (uint32_t)(nbins - 1 - p1); r = rank_left - before - h0; c = h1;
        }
        if (b != 0xffffffffu)                         // exactly one thread: it tells every CTA of the cluster
          for (int q = 0; q < R; ++q) {
            uint32_t* f = R > 1 ? cluster.map_shared_rank(&found[1 + lv][0], q) : &found[1 + lv][0];
            f[0] = b; f[1] = r; f[2] = c;
          }
      }
      if (R > 1) cluster.sync(); else __syncthreads();
      bin = found[1 + lv][0];
      rank_in_bin = found[1 + lv][1];
      in_bin = found[1 + lv][2];
    };
    // A level whose bin is kept as a whole ends the search: the threshold is the bin's lowest key,
    // and every key equal to it is kept.
    uint32_t b1, b2, b3, in_bin, rank_left = (uint32_t)C;
    level(0, 32u, 0u, 21u, 2047u, RADIX_BINS, rank_left, b1, rank_left, in_bin);
    if (rank_left == in_bin) { tau = b1 << 21; need = 0xffffffffu; }
    else {
      level(1, 21u, b1, 10u, 2047u, RADIX_BINS, rank_left, b2, rank_left, in_bin);
      const uint32_t prefix = (b1 << 11) | b2;
      if (rank_left == in_bin) { tau = prefix << 10; need = 0xffffffffu; }
      else {
        level(2, 10u, prefix, 0u, 1023u, 1024, rank_left, b3, rank_left, in_bin);
        tau = (prefix << 10) | b3;
        need = rank_left;                           // how many candidates equal to tau are kept
      }
    }
  }

  // ranks in token order: kept = above tau, plus the first `need` equal to it
  uint32_t packed[TPT], before[TPT];
#pragma unroll
  for (int u = 0; u < TPT; ++u) {
    packed[u] = 0;
    if (slot[u] >= 0) {
      const bool gt = keep_all || (select && key[u] > tau), eq = select && key[u] == tau;
      packed[u] = (gt ? 1u : 0u) | (eq ? 0x10000u : 0u);
    }
  }
  uint32_t tot;
  block_scan_tokens<TPT>(packed, before, wt[4], tot);           // a CTA holds at most 8192 tokens: 16 bits each
  if (R > 1) {
    if (tid < R) *cluster.map_shared_rank(&totals[rank], tid) = tot;
    cluster.sync();                                 // last access to another CTA's shared memory is behind us
  }
  uint32_t gt_base = 0, eq_base = 0;
  for (int r = 0; r < rank; ++r) { gt_base += totals[r] & 0xffffu; eq_base += totals[r] >> 16; }
#pragma unroll
  for (int u = 0; u < TPT; ++u) {
    const int64_t t = tok0 + 32 * u;
    if (slot[u] >= 0) {
      const uint32_t gt_before = gt_base + (before[u] & 0xffffu), eq_before = eq_base + (before[u] >> 16);
      const bool keep = (packed[u] & 1u) || ((packed[u] >> 16) && eq_before < need);
      slot_row[t * slots + slot[u]] = keep ? (int32_t)(off + gt_before + (eq_before < need ? eq_before : need)) : -1;
    }
    if (EXPANDED && dup[u]) slot_row[t * slots + k + (e % m)] = -1;   // that slot is the top-k slot's duplicate
  }
}

// keep_mask[t] from slot_row[t, :]: bit e of a token is set iff the slot that stands for expert e
// holds a row.  One thread per token.
__global__ void __launch_bounds__(256)
k_mask_from_rows(const int32_t* __restrict__ slot_row, const int32_t* __restrict__ topk_idx, int64_t N, int E, int k,
                 int slots, int D, const int32_t* __restrict__ token_group, unsigned long long* __restrict__ keep_mask) {
  allow_next_kernel();
  wait_for_previous_kernel();
  const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (t >= N) return;
  const int W = (E + 63) >> 6;
  unsigned long long w[MAX_E / 64] = {0ull, 0ull, 0ull, 0ull};
  const int32_t* sr = slot_row + t * slots;
  const int m = slots > k ? E / D : 0;
  const int g = slots > k ? home_group(t, N, D, token_group) : 0;
  auto mark = [&](int s, int row) {
    if (row >= 0) {
      const int e = s < k ? topk_idx[t * k + s] : g * m + (s - k);
#pragma unroll
      for (int i = 0; i < MAX_E / 64; ++i)
        if (i == (e >> 6)) w[i] |= 1ull << (e & 63);
    }
  };
  if ((slots & 3) == 0 && (reinterpret_cast<uintptr_t>(slot_row) & 15) == 0) {   // rows of 16-byte pieces: four entries per load
    for (int s = 0; s < slots; s += 4) {
      const int4 q = *reinterpret_cast<const int4*>(sr + s);
      mark(s, q.x); mark(s + 1, q.y); mark(s + 2, q.z); mark(s + 3, q.w);
    }
  } else {
    for (int s = 0; s < slots; ++s) mark(s, sr[s]);
  }
#pragma unroll
  for (int i = 0; i < MAX_E / 64; ++i)
    if (i < W) keep_mask[t * W + i] = w[i];
}

template <bool EXPANDED, int TPT>
cudaError_t launch_inst(unsigned grid, int R, cudaStream_t st, const float* score_src, const int32_t* topk_idx, int64_t N,
                        int E, int k, int64_t C, int D, const int32_t* token_group, const int32_t* load, int64_t T,
                        int32_t* cand_out, int32_t* kept, int32_t* expert_offsets, int32_t* slot_row) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(SEL_THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)R; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see wait_for_previous_kernel()
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, k_select_cluster<EXPANDED, TPT>, score_src, topk_idx, N, E, k, C, D, token_group, load, R,
                            T, cand_out, kept, expert_offsets, slot_row);
}

}  // namespace

// CTAs per expert: enough to occupy the GPU, but at least 512 tokens each.  Two 1024-thread CTAs
// fit an SM, which pays for Token Drop, where only the overloaded experts have a threshold to
// find; under Expanded Drop every expert does, and one CTA per SM measured faster.
static int cluster_size(int64_t N, int E, bool expanded) {
  int R = 1;
  const int sms = sm_count();
  while (R < MAX_R && E * (2 * R) <= (expanded ? sms : 2 * sms) && ceil_div(N, 2 * R) >= 512) R *= 2;
  return R;
}

// Whether the cluster select serves this batch (else the token-parallel select of drop_parallel.cu):
// while a CTA holds at most 8 tokens per thread.  Every cluster reads all N top-k lists, E times in
// total, but out of L2 and in one launch; the token-parallel select takes 13.  Measured (stage call
// replayed from a graph / inside a layer forward): 32768 tokens, 60 experts, Token Drop 28 / 31 us
// against 42 / 58 us; 64 experts 47 / 46 against 50 / 75 us; 16384 tokens, 64 experts, Expanded Drop
// 38 / 54 against 57 / 89 us.
bool drop_cluster_takes(int64_t N, int E, bool expanded) {
  const int max_tpt = 8;
  return N > 0 && ceil_div(N, cluster_size(N, E, expanded)) <= (int64_t)SEL_THREADS * max_tpt;
}

int drop_mask_from_rows(const int32_t* slot_row, const int32_t* topk_idx, int64_t N, int E, int k, int slots, int D,
                        const int32_t* token_group, uint64_t* keep_mask, cudaStream_t st) {
  const int rc = note_cuda(launch_chained(k_mask_from_rows, (unsigned)ceil_div(N, 256), 256, 0, st, slot_row, topk_idx, N,
                                          E, k, slots, D, token_group, reinterpret_cast<unsigned long long*>(keep_mask)));
  count_launch(1);
  return rc;
}

// keep_mask == NULL: the caller derives the mask from slot_row itself (drop_mask_from_rows, or the
// permute kernel of a layer forward).  load: the router's load histogram [E] (device) or NULL.
template <bool EXPANDED>
int drop_cluster(const float* score_src, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C, int D,
                 const int32_t* token_group, const int32_t* load, uint64_t* keep_mask, int32_t* cand_out, int32_t* kept,
                 int32_t* expert_offsets, int32_t* slot_row, cudaStream_t st) {
  const int R = cluster_size(N, E, EXPANDED);
  const int64_t T = ceil_div(N, R);
  const unsigned grid = (unsigned)(E * R);
  cudaError_t err;
#define CAPMOE_SEL_CASE(TPT_)                                                                                      \
  err = launch_inst<EXPANDED, TPT_>(grid, R, st, score_src, topk_idx, N, E, k, C, D, token_group, load, T, cand_out, kept, \
                                    expert_offsets, slot_row)
  if (T <= SEL_THREADS) CAPMOE_SEL_CASE(1);
  else if (T <= 2 * SEL_THREADS) CAPMOE_SEL_CASE(2);
  else if (T <= 4 * SEL_THREADS) CAPMOE_SEL_CASE(4);
  else if (T <= 8 * SEL_THREADS) CAPMOE_SEL_CASE(8);
  else return CAPMOE_EUNSUPPORTED;
#undef CAPMOE_SEL_CASE
  count_launch(1);
  if (err != cudaSuccess) return note_cuda(err);
  if (!keep_mask) return CAPMOE_OK;
  return drop_mask_from_rows(slot_row, topk_idx, N, E, k, EXPANDED ? k + E / D : k, D, token_group, keep_mask, st);
}

template int drop_cluster<false>(const float*, const int32_t*, int64_t, int, int, int64_t, int, const int32_t*,
                                 const int32_t*, uint64_t*, int32_t*, int32_t*, int32_t*, int32_t*, cudaStream_t);
template int drop_cluster<true>(const float*, const int32_t*, int64_t, int, int, int64_t, int, const int32_t*,
                                const int32_t*, uint64_t*, int32_t*, int32_t*, int32_t*, int32_t*, cudaStream_t);

}  // namespace capmoe
