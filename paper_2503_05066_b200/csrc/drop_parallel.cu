// Token-parallel capacity select, used for large batches and for device-level capacity.
//
// The single-CTA-per-expert kernels in drop.cu walk the token list with block scans, which is
// fine up to a few thousand candidates per expert but serialises at N = 65536 or when one
// "segment" is a whole device.  Here every step is spread over all SMs (one CTA per 256 tokens):
//
//   segment        the set that shares one capacity: an expert (Token / Expanded Drop) or a
//                  device (device-level capacity); S = E / seg_m segments.
//   key            64 bits per candidate pair (t, e): score bits in the high word, the inverted
//                  position  (2^P - 1) - (t*E + e)  in the low word.  Descending key order is
//                  (score descending, token ascending, expert ascending): exactly the keep order,
//                  and all keys are distinct, so "keep the C best" is just  key >= tau[segment].
//   pk_hist        one radix level: histogram of one digit of the keys that match the prefix
//                  found so far (integer atomics into [S][2048] counters).
//   pk_find        one CTA per segment: the bin that holds the C-th largest key extends the prefix;
//                  clears the counters for the next level.  Score digits 11/11/10 bits, then
//                  position digits; a segment stops as soon as its whole selected bin is kept
//                  (no ties at the threshold: after the three score levels), and once no segment
//                  is left the remaining levels return at once.
//   pk_count       kept pairs per (chunk, expert)
//   pk_scan        per expert: exclusive scan over chunks -> rank base per chunk, kept[e]
//   pk_place       per chunk: bitmap of kept tokens per expert -> rank inside the chunk by popcount;
//                  row = offset[e] + base[chunk][e] + rank; writes slot_row, keep_mask, offsets.
// Every output word is written exactly once, without atomics, so nothing needs initialising
// except the histogram area (one memset).
#include "common.cuh"

namespace capmoe {
namespace {

constexpr int CHUNK = 256;           // tokens per CTA
constexpr int TPT = 4;               // threads per token in the kernels that walk the candidate pairs:
                                     // thread (token, j) takes slots j, j + TPT, ...  A warp then holds one
                                     // slot of 32 consecutive tokens: for the home-device slots that is one
                                     // expert, and its histogram updates merge in the atomic unit (pairs in
                                     // (token, slot) order across a warp measured 1.5x slower for that reason)
constexpr int PAIR_THREADS = CHUNK * TPT;
constexpr int BINS = 2048;
constexpr int MAX_LEVELS = 6;
constexpr int MAX_SEG = 256;

struct Level { int shift, bits; };


struct SegState {                    // one per segment, in global memory
  unsigned long long prefix;         // key bits fixed so far (tau once done)
  uint32_t rank;                     // how many keys of the current bin are still to be kept
  uint32_t done;                     // 1: tau final
  uint32_t n;                        // candidate pairs of the segment
  uint32_t pad;
};

struct PWs {
  uint32_t* hist;        // [S][BINS]
  uint32_t* active;      // [8] per level: segments that still need another level
  int32_t* cand;         // [256]
  SegState* seg;         // [S]
  int32_t* cnt;          // [chunks][E] kept pairs per chunk and expert
  int32_t* base;         // [chunks][E] exclusive scan of cnt over chunks
};

inline size_t al256(size_t v) { return (v + 255) & ~(size_t)255; }

struct PArgs {
  const float* scores;       // [N,E] or null (then only top-k slots exist and topk_score is used)
  const float* topk_score;   // [N,k] or null
  const int32_t* topk_idx;   // [N,k]
  const int32_t* token_group;
  int64_t N;
  int E, k, D, m, seg_m, slots, expanded, pos_bits;
  unsigned long long C_seg;
};

// Expert and key of slot s of token t; returns false if the slot is not a candidate.
__device__ __forceinline__ bool pair_of(const PArgs& a, int64_t t, int s, const int32_t* row, int home, int& e,
                                        unsigned long long& key) {
  float sc;
  if (s < a.k) {
    e = row[s];
    sc = a.topk_score ? a.topk_score[t * a.k + s] : a.scores[t * a.E + e];
  } else {
    e = home * a.m + (s - a.k);
    for (int j = 0; j < a.k; ++j)
      if (row[j] == e) return false;                 // already a top-k slot
    sc = a.scores[t * a.E + e];
  }
  const unsigned long long pos = (unsigned long long)t * (unsigned)a.E + (unsigned)e;
  const unsigned long long inv = ((1ull << a.pos_bits) - 1ull) - pos;
  key = ((unsigned long long)__float_as_uint(sc) << 32) | inv;
  return true;
}

__global__ void __launch_bounds__(PAIR_THREADS)
pk_hist(PArgs a, PWs w, int level, Level lv, int first_level_counts_cand) {
  allow_next_kernel();
  wait_for_previous_kernel();
  __shared__ int cand_s[MAX_SEG];
  const int tid = threadIdx.x;
  if (level > 0 && __ldcg(&w.active[level - 1]) == 0u) return;       // every segment already has its tau
  if (first_level_counts_cand)
    for (int i = tid; i < a.E; i += PAIR_THREADS) cand_s[i] = 0;
  __syncthreads();
  const int64_t t = (int64_t)blockIdx.x * CHUNK + (tid & (CHUNK - 1));
  const bool tok_ok = t < a.N;
  const int32_t* row = a.topk_idx + (tok_ok ? t : 0) * a.k;
  const int home = (a.expanded && tok_ok) ? home_group(t, a.N, a.D, a.token_group) : 0;
  const int lane = tid & 31;
  // (the slot index is the same for all lanes of a warp, so the warp stays together in this loop)
  for (int s = tid / CHUNK; s < a.slots; s += TPT) {
    int e = 0;
    unsigned long long key = 0;
    bool in = tok_ok && pair_of(a, t, s, row, home, e, key);
    if (in && first_level_counts_cand) atomicAdd(&cand_s[e], 1);
    const int sg = e / a.seg_m;
    if (in && level > 0) {
      const SegState st = w.seg[sg];
      const int hi = lv.shift + lv.bits;                         // < 64 for every level after the first
      in = !st.done && (key >> hi) == (st.prefix >> hi);
    }
    const uint32_t digit = (uint32_t)(key >> lv.shift) & ((1u << lv.bits) - 1u);
    if (level == 0) {
      // Every candidate takes part in the first level, and a warp's lanes hold one slot of 32
      // consecutive tokens: for a home-device slot that is one expert, whose scores fall into a few
      // bins.  One atomic per distinct (segment, bin) of the warp instead of one per lane.
      const uint32_t bin = in ? (uint32_t)sg * BINS + digit : 0xffffffffu - (uint32_t)lane;
      const unsigned same = __match_any_sync(0xffffffffu, bin);
      if (in && lane == __ffs(same) - 1) atomicAdd(&w.hist[bin], (uint32_t)__popc(same));
    } else if (in) {
      atomicAdd(&w.hist[(size_t)sg * BINS + digit], 1u);
    }
  }
  __syncthreads();
  if (first_level_counts_cand)
    for (int i = tid; i < a.E; i += PAIR_THREADS)
      if (cand_s[i]) atomicAdd(&w.cand[i], cand_s[i]);
}

// One CTA per segment: pick the bin that holds the rank-th largest key of this level, extend the
// prefix, clear the counters.  Thread i owns 8 consecutive bins, highest bins first.
__global__ void __launch_bounds__(CHUNK)
pk_find(PWs w, unsigned long long C_seg, int level, Level lv, int n_levels) {
  allow_next_kernel();
  wait_for_previous_kernel();
  __shared__ uint32_t wtot[CHUNK / 32 + 1];
  __shared__ uint32_t res[3];
  const int sg = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (level > 0 && __ldcg(&w.active[level - 1]) == 0u) return;
  uint32_t* h = w.hist + (size_t)sg * BINS;
  SegState st;
  if (level == 0) { st.prefix = 0; st.rank = 0; st.done = 0; st.n = 0; st.pad = 0; }
  else st = w.seg[sg];
  if (st.done) return;                                            // nothing was counted for it
  const int nb = 1 << lv.bits;
  constexpr int PER = BINS / CHUNK;                               // 8
  uint32_t c[PER];
  uint32_t local = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const int b = nb - 1 - (tid * PER + i);
    c[i] = b >= 0 ? __ldcg(&h[b]) : 0u;
    local += c[i];
  }
  uint32_t incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) wtot[wid] = incl;
  if (tid < 3) res[tid] = 0xffffffffu;
  __syncthreads();
  if (tid == 0) {
    uint32_t acc = 0;
    for (int i = 0; i < CHUNK / 32; ++i) { const uint32_t x = wtot[i]; wtot[i] = acc; acc += x; }
    wtot[CHUNK / 32] = acc;
  }
  __syncthreads();
  const uint32_t total = wtot[CHUNK / 32];
  const uint32_t before = wtot[wid] + incl - local;               // keys in bins above this thread's
  if (level == 0) {
    st.n = total;
    if (C_seg == 0) { st.prefix = ~0ull; st.done = 1; }                          // keep nothing
    else if ((unsigned long long)total <= C_seg) { st.prefix = 0; st.done = 1; } // keep everything
    else st.rank = (uint32_t)C_seg;
  }
  if (!st.done) {
    if (before < st.rank && st.rank <= before + local) {          // exactly one thread
      uint32_t acc = before;
#pragma unroll
      for (int i = 0; i < PER; ++i) {
        if (acc < st.rank && st.rank <= acc + c[i]) {
          res[0] = (uint32_t)(nb - 1 - (tid * PER + i)); res[1] = st.rank - acc; res[2] = c[i];
        }
        acc += c[i];
      }
    }
  }
  __syncthreads();
  if (!st.done) {
    st.prefix |= (unsigned long long)res[0] << lv.shift;
    st.rank = res[1];
    if (res[1] == res[2] || level == n_levels - 1) st.done = 1;   // the whole selected bin is kept
  }
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const int b = nb - 1 - (tid * PER + i);
    if (b >= 0) h[b] = 0u;                                         // ready for the next level
  }
  if (tid == 0) {
    w.seg[sg] = st;
    if (!st.done) atomicAdd(&w.active[level], 1u);
  }
}

__global__ void __launch_bounds__(PAIR_THREADS)
pk_count(PArgs a, PWs w) {
  allow_next_kernel();
  wait_for_previous_kernel();
  __shared__ int cnt_s[MAX_SEG];
  const int tid = threadIdx.x;
  for (int i = tid; i < a.E; i += PAIR_THREADS) cnt_s[i] = 0;
  __syncthreads();
  const int64_t t = (int64_t)blockIdx.x * CHUNK + (tid & (CHUNK - 1));
  if (t < a.N) {
    const int32_t* row = a.topk_idx + t * a.k;
    const int home = a.expanded ? home_group(t, a.N, a.D, a.token_group) : 0;
    for (int s = tid / CHUNK; s < a.slots; s += TPT) {
      int e;
      unsigned long long key;
      if (!pair_of(a, t, s, row, home, e, key)) continue;
      if (key >= w.seg[e / a.seg_m].prefix) atomicAdd(&cnt_s[e], 1);
    }
  }
  __syncthreads();
  for (int i = tid; i < a.E; i += PAIR_THREADS) w.cnt[(int64_t)blockIdx.x * a.E + i] = cnt_s[i];
}

// one CTA per expert: exclusive scan of its per-chunk counts
__global__ void __launch_bounds__(CHUNK)
pk_scan(PWs w, int E, int chunks, int32_t* __restrict__ kept, int32_t* __restrict__ cand_out) {
  allow_next_kernel();
  wait_for_previous_kernel();
  __shared__ int warp_tot[CHUNK / 32 + 1];
  const int e = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  int running = 0;
  for (int c0 = 0; c0 < chunks; c0 += CHUNK) {
    const int c = c0 + tid;
    const int v = c < chunks ? w.cnt[(int64_t)c * E + e] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    if (tid == 0) {
      int acc = 0;
      for (int i = 0; i < CHUNK / 32; ++i) { const int x = warp_tot[i]; warp_tot[i] = acc; acc += x; }
      warp_tot[CHUNK / 32] = acc;
    }
    __syncthreads();
    if (c < chunks) w.base[(int64_t)c * E + e] = running + warp_tot[wid] + incl - v;
    running += warp_tot[CHUNK / 32];
    __syncthreads();
  }
  if (tid == 0) {
    kept[e] = running;
    if (cand_out) cand_out[e] = w.cand[e];
  }
}

__global__ void __launch_bounds__(PAIR_THREADS)
pk_place(PArgs a, PWs w, const int32_t* __restrict__ kept, unsigned long long* __restrict__ keep_mask,
         int32_t* __restrict__ expert_offsets, int32_t* __restrict__ slot_row) {
  allow_next_kernel();
  wait_for_previous_kernel();
  __shared__ int off[MAX_SEG + 1];
  __shared__ uint32_t bitmap[MAX_SEG][CHUNK / 32];
  __shared__ unsigned long long mask_s[CHUNK][4];               // keep mask of the chunk's tokens (E <= 256)
  __shared__ int wtot[CHUNK / 32 + 1];
  const int tid = threadIdx.x, lane = tid & 31;
  const int tl = tid & (CHUNK - 1);                             // token of the chunk this thread works for
  const int wt = tl >> 5;                                       // that token's 32-token word in the bitmaps
  const int sub = tid / CHUNK;                                  // which of the token's TPT threads
  // offsets = exclusive prefix of kept (E <= 256 = CHUNK), by the first CHUNK threads
  {
    int v = 0, incl = 0;
    if (tid < CHUNK) {
      v = tid < a.E ? kept[tid] : 0;
      incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (lane == 31) wtot[tid >> 5] = incl;
    }
    __syncthreads();
    if (tid == 0) {
      int acc = 0;
      for (int i = 0; i < CHUNK / 32; ++i) { const int x = wtot[i]; wtot[i] = acc; acc += x; }
      wtot[CHUNK / 32] = acc;
    }
    __syncthreads();
    if (tid < a.E) off[tid] = wtot[tid >> 5] + incl - v;
    if (tid == 0) off[a.E] = wtot[CHUNK / 32];
  }
  for (int i = tid; i < a.E * (CHUNK / 32); i += PAIR_THREADS) (&bitmap[0][0])[i] = 0u;
  for (int i = tid; i < CHUNK * 4; i += PAIR_THREADS) (&mask_s[0][0])[i] = 0ull;
  __syncthreads();
  if (blockIdx.x == 0)
    for (int i = tid; i <= a.E; i += PAIR_THREADS) expert_offsets[i] = off[i];

  const int64_t t = (int64_t)blockIdx.x * CHUNK + tl;
  const bool live = t < a.N;
  const int32_t* row = a.topk_idx + (live ? t : 0) * a.k;
  const int home = (live && a.expanded) ? home_group(t, a.N, a.D, a.token_group) : 0;
  const int W = (a.E + 63) >> 6;
  if (live) {
    for (int s = sub; s < a.slots; s += TPT) {
      int e;
      unsigned long long key;
      if (!pair_of(a, t, s, row, home, e, key)) continue;
      if (key >= w.seg[e / a.seg_m].prefix) atomicOr(&bitmap[e][wt], 1u << lane);
    }
  }
  __syncthreads();
  if (live) {
    for (int s = sub; s < a.slots; s += TPT) {
      int e;
      unsigned long long key;
      int32_t out = -1;
      if (pair_of(a, t, s, row, home, e, key) && ((bitmap[e][wt] >> lane) & 1u)) {
        int r = __popc(bitmap[e][wt] & ((1u << lane) - 1u));
        for (int i = 0; i < wt; ++i) r += __popc(bitmap[e][i]);
        out = off[e] + w.base[(int64_t)blockIdx.x * a.E + e] + r;
        atomicOr(&mask_s[tl][e >> 6], 1ull << (e & 63));
      }
      slot_row[t * a.slots + s] = out;
    }
  }
  __syncthreads();
  if (live && sub == 0)
    for (int i = 0; i < W; ++i) keep_mask[t * W + i] = mask_s[tl][i];
}

PWs carve_p(void* ws, int64_t N, int E, int S) {
  const int64_t chunks = ceil_div(N, CHUNK);
  char* p = (char*)ws;
  PWs w;
  w.hist = (uint32_t*)p;  p += al256(sizeof(uint32_t) * (size_t)S * BINS);
  w.active = (uint32_t*)p; p += 256;
  w.cand = (int32_t*)p;   p += al256(sizeof(int32_t) * 256);
  w.seg = (SegState*)p;   p += al256(sizeof(SegState) * (size_t)S);
  w.cnt = (int32_t*)p;    p += al256(sizeof(int32_t) * (size_t)chunks * E);
  w.base = (int32_t*)p;
  return w;
}

}  // namespace

size_t drop_parallel_ws_bytes(int64_t N, int E) {
  const int64_t chunks = ceil_div(N, CHUNK);
  // sized for the largest segment count (S = E)
  return al256(sizeof(uint32_t) * (size_t)E * BINS) + 256 + al256(sizeof(int32_t) * 256) +
         al256(sizeof(SegState) * (size_t)E) + 2 * al256(sizeof(int32_t) * (size_t)chunks * E);
}

int drop_parallel_clear(void* ws_ptr, int64_t N, int E, int S, cudaStream_t st) {
  PWs w = carve_p(ws_ptr, N, E, S);
  return note_cuda(cudaMemsetAsync(w.hist, 0, (size_t)((char*)w.seg - (char*)w.hist), st));
}

// C_seg: capacity of one segment (expert: C; device: C_dev).  seg_m: experts per segment.
int drop_parallel(const float* scores, const float* topk_score, const int32_t* topk_idx, int64_t N, int E, int k,
                  int64_t C_seg, int D, int seg_m, int expanded, const int32_t* token_group, uint64_t* keep_mask,
                  int32_t* cand_out, int32_t* kept, int32_t* expert_offsets, int32_t* slot_row, void* ws_ptr,
                  size_t ws_bytes, cudaStream_t st, bool counters_cleared) {
  if (E > MAX_SEG) return CAPMOE_EUNSUPPORTED;
  if ((unsigned long long)N * (unsigned)E >= (1ull << 32)) return CAPMOE_EUNSUPPORTED;   // position word
  if (ws_bytes < drop_parallel_ws_bytes(N, E)) return CAPMOE_EWORKSPACE;
  const int S = E / seg_m;
  PWs w = carve_p(ws_ptr, N, E, S);
  PArgs a;
  a.scores = scores; a.topk_score = topk_score; a.topk_idx = topk_idx; a.token_group = token_group;
  a.N = N; a.E = E; a.k = k; a.D = D; a.m = expanded ? E / D : 1; a.seg_m = seg_m;
  a.slots = expanded ? k + E / D : k; a.expanded = expanded;
  int pos_bits = 1;
  while ((1ull << pos_bits) < (unsigned long long)N * (unsigned)E) ++pos_bits;
  a.pos_bits = pos_bits;
  a.C_seg = (unsigned long long)C_seg;
  // radix levels: the score word top down (11, 11, 10 bits), then the position word
  Level lv[MAX_LEVELS];
  int nl = 0;
  lv[nl++] = {53, 11}; lv[nl++] = {42, 11}; lv[nl++] = {32, 10};
  int left = pos_bits;
  while (left > 0) {
    const int b = left > 11 ? (left % 11 ? left % 11 : 11) : left;
    lv[nl++] = {left - b, b};
    left -= b;
  }
  // hist, tickets and candidate counters start at zero
  if (!counters_cleared) {
    const int rc0 = drop_parallel_clear(ws_ptr, N, E, S, st);
    if (rc0 != CAPMOE_OK) return rc0;
  }
  const unsigned chunks = (unsigned)ceil_div(N, CHUNK);
  int rc;
  for (int l = 0; l < nl; ++l) {
    if ((rc = note_cuda(launch_chained(pk_hist, chunks, PAIR_THREADS, 0, st, a, w, l, lv[l], l == 0 ? 1 : 0))) != CAPMOE_OK)
      return rc;
    count_launch(1);
    if ((rc = note_cuda(launch_chained(pk_find, (unsigned)S, CHUNK, 0, st, w, a.C_seg, l, lv[l], nl))) != CAPMOE_OK) return rc;
    count_launch(1);
  }
  if ((rc = note_cuda(launch_chained(pk_count, chunks, PAIR_THREADS, 0, st, a, w))) != CAPMOE_OK) return rc;
  count_launch(1);
  if ((rc = note_cuda(launch_chained(pk_scan, (unsigned)E, CHUNK, 0, st, w, E, (int)chunks, kept, cand_out))) != CAPMOE_OK)
    return rc;
  count_launch(1);
  rc = note_cuda(launch_chained(pk_place, chunks, PAIR_THREADS, 0, st, a, w, (const int32_t*)kept,
                                (unsigned long long*)keep_mask, expert_offsets, slot_row));
  count_launch(1);
  return rc;
}

}  // namespace capmoe
