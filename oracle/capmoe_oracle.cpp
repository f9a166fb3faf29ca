// CPU checker for the capacity-aware MoE layer forward.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
// layer computes; the tests, the smoke check and the CPU-baseline leg of the
// benchmark call it, the product never does.  It shares no code, header, table
// or helper with the CUDA library.
//
// Every function follows the paper's definitions step by step, in the paper's
// notation (N tokens, E experts, top-k, capacity factor gamma, capacity C,
// m = E/D experts per device):
//   router + softmax + top-k ............ Eq. 1, Algorithm 1 (first three statements)
//   mean load, capacity ................. Eq. 3, "C = gamma * N_bar", Algorithm 1 (cap)
//   Token Drop .......................... Eq. 7-10, Algorithm 1
//   Expanded Drop ....................... Section "Expanded Drop ...", Algorithm 2
//   dropped-token fraction .............. Eq. 11
//   expert FFN and weighted combine ..... Eq. 2 (SwiGLU expert: the paper leaves the expert's form open)
// Floating point: all arithmetic in double, except the softmax, whose scores
// decide integer outputs (keep masks); it is evaluated in IEEE binary32 with a
// fixed operation order (see oracle_softmax) so that the decision is taken in
// the same precision as on the GPU.
//
// Pins (tests/test_oracle_*.py): brute-force rank counting on tiny inputs, the
// dense-mask formulation of Algorithms 1/2, kept_e = min(N_e, C) (Eq. 11),
// Eq. 5 and Eq. 6 bounds, gamma = inf reproduces no-drop, D = 1 Expanded Drop
// equals expert-choice routing, k = E with identical experts equals one dense
// SwiGLU FFN (numpy fp64), softmax within 2 ulp of an fp64 softmax.
// No function here is "parity unpinned".
//
// Build: g++ -O3 -fopenmp -ffp-contract=off -shared -fPIC (no -ffast-math).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

enum { DT_F32 = 0, DT_BF16 = 1 };

inline double load_elem(const void* p, int64_t i, int dtype) {
  if (dtype == DT_F32) return (double)((const float*)p)[i];
  uint32_t bits = (uint32_t)((const uint16_t*)p)[i] << 16;   // bf16 is the top half of a binary32
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}

inline float f32_from_bits(uint32_t b) { float f; std::memcpy(&f, &b, 4); return f; }
inline uint32_t bits_from_f32(float f) { uint32_t b; std::memcpy(&b, &f, 4); return b; }

// exp(x) for x <= 0 in binary32 with a fixed sequence of correctly rounded operations.
inline float exp_spec(float x) {
  if (x < -80.0f) return 0.0f;
  const float log2e  = f32_from_bits(0x3fb8aa3bu);
  const float ln2_hi = f32_from_bits(0x3f317200u);
  const float ln2_lo = f32_from_bits(0x35bfbe8eu);
  float n = std::rint(x * log2e);                 // round-half-even, default rounding mode
  float r = std::fmaf(n, -ln2_hi, x);
  r = std::fmaf(n, -ln2_lo, r);
  float q = f32_from_bits(0x39500d01u);           // 1/5040
  q = std::fmaf(q, r, f32_from_bits(0x3ab60b61u)); // 1/720
  q = std::fmaf(q, r, f32_from_bits(0x3c088889u)); // 1/120
  q = std::fmaf(q, r, f32_from_bits(0x3d2aaaabu)); // 1/24
  q = std::fmaf(q, r, f32_from_bits(0x3e2aaaabu)); // 1/6
  q = std::fmaf(q, r, 0.5f);
  q = std::fmaf(q, r, 1.0f);
  q = std::fmaf(q, r, 1.0f);
  int32_t ni = (int32_t)n;                         // n in [-116, 0]
  return f32_from_bits(bits_from_f32(q) + ((uint32_t)ni << 23));   // q * 2^n, result stays normal
}

inline int64_t home_group(int64_t t, int64_t N, int D, const int32_t* token_group) {
  if (token_group) return token_group[t];
  return (t * (int64_t)D) / N;                     // contiguous token blocks
}

struct Cand { float s; int32_t t; int32_t slot; };

// Per-expert selection shared by Token Drop and Expanded Drop: candidates arrive in
// ascending token order; the C best by (score descending, token ascending) are kept
// (Eq. 8-10 with the tie rule "lower token index wins").
void select_and_place(std::vector<std::vector<Cand>>& cands, int64_t N, int E, int slots, int64_t C,
                      uint64_t* keep_mask, int32_t* kept, int32_t* offsets, int32_t* slot_row) {
  const int W = (E + 63) / 64;
  for (int64_t i = 0; i < N * W; ++i) keep_mask[i] = 0;
  for (int64_t i = 0; i < N * slots; ++i) slot_row[i] = -1;
  offsets[0] = 0;
  for (int e = 0; e < E; ++e) {
    std::vector<Cand>& c = cands[e];
    std::vector<Cand> order(c);
    std::stable_sort(order.begin(), order.end(), [](const Cand& a, const Cand& b) { return a.s > b.s; });
    int64_t keep_n = std::min<int64_t>((int64_t)order.size(), C);
    std::vector<char> is_kept(N > 0 ? N : 1, 0);
    for (int64_t i = 0; i < keep_n; ++i) is_kept[order[i].t] = 1;
    kept[e] = (int32_t)keep_n;
    int32_t row = offsets[e];
    for (const Cand& x : c) {                       // ascending token index inside the segment
      if (is_kept[x.t]) {
        keep_mask[(int64_t)x.t * W + (e >> 6)] |= (uint64_t)1 << (e & 63);
        slot_row[(int64_t)x.t * slots + x.slot] = row++;
      }
    }
    offsets[e + 1] = row;
  }
}

}  // namespace

extern "C" {

// Capacity C = gamma * N_bar with N_bar = N k / E (Eq. 3 and the capacity definition), evaluated
// as (gamma * (N*k)) / E in double (Algorithm 1's operation order).  round_mode 0 = ceil,
// 1 = floor (the listing's int()).  Clamped to [0, N]; gamma = +inf gives N (no drop).
int oracle_capacity(int64_t N, int E, int k, double gamma, int round_mode, int64_t* C) {
  if (N < 0 || E < 1 || k < 1 || k > E || !(gamma >= 0.0)) return 1;
  double c;
  if (std::isinf(gamma)) c = (double)N;
  else {
    double v = (gamma * (double)(N * (int64_t)k)) / (double)E;
    c = round_mode == 1 ? std::floor(v) : std::ceil(v);
  }
  if (c > (double)N) c = (double)N;
  if (c < 0.0) c = 0.0;
  *C = (int64_t)c;
  return 0;
}

// Device-level capacity n_l * gamma * N_bar = gamma * N k / D for a device holding n_l = E/D experts
// ("Advanced Variant" paragraph), evaluated as (gamma * (N*k)) / D in double, rounded like
// oracle_capacity, clamped to [0, N * E/D] (a device cannot hold more pairs than that).
int oracle_device_capacity(int64_t N, int E, int k, int D, double gamma, int round_mode, int64_t* C_dev) {
  if (N < 0 || E < 1 || k < 1 || k > E || D < 1 || E % D != 0 || !(gamma >= 0.0)) return 1;
  const double most = (double)N * (double)(E / D);
  double c;
  if (std::isinf(gamma)) c = most;
  else {
    double v = (gamma * (double)(N * (int64_t)k)) / (double)D;
    c = round_mode == 1 ? std::floor(v) : std::ceil(v);
  }
  if (c > most) c = most;
  if (c < 0.0) c = 0.0;
  *C_dev = (int64_t)c;
  return 0;
}

// Router logits l[t,e] = sum_j x[t,j] w[e,j] + b[e] (the gate of Eq. 1), accumulated in
// double, rounded once to binary32.
void oracle_router_logits(const void* x, const void* w, const float* bias, int64_t N, int d, int E,
                          int dtype, float* logits) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < N; ++t)
    for (int e = 0; e < E; ++e) {
      double acc = 0.0;
      for (int j = 0; j < d; ++j) acc += load_elem(x, t * d + j, dtype) * load_elem(w, (int64_t)e * d + j, dtype);
      if (bias) acc += (double)bias[e];
      logits[t * E + e] = (float)acc;
    }
}

// Row-wise softmax (Eq. 1) in binary32: m = max, p_e = exp_spec(l_e - m), S = p_0 + ... + p_{E-1}
// summed left to right, score_e = p_e / S.
void oracle_softmax(const float* logits, int64_t N, int E, float* scores) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < N; ++t) {
    const float* l = logits + t * E;
    float* s = scores + t * E;
    float mx = l[0];
    for (int e = 1; e < E; ++e) mx = l[e] > mx ? l[e] : mx;
    float sum = 0.0f;
    for (int e = 0; e < E; ++e) { s[e] = exp_spec(l[e] - mx); sum = sum + s[e]; }
    for (int e = 0; e < E; ++e) s[e] = s[e] / sum;
  }
}

// Per-token top-k of the scores (Eq. 1): the k largest, ordered by (score descending,
// expert id ascending); raw softmax values, not renormalised.  load[e] = N_e.
void oracle_topk(const float* scores, int64_t N, int E, int k, int32_t* topk_idx, float* topk_score,
                 int32_t* load) {
  for (int e = 0; e < E; ++e) load[e] = 0;
  std::vector<int32_t> ids(E);
  for (int64_t t = 0; t < N; ++t) {
    const float* s = scores + t * E;
    for (int e = 0; e < E; ++e) ids[e] = e;
    std::stable_sort(ids.begin(), ids.end(), [s](int32_t a, int32_t b) { return s[a] > s[b]; });
    for (int j = 0; j < k; ++j) {
      topk_idx[t * k + j] = ids[j];
      topk_score[t * k + j] = s[ids[j]];
      load[ids[j]] += 1;
    }
  }
}

// Token Drop (Eq. 7-10, Algorithm 1): expert e's candidates are the tokens whose top-k holds e;
// it keeps the min(N_e, C) best.  Outputs: keep_mask [N, ceil(E/64)] (bit e of token t),
// kept[E], offsets[E+1] (exclusive prefix of kept), slot_row[N,k] (row of the permuted
// matrix for top-k slot j of token t, or -1 when dropped).
void oracle_token_drop(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C,
                       uint64_t* keep_mask, int32_t* kept, int32_t* offsets, int32_t* slot_row) {
  std::vector<std::vector<Cand>> cands(E);
  for (int64_t t = 0; t < N; ++t)
    for (int j = 0; j < k; ++j) {
      int e = topk_idx[t * k + j];
      cands[e].push_back(Cand{scores[t * E + e], (int32_t)t, j});
    }
  select_and_place(cands, N, E, k, C, keep_mask, kept, offsets, slot_row);
}

// Expanded Drop (Algorithm 2): token t is a candidate of its top-k experts and of all m = E/D
// experts of its home group h(t); every candidate competes on score[t,e]; each expert keeps
// its min(|Cand_e|, C) best.  slot_row[N, k+m]: slots 0..k-1 follow the top-k order, slot
// k+i is local expert h(t)*m+i when that expert is not already one of the top-k.
void oracle_expanded_drop(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C,
                          int D, const int32_t* token_group, uint64_t* keep_mask, int32_t* cand,
                          int32_t* kept, int32_t* offsets, int32_t* slot_row) {
  const int m = E / D;
  std::vector<std::vector<Cand>> cands(E);
  std::vector<char> in_topk(E);
  for (int64_t t = 0; t < N; ++t) {
    std::fill(in_topk.begin(), in_topk.end(), 0);
    for (int j = 0; j < k; ++j) in_topk[topk_idx[t * k + j]] = 1;
    const int64_t g = home_group(t, N, D, token_group);
    // ascending expert id is irrelevant here (lists are per expert); visit top-k then locals
    for (int j = 0; j < k; ++j) {
      int e = topk_idx[t * k + j];
      cands[e].push_back(Cand{scores[t * E + e], (int32_t)t, j});
    }
    for (int i = 0; i < m; ++i) {
      int e = (int)g * m + i;
      if (!in_topk[e]) cands[e].push_back(Cand{scores[t * E + e], (int32_t)t, k + i});
    }
  }
  for (int e = 0; e < E; ++e) cand[e] = (int32_t)cands[e].size();
  select_and_place(cands, N, E, k + m, C, keep_mask, kept, offsets, slot_row);
}

// Drop metrics ("Order", "Reverse Order", "Random", "Score" in the Token Drop paragraph).  Each
// (token, expert) entry gets a 32-bit key; the drop keeps the entries with the largest keys, equal
// keys going to the lower token index.
//   metric 0  Score          key = bit pattern of the score (non-negative floats order like their bits)
//   metric 1  Order          one constant key: everything ties, so earlier tokens fill the capacity
//   metric 2  Reverse Order  key = token index: later tokens win, earlier ones are removed
//   metric 3  Random         key = high word of a 64-bit mix of (seed, t*E + e): every candidate
//                            has the same chance
// scores [N,cols]; idx [N,cols] expert ids, or null when cols == E and column c is expert c.
static inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

void oracle_drop_keys(int metric, uint64_t seed, const float* scores, const int32_t* idx, int64_t N, int cols,
                      int E, uint32_t* keys) {
  for (int64_t t = 0; t < N; ++t)
    for (int c = 0; c < cols; ++c) {
      const int64_t i = t * cols + c;
      const int e = idx ? idx[i] : c;
      uint32_t key;
      if (metric == 0) key = bits_from_f32(scores[i]);
      else if (metric == 1) key = 0x3f800000u;
      else if (metric == 2) key = (uint32_t)t;
      else key = (uint32_t)(mix64(seed + 0x9E3779B97F4A7C15ull * ((uint64_t)t * (uint64_t)E + (uint64_t)e + 1ull)) >> 32);
      keys[i] = key;
    }
}

// Token Drop / Expanded Drop on arbitrary 32-bit keys [N,E] (same candidate sets, capacity rule and
// output layout as oracle_token_drop / oracle_expanded_drop; expanded = 0 ignores D).
void oracle_drop_keyed(const uint32_t* keys, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C, int D,
                       int expanded, const int32_t* token_group, uint64_t* keep_mask, int32_t* cand, int32_t* kept,
                       int32_t* offsets, int32_t* slot_row) {
  const int m = expanded ? E / D : 0;
  const int slots = k + m;
  const int W = (E + 63) / 64;
  struct KC { uint32_t key; int32_t t; int32_t slot; };
  std::vector<std::vector<KC>> cands(E);
  std::vector<char> in_topk(E);
  for (int64_t t = 0; t < N; ++t) {
    std::fill(in_topk.begin(), in_topk.end(), 0);
    for (int j = 0; j < k; ++j) {
      const int e = topk_idx[t * k + j];
      in_topk[e] = 1;
      cands[e].push_back(KC{keys[t * E + e], (int32_t)t, j});
    }
    if (expanded) {
      const int64_t g = home_group(t, N, D, token_group);
      for (int i = 0; i < m; ++i) {
        const int e = (int)g * m + i;
        if (!in_topk[e]) cands[e].push_back(KC{keys[t * E + e], (int32_t)t, k + i});
      }
    }
  }
  for (int64_t i = 0; i < N * W; ++i) keep_mask[i] = 0;
  for (int64_t i = 0; i < N * slots; ++i) slot_row[i] = -1;
  offsets[0] = 0;
  for (int e = 0; e < E; ++e) {
    cand[e] = (int32_t)cands[e].size();
    std::vector<KC> order(cands[e]);
    std::stable_sort(order.begin(), order.end(), [](const KC& a, const KC& b) { return a.key > b.key; });
    const int64_t keep_n = std::min<int64_t>((int64_t)order.size(), C);
    std::vector<char> is_kept(N > 0 ? N : 1, 0);
    for (int64_t i = 0; i < keep_n; ++i) is_kept[order[i].t] = 1;
    kept[e] = (int32_t)keep_n;
    int32_t row = offsets[e];
    for (const KC& x : cands[e])
      if (is_kept[x.t]) {
        keep_mask[(int64_t)x.t * W + (e >> 6)] |= (uint64_t)1 << (e & 63);
        slot_row[(int64_t)x.t * slots + x.slot] = row++;
      }
    offsets[e + 1] = row;
  }
}

// Priority classes on top of a drop metric.  Two of the paper's variants rank candidates first by
// a class and only then by the metric:
//   * dropping by modality (multimodal section, "Image First" / "Text First"): every token of the
//     protected modality outranks every token of the other one, whatever their scores;
//   * Expanded Drop read as substitution only ("makes no change in the token assignments in experts
//     that are overflowed by the top-k"): a token's top-k pairs outrank the pairs it only has
//     through its home device, so the expansion can fill spare capacity but never displace.
// Class P = 2 * [pair (t,e) is one of t's top-k, when topk_idx is given] + [token_class[t] & 1, when
// token_class is given] goes into the two high bits of the key; the metric's key goes below it,
// unchanged when exact != 0 (it must then be below 2^30, as the bit pattern of every score in [0,1]
// is), else shifted right by two bits.  base/out [N,cols]; idx as in oracle_drop_keys.
// Returns 1 if an exact key does not fit.
int oracle_priority_keys(const uint32_t* base, const int32_t* idx, int64_t N, int cols, int E, int exact,
                         const uint8_t* token_class, const int32_t* topk_idx, int k, uint32_t* out) {
  (void)E;
  for (int64_t t = 0; t < N; ++t)
    for (int c = 0; c < cols; ++c) {
      const int64_t i = t * cols + c;
      const int e = idx ? idx[i] : c;
      uint32_t P = 0;
      if (topk_idx)
        for (int j = 0; j < k; ++j)
          if (topk_idx[t * k + j] == e) P = 2;
      if (token_class) P += token_class[t] & 1u;
      uint32_t body = base[i];
      if (exact) {
        if (body >= (1u << 30)) return 1;
      } else {
        body >>= 2;
      }
      out[i] = (P << 30) | body;
    }
  return 0;
}

// "w/ max" ablation of Expanded Drop (appendix "Maximum Number of Selected Experts"): after the
// drop a token may sit on more than k experts; with the constraint it retains only its k_max
// best by gating score (ties to the lower expert id).  One pass: capacity freed this way is not
// handed to anyone else.  keep_mask [N, ceil(E/64)] is edited in place.
void oracle_limit_experts(const float* scores, int64_t N, int E, int k_max, uint64_t* keep_mask) {
  const int W = (E + 63) / 64;
  std::vector<int> es;
  for (int64_t t = 0; t < N; ++t) {
    es.clear();
    for (int e = 0; e < E; ++e)
      if ((keep_mask[t * W + (e >> 6)] >> (e & 63)) & 1u) es.push_back(e);
    if ((int)es.size() <= k_max) continue;
    std::stable_sort(es.begin(), es.end(), [&](int a, int b) { return scores[t * E + a] > scores[t * E + b]; });
    for (size_t i = (size_t)k_max; i < es.size(); ++i)
      keep_mask[t * W + (es[i] >> 6)] &= ~((uint64_t)1 << (es[i] & 63));
  }
}

// Counts, offsets and rows of a given keep mask, in the layout the drop stages produce: segment e
// holds the tokens with bit e set in ascending token order; slot_row [N,slots] maps a token's
// slots (top-k order, then the m = E/D home-device experts when slots = k + m) to rows, -1 where
// the bit is clear.  A set bit whose expert is none of the token's slots is an error (returns 1).
int oracle_rows_from_mask(const uint64_t* keep_mask, const int32_t* topk_idx, int64_t N, int E, int k, int slots,
                          int D, const int32_t* token_group, int32_t* kept, int32_t* offsets, int32_t* slot_row) {
  const int W = (E + 63) / 64;
  const int m = slots > k ? E / D : 0;
  std::vector<int32_t> next(E);
  for (int e = 0; e < E; ++e) kept[e] = 0;
  for (int64_t t = 0; t < N; ++t)
    for (int e = 0; e < E; ++e)
      if ((keep_mask[t * W + (e >> 6)] >> (e & 63)) & 1u) ++kept[e];
  offsets[0] = 0;
  for (int e = 0; e < E; ++e) { offsets[e + 1] = offsets[e] + kept[e]; next[e] = offsets[e]; }
  for (int64_t t = 0; t < N; ++t) {
    const int64_t g = m > 0 ? home_group(t, N, D, token_group) : 0;
    uint64_t seen[4] = {0, 0, 0, 0};
    for (int s = 0; s < slots; ++s) {
      const int e = s < k ? topk_idx[t * k + s] : (int)g * m + (s - k);
      const bool dup = (seen[e >> 6] >> (e & 63)) & 1u;       // a home-device expert that is also a top-k slot
      seen[e >> 6] |= (uint64_t)1 << (e & 63);
      const bool set = (keep_mask[t * W + (e >> 6)] >> (e & 63)) & 1u;
      slot_row[t * slots + s] = (set && !dup) ? -2 : -1;      // -2: row assigned below, in expert order
    }
    for (int e = 0; e < E; ++e)
      if (((keep_mask[t * W + (e >> 6)] >> (e & 63)) & 1u) && !((seen[e >> 6] >> (e & 63)) & 1u)) return 1;
  }
  // rows are handed out expert by expert in ascending token order
  for (int64_t t = 0; t < N; ++t) {
    const int64_t g = m > 0 ? home_group(t, N, D, token_group) : 0;
    for (int s = 0; s < slots; ++s)
      if (slot_row[t * slots + s] == -2) {
        const int e = s < k ? topk_idx[t * k + s] : (int)g * m + (s - k);
        slot_row[t * slots + s] = next[e]++;
      }
  }
  return 0;
}

// Device-level capacity ("Advanced Variant: Device-Level Capacity-Aware Inference"): the constraint
// is on the aggregated load of a device, N_1 + ... + N_{n_l} <= C_dev, not on each expert.  The
// candidates of device g are all (token, expert) pairs with the expert on g (top-k pairs, plus
// the home-device pairs when expanded != 0, as in Expanded Drop); the device keeps its
// min(|Cand_g|, C_dev) best pairs by score, equal scores going to the lower token index and,
// inside one token, to the lower expert id.  Rows stay expert-major, token-ascending.
void oracle_device_drop(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C_dev,
                        int D, int expanded, const int32_t* token_group, uint64_t* keep_mask, int32_t* cand,
                        int32_t* kept, int32_t* offsets, int32_t* slot_row) {
  const int m = E / D;
  const int slots = expanded ? k + m : k;
  const int W = (E + 63) / 64;
  struct Pair { float s; int32_t t; int32_t e; int32_t slot; };
  std::vector<std::vector<Pair>> dev(D);          // per device, ordered by (token, expert)
  std::vector<int32_t> slot_of(E);
  for (int e = 0; e < E; ++e) cand[e] = 0;
  for (int64_t t = 0; t < N; ++t) {
    std::fill(slot_of.begin(), slot_of.end(), -1);
    for (int j = 0; j < k; ++j) slot_of[topk_idx[t * k + j]] = j;
    if (expanded) {
      const int64_t g = home_group(t, N, D, token_group);
      for (int i = 0; i < m; ++i)
        if (slot_of[g * m + i] < 0) slot_of[g * m + i] = k + i;
    }
    for (int e = 0; e < E; ++e)                   // ascending expert id inside the token
      if (slot_of[e] >= 0) {
        dev[e / m].push_back(Pair{scores[t * E + e], (int32_t)t, e, slot_of[e]});
        cand[e] += 1;
      }
  }
  for (int64_t i = 0; i < N * W; ++i) keep_mask[i] = 0;
  for (int64_t i = 0; i < N * slots; ++i) slot_row[i] = -1;
  std::vector<std::vector<std::pair<int32_t, int32_t>>> rows(E);   // per expert: (token, slot) kept
  for (int g = 0; g < D; ++g) {
    std::vector<Pair> order(dev[g]);
    std::stable_sort(order.begin(), order.end(), [](const Pair& a, const Pair& b) { return a.s > b.s; });
    const int64_t keep_n = std::min<int64_t>((int64_t)order.size(), C_dev);
    for (int64_t i = 0; i < keep_n; ++i) {
      const Pair& p = order[i];
      keep_mask[(int64_t)p.t * W + (p.e >> 6)] |= (uint64_t)1 << (p.e & 63);
      rows[p.e].push_back({p.t, p.slot});
    }
  }
  offsets[0] = 0;
  for (int e = 0; e < E; ++e) {
    std::sort(rows[e].begin(), rows[e].end());    // ascending token index inside the segment
    kept[e] = (int32_t)rows[e].size();
    int32_t row = offsets[e];
    for (auto& ts : rows[e]) slot_row[(int64_t)ts.first * slots + ts.second] = row++;
    offsets[e + 1] = row;
  }
}

// Expert id served by slot s of token t (slots < k: top-k order; slots >= k: local experts).
static inline int slot_expert(const int32_t* topk_idx, int64_t t, int s, int k, int m, int64_t g) {
  return s < k ? topk_idx[t * k + s] : (int)g * m + (s - k);
}

// Permutation: row r of the expert-major matrix holds token perm_token[r] with gate weight
// perm_weight[r] = score[t,e]; x_perm[r] = x[t] (same storage dtype, a byte copy).
void oracle_permute(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype,
                    const float* scores, const int32_t* topk_idx, const int32_t* token_group,
                    const int32_t* slot_row, void* x_perm, int32_t* perm_token, float* perm_weight,
                    int32_t* perm_expert) {
  const int m = D > 0 ? E / D : 0;
  const size_t elt = dtype == DT_F32 ? 4 : 2;
  for (int64_t t = 0; t < N; ++t) {
    const int64_t g = D > 0 ? home_group(t, N, D, token_group) : 0;
    for (int s = 0; s < slots; ++s) {
      int32_t r = slot_row[t * slots + s];
      if (r < 0) continue;
      int e = slot_expert(topk_idx, t, s, k, m, g);
      perm_token[r] = (int32_t)t;
      perm_weight[r] = scores[t * E + e];
      if (perm_expert) perm_expert[r] = e;
      if (x_perm) std::memcpy((char*)x_perm + (size_t)r * d * elt, (const char*)x + (size_t)t * d * elt, d * elt);
    }
  }
}

// SwiGLU expert on R rows: y = W_d ( silu(W_g x) * (W_u x) ), silu(g) = g / (1 + exp(-g)).
// row_expert[r] picks the expert; weights [E,F,d], [E,F,d], [E,d,F] in the storage dtype;
// everything in double, no intermediate rounding.
void oracle_expert_ffn(const void* x_rows, const int32_t* row_expert, int64_t R, int d, int F, int dtype,
                       const void* w_gate, const void* w_up, const void* w_down, double* y) {
#pragma omp parallel
  {
    std::vector<double> xr(d), h(F);
#pragma omp for schedule(dynamic, 1)
    for (int64_t r = 0; r < R; ++r) {
      const int64_t e = row_expert ? row_expert[r] : 0;
      for (int j = 0; j < d; ++j) xr[j] = load_elem(x_rows, r * d + j, dtype);
      for (int f = 0; f < F; ++f) {
        double g = 0.0, u = 0.0;
        const int64_t base = (e * F + f) * (int64_t)d;
        for (int j = 0; j < d; ++j) {
          g += load_elem(w_gate, base + j, dtype) * xr[j];
          u += load_elem(w_up, base + j, dtype) * xr[j];
        }
        h[f] = g / (1.0 + std::exp(-g)) * u;
      }
      for (int j = 0; j < d; ++j) {
        double acc = 0.0;
        const int64_t base = (e * d + j) * (int64_t)F;
        for (int f = 0; f < F; ++f) acc += load_elem(w_down, base + f, dtype) * h[f];
        y[r * d + j] = acc;
      }
    }
  }
}

// Combine (Eq. 2): y_t = sum over kept (t,e) of score[t,e] * y_perm[row(t,e)] (+ y_shared[t] with
// weight 1); zero when nothing is kept.  Double throughout.
void oracle_combine(const double* y_perm, const int32_t* slot_row, const float* scores,
                    const int32_t* topk_idx, const int32_t* token_group, int64_t N, int d, int E, int k,
                    int slots, int D, const double* y_shared, double* y) {
  const int m = D > 0 ? E / D : 0;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < N; ++t) {
    const int64_t g = D > 0 ? home_group(t, N, D, token_group) : 0;
    for (int j = 0; j < d; ++j) y[t * d + j] = y_shared ? y_shared[t * d + j] : 0.0;
    for (int s = 0; s < slots; ++s) {
      int32_t r = slot_row[t * slots + s];
      if (r < 0) continue;
      int e = slot_expert(topk_idx, t, s, k, m, g);
      double wgt = (double)scores[t * E + e];
      for (int j = 0; j < d; ++j) y[t * d + j] += wgt * y_perm[(int64_t)r * d + j];
    }
  }
}

// Layer output for a chosen list of tokens (used where the whole layer is too slow on a CPU):
// for each listed token, run the experts it kept and combine.  out [n_tok, d] double.
void oracle_layer_tokens(const void* x, const int32_t* tokens, int64_t n_tok, int64_t N, int d, int E, int k,
                         int slots, int D, int F, int dtype, const float* scores, const int32_t* topk_idx,
                         const int32_t* token_group, const int32_t* slot_row, const void* w_gate,
                         const void* w_up, const void* w_down, double* out) {
  const int m = D > 0 ? E / D : 0;
  const size_t elt = dtype == DT_F32 ? 4 : 2;
  std::vector<int32_t> row_tok, row_exp;
  std::vector<double> row_w;
  for (int64_t i = 0; i < n_tok; ++i) {
    int64_t t = tokens[i];
    const int64_t g = D > 0 ? home_group(t, N, D, token_group) : 0;
    for (int s = 0; s < slots; ++s) {
      if (slot_row[t * slots + s] < 0) continue;
      int e = slot_expert(topk_idx, t, s, k, m, g);
      row_tok.push_back((int32_t)i); row_exp.push_back(e); row_w.push_back((double)scores[t * E + e]);
    }
  }
  const int64_t R = (int64_t)row_tok.size();
  std::vector<char> rows((size_t)std::max<int64_t>(R, 1) * d * elt);
  for (int64_t r = 0; r < R; ++r)
    std::memcpy(rows.data() + (size_t)r * d * elt, (const char*)x + (size_t)tokens[row_tok[r]] * d * elt, d * elt);
  std::vector<double> yr((size_t)std::max<int64_t>(R, 1) * d);
  oracle_expert_ffn(rows.data(), row_exp.data(), R, d, F, dtype, w_gate, w_up, w_down, yr.data());
  for (int64_t i = 0; i < n_tok * d; ++i) out[i] = 0.0;
  for (int64_t r = 0; r < R; ++r)
    for (int j = 0; j < d; ++j) out[(int64_t)row_tok[r] * d + j] += row_w[r] * yr[r * d + j];
}

// Workload statistics: max load / N_bar (Eq. 3, 5) and the dropped fraction
// DT = sum_e relu(N_e - C) / sum_e N_e (Eq. 11).  stats[0] = max N_e / N_bar, stats[1] = DT,
// stats[2] = max N_e, stats[3] = sum_e N_e.
void oracle_stats(const int32_t* load, int E, int64_t N, int k, int64_t C, double* stats) {
  double nbar = (double)N * k / E, mx = 0, tot = 0, drop = 0;
  for (int e = 0; e < E; ++e) {
    mx = std::max(mx, (double)load[e]);
    tot += load[e];
    drop += std::max<double>((double)load[e] - (double)C, 0.0);
  }
  stats[0] = nbar > 0 ? mx / nbar : 0.0;
  stats[1] = tot > 0 ? drop / tot : 0.0;
  stats[2] = mx;
  stats[3] = tot;
}

}  // extern "C"
