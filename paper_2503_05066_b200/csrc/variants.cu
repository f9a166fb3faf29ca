// Variants of the drop stages: priority classes on top of a drop metric (modality-first dropping
// of the multimodal section; Expanded Drop read as substitution only), the "w/ max" limit on
// experts per token (appendix "Maximum Number of Selected Experts"), and the rebuild of counts,
// offsets and rows from an edited keep mask.
#include "common.cuh"

namespace capmoe {
namespace {

constexpr int VT = 256;              // threads per CTA = tokens per chunk
constexpr int MAX_W = 4;             // mask words per token (E <= 256)

__global__ void __launch_bounds__(VT)
k_priority_keys(const uint32_t* __restrict__ base, const int32_t* __restrict__ idx, int64_t total, int cols, int exact,
                const uint8_t* __restrict__ token_class, const int32_t* __restrict__ topk_idx, int k,
                uint32_t* __restrict__ keys) {
  const int64_t i = (int64_t)blockIdx.x * VT + threadIdx.x;
  if (i >= total) return;
  const int64_t t = i / cols;
  const int c = (int)(i - t * cols);
  const int e = idx ? idx[i] : c;
  uint32_t P = 0;
  if (topk_idx)
    for (int j = 0; j < k; ++j)
      if (topk_idx[t * k + j] == e) P = 2;
  if (token_class) P += token_class[t] & 1u;
  const uint32_t b = base[i];
  keys[i] = (P << 30) | (exact ? (b & 0x3fffffffu) : (b >> 2));
}

// One thread per token: if more than k_max bits are set, keep the k_max with the highest score
// (ties to the lower expert id) by k_max rounds of arg-max over the set bits.
__global__ void __launch_bounds__(VT)
k_limit_experts(const float* __restrict__ scores, int64_t N, int E, int W, int k_max,
                unsigned long long* __restrict__ keep_mask) {
  const int64_t t = (int64_t)blockIdx.x * VT + threadIdx.x;
  if (t >= N) return;
  unsigned long long left[MAX_W], out[MAX_W];
  int n = 0;
#pragma unroll
  for (int w = 0; w < MAX_W; ++w) {
    left[w] = w < W ? keep_mask[t * W + w] : 0ull;
    out[w] = 0ull;
    n += __popcll(left[w]);
  }
  if (n <= k_max) return;
  const float* srow = scores + t * E;
  for (int j = 0; j < k_max; ++j) {
    float best = -1.f;
    int be = -1;
#pragma unroll
    for (int w = 0; w < MAX_W; ++w) {
      unsigned long long bits = left[w];
      while (bits) {                                     // ascending expert id: strict '>' keeps the lower id
        const int b = __ffsll((long long)bits) - 1;
        bits &= bits - 1;
        const float s = srow[w * 64 + b];
        if (s > best) { best = s; be = w * 64 + b; }
      }
    }
    if (be < 0) break;
#pragma unroll
    for (int w = 0; w < MAX_W; ++w)
      if (w == (be >> 6)) {
        left[w] &= ~(1ull << (be & 63));
        out[w] |= 1ull << (be & 63);
      }
  }
#pragma unroll
  for (int w = 0; w < MAX_W; ++w)
    if (w < W) keep_mask[t * W + w] = out[w];
}

// ---------------------------------------------------------------- rows from a keep mask
// Chunk = VT consecutive tokens = one CTA.  Per expert the set bits of a chunk are counted with
// warp ballots; a scan over the chunks gives each chunk's first row inside the expert's segment;
// the placing pass repeats the ballots and turns (chunk base, warps before, lanes before) into the
// row, which keeps every segment in ascending token order without atomics.
__global__ void __launch_bounds__(VT)
k_mask_count(const unsigned long long* __restrict__ keep_mask, int64_t N, int E, int W,
             int32_t* __restrict__ chunk_cnt /*[chunks][E]*/) {
  extern __shared__ int wcnt[];                          // [VT/32][E]
  const int64_t t = (int64_t)blockIdx.x * VT + threadIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned long long m[MAX_W];
#pragma unroll
  for (int w = 0; w < MAX_W; ++w) m[w] = (w < W && t < N) ? keep_mask[t * W + w] : 0ull;
#pragma unroll
  for (int w = 0; w < MAX_W; ++w) {                      // static word index: the mask stays in registers
    const int ne = min(64, E - w * 64);
    for (int i = 0; i < ne; ++i) {
      const unsigned b = __ballot_sync(0xffffffffu, (m[w] >> i) & 1ull);
      if (lane == 0) wcnt[warp * E + w * 64 + i] = __popc(b);
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += VT) {
    int s = 0;
    for (int w = 0; w < VT / 32; ++w) s += wcnt[w * E + e];
    chunk_cnt[(int64_t)blockIdx.x * E + e] = s;
  }
}

// One CTA, thread e walks expert e's chunk counts in order (exclusive prefix in place), then the
// experts' totals are scanned into the segment offsets.
__global__ void __launch_bounds__(256)
k_mask_scan(int32_t* __restrict__ chunk_cnt, int64_t chunks, int E, int32_t* __restrict__ kept,
            int32_t* __restrict__ expert_offsets) {
  __shared__ int tot[256];
  const int e = threadIdx.x;
  int run = 0;
  if (e < E) {
    for (int64_t c = 0; c < chunks; ++c) {
      const int v = chunk_cnt[c * E + e];
      chunk_cnt[c * E + e] = run;
      run += v;
    }
    kept[e] = run;
  }
  tot[e] = e < E ? run : 0;
  __syncthreads();
  if (e == 0) {
    int acc = 0;
    for (int i = 0; i < E; ++i) { expert_offsets[i] = acc; acc += tot[i]; }
    expert_offsets[E] = acc;
  }
}

__global__ void __launch_bounds__(VT)
k_mask_place(const unsigned long long* __restrict__ keep_mask, const int32_t* __restrict__ topk_idx, int64_t N, int E,
             int W, int k, int slots, int D, const int32_t* __restrict__ token_group,
             const int32_t* __restrict__ chunk_base, const int32_t* __restrict__ expert_offsets,
             int32_t* __restrict__ slot_row, int32_t* __restrict__ bad) {
  extern __shared__ int wcnt[];                          // [VT/32][E]
  const int64_t t = (int64_t)blockIdx.x * VT + threadIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool live = t < N;
  const int m_loc = slots > k ? E / D : 0;
  unsigned long long m[MAX_W];
#pragma unroll
  for (int w = 0; w < MAX_W; ++w) m[w] = (w < W && live) ? keep_mask[t * W + w] : 0ull;
#pragma unroll
  for (int w = 0; w < MAX_W; ++w) {                      // static word index: the mask stays in registers
    const int ne = min(64, E - w * 64);
    for (int i = 0; i < ne; ++i) {
      const unsigned b = __ballot_sync(0xffffffffu, (m[w] >> i) & 1ull);
      if (lane == 0) wcnt[warp * E + w * 64 + i] = __popc(b);
    }
  }
  if (live)
    for (int s = 0; s < slots; ++s) slot_row[t * slots + s] = -1;
  __syncthreads();
  const int g = (live && m_loc > 0) ? home_group(t, N, D, token_group) : 0;
#pragma unroll
  for (int w = 0; w < MAX_W; ++w) {
    const int ne = min(64, E - w * 64);
    for (int i = 0; i < ne; ++i) {
      const int e = w * 64 + i;
      const bool set = (m[w] >> i) & 1ull;
      const unsigned b = __ballot_sync(0xffffffffu, set);
      if (!set) continue;
      int before = __popc(b & ((1u << lane) - 1u));
      for (int w2 = 0; w2 < warp; ++w2) before += wcnt[w2 * E + e];
      const int row = expert_offsets[e] + chunk_base[(int64_t)blockIdx.x * E + e] + before;
      // the slot that serves expert e: its place among the top-k, else its place on the home device
      int slot = -1;
      for (int j = 0; j < k; ++j)
        if (topk_idx[t * k + j] == e) { slot = j; break; }
      if (slot < 0 && m_loc > 0 && e >= g * m_loc && e < (g + 1) * m_loc) slot = k + (e - g * m_loc);
      if (slot >= 0) slot_row[t * slots + slot] = row;
      else atomicExch(bad, 1);                           // a bit outside the token's slots
    }
  }
}

}  // namespace
}  // namespace capmoe

using namespace capmoe;

extern "C" int capmoe_priority_keys(const uint32_t* base, const int32_t* idx, int64_t N, int cols, int E, int exact,
                                    const uint8_t* token_class, const int32_t* topk_idx, int k, uint32_t* keys,
                                    void* stream) {
  if (N < 0 || cols < 1 || E < 1 || (!idx && cols != E) || (topk_idx && (k < 1 || k > E))) return CAPMOE_EINVAL;
  if (N == 0) return CAPMOE_OK;
  if (!base || !keys) return CAPMOE_EINVAL;
  const int64_t total = N * cols;
  if (total >= ((int64_t)1 << 38)) return CAPMOE_EUNSUPPORTED;
  k_priority_keys<<<(unsigned)ceil_div(total, VT), VT, 0, as_stream(stream)>>>(base, idx, total, cols, exact,
                                                                              token_class, topk_idx, k, keys);
  return check_launch();
}

extern "C" int capmoe_limit_experts(const float* scores, int64_t N, int E, int k_max, uint64_t* keep_mask,
                                    void* stream) {
  if (N < 0 || E < 1 || k_max < 0) return CAPMOE_EINVAL;
  if (E > 64 * MAX_W) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return CAPMOE_OK;
  if (!scores || !keep_mask) return CAPMOE_EINVAL;
  k_limit_experts<<<(unsigned)ceil_div(N, VT), VT, 0, as_stream(stream)>>>(
      scores, N, E, (E + 63) / 64, k_max, reinterpret_cast<unsigned long long*>(keep_mask));
  return check_launch();
}

extern "C" int capmoe_rows_from_mask(const uint64_t* keep_mask, const int32_t* topk_idx, int64_t N, int E, int k,
                                     int slots, int D, const int32_t* token_group, int32_t* kept,
                                     int32_t* expert_offsets, int32_t* slot_row, int32_t* bad, void* ws,
                                     size_t ws_bytes, void* stream) {
  if (N < 0 || E < 1 || k < 1 || k > E || D < 1 || E % D != 0) return CAPMOE_EINVAL;
  if (slots != k && slots != k + E / D) return CAPMOE_EINVAL;
  if (E > 64 * MAX_W) return CAPMOE_EUNSUPPORTED;
  if (!kept || !expert_offsets) return CAPMOE_EINVAL;
  cudaStream_t st = as_stream(stream);
  if (N == 0) {
    cudaError_t err = cudaMemsetAsync(kept, 0, sizeof(int32_t) * E, st);
    if (err == cudaSuccess) err = cudaMemsetAsync(expert_offsets, 0, sizeof(int32_t) * (E + 1), st);
    return note_cuda(err);
  }
  if (!keep_mask || !topk_idx || !slot_row || !bad || !ws) return CAPMOE_EINVAL;
  const int64_t chunks = ceil_div(N, VT);
  if (ws_bytes < sizeof(int32_t) * (size_t)chunks * E) return CAPMOE_EWORKSPACE;
  cudaError_t err = cudaMemsetAsync(bad, 0, sizeof(int32_t), st);
  if (err != cudaSuccess) return note_cuda(err);
  int32_t* chunk_cnt = reinterpret_cast<int32_t*>(ws);
  const unsigned long long* km = reinterpret_cast<const unsigned long long*>(keep_mask);
  const int W = (E + 63) / 64;
  const size_t smem = sizeof(int) * (VT / 32) * E;
  k_mask_count<<<(unsigned)chunks, VT, smem, st>>>(km, N, E, W, chunk_cnt);
  int rc = check_launch();
  if (rc != CAPMOE_OK) return rc;
  k_mask_scan<<<1, 256, 0, st>>>(chunk_cnt, chunks, E, kept, expert_offsets);
  if ((rc = check_launch()) != CAPMOE_OK) return rc;
  k_mask_place<<<(unsigned)chunks, VT, smem, st>>>(km, topk_idx, N, E, W, k, slots, D, token_group, chunk_cnt,
                                                   expert_offsets, slot_row, bad);
  return check_launch();
}
