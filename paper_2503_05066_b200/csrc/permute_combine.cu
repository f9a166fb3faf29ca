// Stage 4 (permute: gather kept tokens into expert-major rows) and stage 6 (combine: the
// gate-weighted sum of Eq. 2 back in token order).  Pure data movement, bound by HBM.
// Work unit = (token, 2 KB chunk of its row): one warp per unit, four 16-byte vectors per lane,
// so that the number of units (N * row bytes / 2 KB) is many times the number of resident warps
// and the last wave stays full.  Each x row is read once and written to every row that keeps it.
#include "common.cuh"

namespace capmoe {
namespace {

constexpr int PC_WARPS = 8;          // warps (work units) per CTA
constexpr int VPL = 4;               // 16-byte vectors per lane per unit
constexpr int CHUNK_VECS = 32 * VPL; // vectors per unit (2 KB)
constexpr int MAX_SLOTS = 288;       // k + m <= 32 + 256

// Where a row of the permuted matrix lives when the matrix is spread over the ranks of an
// expert-parallel group: rows [p*rows_per_peer, (p+1)*rows_per_peer) belong to rank p and sit in
// that rank's buffer (base address table[p]) from row `row0` on, the block this rank owns there.
// table == NULL: one local matrix.
struct PeerRows {
  const unsigned long long* table;
  int rows_per_peer, row0;
};
__device__ __forceinline__ uint4* peer_row(const PeerRows& pr, uint4* local_base, int32_t r, int row_vecs) {
  if (!pr.table) return local_base + (int64_t)r * row_vecs;
  const int p = r / pr.rows_per_peer, i = r - p * pr.rows_per_peer;
  return reinterpret_cast<uint4*>(pr.table[p]) + (int64_t)(pr.row0 + i) * row_vecs;
}

__global__ void __launch_bounds__(PC_WARPS * 32)
k_permute(const uint4* __restrict__ x, int64_t N, int row_vecs /* 16-byte vectors per row */, int chunks, int E,
          int k, int slots, int D, const float* __restrict__ scores, const int32_t* __restrict__ topk_idx,
          const int32_t* __restrict__ token_group, const int32_t* __restrict__ slot_row,
          uint4* __restrict__ x_perm, int32_t* __restrict__ perm_token, float* __restrict__ perm_weight,
          unsigned long long* __restrict__ keep_mask /* NULL, or [N, ceil(E/64)] to be derived from slot_row here */,
          const PeerRows peers) {
  allow_next_kernel();
  wait_for_previous_kernel();
  const int lane = threadIdx.x & 31;
  const int64_t unit = (int64_t)blockIdx.x * PC_WARPS + (threadIdx.x >> 5);
  const int64_t t = unit / chunks;
  const int chunk = (int)(unit - t * chunks);
  if (t >= N) return;
  const int32_t* sr = slot_row + t * slots;
  if (chunk == 0) {                                    // bookkeeping once per token: lane s handles slot s, s+32, ...
    const int m = D > 0 ? E / D : 0;
    const int g = D > 0 ? home_group(t, N, D, token_group) : 0;
    uint32_t bits[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};          // this lane's share of the token's keep mask (E <= 256)
    for (int s = lane; s < slots; s += 32) {
      const int32_t r = sr[s];
      if (r >= 0) {
        const int e = s < k ? topk_idx[t * k + s] : g * m + (s - k);
        perm_token[r] = (int32_t)t;
        perm_weight[r] = scores[t * E + e];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (i == (e >> 5)) bits[i] |= 1u << (e & 31);
      }
    }
    if (keep_mask) {                                   // bit e set iff the slot that stands for expert e holds a row
      const int W = (E + 63) >> 6;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (i < W) {
          const uint32_t lo32 = __reduce_or_sync(0xffffffffu, bits[2 * i]);
          const uint32_t hi32 = __reduce_or_sync(0xffffffffu, bits[2 * i + 1]);
          if (lane == 0) keep_mask[t * W + i] = ((unsigned long long)hi32 << 32) | lo32;
        }
    }
  }
  const int v0 = chunk * CHUNK_VECS + lane;
  const uint4* src = x + t * row_vecs + v0;
  uint4 val[VPL];
  bool loaded = false;
  for (int s0 = 0; s0 < slots; s0 += 32) {
    const int32_t mine = (s0 + lane < slots) ? sr[s0 + lane] : -1;
    unsigned rem = __ballot_sync(0xffffffffu, mine >= 0);
    if (!rem) continue;
    if (!loaded) {                                     // a token nobody keeps is never read
#pragma unroll
      for (int u = 0; u < VPL; ++u)
        val[u] = (v0 + u * 32 < row_vecs) ? __ldcs(src + u * 32) : make_uint4(0u, 0u, 0u, 0u);
      loaded = true;
    }
    while (rem) {
      const int b = __ffs(rem) - 1;
      rem &= rem - 1;
      const int32_t r = __shfl_sync(0xffffffffu, mine, b);
      uint4* dst = peer_row(peers, x_perm, r, row_vecs) + v0;
#pragma unroll
      for (int u = 0; u < VPL; ++u)
        if (v0 + u * 32 < row_vecs) dst[u * 32] = val[u];
    }
  }
}

template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int n = 4;
  static __device__ __forceinline__ void load(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  static __device__ __forceinline__ uint4 store(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int n = 8;
  static __device__ __forceinline__ void load(const uint4& v, float* f) {
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ uint4 store(const float* f) {
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<unsigned*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// acc[u] += wgt * row[u] for the VPL vectors of one kept row
template <typename T>
__device__ __forceinline__ void axpy_row(float (*acc)[Vec16<T>::n], const uint4* raw, float wgt) {
#pragma unroll
  for (int u = 0; u < VPL; ++u) {
    float f[Vec16<T>::n];
    Vec16<T>::load(raw[u], f);
#pragma unroll
    for (int i = 0; i < Vec16<T>::n; ++i) acc[u][i] = fmaf(wgt, f[i], acc[u][i]);
  }
}

template <typename T>
__global__ void __launch_bounds__(PC_WARPS * 32, 4)
k_combine(const uint4* __restrict__ y_perm, const int32_t* __restrict__ slot_row,
          const float* __restrict__ perm_weight, int64_t N, int row_vecs, int chunks, int slots,
          const uint4* __restrict__ y_shared, uint4* __restrict__ y, const PeerRows peers) {
  allow_next_kernel();
  wait_for_previous_kernel();
  constexpr int NV = Vec16<T>::n;
  const int lane = threadIdx.x & 31;
  const int64_t unit = (int64_t)blockIdx.x * PC_WARPS + (threadIdx.x >> 5);
  const int64_t t = unit / chunks;
  const int chunk = (int)(unit - t * chunks);
  if (t >= N) return;
  const int32_t* sr = slot_row + t * slots;
  const int v0 = chunk * CHUNK_VECS + lane;
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  float acc[VPL][NV];
#pragma unroll
  for (int u = 0; u < VPL; ++u) {
#pragma unroll
    for (int i = 0; i < NV; ++i) acc[u][i] = 0.f;
    if (y_shared && v0 + u * 32 < row_vecs) Vec16<T>::load(__ldcs(y_shared + t * row_vecs + v0 + u * 32), acc[u]);
  }
  for (int s0 = 0; s0 < slots; s0 += 32) {
    const int32_t mine = (s0 + lane < slots) ? sr[s0 + lane] : -1;
    const float wmine = mine >= 0 ? perm_weight[mine] : 0.f;
    unsigned rem = __ballot_sync(0xffffffffu, mine >= 0);
    while (rem) {                                      // ascending slot order, two kept rows per round
      const int b0 = __ffs(rem) - 1;
      rem &= rem - 1;
      const bool two = rem != 0;
      const int b1 = two ? __ffs(rem) - 1 : b0;
      rem &= rem - 1;                                  // no-op when rem is already 0
      const int32_t r0 = __shfl_sync(0xffffffffu, mine, b0), r1 = __shfl_sync(0xffffffffu, mine, b1);
      const float w0 = __shfl_sync(0xffffffffu, wmine, b0), w1 = __shfl_sync(0xffffffffu, wmine, b1);
      const uint4* p0 = peer_row(peers, const_cast<uint4*>(y_perm), r0, row_vecs) + v0;
      const uint4* p1 = peer_row(peers, const_cast<uint4*>(y_perm), r1, row_vecs) + v0;
      uint4 raw0[VPL], raw1[VPL];
#pragma unroll
      for (int u = 0; u < VPL; ++u) {                  // all loads first, arithmetic after
        const bool in = v0 + u * 32 < row_vecs;
        raw0[u] = in ? __ldcs(p0 + u * 32) : zero;
        raw1[u] = (in && two) ? __ldcs(p1 + u * 32) : zero;
      }
      axpy_row<T>(acc, raw0, w0);
      if (two) axpy_row<T>(acc, raw1, w1);
    }
  }
#pragma unroll
  for (int u = 0; u < VPL; ++u)
    if (v0 + u * 32 < row_vecs) y[t * row_vecs + v0 + u * 32] = Vec16<T>::store(acc[u]);
}

}  // namespace
}  // namespace capmoe

using namespace capmoe;

namespace capmoe {
namespace {
int permute_rows(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype, const float* scores,
                 const int32_t* topk_idx, const int32_t* token_group, const int32_t* slot_row, void* x_perm,
                 int32_t* perm_token, float* perm_weight, uint64_t* keep_mask_out, const PeerRows& peers, void* stream) {
  if (N < 0 || d < 1 || E < 1 || k < 1 || k > E || slots < k || D < 0) return CAPMOE_EINVAL;
  if (dtype != CAPMOE_F32 && dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (D > 0 && (E % D != 0 || slots != k + E / D)) return CAPMOE_EINVAL;
  if (D == 0 && slots != k) return CAPMOE_EINVAL;
  if (slots > MAX_SLOTS) return CAPMOE_EUNSUPPORTED;
  if (((size_t)d * elt_size(dtype)) % 16 != 0) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return CAPMOE_OK;
  if (!x || !scores || !topk_idx || !slot_row || (!x_perm && !peers.table) || !perm_token || !perm_weight)
    return CAPMOE_EINVAL;
  if (!aligned16(x) || !aligned16(x_perm)) return CAPMOE_EINVAL;
  const int row_vecs = (int)((size_t)d * elt_size(dtype) / 16);
  const int chunks = (row_vecs + CHUNK_VECS - 1) / CHUNK_VECS;
  const int64_t blocks = ceil_div(N * chunks, PC_WARPS);
  if (blocks > 0x7fffffff) return CAPMOE_EUNSUPPORTED;
  const int rc = note_cuda(launch_chained(k_permute, (unsigned)blocks, PC_WARPS * 32, 0, as_stream(stream),
                                          (const uint4*)x, N, row_vecs, chunks, E, k, slots, D, scores, topk_idx,
                                          token_group, slot_row, (uint4*)x_perm, perm_token, perm_weight,
                                          reinterpret_cast<unsigned long long*>(keep_mask_out), peers));
  count_launch(1);
  return rc;
}

int combine_rows(const void* y_perm, const int32_t* slot_row, const float* perm_weight, int64_t N, int d, int slots,
                 int dtype, const void* y_shared, void* y, const PeerRows& peers, void* stream) {
  if (N < 0 || d < 1 || slots < 1) return CAPMOE_EINVAL;
  if (dtype != CAPMOE_F32 && dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (slots > MAX_SLOTS) return CAPMOE_EUNSUPPORTED;
  if (((size_t)d * elt_size(dtype)) % 16 != 0) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return CAPMOE_OK;
  if (!slot_row || !y) return CAPMOE_EINVAL;       // y_perm / perm_weight may be NULL only if A == 0
  if (!aligned16(y_perm) || !aligned16(y) || !aligned16(y_shared)) return CAPMOE_EINVAL;
  const int row_vecs = (int)((size_t)d * elt_size(dtype) / 16);
  const int chunks = (row_vecs + CHUNK_VECS - 1) / CHUNK_VECS;
  const int64_t blocks = ceil_div(N * chunks, PC_WARPS);
  if (blocks > 0x7fffffff) return CAPMOE_EUNSUPPORTED;
  cudaStream_t st = as_stream(stream);
  cudaError_t err;
  if (dtype == CAPMOE_F32)
    err = launch_chained(k_combine<float>, (unsigned)blocks, PC_WARPS * 32, 0, st, (const uint4*)y_perm, slot_row,
                         perm_weight, N, row_vecs, chunks, slots, (const uint4*)y_shared, (uint4*)y, peers);
  else
    err = launch_chained(k_combine<__nv_bfloat16>, (unsigned)blocks, PC_WARPS * 32, 0, st, (const uint4*)y_perm,
                         slot_row, perm_weight, N, row_vecs, chunks, slots, (const uint4*)y_shared, (uint4*)y, peers);
  count_launch(1);
  return note_cuda(err);
}

// Expert parallelism, bookkeeping kernels (see capmoe_ep_plan / capmoe_ep_segments in the header).
__global__ void __launch_bounds__(256)
k_ep_plan(const int32_t* __restrict__ slot_row, const int32_t* __restrict__ topk_idx,
          const int32_t* __restrict__ expert_offsets, int64_t N, int E, int k, int slots, int D,
          const int32_t* __restrict__ token_group, int C_local, int32_t* __restrict__ slot_row_ep,
          int32_t* __restrict__ bad) {
  allow_next_kernel();
  wait_for_previous_kernel();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= N * slots) return;
  const int64_t t = i / slots;
  const int s = (int)(i - t * slots);
  const int32_t r = slot_row[i];
  int32_t out = -1;
  if (r >= 0) {
    const int m = slots > k ? E / D : 0;
    const int e = s < k ? topk_idx[t * k + s] : home_group(t, N, D, token_group) * m + (s - k);
    const int32_t within = r - expert_offsets[e];
    if (within < 0 || within >= C_local) *bad = 1;           // more rows on an expert than its capacity allows
    else out = e * C_local + within;
  }
  slot_row_ep[i] = out;
}

// Debug check: every index a later stage uses as an address lies where it should.  Reads only.
__global__ void __launch_bounds__(256)
k_check_indices(const int32_t* __restrict__ slot_row, const int32_t* __restrict__ topk_idx,
                const int32_t* __restrict__ expert_offsets, int64_t N, int E, int k, int slots, int D,
                const int32_t* __restrict__ token_group, int64_t A_max, int32_t* __restrict__ dev_status) {
  allow_next_kernel();
  wait_for_previous_kernel();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  bool bad = false;
  if (i <= E) {                                          // offsets: non-decreasing, inside the buffers
    const int64_t o = expert_offsets[i];
    bad = o < 0 || o > A_max || (i > 0 && o < expert_offsets[i - 1]);
  }
  if (i < N * slots) {
    const int64_t t = i / slots;
    const int s = (int)(i - t * slots);
    const int32_t r = slot_row[i];
    if (r != -1) {
      const int m = slots > k ? E / D : 0;
      const int e = s < k ? topk_idx[t * k + s] : home_group(t, N, D, token_group) * m + (s - k);
      bad = bad || e < 0 || e >= E || r < expert_offsets[e < 0 || e >= E ? 0 : e] ||
            r >= expert_offsets[e < 0 || e >= E ? 0 : e + 1];
    }
  }
  if (bad) atomicExch(dev_status, (int)CAPMOE_EINDEX);
}

__global__ void __launch_bounds__(256)
k_ep_segments(const int32_t* __restrict__ counts, int S, int C_local, int32_t* __restrict__ seg_begin,
              int32_t* __restrict__ seg_end) {
  allow_next_kernel();
  wait_for_previous_kernel();
  const int s = blockIdx.x * 256 + threadIdx.x;
  if (s >= S) return;
  const int c = counts[s];
  seg_begin[s] = s * C_local;
  seg_end[s] = s * C_local + (c < 0 ? 0 : (c > C_local ? C_local : c));
}

}  // namespace
}  // namespace capmoe

int capmoe::permute_impl(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype,
                         const float* scores, const int32_t* topk_idx, const int32_t* token_group,
                         const int32_t* slot_row, void* x_perm, int32_t* perm_token, float* perm_weight,
                         uint64_t* keep_mask_out, void* stream) {
  return permute_rows(x, N, d, E, k, slots, D, dtype, scores, topk_idx, token_group, slot_row, x_perm, perm_token,
                      perm_weight, keep_mask_out, PeerRows{nullptr, 0, 0}, stream);
}

extern "C" int capmoe_permute(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype,
                              const float* scores, const int32_t* topk_idx, const int32_t* token_group,
                              const int32_t* slot_row, void* x_perm, int32_t* perm_token, float* perm_weight,
                              void* stream) {
  return permute_impl(x, N, d, E, k, slots, D, dtype, scores, topk_idx, token_group, slot_row, x_perm, perm_token,
                      perm_weight, nullptr, stream);
}

extern "C" int capmoe_combine(const void* y_perm, const int32_t* slot_row, const float* perm_weight, int64_t N,
                              int d, int slots, int dtype, const void* y_shared, void* y, void* stream) {
  return combine_rows(y_perm, slot_row, perm_weight, N, d, slots, dtype, y_shared, y, PeerRows{nullptr, 0, 0}, stream);
}

// ---------------------------------------------------------------------------------------------
// Expert parallelism with per-rank capacity (entry points documented in capmoe.h).
namespace {
int check_ep(int R, int rank, int E, int64_t C_local) {
  if (R < 1 || rank < 0 || rank >= R || E < 1 || E % R != 0 || C_local < 0) return CAPMOE_EINVAL;
  if ((int64_t)E * C_local >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  return CAPMOE_OK;
}
}  // namespace

extern "C" int capmoe_ep_plan(const int32_t* slot_row, const int32_t* topk_idx, const int32_t* expert_offsets, int64_t N,
                              int E, int k, int slots, int D, const int32_t* token_group, int64_t C_local,
                              int32_t* slot_row_ep, int32_t* bad, void* stream) {
  if (N < 0 || E < 1 || k < 1 || k > E || slots < k || C_local < 0) return CAPMOE_EINVAL;
  if (slots > k && (D < 1 || E % D != 0 || slots != k + E / D)) return CAPMOE_EINVAL;
  if ((int64_t)E * C_local >= ((int64_t)1 << 31) || N * (int64_t)slots >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return CAPMOE_OK;
  if (!slot_row || !topk_idx || !expert_offsets || !slot_row_ep || !bad) return CAPMOE_EINVAL;
  const int rc = note_cuda(launch_chained(k_ep_plan, (unsigned)ceil_div(N * slots, 256), 256, 0, as_stream(stream),
                                          slot_row, topk_idx, expert_offsets, N, E, k, slots, D < 1 ? 1 : D, token_group,
                                          (int)C_local, slot_row_ep, bad));
  count_launch(1);
  return rc;
}

extern "C" int capmoe_debug_check_indices(const int32_t* slot_row, const int32_t* topk_idx, const int32_t* expert_offsets,
                                          int64_t N, int E, int k, int slots, int D, const int32_t* token_group,
                                          int64_t A_max, int32_t* dev_status, void* stream) {
  if (N < 0 || E < 1 || k < 1 || k > E || slots < k || A_max < 0) return CAPMOE_EINVAL;
  if (slots > k && (D < 1 || E % D != 0 || slots != k + E / D)) return CAPMOE_EINVAL;
  if (!expert_offsets || !dev_status || (N > 0 && (!slot_row || !topk_idx))) return CAPMOE_EINVAL;
  const int64_t items = N * slots > E + 1 ? N * slots : E + 1;
  if (items >= ((int64_t)1 << 38)) return CAPMOE_EUNSUPPORTED;
  const int rc = note_cuda(launch_chained(k_check_indices, (unsigned)ceil_div(items, 256), 256, 0, as_stream(stream),
                                          slot_row, topk_idx, expert_offsets, N, E, k, slots, D < 1 ? 1 : D, token_group,
                                          A_max, dev_status));
  count_launch(1);
  return rc;
}

extern "C" int capmoe_ep_segments(const int32_t* counts, int S, int64_t C_local, int32_t* seg_begin, int32_t* seg_end,
                                  void* stream) {
  if (S < 1 || C_local < 0 || (int64_t)S * C_local >= ((int64_t)1 << 31)) return CAPMOE_EINVAL;
  if (!counts || !seg_begin || !seg_end) return CAPMOE_EINVAL;
  const int rc = note_cuda(launch_chained(k_ep_segments, (unsigned)ceil_div(S, 256), 256, 0, as_stream(stream), counts, S,
                                          (int)C_local, seg_begin, seg_end));
  count_launch(1);
  return rc;
}

extern "C" int capmoe_ep_dispatch(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype,
                                  const float* scores, const int32_t* topk_idx, const int32_t* token_group,
                                  const int32_t* slot_row_ep, const uint64_t* peer_rows, int R, int rank,
                                  int64_t C_local, int32_t* perm_token, float* perm_weight, void* stream) {
  const int rc = check_ep(R, rank, E, C_local);
  if (rc != CAPMOE_OK) return rc;
  if (!peer_rows) return CAPMOE_EINVAL;
  const int per = (int)((E / R) * C_local);
  return permute_rows(x, N, d, E, k, slots, D, dtype, scores, topk_idx, token_group, slot_row_ep, nullptr, perm_token,
                      perm_weight, nullptr,
                      PeerRows{reinterpret_cast<const unsigned long long*>(peer_rows), per > 0 ? per : 1, rank * per},
                      stream);
}

extern "C" int capmoe_ep_combine(const uint64_t* peer_rows, int R, int rank, int E, int64_t C_local,
                                 const int32_t* slot_row_ep, const float* perm_weight, int64_t N, int d, int slots,
                                 int dtype, const void* y_shared, void* y, void* stream) {
  const int rc = check_ep(R, rank, E, C_local);
  if (rc != CAPMOE_OK) return rc;
  if (!peer_rows) return CAPMOE_EINVAL;
  const int per = (int)((E / R) * C_local);
  return combine_rows(nullptr, slot_row_ep, perm_weight, N, d, slots, dtype, y_shared, y,
                      PeerRows{reinterpret_cast<const unsigned long long*>(peer_rows), per > 0 ? per : 1, rank * per},
                      stream);
}
