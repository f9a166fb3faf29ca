// Stage 4 (permute: gather kept tokens into expert-major rows) and stage 6 (combine: the
// gate-weighted sum of Eq. 2 back in token order).  Pure data movement: one warp per token,
// 16-byte accesses, each x row read once and written to every row that keeps it.
#include "common.cuh"

namespace capmoe {
namespace {

constexpr int PC_WARPS = 8;          // warps (tokens) per CTA
constexpr int MAX_SLOTS = 288;       // k + m <= 32 + 256

__global__ void __launch_bounds__(PC_WARPS * 32)
k_permute(const uint4* __restrict__ x, int64_t N, int row_vecs /* 16-byte vectors per row */, int E, int k,
          int slots, int D, const float* __restrict__ scores, const int32_t* __restrict__ topk_idx,
          const int32_t* __restrict__ token_group, const int32_t* __restrict__ slot_row,
          uint4* __restrict__ x_perm, int32_t* __restrict__ perm_token, float* __restrict__ perm_weight) {
  const int lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * PC_WARPS + (threadIdx.x >> 5);
  if (t >= N) return;
  const int m = D > 0 ? E / D : 0;
  const int g = D > 0 ? home_group(t, N, D, token_group) : 0;
  const int32_t* sr = slot_row + t * slots;
  // bookkeeping: lane s handles slot s (+32, +64, ...)
  for (int s = lane; s < slots; s += 32) {
    const int32_t r = sr[s];
    if (r >= 0) {
      const int e = s < k ? topk_idx[t * k + s] : g * m + (s - k);
      perm_token[r] = (int32_t)t;
      perm_weight[r] = scores[t * E + e];
    }
  }
  const uint4* src = x + t * row_vecs;
  for (int s0 = 0; s0 < slots; s0 += 32) {
    const int32_t mine = (s0 + lane < slots) ? sr[s0 + lane] : -1;
    unsigned live = __ballot_sync(0xffffffffu, mine >= 0);
    if (!live) continue;
    for (int v = lane; v < row_vecs; v += 32) {
      const uint4 val = src[v];
      unsigned rem = live;
      while (rem) {
        const int b = __ffs(rem) - 1;
        rem &= rem - 1;
        const int32_t r = __shfl_sync(0xffffffffu, mine, b);
        x_perm[(int64_t)r * row_vecs + v] = val;
      }
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

template <typename T>
__global__ void __launch_bounds__(PC_WARPS * 32)
k_combine(const uint4* __restrict__ y_perm, const int32_t* __restrict__ slot_row,
          const float* __restrict__ perm_weight, int64_t N, int row_vecs, int slots,
          const uint4* __restrict__ y_shared, uint4* __restrict__ y) {
  constexpr int NV = Vec16<T>::n;
  const int lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * PC_WARPS + (threadIdx.x >> 5);
  if (t >= N) return;
  const int32_t* sr = slot_row + t * slots;
  constexpr int VPL = 4;                               // 16-byte vectors per lane in flight per row
  for (int v0 = 0; v0 < row_vecs; v0 += 32 * VPL) {
    float acc[VPL][NV];
#pragma unroll
    for (int u = 0; u < VPL; ++u) {
      const int v = v0 + u * 32 + lane;
#pragma unroll
      for (int i = 0; i < NV; ++i) acc[u][i] = 0.f;
      if (y_shared && v < row_vecs) Vec16<T>::load(y_shared[t * row_vecs + v], acc[u]);
    }
    for (int s0 = 0; s0 < slots; s0 += 32) {
      const int32_t mine = (s0 + lane < slots) ? sr[s0 + lane] : -1;
      const float wmine = mine >= 0 ? perm_weight[mine] : 0.f;
      unsigned rem = __ballot_sync(0xffffffffu, mine >= 0);
      while (rem) {                                    // ascending slot order
        const int b = __ffs(rem) - 1;
        rem &= rem - 1;
        const int32_t r = __shfl_sync(0xffffffffu, mine, b);
        const float wgt = __shfl_sync(0xffffffffu, wmine, b);
        const uint4* src = y_perm + (int64_t)r * row_vecs + v0 + lane;
        uint4 raw[VPL];
#pragma unroll
        for (int u = 0; u < VPL; ++u)                  // independent loads first, arithmetic after
          raw[u] = (v0 + u * 32 + lane < row_vecs) ? __ldcs(src + u * 32) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < VPL; ++u) {
          float f[NV];
          Vec16<T>::load(raw[u], f);
#pragma unroll
          for (int i = 0; i < NV; ++i) acc[u][i] = fmaf(wgt, f[i], acc[u][i]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < VPL; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < row_vecs) y[t * row_vecs + v] = Vec16<T>::store(acc[u]);
    }
  }
}

}  // namespace
}  // namespace capmoe

using namespace capmoe;

extern "C" int capmoe_permute(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype,
                              const float* scores, const int32_t* topk_idx, const int32_t* token_group,
                              const int32_t* slot_row, void* x_perm, int32_t* perm_token, float* perm_weight,
                              void* stream) {
  if (N < 0 || d < 1 || E < 1 || k < 1 || k > E || slots < k || D < 0) return CAPMOE_EINVAL;
  if (dtype != CAPMOE_F32 && dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (D > 0 && (E % D != 0 || slots != k + E / D)) return CAPMOE_EINVAL;
  if (D == 0 && slots != k) return CAPMOE_EINVAL;
  if (slots > MAX_SLOTS) return CAPMOE_EUNSUPPORTED;
  if (((size_t)d * elt_size(dtype)) % 16 != 0) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return CAPMOE_OK;
  if (!x || !scores || !topk_idx || !slot_row || !x_perm || !perm_token || !perm_weight) return CAPMOE_EINVAL;
  if (!aligned16(x) || !aligned16(x_perm)) return CAPMOE_EINVAL;
  const int row_vecs = (int)((size_t)d * elt_size(dtype) / 16);
  k_permute<<<(unsigned)ceil_div(N, PC_WARPS), PC_WARPS * 32, 0, as_stream(stream)>>>(
      (const uint4*)x, N, row_vecs, E, k, slots, D, scores, topk_idx, token_group, slot_row, (uint4*)x_perm,
      perm_token, perm_weight);
  return check_launch();
}

extern "C" int capmoe_combine(const void* y_perm, const int32_t* slot_row, const float* perm_weight, int64_t N,
                              int d, int slots, int dtype, const void* y_shared, void* y, void* stream) {
  if (N < 0 || d < 1 || slots < 1) return CAPMOE_EINVAL;
  if (dtype != CAPMOE_F32 && dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (slots > MAX_SLOTS) return CAPMOE_EUNSUPPORTED;
  if (((size_t)d * elt_size(dtype)) % 16 != 0) return CAPMOE_EUNSUPPORTED;
  if (N == 0) return CAPMOE_OK;
  if (!slot_row || !y) return CAPMOE_EINVAL;       // y_perm / perm_weight may be NULL only if A == 0
  if (!aligned16(y_perm) || !aligned16(y) || !aligned16(y_shared)) return CAPMOE_EINVAL;
  const int row_vecs = (int)((size_t)d * elt_size(dtype) / 16);
  const unsigned grid = (unsigned)ceil_div(N, PC_WARPS);
  cudaStream_t st = as_stream(stream);
  if (dtype == CAPMOE_F32)
    k_combine<float><<<grid, PC_WARPS * 32, 0, st>>>((const uint4*)y_perm, slot_row, perm_weight, N, row_vecs,
                                                      slots, (const uint4*)y_shared, (uint4*)y);
  else
    k_combine<__nv_bfloat16><<<grid, PC_WARPS * 32, 0, st>>>((const uint4*)y_perm, slot_row, perm_weight, N,
                                                              row_vecs, slots, (const uint4*)y_shared, (uint4*)y);
  return check_launch();
}
