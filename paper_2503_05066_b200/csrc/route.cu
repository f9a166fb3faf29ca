// Stage 1: router GEMM, softmax, per-token top-k, expert load histogram (Eq. 1, Eq. 3).
#include "common.cuh"

namespace capmoe {
namespace {

constexpr int RT_TOK = 32;     // tokens per CTA in the GEMM
constexpr int RT_EG = 8;       // expert groups per CTA (threads = RT_TOK * RT_EG)
constexpr int RT_BK = 64;      // K chunk
constexpr int SM_TOK = 64;     // tokens per CTA in the softmax/top-k kernel

// logits[t,e] = sum_j x[t,j] w[e,j] + bias[e], fp32 accumulate.  One CTA: RT_TOK tokens x all E
// experts; thread (lane = token, group = tid/32) owns EPT experts of one token.
template <typename T, int EPT>
__global__ void __launch_bounds__(RT_TOK* RT_EG)
k_router_gemm(const T* __restrict__ x, const T* __restrict__ w, const float* __restrict__ bias,
              int64_t N, int d, int E, float* __restrict__ logits) {
  extern __shared__ float smem[];
  float* xs = smem;                              // [RT_TOK][RT_BK+1]
  float* wsm = smem + RT_TOK * (RT_BK + 1);      // [E][RT_BK+1]
  const int tid = threadIdx.x;
  const int lane_tok = tid & 31, eg = tid >> 5;
  const int64_t t0 = (int64_t)blockIdx.x * RT_TOK;
  float acc[EPT];
#pragma unroll
  for (int i = 0; i < EPT; ++i) acc[i] = 0.f;

  for (int k0 = 0; k0 < d; k0 += RT_BK) {
    for (int i = tid; i < RT_TOK * RT_BK; i += RT_TOK * RT_EG) {
      int r = i / RT_BK, c = i % RT_BK;
      int64_t t = t0 + r;
      xs[r * (RT_BK + 1) + c] = (t < N && k0 + c < d) ? to_float(x[t * d + k0 + c]) : 0.f;
    }
    for (int i = tid; i < E * RT_BK; i += RT_TOK * RT_EG) {
      int r = i / RT_BK, c = i % RT_BK;
      wsm[r * (RT_BK + 1) + c] = (k0 + c < d) ? to_float(w[(int64_t)r * d + k0 + c]) : 0.f;
    }
    __syncthreads();
    const float* xr = xs + lane_tok * (RT_BK + 1);
#pragma unroll 8
    for (int j = 0; j < RT_BK; ++j) {
      float xv = xr[j];
#pragma unroll
      for (int i = 0; i < EPT; ++i) {
        int e = eg * EPT + i;
        float wv = e < E ? wsm[e * (RT_BK + 1) + j] : 0.f;
        acc[i] = fmaf(xv, wv, acc[i]);
      }
    }
    __syncthreads();
  }
  int64_t t = t0 + lane_tok;
  if (t < N) {
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
      int e = eg * EPT + i;
      if (e < E) logits[t * E + e] = acc[i] + (bias ? bias[e] : 0.f);
    }
  }
}

// exp(x), x <= 0, as a fixed sequence of correctly rounded binary32 operations: range
// reduction x = n ln2 + r with a two-word ln2, a degree-7 Taylor polynomial in Horner/fma
// form, scaling by 2^n through the exponent field.  x < -80 gives exactly 0.
__device__ __forceinline__ float exp_fixed(float x) {
  if (x < -80.0f) return 0.0f;
  const float n = rintf(__fmul_rn(x, __uint_as_float(0x3fb8aa3bu)));          // x * log2(e)
  float r = __fmaf_rn(n, -__uint_as_float(0x3f317200u), x);                   // - n * ln2_hi
  r = __fmaf_rn(n, -__uint_as_float(0x35bfbe8eu), r);                         // - n * ln2_lo
  float q = __uint_as_float(0x39500d01u);                                     // 1/7!
  q = __fmaf_rn(q, r, __uint_as_float(0x3ab60b61u));                          // 1/6!
  q = __fmaf_rn(q, r, __uint_as_float(0x3c088889u));                          // 1/5!
  q = __fmaf_rn(q, r, __uint_as_float(0x3d2aaaabu));                          // 1/4!
  q = __fmaf_rn(q, r, __uint_as_float(0x3e2aaaabu));                          // 1/3!
  q = __fmaf_rn(q, r, 0.5f);
  q = __fmaf_rn(q, r, 1.0f);
  q = __fmaf_rn(q, r, 1.0f);
  const int ni = (int)n;
  return __uint_as_float(__float_as_uint(q) + ((unsigned)ni << 23));
}

// One thread per token: softmax over the E logits (left-to-right sum), top-k by repeated
// arg-max (strict '>' keeps the lower expert id on equal scores), load histogram.
__global__ void __launch_bounds__(SM_TOK)
k_softmax_topk(const float* __restrict__ logits, int64_t N, int E, int k, float* __restrict__ scores,
               int32_t* __restrict__ topk_idx, float* __restrict__ topk_score, int32_t* __restrict__ load) {
  extern __shared__ float smem[];
  const int ld = E + 1;
  float* rows = smem;                                     // [SM_TOK][E+1]
  int* hist = reinterpret_cast<int*>(smem + SM_TOK * ld); // [E]
  const int tid = threadIdx.x;
  const int64_t t0 = (int64_t)blockIdx.x * SM_TOK;
  const int64_t nrow = min((int64_t)SM_TOK, N - t0);
  for (int i = tid; i < E; i += SM_TOK) hist[i] = 0;
  for (int64_t i = tid; i < nrow * E; i += SM_TOK) rows[(i / E) * ld + (i % E)] = logits[t0 * E + i];
  __syncthreads();
  float* row = rows + tid * ld;
  if (tid < nrow) {
    float mx = row[0];
    for (int e = 1; e < E; ++e) mx = row[e] > mx ? row[e] : mx;
    float sum = 0.f;
    for (int e = 0; e < E; ++e) {
      float p = exp_fixed(__fsub_rn(row[e], mx));
      row[e] = p;
      sum = __fadd_rn(sum, p);
    }
    for (int e = 0; e < E; ++e) row[e] = __fdiv_rn(row[e], sum);
  }
  __syncthreads();
  for (int64_t i = tid; i < nrow * E; i += SM_TOK) scores[t0 * E + i] = rows[(i / E) * ld + (i % E)];
  __syncthreads();
  if (tid < nrow) {
    const int64_t t = t0 + tid;
    for (int j = 0; j < k; ++j) {
      float best = -1.f;
      int be = 0;
      for (int e = 0; e < E; ++e) {
        float v = row[e];
        if (v > best) { best = v; be = e; }
      }
      row[be] = -2.f;                                     // taken (scores are >= 0)
      topk_idx[t * k + j] = be;
      topk_score[t * k + j] = best;
      atomicAdd(&hist[be], 1);
    }
  }
  __syncthreads();
  for (int i = tid; i < E; i += SM_TOK)
    if (hist[i]) atomicAdd(&load[i], hist[i]);
}

template <typename T>
int launch_gemm(const T* x, const T* w, const float* bias, int64_t N, int d, int E, float* logits,
                cudaStream_t st) {
  const int ept = (E + RT_EG - 1) / RT_EG;
  const size_t smem = (size_t)(RT_TOK + E) * (RT_BK + 1) * sizeof(float);
  const dim3 grid((unsigned)ceil_div(N, RT_TOK)), block(RT_TOK * RT_EG);
#define CAPMOE_RT_CASE(EPT)                                                                      \
  {                                                                                              \
    if (smem > 48 * 1024) {                                                                      \
      cudaError_t e_ = cudaFuncSetAttribute(k_router_gemm<T, EPT>,                               \
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
      if (e_ != cudaSuccess) return note_cuda(e_);                                               \
    }                                                                                            \
    k_router_gemm<T, EPT><<<grid, block, smem, st>>>(x, w, bias, N, d, E, logits);               \
  }
  if (ept <= 1) CAPMOE_RT_CASE(1)
  else if (ept <= 2) CAPMOE_RT_CASE(2)
  else if (ept <= 4) CAPMOE_RT_CASE(4)
  else if (ept <= 8) CAPMOE_RT_CASE(8)
  else if (ept <= 16) CAPMOE_RT_CASE(16)
  else CAPMOE_RT_CASE(32)
#undef CAPMOE_RT_CASE
  return check_launch();
}

}  // namespace
}  // namespace capmoe

using namespace capmoe;

extern "C" int capmoe_route(const void* x, const void* w_router, const float* bias, const float* logits_in,
                            int64_t N, int d, int E, int k, int dtype, float* logits, float* scores,
                            int32_t* topk_idx, float* topk_score, int32_t* load, void* stream) {
  if (N < 0 || E < 1 || k < 1 || k > E || d < 0) return CAPMOE_EINVAL;
  if (E > 256 || k > 32) return CAPMOE_EUNSUPPORTED;
  if (dtype != CAPMOE_F32 && dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (!scores || !topk_idx || !topk_score || !load) return CAPMOE_EINVAL;
  if (!logits_in && (!x || !w_router || !logits || d < 1)) return CAPMOE_EINVAL;
  if (N * (int64_t)E >= (int64_t)1 << 40) return CAPMOE_EUNSUPPORTED;
  cudaStream_t st = as_stream(stream);
  cudaError_t err = cudaMemsetAsync(load, 0, sizeof(int32_t) * E, st);
  if (err != cudaSuccess) return note_cuda(err);
  if (N == 0) return CAPMOE_OK;
  const float* lg = logits_in;
  if (!logits_in) {
    int rc = dtype == CAPMOE_F32
                 ? launch_gemm<float>((const float*)x, (const float*)w_router, bias, N, d, E, logits, st)
                 : launch_gemm<__nv_bfloat16>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w_router, bias,
                                              N, d, E, logits, st);
    if (rc != CAPMOE_OK) return rc;
    lg = logits;
  } else if (logits && logits != logits_in) {
    err = cudaMemcpyAsync(logits, logits_in, sizeof(float) * N * E, cudaMemcpyDeviceToDevice, st);
    if (err != cudaSuccess) return note_cuda(err);
  }
  const size_t smem = (size_t)SM_TOK * (E + 1) * sizeof(float) + (size_t)E * sizeof(int);
  if (smem > 48 * 1024) {
    err = cudaFuncSetAttribute(k_softmax_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return note_cuda(err);
  }
  k_softmax_topk<<<(unsigned)ceil_div(N, SM_TOK), SM_TOK, smem, st>>>(lg, N, E, k, scores, topk_idx,
                                                                       topk_score, load);
  return check_launch();
}
