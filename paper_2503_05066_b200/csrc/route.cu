// Stage 1: router GEMM, softmax, per-token top-k, expert load histogram (Eq. 1, Eq. 3).
#include "common.cuh"
#include "softmax.cuh"

namespace capmoe {
namespace {

constexpr int RT_TOK = 32;     // tokens per CTA in the GEMM
constexpr int RT_EG = 8;       // expert groups per CTA (threads = RT_TOK * RT_EG)
constexpr int RT_BK = 64;      // K chunk

// logits[t,e] = sum_j x[t,j] w[e,j] + bias[e], fp32 accumulate.  One CTA: RT_TOK tokens x all E
// experts; thread (lane = token, group = tid/32) owns EPT experts of one token.
template <typename T, int EPT>
__global__ void __launch_bounds__(RT_TOK* RT_EG)
k_router_gemm(const T* __restrict__ x, const T* __restrict__ w, const float* __restrict__ bias,
              int64_t N, int d, int E, float* __restrict__ logits) {
  allow_next_kernel();
  wait_for_previous_kernel();
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

// Softmax, top-k and load histogram.  One warp per token, EPL = ceil(E/32) experts per lane: the max is a shuffle reduction (exact), every lane evaluates exp for its
// experts, ONE lane adds the E terms left to right (the order the scores are defined with),
// every lane divides; top-k is k rounds of a warp arg-max on (score, lower expert id wins).
constexpr int SW_WARPS = 8;

// The whole warp handles one token: lrow = its E logits (global or shared memory), prow = E floats
// of scratch owned by this warp, hist = the CTA's shared-memory load histogram.
template <int EPL>
__device__ __forceinline__ void softmax_topk_token(const float* lrow, int E, int k, int64_t t, float* prow,
                                                   float* __restrict__ scores, int32_t* __restrict__ topk_idx,
                                                   float* __restrict__ topk_score, int* hist) {
  const int lane = threadIdx.x & 31;
  float v[EPL];
  float mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const int e = lane + 32 * i;
    v[i] = e < E ? lrow[e] : -INFINITY;
    mx = v[i] > mx ? v[i] : mx;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float other = __shfl_xor_sync(0xffffffffu, mx, o);
    mx = other > mx ? other : mx;
  }
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const int e = lane + 32 * i;
    if (e < E) { v[i] = exp_fixed(__fsub_rn(v[i], mx)); prow[e] = v[i]; }
  }
  __syncwarp();
  float sum = 0.f;
  if (lane == 0)
    for (int e = 0; e < E; ++e) sum = __fadd_rn(sum, prow[e]);
  sum = __shfl_sync(0xffffffffu, sum, 0);
  __syncwarp();                                              // prow is rewritten by the next token
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const int e = lane + 32 * i;
    if (e < E) { v[i] = __fdiv_rn(v[i], sum); scores[t * E + e] = v[i]; }
    else v[i] = -1.f;                                        // never selected (scores are >= 0)
  }
  float my_score = 0.f;
  int my_idx = 0;
  for (int j = 0; j < k; ++j) {
    float best = -1.f;
    int be = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < EPL; ++i)                            // ascending expert id inside the lane
      if (v[i] > best) { best = v[i]; be = lane + 32 * i; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oe = __shfl_xor_sync(0xffffffffu, be, o);
      if (ob > best || (ob == best && oe < be)) { best = ob; be = oe; }
    }
#pragma unroll
    for (int i = 0; i < EPL; ++i)
      if (be == lane + 32 * i) v[i] = -2.f;                  // taken
    if (lane == j) { my_score = best; my_idx = be; }
  }
  if (lane < k) {
    topk_idx[t * k + lane] = my_idx;
    topk_score[t * k + lane] = my_score;
    atomicAdd(&hist[my_idx], 1);
  }
}

// The same for few experts (E <= G <= 16): G lanes per token, 32 / G tokens per warp side by side,
// so that a short list of tokens is one step deep.  Lane e of a group holds expert e; the sum is
// still taken left to right (every lane walks the group's exponentials in order), the arg-max
// rounds are butterflies on (score, lower expert id) inside the group.
template <int G>
__device__ __forceinline__ void softmax_topk_group(const float* lrow, bool active, int E, int k, int64_t t,
                                                   float* __restrict__ scores, int32_t* __restrict__ topk_idx,
                                                   float* __restrict__ topk_score, int* hist) {
  const int lane = threadIdx.x & 31, e = lane & (G - 1), first = lane & ~(G - 1);
  const bool mine = active && e < E;
  const float v = mine ? lrow[e] : -INFINITY;
  float mx = v;
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) {
    const float other = __shfl_xor_sync(0xffffffffu, mx, o);
    mx = other > mx ? other : mx;
  }
  const float p = mine ? exp_fixed(__fsub_rn(v, mx)) : 0.f;
  float sum = 0.f;
  for (int j = 0; j < E; ++j) sum = __fadd_rn(sum, __shfl_sync(0xffffffffu, p, first + j));
  float cur = mine ? __fdiv_rn(p, sum) : -1.f;                   // never selected (scores are >= 0)
  if (mine) scores[t * E + e] = cur;
  for (int j = 0; j < k; ++j) {
    float best = cur;
    int be = e;
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oe = __shfl_xor_sync(0xffffffffu, be, o);
      if (ob > best || (ob == best && oe < be)) { best = ob; be = oe; }
    }
    if (be == e) cur = -2.f;                                     // taken
    if (active && e == j) {
      topk_idx[t * k + j] = be;
      topk_score[t * k + j] = best;
      atomicAdd(&hist[be], 1);
    }
  }
}

template <int EPL>
__global__ void __launch_bounds__(SW_WARPS * 32)
k_softmax_topk_warp(const float* __restrict__ logits, int64_t N, int E, int k, float* __restrict__ scores,
                    int32_t* __restrict__ topk_idx, float* __restrict__ topk_score, int32_t* __restrict__ load) {
  allow_next_kernel();
  wait_for_previous_kernel();
  extern __shared__ float smem[];
  float* prow = smem + (threadIdx.x >> 5) * (EPL * 32);       // this warp's E exponentials
  int* hist = reinterpret_cast<int*>(smem + SW_WARPS * EPL * 32);
  for (int i = threadIdx.x; i < E; i += SW_WARPS * 32) hist[i] = 0;
  __syncthreads();
  const int64_t warps_total = (int64_t)gridDim.x * SW_WARPS;
  for (int64_t t = (int64_t)blockIdx.x * SW_WARPS + (threadIdx.x >> 5); t < N; t += warps_total)
    softmax_topk_token<EPL>(logits + t * E, E, k, t, prow, scores, topk_idx, topk_score, hist);
  __syncthreads();
  for (int i = threadIdx.x; i < E; i += SW_WARPS * 32)
    if (hist[i]) atomicAdd(&load[i], hist[i]);
}

template <int EPL>
int launch_softmax_warp(const float* lg, int64_t N, int E, int k, float* scores, int32_t* topk_idx,
                        float* topk_score, int32_t* load, cudaStream_t st) {
  const size_t smem = (size_t)SW_WARPS * EPL * 32 * sizeof(float) + (size_t)E * sizeof(int);
  int64_t blocks = ceil_div(N, SW_WARPS);
  const int64_t cap = (int64_t)sm_count() * 8;                 // resident CTAs; more tokens loop inside
  if (blocks > cap) blocks = cap;
  const int rc = note_cuda(launch_chained(k_softmax_topk_warp<EPL>, (unsigned)blocks, SW_WARPS * 32, smem, st, lg, N, E, k,
                                          scores, topk_idx, topk_score, load));
  count_launch(1);
  return rc;
}

template <typename T>
int launch_gemm(const T* x, const T* w, const float* bias, int64_t N, int d, int E, float* logits,
                cudaStream_t st) {
  const int ept = (E + RT_EG - 1) / RT_EG;
  const size_t smem = (size_t)(RT_TOK + E) * (RT_BK + 1) * sizeof(float);
  const dim3 grid((unsigned)ceil_div(N, RT_TOK)), block(RT_TOK * RT_EG);
  cudaError_t launch_err = cudaSuccess;
#define CAPMOE_RT_CASE(EPT)                                                                      \
  {                                                                                              \
    if (smem > 48 * 1024) {                                                                      \
      cudaError_t e_ = cudaFuncSetAttribute(k_router_gemm<T, EPT>,                               \
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
      if (e_ != cudaSuccess) return note_cuda(e_);                                               \
    }                                                                                            \
    launch_err = launch_chained(k_router_gemm<T, EPT>, grid.x, block.x, smem, st, x, w, bias, N, d, E, logits); \
  }
  if (ept <= 1) CAPMOE_RT_CASE(1)
  else if (ept <= 2) CAPMOE_RT_CASE(2)
  else if (ept <= 4) CAPMOE_RT_CASE(4)
  else if (ept <= 8) CAPMOE_RT_CASE(8)
  else if (ept <= 16) CAPMOE_RT_CASE(16)
  else CAPMOE_RT_CASE(32)
#undef CAPMOE_RT_CASE
  count_launch(1);
  return note_cuda(launch_err);
}

// ---------------------------------------------------------------------------------------------
// bf16 router GEMM, bandwidth-bound form.  The stage has to read X exactly once at HBM speed, so
// X fragments go from global memory straight into tensor-core registers with 16-byte loads:
// a CTA owns 16*MT tokens, its 8 warps split the d columns (split-K), each warp runs
// mma.m16n8k16 (bf16 x bf16 -> fp32) over its column range and the 8 partial sums are added in
// warp order through shared memory (a fixed order, so logits are reproducible).
// The k index inside an MMA is only a summation index, so each thread takes its 8 consecutive
// columns of X (one 16-byte load) as the k slots it owns in two MMAs, and loads the same 8
// columns of W_r for its B fragment; no shared-memory staging or ldmatrix is needed.
constexpr int RM_WARPS = 8;
}  // namespace
// tcgen05 router GEMM (ffn_tc.cu): used when there are enough experts for the MMA work to matter
bool router_tc_supported(int64_t N, int d, int E);
bool router_tc_fusable(int E, int k);
int router_tc(const void* x, const void* w_router, const float* bias, int64_t N, int d, int E, float* logits,
              float* scores, int32_t* topk_idx, float* topk_score, int32_t* load, int k, bool fused,
              cudaStream_t st);
namespace {

__device__ __forceinline__ void mma_bf16_16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// FUSED: the CTA goes on to softmax / top-k / load histogram for its tokens (E <= 32), so the
// router is a single pass over X.
template <int MT, int NT, bool FUSED>
__global__ void __launch_bounds__(RM_WARPS * 32)
k_router_mma(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
             const float* __restrict__ bias, int64_t N, int d, int E, float* __restrict__ logits, int k,
             float* __restrict__ scores, int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
             int32_t* __restrict__ load) {
  allow_next_kernel();
  wait_for_previous_kernel();
  extern __shared__ float red[];                       // [RM_WARPS][16*MT][NT*8 + 1] (+ fused scratch)
  constexpr int ROWS = 16 * MT, EP = NT * 8, LD = EP + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, q = lane & 3;
  const int64_t t0 = (int64_t)blockIdx.x * ROWS;
  const int kw = d / RM_WARPS;                         // columns per warp (multiple of 64)
  const int kbeg = warp * kw;

  float acc[MT][NT][4];
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[i][j][r] = 0.f;

  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  const uint4* xrow[MT][2];
#pragma unroll
  for (int i = 0; i < MT; ++i) {
    const int64_t ta = t0 + i * 16 + g, tb = ta + 8;
    xrow[i][0] = ta < N ? reinterpret_cast<const uint4*>(x + ta * d + kbeg) + 2 * q : nullptr;
    xrow[i][1] = tb < N ? reinterpret_cast<const uint4*>(x + tb * d + kbeg) + 2 * q : nullptr;
  }
  const uint4* wrow[NT];
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    const int e = j * 8 + g;
    wrow[j] = e < E ? reinterpret_cast<const uint4*>(w + (int64_t)e * d + kbeg) + 2 * q : nullptr;
  }

  // 64 columns per step: each lane takes 32 contiguous bytes (two 16-byte loads) of its two rows, so
  // the four lanes of a row cover one full 128-byte line per step
  const int steps = kw / 64;
#pragma unroll 4
  for (int s = 0; s < steps; ++s) {
    uint4 xa[MT][2], xb[MT][2];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        xa[i][h] = xrow[i][0] ? __ldcs(xrow[i][0] + s * 8 + h) : zero;   // streamed once: evict first
        xb[i][h] = xrow[i][1] ? __ldcs(xrow[i][1] + s * 8 + h) : zero;
      }
#pragma unroll
    for (int j = 0; j < NT; ++j) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint4 wv = wrow[j] ? __ldg(wrow[j] + s * 8 + h) : zero;
#pragma unroll
        for (int i = 0; i < MT; ++i) {
          mma_bf16_16816(acc[i][j], xa[i][h].x, xb[i][h].x, xa[i][h].y, xb[i][h].y, wv.x, wv.y);
          mma_bf16_16816(acc[i][j], xa[i][h].z, xb[i][h].z, xa[i][h].w, xb[i][h].w, wv.z, wv.w);
        }
      }
    }
  }

  // partial sums of this warp -> shared memory (accumulator layout: rows g, g+8; columns 2q, 2q+1)
  float* mine = red + (size_t)warp * ROWS * LD;
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const int r0 = i * 16 + g, c0 = j * 8 + 2 * q;
      mine[r0 * LD + c0] = acc[i][j][0];
      mine[r0 * LD + c0 + 1] = acc[i][j][1];
      mine[(r0 + 8) * LD + c0] = acc[i][j][2];
      mine[(r0 + 8) * LD + c0 + 1] = acc[i][j][3];
    }
  __syncthreads();
  for (int i = threadIdx.x; i < ROWS * E; i += RM_WARPS * 32) {
    const int r = i / E, e = i - r * E;
    const int64_t t = t0 + r;
    if (t >= N) continue;
    float sum = 0.f;
#pragma unroll
    for (int wv = 0; wv < RM_WARPS; ++wv) sum += red[((size_t)wv * ROWS + r) * LD + e];
    sum += bias ? bias[e] : 0.f;
    logits[t * E + e] = sum;
    if (FUSED) red[(size_t)RM_WARPS * ROWS * LD + r * 32 + e] = sum;      // final logits tile [ROWS][32]
  }
  if (FUSED) {
    float* fin = red + (size_t)RM_WARPS * ROWS * LD;                       // [ROWS][32]
    float* prow = fin + ROWS * 32 + warp * 32;                             // [RM_WARPS][32]
    int* hist = reinterpret_cast<int*>(fin + ROWS * 32 + RM_WARPS * 32);   // [32]
    if (threadIdx.x < 32) hist[threadIdx.x] = 0;
    __syncthreads();
    if (E <= 8) {
      for (int r0 = warp * 4; r0 < ROWS; r0 += RM_WARPS * 4) {      // four tokens per warp at a time
        const int r = r0 + (lane >> 3);
        const int64_t t = t0 + r;
        softmax_topk_group<8>(fin + (r < ROWS ? r : 0) * 32, r < ROWS && t < N, E, k, t, scores, topk_idx, topk_score, hist);
      }
    } else if (E <= 16) {
      for (int r0 = warp * 2; r0 < ROWS; r0 += RM_WARPS * 2) {
        const int r = r0 + (lane >> 4);
        const int64_t t = t0 + r;
        softmax_topk_group<16>(fin + (r < ROWS ? r : 0) * 32, r < ROWS && t < N, E, k, t, scores, topk_idx, topk_score, hist);
      }
    } else {
      for (int r = warp; r < ROWS; r += RM_WARPS) {
        const int64_t t = t0 + r;
        if (t < N) softmax_topk_token<1>(fin + r * 32, E, k, t, prow, scores, topk_idx, topk_score, hist);
      }
    }
    __syncthreads();
    if (threadIdx.x < E && hist[threadIdx.x]) atomicAdd(&load[threadIdx.x], hist[threadIdx.x]);
  }
}

struct RouteOut { int k; float* scores; int32_t* topk_idx; float* topk_score; int32_t* load; };

bool router_mma_ok(int d, int E) { return d % (RM_WARPS * 64) == 0 && E <= 128; }


template <int MT, int NT, bool FUSED>
int launch_router_mma_inst(const __nv_bfloat16* x, const __nv_bfloat16* w, const float* bias, int64_t N, int d,
                           int E, float* logits, const RouteOut& o, cudaStream_t st) {
  size_t smem = (size_t)RM_WARPS * 16 * MT * (NT * 8 + 1) * sizeof(float);
  if (FUSED) smem += (size_t)(16 * MT * 32 + RM_WARPS * 32 + 32) * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e_ = cudaFuncSetAttribute(k_router_mma<MT, NT, FUSED>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e_ != cudaSuccess) return note_cuda(e_);
  }
  const int rc = note_cuda(launch_chained(k_router_mma<MT, NT, FUSED>, (unsigned)ceil_div(N, 16 * MT), RM_WARPS * 32, smem,
                                          st, x, w, bias, N, d, E, logits, o.k, o.scores, o.topk_idx, o.topk_score,
                                          o.load));
  count_launch(1);
  return rc;
}

// fused = true: the kernel also produced scores, top-k and the load histogram.
int launch_router_mma(const __nv_bfloat16* x, const __nv_bfloat16* w, const float* bias, int64_t N, int d, int E,
                      float* logits, const RouteOut& o, bool* fused, cudaStream_t st) {
  const int nt = (E + 7) / 8;
  *fused = nt <= 2;
  if (nt <= 1) return launch_router_mma_inst<1, 1, true>(x, w, bias, N, d, E, logits, o, st);
  if (nt <= 2) return launch_router_mma_inst<1, 2, true>(x, w, bias, N, d, E, logits, o, st);
  const bool wide = N >= (int64_t)32 * 2 * sm_count();      // enough tokens for 32-token CTAs to fill the GPU
  if (nt <= 4) return wide ? launch_router_mma_inst<2, 4, false>(x, w, bias, N, d, E, logits, o, st)
                           : launch_router_mma_inst<1, 4, false>(x, w, bias, N, d, E, logits, o, st);
  if (nt <= 8) return wide ? launch_router_mma_inst<2, 8, false>(x, w, bias, N, d, E, logits, o, st)
                           : launch_router_mma_inst<1, 8, false>(x, w, bias, N, d, E, logits, o, st);
  return launch_router_mma_inst<1, 16, false>(x, w, bias, N, d, E, logits, o, st);
}

}  // namespace
}  // namespace capmoe

using namespace capmoe;

int capmoe::route_impl(const void* x, const void* w_router, const float* bias, const float* logits_in,
                            int64_t N, int d, int E, int k, int dtype, float* logits, float* scores,
                            int32_t* topk_idx, float* topk_score, int32_t* load, void* stream, bool load_cleared) {
  if (N < 0 || E < 1 || k < 1 || k > E || d < 0) return CAPMOE_EINVAL;
  if (E > 256 || k > 32) return CAPMOE_EUNSUPPORTED;
  if (dtype != CAPMOE_F32 && dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (!scores || !topk_idx || !topk_score || !load) return CAPMOE_EINVAL;
  if (!logits_in && (!x || !w_router || !logits || d < 1)) return CAPMOE_EINVAL;
  if (N * (int64_t)E >= (int64_t)1 << 40) return CAPMOE_EUNSUPPORTED;
  cudaStream_t st = as_stream(stream);
  cudaError_t err = cudaSuccess;
  if (!load_cleared) {
    const int rc0 = clear_words(load, E, nullptr, 0, st);
    if (rc0 != CAPMOE_OK) return rc0;
  }
  if (N == 0) return CAPMOE_OK;
  const float* lg = logits_in;
  if (!logits_in) {
    int rc;
    bool fused = false;
    const RouteOut ro{k, scores, topk_idx, topk_score, load};
    if (dtype == CAPMOE_F32)
      rc = launch_gemm<float>((const float*)x, (const float*)w_router, bias, N, d, E, logits, st);
    else if (E > 16 && router_tc_supported(N, d, E) && aligned16(x) && aligned16(w_router)) {
      fused = router_tc_fusable(E, k);
      rc = router_tc(x, w_router, bias, N, d, E, logits, scores, topk_idx, topk_score, load, k, fused, st);
    }
    else if (router_mma_ok(d, E) && aligned16(x) && aligned16(w_router))
      rc = launch_router_mma((const __nv_bfloat16*)x, (const __nv_bfloat16*)w_router, bias, N, d, E, logits, ro,
                             &fused, st);
    else
      rc = launch_gemm<__nv_bfloat16>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w_router, bias, N, d, E,
                                      logits, st);
    if (rc != CAPMOE_OK) return rc;
    if (fused) return CAPMOE_OK;
    lg = logits;
  } else if (logits && logits != logits_in) {
    err = cudaMemcpyAsync(logits, logits_in, sizeof(float) * N * E, cudaMemcpyDeviceToDevice, st);
    if (err != cudaSuccess) return note_cuda(err);
  }
  const int epl = (E + 31) / 32;
  if (epl <= 1) return launch_softmax_warp<1>(lg, N, E, k, scores, topk_idx, topk_score, load, st);
  if (epl <= 2) return launch_softmax_warp<2>(lg, N, E, k, scores, topk_idx, topk_score, load, st);
  if (epl <= 4) return launch_softmax_warp<4>(lg, N, E, k, scores, topk_idx, topk_score, load, st);
  return launch_softmax_warp<8>(lg, N, E, k, scores, topk_idx, topk_score, load, st);
}

extern "C" int capmoe_route(const void* x, const void* w_router, const float* bias, const float* logits_in,
                            int64_t N, int d, int E, int k, int dtype, float* logits, float* scores,
                            int32_t* topk_idx, float* topk_score, int32_t* load, void* stream) {
  return route_impl(x, w_router, bias, logits_in, N, d, E, k, dtype, logits, scores, topk_idx, topk_score, load, stream,
                    false);
}
