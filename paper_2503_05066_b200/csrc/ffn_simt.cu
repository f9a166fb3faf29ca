// Stage 5, plain-FMA path: grouped SwiGLU expert FFN for fp32 storage and for shapes the
// tensor-core path does not take.  fp32 accumulation with fused multiply-add; two grouped
// GEMMs (gate|up with the SwiGLU epilogue, then down), tiles scheduled from expert_offsets
// on the device.
#include "common.cuh"

namespace capmoe {

namespace {

constexpr int TS = 64;       // tile rows and columns
constexpr int BK = 16;       // K step
constexpr int NT = 256;      // threads: 16 x 16, each a 4 x 4 micro-tile

// C[r, c] = sum_j A[r, j] * B[e][c, j] for the rows of every expert segment.
// SWIGLU: two B operands (gate, up) and out = silu(g) * u.
template <typename T, bool SWIGLU>
__global__ void __launch_bounds__(NT)
k_grouped_gemm(const T* __restrict__ A, const int32_t* __restrict__ seg_begin, const int32_t* __restrict__ seg_end,
               int w_mod, int E, int K, int Nout, const T* __restrict__ B0, const T* __restrict__ B1, T* __restrict__ C) {
  __shared__ float As[BK][TS + 4];
  __shared__ float Bs0[BK][TS + 4];
  __shared__ float Bs1[SWIGLU ? BK : 1][TS + 4];
  __shared__ int seg[3];       // expert, first row, rows in this tile
  const int tid = threadIdx.x;
  if (tid == 0) {
    int slot = blockIdx.y, found = -1, row0 = 0, rows = 0;
    int acc = 0;
    for (int e = 0; e < E; ++e) {
      const int b = seg_begin[e], n = seg_end[e] - b;
      const int nt = (n + TS - 1) / TS;
      if (slot < acc + nt) {
        found = e;
        row0 = b + (slot - acc) * TS;
        rows = min(TS, b + n - row0);
        break;
      }
      acc += nt;
    }
    seg[0] = found; seg[1] = row0; seg[2] = rows;
  }
  __syncthreads();
  const int e = seg[0];
  if (e < 0) return;
  const int row0 = seg[1], rows = seg[2];
  const int col0 = blockIdx.x * TS;
  const int tx = tid & 15, ty = tid >> 4;
  const int we = w_mod > 0 ? e % w_mod : e;             // weight block of this segment
  const T* Be0 = B0 + (int64_t)we * Nout * K;
  const T* Be1 = SWIGLU ? B1 + (int64_t)we * Nout * K : nullptr;

  float acc0[4][4], acc1[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc0[i][j] = 0.f; acc1[i][j] = 0.f; }

  for (int k0 = 0; k0 < K; k0 += BK) {
    for (int i = tid; i < TS * BK; i += NT) {
      const int r = i / BK, c = i % BK;
      const bool kin = k0 + c < K;
      As[c][r] = (r < rows && kin) ? to_float(A[(int64_t)(row0 + r) * K + k0 + c]) : 0.f;
      const bool cin = (col0 + r < Nout) && kin;
      Bs0[c][r] = cin ? to_float(Be0[(int64_t)(col0 + r) * K + k0 + c]) : 0.f;
      if (SWIGLU) Bs1[c][r] = cin ? to_float(Be1[(int64_t)(col0 + r) * K + k0 + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b0[4], b1[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b0[j] = Bs0[kk][tx * 4 + j];
        b1[j] = SWIGLU ? Bs1[kk][tx * 4 + j] : 0.f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc0[i][j] = fmaf(a[i], b0[j], acc0[i][j]);
          if (SWIGLU) acc1[i][j] = fmaf(a[i], b1[j], acc1[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty * 4 + i;
    if (r >= rows) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = col0 + tx * 4 + j;
      if (c >= Nout) continue;
      float v = acc0[i][j];
      if (SWIGLU) v = v / (1.0f + expf(-v)) * acc1[i][j];
      C[(int64_t)(row0 + r) * Nout + c] = from_float<T>(v);
    }
  }
}

template <typename T>
int run(const T* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int d, int F, const T* wg,
        const T* wu, const T* wd, T* h, T* y, int64_t A_max, cudaEvent_t mid, cudaStream_t st) {
  const unsigned slots = (unsigned)(ceil_div(A_max, TS) + E);
  if (slots > 65535u) return CAPMOE_EUNSUPPORTED;
  k_grouped_gemm<T, true><<<dim3((unsigned)ceil_div(F, TS), slots), NT, 0, st>>>(x_perm, seg_begin, seg_end, w_mod, E,
                                                                                d, F, wg, wu, h);
  int rc = check_launch();
  if (rc != CAPMOE_OK) return rc;
  if (mid && (rc = note_cuda(cudaEventRecord(mid, st))) != CAPMOE_OK) return rc;
  k_grouped_gemm<T, false><<<dim3((unsigned)ceil_div(d, TS), slots), NT, 0, st>>>(h, seg_begin, seg_end, w_mod, E, F,
                                                                                 d, wd, nullptr, y);
  return check_launch();
}

}  // namespace

int ffn_simt(const void* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int d, int F,
             int dtype, const void* w_gate, const void* w_up, const void* w_down, void* h_ws, void* y_perm,
             int64_t A_max, cudaEvent_t mid, cudaStream_t st) {
  if (dtype == CAPMOE_F32)
    return run<float>((const float*)x_perm, seg_begin, seg_end, E, w_mod, d, F, (const float*)w_gate,
                      (const float*)w_up, (const float*)w_down, (float*)h_ws, (float*)y_perm, A_max, mid, st);
  return run<__nv_bfloat16>((const __nv_bfloat16*)x_perm, seg_begin, seg_end, E, w_mod, d, F, (const __nv_bfloat16*)w_gate,
                            (const __nv_bfloat16*)w_up, (const __nv_bfloat16*)w_down, (__nv_bfloat16*)h_ws,
                            (__nv_bfloat16*)y_perm, A_max, mid, st);
}

}  // namespace capmoe
