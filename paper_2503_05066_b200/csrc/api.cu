// Host side of the C ABI: helpers, the FFN dispatcher and the whole-layer entry points.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace capmoe {


static std::atomic<uint64_t> g_launches{0};
static thread_local char g_cuda_err[256] = "";

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int note_cuda(cudaError_t err) {
  if (err == cudaSuccess) return CAPMOE_OK;
  std::snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", cudaGetErrorName(err), cudaGetErrorString(err));
  return CAPMOE_ECUDA;
}

int check_launch() {
  count_launch(1);
  return note_cuda(cudaPeekAtLastError());
}

namespace {
__global__ void __launch_bounds__(256) k_clear_words(int32_t* __restrict__ a, int na, int32_t* __restrict__ b, int nb) {
  allow_next_kernel();
  wait_for_previous_kernel();
  for (int i = threadIdx.x; i < na; i += 256) a[i] = 0;
  for (int i = threadIdx.x; i < nb; i += 256) b[i] = 0;
}
}  // namespace

namespace {
// Reads `n` 16-byte vectors once, eight independent loads in flight per thread, and keeps the
// compiler from dropping them; nothing else.  The time of this launch is what ANY kernel needs to
// pull that many bytes out of HBM once, launch included.
__global__ void __launch_bounds__(256) k_read_probe(const uint4* __restrict__ p, size_t n, int32_t* __restrict__ sink) {
  unsigned acc = 0;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i + 7 * stride < n; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = __ldcs(p + i + u * stride);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n; i += stride) {
    const uint4 v = __ldcs(p + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  if (acc == 0x9e3779b9u && sink) *sink = (int32_t)acc;       // practically never: keeps the loads alive
}
}  // namespace

int read_probe(const void* p, size_t bytes, int32_t* sink, cudaStream_t st) {
  k_read_probe<<<(unsigned)(sm_count() * 8), 256, 0, st>>>((const uint4*)p, bytes / 16, sink);
  return check_launch();
}

int clear_words(int32_t* a, int na, int32_t* b, int nb, cudaStream_t st) {
  if (!a) na = 0;
  if (!b) nb = 0;
  if (na <= 0 && nb <= 0) return CAPMOE_OK;
  const int rc = note_cuda(launch_chained(k_clear_words, 1u, 256u, 0, st, a, na, b, nb));
  count_launch(1);
  return rc;
}

int sm_count() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

// defined in ffn_simt.cu / ffn_tc.cu
int ffn_simt(const void* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int d, int F,
             int dtype, const void* w_gate, const void* w_up, const void* w_down, void* h_ws, void* y_perm,
             int64_t A_max, cudaEvent_t mid, cudaStream_t st);
int ffn_tc(const void* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int n_w, int d, int F,
           const void* w_gate, const void* w_up, const void* w_down, void* h_ws, void* y_perm, int64_t A_max,
           int D_straggler, int32_t* dev_status, int sched_slot, bool counters_cleared, cudaEvent_t mid, cudaStream_t st);
int wait_probe(long long limit_cycles, int32_t* dev_status, cudaStream_t st);

// Row segments [seg_begin[e], seg_end[e]), e < E; segment e uses weight block e % w_mod (w_mod = 0:
// block e).  The packed form of the stage is seg_begin = expert_offsets, seg_end = expert_offsets + 1.
static int grouped_ffn_impl(const void* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int d,
                            int F, int dtype, const void* w_gate, const void* w_up, const void* w_down, void* h_ws,
                            void* y_perm, int64_t A_max, int D_straggler, int32_t* dev_status, cudaEvent_t mid,
                            void* stream, int sched_slot = 0, bool counters_cleared = false) {
  if (E < 1 || d < 1 || F < 1 || A_max < 0 || D_straggler < 0 || w_mod < 0 || w_mod > E) return CAPMOE_EINVAL;
  if (dtype != CAPMOE_F32 && dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (D_straggler > 0 && E % D_straggler != 0) return CAPMOE_EINVAL;
  if (E > 256) return CAPMOE_EUNSUPPORTED;
  if (!seg_begin || !seg_end) return CAPMOE_EINVAL;
  if (A_max == 0) return CAPMOE_OK;
  if (!x_perm || !w_gate || !w_up || !w_down || !h_ws || !y_perm) return CAPMOE_EINVAL;
  if (!aligned16(x_perm) || !aligned16(w_gate) || !aligned16(w_up) || !aligned16(w_down) || !aligned16(h_ws) ||
      !aligned16(y_perm))
    return CAPMOE_EINVAL;
  const int n_w = w_mod > 0 ? w_mod : E;
  if (ffn_tc_supported(d, F, dtype))
    return ffn_tc(x_perm, seg_begin, seg_end, E, w_mod, n_w, d, F, w_gate, w_up, w_down, h_ws, y_perm, A_max,
                  D_straggler, dev_status, sched_slot, counters_cleared, mid, as_stream(stream));
  if (D_straggler > 0) return CAPMOE_EUNSUPPORTED;   // SM partitioning exists only in the tensor-core kernel
  return ffn_simt(x_perm, seg_begin, seg_end, E, w_mod, d, F, dtype, w_gate, w_up, w_down, h_ws, y_perm, A_max, mid,
                  as_stream(stream));
}

}  // namespace capmoe

using namespace capmoe;

extern "C" int capmoe_capacity(int64_t N, int E, int k, double gamma, int round, int64_t* C) {
  if (!C || N < 0 || E < 1 || k < 1 || k > E || !(gamma >= 0.0)) return CAPMOE_EINVAL;
  if (round != CAPMOE_CAP_CEIL && round != CAPMOE_CAP_FLOOR) return CAPMOE_EINVAL;
  double c;
  if (std::isinf(gamma)) {
    c = (double)N;
  } else {
    const double v = (gamma * (double)(N * (int64_t)k)) / (double)E;
    c = round == CAPMOE_CAP_FLOOR ? std::floor(v) : std::ceil(v);
  }
  if (c > (double)N) c = (double)N;
  if (c < 0.0) c = 0.0;
  *C = (int64_t)c;
  return CAPMOE_OK;
}

extern "C" int capmoe_device_capacity(int64_t N, int E, int k, int D, double gamma, int round, int64_t* C_dev) {
  if (!C_dev || N < 0 || E < 1 || k < 1 || k > E || D < 1 || E % D != 0 || !(gamma >= 0.0)) return CAPMOE_EINVAL;
  if (round != CAPMOE_CAP_CEIL && round != CAPMOE_CAP_FLOOR) return CAPMOE_EINVAL;
  const double most = (double)N * (double)(E / D);
  double c;
  if (std::isinf(gamma)) {
    c = most;
  } else {
    const double v = (gamma * (double)(N * (int64_t)k)) / (double)D;
    c = round == CAPMOE_CAP_FLOOR ? std::floor(v) : std::ceil(v);
  }
  if (c > most) c = most;
  if (c < 0.0) c = 0.0;
  *C_dev = (int64_t)c;
  return CAPMOE_OK;
}

extern "C" int capmoe_max_rows(int64_t N, int E, int k, int D, int64_t C, int expanded, int64_t* A_max) {
  if (!A_max || N < 0 || E < 1 || k < 1 || k > E || C < 0) return CAPMOE_EINVAL;
  if (expanded && (D < 1 || E % D != 0)) return CAPMOE_EINVAL;
  const int64_t cands = N * (int64_t)(expanded ? k + E / D : k);
  const int64_t cap = (int64_t)E * (C > N ? N : C);
  *A_max = cands < cap ? cands : cap;
  return CAPMOE_OK;
}

extern "C" int capmoe_device_max_rows(int64_t N, int E, int k, int D, int64_t C_dev, int expanded, int64_t* A_max) {
  if (!A_max || N < 0 || E < 1 || k < 1 || k > E || D < 1 || E % D != 0 || C_dev < 0) return CAPMOE_EINVAL;
  const int64_t cands = N * (int64_t)(expanded ? k + E / D : k);
  const int64_t most = N * (int64_t)(E / D);
  const int64_t cap = (int64_t)D * (C_dev > most ? most : C_dev);
  *A_max = cands < cap ? cands : cap;
  return CAPMOE_OK;
}

extern "C" const char* capmoe_status_str(int status) {
  switch (status) {
    case CAPMOE_OK: return "ok";
    case CAPMOE_EINVAL: return "invalid argument";
    case CAPMOE_EUNSUPPORTED: return "unsupported dtype or shape";
    case CAPMOE_EWORKSPACE: return "workspace too small";
    case CAPMOE_ECUDA: return "CUDA error";
    case CAPMOE_ETIMEOUT: return "device-side wait timed out";
    case CAPMOE_EINDEX: return "row index outside its buffer (debug check)";
    default: return "unknown status";
  }
}

extern "C" const char* capmoe_last_cuda_error(void) { return g_cuda_err; }
extern "C" uint64_t capmoe_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
extern "C" int capmoe_ffn_uses_tensor_cores(int d, int F, int dtype) { return ffn_tc_supported(d, F, dtype) ? 1 : 0; }

extern "C" int capmoe_debug_read_probe(const void* p, size_t bytes, int32_t* sink, void* stream) {
  if (!p || !aligned16(p) || bytes < 16) return CAPMOE_EINVAL;
  return read_probe(p, bytes, sink, as_stream(stream));
}

extern "C" int capmoe_debug_wait_probe(int64_t limit_cycles, int32_t* dev_status, void* stream) {
  if (!dev_status || limit_cycles < 1 || limit_cycles > 4000000000LL) return CAPMOE_EINVAL;
  return wait_probe((long long)limit_cycles, dev_status, as_stream(stream));
}

extern "C" int capmoe_grouped_ffn(const void* x_perm, const int32_t* expert_offsets, int E, int d, int F,
                                  int dtype, const void* w_gate, const void* w_up, const void* w_down,
                                  void* h_ws, void* y_perm, int64_t A_max, int D_straggler,
                                  int32_t* dev_status, void* stream) {
  if (!expert_offsets) return CAPMOE_EINVAL;
  return grouped_ffn_impl(x_perm, expert_offsets, expert_offsets + 1, E, 0, d, F, dtype, w_gate, w_up, w_down, h_ws,
                          y_perm, A_max, D_straggler, dev_status, nullptr, stream);
}

extern "C" int capmoe_grouped_ffn_segments(const void* x_rows, const int32_t* seg_begin, const int32_t* seg_end, int S,
                                           int w_mod, int d, int F, int dtype, const void* w_gate, const void* w_up,
                                           const void* w_down, void* h_ws, void* y_rows, int64_t rows,
                                           int32_t* dev_status, void* stream) {
  return grouped_ffn_impl(x_rows, seg_begin, seg_end, S, w_mod, d, F, dtype, w_gate, w_up, w_down, h_ws, y_rows, rows,
                          0, dev_status, nullptr, stream);
}

namespace capmoe {
namespace {

// Rows of the permuted matrix that a forward with these settings can produce at most.
int64_t layer_row_bound(const capmoe_layer* L, int slots) {
  const int64_t cands = L->N * (int64_t)slots;
  int64_t cap;
  if (L->mode == 0) cap = cands;
  else if (L->mode <= 2) cap = (int64_t)L->E * (L->C > L->N ? L->N : L->C);
  else cap = (int64_t)L->D * L->C;
  return cands < cap ? cands : cap;
}

// Every check of capmoe_layer_forward, made before the first event record, memset or launch, so
// that a non-zero return (other than CAPMOE_ECUDA) leaves the stream untouched.
int validate_layer(const capmoe_layer* L) {
  if (L->mode < 0 || L->mode > 4) return CAPMOE_EINVAL;
  if (L->N < 0 || L->d < 1 || L->E < 1 || L->k < 1 || L->k > L->E || L->F < 1 || L->A_max < 0) return CAPMOE_EINVAL;
  if (L->dtype != CAPMOE_F32 && L->dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (L->E > 256 || L->k > 32) return CAPMOE_EUNSUPPORTED;
  if (L->N >= ((int64_t)1 << 31) || L->N * (int64_t)L->E >= ((int64_t)1 << 40)) return CAPMOE_EUNSUPPORTED;
  const bool expanded = L->mode == 2 || L->mode == 4, device_level = L->mode >= 3;
  const bool needs_D = expanded || device_level || L->straggler;
  if (needs_D && (L->D < 1 || L->E % L->D != 0)) return CAPMOE_EINVAL;
  const int slots = expanded ? L->k + L->E / L->D : L->k;
  if (slots > 288) return CAPMOE_EUNSUPPORTED;
  if (L->N * (int64_t)slots >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  if (((size_t)L->d * elt_size(L->dtype)) % 16 != 0) return CAPMOE_EUNSUPPORTED;
  if (L->mode == 1 || L->mode == 2) {
    if (L->C < 0 || L->C > L->N) return CAPMOE_EINVAL;
  } else if (device_level) {
    if (L->C < 0 || L->C > L->N * (int64_t)(L->E / L->D)) return CAPMOE_EINVAL;
  }
  // variants of the drop
  if (L->metric < CAPMOE_METRIC_SCORE || L->metric > CAPMOE_METRIC_RANDOM || L->max_experts < 0) return CAPMOE_EINVAL;
  const bool variant = L->metric != CAPMOE_METRIC_SCORE || L->token_class || L->topk_first || L->max_experts > 0;
  if (device_level && variant) return CAPMOE_EUNSUPPORTED;      // defined for the per-expert capacity
  const bool keyed = (L->mode == 1 || L->mode == 2) &&
                     (L->metric != CAPMOE_METRIC_SCORE || L->token_class || (L->mode == 2 && L->topk_first));
  if (keyed && !L->drop_keys) return CAPMOE_EINVAL;
  if (L->mode != 0 && L->max_experts > 0 && !L->bad) return CAPMOE_EINVAL;
  if (L->debug_checks && !L->dev_status) return CAPMOE_EINVAL;
  // buffers
  if (!L->logits || !L->scores || !L->topk_idx || !L->topk_score || !L->load || !L->kept || !L->expert_offsets)
    return CAPMOE_EINVAL;
  if ((expanded || device_level) && !L->cand) return CAPMOE_EINVAL;
  if (L->stage_events)
    for (int i = 0; i < CAPMOE_N_STAGE_EVENTS; ++i)
      if (!L->stage_events[i]) return CAPMOE_EINVAL;
  if (L->F_shared < 0) return CAPMOE_EINVAL;
  if (L->F_shared > 0 &&
      (!L->ws_gate || !L->ws_up || !L->ws_down || !L->hs_ws || !L->y_shared || !L->one_segment ||
       !aligned16(L->ws_gate) || !aligned16(L->ws_up) || !aligned16(L->ws_down) || !aligned16(L->hs_ws) ||
       !aligned16(L->y_shared)))
    return CAPMOE_EINVAL;
  if (L->straggler && !ffn_tc_supported(L->d, L->F, L->dtype)) return CAPMOE_EUNSUPPORTED;
  if (L->A_max < layer_row_bound(L, slots)) return CAPMOE_EWORKSPACE;   // the permute and the FFN write by row index
  if (L->N > 0) {
    if (!L->x || !L->w_router || !L->keep_mask || !L->slot_row || !L->y || !L->drop_ws) return CAPMOE_EINVAL;
    if (!aligned16(L->x) || !aligned16(L->w_router) || !aligned16(L->y)) return CAPMOE_EINVAL;
    if (L->drop_ws_bytes < drop_ws_required(L->mode, L->N, L->E, L->k, needs_D ? L->D : 1)) return CAPMOE_EWORKSPACE;
  }
  if (L->A_max > 0) {
    if (!L->x_perm || !L->perm_token || !L->perm_weight || !L->h_ws || !L->y_perm || !L->w_gate || !L->w_up ||
        !L->w_down)
      return CAPMOE_EINVAL;
    if (!aligned16(L->x_perm) || !aligned16(L->h_ws) || !aligned16(L->y_perm) || !aligned16(L->w_gate) ||
        !aligned16(L->w_up) || !aligned16(L->w_down))
      return CAPMOE_EINVAL;
  }
  return CAPMOE_OK;
}

}  // namespace
}  // namespace capmoe

extern "C" int capmoe_layer_forward(const capmoe_layer* L, void* stream) {
  if (!L) return CAPMOE_EINVAL;
  {
    const int bad_args = validate_layer(L);
    if (bad_args != CAPMOE_OK) return bad_args;
  }
  cudaStream_t st = as_stream(stream);
  auto mark = [&](int i) -> int {
    if (!L->stage_events) return CAPMOE_OK;
    return note_cuda(cudaEventRecord((cudaEvent_t)L->stage_events[i], st));
  };
  int rc = mark(0);
  if (rc != CAPMOE_OK) return rc;
  // The tile counters of all FFN launches of this forward are cleared here, away from the kernels
  // that use them, so that no memset sits between the permute and the first GEMM.
  // Likewise the load histogram (one small kernel for both) and the drop stage's counters; the
  // stages are told so below.
  if ((rc = clear_words(L->dev_status ? L->dev_status + 1 : nullptr, CAPMOE_FFN_STATUS_WORDS - 1, L->load, L->E, st)) !=
      CAPMOE_OK)
    return rc;
  if ((rc = drop_clear_counters(L->mode, L->N, L->E, L->k, L->D < 1 ? 1 : L->D, L->cand, L->drop_ws, L->drop_ws_bytes,
                                st)) != CAPMOE_OK)
    return rc;
  rc = route_impl(L->x, L->w_router, L->bias, nullptr, L->N, L->d, L->E, L->k, L->dtype, L->logits, L->scores,
                  L->topk_idx, L->topk_score, L->load, stream, true);
  if (rc != CAPMOE_OK) return rc;
  if ((rc = mark(1)) != CAPMOE_OK) return rc;
  int slots, Dp;
  // The permute kernel can write the keep mask while it reads a token's rows, unless something
  // between the drop and the permute needs the mask ("w/ max").
  bool defer_mask = !(L->mode != 0 && L->max_experts > 0);
  if (L->mode >= 3) {                     // device-level capacity: L->C is the per-device bound
    defer_mask = false;                   // the token-parallel select writes the mask itself
    const int expanded = L->mode == 4;
    rc = device_drop_impl(L->scores, L->topk_idx, L->N, L->E, L->k, L->C, L->D, expanded, nullptr, L->keep_mask,
                          L->cand, L->kept, L->expert_offsets, L->slot_row, L->drop_ws, L->drop_ws_bytes, stream,
                          true);
    slots = expanded ? L->k + L->E / L->D : L->k;
    Dp = expanded ? L->D : 0;
  } else {
    // drop keys: the scores themselves, or a metric / priority class worked into 32-bit keys
    const bool expanded = L->mode == 2;
    const bool keyed = L->mode != 0 && (L->metric != CAPMOE_METRIC_SCORE || L->token_class || (expanded && L->topk_first));
    const float* sel = expanded ? L->scores : L->topk_score;
    if (keyed) {
      const int cols = expanded ? L->E : L->k;
      const int32_t* idx = expanded ? nullptr : L->topk_idx;
      uint32_t* keys = reinterpret_cast<uint32_t*>(L->drop_keys);
      rc = capmoe_drop_keys(L->metric, L->metric_seed, sel, idx, L->N, cols, L->E, keys, stream);
      if (rc != CAPMOE_OK) return rc;
      if (L->token_class || (expanded && L->topk_first)) {
        rc = capmoe_priority_keys(keys, idx, L->N, cols, L->E, L->metric == CAPMOE_METRIC_SCORE, L->token_class,
                                  (expanded && L->topk_first) ? L->topk_idx : nullptr, L->k, keys, stream);
        if (rc != CAPMOE_OK) return rc;
      }
      sel = L->drop_keys;
    }
    if (expanded) {
      rc = expanded_drop_impl(sel, L->topk_idx, L->N, L->E, L->k, L->C, L->D, nullptr, L->keep_mask, L->cand,
                              L->kept, L->expert_offsets, L->slot_row, L->drop_ws, L->drop_ws_bytes, stream, true,
                              &defer_mask, L->load);
      slots = L->k + L->E / L->D;
      Dp = L->D;
    } else {
      rc = token_drop_impl(sel, L->topk_idx, L->N, L->E, L->k, L->mode == 0 ? L->N : L->C, L->keep_mask, L->kept,
                           L->expert_offsets, L->slot_row, L->drop_ws, L->drop_ws_bytes, stream, true, &defer_mask,
                           L->load);
      slots = L->k;
      Dp = 0;
    }
    if (rc == CAPMOE_OK && L->mode != 0 && L->max_experts > 0) {        // "w/ max": prune, then renumber the rows
      rc = capmoe_limit_experts(L->scores, L->N, L->E, L->max_experts, L->keep_mask, stream);
      if (rc != CAPMOE_OK) return rc;
      rc = capmoe_rows_from_mask(L->keep_mask, L->topk_idx, L->N, L->E, L->k, slots, expanded ? L->D : 1, nullptr,
                                 L->kept, L->expert_offsets, L->slot_row, L->bad, L->drop_ws, L->drop_ws_bytes,
                                 stream);
    }
  }
  if (rc != CAPMOE_OK) return rc;
  if (L->debug_checks && L->N > 0 &&
      (rc = capmoe_debug_check_indices(L->slot_row, L->topk_idx, L->expert_offsets, L->N, L->E, L->k, slots,
                                       Dp > 0 ? Dp : 1, nullptr, L->A_max, L->dev_status, stream)) != CAPMOE_OK)
    return rc;
  if ((rc = mark(2)) != CAPMOE_OK) return rc;
  rc = permute_impl(L->x, L->N, L->d, L->E, L->k, slots, Dp, L->dtype, L->scores, L->topk_idx, nullptr, L->slot_row,
                    L->x_perm, L->perm_token, L->perm_weight, defer_mask ? L->keep_mask : nullptr, stream);
  if (rc != CAPMOE_OK) return rc;
  if ((rc = mark(3)) != CAPMOE_OK) return rc;
  rc = grouped_ffn_impl(L->x_perm, L->expert_offsets, L->expert_offsets + 1, L->E, 0, L->d, L->F, L->dtype, L->w_gate,
                        L->w_up, L->w_down,
                        L->h_ws, L->y_perm, L->A_max, L->straggler ? L->D : 0, L->dev_status,
                        L->stage_events ? (cudaEvent_t)L->stage_events[4] : nullptr, stream, 0, true);
  if (rc != CAPMOE_OK) return rc;
  if (L->A_max == 0 && (rc = mark(4)) != CAPMOE_OK) return rc;
  if ((rc = mark(5)) != CAPMOE_OK) return rc;
  const void* y_shared = nullptr;
  if (L->F_shared > 0) {
    rc = grouped_ffn_impl(L->x, L->one_segment, L->one_segment + 1, 1, 0, L->d, L->F_shared, L->dtype, L->ws_gate,
                          L->ws_up, L->ws_down,
                          L->hs_ws, L->y_shared, L->N, 0, L->dev_status, nullptr, stream, 1, true);
    if (rc != CAPMOE_OK) return rc;
    y_shared = L->y_shared;
  }
  if ((rc = mark(6)) != CAPMOE_OK) return rc;
  rc = capmoe_combine(L->y_perm, L->slot_row, L->perm_weight, L->N, L->d, slots, L->dtype, y_shared, L->y,
                      stream);
  if (rc != CAPMOE_OK) return rc;
  return mark(7);
}

extern "C" int capmoe_layer_forward_host(const capmoe_layer* L, const void* x_host, void* y_host, void* stream) {
  if (!L || !x_host || !y_host) return CAPMOE_EINVAL;
  const size_t bytes = (size_t)L->N * L->d * elt_size(L->dtype);
  cudaStream_t st = as_stream(stream);
  cudaError_t err = cudaMemcpyAsync(const_cast<void*>(L->x), x_host, bytes, cudaMemcpyHostToDevice, st);
  if (err != cudaSuccess) return note_cuda(err);
  int rc = capmoe_layer_forward(L, stream);
  if (rc != CAPMOE_OK) return rc;
  err = cudaMemcpyAsync(y_host, L->y, bytes, cudaMemcpyDeviceToHost, st);
  return note_cuda(err);
}

namespace capmoe {
static std::atomic<int> g_ffn_variant{FFN_AUTO};
int ffn_variant() { return g_ffn_variant.load(std::memory_order_relaxed); }
}  // namespace capmoe

extern "C" int capmoe_debug_ffn_variant(int variant) {
  if (variant < capmoe::FFN_AUTO || variant > capmoe::FFN_SHORT_DOWN) return CAPMOE_EINVAL;
  capmoe::g_ffn_variant.store(variant, std::memory_order_relaxed);
  return CAPMOE_OK;
}

// ---------------------------------------------------------------------------------------------
// One rank of an expert-parallel group (see capmoe_ep_rank in the header).
namespace {
int validate_ep_rank(const capmoe_ep_rank* P) {
  if (!P) return CAPMOE_EINVAL;
  if (P->N < 0 || P->d < 1 || P->E < 1 || P->k < 1 || P->k > P->E || P->F < 1) return CAPMOE_EINVAL;
  if (P->dtype != CAPMOE_F32 && P->dtype != CAPMOE_BF16) return CAPMOE_EUNSUPPORTED;
  if (P->E > 256 || P->k > 32) return CAPMOE_EUNSUPPORTED;
  if (P->R < 1 || P->rank < 0 || P->rank >= P->R || P->E % P->R != 0) return CAPMOE_EINVAL;
  if (P->mode < 0 || P->mode > 2) return CAPMOE_EINVAL;
  if (P->C_local < 0 || P->C_local > P->N || P->C < P->C_local) return CAPMOE_EINVAL;
  if (P->mode == 0 && P->C_local != P->N) return CAPMOE_EINVAL;
  if ((int64_t)P->E * P->C >= ((int64_t)1 << 31)) return CAPMOE_EUNSUPPORTED;
  if (((size_t)P->d * elt_size(P->dtype)) % 16 != 0) return CAPMOE_EUNSUPPORTED;
  if (!P->logits || !P->scores || !P->topk_idx || !P->topk_score || !P->load || !P->kept || !P->expert_offsets ||
      !P->bad || !P->cnt_recv || !P->seg_begin || !P->seg_end)
    return CAPMOE_EINVAL;
  if (P->mode == 2 && (!P->cand || (P->N > 0 && !P->token_group))) return CAPMOE_EINVAL;
  if (P->N > 0 && (!P->x || !P->w_router || !P->keep_mask || !P->slot_row || !P->slot_row_ep || !P->y || !P->drop_ws))
    return CAPMOE_EINVAL;
  if (P->N > 0 && P->drop_ws_bytes < drop_ws_required(P->mode, P->N, P->E, P->k, P->mode == 2 ? P->R : 1))
    return CAPMOE_EWORKSPACE;
  if ((int64_t)P->E * P->C > 0) {
    if (!P->perm_token || !P->perm_weight || !P->x_recv || !P->h_ws || !P->y_recv || !P->w_gate || !P->w_up || !P->w_down)
      return CAPMOE_EINVAL;
    if (!P->peer_x && !P->x_send) return CAPMOE_EINVAL;
    if (!P->peer_y && !P->y_ret) return CAPMOE_EINVAL;
  }
  return CAPMOE_OK;
}
}  // namespace

extern "C" int capmoe_ep_forward_dispatch(const capmoe_ep_rank* P, void* stream) {
  int rc = validate_ep_rank(P);
  if (rc != CAPMOE_OK) return rc;
  cudaStream_t st = as_stream(stream);
  if ((rc = clear_words(P->load, P->E, P->bad, 1, st)) != CAPMOE_OK) return rc;
  rc = route_impl(P->x, P->w_router, P->bias, nullptr, P->N, P->d, P->E, P->k, P->dtype, P->logits, P->scores, P->topk_idx,
                  P->topk_score, P->load, stream, true);
  if (rc != CAPMOE_OK) return rc;
  const bool expanded = P->mode == 2;
  const int slots = expanded ? P->k + P->E / P->R : P->k;
  if (expanded)
    rc = expanded_drop_impl(P->scores, P->topk_idx, P->N, P->E, P->k, P->C_local, P->R, P->token_group, P->keep_mask, P->cand,
                            P->kept, P->expert_offsets, P->slot_row, P->drop_ws, P->drop_ws_bytes, stream, false, nullptr,
                            P->load);
  else
    rc = token_drop_impl(P->topk_score, P->topk_idx, P->N, P->E, P->k, P->C_local, P->keep_mask, P->kept, P->expert_offsets,
                         P->slot_row, P->drop_ws, P->drop_ws_bytes, stream, false, nullptr, P->load);
  if (rc != CAPMOE_OK) return rc;
  rc = capmoe_ep_plan(P->slot_row, P->topk_idx, P->expert_offsets, P->N, P->E, P->k, slots, expanded ? P->R : 1,
                      P->token_group, P->C, P->slot_row_ep, P->bad, stream);
  if (rc != CAPMOE_OK || P->N == 0 || (int64_t)P->E * P->C == 0) return rc;
  if (P->peer_x)
    return capmoe_ep_dispatch(P->x, P->N, P->d, P->E, P->k, slots, expanded ? P->R : 0, P->dtype, P->scores, P->topk_idx,
                              P->token_group, P->slot_row_ep, P->peer_x, P->R, P->rank, P->C, P->perm_token, P->perm_weight,
                              stream);
  return capmoe_permute(P->x, P->N, P->d, P->E, P->k, slots, expanded ? P->R : 0, P->dtype, P->scores, P->topk_idx,
                        P->token_group, P->slot_row_ep, P->x_send, P->perm_token, P->perm_weight, stream);
}

extern "C" int capmoe_ep_forward_experts(const capmoe_ep_rank* P, void* stream) {
  int rc = validate_ep_rank(P);
  if (rc != CAPMOE_OK) return rc;
  rc = capmoe_ep_segments(P->cnt_recv, P->E, P->C, P->seg_begin, P->seg_end, stream);
  if (rc != CAPMOE_OK || (int64_t)P->E * P->C == 0) return rc;
  return capmoe_grouped_ffn_segments(P->x_recv, P->seg_begin, P->seg_end, P->E, P->E / P->R, P->d, P->F, P->dtype, P->w_gate,
                                     P->w_up, P->w_down, P->h_ws, P->y_recv, (int64_t)P->E * P->C, P->dev_status, stream);
}

extern "C" int capmoe_ep_forward_combine(const capmoe_ep_rank* P, void* stream) {
  int rc = validate_ep_rank(P);
  if (rc != CAPMOE_OK) return rc;
  const int slots = P->mode == 2 ? P->k + P->E / P->R : P->k;
  if (P->peer_y && (int64_t)P->E * P->C > 0)
    return capmoe_ep_combine(P->peer_y, P->R, P->rank, P->E, P->C, P->slot_row_ep, P->perm_weight, P->N, P->d, slots,
                             P->dtype, nullptr, P->y, stream);
  return capmoe_combine(P->y_ret, P->slot_row_ep, P->perm_weight, P->N, P->d, slots, P->dtype, nullptr, P->y, stream);
}
