// Internal helpers of the capmoe CUDA library (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "capmoe.h"

namespace capmoe {

// Bookkeeping shared by the translation units (defined in api.cu).
void count_launch(int n = 1);
int note_cuda(cudaError_t err);            // records the text, returns CAPMOE_ECUDA or CAPMOE_OK
int check_launch();                        // cudaPeekAtLastError -> status, counts one launch
int sm_count();                            // SMs of the current device (cached per device)

// The stages as capmoe_layer_forward calls them.  With the last argument true the caller has
// itself issued, earlier on the stream, the small memsets the stage begins with (load histogram,
// drop counters: see drop_clear_counters): the stage skips them, and its first kernel chains onto
// the previous stage's last one.  Argument lists as in capmoe.h.  defer_mask (may be NULL): on entry
// true if the caller can derive keep_mask from slot_row itself later (permute_impl does); on return
// true if the stage left keep_mask unwritten for that reason.  load (may be NULL): the router's load
// histogram of the same top-k lists, which saves the stage a count.
int route_impl(const void* x, const void* w_router, const float* bias, const float* logits_in, int64_t N, int d, int E,
               int k, int dtype, float* logits, float* scores, int32_t* topk_idx, float* topk_score, int32_t* load,
               void* stream, bool load_cleared);
int token_drop_impl(const float* topk_score, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C,
                    uint64_t* keep_mask, int32_t* kept, int32_t* expert_offsets, int32_t* slot_row, void* ws,
                    size_t ws_bytes, void* stream, bool counters_cleared, bool* defer_mask, const int32_t* load);
int expanded_drop_impl(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C, int D,
                       const int32_t* token_group, uint64_t* keep_mask, int32_t* cand, int32_t* kept,
                       int32_t* expert_offsets, int32_t* slot_row, void* ws, size_t ws_bytes, void* stream,
                       bool counters_cleared, bool* defer_mask, const int32_t* load);
int device_drop_impl(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k, int64_t C_dev, int D,
                     int expanded, const int32_t* token_group, uint64_t* keep_mask, int32_t* cand, int32_t* kept,
                     int32_t* expert_offsets, int32_t* slot_row, void* ws, size_t ws_bytes, void* stream,
                     bool counters_cleared);
// Workspace bytes the drop stage of a layer forward in this mode will ask for (mode as in capmoe_layer).
size_t drop_ws_required(int mode, int64_t N, int E, int k, int D);
bool ffn_tc_supported(int d, int F, int dtype);
// The memsets of the drop stage that would run for these arguments (mode as in capmoe_layer).
int drop_clear_counters(int mode, int64_t N, int E, int k, int D, int32_t* cand, void* ws, size_t ws_bytes,
                        cudaStream_t st);
// keep_mask from slot_row (one thread per token); and the permute stage with the same derivation
// folded into its per-token bookkeeping (keep_mask_out may be NULL).
int drop_mask_from_rows(const int32_t* slot_row, const int32_t* topk_idx, int64_t N, int E, int k, int slots, int D,
                        const int32_t* token_group, uint64_t* keep_mask, cudaStream_t st);
int permute_impl(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype, const float* scores,
                 const int32_t* topk_idx, const int32_t* token_group, const int32_t* slot_row, void* x_perm,
                 int32_t* perm_token, float* perm_weight, uint64_t* keep_mask_out, void* stream);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t elt_size(int dtype) { return dtype == CAPMOE_F32 ? 4 : 2; }
inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Home device of token t: explicit table, or contiguous blocks floor(t*D/N).
__device__ __forceinline__ int home_group(int64_t t, int64_t N, int D, const int32_t* token_group) {
  return token_group ? token_group[t] : (int)((t * (int64_t)D) / N);
}

// Kernels that form a dependent chain on one stream are launched with programmatic stream
// serialisation: the launch of the next kernel is processed while its predecessor still runs, and
// its threads wait in wait_for_previous_kernel(), before touching memory, until the predecessor has
// finished and its writes are visible.  That removes most of the gap (about 3 us) between two
// dependent launches.  Without the launch attribute the wait is a no-op.
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Called first thing in every kernel: once all CTAs of this grid have started, the next kernel on
// the stream (if it was launched with the attribute above) may be scheduled onto free resources.  Its
// CTAs run up to their own wait_for_previous_kernel(), which still returns only when this whole
// grid has finished, so nothing it reads or writes moves ahead; what moves ahead is its launch
// latency and whatever set-up it does before the wait.
__device__ __forceinline__ void allow_next_kernel() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                  cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Which tensor-core FFN kernel serves a call: chosen from the shape (FFN_AUTO), or forced through
// capmoe_debug_ffn_variant (process-wide; tests run every variant on the same inputs with it).
enum { FFN_AUTO = 0, FFN_PAIR = 1, FFN_SINGLE = 2, FFN_SHORT = 3, FFN_SHORT_DOWN = 4 };
int ffn_variant();
int ffn_tc_short(bool gate_up, bool down, const void* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int n_w, int d, int F,
                 const void* w_gate, const void* w_up, const void* w_down, void* h_ws, void* y_perm, int64_t A_max,
                 int D_straggler, int32_t* dev_status, int32_t* sched1, int32_t* sched2, cudaEvent_t mid, cudaStream_t st);

// Zeroes up to two small int32 arrays with one chained kernel launch (a memset node between two
// kernels costs more stream time than this and breaks the chain of overlapped launches).
int clear_words(int32_t* a, int na, int32_t* b, int nb, cudaStream_t st);

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

}  // namespace capmoe
