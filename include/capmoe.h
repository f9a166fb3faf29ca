/* capmoe - capacity-aware Mixture-of-Experts layer forward on one NVIDIA B200 (sm_100a).
 *
 * One MoE layer (Eq. 1-2 of "Capacity-Aware Inference: Mitigating the Straggler Effect in
 * Mixture of Experts") with the paper's two capacity rules, as six stream-ordered stages:
 *
 *   capmoe_route          router GEMM, softmax, per-token top-k, expert load   (Eq. 1, Eq. 3)
 *   capmoe_token_drop     Capacity-Aware Token Drop                           (Eq. 7-10, Algorithm 1)
 *   capmoe_expanded_drop  Capacity-Aware Expanded Drop                        (Algorithm 2)
 *   capmoe_permute        gather kept tokens into expert-major rows
 *   capmoe_grouped_ffn    SwiGLU expert FFN over the per-expert row segments  (E_i(x) of Eq. 2)
 *   capmoe_combine        gate-weighted sum back to token order               (Eq. 2)
 *
 * Conventions, unless an entry point says otherwise
 *   - Pointers named in the argument lists are DEVICE pointers owned by the caller; the library
 *     allocates no device memory, keeps no per-call state and never synchronises the stream.
 *     `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - All tensors are dense, row-major, 16-byte aligned.  dtype selects the storage type of the
 *     activations and weights (CAPMOE_F32 or CAPMOE_BF16); logits, scores and gate weights are
 *     always fp32; accumulation is always fp32.
 *   - The return value is the only error channel (a capmoe_status as int).  Arguments are
 *     validated before anything is launched; on a non-zero return nothing was enqueued, except
 *     CAPMOE_ECUDA which reports a failed launch or driver call.
 *   - Every output is a deterministic function of the inputs (positions come from ordered
 *     prefix scans, integer atomics only where the result is order-independent).
 *   - Notation follows the paper: N tokens, hidden size d, E experts, k experts per token,
 *     capacity factor gamma, capacity C, D (virtual) expert-parallel devices with m = E/D
 *     experts each, F the expert FFN width, A the number of kept (token, expert) assignments.
 */
#ifndef CAPMOE_H_
#define CAPMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CAPMOE_OK = 0,
  CAPMOE_EINVAL = 1,       /* null / misaligned pointer, negative size, k > E, E % D != 0 ... */
  CAPMOE_EUNSUPPORTED = 2, /* well-formed request with no kernel (dtype, row size not 16-byte) */
  CAPMOE_EWORKSPACE = 3,   /* workspace smaller than capmoe_*_workspace_bytes reports        */
  CAPMOE_ECUDA = 4,        /* a CUDA call failed; see capmoe_last_cuda_error                   */
  CAPMOE_ETIMEOUT = 5,     /* a bounded device-side wait ran out (read from dev_status)       */
  CAPMOE_EINDEX = 6        /* debug check: a row index lies outside its buffer or segment (dev_status) */
} capmoe_status;

typedef enum { CAPMOE_F32 = 0, CAPMOE_BF16 = 1 } capmoe_dtype;
typedef enum { CAPMOE_CAP_CEIL = 0, CAPMOE_CAP_FLOOR = 1 } capmoe_round;

/* ---------------------------------------------------------------- host-only helpers */

/* Expert capacity C = gamma * N_bar with N_bar = N*k/E (Eq. 3; "Token Drop" paragraph),
 * evaluated as (gamma*(N*k))/E in double as Algorithm 1 does, rounded up (CAPMOE_CAP_CEIL,
 * default) or down (CAPMOE_CAP_FLOOR, the listing's int()), clamped to [0, N].  gamma = +inf
 * gives C = N, i.e. the layer without capacity limits.  Host pointer out. */
int capmoe_capacity(int64_t N, int E, int k, double gamma, int round, int64_t* C);

/* Upper bound on A (rows of the permuted matrix) known before routing:
 * min(E*C, N*k) for Token Drop, min(E*C, N*(k+E/D)) for Expanded Drop.  Host pointer out. */
int capmoe_max_rows(int64_t N, int E, int k, int D, int64_t C, int expanded, int64_t* A_max);

/* The same bound under device-level capacity (capmoe_device_drop with a per-device bound C_dev):
 * min(D*C_dev, N*k) or, with the expanded candidate set, min(D*C_dev, N*(k+E/D)).  Host pointer out. */
int capmoe_device_max_rows(int64_t N, int E, int k, int D, int64_t C_dev, int expanded, int64_t* A_max);

/* Scratch needed by capmoe_token_drop (expanded = 0) / capmoe_expanded_drop (expanded = 1). */
int capmoe_drop_workspace_bytes(int64_t N, int E, int k, int D, int expanded, size_t* bytes);

const char* capmoe_status_str(int status);
/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char* capmoe_last_cuda_error(void);
/* Number of kernels this library has launched in this process (all threads). */
uint64_t capmoe_launch_count(void);
/* 1 if grouped_ffn would take the tcgen05/TMA tensor-core path for this shape, else 0. */
int capmoe_ffn_uses_tensor_cores(int d, int F, int dtype);

/* ---------------------------------------------------------------- stage 1: router
 * logits[t,e] = sum_j x[t,j]*w_router[e,j] + bias[e]; scores = softmax(logits) per token;
 * top-k of the scores per token (Eq. 1; Algorithm 1, first three statements); load[e] = N_e,
 * the number of tokens whose top-k holds e (Eq. 3's N_i).
 *   x [N,d], w_router [E,d] in `dtype`; bias [E] fp32 or NULL.
 *   out: logits [N,E] fp32, scores [N,E] fp32, topk_idx [N,k] int32 (score descending, ties to
 *        the lower expert id), topk_score [N,k] fp32 (raw softmax values, not renormalised),
 *        load [E] int32.
 * The softmax is evaluated in binary32 in a fixed order (max; exp by range reduction and a
 * degree-7 polynomial in fma form; left-to-right sum; IEEE division), so scores are a pure
 * function of the fp32 logits.  logits_in, when not NULL, replaces the GEMM: the stage then
 * starts from the caller's fp32 logits [N,E] (x and w_router may be NULL).
 * Requires 1 <= k <= E <= 256, k <= 32. */
int capmoe_route(const void* x, const void* w_router, const float* bias, const float* logits_in,
                 int64_t N, int d, int E, int k, int dtype,
                 float* logits, float* scores, int32_t* topk_idx, float* topk_score, int32_t* load,
                 void* stream);

/* ---------------------------------------------------------------- stage 2: Token Drop
 * For every expert e, among the tokens whose top-k holds e keep the C with the highest score
 * (all of them if N_e <= C); equal scores go to the lower token index (Eq. 7-10, Algorithm 1).
 *   in : topk_score [N,k] fp32, topk_idx [N,k] int32, capacity C in [0,N].
 *   out: keep_mask [N, ceil(E/64)] uint64, bit (e%64) of word e/64 set iff (t,e) is kept;
 *        kept [E] int32 = min(N_e, C); expert_offsets [E+1] int32, exclusive prefix of kept
 *        (expert_offsets[E] = A); slot_row [N,k] int32 = row of the permuted matrix that holds
 *        top-k slot j of token t, or -1 if dropped.  Rows of expert e are
 *        [expert_offsets[e], expert_offsets[e+1]) in ascending token index.
 *   ws : capmoe_drop_workspace_bytes(N,E,k,0,0) bytes, contents undefined on entry and exit.
 * C = N is the layer without dropping. */
int capmoe_token_drop(const float* topk_score, const int32_t* topk_idx, int64_t N, int E, int k,
                      int64_t C, uint64_t* keep_mask, int32_t* kept, int32_t* expert_offsets,
                      int32_t* slot_row, void* ws, size_t ws_bytes, void* stream);

/* Token Drop without caller-provided scratch.  The paper has no counterpart: this entry point
 * exists for callers that can neither allocate device memory nor carve a workspace out of memory
 * they own - a serving runtime whose memory pool is fixed at start-up, a host that forbids
 * allocation after initialisation, or a language binding that only holds the input and output
 * tensors.  Same inputs, outputs and results as capmoe_token_drop; the scratch is a fixed array in
 * device memory that the library owns (about 12 MiB on every GPU that loads the library, held
 * until the process exits).
 *   - Limit: N*k <= CAPMOE_STATIC_DROP_MAX_PAIRS; larger calls return CAPMOE_EWORKSPACE and
 *     launch nothing.
 *   - It calls no cudaMalloc/cudaFree and no allocating library routine.  The first call on each
 *     device looks up the array's device address (the device must be current); make that first
 *     call outside of any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents: the
 *     call clears the part that has to start at zero itself, but two calls that overlap on the
 *     GPU (different streams, or several host threads) race on it.  Serialise them.
 *   - Whatever the batch size it runs the select with one thread block per expert, which walks
 *     all N tokens; from a few ten thousand tokens on capmoe_token_drop, which spreads the select
 *     over the whole GPU, is several times faster. */
#define CAPMOE_STATIC_DROP_MAX_PAIRS (1 << 20)
int capmoe_token_drop_static(const float* topk_score, const int32_t* topk_idx, int64_t N, int E, int k,
                             int64_t C, uint64_t* keep_mask, int32_t* kept, int32_t* expert_offsets,
                             int32_t* slot_row, void* stream);

/* ---------------------------------------------------------------- stage 3: Expanded Drop
 * Token t is a candidate of its top-k experts and of all m = E/D experts of its home device
 * h(t); all candidates of an expert compete on scores[t,e]; the expert keeps its C best, ties
 * to the lower token index (Algorithm 2).  A token may end with more than k experts.
 *   in : scores [N,E] fp32, topk_idx [N,k], C, D (E % D == 0), token_group [N] int32 with
 *        h(t) in [0,D) or NULL for contiguous blocks h(t) = floor(t*D/N).
 *   out: keep_mask, kept, expert_offsets as above; cand [E] int32 = candidates per expert;
 *        slot_row [N, k+m] int32: slots 0..k-1 are the top-k slots, slot k+i is local expert
 *        h(t)*m+i when it is not one of the token's top-k (else -1).
 *   ws : capmoe_drop_workspace_bytes(N,E,k,D,1) bytes. */
int capmoe_expanded_drop(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k,
                         int64_t C, int D, const int32_t* token_group, uint64_t* keep_mask,
                         int32_t* cand, int32_t* kept, int32_t* expert_offsets, int32_t* slot_row,
                         void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------- drop metrics
 * The Token Drop paragraph names four ways to rank the tokens an overloaded expert received:
 * Score (the gating score, the default), Order (later tokens are discarded once earlier ones
 * filled the capacity), Reverse Order (earlier tokens are removed) and Random (every token has
 * the same chance).  capmoe_drop_keys turns a metric into one 32-bit key per entry; the drop
 * stages compare their score input by bit pattern (larger = kept first, equal = lower token
 * index first), so the key array, passed where capmoe_token_drop expects topk_score [N,k] or
 * capmoe_expanded_drop / capmoe_device_drop expect scores [N,E], selects by that metric.  The
 * gate weights of the kept rows still come from the real scores (stage 4).
 *   scores [N,cols] fp32 (read for CAPMOE_METRIC_SCORE only), idx [N,cols] expert ids or NULL when
 *   cols == E and column c is expert c; keys [N,cols] uint32 out.
 *   Random keys are the high word of a 64-bit mix of (seed, t*E + e): a pure function of the
 *   seed and the (token, expert) position. */
typedef enum {
  CAPMOE_METRIC_SCORE = 0, CAPMOE_METRIC_ORDER = 1, CAPMOE_METRIC_REVERSE_ORDER = 2, CAPMOE_METRIC_RANDOM = 3
} capmoe_metric;
int capmoe_drop_keys(int metric, uint64_t seed, const float* scores, const int32_t* idx, int64_t N, int cols,
                     int E, uint32_t* keys, void* stream);

/* ---------------------------------------------------------------- device-level capacity
 * The paper's "Advanced Variant: Device-Level Capacity-Aware Inference": the bound applies to the
 * aggregated load of a device, N_1 + ... + N_{n_l} <= C_dev = n_l * gamma * N_bar, not to each
 * expert.  capmoe_device_capacity evaluates (gamma*(N*k))/D like capmoe_capacity (host pointer
 * out; clamped to [0, N*E/D]).  capmoe_device_drop keeps, per device, the C_dev best of all
 * (token, expert) pairs whose expert lives on it - the top-k pairs, plus every pair of the token's
 * home device when expanded != 0 (the candidate set of Expanded Drop) - by scores[t,e]; equal scores
 * go to the lower token index and, inside a token, to the lower expert id.  Outputs have the
 * layout of stages 2/3 (slot_row [N,k] or [N,k+E/D]; rows expert-major, token-ascending).
 * ws: capmoe_drop_workspace_bytes(N,E,k,D,expanded) bytes. */
int capmoe_device_capacity(int64_t N, int E, int k, int D, double gamma, int round, int64_t* C_dev);
int capmoe_device_drop(const float* scores, const int32_t* topk_idx, int64_t N, int E, int k,
                       int64_t C_dev, int D, int expanded, const int32_t* token_group,
                       uint64_t* keep_mask, int32_t* cand, int32_t* kept, int32_t* expert_offsets,
                       int32_t* slot_row, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------- priority classes, "w/ max"
 * capmoe_priority_keys puts a priority class above a metric's key, for the two variants that
 * rank candidates by a class before the metric:
 *   - dropping by modality (multimodal section: "Image First" drops image tokens before any text
 *     token, "Text First" the other way round): token_class[t] = 1 for the protected modality;
 *   - Expanded Drop as substitution only (Expanded Drop paragraph: the expansion "makes no change
 *     in the token assignments in experts that are overflowed by the top-k"): pass topk_idx and a
 *     token's top-k pairs outrank the pairs it only has through its home device.  Without this
 *     class all candidates compete equally, as in Algorithm 2.
 * keys[i] = ((2*[pair is a top-k pair] + token_class[t]) << 30) | body, body = base[i] when exact != 0
 * (the caller guarantees base < 2^30, true of every score in [0,1]; higher bits are masked off)
 * else base[i] >> 2.  base/keys [N,cols] uint32 (may alias); idx as in capmoe_drop_keys;
 * token_class [N] uint8 or NULL; topk_idx [N,k] or NULL.
 *
 * capmoe_limit_experts is the "w/ max" ablation (appendix "Maximum Number of Selected Experts"):
 * every token retains at most k_max of the experts that kept it, the best by scores[t,e], ties to
 * the lower expert id; keep_mask [N, ceil(E/64)] is edited in place, freed capacity is not handed
 * on.  capmoe_rows_from_mask then rebuilds kept [E], expert_offsets [E+1] and slot_row [N,slots]
 * (slots = k, or k + E/D with the home-device slots of stage 3) for that mask - or for any mask
 * whose bits lie on the token's slots; *bad (device int32) is set to 1 if one does not, else 0.
 * ws: ceil(N/256)*E*4 bytes (capmoe_drop_workspace_bytes(...) is enough).
 * Global expansion (candidates = the token's k+m best experts anywhere) needs no call of its own:
 * capmoe_route with k+m choices followed by capmoe_token_drop. */
int capmoe_priority_keys(const uint32_t* base, const int32_t* idx, int64_t N, int cols, int E, int exact,
                         const uint8_t* token_class, const int32_t* topk_idx, int k, uint32_t* keys,
                         void* stream);
int capmoe_limit_experts(const float* scores, int64_t N, int E, int k_max, uint64_t* keep_mask,
                         void* stream);
int capmoe_rows_from_mask(const uint64_t* keep_mask, const int32_t* topk_idx, int64_t N, int E, int k,
                          int slots, int D, const int32_t* token_group, int32_t* kept,
                          int32_t* expert_offsets, int32_t* slot_row, int32_t* bad, void* ws,
                          size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------- stage 4: permute
 * x_perm[r] = x[t], perm_token[r] = t, perm_weight[r] = scores[t,e] for every kept (t,e) with
 * r = its slot_row entry.  slots = k after Token Drop (pass D = 0) or k+E/D after Expanded Drop.
 *   in : x [N,d] `dtype`, scores [N,E] fp32, topk_idx [N,k], token_group (as in stage 3),
 *        slot_row [N,slots].
 *   out: x_perm [A,d] `dtype`, perm_token [A] int32, perm_weight [A] fp32 (A rows written).
 * Requires d*sizeof(elt) to be a multiple of 16. */
int capmoe_permute(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype,
                   const float* scores, const int32_t* topk_idx, const int32_t* token_group,
                   const int32_t* slot_row, void* x_perm, int32_t* perm_token, float* perm_weight,
                   void* stream);

/* ---------------------------------------------------------------- stage 5: grouped SwiGLU FFN
 * For every expert e and every row r in [expert_offsets[e], expert_offsets[e+1]):
 *   h = silu(W_g[e] x_perm[r]) * (W_u[e] x_perm[r]),  y_perm[r] = W_d[e] h      (E_i(x) in Eq. 2).
 *   in : x_perm [A_max,d], expert_offsets [E+1] (device), w_gate, w_up [E,F,d], w_down [E,d,F].
 *   ws : h_ws [A_max,F] in `dtype` (the hidden activations; contents undefined afterwards).
 *   out: y_perm [A_max,d] in `dtype`; rows >= expert_offsets[E] are left untouched.
 * A_max is the allocated row count of x_perm / h_ws / y_perm (>= A).  No host-device sync:
 * tiles are scheduled on the device from expert_offsets.
 * D_straggler > 0 (E % D_straggler == 0) turns on straggler emulation: the experts of virtual
 * device g run only on a fixed share floor(#SM/D) of the SMs, so the most loaded device sets
 * the latency as under expert parallelism (Eq. 4, L proportional to max_i N_i).
 * dev_status: NULL, or a device block of CAPMOE_FFN_STATUS_WORDS int32.  Word 0 is set to
 * CAPMOE_ETIMEOUT if a bounded wait inside the tensor-core kernel ran out; the caller zeroes it
 * and reads it after synchronising.  The other words are scratch that the call itself clears: the
 * tile counters from which the kernels take their work in list order (so that tiles sharing an
 * operand run at the same time whatever the speed of their SMs); with NULL, or more than
 * CAPMOE_FFN_SCHED_GROUPS straggler groups, every CTA walks a fixed list of tiles instead.  Calls
 * that overlap on the GPU need a block each.
 * bf16 with d % 64 == 0 and F % 64 == 0 runs on tcgen05 tensor cores with TMA-fed tiles (the last
 * 128-column block of the gate/up GEMM is half filled when F is an odd multiple of 64); everything
 * else (fp32, odd shapes) runs a plain fp32-FMA kernel, which has no straggler emulation
 * (D_straggler > 0 then returns CAPMOE_EUNSUPPORTED).  capmoe_ffn_uses_tensor_cores tells which. */
#define CAPMOE_FFN_SCHED_GROUPS 62
#define CAPMOE_FFN_STATUS_WORDS (1 + 2 * CAPMOE_FFN_SCHED_GROUPS + 3)   /* 128: status, counters of the routed
                                                                           experts' two GEMMs, two counters for
                                                                           the layer's shared expert, one spare */
int capmoe_grouped_ffn(const void* x_perm, const int32_t* expert_offsets, int E, int d, int F,
                       int dtype, const void* w_gate, const void* w_up, const void* w_down,
                       void* h_ws, void* y_perm, int64_t A_max, int D_straggler,
                       int32_t* dev_status, void* stream);

/* The same stage over explicit row segments: segment s holds the rows [seg_begin[s], seg_end[s]) of
 * x_rows (seg_begin, seg_end: device int32 [S], non-overlapping, ascending) and is multiplied with
 * weight block s % w_mod of w_gate / w_up [w_mod,F,d] and w_down [w_mod,d,F] (w_mod = 0: block s of
 * S).  This is the form the owner of a few experts runs under expert parallelism, where every
 * (source rank, local expert) pair is a segment of at most C_local rows at a fixed place (see
 * capmoe_ep_segments).  rows = allocated rows of x_rows / h_ws / y_rows; rows outside every segment
 * are neither read into a result nor written.  dev_status as above (no straggler emulation here). */
int capmoe_grouped_ffn_segments(const void* x_rows, const int32_t* seg_begin, const int32_t* seg_end, int S,
                                int w_mod, int d, int F, int dtype, const void* w_gate, const void* w_up,
                                const void* w_down, void* h_ws, void* y_rows, int64_t rows,
                                int32_t* dev_status, void* stream);

/* ---------------------------------------------------------------- expert parallelism
 * The paper's deployment (experimental set-up: data parallel over the tokens, expert parallel over
 * the experts) with the capacity applied "within each local device" (Capacity-Aware Token Drop
 * paragraph), so that tokens are "discarded prior to All-to-All" (Figure 3) and no rank needs to
 * know another rank's load: rank r of R routes and drops its own N_local tokens with
 * C_local = capmoe_capacity(N_local, E, k, gamma) - stages 1 to 3 unchanged, Expanded Drop with
 * D = R and every token's home device = r - and owns the m = E/R experts r*m .. r*m+m-1.
 * Because a rank keeps at most C_local rows per expert, every message has a fixed place and a
 * fixed bound: the row space of a rank is [E][C_local] (row e*C_local + i = the i-th kept row of
 * expert e, token-ascending), its block [r'*m*C_local, (r'+1)*m*C_local) goes to rank r', and the
 * owner receives [R][m][C_local] rows (source-major).  No counts cross the host.
 *
 * capmoe_ep_plan      slot_row (rows of the packed matrix, stages 2/3) -> slot_row_ep (rows of the
 *                     [E][C_local] space, or -1); *bad (device int32) is set to 1 if an expert holds
 *                     more than C_local rows.  The send counts are the stage's kept[E].
 * capmoe_permute / capmoe_combine with slot_row_ep and [E*C_local, d] buffers then fill the send
 *                     buffer and read the returned rows when the exchange is a collective (two
 *                     equal-split all-to-alls each way: rows and counts).
 * capmoe_ep_dispatch  the permute stage writing each kept row straight into its owner's receive
 *                     buffer: peer_rows[r'] (device array of R addresses) = base of rank r''s
 *                     [R*m*C_local, d] buffer, mapped into this process (peer access within a node);
 *                     this rank's rows land in block `rank` of it.  perm_token / perm_weight
 *                     [E*C_local] stay local.  Plain stores, no multicast.
 * capmoe_ep_segments  counts [R*m] (received: kept of (source, local expert)) -> seg_begin / seg_end
 *                     of the R*m segments for capmoe_grouped_ffn_segments (w_mod = m).
 * capmoe_ep_combine   the combine stage reading each kept row's result straight from its owner's
 *                     [R*m*C_local, d] output buffer (peer_rows as above).
 * The caller orders the ranks (all rows and counts have arrived before the owner's FFN starts, all
 * results are written before a combine reads them); no kernel of this library waits for another rank. */
int capmoe_ep_plan(const int32_t* slot_row, const int32_t* topk_idx, const int32_t* expert_offsets, int64_t N,
                   int E, int k, int slots, int D, const int32_t* token_group, int64_t C_local,
                   int32_t* slot_row_ep, int32_t* bad, void* stream);
int capmoe_ep_segments(const int32_t* counts, int S, int64_t C_local, int32_t* seg_begin, int32_t* seg_end,
                       void* stream);
int capmoe_ep_dispatch(const void* x, int64_t N, int d, int E, int k, int slots, int D, int dtype,
                       const float* scores, const int32_t* topk_idx, const int32_t* token_group,
                       const int32_t* slot_row_ep, const uint64_t* peer_rows, int R, int rank,
                       int64_t C_local, int32_t* perm_token, float* perm_weight, void* stream);
int capmoe_ep_combine(const uint64_t* peer_rows, int R, int rank, int E, int64_t C_local,
                      const int32_t* slot_row_ep, const float* perm_weight, int64_t N, int d, int slots,
                      int dtype, const void* y_shared, void* y, void* stream);

/* One rank's forward under expert parallelism, in the three phases between which the caller orders
 * the ranks.  Every pointer is a device pointer; sizes in brackets.
 *   capmoe_ep_forward_dispatch  stages 1-3 on the rank's own N tokens with C_local (mode 1 = Token Drop,
 *                               2 = Expanded Drop with D = R and every token at home on `rank`, 0 = no
 *                               drop, C_local = N), capmoe_ep_plan with row stride C (>= C_local, the same
 *                               on all ranks), then the rows go out: into the owners' x_recv buffers
 *                               through peer_x (a table of R addresses), or, with peer_x == NULL, into
 *                               this rank's send buffer x_send for an all-to-all.  kept [E] = [R][m] are
 *                               the counts the owners need (cnt_recv block `rank` of owner r').
 *   capmoe_ep_forward_experts   the owner's part, once rows (x_recv) and counts (cnt_recv [R*m]) of all
 *                               ranks have arrived: segments, SwiGLU FFN with the rank's own m experts,
 *                               results in y_recv.
 *   capmoe_ep_forward_combine   once all owners are done: Eq. 2 for the rank's tokens, reading the
 *                               results through peer_y, or, with peer_y == NULL, from y_ret (the
 *                               all-to-all's output).  Writes y [N,d].
 * All fields are checked before anything is enqueued.  dev_status [CAPMOE_FFN_STATUS_WORDS] and
 * bad [1] report as in capmoe_grouped_ffn / capmoe_ep_plan. */
typedef struct {
  int64_t N; int d, E, k, F, dtype;
  int R, rank, mode;           /* mode: 0 no drop, 1 Token Drop, 2 Expanded Drop */
  int64_t C_local, C;          /* the rank's capacity; the row stride all ranks agreed on */
  const void* x; const void* w_router; const float* bias;
  const void* w_gate; const void* w_up; const void* w_down;            /* this rank's m = E/R experts */
  float* logits; float* scores; int32_t* topk_idx; float* topk_score; int32_t* load;   /* [N,E] .. [E] */
  uint64_t* keep_mask; int32_t* cand; int32_t* kept; int32_t* expert_offsets; int32_t* slot_row;
  int32_t* slot_row_ep;        /* [N, slots] rows of the [E][C] space */
  const int32_t* token_group;  /* [N] filled with `rank` (mode 2), else NULL */
  int32_t* perm_token; float* perm_weight;                              /* [E*C] */
  void* x_send; void* y_ret;                                            /* [E*C, d]: collective transport */
  const uint64_t* peer_x; const uint64_t* peer_y;                       /* [R] addresses: peer transport */
  void* x_recv; void* h_ws; void* y_recv;                               /* [R*m*C, d], [.., F], [.., d] */
  int32_t* cnt_recv; int32_t* seg_begin; int32_t* seg_end;              /* [R*m] */
  void* y;                                                              /* [N, d] */
  void* drop_ws; size_t drop_ws_bytes;
  int32_t* dev_status; int32_t* bad;
} capmoe_ep_rank;
int capmoe_ep_forward_dispatch(const capmoe_ep_rank* P, void* stream);
int capmoe_ep_forward_experts(const capmoe_ep_rank* P, void* stream);
int capmoe_ep_forward_combine(const capmoe_ep_rank* P, void* stream);

/* Which tensor-core kernel capmoe_grouped_ffn* and the layer forward use for bf16 shapes, for the whole
 * process: 0 = chosen from the shape (the default), 1 = CTA pairs with 256-token tiles, 2 = one CTA per
 * 128-token tile, 3 = the short-segment form (256 weight rows x up to 256 tokens per pair, tokens in
 * steps of 16), 4 = that form for the down GEMM only, behind the gate/up kernel the shape selects.  All compute the same thing (Eq. 2's experts); tests force each on the same inputs.
 * A variant the device cannot run (fewer than two SMs per straggler group) returns
 * CAPMOE_EUNSUPPORTED at the next FFN call.  Not stream-ordered: set it while no FFN call is being issued. */
int capmoe_debug_ffn_variant(int variant);

/* Self-test of the bounded device-side wait used inside the tensor-core kernels (no counterpart
 * in the paper).  Launches one warp that waits on a barrier nothing will ever signal, with the
 * same wait routine and a limit of limit_cycles SM clock cycles (1 .. 4e9); the wait must run
 * out, the kernel must return normally and *dev_status must read CAPMOE_ETIMEOUT afterwards
 * (the caller zeroes it first).  The context stays usable. */
int capmoe_debug_wait_probe(int64_t limit_cycles, int32_t* dev_status, void* stream);

/* Debug check of the indices the later stages will use as addresses (no counterpart in the paper;
 * the stand-in for a memory checker on machines where none can run).  Reads only: expert_offsets must
 * be non-decreasing with expert_offsets[E] <= A_max, and every slot_row[t,s] must be -1 or lie inside
 * the segment of the expert the slot stands for (slots = k, or k + E/D with the home-device slots).
 * On a violation *dev_status is set to CAPMOE_EINDEX (never a trap); the caller zeroes it first and
 * reads it after synchronising.  capmoe_layer_forward runs it after the drop stage when the struct's
 * debug_checks field is non-zero. */
int capmoe_debug_check_indices(const int32_t* slot_row, const int32_t* topk_idx, const int32_t* expert_offsets,
                               int64_t N, int E, int k, int slots, int D, const int32_t* token_group,
                               int64_t A_max, int32_t* dev_status, void* stream);

/* Measurement aid (no counterpart in the paper): one launch that reads `bytes` bytes from p once,
 * as fast as plain loads go, and does nothing else.  Its device time is the floor for any kernel
 * that has to read that much from HBM once, launch included - for the few ten megabytes of a small
 * batch that floor is well below the bandwidth of a long copy, which is what the bandwidth-bound
 * stages are otherwise compared with.  p: device, 16-byte aligned; sink: device int32 or NULL. */
int capmoe_debug_read_probe(const void* p, size_t bytes, int32_t* sink, void* stream);

/* ---------------------------------------------------------------- stage 6: combine
 * y[t] = sum over slots s with slot_row[t,s] >= 0 of perm_weight[row] * y_perm[row], added in
 * ascending slot order in fp32, plus y_shared[t] (weight 1) when y_shared is not NULL; a token
 * with nothing kept gets y_shared[t] or zeros (Eq. 2 with the kept set in place of K).
 *   in : y_perm [A,d] `dtype`, slot_row [N,slots], perm_weight [A] fp32, y_shared [N,d] or NULL.
 *   out: y [N,d] `dtype`. */
int capmoe_combine(const void* y_perm, const int32_t* slot_row, const float* perm_weight,
                   int64_t N, int d, int slots, int dtype, const void* y_shared, void* y,
                   void* stream);

/* ---------------------------------------------------------------- whole layer
 * Buffers for one layer forward.  Every pointer is a device pointer sized as noted. */
typedef struct {
  /* problem */
  int64_t N; int d, E, k, F, D, dtype;
  int mode;              /* 0 = no drop (C = N), 1 = Token Drop, 2 = Expanded Drop,
                            3 / 4 = Token / Expanded Drop candidates under device-level capacity */
  int64_t C;             /* capacity per expert (modes 1, 2) or per device (modes 3, 4); ignored for mode 0 */
  int straggler;         /* 0/1: run the FFN in straggler-emulation mode over D devices */
  /* inputs */
  const void* x; const void* w_router; const float* bias;
  const void* w_gate; const void* w_up; const void* w_down;
  const void* ws_gate; const void* ws_up; const void* ws_down; int F_shared; /* shared expert or NULL/0 */
  /* outputs and intermediates */
  float* logits; float* scores; int32_t* topk_idx; float* topk_score; int32_t* load;
  uint64_t* keep_mask; int32_t* cand; int32_t* kept; int32_t* expert_offsets; int32_t* slot_row;
  void* x_perm; int32_t* perm_token; float* perm_weight;
  void* h_ws; void* y_perm; int64_t A_max;
  void* hs_ws; void* y_shared;  /* shared expert scratch: [N,F_shared], [N,d] */
  const int32_t* one_segment;   /* [2] int32 holding {0, N}: the shared expert's single row segment */
  void* y;
  void* drop_ws; size_t drop_ws_bytes;
  int32_t* dev_status;   /* CAPMOE_FFN_STATUS_WORDS int32, see capmoe_grouped_ffn */
  /* Optional stage timing.  NULL, or CAPMOE_N_STAGE_EVENTS cudaEvent_t handles (as void*) that the
   * layer records on `stream`: [0] start, [1] after route, [2] after drop, [3] after permute,
   * [4] after the gate/up GEMM + SwiGLU, [5] after the down GEMM, [6] after the shared expert,
   * [7] after combine. */
  void** stage_events;
  /* Variants of the drop for modes 1 and 2 (all zero / NULL = the default reading: Score metric,
   * equal competition, no limit on experts per token).  See capmoe_drop_keys,
   * capmoe_priority_keys, capmoe_limit_experts. */
  int metric;                  /* capmoe_metric */
  uint64_t metric_seed;        /* CAPMOE_METRIC_RANDOM */
  const uint8_t* token_class;  /* [N] or NULL: 1 = token of the protected modality (modality-first dropping) */
  int topk_first;              /* mode 2: a token's top-k pairs outrank its home-device-only pairs */
  int max_experts;             /* > 0: every token retains at most this many experts ("w/ max") */
  float* drop_keys;            /* scratch for the keys, [N,k] (mode 1) or [N,E] (mode 2) 32-bit words; needed
                                  unless metric is Score, token_class is NULL and topk_first is 0 */
  int32_t* bad;                /* device int32, needed when max_experts > 0 (see capmoe_rows_from_mask) */
  int debug_checks;            /* non-zero: run capmoe_debug_check_indices after the drop (needs dev_status) */
} capmoe_layer;
#define CAPMOE_N_STAGE_EVENTS 8

/* Runs the stages above in order on `stream` (route, drop, permute, FFN, [shared FFN], combine).
 * Every field is checked before the first event record, memset or launch: missing pointers for the
 * chosen mode and variants (CAPMOE_EINVAL), E % D, capacities out of range, a drop workspace below
 * what the mode needs or A_max below the row bound of the mode (capmoe_max_rows /
 * capmoe_device_max_rows; N*k without dropping) (CAPMOE_EWORKSPACE), straggler emulation off the
 * tensor-core path (CAPMOE_EUNSUPPORTED).  x_perm, h_ws and y_perm must hold A_max rows. */
int capmoe_layer_forward(const capmoe_layer* L, void* stream);

/* Same, with the activations on the HOST: copies x_host [N,d] (pinned) to L->x, runs the layer,
 * copies L->y to y_host [N,d] (pinned), all on `stream`; weights stay resident on the device.
 * L->x is used as the device staging buffer and must be writable. */
int capmoe_layer_forward_host(const capmoe_layer* L, const void* x_host, void* y_host, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CAPMOE_H_ */
