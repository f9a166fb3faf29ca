// Stage 5, tensor-core path for SHORT expert segments: the grouped SwiGLU FFN with the operand
// roles exchanged.  The kernels of ffn_tc.cu put tokens on the M side of the MMA (128 or 256 rows per
// tile), so a segment of a few hundred rows pays for the padding of its last tile in tensor time.
// Here the WEIGHTS are the M side and the tokens the N side, which tcgen05.mma takes in steps of 16:
//   GEMM1  H^T[f, t]      = silu(W_g[e,f,:] . x_perm[t,:]) * (W_u[e,f,:] . x_perm[t,:])
//   GEMM2  y_perm^T[j, t] = W_d[e,j,:] . H[t,:]
// A tile is 256 weight rows (128 per CTA of a pair, cta_group::2, M = 256) by up to 256 tokens
// (N = the tile's token count rounded up to 16; each CTA loads half of them).  Every weight tile
// passes through the pair's shared memory once per 256 tokens of its segment, which is what bounds
// these launches: they move far more bytes from L2 to the SMs than from DRAM.  GEMM1 issues two MMAs
// per k-step on the same token tile, one with the W_g rows and one with the W_u rows, into two
// accumulators 256 columns apart, so a thread of the epilogue finds gate and up of its (f, t) in its
// own TMEM lane; that fills tensor memory, so GEMM1's next tile starts its MMAs when the epilogue has
// read the accumulators (its loads run ahead meanwhile).  GEMM2's accumulators ping-pong between the
// two 256-column halves.
// The epilogue transposes through shared memory: a warp holds 32 weight rows (lanes) by 32 tokens
// (columns), writes them as a 32-token x 32-column bf16 box and stores the box by TMA when all 32
// tokens are inside the segment, else element by element.
// Pipeline, tile queue, bounded waits and the straggler partition are those of k_ffn_tc2.
#include "tc_common.cuh"

namespace capmoe {
namespace {

constexpr int TT_MAX = 256;                   // tokens per tile at most (MMA N)
constexpr int TT_HALF = TT_MAX / 2;           // token rows one CTA loads per k-block
constexpr int WT = 256;                       // weight rows (output columns) per tile, 128 per CTA
constexpr int RING_BYTES = STAGES * STAGE_BYTES;
constexpr int TB_BYTES = TT_HALF * BK * 2;    // 16 KB: one CTA's half of the token tile
template <bool SWIGLU> struct StageT {
  static constexpr int W_BYTES = (SWIGLU ? 2 : 1) * A_BYTES;       // 128 rows of W_g and of W_u, or of W_d
  static constexpr int BYTES = W_BYTES + TB_BYTES;                 // 48 KB / 32 KB per CTA
  static constexpr int N = RING_BYTES / BYTES;                     // 4 / 6 stages
};
static_assert(StageT<true>::N >= 3 && StageT<false>::N <= MAX_STAGES, "ring depth");
static_assert(StageT<true>::BYTES % 1024 == 0 && StageT<false>::BYTES % 1024 == 0, "swizzle atoms stay aligned");

struct TileT { int e, row0, rows, nt, w0; };   // segment, first token row, tokens, MMA N, first weight row

// Tiles of a segment: token block fastest, then weight block (the pairs that run side by side then
// share one weight tile through L2 and differ in their tokens).
__device__ __forceinline__ bool locate_tile_t(int tile, int& cursor, const int* tile_start, const int* offs,
                                              const int* ends, int E, TileT& t) {
  while (cursor < E && tile >= tile_start[cursor + 1]) ++cursor;
  if (cursor >= E) return false;
  const int local = tile - tile_start[cursor];
  const int cnt = ends[cursor] - offs[cursor];
  const int ntb = (cnt + TT_MAX - 1) / TT_MAX;
  const int wb = local / ntb, tb = local - wb * ntb;
  t.e = cursor;
  t.row0 = offs[cursor] + tb * TT_MAX;
  t.rows = min(TT_MAX, cnt - tb * TT_MAX);
  t.nt = (t.rows + 15) & ~15;
  t.w0 = wb * WT;
  return true;
}

template <int MODE>
__global__ void __launch_bounds__(TC_THREADS, 1)
k_ffn_tc2t(const __grid_constant__ CUtensorMap map_x /* token rows, box 128 x 64 */,
           const __grid_constant__ CUtensorMap map_w0 /* W_g or W_d, box 128 x 64, 3-D */,
           const __grid_constant__ CUtensorMap map_w1 /* W_u */, const __grid_constant__ CUtensorMap map_out /* the
           output as 32 x 32 boxes */, const int32_t* __restrict__ seg_begin, const int32_t* __restrict__ seg_end, int w_mod,
           int E, int K, int Nout, __nv_bfloat16* __restrict__ out, int D_straggler, int32_t* __restrict__ dev_status,
           int32_t* __restrict__ sched) {
  constexpr bool SWIGLU = MODE == 0;
  using SG = StageT<SWIGLU>;
  constexpr int NST = SG::N;
  allow_next_kernel();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + TAIL_OFF);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* offs = reinterpret_cast<int*>(gen + TAIL_OFF + 512);
  int* tile_start = offs + (MAX_E + 1);
  int* ends = reinterpret_cast<int*>(reinterpret_cast<float*>(tile_start + (MAX_E + 1) + 2) + 256 + RF_XCH_FLOATS);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();                      // 0 = leader (issues the MMAs)
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(MAX_STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (uint32_t)(2 * MAX_STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (uint32_t)(2 * MAX_STAGES + 2 + b); };
  const TileQueue<true> tq{bar0 + 8u * 40u, bar0 + 8u * 44u, bar0 + 8u * 48u, rank, abort_flag};

  // set-up that touches no global memory comes before the wait for the previous kernel
  if (tid == 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w0) : "memory");
    if (SWIGLU) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w1) : "memory");
  }
  if (tid == 0) {
    for (int s = 0; s < NST; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 2 * EPI_WARPS * 32); }
    for (int i = 0; i < TQ; ++i) { mbar_init(tq.full(i), 1); mbar_init(tq.empty(i), TQ_READERS_PAIR); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  wait_for_previous_kernel();
  for (int i = tid; i < E; i += TC_THREADS) { offs[i] = seg_begin[i]; ends[i] = seg_end[i]; }
  __syncthreads();
  if (tid == 0) {
    const int w_blocks = (Nout + WT - 1) / WT;
    int acc = 0;
    for (int e = 0; e < E; ++e) {
      tile_start[e] = acc;
      acc += ((ends[e] - offs[e] + TT_MAX - 1) / TT_MAX) * w_blocks;
    }
    tile_start[E] = acc;
  }
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();             // the peer's barriers are initialised and its tensor memory allocated
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  int tile_lo, tile_hi, stride, first;
  int32_t* counter = sched;
  if (D_straggler > 0) {
    const int per = npairs / D_straggler;
    const int g = pair / per;
    if (g >= D_straggler) { tile_lo = tile_hi = 0; first = 0; stride = 1; counter = nullptr; }
    else {
      const int m = E / D_straggler;
      tile_lo = tile_start[g * m];
      tile_hi = tile_start[(g + 1) * m];
      first = tile_lo + (pair - g * per); stride = per;
      if (sched) counter = sched + g;
    }
  } else {
    tile_lo = 0; tile_hi = tile_start[E]; first = pair; stride = npairs;
  }
  const bool dyn = sched != nullptr;
  auto next_tile = [&](int j, bool whole_warp) -> int {   // every role but the scheduler
    if (!dyn) { const int tile = first + j * stride; return tile < tile_hi ? tile : -1; }
    return tq.get(j, whole_warp);
  };
  const int num_kb = (K + BK - 1) / BK;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (elect_one()) {
      int cursor = 0, s = 0;
      uint32_t ph = 0;
      TileT t;
      bool ok = true;
      const bool scheduler = dyn && rank == 0;
      int cur = -1, claim = 0;
      if (scheduler) {
        if (counter) {
          cur = tile_lo + atomicAdd(counter, 1);
          if (cur >= tile_hi) cur = -1;
        }
        ok = tq.put(0, cur);
        if (ok && cur >= 0) claim = atomicAdd(counter, 1);
      }
      const int pub_kb = num_kb / 2;
      for (int j = 0; ok; ++j) {
        const int tile = scheduler ? cur : next_tile(j, false);
        if (tile < 0) break;
        if (!locate_tile_t(tile, cursor, tile_start, offs, ends, E, t)) break;
        const int my_w0 = t.w0 + (int)rank * BM;                 // this CTA's 128 weight rows
        const int my_t0 = t.row0 + (int)rank * (t.nt >> 1);      // and its half of the tokens
        const int we = w_mod > 0 ? t.e % w_mod : t.e;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (scheduler && kb == pub_kb) {
            cur = tile_lo + claim;
            if (cur >= tile_hi) cur = -1;
            if (!tq.put(j + 1, cur)) { ok = false; break; }
            if (cur >= 0) claim = atomicAdd(counter, 1);
          }
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t lead_full = full_bar(s) & PEER_MASK;   // the leader's barrier counts both CTAs' bytes
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * SG::BYTES);
          const uint32_t w_dst = tiles + (uint32_t)s * SG::BYTES;
          tma2_load_3d(w_dst, &map_w0, kb * BK, my_w0, we, lead_full);
          if (SWIGLU) tma2_load_3d(w_dst + A_BYTES, &map_w1, kb * BK, my_w0, we, lead_full);
          tma2_load_2d(w_dst + SG::W_BYTES, &map_x, kb * BK, my_t0, lead_full);
          if (++s == NST) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (rank == 0 && elect_one()) {
      int cursor = 0, s = 0;
      uint32_t it = 0, ph = 0;
      const uint64_t wdesc0 = umma_desc(tiles);
      const uint64_t xdesc0 = umma_desc(tiles + SG::W_BYTES);
      const uint64_t stage_step = (uint64_t)(SG::BYTES >> 4);
      uint64_t stage_off = 0;
      TileT t;
      bool ok = true;
      for (int j = 0; ok; ++j, ++it) {
        const int tile = next_tile(j, false);
        if (tile < 0) break;
        if (!locate_tile_t(tile, cursor, tile_start, offs, ends, E, t)) break;
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(t.nt >> 3) << 17) |
                               ((uint32_t)((2 * BM) >> 4) << 24);     // M = 256, N = nt
        const uint32_t b = SWIGLU ? 0u : it & 1u, use = SWIGLU ? it : it >> 1;
        if (!mbar_wait(tempty_bar(b), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + b * (uint32_t)BNB;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t wdesc = wdesc0 + stage_off, xdesc = xdesc0 + stage_off;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
            umma2(tmem_d, wdesc + (uint64_t)(2 * k), xdesc + (uint64_t)(2 * k), idesc, accum);
            if (SWIGLU)
              umma2(tmem_d + (uint32_t)TT_MAX, wdesc + (uint64_t)((A_BYTES >> 4) + 2 * k), xdesc + (uint64_t)(2 * k), idesc,
                    accum);
          }
          umma2_commit_both(empty_bar(s));
          stage_off += stage_step;
          if (++s == NST) { s = 0; ph ^= 1u; stage_off = 0; }
        }
        if (ok) umma2_commit_both(tfull_bar(b));
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (both CTAs, own 128 weight rows)
    const int quarter = warp & 3;                         // TMEM lane quarter = 32 output columns
    const int half = (warp - 2) >> 2;                     // token chunks half, half + 2
    int cursor = 0;
    uint32_t it = 0;
    TileT t;
    uint8_t* stg = gen + STAGES * STAGE_BYTES + (warp - 2) * STG_WARP_BYTES;
    const uint32_t stg_a = smem_u32(stg);
    for (int j = 0;; ++j, ++it) {
      const int tile = next_tile(j, true);
      if (tile < 0) break;
      if (!locate_tile_t(tile, cursor, tile_start, offs, ends, E, t)) break;
      const uint32_t b = SWIGLU ? 0u : it & 1u, use = SWIGLU ? it : it >> 1;
      bool ready = mbar_wait(tfull_bar(b), use & 1u, abort_flag);
      ready = __all_sync(0xffffffffu, ready);
      if (!ready) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * (uint32_t)BNB;
      const int col0 = t.w0 + (int)rank * BM + quarter * 32;        // first output column of this warp
      const int col = col0 + lane;                                  // this thread's output column
      if (col0 < Nout) {
#pragma unroll 1
        for (int c = half * 32; c < t.nt; c += 64) {                // 32-token chunks
          uint32_t g[32];
          uint32_t hv[16];                                           // 32 bf16: tokens c .. c+31 of this column
          if (SWIGLU) {
            uint32_t u[32];
            tmem_ld32(taddr + (uint32_t)c, g);
            tmem_ld32(taddr + (uint32_t)(TT_MAX + c), u);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
              const float u0 = __uint_as_float(u[2 * i]), u1 = __uint_as_float(u[2 * i + 1]);
              hv[i] = pack_bf16(__fdividef(g0, 1.0f + __expf(-g0)) * u0, __fdividef(g1, 1.0f + __expf(-g1)) * u1);
            }
          } else {
            tmem_ld32(taddr + (uint32_t)c, g);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) hv[i] = pack_bf16(__uint_as_float(g[2 * i]), __uint_as_float(g[2 * i + 1]));
          }
          const int tok0 = t.row0 + c;
          const bool whole = c + 32 <= t.rows && col0 + 32 <= Nout;   // all 32 tokens and columns exist
          if (whole) {
            if (lane == 0) bulk_wait_read_all();                     // the previous box has left the staging buffer
            __syncwarp();
            // box row = token (64 bytes = 32 columns), 64-byte swizzle: 16-byte chunk ^ ((row >> 1) & 3)
            const uint32_t in_chunk = (uint32_t)(lane & 7) * 2u, chunk = (uint32_t)lane >> 3;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const uint32_t r0 = 2 * i, r1 = 2 * i + 1;             // two tokens share (row >> 1)
              const uint32_t sw = (chunk ^ ((uint32_t)i & 3u)) * 16u + in_chunk;
              asm volatile("st.shared.u16 [%0], %1;" ::"r"(stg_a + r0 * 64u + sw), "h"((uint16_t)(hv[i] & 0xffffu)) : "memory");
              asm volatile("st.shared.u16 [%0], %1;" ::"r"(stg_a + r1 * 64u + sw), "h"((uint16_t)(hv[i] >> 16)) : "memory");
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&map_out, col0, tok0, stg_a);
              bulk_commit();
            }
          } else if (col < Nout) {
            __nv_bfloat16* o = out + (int64_t)tok0 * Nout + col;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              if (c + 2 * i < t.rows) o[(int64_t)(2 * i) * Nout] = __ushort_as_bfloat16((uint16_t)(hv[i] & 0xffffu));
              if (c + 2 * i + 1 < t.rows) o[(int64_t)(2 * i + 1) * Nout] = __ushort_as_bfloat16((uint16_t)(hv[i] >> 16));
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive_cluster(tempty_bar(b) & PEER_MASK);   // the leader waits for both CTAs' epilogues
    }
    if (lane == 0) bulk_wait_all();
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
  if (tid == 0 && *abort_flag && dev_status) atomicExch(dev_status, (int)CAPMOE_ETIMEOUT);
}

}  // namespace

// The launches of the short-segment form (either GEMM, or both).  `sched1` / `sched2`: zeroed tile
// counters (one per straggler group) or NULL.
int ffn_tc_short(bool gate_up, bool down, const void* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int n_w, int d, int F,
                 const void* w_gate, const void* w_up, const void* w_down, void* h_ws, void* y_perm, int64_t A_max,
                 int D_straggler, int32_t* dev_status, int32_t* sched1, int32_t* sched2, cudaEvent_t mid, cudaStream_t st) {
  alignas(64) CUtensorMap x1, wg, wu, x2, wd, o1, o2;
  if (!make_store_map(&o1, h_ws, (uint64_t)F, (uint64_t)A_max) ||
      !make_store_map(&o2, y_perm, (uint64_t)d, (uint64_t)A_max) ||
      !make_map(&x1, x_perm, (uint64_t)d, (uint64_t)A_max, 0, TT_HALF) ||
      !make_map(&wg, w_gate, (uint64_t)d, (uint64_t)F, (uint64_t)n_w, BM) ||
      !make_map(&wu, w_up, (uint64_t)d, (uint64_t)F, (uint64_t)n_w, BM) ||
      !make_map(&x2, h_ws, (uint64_t)F, (uint64_t)A_max, 0, TT_HALF) ||
      !make_map(&wd, w_down, (uint64_t)F, (uint64_t)d, (uint64_t)n_w, BM))
    return note_cuda(cudaErrorInvalidValue);
  int pairs = sm_count() / 2;
  if (pairs < 1 || (D_straggler > 0 && pairs < D_straggler)) return CAPMOE_EUNSUPPORTED;
  if (D_straggler > 0) pairs = (pairs / D_straggler) * D_straggler;
  cudaError_t err = cudaFuncSetAttribute(k_ffn_tc2t<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (err != cudaSuccess) return note_cuda(err);
  err = cudaFuncSetAttribute(k_ffn_tc2t<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (err != cudaSuccess) return note_cuda(err);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (gate_up) {
    err = cudaLaunchKernelEx(&cfg, k_ffn_tc2t<0>, x1, wg, wu, o1, seg_begin, seg_end, w_mod, E, d, F, (__nv_bfloat16*)h_ws,
                             D_straggler, dev_status, sched1);
    count_launch(1);
    if (err != cudaSuccess) return note_cuda(err);
    int rc;
    if (mid && (rc = note_cuda(cudaEventRecord(mid, st))) != CAPMOE_OK) return rc;
  }
  if (!down) return CAPMOE_OK;
  err = cudaLaunchKernelEx(&cfg, k_ffn_tc2t<1>, x2, wd, wd, o2, seg_begin, seg_end, w_mod, E, F, d, (__nv_bfloat16*)y_perm,
                           D_straggler, dev_status, sched2);
  count_launch(1);
  return note_cuda(err);
}

}  // namespace capmoe
