// Stage 5, tensor-core path: grouped SwiGLU expert FFN in bf16 on tcgen05 (5th-generation
// tensor cores) with TMA-fed shared-memory tiles and fp32 accumulators in tensor memory; the
// router (stage 1) for bf16 inputs with more than 16 experts runs on the same pipeline.
//
// Two persistent, warp-specialised launches per layer:
//   GEMM1  H[r, f]  = silu(x_perm[r,:] . W_g[e,f,:]) * (x_perm[r,:] . W_u[e,f,:])
//   GEMM2  y_perm[r, j] = H[r,:] . W_d[e,j,:]
// Both operands of both GEMMs are K-major (row-major activations, [out,in] weights), so every
// tile is loaded by TMA with the 128-byte swizzle and consumed by tcgen05.mma straight from
// shared memory.  k_ffn_tc, one CTA per SM:
//   warp 0      TMA producer (one elected lane): ring of STAGES {A 128x64, B 256x64} bf16 tiles
//   warp 1      MMA issuer (one elected lane): 128 x 256 x 16 tcgen05.mma, accumulators ping-pong
//               between two 256-column halves of the CTA's 512 TMEM columns
//   warps 2-9   epilogue: tcgen05.ld the finished accumulator, SwiGLU / convert, 16-byte stores,
//               overlapping the next tile's MMAs
// GEMM1 puts 128 gate rows and 128 up rows of the same output columns into one 256-row B tile,
// so one MMA yields both halves of the SwiGLU pair.  k_ffn_tc2 is the same pipeline on CTA pairs
// (cta_group::2, 256 x 256 tiles, each CTA loads half of B) and serves long expert segments.
// Tiles are enumerated on the device from the segment bounds (no host synchronisation); within an
// expert the row-block index runs fastest so that concurrently running CTAs share weight tiles
// through L2.  With a status block from the caller the CTAs take their tiles from a device counter
// (TileQueue below), else each walks a fixed list.  In straggler-emulation mode the CTAs are split
// into D equal groups and group g only serves the experts of virtual device g.
// MODE_ROUTER / MODE_ROUTER_FUSED reuse k_ffn_tc for logits = x . W_r^T + bias, the fused form with
// softmax, top-k and the load histogram in a 16-warp epilogue.
// Every mbarrier wait is bounded; on expiry the CTA raises a flag, all roles drain and the
// kernel reports CAPMOE_ETIMEOUT through dev_status.
#include "softmax.cuh"
#include "tc_common.cuh"

namespace capmoe {
namespace {


// MODE_GATE_UP: B tile = 128 rows of W_g + 128 rows of W_u, output columns n0..n0+127 of H (bf16)
// MODE_DOWN   : B tile = 256 rows of W_d, output columns n0..n0+255 of y_perm (bf16)
// MODE_ROUTER : one row segment [0, single_rows), B tile = all n_mma (>= Nout) rows of W_r,
//               output = fp32 logits [rows, Nout] + bias  (Eq. 1's gate)
// MODE_ROUTER_FUSED : MODE_ROUTER whose epilogue goes on, one thread per token with the token's
//               Nout <= EPAD logits in registers, to softmax, top-k and the load histogram
//               (Eq. 1, Eq. 3): the whole router stage in one launch
enum { MODE_GATE_UP = 0, MODE_DOWN = 1, MODE_ROUTER = 2, MODE_ROUTER_FUSED = 3 };

// Outputs of the fused router epilogue (unused by the other modes).
struct RouterFused { float* scores; int32_t* topk_idx; float* topk_score; int32_t* load; int k; };

template <int MODE, int EPAD = 32>
__global__ void __launch_bounds__(MODE == MODE_ROUTER_FUSED ? RF_THREADS : TC_THREADS, 1)
k_ffn_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
         const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_out /* FFN modes: the
         output as 32 x 32 boxes */, const int32_t* __restrict__ seg_begin, const int32_t* __restrict__ seg_end /* [E]:
         rows [seg_begin[e], seg_end[e]) form segment e; for packed segments seg_end = seg_begin + 1 */,
         int w_mod /* > 0: segment e uses weight block e % w_mod */, int E,
         int K /* reduction length */, int Nout /* output columns */, void* __restrict__ out_ptr,
         int D_straggler, int32_t* __restrict__ dev_status, int n_mma, int single_rows,
         const float* __restrict__ bias, int tile_rows /* rows per tile actually loaded (<= 128) */,
         int n_stages, int stage_stride, const RouterFused rf,
         int32_t* __restrict__ sched /* FFN modes: tile counters, one per straggler group, zeroed; NULL = fixed lists */) {
  constexpr bool SWIGLU = MODE == MODE_GATE_UP;
  constexpr bool ROUTER = MODE == MODE_ROUTER || MODE == MODE_ROUTER_FUSED;
  constexpr bool FUSED = MODE == MODE_ROUTER_FUSED;
  allow_next_kernel();
  constexpr int N_TILE = SWIGLU ? 128 : 256;
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(out_ptr);
  const uint32_t idesc = make_idesc(n_mma);
  // The MMA always spans 128 rows; with tile_rows < 128 (router, few tokens) only the first
  // tile_rows rows of the A tile are loaded and stored, the rest of the accumulator is ignored.
  const uint32_t a_bytes = (uint32_t)(tile_rows * BK * 2);
  const uint32_t stage_tx = a_bytes + (uint32_t)(n_mma * BK * 2);
  extern __shared__ uint8_t smem_raw[];
  // carve: tiles (1024-byte aligned), barriers, expert tables
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + TAIL_OFF);
  // bars[0..16) full, [16..32) empty, [32..34) tmem_full, [34..36) tmem_empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* offs = reinterpret_cast<int*>(gen + TAIL_OFF + 512);
  int* tile_start = offs + (MAX_E + 1);
  float* bias_s = reinterpret_cast<float*>(tile_start + (MAX_E + 1) + 2);   // [256], router mode only
  int* hist = tile_start + 8;                          // [<= 128] load histogram, fused router only
  float* xch = bias_s + 256;                           // [RF_XCH_FLOATS] exchange between a token's threads
  int* ends = reinterpret_cast<int*>(xch + RF_XCH_FLOATS);   // [MAX_E] row after the last of each segment
  const int nthreads = (int)blockDim.x;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(MAX_STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (uint32_t)(2 * MAX_STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (uint32_t)(2 * MAX_STAGES + 2 + b); };
  // tile queue: barriers 40..47 and four ints behind them, inside the 512-byte barrier block
  const TileQueue<false> tq{bar0 + 8u * 40u, bar0 + 8u * 44u, bar0 + 8u * 48u, 0u, abort_flag};
  // Set-up that touches no global memory (barriers, tensor memory) runs before the wait for the
  // previous kernel, so that it overlaps that kernel's tail.
  if (tid == 32) {                                       // the descriptors the first loads will need
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b0) : "memory");
    if (SWIGLU) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b1) : "memory");
  }
  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), nthreads - 64); }
    for (int i = 0; i < TQ; ++i) { mbar_init(tq.full(i), 1); mbar_init(tq.empty(i), TQ_READERS_ONE); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  wait_for_previous_kernel();
  if (ROUTER) {
    // (the bias is fetched by the epilogue warps, which are the only ones to use it: the first
    // loads do not wait for that round trip to global memory)
    if (tid == 0) { offs[0] = 0; ends[0] = single_rows; }
    if (FUSED)
      for (int i = tid; i < EPAD; i += nthreads) hist[i] = 0;
  } else {
    for (int i = tid; i < E; i += nthreads) { offs[i] = seg_begin[i]; ends[i] = seg_end[i]; }
  }
  __syncthreads();
  if (tid == 0) {
    const int n_blocks = (Nout + N_TILE - 1) / N_TILE;
    int acc = 0;
    for (int e = 0; e < E; ++e) {
      tile_start[e] = acc;
      acc += ((ends[e] - offs[e] + tile_rows - 1) / tile_rows) * n_blocks;
    }
    tile_start[E] = acc;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // this CTA's share of the tile list
  int tile_lo, tile_hi, stride, first;
  int32_t* counter = sched;                             // this CTA's group counter
  if (D_straggler > 0) {
    const int per = gridDim.x / D_straggler;            // CTAs per virtual device
    const int g = blockIdx.x / per;
    if (g >= D_straggler) { tile_lo = tile_hi = 0; first = 0; stride = 1; counter = nullptr; }
    else {
      const int m = E / D_straggler;
      tile_lo = tile_start[g * m]; tile_hi = tile_start[(g + 1) * m];
      first = tile_lo + (blockIdx.x - g * per); stride = per;
      if (sched) counter = sched + g;
    }
  } else {
    tile_lo = 0; tile_hi = tile_start[E]; first = blockIdx.x; stride = gridDim.x;
  }
  const int num_kb = (K + BK - 1) / BK;
  const bool dyn = !ROUTER && sched != nullptr;
  auto next_tile = [&](int j, bool whole_warp) -> int {   // every role but the scheduler
    if (!dyn) { const int tile = first + j * stride; return tile < tile_hi ? tile : -1; }
    return tq.get(j, whole_warp);
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      int cursor = 0;
      int s = 0;                                         // ring position and phase, advanced without division
      uint32_t ph = 0;
      Tile t;
      bool ok = true;
      // With a counter the producer is the CTA's scheduler: halfway through the loads of tile j it
      // publishes entry j+1 and asks the counter for the one after, so the counter's round trip
      // never sits between two tiles' loads.
      int cur = -1, claim = 0;
      if (dyn) {
        if (counter) {
          cur = tile_lo + atomicAdd(counter, 1);
          if (cur >= tile_hi) cur = -1;
        }
        ok = tq.put(0, cur);
        if (ok && cur >= 0) claim = atomicAdd(counter, 1);
      }
      const int pub_kb = num_kb / 2;
      for (int j = 0; ok; ++j) {
        const int tile = dyn ? cur : next_tile(j, false);
        if (tile < 0) break;
        if (!locate_tile(tile, cursor, tile_start, offs, ends, E, N_TILE, tile_rows, t)) break;
        const int we = w_mod > 0 ? t.e % w_mod : t.e;     // weight block of this segment
        for (int kb = 0; kb < num_kb; ++kb) {
          if (dyn && kb == pub_kb) {
            cur = tile_lo + claim;
            if (cur >= tile_hi) cur = -1;
            if (!tq.put(j + 1, cur)) { ok = false; break; }
            if (cur >= 0) claim = atomicAdd(counter, 1);
          }
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(full_bar(s), stage_tx);
          const uint32_t a_dst = tiles + (uint32_t)s * (uint32_t)stage_stride;
          const uint32_t b_dst = a_dst + a_bytes;
          tma_load_2d(a_dst, &map_a, kb * BK, t.row0, full_bar(s));
          if (SWIGLU) {
            tma_load_3d(b_dst, &map_b0, kb * BK, t.n0, we, full_bar(s));
            tma_load_3d(b_dst + B_BYTES / 2, &map_b1, kb * BK, t.n0, we, full_bar(s));
          } else {
            tma_load_3d(b_dst, &map_b0, kb * BK, ROUTER ? 0 : t.n0, we, full_bar(s));
          }
          if (++s == n_stages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      int cursor = 0;
      uint32_t it = 0;
      int s = 0;                                         // ring position and phase, advanced without division
      uint32_t ph = 0;
      // descriptors of stage 0; a stage further on adds its byte offset >> 4 to the address field
      const uint64_t adesc0 = umma_desc(tiles);
      const uint64_t bdesc0 = umma_desc(tiles + a_bytes);
      const uint64_t stage_step = (uint64_t)((uint32_t)stage_stride >> 4);
      uint64_t stage_off = 0;
      Tile t;
      bool ok = true;
      for (int j = 0; ok; ++j, ++it) {
        const int tile = next_tile(j, false);
        if (tile < 0) break;
        if (!locate_tile(tile, cursor, tile_start, offs, ends, E, N_TILE, tile_rows, t)) break;
        const uint32_t b = it & 1u, use = it >> 1;
        if (!mbar_wait(tempty_bar(b), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + b * (uint32_t)BNB;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = adesc0 + stage_off;
          const uint64_t bdesc = bdesc0 + stage_off;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advance 32 bytes (16 bf16) inside the swizzled 128-byte row: +2 in 16-byte units
            umma(tmem_d, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(empty_bar(s));                    // frees the stage when these MMAs have read it
          stage_off += stage_step;
          if (++s == n_stages) { s = 0; ph ^= 1u; stage_off = 0; }
        }
        if (ok) umma_commit(tfull_bar(b));              // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9)
    if (ROUTER) {
      for (int i = tid - 64; i < 256; i += nthreads - 64) bias_s[i] = (bias && i < Nout) ? bias[i] : 0.f;
      group_sync(6, nthreads - 64);
    }
    const int quarter = warp & 3;                        // TMEM lane quarter this warp may read
    const int row_in_tile = quarter * 32 + lane;
    const int half = (warp - 2) >> 2;                    // which half of the columns this warp converts
    int cursor = 0;
    uint32_t it = 0;
    Tile t;
    for (int j = 0;; ++j, ++it) {
      const int tile = next_tile(j, true);
      if (tile < 0) break;
      if (!locate_tile(tile, cursor, tile_start, offs, ends, E, N_TILE, tile_rows, t)) break;
      const uint32_t b = it & 1u, use = it >> 1;
      bool ready = mbar_wait(tfull_bar(b), use & 1u, abort_flag);
      ready = __all_sync(0xffffffffu, ready);            // warp-uniform: tcgen05.ld below is .sync.aligned
      if (FUSED) ready = group_all(1 + quarter, RF_SUBS * 32, ready);   // a token's threads stop together
      if (!ready) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * (uint32_t)BNB;
      const bool row_ok = row_in_tile < t.rows;
      if constexpr (FUSED) {
        if (tile_rows <= RF_SPREAD_ROWS) {
          // Small row tiles (few tokens per SM): with one thread per (token, column quarter) only the
          // warps of the first one or two TMEM lane quarters would have tokens, i.e. one or two of the
          // SM's four warp schedulers.  Instead those warps only move the logits out (global memory and
          // a shared-memory tile), and then all sixteen warps share the tokens, eight threads per token
          // (eight consecutive lanes, an eighth of the columns each, exchange by shuffles).
          constexpr int COLS = EPAD / RF_SUBS;                 // columns a dumping thread reads from TMEM
          constexpr int CS = EPAD / 8;                         // columns per thread afterwards
          float* lt = reinterpret_cast<float*>(gen + STAGES * STAGE_BYTES);   // [RF_SPREAD_ROWS][EPAD] logits + bias
          const int sub = (warp - 2) >> 2;
          const int cbase = sub * COLS;
          if (quarter * 32 < t.rows) {
            uint32_t g[COLS];
            if constexpr (COLS == 16) tmem_ld16(taddr + (uint32_t)cbase, g);
            else tmem_ld8(taddr + (uint32_t)cbase, g);
            tmem_ld_wait();
            float v[COLS];
#pragma unroll
            for (int i = 0; i < COLS; ++i)
              v[i] = cbase + i < Nout ? __fadd_rn(__uint_as_float(g[i]), bias_s[cbase + i]) : -INFINITY;
            if (row_ok) {
              float* lrow = reinterpret_cast<float*>(out_ptr) + ((int64_t)t.row0 + row_in_tile) * Nout + cbase;
              if ((Nout & 3) == 0) {
#pragma unroll
                for (int i = 0; i < COLS; i += 4)
                  if (cbase + i < Nout) *reinterpret_cast<float4*>(lrow + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
              } else {
#pragma unroll
                for (int i = 0; i < COLS; ++i)
                  if (cbase + i < Nout) lrow[i] = v[i];
              }
            }
            if (row_in_tile < RF_SPREAD_ROWS) {
#pragma unroll
              for (int i = 0; i < COLS; i += 4)
                *reinterpret_cast<float4*>(lt + row_in_tile * EPAD + cbase + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            }
          }
          tc_fence_before();
          mbar_arrive(tempty_bar(b));
          group_sync(5, 4 * RF_SUBS * 32);                     // the tile of logits is complete
          const int et = tid - 64;                             // 0 .. 511
          const int r = et >> 3, j = et & 7;
          if (((et >> 5) << 2) >= t.rows) {                    // none of this warp's four tokens exists:
            group_sync(5, 4 * RF_SUBS * 32);                   // leave the issue slots to the warps that have some
            continue;
          }
          const bool tok_ok = r < t.rows;
          const int64_t tok = (int64_t)t.row0 + r;
          const int c0 = j * CS;
          float v[CS];
#pragma unroll
          for (int i = 0; i < CS; i += 4) {
            const float4 q4 = *reinterpret_cast<const float4*>(lt + (r & (RF_SPREAD_ROWS - 1)) * EPAD + c0 + i);
            v[i] = q4.x; v[i + 1] = q4.y; v[i + 2] = q4.z; v[i + 3] = q4.w;
          }
          if (!tok_ok) {
#pragma unroll
            for (int i = 0; i < CS; ++i) v[i] = 0.f;          // rows past the tile: defined values, results unused
          }
          float mx = v[0];
#pragma unroll
          for (int i = 1; i < CS; ++i) mx = v[i] > mx ? v[i] : mx;
#pragma unroll
          for (int o = 4; o > 0; o >>= 1) { const float ov = __shfl_xor_sync(0xffffffffu, mx, o); mx = ov > mx ? ov : mx; }
#pragma unroll
          for (int i = 0; i < CS; ++i) v[i] = exp_fixed(__fsub_rn(v[i], mx));      // padding: exp(-inf) = 0
          // the E terms are added left to right: the partial sum walks through the token's eight threads
          float acc = 0.f;
#pragma unroll
          for (int s2 = 0; s2 < 8; ++s2) {
            const float incoming = __shfl_up_sync(0xffffffffu, acc, 1, 8);
            if (j == s2) {
              acc = s2 ? incoming : 0.f;
#pragma unroll
              for (int i = 0; i < CS; ++i) acc = __fadd_rn(acc, v[i]);             // + 0 (padding) is exact
            }
          }
          const float sum = __shfl_sync(0xffffffffu, acc, 7, 8);                   // in [1, E]
          const float rsum = __frcp_rn(sum);
#pragma unroll
          for (int i = 0; i < CS; ++i) v[i] = c0 + i < Nout ? div_by(v[i], sum, rsum) : -1.f;   // padding never selected
          if (tok_ok) {
            float* srow = rf.scores + tok * Nout + c0;
            if ((Nout & 3) == 0) {
#pragma unroll
              for (int i = 0; i < CS; i += 4)
                if (c0 + i < Nout) *reinterpret_cast<float4*>(srow + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            } else {
#pragma unroll
              for (int i = 0; i < CS; ++i)
                if (c0 + i < Nout) srow[i] = v[i];
            }
          }
          // top-k: k rounds; each thread offers the best of its columns (lower id on ties), the eight
          // offers meet in a butterfly on (score, lower id), the owner marks its column taken
#pragma unroll 1
          for (int kk = 0; kk < rf.k; ++kk) {
            float best = -1.f;
            int bi = 0;
#pragma unroll
            for (int i = 0; i < CS; ++i) { const bool gt = v[i] > best; best = gt ? v[i] : best; bi = gt ? i : bi; }
            int be = c0 + bi;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
              const float ob = __shfl_xor_sync(0xffffffffu, best, o);
              const int oe = __shfl_xor_sync(0xffffffffu, be, o);
              const bool take = ob > best || (ob == best && oe < be);
              best = take ? ob : best;
              be = take ? oe : be;
            }
            if (be >= c0 && be < c0 + CS) {                                        // this thread's offer won
#pragma unroll
              for (int i = 0; i < CS; ++i) v[i] = (c0 + i == be) ? -2.f : v[i];    // taken
              if (tok_ok) {
                rf.topk_idx[tok * rf.k + kk] = be;
                rf.topk_score[tok * rf.k + kk] = best;
                atomicAdd(&hist[be], 1);
              }
            }
          }
          group_sync(5, 4 * RF_SUBS * 32);                     // the next tile may overwrite the shared tile
          continue;
        }
        // RF_SUBS threads per token (same lane of the quarter's four warps), each with COLS of the
        // token's columns in registers.  The accumulator goes back to the MMA issuer as soon as it
        // has been read; what is not local to a thread passes through shared memory between the
        // quarter's named-barrier phases.
        constexpr int COLS = EPAD / RF_SUBS;
        static_assert(COLS == 8 || COLS == 16, "fused router: 32 or 64 padded experts");
        const int sub = (warp - 2) >> 2;
        const int cbase = sub * COLS;
        const int bar_id = 1 + quarter;
        float* xmax = xch;                                                 // [RF_SUBS][128]
        float* xsum = xch + RF_SUBS * 128;                                 // [128]
        float* xb = xsum + 128;                                            // [2][RF_SUBS][128]
        int* xi = reinterpret_cast<int*>(xb + 2 * RF_SUBS * 128);          // [2][RF_SUBS][128]
        uint32_t g[COLS];
        if constexpr (COLS == 16) tmem_ld16(taddr + (uint32_t)cbase, g);
        else tmem_ld8(taddr + (uint32_t)cbase, g);
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive(tempty_bar(b));
        if (quarter * 32 >= t.rows) continue;            // no token of this tile in this quarter (all four warps agree)
        float v[COLS];
#pragma unroll
        for (int i = 0; i < COLS; ++i)
          v[i] = cbase + i < Nout ? __fadd_rn(__uint_as_float(g[i]), bias_s[cbase + i]) : -INFINITY;
        const int64_t tok = (int64_t)t.row0 + row_in_tile;
        float* lrow = reinterpret_cast<float*>(out_ptr) + tok * Nout + cbase;
        float* srow = rf.scores + tok * Nout + cbase;
        const bool vec = (Nout & 3) == 0;                // rows are 16-byte aligned: vector stores
        if (row_ok) {
          if (vec) {
#pragma unroll
            for (int i = 0; i < COLS; i += 4)
              if (cbase + i < Nout) *reinterpret_cast<float4*>(lrow + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < COLS; ++i)
              if (cbase + i < Nout) lrow[i] = v[i];
          }
        }
        float mx = v[0];
#pragma unroll
        for (int i = 1; i < COLS; ++i) mx = v[i] > mx ? v[i] : mx;
        xmax[sub * 128 + row_in_tile] = mx;
        group_sync(bar_id, RF_SUBS * 32);
#pragma unroll
        for (int s2 = 0; s2 < RF_SUBS; ++s2) { const float o = xmax[s2 * 128 + row_in_tile]; mx = o > mx ? o : mx; }
#pragma unroll
        for (int i = 0; i < COLS; ++i) v[i] = exp_fixed(__fsub_rn(v[i], mx));     // padding: exp(-inf) = 0
        // the E terms are added left to right: the partial sum is handed from thread to thread
#pragma unroll
        for (int s2 = 0; s2 < RF_SUBS; ++s2) {
          if (sub == s2) {
            float acc = s2 ? xsum[row_in_tile] : 0.f;
#pragma unroll
            for (int i = 0; i < COLS; ++i) acc = __fadd_rn(acc, v[i]);            // + 0 (padding) is exact
            xsum[row_in_tile] = acc;
          }
          group_sync(bar_id, RF_SUBS * 32);
        }
        const float sum = xsum[row_in_tile];                                      // in [1, E]
        const float rsum = __frcp_rn(sum);
#pragma unroll
        for (int i = 0; i < COLS; ++i) v[i] = cbase + i < Nout ? div_by(v[i], sum, rsum) : -1.f;   // padding never selected
        if (row_ok) {
          if (vec) {
#pragma unroll
            for (int i = 0; i < COLS; i += 4)
              if (cbase + i < Nout) *reinterpret_cast<float4*>(srow + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < COLS; ++i)
              if (cbase + i < Nout) srow[i] = v[i];
          }
        }
        // top-k: k rounds; each thread offers the best of its columns (lower id on ties), the
        // four offers are compared in id order with strict '>', the owner marks its column taken.
#pragma unroll 1
        for (int j = 0; j < rf.k; ++j) {
          float cb0 = -1.f, cb1 = -1.f;
          int ci0 = 0, ci1 = 0;
#pragma unroll
          for (int i = 0; i < COLS / 2; ++i) {
            const bool g0 = v[i] > cb0, g1 = v[COLS / 2 + i] > cb1;
            cb0 = g0 ? v[i] : cb0; ci0 = g0 ? i : ci0;
            cb1 = g1 ? v[COLS / 2 + i] : cb1; ci1 = g1 ? COLS / 2 + i : ci1;
          }
          const bool g1 = cb1 > cb0;
          const float mine = g1 ? cb1 : cb0;
          const int mine_i = g1 ? ci1 : ci0;
          const int slot = (j & 1) * RF_SUBS * 128 + row_in_tile;
          xb[slot + sub * 128] = mine;
          xi[slot + sub * 128] = cbase + mine_i;
          group_sync(bar_id, RF_SUBS * 32);
          float best = xb[slot];
          int be = xi[slot];
#pragma unroll
          for (int s2 = 1; s2 < RF_SUBS; ++s2) {
            const float ob = xb[slot + s2 * 128];
            const int oe = xi[slot + s2 * 128];
            const bool gt = ob > best;
            best = gt ? ob : best;
            be = gt ? oe : be;
          }
          if (be == cbase + mine_i) {                                              // this thread's offer won
#pragma unroll
            for (int i = 0; i < COLS; ++i) v[i] = i == mine_i ? -2.f : v[i];      // taken
            if (row_ok) {
              rf.topk_idx[tok * rf.k + j] = be;
              rf.topk_score[tok * rf.k + j] = best;
              atomicAdd(&hist[be], 1);
            }
          }
        }
        continue;
      }
      if (MODE == MODE_ROUTER) {
        float* lrow = reinterpret_cast<float*>(out_ptr) + (int64_t)(t.row0 + row_in_tile) * Nout;
#pragma unroll 1
        for (int c = half * 32; c < n_mma; c += 64) {
          uint32_t g[32];
          tmem_ld32(taddr + (uint32_t)c, g);
          tmem_ld_wait();
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(g[j]) + bias_s[c + j];
          if (row_ok) {
            if ((Nout & 3) == 0) {                       // rows are 16-byte aligned: vector stores
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                if (c + j < Nout) *reinterpret_cast<float4*>(lrow + c + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (c + j < Nout) lrow[c + j] = v[j];
            }
          }
        }
        tc_fence_before();
        mbar_arrive(tempty_bar(b));
        continue;
      }
      __nv_bfloat16* orow = out + (int64_t)(t.row0 + row_in_tile) * Nout + t.n0;
      const bool full_rows = quarter * 32 + 32 <= t.rows;      // all 32 rows of this warp are inside the segment
      uint8_t* stg = gen + STAGES * STAGE_BYTES + (warp - 2) * STG_WARP_BYTES;
#pragma unroll 1
      for (int c = half * (N_TILE / 2); c < (half + 1) * (N_TILE / 2); c += 32) {
        uint32_t g[32];
        uint32_t packed[16];
        if (SWIGLU) {
          uint32_t u[32];
          tmem_ld32(taddr + (uint32_t)c, g);
          tmem_ld32(taddr + (uint32_t)(128 + c), u);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float g0 = __uint_as_float(g[2 * j]), g1 = __uint_as_float(g[2 * j + 1]);
            const float u0 = __uint_as_float(u[2 * j]), u1 = __uint_as_float(u[2 * j + 1]);
            const float h0 = __fdividef(g0, 1.0f + __expf(-g0)) * u0;
            const float h1 = __fdividef(g1, 1.0f + __expf(-g1)) * u1;
            packed[j] = pack_bf16(h0, h1);
          }
        } else {
          tmem_ld32(taddr + (uint32_t)c, g);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j)
            packed[j] = pack_bf16(__uint_as_float(g[2 * j]), __uint_as_float(g[2 * j + 1]));
        }
        store_piece(packed, full_rows, row_ok, stg, &map_out, t.n0 + c, t.row0 + quarter * 32, orow + c,
                    Nout - (t.n0 + c));
      }
      tc_fence_before();
      mbar_arrive(tempty_bar(b));
    }
    if (!ROUTER && lane == 0) bulk_wait_all();           // this lane's stores have landed before the CTA ends
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
  if (tid == 0 && *abort_flag && dev_status) atomicExch(dev_status, (int)CAPMOE_ETIMEOUT);
  if (FUSED)
    for (int i = tid; i < Nout; i += nthreads)
      if (hist[i]) atomicAdd(&rf.load[i], hist[i]);
}

template <int MODE>
__global__ void __launch_bounds__(TC_THREADS, 1)
k_ffn_tc2(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
          const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_out /* the output as
          32 x 32 boxes */, const int32_t* __restrict__ seg_begin, const int32_t* __restrict__ seg_end, int w_mod, int E,
          int K, int Nout, __nv_bfloat16* __restrict__ out, int D_straggler, int32_t* __restrict__ dev_status,
          int32_t* __restrict__ sched /* tile counters, one per straggler group, zeroed; NULL = fixed lists */) {
  constexpr bool SWIGLU = MODE == MODE_GATE_UP;
  constexpr int N_TILE = SWIGLU ? 128 : 256;
  constexpr int BM2 = 2 * BM;                                   // rows of a pair's tile
  allow_next_kernel();
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BNB >> 3) << 17) |
                         ((uint32_t)(BM2 >> 4) << 24);          // M = 256, N = 256
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
  // tile queue: barriers 40..47 and four ints behind them, inside the 512-byte barrier block
  const TileQueue<true> tq{bar0 + 8u * 40u, bar0 + 8u * 44u, bar0 + 8u * 48u, rank, abort_flag};

  // set-up that touches no global memory comes before the wait for the previous kernel (see k_ffn_tc)
  if (tid == 0) {
    for (int s = 0; s < STAGES2; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
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
    const int n_blocks = (Nout + N_TILE - 1) / N_TILE;
    int acc = 0;
    for (int e = 0; e < E; ++e) {
      tile_start[e] = acc;
      acc += ((ends[e] - offs[e] + BM2 - 1) / BM2) * n_blocks;
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
  int32_t* counter = sched;                                     // this pair's group counter
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
  // Next tile of this pair for a role: the fixed list, or the queue (the leader's producer thread
  // fills it).  Returns a negative number when there is no further tile or a wait ran out.
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
      Tile t;
      bool ok = true;
      // The leader's producer is the pair's scheduler when tiles come from the counter.  It claims
      // half a tile ahead: halfway through the loads of tile j it publishes entry j+1 (so the peer's
      // producer has it before it runs out of work) and asks the counter for the entry after that
      // (so the counter's round trip never sits between two tiles' loads).
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
        if (!locate_tile(tile, cursor, tile_start, offs, ends, E, N_TILE, BM2, t)) break;
        const int my_row0 = t.row0 + (int)rank * BM;
        const int we = w_mod > 0 ? t.e % w_mod : t.e;     // weight block of this segment
        for (int kb = 0; kb < num_kb; ++kb) {
          if (scheduler && kb == pub_kb) {
            cur = tile_lo + claim;
            if (cur >= tile_hi) cur = -1;
            if (!tq.put(j + 1, cur)) { ok = false; break; }
            if (cur >= 0) claim = atomicAdd(counter, 1);
          }
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t lead_full = full_bar(s) & PEER_MASK;   // the leader's barrier counts both CTAs' bytes
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * STAGE2_BYTES);
          const uint32_t a_dst = tiles + (uint32_t)s * STAGE2_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          tma2_load_2d(a_dst, &map_a, kb * BK, my_row0, lead_full);
          if (SWIGLU) tma2_load_3d(b_dst, rank == 0 ? &map_b0 : &map_b1, kb * BK, t.n0, we, lead_full);
          else tma2_load_3d(b_dst, &map_b0, kb * BK, t.n0 + (int)rank * 128, we, lead_full);
          if (++s == STAGES2) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (rank == 0 && elect_one()) {
      int cursor = 0, s = 0;
      uint32_t it = 0, ph = 0;
      const uint64_t adesc0 = umma_desc(tiles);
      const uint64_t bdesc0 = umma_desc(tiles + A_BYTES);
      const uint64_t stage_step = (uint64_t)(STAGE2_BYTES >> 4);
      uint64_t stage_off = 0;
      Tile t;
      bool ok = true;
      for (int j = 0; ok; ++j, ++it) {
        const int tile = next_tile(j, false);
        if (tile < 0) break;
        if (!locate_tile(tile, cursor, tile_start, offs, ends, E, N_TILE, BM2, t)) break;
        const uint32_t b = it & 1u, use = it >> 1;
        if (!mbar_wait(tempty_bar(b), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + b * (uint32_t)BNB;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = adesc0 + stage_off, bdesc = bdesc0 + stage_off;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma2(tmem_d, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          umma2_commit_both(empty_bar(s));              // both CTAs may refill this stage
          stage_off += stage_step;
          if (++s == STAGES2) { s = 0; ph ^= 1u; stage_off = 0; }
        }
        if (ok) umma2_commit_both(tfull_bar(b));        // both halves of the accumulator are complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
    const int quarter = warp & 3;
    const int row_in_half = quarter * 32 + lane;
    const int half = (warp - 2) >> 2;
    int cursor = 0;
    uint32_t it = 0;
    Tile t;
    for (int j = 0;; ++j, ++it) {
      const int tile = next_tile(j, true);
      if (tile < 0) break;
      if (!locate_tile(tile, cursor, tile_start, offs, ends, E, N_TILE, BM2, t)) break;
      const uint32_t b = it & 1u, use = it >> 1;
      bool ready = mbar_wait(tfull_bar(b), use & 1u, abort_flag);
      ready = __all_sync(0xffffffffu, ready);
      if (!ready) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * (uint32_t)BNB;
      const int row_in_tile = (int)rank * BM + row_in_half;
      const bool row_ok = row_in_tile < t.rows;
      __nv_bfloat16* orow = out + (int64_t)(t.row0 + row_in_tile) * Nout + t.n0;
      const int warp_row0 = (int)rank * BM + quarter * 32;     // first of this warp's 32 rows in the pair's tile
      const bool full_rows = warp_row0 + 32 <= t.rows;
      uint8_t* stg = gen + STAGES * STAGE_BYTES + (warp - 2) * STG_WARP_BYTES;
#pragma unroll 1
      for (int c = half * (N_TILE / 2); c < (half + 1) * (N_TILE / 2); c += 32) {
        uint32_t g[32];
        uint32_t packed[16];
        if (SWIGLU) {
          uint32_t u[32];
          tmem_ld32(taddr + (uint32_t)c, g);
          tmem_ld32(taddr + (uint32_t)(128 + c), u);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float g0 = __uint_as_float(g[2 * j]), g1 = __uint_as_float(g[2 * j + 1]);
            const float u0 = __uint_as_float(u[2 * j]), u1 = __uint_as_float(u[2 * j + 1]);
            const float h0 = __fdividef(g0, 1.0f + __expf(-g0)) * u0;
            const float h1 = __fdividef(g1, 1.0f + __expf(-g1)) * u1;
            packed[j] = pack_bf16(h0, h1);
          }
        } else {
          tmem_ld32(taddr + (uint32_t)c, g);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j)
            packed[j] = pack_bf16(__uint_as_float(g[2 * j]), __uint_as_float(g[2 * j + 1]));
        }
        store_piece(packed, full_rows, row_ok, stg, &map_out, t.n0 + c, t.row0 + warp_row0, orow + c,
                    Nout - (t.n0 + c));
      }
      tc_fence_before();
      mbar_arrive_cluster(tempty_bar(b) & PEER_MASK);   // the leader waits for both CTAs' epilogues
    }
    if (lane == 0) bulk_wait_all();                      // this lane's stores have landed before the CTA ends
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();             // no signal of the peer can still be on its way to this CTA
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
  if (tid == 0 && *abort_flag && dev_status) atomicExch(dev_status, (int)CAPMOE_ETIMEOUT);
}


// Exercises the bounded wait on a barrier that nothing ever signals: the wait must run out, the
// kernel must return, and the status word must say so.  One warp, no tensor memory.
__global__ void k_wait_probe(long long limit_cycles, int32_t* __restrict__ dev_status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_cycles);
    if (!ok && dev_status) atomicExch(dev_status, (int)CAPMOE_ETIMEOUT);
  }
}

}  // namespace

int wait_probe(long long limit_cycles, int32_t* dev_status, cudaStream_t st) {
  k_wait_probe<<<1, 32, 0, st>>>(limit_cycles, dev_status);
  return check_launch();
}

bool ffn_tc_supported(int d, int F, int dtype) {
  return dtype == CAPMOE_BF16 && d % 64 == 0 && F % 64 == 0 && d >= 64 && F >= 64;
}

// E row segments [seg_begin[e], seg_end[e]); segment e multiplies with weight block e % w_mod
// (w_mod = 0: block e) out of n_w blocks.
int ffn_tc(const void* x_perm, const int32_t* seg_begin, const int32_t* seg_end, int E, int w_mod, int n_w, int d, int F,
           const void* w_gate, const void* w_up, const void* w_down, void* h_ws, void* y_perm, int64_t A_max,
           int D_straggler, int32_t* dev_status, int sched_slot, bool counters_cleared, cudaEvent_t mid, cudaStream_t st) {
  if (E > MAX_E) return CAPMOE_EUNSUPPORTED;
  alignas(64) CUtensorMap a1, bg, bu, a2, bd, o1, o2;
  if (!make_store_map(&o1, h_ws, (uint64_t)F, (uint64_t)A_max) ||
      !make_store_map(&o2, y_perm, (uint64_t)d, (uint64_t)A_max) ||
      !make_map(&a1, x_perm, (uint64_t)d, (uint64_t)A_max, 0, BM) ||
      !make_map(&bg, w_gate, (uint64_t)d, (uint64_t)F, (uint64_t)n_w, 128) ||
      !make_map(&bu, w_up, (uint64_t)d, (uint64_t)F, (uint64_t)n_w, 128) ||
      !make_map(&a2, h_ws, (uint64_t)F, (uint64_t)A_max, 0, BM) ||
      !make_map(&bd, w_down, (uint64_t)F, (uint64_t)d, (uint64_t)n_w, 256))
    return note_cuda(cudaErrorInvalidValue);
  cudaError_t err = cudaFuncSetAttribute(k_ffn_tc<MODE_GATE_UP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         SMEM_BYTES);
  if (err != cudaSuccess) return note_cuda(err);
  err = cudaFuncSetAttribute(k_ffn_tc<MODE_DOWN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (err != cudaSuccess) return note_cuda(err);
  int grid = sm_count();
  // Tile counters of the two launches (one per straggler group), in the caller's status block.
  // Against fixed lists the counter halved the DRAM reads of the Mixtral-shape gate/up GEMM and
  // measured 2-5 % faster on the gate/up GEMMs of the other long-segment shapes, equal on their
  // down GEMMs and on the single-CTA kernel's ragged workloads.
  int32_t *sched1 = nullptr, *sched2 = nullptr;
  if (dev_status && sched_slot == 0 && D_straggler <= CAPMOE_FFN_SCHED_GROUPS) {
    sched1 = dev_status + 1;
    sched2 = dev_status + 1 + CAPMOE_FFN_SCHED_GROUPS;
  } else if (dev_status && sched_slot == 1 && D_straggler == 0) {   // a layer's shared expert: one group
    sched1 = dev_status + 1 + 2 * CAPMOE_FFN_SCHED_GROUPS;
    sched2 = sched1 + 1;
  }
  if (sched1 && !counters_cleared) {
    const int rc0 = clear_words(dev_status + 1, CAPMOE_FFN_STATUS_WORDS - 1, nullptr, 0, st);
    if (rc0 != CAPMOE_OK) return rc0;
  }
  const int64_t avg_rows = A_max / E;
  const int variant = ffn_variant();
  const bool pairs_fit = grid >= 2 && (D_straggler == 0 || grid / 2 >= D_straggler);
  if (variant == FFN_SHORT && !pairs_fit) return CAPMOE_EUNSUPPORTED;
  if (variant == FFN_SHORT)
    return ffn_tc_short(true, true, x_perm, seg_begin, seg_end, E, w_mod, n_w, d, F, w_gate, w_up, w_down, h_ws, y_perm, A_max,
                        D_straggler, dev_status, sched1, sched2, mid, st);
  // Down GEMM of segments below about a thousand rows: the short-segment kernel (tokens in steps of
  // 16 on the N side).  With 256-row tiles most of such a launch's tensor and L2->SM time goes into the
  // padding of last tiles (a 547-row segment costs three tiles); measured 5-15 % faster on every
  // many-expert shape, drop mode and token count tried.  For the gate/up GEMM that form needs all of
  // tensor memory for one tile (gate and up accumulators), loses the overlap of epilogue and MMAs, and
  // measured slower except on the shortest segments: it keeps the token-major kernels.
  if (variant == FFN_SHORT_DOWN && !pairs_fit) return CAPMOE_EUNSUPPORTED;
  const bool short_down = variant == FFN_SHORT_DOWN || (variant == FFN_AUTO && pairs_fit && avg_rows < 1024);
  auto down_short = [&]() {
    return ffn_tc_short(false, true, x_perm, seg_begin, seg_end, E, w_mod, n_w, d, F, w_gate, w_up, w_down, h_ws, y_perm,
                        A_max, D_straggler, dev_status, sched1, sched2, nullptr, st);
  };
  // CTA pairs (256-row tiles) when the expert segments are long enough that the extra tail
  // padding does not matter, or when a typical segment (A_max / E rows) pads to about the same number
  // of rows with 256-row tiles as with 128-row ones (the pair kernel moves a third less through
  // shared memory per flop: 134 against 154 us on 137-row segments, Qwen shape at 2048 tokens; the
  // other way round on 547-row segments, 179 against 170 us)
  const int64_t pad256 = ceil_div(avg_rows, (int64_t)256) * 256, pad128 = ceil_div(avg_rows, (int64_t)128) * 128;
  const bool want_pairs = variant == FFN_AUTO || variant == FFN_SHORT_DOWN
                              ? avg_rows >= 1024 || (avg_rows > 0 && pad256 * 10 <= pad128 * 11)
                              : variant == FFN_PAIR;
  if (want_pairs && !pairs_fit && variant == FFN_PAIR) return CAPMOE_EUNSUPPORTED;
  if (want_pairs && pairs_fit) {
    alignas(64) CUtensorMap bd128;
    if (!make_map(&bd128, w_down, (uint64_t)F, (uint64_t)d, (uint64_t)n_w, 128)) return note_cuda(cudaErrorInvalidValue);
    int pairs = grid / 2;
    if (D_straggler > 0) pairs = (pairs / D_straggler) * D_straggler;
    err = cudaFuncSetAttribute(k_ffn_tc2<MODE_GATE_UP>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (err != cudaSuccess) return note_cuda(err);
    err = cudaFuncSetAttribute(k_ffn_tc2<MODE_DOWN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (err != cudaSuccess) return note_cuda(err);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see wait_for_previous_kernel()
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    err = cudaLaunchKernelEx(&cfg, k_ffn_tc2<MODE_GATE_UP>, a1, bg, bu, o1, seg_begin, seg_end, w_mod, E, d, F,
                             (__nv_bfloat16*)h_ws, D_straggler, dev_status, sched1);
    count_launch(1);
    if (err != cudaSuccess) return note_cuda(err);
    int rc2;
    if (mid && (rc2 = note_cuda(cudaEventRecord(mid, st))) != CAPMOE_OK) return rc2;
    if (short_down) return down_short();
    err = cudaLaunchKernelEx(&cfg, k_ffn_tc2<MODE_DOWN>, a2, bd128, bd128, o2, seg_begin, seg_end, w_mod, E, F, d,
                             (__nv_bfloat16*)y_perm, D_straggler, dev_status, sched2);
    count_launch(1);
    return note_cuda(err);
  }
  if (D_straggler > 0) {
    if (grid < D_straggler) return CAPMOE_EUNSUPPORTED;
    grid = (grid / D_straggler) * D_straggler;          // equal share of SMs per virtual device
  }
  int rc = note_cuda(launch_chained(k_ffn_tc<MODE_GATE_UP, 32>, (unsigned)grid, TC_THREADS, SMEM_BYTES, st, a1, bg, bu, o1,
                                    seg_begin, seg_end, w_mod, E, d, F, h_ws, D_straggler, dev_status, BNB, 0,
                                    (const float*)nullptr, BM, STAGES, STAGE_BYTES, RouterFused{}, sched1));
  count_launch(1);
  if (rc != CAPMOE_OK) return rc;
  if (mid && (rc = note_cuda(cudaEventRecord(mid, st))) != CAPMOE_OK) return rc;
  if (short_down) return down_short();
  rc = note_cuda(launch_chained(k_ffn_tc<MODE_DOWN, 32>, (unsigned)grid, TC_THREADS, SMEM_BYTES, st, a2, bd, bd, o2,
                                seg_begin, seg_end, w_mod, E, F, d, y_perm, D_straggler, dev_status, BNB, 0,
                                (const float*)nullptr, BM, STAGES, STAGE_BYTES, RouterFused{}, sched2));
  count_launch(1);
  return rc;
}

// Router on the same pipeline: logits[N,E] = x[N,d] . w_router[E,d]^T + bias in fp32 and, when
// `fused` points at the other outputs and E <= 64, softmax / top-k / load histogram in the epilogue.
bool router_tc_supported(int64_t N, int d, int E) { return d % 64 == 0 && d >= 64 && E <= 256 && N < (1ll << 31); }
bool router_tc_fusable(int E, int k) { return E <= 64 && k <= E; }

template <int MODE, int EPAD>
static int launch_router_tc(const CUtensorMap& ax, const CUtensorMap& bw, int grid, int d, int E, float* logits,
                            int n_mma, int64_t N, const float* bias, int tile_rows, int n_stages, int stage_stride,
                            const RouterFused& rf, cudaStream_t st) {
  cudaError_t err = cudaFuncSetAttribute(k_ffn_tc<MODE, EPAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         SMEM_BYTES);
  if (err != cudaSuccess) return note_cuda(err);
  // (the fourth tensor map is the FFN modes' output map: unused here)
  const int rc = note_cuda(launch_chained(k_ffn_tc<MODE, EPAD>, (unsigned)grid,
                                          MODE == MODE_ROUTER_FUSED ? RF_THREADS : TC_THREADS, SMEM_BYTES, st, ax, bw, bw, bw,
                                          (const int32_t*)nullptr, (const int32_t*)nullptr, 0, 1, d, E, (void*)logits, 0,
                                          (int32_t*)nullptr, n_mma, (int)N, bias, tile_rows, n_stages, stage_stride, rf,
                                          (int32_t*)nullptr));
  count_launch(1);
  return rc;
}

int router_tc(const void* x, const void* w_router, const float* bias, int64_t N, int d, int E, float* logits,
              float* scores, int32_t* topk_idx, float* topk_score, int32_t* load, int k, bool fused,
              cudaStream_t st) {
  const int n_mma = (E + 15) / 16 * 16;
  // The stage reads X once and is bound by HBM, so what matters is bytes in flight and an even
  // share of rows per SM: the tokens are cut into `rounds` tiles per SM of equal height (a
  // multiple of 8 rows, the swizzle atom; at most 128, the MMA's M).  The MMA always spans 128
  // rows; the rows past tile_rows cost nothing that is on the critical path.
  const int sms = sm_count();
  // (Every tile re-reads W_r through L2, and an SM's L2 port, not HBM, bounds the k-loop of small
  // tiles: capping tiles at 64 rows so that their epilogue hides under the next tile's loads measured
  // no faster at 16384 tokens and 5 % slower at 65536.)
  const int max_rows = 128;
  const int64_t rounds = ceil_div(N, (int64_t)max_rows * sms);
  int tile_rows = (int)((ceil_div(N, (int64_t)sms * rounds) + 7) / 8 * 8);
  if (tile_rows < 32) tile_rows = 32;
  if (tile_rows > max_rows) tile_rows = max_rows;
  // A stage holds tile_rows rows of A followed by n_mma rows of B (both multiples of 1 KB).  The
  // MMA reads 128 A rows whatever tile_rows is, so the last stage must leave room for that.
  const int b_bytes = n_mma * BK * 2;
  const int stage_stride = tile_rows * BK * 2 + b_bytes;
  int n_stages = (STAGES * STAGE_BYTES - A_BYTES - b_bytes) / stage_stride + 1;
  if (n_stages > MAX_STAGES) n_stages = MAX_STAGES;
  if (n_stages > (STAGES * STAGE_BYTES) / stage_stride) n_stages = (STAGES * STAGE_BYTES) / stage_stride;
  alignas(64) CUtensorMap ax, bw;
  if (!make_map(&ax, x, (uint64_t)d, (uint64_t)N, 0, (uint32_t)tile_rows) ||
      !make_map(&bw, w_router, (uint64_t)d, (uint64_t)E, 1, (uint32_t)n_mma))
    return note_cuda(cudaErrorInvalidValue);
  int grid = (int)ceil_div(N, tile_rows);
  if (grid > sms) grid = sms;
  const RouterFused rf{scores, topk_idx, topk_score, load, k};
  if (fused && router_tc_fusable(E, k)) {
    if (E <= 32)
      return launch_router_tc<MODE_ROUTER_FUSED, 32>(ax, bw, grid, d, E, logits, n_mma, N, bias, tile_rows, n_stages,
                                                     stage_stride, rf, st);
    return launch_router_tc<MODE_ROUTER_FUSED, 64>(ax, bw, grid, d, E, logits, n_mma, N, bias, tile_rows, n_stages,
                                                   stage_stride, rf, st);
  }
  return launch_router_tc<MODE_ROUTER, 32>(ax, bw, grid, d, E, logits, n_mma, N, bias, tile_rows, n_stages,
                                           stage_stride, rf, st);
}

}  // namespace capmoe
