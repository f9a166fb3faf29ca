// Shared pieces of the tcgen05 kernels: tile geometry, PTX wrappers (TMA, tensor memory, MMA),
// the tile queue, tile enumeration over row segments, and the host-side tensor-map builders.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "mbarrier.cuh"

namespace capmoe {
namespace {

constexpr int BM = 128;              // rows per tile (TMEM lanes)
constexpr int BK = 64;               // K elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int BNB = 256;             // B rows per stage = MMA N
constexpr int UMMA_K = 16;
constexpr int STAGES = 4;              // FFN ring depth (48 KB stages)
constexpr int MAX_STAGES = 16;         // router ring depth limit (smaller stages, deeper ring)
constexpr int A_BYTES = BM * BK * 2;         // 16 KB
constexpr int B_BYTES = BNB * BK * 2;        // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_WARPS = 8;              // two warps per TMEM lane quarter, each takes half the columns
constexpr int TC_THREADS = 64 + EPI_WARPS * 32;
// Fused router: four warps per lane quarter, each thread takes a quarter of its token's columns.
constexpr int RF_SUBS = 4;
constexpr int RF_THREADS = 64 + 4 * RF_SUBS * 32;
constexpr int RF_XCH_FLOATS = RF_SUBS * 128 + 128 + 4 * RF_SUBS * 128;   // max, sum relay, top-k candidates
constexpr int RF_SPREAD_ROWS = 64;        // row tiles up to this size share their tokens among all epilogue warps

constexpr int MAX_E = 256;
// Epilogue staging: each FFN epilogue warp packs a 32-row x 32-column bf16 piece of the output into
// 2 KB of shared memory (64-byte rows, 64-byte swizzle) and one lane hands it to TMA to store.
constexpr int STG_WARP_BYTES = 32 * 64;
constexpr int STG_BYTES = EPI_WARPS * STG_WARP_BYTES;      // 16 KB, right behind the operand ring
constexpr int TAIL_OFF = STAGES * STAGE_BYTES + STG_BYTES; // barriers and tables start here
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STG_BYTES + 1024 /*alignment slack*/ + 512 /*barriers*/ +
                           2 * (MAX_E + 1) * 4 + 8 + 256 * 4 /*router bias*/ + RF_XCH_FLOATS * 4 + MAX_E * 4 /*segment ends*/;
static_assert(SMEM_BYTES <= 227 * 1024, "dynamic shared memory limit of a thread block");
static_assert(RF_SPREAD_ROWS * 64 * 4 <= STG_BYTES, "the fused router's shared logits tile lives in the staging area");

// ---------------------------------------------------------------- PTX wrappers (mbarriers: mbarrier.cuh)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

// One lane of a converged warp, chosen by the hardware.  The compiler knows that the region this
// guards is single-threaded and issues the asynchronous instructions from uniform registers; with
// a plain `lane == 0` test each tcgen05.mma took ~90 cycles to issue, this way ~30.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
// Store of a shared-memory box through TMA (bulk async group of the issuing thread).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int c0, int c1, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all but the newest 0 groups of this thread have finished READING their shared-memory source
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// makes this thread's shared-memory writes visible to the async proxy (TMA) that will read them
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// One 32 x 32 bf16 piece of the output: lane r holds row r as 16 packed words.  With all 32 rows
// inside the segment the piece goes out as one TMA store (full 64-byte runs per row instead of 32
// scattered 16-byte stores per instruction, which made short-K GEMMs wait on their epilogue);
// otherwise the rows that exist are written directly.
__device__ __forceinline__ void store_piece(const uint32_t* packed, bool full_rows, bool row_ok, uint8_t* stg,
                                            const CUtensorMap* map_out, int col, int row0_of_warp,
                                            __nv_bfloat16* orow_c, int cols_left) {
  const int lane = threadIdx.x & 31;
  if (full_rows) {
    if (lane == 0) bulk_wait_read_all();                 // the previous piece has left the staging buffer
    __syncwarp();
    const uint32_t base = smem_u32(stg) + (uint32_t)lane * 64u;
#pragma unroll
    for (int v = 0; v < 4; ++v)
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + (uint32_t)((v ^ ((lane >> 1) & 3)) * 16)),
                   "r"(packed[4 * v]), "r"(packed[4 * v + 1]), "r"(packed[4 * v + 2]), "r"(packed[4 * v + 3])
                   : "memory");
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      tma_store_2d(map_out, col, row0_of_warp, smem_u32(stg));
      bulk_commit();
    }
  } else if (row_ok) {
#pragma unroll
    for (int v = 0; v < 4; ++v)
      if (v * 8 + 8 <= cols_left)
        *reinterpret_cast<uint4*>(orow_c + v * 8) =
            make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
  }
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows 128 bytes apart,
// 8-row groups 1024 bytes apart (stride byte offset), descriptor version 1 (Blackwell).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffffu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset
  d |= (uint64_t)1 << 46;                            // version
  d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
  return d;
}
// Instruction descriptor, kind::f16: D = fp32, A = B = bf16, both K-major, M = 128, N = n_mma
// (a multiple of 16 up to 256).
__host__ __device__ constexpr uint32_t make_idesc(int n_mma) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                     uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets row (lane base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
      : "r"(taddr)
      : "memory");
}
// Named barrier over `count` threads (whole warps), and the same with an AND over a predicate.
__device__ __forceinline__ void group_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ bool group_all(int id, int count, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %3, 0;\n\t"
      "bar.red.and.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(count), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;                // shared::cluster address of the even CTA's copy
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Tile queue of a CTA or a CTA pair.  With a scheduler counter the CTAs do not walk fixed lists of
// tiles: the (leader's) producer thread takes the next tile index from a global counter shortly
// before it needs it and hands it to every role (of both CTAs) through a small ring in shared
// memory (value + "full" barrier in each CTA, one "empty" barrier in the leader that all readers
// arrive on).  Tiles that are neighbours in the list (same weight tile, next row block) are then
// started within microseconds of each other whatever the speed of the SMs they run on, so their
// shared operand tiles meet in L2, and no pair is left with a longer list than the others.
__device__ __forceinline__ uint32_t peer_addr(uint32_t own) {   // same offset in CTA 1 of the pair
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, 1;" : "=r"(r) : "r"(own));
  return r;
}
constexpr int TQ = 4;
constexpr int TQ_READERS_PAIR = 2 + 2 * EPI_WARPS; // leader MMA thread, peer producer, epilogue warps of both CTAs
constexpr int TQ_READERS_ONE = 1 + EPI_WARPS;      // a CTA on its own: MMA thread and epilogue warps
template <bool PAIRED>
struct TileQueue {
  uint32_t full0, empty0, val0;      // shared::cta addresses of full[TQ], empty[TQ] (leader's used), tile[TQ]
  uint32_t rank;                     // CTA rank in the pair (0 for a CTA on its own)
  volatile int* abort_flag;
  __device__ __forceinline__ uint32_t full(int q) const { return full0 + 8u * (uint32_t)(q & (TQ - 1)); }
  __device__ __forceinline__ uint32_t empty(int q) const { return empty0 + 8u * (uint32_t)(q & (TQ - 1)); }
  __device__ __forceinline__ uint32_t val(int q) const { return val0 + 4u * (uint32_t)(q & (TQ - 1)); }
  // leader's producer thread: publish tile (or -1 = no more) as entry q; false if a wait ran out
  __device__ __forceinline__ bool put(int q, int tile) const {
    const uint32_t par = (((uint32_t)q / TQ) & 1u) ^ 1u;
    if (!mbar_wait(empty(q), par, abort_flag)) return false;     // only the count matters here
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(val(q)), "r"((uint32_t)tile) : "memory");
    mbar_arrive(full(q));
    if constexpr (PAIRED) {
      // the peer CTA's copy: a store that reports to the peer's barrier itself (no fence on this
      // thread, which has loads to issue)
      const uint32_t pfull = peer_addr(full(q));
      asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(pfull), "r"(4u) : "memory");
      asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.u32 [%0], %1, [%2];"
                   ::"r"(peer_addr(val(q))), "r"((uint32_t)tile), "r"(pfull)
                   : "memory");
    }
    return true;
  }
  // any other role (one thread, or one whole warp): entry q, or -2 if the wait ran out
  __device__ __forceinline__ int get(int q, bool whole_warp) const {
    const uint32_t par = ((uint32_t)q / TQ) & 1u;
    bool ok = mbar_wait(full(q), par, abort_flag);
    if (whole_warp) ok = __all_sync(0xffffffffu, ok);
    if (!ok) return -2;
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(val(q)) : "memory");
    if (whole_warp) __syncwarp();
    if (!whole_warp || (threadIdx.x & 31) == 0) {
      if (!PAIRED || rank == 0) mbar_arrive(empty(q));
      else mbar_arrive_cluster(empty(q) & PEER_MASK);
    }
    return (int)v;
  }
};

// ---------------------------------------------------------------- tile enumeration
struct Tile { int e, row0, rows, n0; };

// tile_start[e] = first tile of expert e; tiles of an expert: row block fastest, then column block.
// offs[e] / ends[e]: first row of segment e and the row after its last.
__device__ __forceinline__ bool locate_tile(int tile, int& cursor, const int* tile_start, const int* offs,
                                            const int* ends, int E, int n_tile, int bm, Tile& t) {
  while (cursor < E && tile >= tile_start[cursor + 1]) ++cursor;
  if (cursor >= E) return false;
  const int local = tile - tile_start[cursor];
  const int cnt = ends[cursor] - offs[cursor];
  const int nmb = (cnt + bm - 1) / bm;
  const int nb = local / nmb, mb = local - nb * nmb;
  t.e = cursor;
  t.row0 = offs[cursor] + mb * bm;
  t.rows = min(bm, cnt - mb * bm);
  t.n0 = nb * n_tile;
  return true;
}

// ---------------------------------------------------------------- CTA-pair variant (cta_group::2)
// Two CTAs of a cluster work on one 256 x 256 tile: each loads its own 128 rows of A and half of
// the B rows (for gate/up: CTA 0 the W_g tile, CTA 1 the W_u tile), the even CTA issues
// tcgen05.mma.cta_group::2 (M = 256) for both, and each CTA's tensor memory receives the 128
// accumulator rows it loaded A for.  Per k-block a CTA now fills 32 KB of shared memory instead of
// 48 KB for the same MMA work, which cuts L2->SM traffic by a third, and the ring is six deep.
// Every TMA load goes to the shared memory of the CTA that issued it; only the "stage free" and
// "accumulator ready" barrier signals of tcgen05.commit reach both CTAs.
constexpr int STAGES2 = 6;
constexpr int HALF_B_BYTES = 128 * BK * 2;                 // 16 KB
constexpr int STAGE2_BYTES = A_BYTES + HALF_B_BYTES;       // 32 KB per CTA
static_assert(STAGES2 * STAGE2_BYTES == STAGES * STAGE_BYTES, "both variants share one smem layout");

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                             uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void umma2(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                      uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the barrier at this offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3)
      : "memory");
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// bf16 tensor [rows, cols] (2D) or [batch, rows, cols] (3D), cols contiguous; box = box_rows x 64 columns.
bool make_map(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t batch, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {cols, rows, batch};
  cuuint64_t strides[2] = {cols * 2, cols * rows * 2};
  cuuint32_t box[3] = {(cuuint32_t)BK, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  const cuuint32_t rank = batch > 0 ? 3 : 2;
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// bf16 matrix [rows, cols] as 32 x 32 boxes with the 64-byte swizzle: the epilogue's TMA stores.
bool make_store_map(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {32, 32};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace
}  // namespace capmoe
