// Tensor-core product engine for sm_100a: persistent, warp-specialised tcgen05 kernel.
//
//   warp 0      TMA producer: cp.async.bulk.tensor loads of the A and B operand tiles into a ring of
//               128-byte-swizzled shared-memory stages, signalled through mbarriers
//   warp 1      allocates tensor memory and issues tcgen05.mma (one elected lane), fp32 accumulators
//               in tensor memory
//   warps 2..9  epilogue: tcgen05.ld of the accumulator (two warps per 32-lane quarter, alternating 32-column
//               blocks), the element-wise epilogue (store / polynomial / residual / norm partials), global
//               accesses coalesced through a per-warp staging buffer in shared memory
//
// Tile forms (BN = tile width, a multiple of 16 up to 256; K is walked in blocks of 128 bytes = 64 bf16 or
// 32 tf32 values):
//   M <= 128    one CTA, 128 x BN tile, two accumulator buffers (epilogue of tile i overlaps tile i+1)
//   M >  128    a cluster of two CTAs per 256 x BN tile (tcgen05 cta_group::2): each CTA stages 128 rows of A
//               and half of the B columns, the leader CTA issues one 256-row product for both, each CTA holds
//               its 128 accumulator rows in its own tensor memory, two accumulator buffers. A pipeline stage
//               covers two K blocks: the cost of one step of the two issuing threads (barrier wait, four
//               products at ~75 cycles of issue each, commit) otherwise exceeds the 512 cycles the tensor
//               pipe needs per K block (one K block per stage when two would not leave three stages).
//               DEFL_TC_PAIR=0 selects the older single-CTA form of the 256-row tile (two 128-row halves
//               sharing the B tile, one accumulator buffer).
// Either operand may be K-major (K contiguous in global memory) or MN-major; the shared-memory matrix
// descriptors and the instruction descriptor are built to match. No multicast copies: every CTA loads its own
// operands. Every wait is bounded: when one runs out the kernel raises DEFL_ST_DEVICE_WAIT in the status word,
// stops waiting and drains.
#include "common.cuh"
#include <cuda.h>
#include <cudaTypedefs.h>
#include <mutex>
#include <cstdlib>
#include <cstdio>

namespace defl {

namespace {

constexpr int KBYTES = 128;                 // bytes of K per stage row (one swizzle span)
constexpr int NUM_THREADS = 320;            // producer warp, MMA warp, eight epilogue warps
constexpr int EPI_WARPS = 8;
constexpr int STAGING_BYTES = 4096;         // per epilogue warp: one 32 x 32 block of 4-byte values
constexpr int AUX_AHEAD = 3;                // tiles (per CTA) by which the aux prefetch runs ahead
constexpr int MAX_STAGES = 6;
constexpr int SCHED_SLOTS = 8;              // tile numbers published ahead of the slowest reader (pair form)

struct TcParams {
  CUtensorMap tmA[2];
  CUtensorMap tmB[2];
  CUtensorMap tmAux;           // [batch, M, N] view of `aux`, used only to prefetch the epilogue's tile into L2
  int aux_prefetch;
  int nseg;
  int seg1_ident;              // segment 1 = A[1] tile (K offset by the tile's first column) x identity tile (same for every tile and matrix)
  int b_split;                 // 2: B is the sum of two operands (tmB[0] + tmB[1]) that share A; else 1
  int kblocks[2];              // pipeline steps per segment (a step covers `ksub` K blocks of 128 bytes)
  int ksub;                    // K blocks per pipeline stage (1 or 2)
  int kreal[2];                // K blocks of 128 bytes per segment (the last step of a segment may hold fewer than ksub)
  int M, N, batch;
  int BN;                      // tile width (UMMA N)
  int tile_m;                  // 128 or 256 rows per tile
  int pair;                    // 1: a cluster of two CTAs per 256-row tile (tcgen05 cta_group::2), each CTA 128 rows
  int tiles_m, tiles_n;
  int tiles_per_matrix;        // tiles enumerated per matrix (fewer than tiles_m * tiles_n for symmetric output)
  long long total_tiles;
  int a_mn_major, b_mn_major;  // 0 = K-major, 1 = MN-major
  int esize;                   // operand element size in bytes (2 bf16, 4 tf32)
  int stages;
  uint32_t a_stage_bytes, b_stage_bytes;   // b_stage_bytes covers all splits
  uint32_t b_split_bytes;                  // bytes of one B split within a stage
  uint32_t a_boxes, b_boxes;   // TMA boxes per stage per operand
  uint32_t a_box_bytes, b_box_bytes;
  uint32_t a_box_rows, b_box_rows;   // MN extent covered by one box (K-major) or 128B/esize (MN-major)
  uint32_t idesc;
  // epilogue
  int epilogue, out_dtype, aux_dtype, symmetric, round_tf32;
  int transposed;              // EPI_STORE: the tile is written transposed, element (i, j) at C[j * ldc + i]
  int dup_ok;                  // symmetric pair-form product of a matrix with itself, BN = 256: diagonal tiles share one operand fetch
  int diag_exact;              // symmetric output of two different operands: diagonal blocks mirrored element by element
  int aux_f16, out_f16;        // a 16-bit aux / output is IEEE half (else bf16); the operands' kind is in idesc
  void* C; long long ldc, batch_c;
  const void* aux; long long ld_aux, batch_aux;
  float alpha, aux_scale, pa, pb, pc;
  const float* alpha_dev; const float* aux_scale_dev;
  double* partials; int partials_per_batch;
  int* status;
  unsigned int* tile_counter;  // pair form: tiles beyond each pair's first are handed out through this counter (null: fixed stride)
  unsigned long long wait_ns;  // limit of every bounded wait
  int hold_stage;              // test hook (single-CTA form): the producer withholds the copies of this pipeline step (-1: none)
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One poll. The suspend-time hint lets the hardware park the thread until the phase completes or the time is up,
// instead of returning at once: a waiting producer or issuing thread then executes a handful of instructions per
// wait, not a spin loop that competes with the epilogue warps of its scheduler for issue slots.
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(20000u)
      : "memory");
  return ok;
}
// non-blocking probe of a barrier phase
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait. A short burst of polls first (the common case: the barrier flips within the hardware
// suspend window of try_wait); after that every poll also checks the CTA's abort flag and a wall-clock
// budget, so that a protocol error or a lost copy ends in a status bit instead of a hang.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, unsigned long long wait_ns) {
#pragma unroll 1
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > wait_ns) {
      *abort_flag = 1;
      if (status) atomicOr(status, 8);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// Pair mode (two CTAs of a cluster drive one tcgen05.mma.cta_group::2): the copy lands in the executing CTA's
// shared memory, its completion is counted on an mbarrier that may live in the peer CTA (a shared::cluster
// address). No multicast: every CTA fetches its own operand halves.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t bar_cluster, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
// (default semantics, release at CTA scope: what the arrival orders is the tensor-memory read-out, which the
// tcgen05 fences cover; a cluster-scope release would also wait for every global store of the thread to drain)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// 4-byte store into the other CTA's shared memory that counts as 4 transaction bytes on a barrier there: readers
// that wait on that barrier see the value, with no fence on either side (the way a bulk copy is seen)
__device__ __forceinline__ void st_async_u32(uint32_t addr_cluster, uint32_t v, uint32_t bar_cluster) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
               ::"r"(addr_cluster), "r"(v), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// asks the memory system to bring one tile of a tensor into L2 (no shared memory, no completion to wait for)
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* tm, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
               ::"l"(tm), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

template <int KIND_TF32>
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if (KIND_TF32) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
// 256-row product of a CTA pair: each CTA supplies 128 rows of A and half of the B columns from its own shared
// memory (same offsets in both), and receives its 128 rows of the accumulator in its own tensor memory
template <int KIND_TF32>
__device__ __forceinline__ void umma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if (KIND_TF32) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
// pair mode: arrives on the mbarrier at this shared-memory offset in BOTH CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
// arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading/stride byte offsets (all >> 4),
// version 1 at bit 46, 128-byte swizzle (layout type 2) at bits 61..63.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// constant upper part of a descriptor; the 14-bit start-address field (address >> 4) is added per product
__device__ __forceinline__ uint64_t smem_desc_hi(uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return make_smem_desc(0, lbo_bytes, sbo_bytes);
}

// ----------------------------------------------------------------------------- the kernel
// Tile geometry. tile_m = 128: one 128-row accumulator per tile, two accumulator buffers (the epilogue
// of tile i overlaps the products of tile i+1). tile_m = 256: two 128-row halves that share the B tile
// (half the shared-memory -> tensor-core operand traffic per flop, which is what bounds this kernel: the
// L2 -> SM path), both halves resident in tensor memory, so a single accumulator buffer.
struct TileInfo {
  int tn, tm, bz;
  int halves;     // bit mask of the 128-row halves this tile computes
  int n_eff;      // columns actually computed (multiple of 16)
  bool skip;
  bool dup;       // a full tile on the diagonal of a product of a matrix with itself: its B tile IS its A tile
};

__device__ __forceinline__ TileInfo tile_info(const TcParams& p, long long tile64) {
  TileInfo t;
  const int tile = (int)tile64;          // the host refuses launches with 2^31 tiles or more: 32-bit divisions
  if (p.symmetric) {
    // only tiles that reach the diagonal or lie right of it are enumerated, so that every CTA gets the same
    // share of real work: tile row tm starts at column tile (tm * tile_m) / BN
    t.bz = tile / p.tiles_per_matrix;
    int idx = tile - t.bz * p.tiles_per_matrix;
    int tm = 0;
    for (; tm < p.tiles_m; ++tm) {
      const int first = (tm * p.tile_m) / p.BN;
      const int cnt = p.tiles_n - first;
      if (idx < cnt) { t.tn = first + idx; break; }
      idx -= cnt;
    }
    t.tm = tm;
  } else {
    t.bz = tile / p.tiles_per_matrix;
    const int idx = tile - t.bz * p.tiles_per_matrix;
    t.tm = idx / p.tiles_n;
    t.tn = idx - t.tm * p.tiles_n;
  }
  const int row0 = t.tm * p.tile_m, col_end = (t.tn + 1) * p.BN;
  t.skip = p.symmetric && col_end <= row0;               // entirely below the diagonal
  t.halves = 1;
  if (p.tile_m == 256 && p.M - row0 > 128 && !(p.symmetric && col_end <= row0 + 128)) t.halves = 3;
  int rem = p.N - t.tn * p.BN;
  rem = p.pair ? ((rem + 31) & ~31) : ((rem + 15) & ~15);    // a pair splits the columns in two halves of 16k
  t.n_eff = rem < p.BN ? rem : p.BN;
  // X X^T / A A on the diagonal: the tile's B operand (this CTA's half of the tile's columns) is the same block of the
  // same matrix as its A operand (this CTA's 128 rows), in the same shared-memory layout: it is fetched once. Operand
  // fetch from L2 is what bounds the product, and a diagonal tile then moves half the bytes.
  t.dup = p.dup_ok && !t.skip && t.tn * p.BN == row0 && t.n_eff == p.BN;
  return t;
}


// Epilogue of one 128-row half of a tile for the calling warp's 32 rows (one row per lane). The two warps
// that share a tensor-memory lane quarter take alternate 32-column blocks. Per block: two 16-column
// tensor-memory loads and (when the operation reads `aux`) the global loads of both chunks are issued before
// anything is consumed, so that several requests per warp are in flight; then the element-wise operation and
// 16-byte stores. The kind is a template parameter so that the per-element code is branch-free.
template <int EPI>
__device__ __forceinline__ void load_aux16(const TcParams& p, bool take, bool vec, bool aux_bf16, size_t xoff, int gj0,
                                           float* x) {
  if (EPI == EPI_STORE) return;
  const uint16_t* auxh = reinterpret_cast<const uint16_t*>(p.aux);
  const float* auxf = reinterpret_cast<const float*>(p.aux);
  const bool f16 = p.aux_f16 != 0;
  if (!take) {
#pragma unroll
    for (int j = 0; j < 16; ++j) x[j] = 0.f;
  } else if (vec && aux_bf16) {
    const uint4* src = reinterpret_cast<const uint4*>(auxh + xoff);
    uint4 pk[2] = {src[0], src[1]};
    const uint32_t* hh = reinterpret_cast<const uint32_t*>(pk);
#pragma unroll
    for (int j = 0; j < 8; ++j) { const float2 f = unpack16x2(hh[j], f16); x[2 * j] = f.x; x[2 * j + 1] = f.y; }
  } else if (vec) {
    const float4* src = reinterpret_cast<const float4*>(auxf + xoff);
#pragma unroll
    for (int j = 0; j < 4; ++j) { const float4 f = src[j]; x[4 * j] = f.x; x[4 * j + 1] = f.y; x[4 * j + 2] = f.z; x[4 * j + 3] = f.w; }
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      x[j] = (gj0 + j < p.N) ? (aux_bf16 ? unpack16x2((uint32_t)auxh[xoff + j], f16).x : auxf[xoff + j]) : 0.f;
  }
}

template <int EPI>
__device__ __forceinline__ void finish16(const TcParams& p, const uint32_t* r, const float* x, int gi, int gi_warp0,
                                         int gj0, bool row_ok, bool vec, size_t crow, size_t cbatch, float alpha,
                                         float aux_scale, float& sq) {
  if (gj0 >= p.N) return;
  const bool out_bf16 = (p.out_dtype != F32);       // a 16-bit output type
  const bool f16 = p.out_f16 != 0;
  uint16_t* outh = reinterpret_cast<uint16_t*>(p.C);
  float* outf = reinterpret_cast<float*>(p.C);
  float v[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float a = __uint_as_float(r[j]);
    if (EPI == EPI_STORE) v[j] = alpha * a;
    else if (EPI == EPI_POLY) v[j] = p.pb * x[j] + p.pc * a + ((gi == gj0 + j) ? p.pa : 0.f);
    else if (EPI == EPI_AUX_PLUS) v[j] = aux_scale * x[j] + alpha * a;
    else v[j] = (row_ok && gj0 + j < p.N) ? (x[j] - a) : 0.f;
  }
  if (p.round_tf32) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = round_to_tf32(v[j]);
  }
  if (EPI == EPI_RESID_NORM) {
    float sqf = 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) sqf = fmaf(v[j], v[j], sqf);
    sq += sqf;
    return;
  }
  if (!row_ok) return;
  if (p.transposed) {
    // for a fixed column the 32 lanes are 32 consecutive rows of the product, one contiguous run of C
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int gj = gj0 + j;
      if (gj < p.N) {
        const size_t m = cbatch + (size_t)gj * p.ldc + gi;
        if (out_bf16) outh[m] = (uint16_t)pack16x2(v[j], 0.f, f16); else outf[m] = v[j];
      }
    }
    return;
  }
  // symmetric output: chunks entirely right of the warp's rows are stored like any other chunk and mirrored;
  // chunks that touch the diagonal go element by element; chunks left of it are skipped by the caller
  const bool mirror_all = p.symmetric && gj0 > gi_warp0 + 31;
  if (vec && (!p.symmetric || mirror_all)) {
    if (out_bf16) {
      uint4 pk[2];
      uint32_t* hh = reinterpret_cast<uint32_t*>(pk);
#pragma unroll
      for (int j = 0; j < 8; ++j) hh[j] = pack16x2(v[2 * j], v[2 * j + 1], f16);
      uint4* dst = reinterpret_cast<uint4*>(outh + crow + gj0);
      dst[0] = pk[0]; dst[1] = pk[1];
    } else {
      float4* dst = reinterpret_cast<float4*>(outf + crow + gj0);
#pragma unroll
      for (int j = 0; j < 4; ++j) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int gj = gj0 + j;
      if (gj < p.N && (!p.symmetric || gj >= gi)) {
        if (out_bf16) outh[crow + gj] = (uint16_t)pack16x2(v[j], 0.f, f16); else outf[crow + gj] = v[j];
      }
    }
  }
  if (p.symmetric) {
    // mirror image: for a fixed column the 32 lanes are 32 consecutive rows, i.e. one contiguous run
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int gj = gj0 + j;
      if (gj < p.N && gj > gi) {
        const size_t m = cbatch + (size_t)gj * p.ldc + gi;
        if (out_bf16) outh[m] = (uint16_t)pack16x2(v[j], 0.f, f16); else outf[m] = v[j];
      }
    }
  }
}

// Fast path of the epilogue for a full, aligned 32-row x 32-column block of a non-symmetric output: global
// memory is touched only in runs of 64 or 128 contiguous bytes. The accumulator comes out of tensor memory one
// ROW per lane, which would make every global access a 32-way scatter (one 16-byte piece in each of 32 rows:
// measured 2.3 TB/s for stores, 1.2 TB/s for loads). So the block goes through a 4 KB per-warp staging buffer in
// shared memory with an XOR swizzle: `aux` is fetched with coalesced loads, written to the buffer, and each lane
// reads back its row; the results take the same way in the other direction.
__device__ __forceinline__ uint32_t stage_off(int row, int piece, int rowb, int pp) {
  // rowb = bytes per row (64 or 128), pp = 16-byte pieces per row (4 or 8); rows of 64 bytes share a 128-byte line.
  // The key of a 64-byte row also takes in row >> 3: the transposed gather of a mirrored block reads, in one
  // instruction, the same column of rows 8 apart, which the key (row >> 1) & 3 alone left on one bank.
  const int key = (rowb == 64) ? (((row >> 1) ^ (row >> 3)) & 3) : (row & 7);
  return (uint32_t)(row * rowb + ((piece ^ key) << 4));
}

// Coalesced fetch of one 32 x 32 block of `aux` (rows gi_warp0.., columns gj0..) into a staging buffer, 16 bytes per
// lane and instruction, whole 64- or 128-byte row segments per warp instruction. The asynchronous form
// (cp.async) needs no registers for the data, so that the fetch of a warp's next block can be in flight while
// the current one is processed; rows past M are filled with zeros.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int ES>
__device__ __forceinline__ void aux_fetch_async(const TcParams& p, int lane, int gi_warp0, int gj0, int bz, uint8_t* stg) {
  constexpr int rowb = 32 * ES, pp = rowb >> 4, rpi = 32 / pp;     // rpi = rows covered by one warp instruction
  const uint8_t* abase = reinterpret_cast<const uint8_t*>(p.aux) +
                         ((size_t)bz * p.batch_aux + (size_t)gi_warp0 * p.ld_aux + gj0) * ES;
  const int prow = lane / pp, piece = lane % pp;
  const uint32_t sbase = smem_u32(stg);
#pragma unroll
  for (int i = 0; i < pp; ++i) {
    const int row = prow + rpi * i;
    const bool ok = gi_warp0 + row < p.M;
    cp_async16(sbase + stage_off(row, piece, rowb, pp), abase + (size_t)(ok ? row : 0) * p.ld_aux * ES + piece * 16, ok ? 16u : 0u);
  }
  cp_async_commit();
}

// Transposed store of one 32 x 32 block of 16-bit results (EPI_STORE): C[(gj0 + c) * ldc + gi_warp0 + r] = alpha acc[r][c].
// Each lane packs its row into 16 words of two columns, trades words with its neighbour lane so that a word holds
// two ROWS of one column, and writes it into the staging buffer laid out as the transposed block (32 columns x 64
// bytes, conflict-free); the block then leaves in 64-byte rows, 16 bytes per lane. A third of the instructions of
// gathering the transposed block element by element out of a row-major staging buffer. (Writing the block with one
// 2-byte store per lane and column instead, 64 contiguous bytes per warp instruction and no staging, takes the same
// 1.48 ms for the 48 x 1600 x 6400 apply product under the board's power cap: the epilogue is not what bounds it.)
template <bool F16O>
__device__ __forceinline__ void store_block_transposed16(const TcParams& p, const uint32_t* r, uint8_t* stg, int lane,
                                                         int gi_warp0, int gj0, int bz, float alpha) {
  uint32_t* T = reinterpret_cast<uint32_t*>(stg);          // [32 columns][16 words]
  const bool odd = (lane & 1) != 0;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const uint32_t w = pack16x2(alpha * __uint_as_float(r[2 * j]), alpha * __uint_as_float(r[2 * j + 1]), F16O);
    const uint32_t y = __shfl_xor_sync(0xffffffffu, w, 1);
    // even lane: column 2j, rows (mine, neighbour's); odd lane: column 2j + 1, rows (neighbour's, mine)
    const uint32_t word = odd ? __byte_perm(y, w, 0x7632) : __byte_perm(w, y, 0x5410);
    T[(2 * j + (odd ? 1 : 0)) * 16 + (lane >> 1)] = word;
  }
  __syncwarp();
  uint8_t* mbase = reinterpret_cast<uint8_t*>(p.C) + ((size_t)bz * p.batch_c + (size_t)gj0 * p.ldc + gi_warp0) * 2;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = (lane >> 2) + 8 * i;
    const uint4 q = *reinterpret_cast<const uint4*>(stg + c * 64 + (lane & 3) * 16);
    *reinterpret_cast<uint4*>(mbase + (size_t)c * p.ldc * 2 + (lane & 3) * 16) = q;
  }
  __syncwarp();
}

// The calling lane's row of one staged 32 x 32 block, 16 bytes at a time and in place: `aux` values in, results out
// (nothing is written for the residual norm, whose partial sum of squares is returned). The formats of two-byte
// values (F16A: `aux` is IEEE half, F16O: the output is; else bf16) and whether the block meets the diagonal (DIAG,
// the polynomial's identity term) are template parameters, so that the loop has no per-element tests. Rows past M
// need no test either: their `aux` was filled with zeros and so was their part of the A operand.
template <int EPI, int ES, bool F16A, bool F16O, bool DIAG>
__device__ __forceinline__ float transform_row(const TcParams& p, const uint32_t* r, uint8_t* stg, int lane, int gi, int gj0,
                                               float alpha, float aux_scale) {
  constexpr int rowb = 32 * ES, pp = rowb >> 4, epp = 16 / ES;   // epp = elements per 16-byte piece
  const bool rnd = (ES == 4) && p.round_tf32 != 0;
  float sqf = 0.f;
#pragma unroll
  for (int pc = 0; pc < pp; ++pc) {
    uint4* slot = reinterpret_cast<uint4*>(stg + stage_off(lane, pc, rowb, pp));
    float x[epp], v[epp];
    if (EPI != EPI_STORE) {
      const uint4 q = *slot;
      if (ES == 2) {
        const uint32_t* hh = reinterpret_cast<const uint32_t*>(&q);
#pragma unroll
        for (int j = 0; j < epp / 2; ++j) { const float2 f = unpack16x2(hh[j], F16A); x[2 * j] = f.x; x[2 * j + 1] = f.y; }
      } else {
        x[0] = __uint_as_float(q.x); x[1] = __uint_as_float(q.y); x[2 % epp] = __uint_as_float(q.z); x[3 % epp] = __uint_as_float(q.w);
      }
    }
#pragma unroll
    for (int j = 0; j < epp; ++j) {
      const int c = pc * epp + j;
      const float a = __uint_as_float(r[c]);
      if (EPI == EPI_STORE) v[j] = alpha * a;
      else if (EPI == EPI_POLY) v[j] = p.pb * x[j] + p.pc * a + ((DIAG && gi == gj0 + c) ? p.pa : 0.f);
      else if (EPI == EPI_AUX_PLUS) v[j] = aux_scale * x[j] + alpha * a;
      else v[j] = x[j] - a;
      if (rnd) v[j] = round_to_tf32(v[j]);
      if (EPI == EPI_RESID_NORM) sqf = fmaf(v[j], v[j], sqf);
    }
    if (EPI != EPI_RESID_NORM) {
      uint4 q;
      if (ES == 2) {
        uint32_t* hh = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
        for (int j = 0; j < epp / 2; ++j) hh[j] = pack16x2(v[2 * j], v[2 * j + 1], F16O);
      } else {
        q = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2 % epp]), __float_as_uint(v[3 % epp]));
      }
      *slot = q;
    }
  }
  return sqf;
}

// One complete 32 x 32 block whose `aux` values already sit (or are about to land) in `stg`. ES = element size of
// `aux` and of the output (the same type). Each lane turns its row of the staged block into results 16 bytes at
// a time, in place; the block then leaves with coalesced 16-byte stores. `pending` = number of cp.async groups
// that may still be in flight after this block's own (0 or 1).
template <int EPI, int ES, int PENDING>
__device__ __forceinline__ void epilogue_block_fast(const TcParams& p, uint32_t taddr, uint8_t* stg, int lane, int gi_warp0,
                                                    int gj0, int bz, float alpha, float aux_scale, float& sq) {
  constexpr int rowb = 32 * ES, pp = rowb >> 4, rpi = 32 / pp, epp = 16 / ES;   // epp = elements per 16-byte piece
  const int prow = lane / pp, piece = lane % pp;
  uint32_t r[32];
  tmem_ld16(taddr, r);
  tmem_ld16(taddr + 16u, r + 16);
  if (EPI != EPI_STORE) {
    cp_async_wait<PENDING>();
    __syncwarp();
  }
  tmem_ld_wait();
  if (EPI == EPI_STORE && ES == 2) {
    if (p.transposed) {            // (warp-uniform)
      if (p.out_f16) store_block_transposed16<true>(p, r, stg, lane, gi_warp0, gj0, bz, alpha);
      else store_block_transposed16<false>(p, r, stg, lane, gi_warp0, gj0, bz, alpha);
      return;
    }
  }
  const int gi = gi_warp0 + lane;
  // the formats of the two-byte types and the position of the diagonal are the same for the whole warp: one
  // branch per block selects a row loop without per-element tests
  const bool diag = (EPI == EPI_POLY) && gj0 < gi_warp0 + 32 && gj0 + 32 > gi_warp0;
  const int fmt = (ES == 2 ? ((EPI != EPI_STORE && p.aux_f16) ? 1 : 0) | ((EPI != EPI_RESID_NORM && p.out_f16) ? 2 : 0) : 0) |
                  (diag ? 4 : 0);
  float sqf;
  switch (fmt) {
    case 0: sqf = transform_row<EPI, ES, false, false, false>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
    case 1: sqf = transform_row<EPI, ES, true, false, false>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
    case 2: sqf = transform_row<EPI, ES, false, true, false>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
    case 3: sqf = transform_row<EPI, ES, true, true, false>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
    case 4: sqf = transform_row<EPI, ES, false, false, true>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
    case 5: sqf = transform_row<EPI, ES, true, false, true>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
    case 6: sqf = transform_row<EPI, ES, false, true, true>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
    default: sqf = transform_row<EPI, ES, true, true, true>(p, r, stg, lane, gi, gj0, alpha, aux_scale); break;
  }
  if (EPI == EPI_RESID_NORM) {
    sq += sqf;
    __syncwarp();
    return;
  }
  __syncwarp();
  if (!p.transposed) {
    uint8_t* cbase = reinterpret_cast<uint8_t*>(p.C) + ((size_t)bz * p.batch_c + (size_t)gi_warp0 * p.ldc + gj0) * ES;
#pragma unroll
    for (int i = 0; i < pp; ++i) {
      const int row = prow + rpi * i;
      const uint4 q = *reinterpret_cast<const uint4*>(stg + stage_off(row, piece, rowb, pp));
      if (gi_warp0 + row < p.M) *reinterpret_cast<uint4*>(cbase + (size_t)row * p.ldc * ES + piece * 16) = q;
    }
  }
  // (a transposed output is written the way a symmetric one is mirrored)
  if (p.transposed || (p.symmetric && gj0 > gi_warp0)) {
    // mirror image of a block above the diagonal (the caller guarantees 32 complete rows): transposed row c of the
    // block is 32 values = pp pieces of 16 bytes; pp consecutive lanes write one such row, each lane gathering its
    // epp values from one column of the staged block
    uint8_t* mbase = reinterpret_cast<uint8_t*>(p.C) + ((size_t)bz * p.batch_c + (size_t)gj0 * p.ldc + gi_warp0) * ES;
#pragma unroll
    for (int i = 0; i < pp; ++i) {
      const int c = rpi * i + prow;                 // column of the block = row of the mirror image
      const int cp = c / epp, ce = (c % epp) * ES;  // its piece and byte offset within a staged row
      uint4 q;
      if (ES == 2) {
        uint16_t h[8];
#pragma unroll
        for (int e = 0; e < 8; ++e)
          h[e] = *reinterpret_cast<const uint16_t*>(stg + stage_off(piece * epp + e, cp, rowb, pp) + ce);
        q = make_uint4((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16),
                       (uint32_t)h[4] | ((uint32_t)h[5] << 16), (uint32_t)h[6] | ((uint32_t)h[7] << 16));
      } else {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          w[e] = *reinterpret_cast<const uint32_t*>(stg + stage_off(piece * epp + e, cp, rowb, pp) + ce);
        q = make_uint4(w[0], w[1], w[2], w[3]);
      }
      *reinterpret_cast<uint4*>(mbase + (size_t)c * p.ldc * ES + piece * 16) = q;
    }
  }
  __syncwarp();
}

// the warp's complete 32-column blocks c0, c0 + 64, ... below `lim`; returns the first block not done. Two-byte
// types: the 4 KB staging buffer holds two blocks, and the fetch of block i+1 is issued before block i is
// processed. Four-byte types: one block at a time.
template <int EPI, int ES>
__device__ __forceinline__ int epilogue_fast_blocks(const TcParams& p, uint32_t taddr, uint8_t* stg, int lane, int gi_warp0,
                                                    int col0, int c0, int lim, int bz, float alpha, float aux_scale,
                                                    float& sq, int skip_c) {
  constexpr bool AHEAD = (ES == 2) && (EPI != EPI_STORE);
  int half = 0;
  // symmetric output: nothing to do for blocks entirely left of the warp's rows (they are written as mirror images)
  if (p.symmetric) while (c0 + 32 <= lim && col0 + c0 + 31 < gi_warp0) c0 += 64;
  // (the block on the diagonal of a plain symmetric store is left to the caller: see epilogue_half; it is the first
  // block of this walk when it belongs to this warp)
  if (c0 == skip_c) c0 += 64;
  __syncwarp();
  if (AHEAD && c0 + 32 <= lim) aux_fetch_async<ES>(p, lane, gi_warp0, col0 + c0, bz, stg);
#pragma unroll 1
  for (; c0 + 32 <= lim; c0 += 64) {
    uint8_t* cur = stg + (AHEAD ? half * (STAGING_BYTES / 2) : 0);
    if (AHEAD) {
      if (c0 + 96 <= lim) {
        aux_fetch_async<ES>(p, lane, gi_warp0, col0 + c0 + 64, bz, stg + (half ^ 1) * (STAGING_BYTES / 2));
        epilogue_block_fast<EPI, ES, 1>(p, taddr + (uint32_t)c0, cur, lane, gi_warp0, col0 + c0, bz, alpha, aux_scale, sq);
      } else {
        epilogue_block_fast<EPI, ES, 0>(p, taddr + (uint32_t)c0, cur, lane, gi_warp0, col0 + c0, bz, alpha, aux_scale, sq);
      }
      half ^= 1;
    } else {
      if (EPI != EPI_STORE) aux_fetch_async<ES>(p, lane, gi_warp0, col0 + c0, bz, cur);
      epilogue_block_fast<EPI, ES, 0>(p, taddr + (uint32_t)c0, cur, lane, gi_warp0, col0 + c0, bz, alpha, aux_scale, sq);
    }
  }
  return c0;
}

// One 32-column block (two 16-column chunks) through the general path: any alignment, ragged edges, and for a
// symmetric output exactly one computed value per pair (i, j), (j, i), stored at both places.
template <int EPI>
__device__ __forceinline__ void epilogue_block_general(const TcParams& p, uint32_t taddr, int c0, int gi, int gi_warp0, int col0,
                                                       int n_eff, bool row_ok, bool vec_ok, bool aux_bf16, size_t crow,
                                                       size_t cbatch, size_t xrow, float alpha, float aux_scale, float& sq) {
  const int gj0 = col0 + c0, gj1 = gj0 + 16;
  // symmetric output: nothing to do for a block entirely left of the warp's rows (warp-uniform)
  if (p.symmetric && gj0 + 31 < gi_warp0) return;
  const bool second = (c0 + 16 < n_eff);
  uint32_t r0[16], r1[16];
  __syncwarp();
  tmem_ld16(taddr + (uint32_t)c0, r0);
  if (second) tmem_ld16(taddr + (uint32_t)c0 + 16u, r1);
  const bool vec0 = vec_ok && (gj0 + 16 <= p.N) && ((gj0 & 7) == 0);
  const bool vec1 = vec_ok && (gj1 + 16 <= p.N) && ((gj1 & 7) == 0);
  float x0[16], x1[16];
  load_aux16<EPI>(p, row_ok && gj0 < p.N, vec0, aux_bf16, xrow + gj0, gj0, x0);
  load_aux16<EPI>(p, second && row_ok && gj1 < p.N, vec1, aux_bf16, xrow + gj1, gj1, x1);
  tmem_ld_wait();
  finish16<EPI>(p, r0, x0, gi, gi_warp0, gj0, row_ok, vec0, crow, cbatch, alpha, aux_scale, sq);
  if (second) finish16<EPI>(p, r1, x1, gi, gi_warp0, gj1, row_ok, vec1, crow, cbatch, alpha, aux_scale, sq);
}

template <int EPI>
__device__ __forceinline__ void epilogue_half(const TcParams& p, uint32_t taddr, int gi, int gi_warp0, int col0, int n_eff,
                                              int bz, int wsel, float alpha, float aux_scale, float& sq, uint8_t* stg,
                                              int lane) {
  const bool row_ok = gi < p.M;
  const bool aux_bf16 = (p.aux_dtype != F32);       // a 16-bit aux type
  const size_t cbatch = (size_t)bz * p.batch_c;
  const size_t crow = cbatch + (size_t)gi * p.ldc;
  const size_t xrow = (size_t)bz * p.batch_aux + (size_t)gi * p.ld_aux;
  const bool vec_ok = ((p.ldc & 7) == 0) && ((p.batch_c & 7) == 0) && ((p.ld_aux & 7) == 0 || EPI == EPI_STORE) &&
                      ((p.batch_aux & 7) == 0 || EPI == EPI_STORE);
  const bool a2 = (p.aux_dtype != F32), o2 = (p.out_dtype != F32);
  // the coalesced path wants `aux` and the output in the same type (true of every product the library makes)
  // (symmetric output: the mirror stores of the coalesced path assume 32 complete rows)
  const bool fast_ok = vec_ok && (EPI == EPI_STORE || EPI == EPI_RESID_NORM || a2 == o2) &&
                       (!p.symmetric || (gi_warp0 + 32 <= p.M && EPI != EPI_RESID_NORM)) &&
                       (!p.transposed || gi_warp0 + 32 <= p.M);
  int c0 = wsel * 32;
  if (fast_ok) {
    // the complete 32-column blocks come first; whatever is left (a ragged edge) takes the general path below
    int lim = p.N - col0;
    if (lim > n_eff) lim = n_eff;
    // A symmetric output may be the product of two DIFFERENT symmetric matrices (the apply step of the symmetric
    // filter, the Horner steps of a polynomial in the Gram matrix), whose computed (i, j) and (j, i) differ in the last
    // bits. Off the diagonal the mirror store makes the pair equal; the 32 x 32 block ON the diagonal must do the same
    // element by element, or an iterate picks up an antisymmetric part that the symmetric filter doubles at every step:
    // it takes the general path.
    // (A product of a matrix with itself, X X^T or A A, computes (i, j) and (j, i) from the same terms in the same
    // order: its diagonal blocks are symmetric to the bit and stay on the coalesced path.)
    int c_diag = -1;
    if ((EPI == EPI_STORE || EPI == EPI_POLY) && p.symmetric && p.diag_exact && gi_warp0 >= col0 && gi_warp0 - col0 < lim &&
        (((gi_warp0 - col0) >> 5) & 1) == wsel)
      c_diag = gi_warp0 - col0;
    const bool two = (EPI == EPI_STORE) ? o2 : a2;
    if (two) c0 = epilogue_fast_blocks<EPI, 2>(p, taddr, stg, lane, gi_warp0, col0, c0, lim, bz, alpha, aux_scale, sq, c_diag);
    else c0 = epilogue_fast_blocks<EPI, 4>(p, taddr, stg, lane, gi_warp0, col0, c0, lim, bz, alpha, aux_scale, sq, c_diag);
    if (c_diag >= 0)
      epilogue_block_general<EPI>(p, taddr, c_diag, gi, gi_warp0, col0, n_eff, row_ok, vec_ok, aux_bf16, crow, cbatch, xrow,
                                  alpha, aux_scale, sq);
  }
  for (; c0 < n_eff; c0 += 64)
    epilogue_block_general<EPI>(p, taddr, c0, gi, gi_warp0, col0, n_eff, row_ok, vec_ok, aux_bf16, crow, cbatch, xrow, alpha,
                                aux_scale, sq);
}

template <int KIND_TF32, int BSPLIT, int PAIR>
__global__ void __launch_bounds__(NUM_THREADS, 1) gemm_tc_kernel(const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t acc_full_bar[2];
  __shared__ __align__(8) uint64_t acc_empty_bar[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  // Pair form with a tile counter: the leader's producer publishes each tile number to both CTAs (sched_tile,
  // sched_full: a plain store and arrive at home, a 4-byte asynchronous store that completes the peer's barrier
  // there); every reader (the peer's producer, the issuing thread, the epilogue warps of both CTAs: 18 in all)
  // acknowledges on the leader's sched_empty before the slot is reused.
  __shared__ __align__(8) uint64_t sched_full[SCHED_SLOTS];
  __shared__ __align__(8) uint64_t sched_empty[SCHED_SLOTS];
  __shared__ int sched_tile[SCHED_SLOTS];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzled tiles need 1024-byte alignment
  const uint32_t sub_bytes = p.a_stage_bytes + p.b_stage_bytes;      // one K block of A and B
  const uint32_t stage_bytes = sub_bytes * (uint32_t)p.ksub;
  const int total_kblocks = p.kblocks[0] + (p.nseg > 1 ? p.kblocks[1] : 0);
  // Pair mode: CTA 0 of the cluster (the leader) issues the products for both CTAs and owns the barriers that
  // gate them (full_bar, acc_empty_bar); empty_bar and acc_full_bar exist in both CTAs and are signalled in both
  // by one commit. Every CTA loads, and writes out, its own 128 rows.
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const long long tile0 = PAIR ? (long long)(blockIdx.x >> 1) : (long long)blockIdx.x;
  const long long tile_step = PAIR ? (long long)(gridDim.x >> 1) : (long long)gridDim.x;
  const uint32_t nacc = (!PAIR && p.tile_m == 256) ? 1u : 2u;
  // Tiles: every pair starts on tile number = its own number; with a tile counter the later ones are whatever
  // the counter hands out next (so a pair that starts late, or meets costlier tiles, simply takes fewer),
  // otherwise they follow at a fixed stride.
  const bool dynamic = PAIR && p.tile_counter != nullptr;
  const uint32_t sfull0 = smem_u32(&sched_full[0]);
  const uint32_t sempty0_leader = PAIR ? map_to_cta(smem_u32(&sched_empty[0]), 0) : smem_u32(&sched_empty[0]);
  // one reader's step: wait for slot `it`, read the tile number, acknowledge; -1 = no more tiles, -2 = a wait ran out
  auto sched_read = [&](int it) -> long long {
    const uint32_t s2 = (uint32_t)it % SCHED_SLOTS, ph = ((uint32_t)it / SCHED_SLOTS) & 1u;
    if (!mbar_wait(sfull0 + 8u * s2, ph, &abort_flag, p.status, p.wait_ns)) return -2;
    const int tnum = *reinterpret_cast<volatile int*>(&sched_tile[s2]);
    mbar_arrive_cluster(sempty0_leader + 8u * s2);
    return (long long)tnum;
  };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&acc_full_bar[a]), 1);
      mbar_init(smem_u32(&acc_empty_bar[a]), PAIR ? 2 * EPI_WARPS : EPI_WARPS);
    }
    for (int s2 = 0; s2 < SCHED_SLOTS; ++s2) {
      mbar_init(smem_u32(&sched_full[s2]), 1);
      mbar_init(smem_u32(&sched_empty[s2]), 2 * EPI_WARPS + 2);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (PAIR) { tmem_alloc_pair(smem_u32(&tmem_base_slot), 512); tmem_relinquish_pair(); }
    else { tmem_alloc(smem_u32(&tmem_base_slot), 512); tmem_relinquish(); }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();      // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // The whole warp runs the loop: lane 0 waits for the stage and posts the expected byte count, then every lane
    // issues ONE of the step's copies (operand, K block, box, split fixed per lane), so that the copies of a step
    // leave in one warp instruction instead of one thread instruction each (a thread-serial issue of 4-6 copies
    // took longer than the tensor pipe needs for the step). Everything the loop needs sits in registers.
    {
      uint32_t stage = 0, phase = 0;
      const int arow = PAIR ? (int)rank * 128 : 0;              // this CTA's rows within the tile
      const int kstep = KBYTES / p.esize;
      const int a_boxes = (int)p.a_boxes, b_boxes = (int)p.b_boxes;
      const uint32_t nstages = (uint32_t)p.stages;
      const int ksub = p.ksub;
      const uint32_t tx_bytes = PAIR ? 2u * stage_bytes : stage_bytes;   // a pair counts both CTAs' copies on the leader's barrier
      const uint32_t tx_sub_bytes = PAIR ? 2u * sub_bytes : sub_bytes;
      const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
      const uint32_t full0_sig = PAIR ? map_to_cta(full0, 0) : full0;    // the barrier the copies signal
      const int BN = p.BN, tile_m = p.tile_m, nseg = p.nseg;
      const bool aux_prefetch = p.aux_prefetch != 0;
      // this lane's copy within a step (the host guarantees at most 32 copies per step), fixed for the launch
      const int per_sub = a_boxes + BSPLIT * b_boxes;
      const int ops = ksub * per_sub;
      const int my_sub = lane / per_sub;
      int my_r = lane - my_sub * per_sub;
      const bool my_on = lane < ops;
      const bool my_a = my_r < a_boxes;
      int my_sp = 0;
      if (!my_a) { my_r -= a_boxes; my_sp = my_r / b_boxes; my_r -= my_sp * b_boxes; }
      const int my_mn_off = my_r * (int)(my_a ? p.a_box_rows : p.b_box_rows);
      const uint32_t my_dst_off = (uint32_t)my_sub * sub_bytes +
                                  (my_a ? (uint32_t)my_r * p.a_box_bytes
                                        : p.a_stage_bytes + (uint32_t)my_sp * p.b_split_bytes + (uint32_t)my_r * p.b_box_bytes);
      const bool my_mn_major = (my_a ? p.a_mn_major : p.b_mn_major) != 0;
      const int my_k_off = my_sub * kstep;
      const CUtensorMap* my_tm0 = my_a ? &p.tmA[0] : &p.tmB[BSPLIT > 1 ? my_sp : 0];
      const CUtensorMap* my_tm1 = my_a ? &p.tmA[1] : &p.tmB[BSPLIT > 1 ? my_sp : 1];
      const int kblocks0 = p.kblocks[0], kblocks1 = p.kblocks[1], kreal0 = p.kreal[0], kreal1 = p.kreal[1];
      const long long total_tiles = p.total_tiles;
      const uint32_t sfull0_peer = PAIR ? map_to_cta(sfull0, 1) : 0u;
      const uint32_t stile0_peer = PAIR ? map_to_cta(smem_u32(&sched_tile[0]), 1) : 0u;
      const long long npairs = tile_step;
      // tickets drawn from the counter by all pairs together: one per tile beyond the first round, plus the one
      // per pair that tells it to stop; whoever draws the last one puts the counter back to zero
      const long long last_ticket = (total_tiles > npairs ? total_tiles - npairs : 0) + npairs - 1;
      unsigned int ticket = 0;
      for (int it = 0;; ++it) {
        long long tile;
        if (!dynamic) {
          tile = tile0 + (long long)it * tile_step;
          if (tile >= total_tiles) break;
        } else {
          long long tl = 0;
          if (lane == 0) {
            if (rank == 0) {
              if (it == 0) {
                tl = tile0;
              } else {
                tl = npairs + (long long)ticket;
                if ((long long)ticket == last_ticket) atomicExch(p.tile_counter, 0u);
                if (tl >= total_tiles) tl = -1;
              }
              const uint32_t s2 = (uint32_t)it % SCHED_SLOTS, ph = ((uint32_t)it / SCHED_SLOTS) & 1u;
              if (!mbar_wait(smem_u32(&sched_empty[s2]), ph ^ 1u, &abort_flag, p.status, p.wait_ns)) tl = -2;
              if (tl != -2) {
                sched_tile[s2] = (int)tl;
                mbar_arrive(sfull0 + 8u * s2);
                st_async_u32(stile0_peer + 4u * s2, (uint32_t)(int)tl, sfull0_peer + 8u * s2);
                // the next tile's ticket: its latency hides behind this tile's copies
                if (tl >= 0) ticket = atomicAdd(p.tile_counter, 1u);
              }
            } else {
              // the peer's slot completes on this arrival plus the 4 bytes the leader sends
              mbar_expect_tx(sfull0 + 8u * ((uint32_t)it % SCHED_SLOTS), 4u);
              tl = sched_read(it);
            }
          }
          tile = __shfl_sync(0xffffffffu, tl, 0);
          if (tile < 0) break;
        }
        const TileInfo t = tile_info(p, tile);
        if (t.skip) continue;
        // the epilogues read the matching tile of `aux`: start moving it from HBM into L2 well ahead
        // (AUX_AHEAD tiles of this CTA; short main loops leave no time otherwise)
        if (aux_prefetch && !dynamic && lane == 0) {
          if (tile == tile0) {
            for (int d = 0; d < AUX_AHEAD; ++d) {
              const long long tp = tile + (long long)d * tile_step;
              if (tp >= p.total_tiles) break;
              const TileInfo u = tile_info(p, tp);
              if (!u.skip) tma_prefetch_3d(&p.tmAux, u.tn * BN, u.tm * tile_m + arow, u.bz);
            }
          }
          const long long tp = tile + (long long)AUX_AHEAD * tile_step;
          if (tp < p.total_tiles) {
            const TileInfo u = tile_info(p, tp);
            if (!u.skip) tma_prefetch_3d(&p.tmAux, u.tn * BN, u.tm * tile_m + arow, u.bz);
          }
        }
        const int a_mn0 = t.tm * tile_m + arow;
        const int b_loc0 = PAIR ? (int)rank * (t.n_eff >> 1) : 0;                // a pair: this CTA's half of the columns
        const int b_mn0 = t.tn * BN + b_loc0;
        bool live = true;
        for (int seg = 0; seg < nseg && live; ++seg) {
          const int nkb = seg ? kblocks1 : kblocks0;
          int left = seg ? kreal1 : kreal0;                   // K blocks of the segment not yet requested
          const CUtensorMap* tm = seg ? my_tm1 : my_tm0;
          // identity segment: A is read at K = the tile's own columns, B is the same identity tile for every tile
          const bool ident = seg == 1 && p.seg1_ident != 0;
          const int my_mn = (my_a ? a_mn0 : (ident ? b_loc0 : b_mn0)) + my_mn_off;
          const int bz = (ident && !my_a) ? 0 : t.bz;
          int kc = my_k_off + ((ident && my_a) ? t.tn * BN : 0);
          for (int kb = 0; kb < nkb; ++kb, left -= ksub, kc += ksub * kstep) {
            int ok = 1;
            if (lane == 0) ok = mbar_wait(empty0 + 8u * stage, phase ^ 1u, &abort_flag, p.status, p.wait_ns) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) { live = false; break; }
            const int nsub = left < ksub ? left : ksub;       // the last step of a segment may be short
            const bool dup = t.dup;
            // test hook of the bounded waits (single-CTA form): this step of the CTA's first tile is neither announced
            // nor copied, so the consumer's wait for it runs out with nothing in flight
            if (!PAIR && p.hold_stage >= 0 && it == 0 && seg == 0 && kb == p.hold_stage) {
              if (++stage == nstages) { stage = 0; phase ^= 1u; }
              continue;
            }
            if (lane == 0 && (!PAIR || rank == 0))
              mbar_expect_tx(full0 + 8u * stage, dup ? (PAIR ? 2u : 1u) * p.a_stage_bytes * (uint32_t)nsub
                                                     : (nsub == ksub ? tx_bytes : tx_sub_bytes * (uint32_t)nsub));
            // (the part of a K block past the end of K is filled with zeros by the copy engine and adds nothing)
            if (my_on && my_sub < nsub && (my_a || !dup)) {
              const uint32_t fb = full0_sig + 8u * stage;
              const uint32_t dst = smem_base + stage * stage_bytes + my_dst_off;
              const int c0 = my_mn_major ? my_mn : kc, c1 = my_mn_major ? kc : my_mn;
              if (PAIR) tma_load_3d_pair(dst, tm, fb, c0, c1, bz);
              else tma_load_3d(dst, tm, fb, c0, c1, bz);
            }
            __syncwarp();
            if (++stage == nstages) { stage = 0; phase ^= 1u; }
          }
        }
        if (!live) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      // descriptor start addresses advance in units of 16 bytes
      const uint32_t a_kstep16 = (p.a_mn_major ? (uint32_t)(32 / p.esize) * 128u : 32u) >> 4;   // per UMMA K step
      const uint32_t b_kstep16 = (p.b_mn_major ? (uint32_t)(32 / p.esize) * 128u : 32u) >> 4;
      const uint64_t a_hi = smem_desc_hi(p.a_mn_major ? p.a_box_bytes : 16u, 1024u);
      const uint64_t b_hi = smem_desc_hi(p.b_mn_major ? p.b_box_bytes : 16u, 1024u);
      const uint32_t a_half16 = (128u * KBYTES) >> 4;   // rows 128..255 of the A tile (either major)
      const uint32_t split16 = p.b_split_bytes >> 4;
      const uint32_t stage16 = stage_bytes >> 4, sub16 = sub_bytes >> 4, a_stage16 = p.a_stage_bytes >> 4, base16 = smem_base >> 4;
      const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
      const uint32_t nstages = (uint32_t)p.stages;
      const int ksub = p.ksub;
      const int kreal0 = p.kreal[0], kreal1 = p.kreal[1], steps0 = p.kblocks[0];
      const uint32_t idesc0 = p.idesc;
      const bool tall = !PAIR && p.tile_m == 256;
      // The number and geometry of the NEXT tile are worked out in the middle of the current one (after the products
      // of its last step but one have been issued, while the tensor pipe is busy with them), so that at the tile
      // boundary the thread goes straight from the last commit to the first product of the next tile.
      auto next_tile = [&](int it) -> long long {
        if (dynamic) return sched_read(it);
        const long long tl = tile0 + (long long)it * tile_step;
        return tl < p.total_tiles ? tl : -1;
      };
      const int prep = total_kblocks >= 2 ? total_kblocks - 2 : 0;
      int it = 0;
      long long nxt = next_tile(it);
      TileInfo tnx;
      if (nxt >= 0) tnx = tile_info(p, nxt);
      while (nxt >= 0) {
        const TileInfo t = tnx;
        ++it;
        if (t.skip) {
          nxt = next_tile(it);
          if (nxt >= 0) tnx = tile_info(p, nxt);
          continue;
        }
        if (!mbar_wait(smem_u32(&acc_empty_bar[acc]), acc_phase ^ 1u, &abort_flag, p.status, p.wait_ns)) break;
        tc_fence_after();
        const uint32_t idesc = idesc0 | ((uint32_t)(t.n_eff >> 3) << 17);
        const uint32_t d0 = tmem_base + (tall ? 0u : acc * 256u);
        const bool two = !PAIR && (t.halves & 2) != 0;
        bool ok = true;
        uint32_t accum = 0;                                   // the first product of a tile overwrites the accumulator
        int left = kreal0;                                    // K blocks not yet multiplied in the current segment
        uint32_t ready = 0;                                   // the next stage was seen full while this one was issued
        for (int kb = 0; kb < total_kblocks; ++kb, left -= ksub) {
          if (kb == steps0) left = kreal1;
          if (!ready && !mbar_wait(full0 + 8u * stage, phase, &abort_flag, p.status, p.wait_ns)) { ok = false; break; }
          tc_fence_after();
          {
            // probe the following stage now: the answer arrives while this stage's products are issued
            const uint32_t ns = (stage + 1 == nstages) ? 0u : stage + 1;
            ready = (kb + 1 < total_kblocks) ? mbar_test(full0 + 8u * ns, ns == 0u ? phase ^ 1u : phase) : 0u;
          }
          const int nsub = left < ksub ? left : ksub;
          for (int sub = 0; sub < nsub; ++sub) {
            const uint32_t sa16 = base16 + stage * stage16 + (uint32_t)sub * sub16;
            const uint32_t sb16 = t.dup ? sa16 : sa16 + a_stage16;
#pragma unroll
            for (int kk = 0; kk < KBYTES / 32; ++kk) {
              const uint64_t adesc = a_hi | (uint64_t)(sa16 + kk * a_kstep16);
              const uint64_t bdesc = b_hi | (uint64_t)(sb16 + kk * b_kstep16);
              if (PAIR) {
                umma_pair<KIND_TF32>(d0, adesc, bdesc, idesc, accum);
                if (BSPLIT == 2) umma_pair<KIND_TF32>(d0, adesc, bdesc + split16, idesc, 1u);
              } else {
                umma<KIND_TF32>(d0, adesc, bdesc, idesc, accum);
                if (two) umma<KIND_TF32>(d0 + 256u, adesc + a_half16, bdesc, idesc, accum);
                if (BSPLIT == 2) {
                  umma<KIND_TF32>(d0, adesc, bdesc + split16, idesc, 1u);
                  if (two) umma<KIND_TF32>(d0 + 256u, adesc + a_half16, bdesc + split16, idesc, 1u);
                }
              }
              accum = 1u;
            }
          }
          // frees the stage (in both CTAs of a pair) once these products are done
          if (PAIR) umma_commit_pair(empty0 + 8u * stage); else umma_commit(empty0 + 8u * stage);
          if (++stage == nstages) { stage = 0; phase ^= 1u; }
          if (kb == prep) {
            if (total_kblocks == 1) {      // a one-step tile: the accumulator is complete, say so before looking ahead
              if (PAIR) umma_commit_pair(smem_u32(&acc_full_bar[acc])); else umma_commit(smem_u32(&acc_full_bar[acc]));
            }
            nxt = next_tile(it);
            if (nxt >= 0) tnx = tile_info(p, nxt);
          }
        }
        if (!ok) break;
        if (total_kblocks != 1) {
          if (PAIR) umma_commit_pair(smem_u32(&acc_full_bar[acc])); else umma_commit(smem_u32(&acc_full_bar[acc]));   // accumulator complete
        }
        if (++acc == nacc) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;                 // tensor-memory lane quarter this warp may read
    const int wsel = (warp - 2) >> 2;       // which of the two warps of that quarter: alternate 32-column blocks
    uint8_t* stg = smem_raw + (smem_base - smem_u32(smem_raw)) + (uint32_t)p.stages * stage_bytes + (uint32_t)(warp - 2) * STAGING_BYTES;
    uint32_t acc = 0, acc_phase = 0;
    const int h_first = PAIR ? (int)rank : 0;
    const int h_last = PAIR ? (int)rank : ((p.tile_m == 256) ? 1 : 0);
    for (int it = 0;; ++it) {
      long long tile;
      if (!dynamic) {
        tile = tile0 + (long long)it * tile_step;
        if (tile >= p.total_tiles) break;
      } else {
        long long tl = 0;
        if (lane == 0) tl = sched_read(it);
        tile = __shfl_sync(0xffffffffu, tl, 0);
        if (tile < 0) break;
      }
      const TileInfo t = tile_info(p, tile);
      if (t.skip) continue;
      const int tn = t.tn, tm = t.tm, bz = t.bz;
      const bool ok = mbar_wait(smem_u32(&acc_full_bar[acc]), acc_phase, &abort_flag, p.status, p.wait_ns);
      if (!ok) break;
      tc_fence_after();
      float alpha = p.alpha, aux_scale = p.aux_scale;
      if (p.alpha_dev) alpha *= p.alpha_dev[bz];
      if (p.aux_scale_dev) aux_scale *= p.aux_scale_dev[bz];
      for (int h = h_first; h <= h_last; ++h) {
        float sq = 0.f;      // the warp's sum of squares over this tile half (at most 32 x 256 values), fp32
        if (t.halves & (1 << h)) {
          const uint32_t tcol = (!PAIR && p.tile_m == 256) ? (uint32_t)h * 256u : acc * 256u;
          const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + tcol;
          const int gi0 = tm * p.tile_m + h * 128 + q * 32, gi = gi0 + lane;
          switch (p.epilogue) {
            case EPI_STORE: epilogue_half<EPI_STORE>(p, taddr, gi, gi0, tn * p.BN, t.n_eff, bz, wsel, alpha, aux_scale, sq, stg, lane); break;
            case EPI_POLY: epilogue_half<EPI_POLY>(p, taddr, gi, gi0, tn * p.BN, t.n_eff, bz, wsel, alpha, aux_scale, sq, stg, lane); break;
            case EPI_AUX_PLUS: epilogue_half<EPI_AUX_PLUS>(p, taddr, gi, gi0, tn * p.BN, t.n_eff, bz, wsel, alpha, aux_scale, sq, stg, lane); break;
            default: epilogue_half<EPI_RESID_NORM>(p, taddr, gi, gi0, tn * p.BN, t.n_eff, bz, wsel, alpha, aux_scale, sq, stg, lane); break;
          }
        }
        if (p.epilogue == EPI_RESID_NORM) {
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
          if (lane == 0)
            p.partials[(long long)bz * p.partials_per_batch + (((long long)tm * p.tiles_n + tn) * (p.tile_m == 256 ? 2 : 1) + h) * EPI_WARPS + (warp - 2)] = sq;
        }
      }
      // release the accumulator buffer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty_bar[acc]), 0));
        else mbar_arrive(smem_u32(&acc_empty_bar[acc]));
      }
      if (++acc == nacc) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (abort_flag && threadIdx.x == 0) {
    // a wait ran out: give copies that may still be in flight a bounded time to land before the
    // shared memory is released
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) { }
  }
  __syncthreads();
  if (PAIR) cluster_sync_all();      // nothing of this CTA is released while the peer may still signal or read it
  if (warp == 1) {
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512);
  }
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

struct OperandPlan {
  bool mn_major;
  uint32_t boxes, box_bytes, box_rows, stage_bytes;
};

// Operand viewed as [batch][MN][K] with element strides s_mn, s_k. One of the strides must be 1.
bool plan_operand(long long s_mn, long long s_k, int tile_mn, int esize, OperandPlan* pl) {
  const int span = KBYTES / esize;   // elements per 128 bytes
  if (s_k == 1) {
    pl->mn_major = false;
    pl->boxes = 1;
    pl->box_rows = tile_mn;
    pl->box_bytes = (uint32_t)tile_mn * KBYTES;
    pl->stage_bytes = pl->box_bytes;
    return true;
  }
  if (s_mn == 1) {
    pl->mn_major = true;
    pl->boxes = (tile_mn + span - 1) / span;
    pl->box_rows = span;
    pl->box_bytes = (uint32_t)span * KBYTES;     // span K-rows of 128 bytes
    pl->stage_bytes = pl->boxes * pl->box_bytes;
    return true;
  }
  return false;
}

bool encode_map(CUtensorMap* tm, const void* base, int esize, bool tf32, bool mn_major, long long MN, long long K,
                long long s_mn, long long s_k, long long batch, long long batch_stride, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  const uint32_t span = KBYTES / esize;
  cuuint64_t dims[3];
  cuuint64_t strides[2];
  cuuint32_t box[3];
  cuuint32_t estr[3] = {1, 1, 1};
  if (!mn_major) {          // inner = K
    dims[0] = (cuuint64_t)K; dims[1] = (cuuint64_t)MN; dims[2] = (cuuint64_t)batch;
    strides[0] = (cuuint64_t)s_mn * esize; strides[1] = (cuuint64_t)batch_stride * esize;
    box[0] = span; box[1] = box_rows; box[2] = 1;
  } else {                  // inner = MN
    dims[0] = (cuuint64_t)MN; dims[1] = (cuuint64_t)K; dims[2] = (cuuint64_t)batch;
    strides[0] = (cuuint64_t)s_k * esize; strides[1] = (cuuint64_t)batch_stride * esize;
    box[0] = span; box[1] = span; box[2] = 1;
  }
  if (batch == 1) strides[1] = strides[0] * dims[1];
  // (16-bit operands: the copy engine only needs the element size; bf16 and IEEE half tiles move alike)
  const CUtensorMapDataType dt = (esize == 2) ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                              : (tf32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32);
  const CUresult r = enc(tm, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

const TcKnobs kDefaultKnobs = {0, 0, 0, 0, -1, 0, 0, 0, 0, 0};

int choose_bn(int N, bool pair, const TcKnobs& kn) {
  const int q = pair ? 32 : 16;
  if (kn.bn >= q && kn.bn <= 256 && kn.bn % q == 0) return kn.bn;
  // widest tile; edge tiles only compute the columns that exist (rounded up to 16, or 32 for a CTA pair), so
  // a wide tile wastes at most q - 1 columns per tile row
  const int r = (N + q - 1) & ~(q - 1);
  return r < 256 ? r : 256;
}

int choose_tile_m_impl(int M, const TcKnobs& kn) {
  if (kn.tile_m == 128 || kn.tile_m == 256) return kn.tile_m;
  // (128-row tiles for narrow outputs whose 256-row tiles fill the last wave of CTAs badly were measured: slower)
  return M > 128 ? 256 : 128;
}

// 256-row tiles are computed by a cluster of two CTAs (tcgen05 cta_group::2) unless the knob asks for the
// single-CTA form (two 128-row halves in one CTA)
bool choose_pair(int M, int N, const TcKnobs& kn) {
  if (choose_tile_m_impl(M, kn) != 256) return false;
  if (kn.pair >= 0) return kn.pair != 0;
  // (pair_min_n: outputs narrower than this take the single-CTA form; measured on the range finder's
  // 48-column panels the pair streams A faster, 4.9-5.1 against 4.3-4.6 TB/s, so the default keeps every width)
  return N >= kn.pair_min_n;
}

// cached encode: the same (address, shape, strides, box) gives the same descriptor
bool cached_map(TmCache* cache, CUtensorMap* tm, const void* base, int esize, bool tf32, bool mn_major, long long MN, long long K,
                long long s_mn, long long s_k, long long batch, long long batch_stride, uint32_t box_rows) {
  static_assert(sizeof(CUtensorMap) <= sizeof(TmCacheEntry::map), "descriptor size");
  if (cache) {
    for (int i = 0; i < cache->used; ++i) {
      const TmCacheEntry& c = cache->e[i];
      if (c.base == base && c.MN == MN && c.K == K && c.s_mn == s_mn && c.s_k == s_k && c.batch == batch &&
          c.batch_stride == batch_stride && c.esize == esize && c.mn_major == (int)mn_major && c.box_rows == box_rows) {
        memcpy(tm, c.map, sizeof(CUtensorMap));
        ++cache->hits;
        return true;
      }
    }
  }
  if (!encode_map(tm, base, esize, tf32, mn_major, MN, K, s_mn, s_k, batch, batch_stride, box_rows)) return false;
  if (cache) {
    int slot = cache->used < TmCache::SLOTS ? cache->used++ : (cache->next = (cache->next + 1) % TmCache::SLOTS);
    TmCacheEntry& c = cache->e[slot];
    c.base = base; c.MN = MN; c.K = K; c.s_mn = s_mn; c.s_k = s_k; c.batch = batch; c.batch_stride = batch_stride;
    c.esize = esize; c.mn_major = (int)mn_major; c.box_rows = box_rows;
    memcpy(c.map, tm, sizeof(CUtensorMap));
    ++cache->misses;
  }
  return true;
}

}  // namespace

bool gemm_tc_supported(const GemmDesc& g) {
  if (g.batch <= 0 || g.M <= 0 || g.N <= 0) return false;
  if (g.nseg < 1 || g.nseg > 2) return false;
  if (g.b_split == 2 && (g.nseg != 1 || !aligned16(g.B[1]))) return false;
  if (g.b_dtype != g.in_dtype) return false;
  const int esize = (int)dtype_size(g.in_dtype);
  if (g.symmetric && g.M != g.N) return false;
  if (g.transpose_out && (g.epilogue != EPI_STORE || g.symmetric)) return false;
  if (g.seg1_identity && (g.nseg != 2 || g.sa_k[0] != 1 || g.sb_k[0] != 1 || g.sa_k[1] != 1 || esize != 2 || g.b_split == 2)) return false;
  for (int s = 0; s < g.nseg; ++s) {
    if (s == 1 && g.seg1_identity) {
      if (!aligned16(g.A[1]) || !aligned16(g.B[1]) || (g.sa_i[1] * esize) % 16 || (g.batch > 1 && (g.batch_a[1] * esize) % 16)) return false;
      continue;
    }
    if (g.K[s] <= 0) return false;
    if (!aligned16(g.A[s]) || !aligned16(g.B[s])) return false;
    // one unit stride per operand, the other stride and the batch stride multiples of 16 bytes
    const long long a_other = (g.sa_k[s] == 1) ? g.sa_i[s] : g.sa_k[s];
    const long long b_other = (g.sb_k[s] == 1) ? g.sb_j[s] : g.sb_k[s];
    if (g.sa_k[s] != 1 && g.sa_i[s] != 1) return false;
    if (g.sb_k[s] != 1 && g.sb_j[s] != 1) return false;
    // tf32 operands are taken K-major only (an MN-major tf32 tile needs a different swizzle atom;
    // the symmetric fp32 products this engine serves never need it)
    if (esize == 4 && (g.sa_k[s] != 1 || g.sb_k[s] != 1)) return false;
    if ((a_other * esize) % 16 || (b_other * esize) % 16) return false;
    if (g.batch > 1 && ((g.batch_a[s] * esize) % 16 || (g.batch_b[s] * esize) % 16)) return false;
    // both segments must agree on the operand orientation (one instruction descriptor per launch)
    if (s > 0) {
      if ((g.sa_k[s] == 1) != (g.sa_k[0] == 1) || (g.sb_k[s] == 1) != (g.sb_k[0] == 1)) return false;
    }
  }
  return get_encode_fn() != nullptr;
}


TcKnobs tc_knobs_from_env() {
  TcKnobs k = kDefaultKnobs;
  auto geti = [](const char* name, int dflt) { const char* e = getenv(name); return e ? atoi(e) : dflt; };
  k.bn = geti("DEFL_TC_BN", 0); k.tile_m = geti("DEFL_TC_TILE_M", 0); k.stages = geti("DEFL_TC_STAGES", 0);
  k.ksub = geti("DEFL_TC_KSUB", 0); k.pair = geti("DEFL_TC_PAIR", -1); k.pair_min_n = geti("DEFL_TC_PAIR_MIN_N", 0);
  k.dynamic = getenv("DEFL_TC_DYNAMIC") ? 1 : 0; k.aux_prefetch = getenv("DEFL_TC_AUX_PREFETCH") ? 1 : 0;
  k.debug = getenv("DEFL_TC_DEBUG") ? 1 : 0; k.wait_ms = geti("DEFL_TC_WAIT_MS", 0);
  return k;
}

int gemm_tc_partials_per_batch(const GemmDesc& g, const TcKnobs* knobs) {
  const TcKnobs& kn = knobs ? *knobs : kDefaultKnobs;
  const int bn = choose_bn(g.N, choose_pair(g.M, g.N, kn), kn), tmh = choose_tile_m_impl(g.M, kn);
  return ((g.M + tmh - 1) / tmh) * ((g.N + bn - 1) / bn) * (tmh == 256 ? 2 : 1) * EPI_WARPS;
}

cudaError_t gemm_tc_launch(const GemmDesc& g, cudaStream_t st, int* status_word, int num_sms, long long* launches,
                           const TcKnobs* knobs, TmCache* cache) {
  if (!gemm_tc_supported(g)) return cudaErrorNotSupported;
  const TcKnobs& kn = knobs ? *knobs : kDefaultKnobs;
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.wait_ns = (unsigned long long)(kn.wait_ms > 0 ? kn.wait_ms : 2000) * 1000000ull;
  p.hold_stage = g.debug_hold_stage - 1;      // 0 in a zeroed descriptor = no hold
  const int esize = (int)dtype_size(g.in_dtype);
  const bool tf32 = (g.in_dtype == F32);
  p.esize = esize;
  p.M = g.M; p.N = g.N; p.batch = g.batch;
  p.tile_m = choose_tile_m_impl(g.M, kn);
  p.pair = choose_pair(g.M, g.N, kn) ? 1 : 0;
  p.BN = choose_bn(g.N, p.pair != 0, kn);
  p.tiles_m = (g.M + p.tile_m - 1) / p.tile_m;
  p.tiles_n = (g.N + p.BN - 1) / p.BN;
  p.tiles_per_matrix = p.tiles_m * p.tiles_n;
  if (g.symmetric) {
    p.tiles_per_matrix = 0;
    for (int tm = 0; tm < p.tiles_m; ++tm) {
      const int first = (tm * p.tile_m) / p.BN;
      if (first < p.tiles_n) p.tiles_per_matrix += p.tiles_n - first;
    }
  }
  p.total_tiles = (long long)p.tiles_per_matrix * g.batch;
  if (p.total_tiles >= (1ll << 31)) return cudaErrorNotSupported;      // the kernel's tile arithmetic is 32-bit
  p.nseg = g.nseg;
  OperandPlan pa, pb;
  // when a dimension has extent 1 both strides may look "unit"; prefer K-major
  // (per CTA: in pair mode each CTA stages 128 rows of A and half of the tile's B columns)
  if (!plan_operand(g.sa_i[0], g.sa_k[0], p.pair ? 128 : p.tile_m, esize, &pa)) return cudaErrorNotSupported;
  if (!plan_operand(g.sb_j[0], g.sb_k[0], p.pair ? p.BN / 2 : p.BN, esize, &pb)) return cudaErrorNotSupported;
  p.a_mn_major = pa.mn_major; p.b_mn_major = pb.mn_major;
  p.a_boxes = pa.boxes; p.a_box_bytes = pa.box_bytes; p.a_box_rows = pa.box_rows; p.a_stage_bytes = pa.stage_bytes;
  p.b_split = (g.b_split == 2) ? 2 : 1;
  p.b_boxes = pb.boxes; p.b_box_bytes = pb.box_bytes; p.b_box_rows = pb.box_rows;
  p.b_split_bytes = pb.stage_bytes; p.b_stage_bytes = pb.stage_bytes * p.b_split;
  const int span = KBYTES / esize;
  if (p.b_split == 2) {
    if (!cached_map(cache, &p.tmB[1], g.B[1], esize, tf32, pb.mn_major, g.N, g.K[0], g.sb_j[0], g.sb_k[0], g.batch,
                    g.batch_b[0], pb.box_rows))
      return cudaErrorInvalidValue;
  }
  // a pair's K block is half the work per CTA of the single-CTA form, too short to hide the per-step cost of the
  // two issuing threads (barrier wait, commit): its pipeline steps cover two K blocks when three such stages fit
  const uint32_t smem_budget = 224 * 1024 - EPI_WARPS * STAGING_BYTES;
  const uint32_t sub_bytes = p.a_stage_bytes + p.b_stage_bytes;
  p.ksub = (p.pair && 3u * 2u * sub_bytes <= smem_budget) ? 2 : 1;
  if ((kn.ksub == 1 || kn.ksub == 2) && (uint32_t)kn.ksub * sub_bytes * 2u <= smem_budget) p.ksub = kn.ksub;
  p.seg1_ident = (g.nseg == 2 && g.seg1_identity) ? 1 : 0;
  for (int s = 0; s < g.nseg; ++s) {
    if (s == 1 && p.seg1_ident) {
      // A[1] is [M, N] with K running over the output's columns (all of them: the copy engine zero-fills past N);
      // a tile walks its own BN columns; B[1] is one 256 x 256 identity, shared by all tiles and matrices
      p.kreal[s] = (p.BN + span - 1) / span;
      p.kblocks[s] = (p.kreal[s] + p.ksub - 1) / p.ksub;
      if (!cached_map(cache, &p.tmA[s], g.A[s], esize, tf32, false, g.M, g.N, g.sa_i[s], 1, g.batch, g.batch_a[s], pa.box_rows))
        return cudaErrorInvalidValue;
      if (!cached_map(cache, &p.tmB[s], g.B[s], esize, tf32, false, 256, 256, 256, 1, 1, 256 * 256, pb.box_rows))
        return cudaErrorInvalidValue;
      continue;
    }
    p.kreal[s] = (g.K[s] + span - 1) / span;
    p.kblocks[s] = (p.kreal[s] + p.ksub - 1) / p.ksub;
    if (!cached_map(cache, &p.tmA[s], g.A[s], esize, tf32, pa.mn_major, g.M, g.K[s], g.sa_i[s], g.sa_k[s], g.batch,
                    g.batch_a[s], pa.box_rows))
      return cudaErrorInvalidValue;
    if (!cached_map(cache, &p.tmB[s], g.B[s], esize, tf32, pb.mn_major, g.N, g.K[s], g.sb_j[s], g.sb_k[s], g.batch,
                    g.batch_b[s], pb.box_rows))
      return cudaErrorInvalidValue;
  }
  if ((uint32_t)p.ksub * (p.a_boxes + (uint32_t)p.b_split * p.b_boxes) > 32u) return cudaErrorNotSupported;   // one copy per producer lane
  const uint32_t stage_bytes = sub_bytes * (uint32_t)p.ksub;
  int stages = (int)(smem_budget / stage_bytes);
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (kn.stages >= 2 && kn.stages <= stages) stages = kn.stages;
  if (stages < 2) return cudaErrorNotSupported;
  p.stages = stages;
  // instruction descriptor: fp32 accumulate, operand format, majors, N >> 3 at bit 17, M >> 4 at bit 24
  const uint32_t fmt = tf32 ? 2u : (g.in_dtype == F16 ? 0u : 1u);      // kind::tf32: TF32 = 2; kind::f16: F16 = 0, BF16 = 1
  // (N is filled in per tile by the kernel: edge tiles compute fewer columns)
  p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)p.a_mn_major << 15) | ((uint32_t)p.b_mn_major << 16) |
            ((uint32_t)((p.pair ? 256 : 128) >> 4) << 24);
  p.epilogue = g.epilogue; p.out_dtype = g.out_dtype; p.aux_dtype = g.aux_dtype; p.symmetric = g.symmetric; p.round_tf32 = g.round_tf32;
  p.transposed = g.transpose_out ? 1 : 0;
  p.dup_ok = (p.pair && g.symmetric && p.BN == 256 && p.tile_m == 256 && g.nseg == 1 && p.b_split != 2 && g.A[0] == g.B[0] &&
              g.sa_i[0] == g.sb_j[0] && g.sa_k[0] == g.sb_k[0] && g.batch_a[0] == g.batch_b[0]) ? 1 : 0;
  p.diag_exact = !(g.nseg == 1 && g.b_split != 2 && g.A[0] == g.B[0] && g.sa_i[0] == g.sb_j[0] && g.sa_k[0] == g.sb_k[0] &&
                   g.batch_a[0] == g.batch_b[0]) ? 1 : 0;
  p.aux_f16 = (g.epilogue != EPI_STORE && g.aux_dtype == F16) ? 1 : 0;
  p.out_f16 = (g.out_dtype == F16) ? 1 : 0;
  p.C = g.C; p.ldc = g.ldc; p.batch_c = g.batch_c;
  p.aux = g.aux; p.ld_aux = g.ld_aux; p.batch_aux = g.batch_aux;
  p.alpha = g.alpha; p.aux_scale = g.aux_scale; p.pa = g.pa; p.pb = g.pb; p.pc = g.pc;
  p.alpha_dev = g.alpha_dev; p.aux_scale_dev = g.aux_scale_dev;
  p.partials = g.partials; p.partials_per_batch = g.partials_per_batch;
  p.aux_prefetch = 0;
  // (Off unless the aux_prefetch knob is set: with the epilogue's own fetch one block ahead the extra L2 prefetch
  // made the deflation passes 6 % slower and raised their DRAM reads to 1.6x the matrix, measured.)
  if (g.aux && g.epilogue != EPI_STORE && aligned16(g.aux) && kn.aux_prefetch) {
    const int aes = (int)dtype_size(g.aux_dtype);
    if ((g.ld_aux * aes) % 16 == 0 && (g.batch == 1 || (g.batch_aux * aes) % 16 == 0)) {
      EncodeTiledFn enc = get_encode_fn();
      cuuint64_t dims[3] = {(cuuint64_t)g.N, (cuuint64_t)g.M, (cuuint64_t)g.batch};
      cuuint64_t strides[2] = {(cuuint64_t)g.ld_aux * aes, (cuuint64_t)(g.batch == 1 ? g.ld_aux * (long long)g.M : g.batch_aux) * aes};
      // 16-bit types: a full 256-column tile per box; 32-bit types: box columns are capped at 256 elements too
      cuuint32_t box[3] = {(cuuint32_t)(p.BN < 256 ? p.BN : 256), (cuuint32_t)(p.pair ? 128 : p.tile_m), 1};
      cuuint32_t estr[3] = {1, 1, 1};
      const CUtensorMapDataType dt = (aes == 2) ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
      if (enc && enc(&p.tmAux, dt, 3, const_cast<void*>(g.aux), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
        p.aux_prefetch = 1;
    }
  }
  p.status = status_word;
  // The `dynamic` knob: tiles handed out through a counter instead of a fixed stride. The word after the status word
  // is this context's counter (zero between launches: the kernel that uses it puts it back; launches of one
  // context are ordered on its stream, so they never share it in time). Off by default: measured on the filter's
  // products it gains 2 % where tiles are long and uneven (the symmetric Gram product) and loses 2-3 % where they
  // are short (one more hand-off per tile), and the whole step comes out the same.
  p.tile_counter = (p.pair && status_word && kn.dynamic) ? reinterpret_cast<unsigned int*>(status_word + 1) : nullptr;

  const size_t smem = (size_t)stages * stage_bytes + 1024 + EPI_WARPS * STAGING_BYTES;
  cudaError_t e;
  if (p.pair) {
    auto kern = tf32 ? (p.b_split == 2 ? gemm_tc_kernel<1, 2, 1> : gemm_tc_kernel<1, 1, 1>)
                     : (p.b_split == 2 ? gemm_tc_kernel<0, 2, 1> : gemm_tc_kernel<0, 1, 1>);
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // how many CTA pairs the device can hold at once (a GPC with an odd number of free SMs leaves one out)
    static int max_pairs[4][64];   // per kernel variant and device; 0 = not asked yet
    int dev = 0;
    cudaGetDevice(&dev);
    const int variant = (tf32 ? 2 : 0) + (p.b_split == 2 ? 1 : 0);
    int pairs = (dev >= 0 && dev < 64) ? max_pairs[variant][dev] : 0;
    if (pairs <= 0) {
      cfg.gridDim = dim3((unsigned)(num_sms & ~1), 1, 1);
      int n = 0;
      e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
      if (e != cudaSuccess) return e;
      pairs = n > 0 ? n : 1;
      if (pairs > num_sms / 2) pairs = num_sms / 2;
      if (dev >= 0 && dev < 64) max_pairs[variant][dev] = pairs;
      if (kn.debug) fprintf(stderr, "gemm_tc: %d CTA pairs resident (occupancy query %d), %d stages\n", pairs, n, stages);
    }
    long long npairs = p.total_tiles < pairs ? p.total_tiles : pairs;
    if (npairs < 1) npairs = 1;
    cfg.gridDim = dim3((unsigned)(2 * npairs), 1, 1);
    e = cudaLaunchKernelEx(&cfg, kern, p);
    if (launches) ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  auto kern = tf32 ? (p.b_split == 2 ? gemm_tc_kernel<1, 2, 0> : gemm_tc_kernel<1, 1, 0>)
                   : (p.b_split == 2 ? gemm_tc_kernel<0, 2, 0> : gemm_tc_kernel<0, 1, 0>);
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  long long grid = p.total_tiles < num_sms ? p.total_tiles : num_sms;
  if (grid < 1) grid = 1;
  kern<<<(unsigned)grid, NUM_THREADS, smem, st>>>(p);
  if (launches) ++*launches;
  return cudaGetLastError();
}

}  // namespace defl
