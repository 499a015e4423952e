// tcgen05 tensor-core contraction for sm_100a with the fused epilogues of
// Algorithm 1:  acc(i,j) = sum_k A(i,k) B(j,k), bf16 operands, fp32 accumulators
// in tensor memory.
//
// With CTAS == 2 (the default) two CTAs on neighbouring SMs form a cluster and share one
// 256x256 tile: each loads its own 128 rows of A and its own 128 columns of B, the leader issues
// tcgen05.mma.cta_group::2 for both, each keeps the accumulator of its 128 rows in its own tensor
// memory and runs its own epilogue.  B then crosses L2 -> shared memory once per pair instead of
// once per CTA, and the freed shared memory deepens the ring to six stages.
// The dW contraction (template parameter MT = 2) instead puts both accumulators on one 512x256
// tile: two 128-row sub-tiles of A per CTA and stage, four 48 KB stages, epilogue after the tile.
// Tiles are handed out in bands of row tiles (decode_unit) so that the CTA pairs running at the
// same time share operand panels in L2; a contraction with few output tiles can be cut along k
// (EPI_ACCUM_F32, one accumulator slab per range).
//
// One persistent CTA per SM, 192 or 320 threads in three roles:
//   warp 0      TMA producer: 128-byte-swizzled operand tiles into a 5- or 6-stage ring
//   warp 1      MMA issuer (in the pair's leader): tcgen05.mma 256x256x16 from shared-memory
//               descriptors into one of two 256-column accumulators in tensor memory
//   warps 2..   epilogue, 4 or 8 warps (template parameter EW): tcgen05.ld (one accumulator
//               row per thread; with 8 warps two share a tensor-memory lane quarter and take
//               128 columns each), the fused arithmetic, stores (staged through shared
//               memory and written by TMA for dlogits, dX, dW); runs while the next tile's
//               MMAs issue
// Operands may be K-major (k contiguous) or MN-major (the transposed storage),
// chosen at run time through the descriptors, so that dX += dZ W and
// dW = dZ^T X need no transposed copies.
//
// Every mbarrier wait is bounded: after about two seconds a wait stores a code
// in the caller's status word, raises a CTA-wide abort flag and every role
// leaves its loop; the CTA then waits (bounded, whatever the abort flag says)
// for the copies and MMAs it has issued, lingers a millisecond for what its
// peer may still have in flight, frees its tensor memory and returns.
#include "pctc_internal.h"

#include <cuda.h>

#include <atomic>
#include <math_constants.h>

namespace pctc {

namespace {

// Tunables (overridable at compile time for experiments)
#ifndef PCTC_TUNE_RASTER_G
#define PCTC_TUNE_RASTER_G 8      // row tiles per band of the tile order (kernels with one tile per unit)
#endif
#ifndef PCTC_TUNE_WALK_MB
#define PCTC_TUNE_WALK_MB 32      // MB of A rows that a band of the column-walking kernels keeps hot in L2
#endif

#ifndef PCTC_TUNE_L2_PROMOTION
#define PCTC_TUNE_L2_PROMOTION CU_TENSOR_MAP_L2_PROMOTION_L2_256B   // L2 fetch granularity of the TMA loads
#endif

#ifndef PCTC_TUNE_MT2
#define PCTC_TUNE_MT2 1           // 1: the dW contraction may use 512 x 256 tiles (see k_umma_gemm, MT)
#endif

#ifndef PCTC_TUNE_CTAS
#define PCTC_TUNE_CTAS 2          // CTAs per tile: 2 = tcgen05 cta_group::2 pairs, 1 = independent CTAs
#endif

// Measurement probes (never set in the regular build; results are then wrong on purpose).  They knock
// out one part of the kernel at a time to show what a launch is bound by:
//   bit 0  the LSE and dlogits epilogues do not read tensor memory (they work on constants)
//   bit 1  ... do no arithmetic (no exponentials, no maxima)
//   bit 2  the dlogits epilogue does not stage or store the chunk
//   bit 3  the column-walking kernels load their A rows only for the first tile of a unit
#ifndef PCTC_PROBE
#define PCTC_PROBE 0
#endif
constexpr bool PROBE_NO_TMEM_LD = (PCTC_PROBE & 1) != 0;
constexpr bool PROBE_NO_MATH = (PCTC_PROBE & 2) != 0;
constexpr bool PROBE_NO_STORE = (PCTC_PROBE & 4) != 0;
constexpr bool PROBE_SKIP_A = (PCTC_PROBE & 8) != 0;

#ifndef PCTC_TUNE_CHUNK_HINT
#define PCTC_TUNE_CHUNK_HINT 0    // L2 eviction priority for the bf16 dlogits chunk: bit 0 evict-first on its stores
#endif                            // (dlogits), bit 1 evict-first on its loads (A operand of the dX and dW kernels)

#ifndef PCTC_TUNE_WALK_HINT
#define PCTC_TUNE_WALK_HINT 0     // column-walking kernels (LSE, arg-max): bit 0 evict-last on the A rows (re-read for
#endif                            // every column tile), bit 1 evict-first on the B panels (each used once per band)

#ifndef PCTC_TUNE_PDL
#define PCTC_TUNE_PDL 0           // 1: programmatic dependent launch: a contraction kernel's CTAs may start and set up
#endif                            // (barriers, tensor memory) while the kernel before it in the stream drains

#ifndef PCTC_TUNE_EPI_WARPS
#define PCTC_TUNE_EPI_WARPS 0     // 0: by the contraction depth; 4 or 8: forced
#endif

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int MAX_STAGES = 6;
// Epilogue warps per CTA (template parameter EW): 4 = one per tensor-memory lane quarter, 256
// columns each; 8 = two per quarter, 128 columns each.  Eight hide the latency of a math-heavy
// epilogue when the main loop of a tile is short (narrow heads); four leave the ring one stage
// deeper and the SM cooler when the main loop is long.
constexpr int warp_cols(int ew) { return BN / (ew / 4); }   // accumulator columns per epilogue warp
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int b_stage_bytes(int ctas) { return (BN / ctas) * BK * 2; }   // each CTA of a pair holds half of B
constexpr int num_threads(int ew) { return 64 + ew * 32; }
constexpr int TMEM_COLS = 512;
constexpr int MN_GROUP_BYTES = 64 * BK * 2;          // one 64-wide MN group of an MN-major tile
#ifndef PCTC_WAIT_LIMIT_CYCLES
#define PCTC_WAIT_LIMIT_CYCLES 4000000000LL   // about two seconds; a test build shortens it so that a wait runs out
#endif
#ifndef PCTC_WAIT_POLL_MASK
#define PCTC_WAIT_POLL_MASK 255u              // the clock and the abort flag are looked at every 256th poll
#endif
constexpr long long WAIT_LIMIT_CYCLES = PCTC_WAIT_LIMIT_CYCLES;
constexpr long long DRAIN_LIMIT_CYCLES = 200000000LL;   // the waits of an aborting CTA for its own copies and MMAs
constexpr long long ABORT_LINGER_CYCLES = 2000000LL;    // an aborting CTA stays this long before it leaves (see the kernel's end)
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

struct UmmaArgs {
  int m, n, k;
  int a_mn, b_mn;
  int nsplit;          // EPI_LSE_PARTIAL: column splits per row tile
  int raster_g;        // tile order: row tiles per band (see decode_unit)
  int tile_mt;         // host only: 2 = launch the 512-row tile form (store epilogue, long contractions)
  int ksplit;          // EPI_ACCUM_F32: units per output tile, each contracting its own range of k
  int ksplit_rows;     //   ... and writing its own accumulator slab, this many rows further down
  int* status;
  Epilogue e;
};

struct SharedTail {   // barriers and flags
  unsigned long long full[MAX_STAGES];
  unsigned long long empty[MAX_STAGES];
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
  unsigned long long done;
  unsigned tmem_base;
  int abort;
};

// Dynamic shared memory after the operand ring, by epilogue kind:
//   store staging  8 warps x 2 buffers of 32 rows x 64 B (32 bf16 or 16 fp32 columns), 64-byte
//                  swizzle, written out by TMA stores while the other buffer fills
//   SharedTail
//   bias           8 warps x 128 floats (lse, subset, dlogits)
//   list           8 warps x (128 indices in U, -1 if the column's class is not selected, + group masks) (dlogits)
constexpr int STAGE_BOX_BYTES = 2048;                      // one staged box: 32 rows x 64 B
constexpr int STAGE_WARP_BYTES = 2 * STAGE_BOX_BYTES;      // double-buffered
constexpr bool epi_uses_tma_store(int epi) {
  return epi == EPI_DLOGITS || epi == EPI_ACCUM_F32 || epi == EPI_STORE_OUT || epi == EPI_SUBSET_LOGP;
}
constexpr bool epi_fp32_boxes(int epi) { return epi == EPI_ACCUM_F32 || epi == EPI_SUBSET_LOGP; }
constexpr bool epi_uses_bias(int epi) {
  return epi == EPI_LSE_PARTIAL || epi == EPI_SUBSET_LOGP || epi == EPI_DLOGITS || epi == EPI_ARGMAX_PARTIAL;
}
constexpr bool epi_walks_splits(int epi) { return epi == EPI_LSE_PARTIAL || epi == EPI_ARGMAX_PARTIAL; }
// ring depth: what is left of the 227 KB after the epilogue's own buffers
// (mt = 2: two 128-row sub-tiles of A per CTA and stage, both accumulators on one tile: 48 KB stages, four of them)
constexpr int stages_of(int ctas, int epi, int ew, int mt = 1) {
  return mt == 2 ? 4
                 : (ctas == 2 ? ((epi_uses_tma_store(epi) && ew == 8) ? 5 : 6) : (epi_uses_tma_store(epi) ? 3 : 4));
}
constexpr size_t ring_bytes(int ctas, int epi, int ew, int mt = 1) {
  return (size_t)stages_of(ctas, epi, ew, mt) * (mt * A_STAGE_BYTES + b_stage_bytes(ctas));
}
constexpr size_t off_stage(int ctas, int epi, int ew, int mt = 1) { return ring_bytes(ctas, epi, ew, mt); }
constexpr size_t off_tail(int ctas, int epi, int ew, int mt = 1) {
  return ring_bytes(ctas, epi, ew, mt) + (epi_uses_tma_store(epi) ? ew * STAGE_WARP_BYTES : 0);
}
constexpr size_t off_bias(int ctas, int epi, int ew, int mt = 1) { return off_tail(ctas, epi, ew, mt) + 256; }
constexpr size_t off_list(int ctas, int epi, int ew, int mt = 1) {
  return off_bias(ctas, epi, ew, mt) + (epi_uses_bias(epi) ? ew * warp_cols(ew) * 4 : 0);
}
constexpr int list_words(int ew) { return warp_cols(ew) + 32; }
constexpr size_t smem_bytes(int ctas, int epi, int ew, int mt = 1) {
  return 1024 + off_list(ctas, epi, ew, mt) + (epi == EPI_DLOGITS ? ew * list_words(ew) * 4 : 0);
}
static_assert(sizeof(SharedTail) <= 256, "tail layout");

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting or the limit ran out (then it raises the abort).
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, volatile int* abort_flag,
                                          int* status, int code, long long limit = WAIT_LIMIT_CYCLES) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (unsigned it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & PCTC_WAIT_POLL_MASK) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) {
        *abort_flag = 1;
        if (status) atomicCAS(status, 0, code);
        return false;
      }
    }
  }
}
// The waits of the drain: for copies and MMAs this CTA has already issued.  They run when the CTA is
// aborting too, so they ignore the abort flag and keep only their own limit.
__device__ __forceinline__ bool mbar_wait_drain(unsigned long long* bar, unsigned parity) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (unsigned it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 255u) == 0u && clock64() - t0 > DRAIN_LIMIT_CYCLES) return false;
  }
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int c0, int c1,
                                            unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
      : "memory");
}

// Store (or fp32 add-reduce) of one staged box; the tensor map clips rows and columns past the extents.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(smem_u32(smem_src))
               : "memory");
}
// The same copies with an L2 eviction-priority hint (a policy word from make_evict_first_policy).
__device__ __forceinline__ unsigned long long make_evict_first_policy() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ unsigned long long make_evict_last_policy() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* map, const void* smem_src, int c0, int c1,
                                                  unsigned long long policy) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%1, %2}], [%3], %4;"
               ::"l"(map), "r"(c0), "r"(c1), "r"(smem_u32(smem_src)), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, const void* smem_src, int c0, int c1) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(smem_u32(smem_src))
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// --- two-CTA (cluster) forms ---
constexpr unsigned PEER_MASK = 0xFEFFFFFFu;   // shared::cluster address of the same offset in the pair's CTA 0
__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load issued by either CTA of a pair into its own shared memory; the bytes are counted on the
// leader's barrier (no multicast: every CTA fetches its own box).
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, int c0, int c1,
                                                 unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar) & PEER_MASK)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair_hint(void* smem_dst, const CUtensorMap* map, int c0, int c1,
                                                      unsigned long long* bar, unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar) & PEER_MASK), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_leader(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(smem_u32(bar) & PEER_MASK) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(unsigned long long* bar) {       // arrives in both CTAs
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((unsigned short)3)
               : "memory");
}
__device__ __forceinline__ void tc_commit_pair_local(unsigned long long* bar) { // arrives in the issuing CTA only
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(unsigned tmem_d, unsigned long long adesc, unsigned long long bdesc,
                                                 unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ void tc_mma_bf16(unsigned tmem_d, unsigned long long adesc, unsigned long long bdesc,
                                            unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread `lane` of the warp receives its row.
__device__ __forceinline__ void tmem_ld32(unsigned taddr, float* v) {
  unsigned r[32];
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
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// Two fp32 FMAs in one instruction (sm_100 packed fp32): d = a * b + c on both halves.
__device__ __forceinline__ void ffma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void fadd2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
// max of three (one instruction on sm_100)
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ void fmul2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
// v[0..31] += b[0..31]: the staged bias of a column group, read as eight 16-byte words
__device__ __forceinline__ void add_bias32(float (&v)[32], const float* b) {
#pragma unroll
  for (int c = 0; c < 32; c += 4) {
    const float4 bb = *reinterpret_cast<const float4*>(b + c);
    v[c] += bb.x; v[c + 1] += bb.y; v[c + 2] += bb.z; v[c + 3] += bb.w;
  }
}
__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor of a 128-byte-swizzled bf16 tile.
//   K-major : rows of 64 k (128 bytes); 8-row groups 1024 bytes apart (stride byte offset).
//   MN-major: rows of 64 m/n (128 bytes), one row per k; 8-k groups 1024 bytes apart (stride byte
//             offset); 64-wide m/n groups MN_GROUP_BYTES apart (leading byte offset).
__device__ __forceinline__ unsigned long long make_smem_desc(unsigned addr, bool mn_major) {
  unsigned long long d = 0;
  d |= (unsigned long long)((addr & 0x3FFFFu) >> 4);
  d |= (unsigned long long)(mn_major ? (MN_GROUP_BYTES >> 4) : 1) << 16;
  d |= (unsigned long long)(1024 >> 4) << 32;
  d |= 1ull << 46;     // descriptor version of sm_100
  d |= 2ull << 61;     // 128-byte swizzle
  return d;
}

// x / d for 0 <= x < 2^22, 1 <= d: a float quotient and one correction step instead of the long
// integer-division sequence (the tile decode runs in every warp for every tile).
__device__ __forceinline__ int fast_div(int x, int d, int& rem) {
  int q = __float2int_rz(__fdividef((float)x, (float)d));
  int r = x - q * d;
  if (r < 0) { --q; r += d; }
  else if (r >= d) { ++q; r -= d; }
  rem = r;
  return q;
}

__device__ __forceinline__ void split_range(int n_tiles, int splits, int sp, int& start, int& cnt) {
  int rem;
  const int base = fast_div(n_tiles, splits, rem);
  cnt = base + (sp < rem ? 1 : 0);
  start = sp * base + min(sp, rem);
}

// Unit u -> (row tile, first column tile, number of column tiles).  The order decides what the
// CTA groups that run at the same time have in common, i.e. what L2 serves more than once per DRAM
// read.  Row tiles are taken in bands of g: inside a band the row tile runs fastest, then the
// column split, so a wave of W groups covers g row tiles x W/g column splits and touches
// g A-panels + W/g B-panels instead of all A-panels (g = m_tiles) or all B-panels (g = 1).
// Odd bands walk the splits backwards, so a band starts on the B-panels the previous one ended on.
__device__ __forceinline__ void decode_unit(int u, int m_tiles, int n_tiles, int splits, int ksplit, int g,
                                            int& mt, int& sp, int& ks, int& nt0, int& cnt) {
  const int cols = splits * ksplit;              // a column split may itself be cut along k
  int r, row;
  const int band = fast_div(u, g * cols, r);
  const int rows = min(g, m_tiles - band * g);
  int c = fast_div(r, rows, row);
  mt = band * g + row;
  if (band & 1) c = cols - 1 - c;
  if (ksplit == 1) { sp = c; ks = 0; }
  else sp = fast_div(c, ksplit, ks);
  if (splits == n_tiles) { nt0 = sp; cnt = 1; }  // one tile per unit
  else split_range(n_tiles, splits, sp, nt0, cnt);
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
// MT = 2 (store epilogues only, two-CTA form): a tile is 512 x 256; every CTA stages two 128-row
// sub-tiles of A per k-block next to its half of B, the two accumulators hold the two sub-tiles of ONE
// tile (25% fewer operand bytes per FLOP than two 256 x 256 tiles), and the epilogue is not
// overlapped with the next tile's MMAs.
template <int EPI, int CTAS, int EW, int MT = 1>
__global__ void __launch_bounds__(num_threads(EW), 1)
k_umma_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, UmmaArgs a) {
  static_assert(MT == 1 || (MT == 2 && CTAS == 2 && (EPI == EPI_STORE_OUT || EPI == EPI_ACCUM_F32)), "tile height");
  constexpr int STAGES = stages_of(CTAS, EPI, EW, MT);
  constexpr int B_STAGE_BYTES = b_stage_bytes(CTAS);
  constexpr int A_STAGE = MT * A_STAGE_BYTES;  // this CTA's rows of A per stage
  constexpr int WARP_COLS = warp_cols(EW);
  constexpr int LIST_WORDS = list_words(EW);
  constexpr int SUB_M = BM * CTAS;             // rows one MMA covers
  constexpr int TILE_M = SUB_M * MT;           // rows of the tile a CTA (pair) works on
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((size_t)smem_raw + 1023) & ~(size_t)1023);
  unsigned char* sA = smem;
  unsigned char* sB = smem + (size_t)STAGES * A_STAGE;
  SharedTail* st = (SharedTail*)(smem + off_tail(CTAS, EPI, EW, MT));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (CTAS == 2) ? (int)cluster_ctarank() : 0;     // position inside the pair
  const int group = blockIdx.x / CTAS, ngroups = gridDim.x / CTAS;

  // With programmatic dependent launch this CTA may be running before the kernel ahead of it in the
  // stream has finished: nothing that kernel wrote may be read, and nothing it reads may be overwritten,
  // before griddepcontrol.wait.  The set-up below touches shared and tensor memory only, except for the
  // selected-class count, which the kernel ahead may still be writing.
  if (PCTC_TUNE_PDL && EPI == EPI_SUBSET_LOGP) asm volatile("griddepcontrol.wait;" ::: "memory");
  // problem decomposition, identical in every role
  int n_eff = a.n;
  if (EPI == EPI_SUBSET_LOGP) n_eff = min(a.n, *a.e.Kdev);
  const int m_tiles = (a.m + TILE_M - 1) / TILE_M;
  const int n_tiles = (n_eff + BN - 1) / BN;
  const int splits = epi_walks_splits(EPI) ? a.nsplit : n_tiles;
  const int ksplit = (EPI == EPI_ACCUM_F32) ? a.ksplit : 1;
  const int units = m_tiles * splits * ksplit;
  const int k_blocks = (a.k + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&st->full[s], 1); mbar_init(&st->empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&st->tmem_full[s], 1); mbar_init(&st->tmem_empty[s], EW * CTAS); }
    mbar_init(&st->done, 1);
    st->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (CTAS == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&st->tmem_base)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&st->tmem_base)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();     // the peer's barriers exist before anything signals them
  tc_fence_after();
  const unsigned tmem_base = st->tmem_base;
  volatile int* abort_flag = &st->abort;
  if (PCTC_TUNE_PDL) {
    asm volatile("griddepcontrol.wait;" ::: "memory");                 // the kernels ahead are complete and visible
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");    // the next one may set up as SMs free up
  }

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      unsigned g = 0;
      bool ok = true;
      auto load = [&](void* dst, const CUtensorMap* map, int c0, int c1, unsigned long long* bar) {
        if (CTAS == 2) tma_load_2d_pair(dst, map, c0, c1, bar);
        else tma_load_2d(dst, map, c0, c1, bar);
      };
      // the A operand of the dX and dW contractions is the dlogits chunk
      constexpr bool WALK_A = (PCTC_TUNE_WALK_HINT & 1) && CTAS == 2 && epi_walks_splits(EPI);
      constexpr bool WALK_B = (PCTC_TUNE_WALK_HINT & 2) && CTAS == 2 && epi_walks_splits(EPI);
      constexpr bool HINT_A = ((PCTC_TUNE_CHUNK_HINT & 2) && CTAS == 2 && (EPI == EPI_ACCUM_F32 || EPI == EPI_STORE_OUT)) || WALK_A;
      const unsigned long long a_policy = WALK_A ? make_evict_last_policy() : (HINT_A ? make_evict_first_policy() : 0ull);
      const unsigned long long b_policy = WALK_B ? make_evict_first_policy() : 0ull;
      auto load_a = [&](void* dst, const CUtensorMap* map, int c0, int c1, unsigned long long* bar) {
        if (HINT_A) tma_load_2d_pair_hint(dst, map, c0, c1, bar, a_policy);
        else load(dst, map, c0, c1, bar);
      };
      auto load_b = [&](void* dst, const CUtensorMap* map, int c0, int c1, unsigned long long* bar) {
        if (WALK_B) tma_load_2d_pair_hint(dst, map, c0, c1, bar, b_policy);
        else load(dst, map, c0, c1, bar);
      };
      for (int u = group; u < units && ok; u += ngroups) {
        int mt, sp, ks, nt0, cnt, kb0, kcnt;
        decode_unit(u, m_tiles, n_tiles, splits, ksplit, a.raster_g, mt, sp, ks, nt0, cnt);
        split_range(k_blocks, ksplit, ks, kb0, kcnt);            // this unit's share of the contraction
        const int row_a = mt * TILE_M + rank * BM;               // this CTA's rows of A
        for (int nt = nt0; nt < nt0 + cnt && ok; ++nt) {
          const int row_b = nt * BN + rank * (BN / CTAS);        // this CTA's columns of the tile (rows of B)
          for (int kb = kb0; kb < kb0 + kcnt; ++kb, ++g) {
            const int s = g % STAGES;
            const unsigned ph = (g / STAGES) & 1u;
            if (!mbar_wait(&st->empty[s], ph ^ 1u, abort_flag, a.status, 1)) { ok = false; break; }
            // the leader's barrier counts the bytes of both CTAs
            const bool skip_a = PROBE_SKIP_A && epi_walks_splits(EPI) && nt != nt0;
            if (rank == 0) mbar_expect_tx(&st->full[s], CTAS * ((skip_a ? 0 : A_STAGE) + B_STAGE_BYTES));
            unsigned char* dA = sA + (size_t)s * A_STAGE;
            unsigned char* dB = sB + (size_t)s * B_STAGE_BYTES;
#pragma unroll
            for (int h = 0; h < MT; ++h) {               // sub-tile h: this CTA's 128 rows of pair rows h*256..
              if (skip_a) break;
              unsigned char* dAh = dA + h * A_STAGE_BYTES;
              const int row_ah = row_a + h * SUB_M;
              if (!a.a_mn) {
                load_a(dAh, &tmA, kb * BK, row_ah, &st->full[s]);
              } else {
#pragma unroll
                for (int q = 0; q < BM / 64; ++q)
                  load_a(dAh + q * MN_GROUP_BYTES, &tmA, row_ah + q * 64, kb * BK, &st->full[s]);
              }
            }
            if (!a.b_mn) {
              load_b(dB, &tmB, kb * BK, row_b, &st->full[s]);
            } else {
#pragma unroll
              for (int q = 0; q < BN / CTAS / 64; ++q)
                load_b(dB + q * MN_GROUP_BYTES, &tmB, row_b + q * 64, kb * BK, &st->full[s]);
            }
          }
        }
      }
      // drain: every copy issued has landed before the CTA may exit.  The leader's barriers count
      // the peer's bytes too; the peer itself stays alive until the closing cluster barrier.
      if (rank == 0) {
        const unsigned issued = g;
        for (unsigned j = (issued > STAGES ? issued - STAGES : 0); j < issued; ++j)
          mbar_wait_drain(&st->full[j % STAGES], (j / STAGES) & 1u);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0 && rank == 0) {        // the leader issues the MMAs of the pair
      const unsigned idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(a.a_mn ? 1 : 0) << 15) |
                             ((unsigned)(a.b_mn ? 1 : 0) << 16) | ((unsigned)(BN >> 3) << 17) |
                             ((unsigned)(SUB_M >> 4) << 24);
      const unsigned a_step = a.a_mn ? (2048u >> 4) : (32u >> 4);   // descriptor advance per 16 k
      const unsigned b_step = a.b_mn ? (2048u >> 4) : (32u >> 4);
      unsigned g = 0, it = 0;
      bool ok = true;
      for (int u = group; u < units && ok; u += ngroups) {
        int mt, sp, ks, nt0, cnt, kb0, kcnt;
        decode_unit(u, m_tiles, n_tiles, splits, ksplit, a.raster_g, mt, sp, ks, nt0, cnt);
        split_range(k_blocks, ksplit, ks, kb0, kcnt);
        (void)mt;
        for (int nt = nt0; nt < nt0 + cnt && ok; ++nt, ++it) {
          // MT == 1: the two accumulators alternate between tiles.  MT == 2: both belong to this tile
          // (sub-tile h in accumulator h), so both must have been drained, and each is used once per tile.
          const unsigned acc = (MT == 2) ? 0u : (it & 1u), aph = (MT == 2) ? (it & 1u) : ((it >> 1) & 1u);
          if (!mbar_wait(&st->tmem_empty[acc], aph ^ 1u, abort_flag, a.status, 2)) { ok = false; break; }
          if (MT == 2 && !mbar_wait(&st->tmem_empty[1], aph ^ 1u, abort_flag, a.status, 2)) { ok = false; break; }
          tc_fence_after();
          const unsigned d_tmem = tmem_base + acc * BN;
          for (int kb = kb0; kb < kb0 + kcnt; ++kb, ++g) {
            const int s = g % STAGES;
            const unsigned ph = (g / STAGES) & 1u;
            if (!mbar_wait(&st->full[s], ph, abort_flag, a.status, 3)) { ok = false; break; }
            tc_fence_after();
            const unsigned long long adesc = make_smem_desc(smem_u32(sA + (size_t)s * A_STAGE), a.a_mn);
            const unsigned long long bdesc = make_smem_desc(smem_u32(sB + (size_t)s * B_STAGE_BYTES), a.b_mn);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
              const unsigned long long bd = bdesc + (unsigned long long)(kk * b_step);
#pragma unroll
              for (int h = 0; h < MT; ++h) {
                const unsigned long long ad =
                    adesc + (unsigned long long)(kk * a_step) + (unsigned long long)(h * (A_STAGE_BYTES >> 4));
                if (CTAS == 2) tc_mma_bf16_pair(d_tmem + h * BN, ad, bd, idesc, (kb != kb0 || kk != 0) ? 1u : 0u);
                else tc_mma_bf16(d_tmem + h * BN, ad, bd, idesc, (kb != kb0 || kk != 0) ? 1u : 0u);
              }
            }
            // frees the stage (in both CTAs) once these MMAs have read it
            if (CTAS == 2) tc_commit_pair(&st->empty[s]); else tc_commit(&st->empty[s]);
          }
          if (ok) {
            if (CTAS == 2) tc_commit_pair(&st->tmem_full[acc]); else tc_commit(&st->tmem_full[acc]);
            if (MT == 2) tc_commit_pair(&st->tmem_full[1]);
          }
        }
      }
      // all MMAs issued by this thread have completed before tensor memory is freed
      if (CTAS == 2) tc_commit_pair_local(&st->done); else tc_commit(&st->done);
      mbar_wait_drain(&st->done, 0);
    }
  } else {
    // ===================== epilogue warps =====================
    const int ew = warp - 2;                 // private staging slot, 0..EW-1
    const int q = warp & 3;                  // tensor-memory lane quarter this warp may read
    const int r = q * 32 + lane;             // accumulator row of this thread
    const int c_base = (ew >> 2) * WARP_COLS;   // this warp's columns of the tile: [c_base, c_base + WARP_COLS)
    float* sb = (float*)(smem + off_bias(CTAS, EPI, EW, MT)) + ew * WARP_COLS;     // bias of the warp's columns
    int* sj = (int*)(smem + off_list(CTAS, EPI, EW, MT)) + ew * LIST_WORDS;         // index in U of each of them, or -1
    unsigned* sg = (unsigned*)sj + WARP_COLS;                              // one mask of selected columns per 32
    unsigned char* stage = smem + off_stage(CTAS, EPI, EW, MT) + ew * STAGE_WARP_BYTES;   // this warp's two staging boxes
    const unsigned swz64 = (unsigned)((lane >> 1) & 3); // 64-byte swizzle of a staged 64-byte row
    unsigned nbox = 0;                                  // boxes stored so far by this warp (buffer parity)
    const int pstride = a.e.partial_stride ? a.e.partial_stride : a.nsplit;   // split slots per row
    unsigned it = 0;
    bool ok = true;
    // EPI_DLOGITS: the per-row and per-column inputs of a tile (lambda, row weight, class map) are
    // fetched one unit ahead, so their latency is spent under the previous tile's epilogue
    constexpr int NGRP = WARP_COLS / 32;
    float pre_lam = 0.f, pre_w = 0.f;
    int pre_jj[NGRP];
    auto prefetch = [&](int u2) {
      int mt2, sp2, ks2, nt2, cnt2;
      decode_unit(u2, m_tiles, n_tiles, splits, ksplit, a.raster_g, mt2, sp2, ks2, nt2, cnt2);
      const int i2 = mt2 * TILE_M + rank * BM + r;
      pre_lam = 0.f; pre_w = 0.f;
      if (i2 < a.m) { pre_lam = a.e.lambda[i2]; pre_w = a.e.roww[i2]; }
#pragma unroll
      for (int gq = 0; gq < NGRP; ++gq) {
        const int j = nt2 * BN + c_base + gq * 32 + lane;
        int jj = (j < n_eff) ? a.e.vmap[a.e.v0 + j] : -1;
        if (!index_ok(jj, -1, a.e.ld_gamma, a.status, 9)) jj = -1;      // the class map indexes a row of gamma
        pre_jj[gq] = jj;
      }
    };
    if (EPI == EPI_DLOGITS && group < units) prefetch(group);
    for (int u = group; u < units && ok; u += ngroups) {
      int mt, sp, ks, nt0, cnt;
      decode_unit(u, m_tiles, n_tiles, splits, ksplit, a.raster_g, mt, sp, ks, nt0, cnt);
      const int row0_cta = mt * TILE_M + rank * BM;      // first row of this CTA's half of the tile
      const int row0_out = row0_cta + ks * a.ksplit_rows; // ... and where it lands in the output (k-split slab)
      const int i = row0_cta + r;
      const bool row_ok = i < a.m;
      float lam2 = 0.f, lam = 0.f, w = 0.f;
      if (EPI == EPI_SUBSET_LOGP && a.e.lambda && row_ok) lam = a.e.lambda[i];
      int cur_jj[NGRP];
      if (EPI == EPI_DLOGITS) {
        lam = pre_lam; w = pre_w; lam2 = lam * LOG2E;
#pragma unroll
        for (int gq = 0; gq < NGRP; ++gq) cur_jj[gq] = pre_jj[gq];
        if (u + ngroups < units) prefetch(u + ngroups);
      }
      // a positive row weight goes into the exponent; any other (zero, negative) is multiplied in afterwards
      const float wmul = (w > 0.f) ? 1.f : w;
      const float off2 = (w > 0.f) ? lg2(w) - lam2 : -lam2;
      float run_max2 = -CUDART_INF_F, run_sum = 0.f;     // EPI_LSE_PARTIAL, base-2 domain
      float best_z = -CUDART_INF_F;                      // EPI_ARGMAX_PARTIAL
      int best_j = -1;

      for (int nt = nt0; nt < nt0 + cnt && ok; ++nt, ++it) {
        const int n0 = nt * BN;
        // ---- warp-private staging of per-column data (overlaps the MMAs of this tile) ----
        const bool has_bias = a.e.bias != nullptr;        // without a bias the staged zeros are never read
        if (epi_uses_bias(EPI) && has_bias) {
          const __nv_bfloat16* bias = (const __nv_bfloat16*)a.e.bias;
#pragma unroll
          for (int c = lane; c < WARP_COLS; c += 32) {
            const int j = n0 + c_base + c;
            float b = 0.f;
            if (bias && j < n_eff) {
              if (EPI == EPI_SUBSET_LOGP) {
                const int cls = a.e.U[j];
                if (index_ok(cls, 0, a.e.vocab, a.status, 10)) b = __bfloat162float(bias[cls]);
              }
              else b = __bfloat162float(bias[a.e.v0 + j]);
            }
            sb[c] = b;
          }
        }
        if (EPI == EPI_DLOGITS) {                       // one tile per unit: the prefetched class map is this tile's
#pragma unroll
          for (int gq = 0; gq < NGRP; ++gq) {
            const int jj = cur_jj[gq];
            const unsigned mask = __ballot_sync(0xffffffffu, jj >= 0);
            sj[gq * 32 + lane] = jj;
            if (lane == 0) sg[gq] = mask;
          }
        }
        __syncwarp();

#pragma unroll 1
        for (int h = 0; h < MT && ok; ++h) {       // MT == 2: sub-tile h of this tile sits in accumulator h
        const unsigned acc = (MT == 2) ? (unsigned)h : (it & 1u), aph = (MT == 2) ? (it & 1u) : ((it >> 1) & 1u);
        int got = 0;
        if (lane == 0) got = mbar_wait(&st->tmem_full[acc], aph, abort_flag, a.status, 4) ? 1 : 0;
        got = __shfl_sync(0xffffffffu, got, 0);
        if (!got) { ok = false; break; }
        tc_fence_after();
        const unsigned taddr = tmem_base + ((unsigned)(q * 32) << 16) + acc * BN + c_base;   // lane quarter, buffer, column half

        if (epi_uses_tma_store(EPI)) {
          // ---- staged epilogues: the warp's 32 rows go out as 64-byte-wide boxes through TMA ----
          // 32 bf16 columns (one box) or 2 x 16 fp32 columns (two boxes) per 32-column group.  Two
          // buffers alternate, so a box is filled while the TMA engine still reads the previous one.
#pragma unroll 1
          for (int cg = 0; cg < WARP_COLS / 32; ++cg) {
            const int g0 = cg * 32;                   // first of the warp's columns in this group
            const int j0 = n0 + c_base + g0;
            if (j0 >= n_eff) break;                   // warp-uniform
            float v[32];
            if (PROBE_NO_TMEM_LD && EPI == EPI_DLOGITS) {
#pragma unroll
              for (int c = 0; c < 32; ++c) v[c] = (float)(lane + c) * 1e-3f;
            } else {
              tmem_ld32(taddr + g0, v);
            }
            if (EPI == EPI_SUBSET_LOGP) {               // Z_U (or S = Z_U - lambda); columns past K are written as 0
#pragma unroll
              for (int c = 0; c < 32; ++c)
                v[c] = (j0 + c < n_eff) ? v[c] + (has_bias ? sb[g0 + c] : 0.f) - lam : 0.f;
            }
            if (EPI == EPI_DLOGITS) {
              if (has_bias) add_bias32(v, sb + g0);
              // w p = exp2(z log2(e) + off2), off2 = log2(w) - lambda log2(e): one packed FMA per two logits
              if (!PROBE_NO_MATH) {
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                  float x0, x1;
                  ffma2(x0, x1, v[c], v[c + 1], LOG2E, LOG2E, off2, off2);
                  v[c] = ex2(x0);
                  v[c + 1] = ex2(x1);
                }
              }
              if (sg[cg] != 0u) {
                // the group holds selected classes: subtract their weighted occupancy in fp32, before
                // the rounding to bf16; the loads are issued together, the unselected ones predicated off
                float g[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                  const int jj = sj[g0 + c];
                  g[c] = (jj >= 0 && row_ok) ? a.e.gamma[(long long)i * a.e.ld_gamma + jj] : 0.f;
                }
#pragma unroll
                for (int c = 0; c < 32; ++c) v[c] = fmaf(-w, g[c], wmul * v[c]);
              } else if (__any_sync(0xffffffffu, wmul != 1.f)) {      // rows whose weight is not in the exponent
#pragma unroll
                for (int c = 0; c < 32; ++c) v[c] *= wmul;
              }
              if (__any_sync(0xffffffffu, w == 0.f)) {
                if (w == 0.f) {                        // excluded utterance: exact zeros, whatever its logits are
#pragma unroll
                  for (int c = 0; c < 32; ++c) v[c] = 0.f;
                }
              }
            }
            constexpr int NBOX = epi_fp32_boxes(EPI) ? 2 : 1;        // boxes per group
            if (PROBE_NO_STORE && EPI == EPI_DLOGITS) {              // keep the values alive, store nothing
              float t = 0.f;
#pragma unroll
              for (int c = 0; c < 32; ++c) t += v[c];
              if (t == 12345.678f) a.status[1] = 1;
              continue;
            }
#pragma unroll
            for (int b = 0; b < NBOX; ++b) {
              if (NBOX == 2 && j0 + b * 16 >= n_eff) break;          // warp-uniform
              if (lane == 0) bulk_wait_read1();        // the box stored two boxes ago has left its buffer
              __syncwarp();
              unsigned char* box = stage + (nbox & 1u) * STAGE_BOX_BYTES;
              unsigned char* row = box + lane * 64;
              if (epi_fp32_boxes(EPI)) {
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4)
                  *reinterpret_cast<float4*>(row + (((unsigned)c4 ^ swz64) << 4)) =
                      make_float4(v[b * 16 + c4 * 4], v[b * 16 + c4 * 4 + 1], v[b * 16 + c4 * 4 + 2], v[b * 16 + c4 * 4 + 3]);
              } else {
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                  uint4 o;
                  __nv_bfloat162 p0 = __floats2bfloat162_rn(v[c8 * 8 + 0], v[c8 * 8 + 1]);
                  __nv_bfloat162 p1 = __floats2bfloat162_rn(v[c8 * 8 + 2], v[c8 * 8 + 3]);
                  __nv_bfloat162 p2 = __floats2bfloat162_rn(v[c8 * 8 + 4], v[c8 * 8 + 5]);
                  __nv_bfloat162 p3 = __floats2bfloat162_rn(v[c8 * 8 + 6], v[c8 * 8 + 7]);
                  o.x = *(unsigned*)&p0; o.y = *(unsigned*)&p1; o.z = *(unsigned*)&p2; o.w = *(unsigned*)&p3;
                  *reinterpret_cast<uint4*>(row + (((unsigned)c8 ^ swz64) << 4)) = o;
                }
              }
              fence_async_smem();                      // staged data visible to the TMA engine
              __syncwarp();
              if (EPI == EPI_DLOGITS && a.e.colpart != nullptr && row0_cta + q * 32 < a.m) {
                // db_c = dZ_c^T 1, first stage: lane c sums column c of the staged box, i.e. the rounded
                // values of this warp's 32 rows (rows past m hold exact zeros), into the row block's slot
                // lanes 0-15 take rows 0-15, lanes 16-31 rows 16-31; each reads column pair (lane & 15)
                // as one 32-bit word, widens both halves and adds them with one packed fp32 add
                const int cp = lane & 15, rbase = lane & 16;
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int rr = 0; rr < 16; ++rr) {
                  const int row = rbase + rr;
                  const unsigned piece = (unsigned)(cp >> 2) ^ (unsigned)((row >> 1) & 3);
                  const unsigned wv = *reinterpret_cast<const unsigned*>(box + row * 64 + (piece << 4) + (cp & 3) * 4);
                  s0 += __uint_as_float(wv << 16);
                  s1 += __uint_as_float(wv & 0xffff0000u);
                }
                s0 += __shfl_xor_sync(0xffffffffu, s0, 16);
                s1 += __shfl_xor_sync(0xffffffffu, s1, 16);
                const float cs = (lane & 16) ? s1 : s0;                    // lanes 0-15: even columns, 16-31: odd
                const int col = 2 * cp + ((lane >> 4) & 1);
                if (j0 + col < n_eff)
                  a.e.colpart[(long long)((row0_cta + q * 32) >> 5) * a.e.ld_colpart + j0 + col] = cs;
              }
              if (lane == 0) {
                if ((EPI == EPI_ACCUM_F32 || EPI == EPI_STORE_OUT) && a.e.accumulate)
                  tma_reduce_add_2d(&tmC, box, j0 + b * 16, row0_out + h * SUB_M + q * 32);
                else if ((PCTC_TUNE_CHUNK_HINT & 1) && EPI == EPI_DLOGITS)
                  tma_store_2d_hint(&tmC, box, j0 + b * 16, row0_out + h * SUB_M + q * 32, make_evict_first_policy());
                else tma_store_2d(&tmC, box, j0 + b * 16, row0_out + h * SUB_M + q * 32);
                bulk_commit();
              }
              ++nbox;
            }
          }
        }

#pragma unroll 1
        for (int cg = 0; cg < WARP_COLS / 32 && !epi_uses_tma_store(EPI); ++cg) {
          const int j0 = n0 + c_base + cg * 32;
          if (j0 >= n_eff) break;                    // warp-uniform
          float v[32];
          if (PROBE_NO_TMEM_LD && EPI == EPI_LSE_PARTIAL) {
#pragma unroll
            for (int c = 0; c < 32; ++c) v[c] = (float)(lane + c) * 1e-3f;
          } else {
            tmem_ld32(taddr + cg * 32, v);
          }
          if (PROBE_NO_MATH && EPI == EPI_LSE_PARTIAL) {
            float t = 0.f;
#pragma unroll
            for (int c = 0; c < 32; ++c) t += v[c];
            run_sum += t;
            continue;
          }
          if (EPI == EPI_STORE_F32) {
            if (row_ok) {
              float* dst = (float*)a.e.out + (long long)i * a.e.ld + j0;
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (j0 + c < n_eff) dst[c] = v[c];
            }
          } else if (EPI == EPI_ARGMAX_PARTIAL) {
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const float z = has_bias ? v[c] + sb[cg * 32 + c] : v[c];
              if (j0 + c < n_eff && z > best_z) { best_z = z; best_j = j0 + c; }   // ascending columns: first maximum wins
            }
          } else if (EPI == EPI_LSE_PARTIAL) {
            // running (max, sum of exp) in the base-2 domain: x = z * log2(e)
            if (j0 + 32 <= n_eff) {
              // whole group inside the matrix: max over the logits, then one packed FMA per two logits
              // forms x - max and feeds the exponentials
              if (has_bias) add_bias32(v, sb + cg * 32);
              // two chains of three-input maxima (a NaN logit is caught by the sum below, not here)
              float gm0 = fmax3(v[0], v[1], v[2]), gm1 = fmax3(v[3], v[4], v[5]);
#pragma unroll
              for (int c = 6; c + 3 < 32; c += 4) {
                gm0 = fmax3(gm0, v[c], v[c + 1]);
                gm1 = fmax3(gm1, v[c + 2], v[c + 3]);
              }
              const float gm = fmax3(gm0, gm1, fmaxf(v[30], v[31]));
              const float gmax = gm * LOG2E;
              if (gmax > run_max2) {
                run_sum *= ex2(run_max2 - gmax);     // ex2(-inf) = 0 on the first group
                run_max2 = gmax;
              }
              const float nm = -run_max2;
              float s0 = 0.f, s1 = 0.f;
#pragma unroll
              for (int c = 0; c < 32; c += 2) {
                float x0, x1;
                ffma2(x0, x1, v[c], v[c + 1], LOG2E, LOG2E, nm, nm);
                fadd2(s0, s1, s0, s1, ex2(x0), ex2(x1));   // one packed add per two exponentials
              }
              run_sum += s0 + s1;                    // a NaN logit makes the sum NaN
            } else {
              float gmax = -CUDART_INF_F;
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                v[c] = (j0 + c < n_eff) ? (has_bias ? v[c] + sb[cg * 32 + c] : v[c]) * LOG2E : -CUDART_INF_F;
                gmax = fmaxf(gmax, v[c]);
              }
              if (gmax > run_max2) {
                run_sum *= ex2(run_max2 - gmax);
                run_max2 = gmax;
              }
              float s = 0.f;
#pragma unroll
              for (int c = 0; c < 32; ++c) s += ex2(v[c] - run_max2);
              run_sum += s;
              if (gmax != gmax) run_sum = gmax;      // NaN logits poison the normaliser
            }
          }
        }

        tc_fence_before();
        __syncwarp();
        if (lane == 0) { if (CTAS == 2) mbar_arrive_leader(&st->tmem_empty[acc]); else mbar_arrive(&st->tmem_empty[acc]); }
        }
      }

      if (EPI == EPI_LSE_PARTIAL && ok && row_ok)
        a.e.partial[((long long)i * pstride + a.e.partial_offset + sp) * (EW / 4) + (ew >> 2)] =
            make_float2(run_max2 * LN2, run_sum);
      if (EPI == EPI_ARGMAX_PARTIAL && ok && row_ok)
        a.e.partial[((long long)i * pstride + a.e.partial_offset + sp) * (EW / 4) + (ew >> 2)] =
            make_float2(best_z, __int_as_float(best_j));
    }
    if (epi_uses_tma_store(EPI) && lane == 0) bulk_wait0();   // this warp's stores have completed
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait gave up somewhere in this CTA.  The leader has waited above for the copies of the stages
    // it issued itself (its barriers count the peer's bytes of those stages too) and for its MMAs.
    // What that cannot cover is a copy the peer issued for a stage the leader never reached: such a
    // copy lands within microseconds, so both CTAs simply stay for a fixed while before they leave.
    const long long t0 = clock64();
    while (clock64() - t0 < ABORT_LINGER_CYCLES) { }
    __syncthreads();
  }
  if (CTAS == 2) cluster_sync_all();     // no CTA of a pair leaves while the other may still signal it
  if (warp == 1) {
    tc_fence_after();
    if (CTAS == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// 2-D bf16 tensor map: `inner` contiguous elements per row, `rows` rows of pitch `ld` elements.
bool make_map(CUtensorMap* map, const void* base, unsigned long long inner, unsigned long long rows,
              unsigned long long ld, unsigned box_inner, unsigned box_rows, bool fp32 = false) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {ld * (fp32 ? 4 : 2)};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle swizzle =
      (box_inner * (fp32 ? 4u : 2u) == 64u) ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  return fn(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, PCTC_TUNE_L2_PROMOTION,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Per-device state: a process may drive several GPUs, and both the shared-memory opt-in of a kernel
// and the SM count belong to one device.  Entries are filled on first use; the values are the same
// whichever thread fills them.
constexpr int MAX_DEVICES = 64;
int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return 0;
  return dev;
}

int sm_count() {
  static std::atomic<int> table[MAX_DEVICES];
  const int dev = current_device();
  int n = table[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    n = v;
    table[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

constexpr int CTAS_DEFAULT = PCTC_TUNE_CTAS;

template <int EPI, int EW, int MT = 1>
cudaError_t launch_ew(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const UmmaArgs& a,
                      int grid, cudaStream_t stream) {
  // per device: 0 = this kernel has not been configured there yet, else the number of CTA groups
  // (clusters) that can be resident at once
  static std::atomic<int> groups_on[MAX_DEVICES];
  constexpr size_t SMEM = smem_bytes(CTAS_DEFAULT, EPI, EW, MT);
  static_assert(SMEM <= 227 * 1024, "shared memory budget");
  auto kern = k_umma_gemm<EPI, CTAS_DEFAULT, EW, MT>;
  const int dev = current_device();
  int max_groups = groups_on[dev].load(std::memory_order_acquire);
  if (max_groups == 0) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS_DEFAULT;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(num_threads(EW));
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = PCTC_TUNE_PDL ? 2 : 1;
  if (max_groups == 0) {
    cfg.gridDim = dim3((unsigned)(sm_count() / CTAS_DEFAULT * CTAS_DEFAULT));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) n = sm_count() / CTAS_DEFAULT;
    max_groups = n;
    groups_on[dev].store(n, std::memory_order_release);
  }
  if (grid > max_groups * CTAS_DEFAULT) grid = max_groups * CTAS_DEFAULT;
  cfg.gridDim = dim3((unsigned)grid);
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmC, a);
}

// Eight epilogue warps when a tile's main loop is short next to its epilogue (k <= 2048), else four.
constexpr int EW_SWITCH_K = 2048;
inline int epi_warps_for(int k) {
  if (PCTC_TUNE_EPI_WARPS == 4 || PCTC_TUNE_EPI_WARPS == 8) return PCTC_TUNE_EPI_WARPS;
  return k <= EW_SWITCH_K ? 8 : 4;
}

template <int EPI>
cudaError_t launch(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const UmmaArgs& a,
                   int grid, cudaStream_t stream) {
  if constexpr (EPI == EPI_STORE_OUT && CTAS_DEFAULT == 2) {
    if (a.tile_mt == 2) return launch_ew<EPI, 4, 2>(tmA, tmB, tmC, a, grid, stream);
  }
  return epi_warps_for(a.k) == 8 ? launch_ew<EPI, 8>(tmA, tmB, tmC, a, grid, stream)
                                 : launch_ew<EPI, 4>(tmA, tmB, tmC, a, grid, stream);
}

}  // namespace

bool umma_available() { return encode_fn() != nullptr; }

int umma_lse_partials_per_split(int k) { return epi_warps_for(k) / 4; }

#ifndef PCTC_TUNE_LSE_SPLITS
#define PCTC_TUNE_LSE_SPLITS 0    // > 0: force this many column splits in the column-walking kernels (experiments)
#endif

int umma_lse_splits(int m, int n) {
  if (PCTC_TUNE_LSE_SPLITS > 0) return PCTC_TUNE_LSE_SPLITS < (n + BN - 1) / BN ? PCTC_TUNE_LSE_SPLITS : (n + BN - 1) / BN;
  // column splits per row tile such that the (row tile, split) units fill whole waves of CTAs
  const int sms = sm_count() / CTAS_DEFAULT;       // CTA groups that run at once
  const int m_tiles = (m + BM * CTAS_DEFAULT - 1) / (BM * CTAS_DEFAULT), n_tiles = (n + BN - 1) / BN;
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= 32 && s <= n_tiles; ++s) {     // each split yields two partials per frame (column halves)
    const long long units = (long long)m_tiles * s;
    const long long waves = (units + sms - 1) / sms;
    const int per = (n_tiles + s - 1) / s;                 // column tiles of the largest split
    const double cost = (double)waves * per + 0.05 * waves; // tile-times on the critical CTA + per-unit overhead
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  return best;
}

int umma_accum_slab_rows(int m) {
  const int tile_m = BM * CTAS_DEFAULT;
  return (m + tile_m - 1) / tile_m * tile_m;
}

int umma_accum_splits(int m, int n, int k, size_t max_extra_bytes) {
  const int groups = 148 / CTAS_DEFAULT;            // planned for a full B200, without asking the device: the
                                                    // workspace size must not depend on where it is computed
  const long long tiles = (long long)(umma_accum_slab_rows(m) / (BM * CTAS_DEFAULT)) * ((n + BN - 1) / BN);
  const int k_blocks = (k + BK - 1) / BK;
  if (tiles >= 4LL * groups) return 1;              // enough tiles: the last wave is a small share
  const size_t slab = (size_t)umma_accum_slab_rows(m) * n * 4;
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= 16; ++s) {
    if (s > 1 && ((size_t)(s - 1) * slab > max_extra_bytes || k_blocks / s < 16)) break;
    const long long waves = (tiles * s + groups - 1) / groups;
    // k-blocks on the busiest CTA group; a unit costs about 12 k-blocks on top of its own (pipeline
    // refill, accumulator hand-over)
    const double cost = (double)waves * ((double)k_blocks / s + 12.0);
    if (cost < best_cost * 0.97) { best_cost = cost; best = s; }       // split only for a clear gain
  }
  return best;
}

cudaError_t umma_gemm(const __nv_bfloat16* A, long long lda, bool a_mn_major,
                      const __nv_bfloat16* B, long long ldb, bool b_mn_major,
                      int m, int n, int k, const Epilogue& e, int* status, cudaStream_t stream) {
  if (m <= 0 || n <= 0 || k <= 0) return cudaSuccess;
  if ((lda % 8) || (ldb % 8) || ((size_t)A & 15) || ((size_t)B & 15)) return cudaErrorInvalidValue;
  alignas(64) CUtensorMap tmA, tmB, tmC;
  bool ok = true;
  tmC = CUtensorMap{};
  // output boxes of the staged epilogues: 32 rows x 32 columns, clipped to the [m, n] extent
  const int ksplit = (e.kind == EPI_ACCUM_F32 && e.ksplit > 1) ? e.ksplit : 1;
  if (ksplit > 1 && (ksplit > (k + BK - 1) / BK || e.ksplit_rows < umma_accum_slab_rows(m))) return cudaErrorInvalidValue;
  if (e.kind == EPI_ACCUM_F32 || e.kind == EPI_SUBSET_LOGP) {
    if ((e.ld % 4) || ((size_t)e.out & 15)) return cudaErrorInvalidValue;
    const unsigned long long out_rows = (unsigned long long)(ksplit - 1) * e.ksplit_rows + m;   // k-split slabs stacked
    ok = ok && make_map(&tmC, e.out, (unsigned long long)n, out_rows, (unsigned long long)e.ld, 16, 32, true);
  } else if (e.kind == EPI_DLOGITS || e.kind == EPI_STORE_OUT) {
    if ((e.ld % 8) || ((size_t)e.out & 15)) return cudaErrorInvalidValue;
    ok = ok && make_map(&tmC, e.out, (unsigned long long)n, (unsigned long long)m, (unsigned long long)e.ld, 32, 32);
  }
  if (!a_mn_major) ok = ok && make_map(&tmA, A, (unsigned long long)k, (unsigned long long)m, lda, BK, BM);
  else ok = ok && make_map(&tmA, A, (unsigned long long)m, (unsigned long long)k, lda, 64, BK);
  if (!b_mn_major) ok = ok && make_map(&tmB, B, (unsigned long long)k, (unsigned long long)n, ldb, BK, BN / CTAS_DEFAULT);
  else ok = ok && make_map(&tmB, B, (unsigned long long)n, (unsigned long long)k, ldb, 64, BK);
  if (!ok) return cudaErrorInvalidValue;

  UmmaArgs a;
  a.m = m; a.n = n; a.k = k;
  a.a_mn = a_mn_major ? 1 : 0;
  a.b_mn = b_mn_major ? 1 : 0;
  a.nsplit = e.nsplit;
  a.ksplit = ksplit;
  a.ksplit_rows = ksplit > 1 ? e.ksplit_rows : 0;
  a.status = status;
  a.e = e;
  const int n_tiles = (n + BN - 1) / BN;
  const int groups = sm_count() / CTAS_DEFAULT;
  // 512-row tiles for the dW contraction when its main loop is long (the un-overlapped epilogue is then
  // a small share) and whole waves of the taller tiles cost no more than whole waves of the usual ones
  a.tile_mt = 1;
  if (PCTC_TUNE_MT2 && CTAS_DEFAULT == 2 && e.kind == EPI_STORE_OUT && k > EW_SWITCH_K && m >= 2 * BM * CTAS_DEFAULT) {
    const long long t1 = (long long)((m + 255) / 256) * n_tiles, t2 = (long long)((m + 511) / 512) * n_tiles;
    const long long w1 = (t1 + groups - 1) / groups, w2 = 2 * ((t2 + groups - 1) / groups);
    if (w2 <= w1) a.tile_mt = 2;
  }
  const int tile_m = BM * CTAS_DEFAULT * a.tile_mt;
  const int m_tiles = (m + tile_m - 1) / tile_m;
  const bool walks = e.kind == EPI_LSE_PARTIAL || e.kind == EPI_ARGMAX_PARTIAL;
  {
    // a unit of the walking kernels re-reads its A rows for every column tile: the band's A rows must
    // stay in L2 (and leave room for the streaming B); the other kernels read each panel once per
    // unit, and a near-square patch of tiles per wave touches the fewest panels
    long long g = PCTC_TUNE_RASTER_G / a.tile_mt;
    if (walks) g = ((long long)PCTC_TUNE_WALK_MB << 20) / ((long long)BM * CTAS_DEFAULT * k * 2);
    if (g < 1) g = 1;
    if (g > m_tiles) g = m_tiles;
    const int bands = (int)((m_tiles + g - 1) / g);
    a.raster_g = (m_tiles + bands - 1) / bands;          // bands of equal height
  }
  long long units = (long long)m_tiles * (walks ? e.nsplit : n_tiles) * ksplit;
  if (walks && (e.nsplit < 1 || e.nsplit > n_tiles)) return cudaErrorInvalidValue;
  const int grid = (int)(units < groups ? units : groups) * CTAS_DEFAULT;
  switch (e.kind) {
    case EPI_STORE_F32: return launch<EPI_STORE_F32>(tmA, tmB, tmC, a, grid, stream);
    case EPI_LSE_PARTIAL: return launch<EPI_LSE_PARTIAL>(tmA, tmB, tmC, a, grid, stream);
    case EPI_SUBSET_LOGP: return launch<EPI_SUBSET_LOGP>(tmA, tmB, tmC, a, grid, stream);
    case EPI_DLOGITS: return launch<EPI_DLOGITS>(tmA, tmB, tmC, a, grid, stream);
    case EPI_ACCUM_F32: return launch<EPI_ACCUM_F32>(tmA, tmB, tmC, a, grid, stream);
    case EPI_STORE_OUT: return launch<EPI_STORE_OUT>(tmA, tmB, tmC, a, grid, stream);
    case EPI_ARGMAX_PARTIAL: return launch<EPI_ARGMAX_PARTIAL>(tmA, tmB, tmC, a, grid, stream);
  }
  return cudaErrorInvalidValue;
}

}  // namespace pctc
