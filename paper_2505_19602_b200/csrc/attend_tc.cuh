// Tensor-core attention over the paged store for bf16, head_dim 128 (Sec. 3.3, Eq. 5):
// O = softmax(scale * Q K^T) V with online softmax.  One CTA owns up to two 128-query tiles (A, B)
// of one slice and streams the slice's K/V pages once for both.
//
// Roles inside a CTA of 384 threads:
//   warp 0 (one thread) : TMA producer.  The query tiles once; then per 128-key tile the K and V rows into
//                         128B-swizzled shared memory: history tiles page by page through the slice's
//                         page table, tiles of a not yet appended current map from the caller's tensors.
//   warp 1 (one thread) : tcgen05.mma issuer; owns the TMEM allocation (512 columns: two S/P buffers
//                         and two O accumulators).  With two query tiles the issue order is
//                         S_A(0), S_B(0), then per key tile j  PV_A(j), S_A(j+1), PV_B(j), S_B(j+1): while one
//                         tile's softmax runs, the tensor pipe works for the other tile, and a tile's next S
//                         product follows its PV product without a wait in between.  With one query tile the two S buffers
//                         alternate and S(j+1) is issued ahead of PV(j).
//   warps 4-7, 8-11     : softmax, one warpgroup per query tile (warps 4-7 tile A, warps 8-11 tile B), one
//                         thread per query row (TMEM lane), so that no row state is shared between threads and
//                         the two tiles' chains  S -> softmax -> PV  run concurrently, each hiding the other's
//                         hand-over latencies.  A thread sweeps its row of an S tile once, in four chunks of 32
//                         columns (tcgen05.ld), software-pipelined: p = exp2(s * c - m) of chunk cc + 1 against
//                         a lazy reference m (packed f32x2 arithmetic, in place) is issued before chunk cc is
//                         summed, checked and written as bf16 pairs over the first 64 columns of the row's S
//                         buffer (tcgen05.st; a chunk's P only covers columns already read), from where the PV
//                         product takes its A operand.  Only when a chunk's sum shows that an exponent left
//                         the lazy band (2^8) does the warp raise the reference: the chunk is recomputed, the
//                         P chunks already stored for this tile, the running sum and the O accumulator are
//                         scaled down, and the exponentials taken ahead for the next chunk are taken again.  Threads that own a row of the observation window also
//                         store that row's raw products (16-byte stores, key tile j in columns 128 j ..) for
//                         the compress that follows.  At the end each warpgroup normalises its O tile, stages
//                         it in the query tile's shared memory and one thread sends it out with TMA stores.
//                         With a single query tile (n_k <= 128, or the last odd tile of a map) warps 4-7 serve
//                         both S buffers and warps 8-11 idle.
//   warps 2-3           : append.  When the current map has not been copied into the store yet, its K/V
//                         tiles come from the caller's tensors, and the CTA whose turn it is writes each
//                         tile's rows from shared memory to the slice's pages (and their original
//                         positions), so the copy costs no extra read and stays off the critical path.
// Every mbarrier wait is bounded; a wait that gives up raises the sticky device status, sets a
// CTA-wide abort flag and all roles fall through to the common exit where TMEM is released.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>
#include <type_traits>
#include <string>

#include "common.cuh"

namespace scalekv {
namespace tc {

constexpr int kChunks = 4;                       // tcgen05.ld x32 loads per softmax thread (= query row) and S tile
// With two query tiles a PV product is issued in two parts: the steps over the keys of the first kEarlyChunks chunks
// as soon as their P is stored, under the sweep of the remaining chunks, and the rest when the tile's P is complete.
// What stands between the end of a sweep and the tile's next S tile is then 2 (4 - kEarlyChunks) + 8 MMAs, not 16.
constexpr int kEarlyChunks = 3;
static_assert(kEarlyChunks >= 1 && kEarlyChunks < kChunks, "both parts of a PV product need at least one chunk");
constexpr int kThreads = 128 + 2 * 128;          // warps: TMA, MMA, 2 x append, one softmax warpgroup per query tile
constexpr int kStages = 5;                       // one ring for the K and V tiles: K_0, V_0, K_1, V_1, ...
constexpr uint32_t kTileBytes = 128 * 128 * 2;   // one 128 x 128 bf16 operand tile
constexpr uint32_t kHalfBytes = kTileBytes / 2;  // 64 head-dim columns = one 128-byte swizzle span
constexpr uint32_t kOffQ = 0;                    // two query tiles (the dynamic shared memory must start 1024-byte aligned)
constexpr uint32_t kOffRing = kOffQ + 2 * kTileBytes;
constexpr uint32_t kOffBar = kOffRing + kStages * kTileBytes;
constexpr uint32_t kSmemBytes = kOffBar + 256;
static_assert(kSmemBytes <= 232448, "more shared memory than a CTA can have");
// barrier slots (8 bytes each): one full/empty pair per ring stage, one S/P/PV barrier per S buffer or query tile
enum { bQFull = 0, bFull = 1, bEmpty = bFull + kStages, bSFull = bEmpty + kStages, bPFull = bSFull + 2, bPvDone = bPFull + 2,
       bFinal = bPvDone + 2, bOut = bFinal + 2, bPEarly = bOut + 2, bPvEarly = bPEarly + 2, bCount = bPvEarly + 2 };
constexpr uint32_t kOffTmemSlot = 208;            // inside the barrier area, behind the barriers
static_assert(bCount * 8 <= kOffTmemSlot, "barriers overlap the TMEM slot");
static_assert(bCount <= 32, "one lane of the first warp initialises each barrier");
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256;       // S/P buffers at 0 and 128, O accumulators at 256 and 384
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the CTA is aborting or the time limit ran out (status raised).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                            unsigned long long limit_ns = kWaitLimitNs) {
  const unsigned long long t0 = globaltimer();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*abort_flag || *reinterpret_cast<volatile int *>(status) != 0) return false;
    if (globaltimer() - t0 > limit_ns) {
      *abort_flag = 1;
      atomicExch(status, kDevTimeout);
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status);
}
// Self-test of the bounded wait (scalekv_selftest_wait): one warp waits, with the given limit, on a barrier
// that nobody ever arrives at.  The wait must give up, raise the sticky status and return; a second warp that
// polls the CTA's abort flag (also bounded) shows that the other roles of a CTA see the give-up.
// out[0] = 1 when the wait returned false, out[1] = 1 when the second warp saw the abort flag.
__global__ void wait_probe_kernel(int *status, unsigned long long limit_ns, int *out) {
  __shared__ __align__(8) unsigned long long probe_bar;
  __shared__ int abort_word;
  const uint32_t bar = smem_u32(&probe_bar);
  if (threadIdx.x == 0) {
    abort_word = 0;
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int *abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    const bool ok = mbar_try(bar, 0) || mbar_wait_slow(bar, 0, abort_flag, status, limit_ns);
    out[0] = ok ? 0 : 1;
  } else if (threadIdx.x == 32) {
    const unsigned long long t0 = globaltimer();
    int seen = 0;
    while (!seen && globaltimer() - t0 < 4 * limit_ns + 1000000ull) seen = *abort_flag;
    out[1] = seen;
  }
}
// Same, with a warp-uniform result (the callers go on to warp-collective tcgen05 instructions).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status));
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(tm), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, int w, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap *tm, uint32_t src, int x, int y, int z, int w) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(tm), "r"(src), "r"(x), "r"(y),
               "r"(z), "r"(w)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// waits until the bulk stores committed so far have READ their shared-memory source (the CTA may then leave; the
// writes to global memory complete on their own)
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// orders this thread's shared-memory writes before later reads of the asynchronous (TMA) proxy
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// True in exactly one lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// The 64-bit shared-memory descriptors are passed as (low word, high word): the low word holds the
// start address field, so stepping through a tile is one 32-bit add per operand.
// Eight back-to-back MMAs of one 128 x 128 x 128 product, issued by the elected lane of a converged
// warp; the descriptors' start addresses advance by constant steps.  SS: both operands in shared
// memory (K-major tiles: steps of 32 B inside a 64-column half, then the next half).
__device__ __forceinline__ void tc_mma_ss_x8(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred e, pf, pt;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
      "elect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 pf, 0, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pf;\n\t"
      "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
      "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
      "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
      "add.u32 al, %1, 1024;\n\tadd.u32 bl, %2, 1024;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
      "add.u32 al, %1, 1026;\n\tadd.u32 bl, %2, 1026;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
      "add.u32 al, %1, 1028;\n\tadd.u32 bl, %2, 1028;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
      "add.u32 al, %1, 1030;\n\tadd.u32 bl, %2, 1030;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
      "}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc)
      : "memory");
}
// TS: A = P in TMEM (16 keys = 8 columns per step; a row's 128 bf16 values of P fill the first 64 columns of
// its S buffer), B = V in shared memory as the MN-major operand (16 keys = 2048 B per step).
__device__ __forceinline__ constexpr uint32_t p_col(int kk) { return (uint32_t)(kk * 8); }
__device__ __forceinline__ void tc_mma_ts_x8(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                             uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred e, pf, pt;\n\t.reg .b64 db;\n\t.reg .b32 at, bl;\n\t"
      "elect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 pf, %5, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, pf;\n\t"
      "add.u32 at, %1, %6;\n\tadd.u32 bl, %2, 128;\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "add.u32 at, %1, %7;\n\tadd.u32 bl, %2, 256;\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "add.u32 at, %1, %8;\n\tadd.u32 bl, %2, 384;\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "add.u32 at, %1, %9;\n\tadd.u32 bl, %2, 512;\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "add.u32 at, %1, %10;\n\tadd.u32 bl, %2, 640;\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "add.u32 at, %1, %11;\n\tadd.u32 bl, %2, 768;\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "add.u32 at, %1, %12;\n\tadd.u32 bl, %2, 896;\n\tmov.b64 db, {bl, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate_first), "n"(p_col(1)), "n"(p_col(2)), "n"(p_col(3)), "n"(p_col(4)),
      "n"(p_col(5)), "n"(p_col(6)), "n"(p_col(7))
      : "memory");
}
// The first N of the eight steps (a_tmem and b_lo address the first of them).
template <int N>
__device__ __forceinline__ void tc_mma_ts_n(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                            uint32_t accumulate_first) {
  static_assert(N >= 1 && N <= 8, "one to eight steps");
  asm volatile(
      "{\n\t.reg .pred e, pf, pt, q;\n\t.reg .b64 db;\n\t.reg .b32 at, bl, nn;\n\t"
      "elect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 pf, %5, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\tmov.u32 nn, %13;\n\t"
      "mov.b64 db, {%2, %3};\n\t@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, pf;\n\t"
      "setp.gt.and.u32 q, nn, 1, e;\n\tadd.u32 at, %1, %6;\n\tadd.u32 bl, %2, 128;\n\tmov.b64 db, {bl, %3};\n\t@q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "setp.gt.and.u32 q, nn, 2, e;\n\tadd.u32 at, %1, %7;\n\tadd.u32 bl, %2, 256;\n\tmov.b64 db, {bl, %3};\n\t@q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "setp.gt.and.u32 q, nn, 3, e;\n\tadd.u32 at, %1, %8;\n\tadd.u32 bl, %2, 384;\n\tmov.b64 db, {bl, %3};\n\t@q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "setp.gt.and.u32 q, nn, 4, e;\n\tadd.u32 at, %1, %9;\n\tadd.u32 bl, %2, 512;\n\tmov.b64 db, {bl, %3};\n\t@q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "setp.gt.and.u32 q, nn, 5, e;\n\tadd.u32 at, %1, %10;\n\tadd.u32 bl, %2, 640;\n\tmov.b64 db, {bl, %3};\n\t@q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "setp.gt.and.u32 q, nn, 6, e;\n\tadd.u32 at, %1, %11;\n\tadd.u32 bl, %2, 768;\n\tmov.b64 db, {bl, %3};\n\t@q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "setp.gt.and.u32 q, nn, 7, e;\n\tadd.u32 at, %1, %12;\n\tadd.u32 bl, %2, 896;\n\tmov.b64 db, {bl, %3};\n\t@q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, pt;\n\t"
      "}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate_first), "n"(p_col(1)), "n"(p_col(2)), "n"(p_col(3)), "n"(p_col(4)),
      "n"(p_col(5)), "n"(p_col(6)), "n"(p_col(7)), "n"(N)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float *v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const float *v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
      "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
      "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
      "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
      "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
      "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
// 16 consecutive 32-bit columns (32 bf16 values of P) of this thread's TMEM lane
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t *r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t *v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
      "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// packed pairs of fp32 in one 64-bit register
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// Shared-memory matrix descriptor, 128-byte swizzle, operand tiles whose 8-row groups are 1024 B
// apart.  K-major operands (Q, K): rows of 128 B, the leading offset is not used.  MN-major
// operand (V as [key][d]): 64 d-columns are contiguous, the next 64 start `lbo` bytes further.
// Low word: start address >> 4 (bits 0-13), leading byte offset >> 4 (bits 16-29).
// High word: stride byte offset >> 4 (bits 0-13), descriptor version (bit 14), swizzle mode (bits 29-31).
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128, A K-major; B K-major or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// Rare path of the softmax, taken by a whole warp when the sum of one of its rows' chunks shows that an
// exponent left the lazy band.  The chunk's 32 raw products are still intact in the row's S buffer (chunk cc
// sits in columns [32 cc, 32 cc + 32) of s_addr, the P chunks stored so far only cover columns below 16 cc) and
// are read again; `valid` of them are real keys.  Per lane the reference moves up to the chunk's maximum if
// that is larger (a lane that needs nothing gets the factor 1): the chunk's P is recomputed against the new
// reference and stored, and everything accumulated under the old one is multiplied by f = 2^(old - new): the
// running row sum, the P chunks p_first .. cc-1 stored for this tile that the tensor core has not been given yet
// (16 columns each), and - once the product that `pv_bar` stands for has landed: the previous PV product of the
// tile, or the early part of this one when its chunks have been handed over - the row's 128 columns of the O
// accumulator at o_addr.
// Everything goes in and out by value so that the caller's state stays in registers.
struct Raised { float m, l, sum; int o_landed, ok; };
__device__ __noinline__ Raised raise_reference(int valid, float c, float m, float l_run, uint32_t s_addr, int cc, int p_first,
                                               uint32_t o_addr, int with_o, int o_landed, uint32_t pv_bar, uint32_t pv_parity,
                                               volatile int *abort_flag, int *status) {
  float x[32];
  tc_ld32(s_addr + cc * 32, x);
  tc_wait_ld();
  float mt = -INFINITY;
#pragma unroll
  for (int i = 0; i < 32; ++i)
    if (i < valid) mt = fmaxf(mt, x[i]);
  const float m_new = fmaxf(m, mt * c);
  const float f = ex2(m - m_new);
  float sum = 0.f;
  uint32_t pk[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float p0 = (2 * i < valid) ? ex2(fmaf(x[2 * i], c, -m_new)) : 0.f;
    const float p1 = (2 * i + 1 < valid) ? ex2(fmaf(x[2 * i + 1], c, -m_new)) : 0.f;
    sum += p0 + p1;
    pk[i] = pack_bf16(p0, p1);
  }
  tc_st16(s_addr + cc * 16, pk);
#pragma unroll 1
  for (int e = p_first; e < cc; ++e) {
    uint32_t r[16];
    tc_ld16(s_addr + e * 16, r);
    tc_wait_ld();
#pragma unroll
    for (int i = 0; i < 16; ++i)
      r[i] = pack_bf16(__uint_as_float(r[i] << 16) * f, __uint_as_float(r[i] & 0xffff0000u) * f);
    tc_st16(s_addr + e * 16, r);
  }
  if (with_o) {
    if (!o_landed) {
      if (!mbar_wait_warp(pv_bar, pv_parity, abort_flag, status)) return {m_new, l_run * f, sum, 0, 0};
      tc_fence_after();
      o_landed = 1;
    }
#pragma unroll 1
    for (int e = 0; e < 4; ++e) {
      float o[32];
      tc_ld32(o_addr + e * 32, o);
      tc_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) o[i] *= f;
      tc_st32(o_addr + e * 32, o);
    }
  }
  tc_wait_st();
  return {m_new, l_run * f, sum, o_landed, 1};
}

struct Params {
  LayerView lv;
  TensorView O;
  float *lse;
  int n_k;
  float scale_log2e;   // softmax scale * log2(e)
  int box_rows;        // rows per K/V TMA box = min(page_tokens, 128)
  int fused_append;    // 1: the current map's K/V rows are still in the caller's tensors; read them there
  int copy_in;         // 1: and copy them into the pages on the way
  int n_prev;          // original position of the current map's first token
  // observation window (Sec. 3.3): when win_logits is not null, the raw products <q, k> of the w window rows
  // against every cache entry are recorded in win_logits[slice][rank][column], column = 128 j + position in key tile j
  float *win_logits;
  float *win_lse;      // [slice][rank]: base-2 log-sum-exp of each window row's logits (its softmax normaliser)
  int ld_l;            // leading dimension of a logit row
  int w;
  int win_pos[kMaxWindow];   // ascending raster indices of the window rows inside the current map
};

// kWindow: the launch records the observation window's logits; the instance without that code serves the launches
// that record nothing (its mere presence costs every warp's sweep 2-3 %).
template <bool kWindow>
__global__ void __launch_bounds__(kThreads, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKc,
                 const __grid_constant__ CUtensorMap tmVc, const __grid_constant__ CUtensorMap tmO, const Params prm) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  uint8_t *base_ptr = smem_raw;
  const uint32_t bars = base + kOffBar;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + kOffBar + kOffTmemSlot);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + kOffBar + kOffTmemSlot + 4);
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LayerView &lv = prm.lv;
  const int slice = blockIdx.y;
  const int b = slice / lv.n_heads, h = slice % lv.n_heads;
  const int n_k = prm.n_k;
  const int q_first = blockIdx.x * 256;                  // first query row of tile A
  const bool single = q_first + 128 >= n_k;              // tile B would be empty
  // What needs no global memory comes first: the lanes of warp 0 initialise one barrier each, warp 1 allocates the
  // TMEM.  When the launch allows it (programmatic stream serialisation) this part runs while the kernel before this
  // one in the stream is still finishing; `griddepcontrol.wait` then holds every thread until that kernel's writes
  // - cache lengths, page tables, pages, the status word - are visible.  The grid behind this one may come up as
  // soon as all of this grid's CTAs are running.
  if (warp == 0) {
    if (lane < bCount) {
      // arrivals per phase: a ring stage is released by the MMA warp's commit and the two append warps; P, early P and
      // the staged output tile are announced by one lane of each of the four warps of a softmax warpgroup
      const bool four = (lane >= bPFull && lane < bPFull + 2) || (lane >= bPEarly && lane < bPEarly + 2) ||
                        (lane >= bOut && lane < bOut + 2);
      const bool three = lane >= bEmpty && lane < bEmpty + kStages;
      mbar_init(bar(lane), four ? 4u : (three ? 3u : 1u));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  } else if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kOffBar + kOffTmemSlot), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int hist = lv.hist_len[slice];
  const int L = hist + n_k;
  // key tiles: Th from the pages (all of them unless the current map still waits in the caller's
  // tensors), then Tc of the current map; each source ends in a ragged tile
  const bool fused = prm.fused_append != 0;
  const int Th = ((fused ? hist : L) + 127) >> 7;
  const int Tc = fused ? (n_k + 127) >> 7 : 0;
  const int T = Th + Tc;
  auto tile_valid = [&](int j) {   // number of real keys in tile j
    const int rest = j < Th ? (fused ? hist : L) - j * 128 : n_k - (j - Th) * 128;
    return rest < 128 ? rest : 128;
  };
  int *status = lv.status;
  // Set-up, one rendezvous for everything.  Warp 0: its first lane decides for the whole CTA whether it runs at all
  // (one thread, because the status word may change between two threads' reads, and a CTA of which only a part
  // left would go on with barriers and TMEM nobody set up): an earlier CTA gave up - do not pile on; swizzled
  // tiles need the alignment, and a slice must not outgrow its page table - report, do not fault.  Meanwhile the
  // warp's lanes initialise one barrier each.  Warp 1 allocates the TMEM.  Everybody but warp 0 then waits on a
  // named barrier for the barriers, the decision and the allocation; warp 0 (the TMA producer) needs neither the
  // TMEM address nor anybody else: it only announces its part and goes on to issue the first loads while the
  // allocation is still under way.
  volatile int *leave_slot = reinterpret_cast<volatile int *>(base_ptr + kOffBar + kOffTmemSlot + 8);
  int leave = 0;
  if (warp == 0) {
    if (lane == 0) {
      if (*reinterpret_cast<volatile int *>(status) != 0) leave = 1;
      else if ((base & 1023u) || L > (lv.pages_per_slice << lv.page_shift)) { atomicExch(status, kDevCheck); leave = 1; }
      *abort_flag = 0;
      *leave_slot = leave;
    }
    leave = __shfl_sync(0xffffffffu, leave, 0);
    __syncwarp();
    __threadfence_block();
    asm volatile("bar.arrive 1, %0;" ::"n"(kThreads) : "memory");
  } else {
    tc_fence_before();
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
    tc_fence_after();
    leave = *leave_slot;
  }
  if (leave) {
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(kTmemCols) : "memory");
    return;
  }
  const uint32_t tmem = warp == 0 ? 0u : *tmem_slot;

  if (warp < 4) {
  if (warp == 0) {
    {
      // ---------------------------------------------------------------- TMA producer
      // (the whole warp walks the loop so that addresses stay warp-uniform; one lane issues)
      const int nq = single ? 1 : 2;
      if (elect_one()) {
        mbar_expect_tx(bar(bQFull), nq * kTileBytes);
        for (int t = 0; t < nq; ++t) {
          tma_load_4d(base + kOffQ + t * kTileBytes, &tmQ, 0, q_first + t * 128, h, b, bar(bQFull));
          tma_load_4d(base + kOffQ + t * kTileBytes + kHalfBytes, &tmQ, 64, q_first + t * 128, h, b, bar(bQFull));
        }
      }
      const int R = prm.box_rows;
      const int last_page = fused ? (hist > 0 ? (hist - 1) >> lv.page_shift : 0) : (L - 1) >> lv.page_shift;
      const int *pt = lv.page_table + (size_t)slice * lv.pages_per_slice;
      bool ok = true;
      // ring tile t = 2 j is K_j, t = 2 j + 1 is V_j
      for (int t = 0; t < 2 * T && ok; ++t) {
        const int st = t % kStages, j = t >> 1;
        ok = mbar_wait_warp(bar(bEmpty + st), ((t / kStages) & 1) ^ 1, abort_flag, status);
        if (!ok) break;
        const CUtensorMap *tm = (t & 1) ? &tmV : &tmK;
        if (j >= Th) {
          if (elect_one()) {
            const CUtensorMap *tc = (t & 1) ? &tmVc : &tmKc;
            const uint32_t dst = base + kOffRing + st * kTileBytes;
            mbar_expect_tx(bar(bFull + st), kTileBytes);
            tma_load_4d(dst, tc, 0, (j - Th) * 128, h, b, bar(bFull + st));
            tma_load_4d(dst + kHalfBytes, tc, 64, (j - Th) * 128, h, b, bar(bFull + st));
          }
        } else if (elect_one()) {
          mbar_expect_tx(bar(bFull + st), kTileBytes);
          for (int r0 = 0; r0 < 128; r0 += R) {
            const int slot = j * 128 + r0;
            int lp = slot >> lv.page_shift;
            lp = lp > last_page ? last_page : lp;
            const int row = (__ldg(pt + lp) << lv.page_shift) + (slot & lv.page_mask);
            const uint32_t dst = base + kOffRing + st * kTileBytes + r0 * 128;
            tma_load_2d(dst, tm, 0, row, bar(bFull + st));
            tma_load_2d(dst + kHalfBytes, tm, 64, row, bar(bFull + st));
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    {
      // ---------------------------------------------------------------- MMA issuer
      // (the whole warp walks the loop and waits; one elected lane issues the MMAs and commits)
      constexpr uint32_t idesc_qk = instr_desc(false);
      constexpr uint32_t idesc_pv = instr_desc(true);
      bool ok = mbar_wait_warp(bar(bQFull), 0, abort_flag, status);
      // S buffer `buf` = Q tile `qt` times K tile j (transposed)
      constexpr uint32_t dhi = desc_hi(1024);
      const bool leader = elect_one();
      const uint32_t q_lo[2] = {desc_lo(base + kOffQ, 16), desc_lo(base + kOffQ + kTileBytes, 16)};
      auto issue_s = [&](int j, int qt, int buf) {
        const uint32_t a_lo = q_lo[qt], b_lo = desc_lo(base + kOffRing + ((2 * j) % kStages) * kTileBytes, 16);
        const uint32_t d = tmem + kColS + buf * 128;
        tc_mma_ss_x8(d, a_lo, b_lo, dhi, idesc_qk);
        if (leader) tc_commit(bar(bSFull + buf));
        __syncwarp();
      };
      // O of tile `qt` += P (bf16 pairs in the first 32 columns of each half of S buffer `buf`) times V tile t
      auto issue_pv = [&](int t, int qt, int buf, uint32_t p_parity, bool release_v) -> bool {
        const int vt = 2 * t + 1, vs = vt % kStages;
        if (!mbar_wait_warp(bar(bFull + vs), (vt / kStages) & 1, abort_flag, status)) return false;
        if (!mbar_wait_warp(bar(bPFull + buf), p_parity, abort_flag, status)) return false;
        tc_fence_after();
        const uint32_t b_lo = desc_lo(base + kOffRing + vs * kTileBytes, kHalfBytes);
        const uint32_t d = tmem + kColO + qt * 128, a = tmem + kColS + buf * 128;
        const uint32_t acc0 = t > 0 ? 1u : 0u;
        tc_mma_ts_x8(d, a, b_lo, dhi, idesc_pv, acc0);
        if (leader) {
          tc_commit(bar(bPvDone + qt));
          if (release_v) tc_commit(bar(bEmpty + vs));
        }
        __syncwarp();
        return true;
      };
      if (!single) {
        // A tile's chain is  sweep -> PV(j) -> S(j+1) -> sweep ..., so between the moment a tile's P is complete
        // and the issue of its next S product this warp does nothing but issue: the operands of both products
        // are waited for beforehand (they arrive long before P does), the two products go out back to back, and the
        // commits follow them.
        auto ring_full = [&](int t) { return mbar_wait_warp(bar(bFull + t % kStages), (t / kStages) & 1, abort_flag, status); };
        auto mma_s = [&](int j, int qt) {
          tc_mma_ss_x8(tmem + kColS + qt * 128, q_lo[qt], desc_lo(base + kOffRing + ((2 * j) % kStages) * kTileBytes, 16), dhi, idesc_qk);
        };
        constexpr int kEarlySteps = 2 * kEarlyChunks;      // a chunk of 32 keys is two steps of 16
        auto mma_pv_early = [&](int j, int qt) {
          tc_mma_ts_n<kEarlySteps>(tmem + kColO + qt * 128, tmem + kColS + qt * 128,
                                   desc_lo(base + kOffRing + ((2 * j + 1) % kStages) * kTileBytes, kHalfBytes), dhi, idesc_pv,
                                   j > 0 ? 1u : 0u);
        };
        auto mma_pv_rest = [&](int j, int qt) {
          tc_mma_ts_n<8 - kEarlySteps>(tmem + kColO + qt * 128, tmem + kColS + qt * 128 + p_col(kEarlySteps),
                                       desc_lo(base + kOffRing + ((2 * j + 1) % kStages) * kTileBytes, kHalfBytes) + 128 * kEarlySteps,
                                       dhi, idesc_pv, 1u);
        };
        ok = ok && ring_full(0);
        if (ok) {
          tc_fence_after();
          mma_s(0, 0);
          if (leader) tc_commit(bar(bSFull + 0));
          __syncwarp();
          mma_s(0, 1);
          if (leader) { tc_commit(bar(bSFull + 1)); tc_commit(bar(bEmpty + 0)); }
          __syncwarp();
        }
        for (int j = 0; j < T && ok; ++j) {
          const bool more = j + 1 < T;
          ok = ring_full(2 * j + 1) && (!more || ring_full(2 * j + 2));
          for (int qt = 0; qt < 2 && ok; ++qt) {
            ok = mbar_wait_warp(bar(bPEarly + qt), j & 1, abort_flag, status);
            if (!ok) break;
            tc_fence_after();
            mma_pv_early(j, qt);
            if (leader) tc_commit(bar(bPvEarly + qt));
            __syncwarp();
            ok = mbar_wait_warp(bar(bPFull + qt), j & 1, abort_flag, status);
            if (!ok) break;
            tc_fence_after();
            mma_pv_rest(j, qt);
            if (more) mma_s(j + 1, qt);
            if (leader) {
              // after the last key tile the tile's one-shot barrier for the epilogue instead of an S barrier:
              // tile A normalises and stores its rows while tile B is still in its last sweep
              tc_commit(bar((more ? bSFull : bFinal) + qt));
              tc_commit(bar(bPvDone + qt));
              if (qt == 1) {
                tc_commit(bar(bEmpty + (2 * j + 1) % kStages));
                if (more) tc_commit(bar(bEmpty + (2 * j + 2) % kStages));
              }
            }
            __syncwarp();
          }
        }
      } else {
        for (int j = 0; j < T && ok; ++j) {
          ok = mbar_wait_warp(bar(bFull + (2 * j) % kStages), ((2 * j) / kStages) & 1, abort_flag, status);
          if (!ok) break;
          tc_fence_after();
          issue_s(j, 0, j & 1);
          if (leader) tc_commit(bar(bEmpty + (2 * j) % kStages));
          if (j > 0) ok = issue_pv(j - 1, 0, (j - 1) & 1, ((j - 1) >> 1) & 1, true);
        }
        if (ok) ok = issue_pv(T - 1, 0, (T - 1) & 1, ((T - 1) >> 1) & 1, true);
        if (ok && leader) tc_commit(bar(bFinal + 0));
      }
    }
  } else {
    // ------------------------------------------------------------------ append (warps 2 and 3)
    // Every ring tile is waited for and released, so that the empty barrier's phases stay in step;
    // only current-map tiles whose turn falls on this CTA are copied: rows [0, valid) of the tile go
    // to slots hist + 128 (j - Th) + r of the slice, un-swizzled, 16 bytes per thread and step.
    const int u = (warp - 2) * 32 + lane;
    const int chunk = u & 15, rsub = u >> 4;
    const uint32_t src_off = (uint32_t)(chunk >> 3) * kHalfBytes;
    bool ok = true;
    for (int t = 0; t < 2 * T && ok; ++t) {
      const int st = t % kStages, j = t >> 1;
      ok = mbar_wait_warp(bar(bFull + st), (t / kStages) & 1, abort_flag, status);
      if (!ok) break;
      if (prm.copy_in && j >= Th && (j - Th) % (int)gridDim.x == (int)blockIdx.x) {
        const int first = (j - Th) * 128;
        const int nvalid = tile_valid(j);
        char *pool = (t & 1) ? lv.v_pool : lv.k_pool;
        const uint32_t tile = base + kOffRing + st * kTileBytes + src_off;
        for (int r = rsub; r < nvalid; r += 4) {
          uint4 val;
          const uint32_t addr = tile + r * 128 + (((chunk & 7) ^ (r & 7)) << 4);
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(addr));
          const size_t row = slot_row(lv, slice, hist + first + r);
          reinterpret_cast<uint4 *>(pool + row * 256)[chunk] = val;
          if ((t & 1) == 0 && chunk == 0) lv.pos_pool[row] = prm.n_prev + first + r;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(bEmpty + st));
    }
  }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    const int qt = (warp - 4) >> 2;              // the query tile this warpgroup serves
    const int quarter = warp & 3;                // the TMEM lane quarter this warp may access
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const float c = prm.scale_log2e;
    const uint64_t c2 = pack2(c, c);
    const bool active = qt == 0 || !single;      // with one query tile the second warpgroup has nothing to do
    float m = -INFINITY, l = 0.f;
    // window row of this thread (rank in the window, or -1) and whether its warp has any
    int wrank = -1;
    bool wwarp = false;
    if (kWindow && prm.win_logits != nullptr && active) {
      const int qi = q_first + qt * 128 + row;
      for (int e = 0; e < prm.w; ++e)
        if (prm.win_pos[e] == qi) wrank = e;
      wwarp = __any_sync(0xffffffffu, wrank >= 0);
    }
    // (the window row's address is taken once: inside the sweep it would cost 64-bit arithmetic in every chunk)
    float *win_row = wrank >= 0 ? prm.win_logits + ((size_t)slice * prm.w + wrank) * prm.ld_l : nullptr;
    const uint32_t o_addr = lane_addr + kColO + qt * 128;
    bool ok = true;
    for (int j = 0; j < T && ok && active; ++j) {
      const int buf = single ? (j & 1) : qt;
      const uint32_t par = single ? ((j >> 1) & 1) : (j & 1);
      ok = mbar_wait_warp(bar(bSFull + buf), par, abort_flag, status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t s_addr = lane_addr + kColS + buf * 128;
      const int valid = tile_valid(j);           // < 128 only in a ragged tile
      int o_landed = 0;                          // the previous PV product of this tile has been waited for
      // The sweep is software-pipelined over the chunks: while chunk cc is summed, packed, checked and stored
      // ("back"), the exponentials of chunk cc + 1 ("front": x = s c - m and 2^x, in place in the chunk's registers)
      // are already issued, against the reference as it stands.  They are independent of chunk cc's check, so the
      // transcendental unit stays busy across the vote and the stores; in the rare case that the check raises the
      // reference, chunk cc + 1 is read again and redone.
      float v[2][32];
      auto log_window = [&](const float *x, int cc) {
        // The row's raw products go out as they are (the score kernel applies the softmax scale), 32
        // columns as eight 16-byte stores, at column 128 j + ...: key tile j owns columns [128 j, 128 j + 128)
        // of a logit row, so the current map starts at the next multiple of 128 behind the history and
        // every store is aligned.  Columns of a ragged tile beyond its keys hold finite values nobody reads.
        if (wrank >= 0) {
          float4 *dst = reinterpret_cast<float4 *>(win_row + (j * 128 + cc * 32));
#pragma unroll
          for (int i = 0; i < 8; ++i) dst[i] = make_float4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
        }
        __syncwarp();   // the tcgen05 instructions that follow want the warp converged
      };
      // (masked: a ragged tile, whose columns beyond the last key must not count)
      auto front = [&](float *x, int vc, auto masked) {      // vc: real keys in this chunk (>= 32: all)
        const uint64_t negm2 = pack2(-m, -m);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float a0, a1;
          unpack2(fma2(pack2(x[2 * i], x[2 * i + 1]), c2, negm2), a0, a1);
          if constexpr (decltype(masked)::value) {
            if (2 * i >= vc) a0 = -INFINITY;
            if (2 * i + 1 >= vc) a1 = -INFINITY;
          }
          x[2 * i] = ex2(a0);
          x[2 * i + 1] = ex2(a1);
        }
      };
      // 32 values of at most 2^8 sum to at most 2^13; a larger, infinite or NaN sum means that some x exceeded 8.
      auto back = [&](const float *pv, uint32_t *pk) -> float {
        uint64_t sum2a = pack2(0.f, 0.f), sum2b = sum2a;
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          sum2a = add2(sum2a, pack2(pv[2 * i], pv[2 * i + 1]));
          sum2b = add2(sum2b, pack2(pv[2 * i + 2], pv[2 * i + 3]));
          pk[i] = pack_bf16(pv[2 * i], pv[2 * i + 1]);
          pk[i + 1] = pack_bf16(pv[2 * i + 2], pv[2 * i + 3]);
        }
        float s0, s1, s2, s3;
        unpack2(sum2a, s0, s1);
        unpack2(sum2b, s2, s3);
        return (s0 + s1) + (s2 + s3);
      };
      auto sweep = [&](auto masked) {
      tc_ld32(s_addr, v[0]);
      tc_ld32(s_addr + 32, v[1]);
      tc_wait_ld();
      if (kWindow && wwarp) { log_window(v[0], 0); log_window(v[1], 1); }
      if (j == 0) {
        // no reference yet: the largest of the row's first 32 products serves (column 0 of the first tile
        // always holds a key, so it is finite); a later chunk that exceeds the band raises it like any other
        float mt = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float e0 = (i < valid) ? v[0][i] : -INFINITY;
          const float e1 = (i + 1 < valid) ? v[0][i + 1] : -INFINITY;
          mt = max3(mt, e0, e1);
        }
        m = mt * c;
      }
      front(v[0], valid, masked);
#pragma unroll
      for (int cc = 0; cc < kChunks; ++cc) {
        uint32_t pk[16];
        const int vc = valid - cc * 32;
        if (cc + 1 < kChunks) front(v[(cc + 1) & 1], vc - 32, masked);
        const float lt = back(v[cc & 1], pk);
        if (cc + 2 < kChunks) tc_ld32(s_addr + (cc + 2) * 32, v[cc & 1]);
        if (__any_sync(0xffffffffu, !(lt <= 8192.f))) {
          // Once the early chunks' P is with the tensor core, their product has to land before O is scaled, and only
          // the later chunks' P is still this thread's to scale.
          const bool late = !single && cc >= kEarlyChunks;
          const Raised r = raise_reference(vc, c, m, l, s_addr, cc, late ? kEarlyChunks : 0, o_addr, (late || j > 0) ? 1 : 0,
                                           late ? (o_landed == 2) : (o_landed >= 1), bar((late ? bPvEarly : bPvDone) + qt),
                                           (late ? j : j - 1) & 1, abort_flag, status);
          ok = __all_sync(0xffffffffu, r.ok != 0);
          if (!ok) return;
          m = r.m; l = r.l + r.sum;
          if (r.o_landed) o_landed = late ? 2 : 1;
          if (cc + 1 < kChunks) {
            // the next chunk's exponentials were taken against the old reference: once more, from its raw products
            tc_ld32(s_addr + (cc + 1) * 32, v[(cc + 1) & 1]);
            tc_wait_ld();
            front(v[(cc + 1) & 1], vc - 32, masked);
          }
        } else {
          tc_st16(s_addr + cc * 16, pk);
          l += lt;
        }
        if (!single && cc == kEarlyChunks - 1) {
          // P of the first chunks is complete: that part of the PV product may start under the rest of the sweep
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(bPEarly + buf));
        }
        if (cc + 2 < kChunks) tc_wait_ld();
      }
      // The window rows' products of the tile's second half are recorded here, not between the chunks (a branch
      // there costs every warp's schedule 2-3 %): columns 64-127 of the S buffer still hold them, P only covers
      // columns 0-63, and the buffer is not written again before this warp has arrived below.
      if (kWindow && wwarp && ok) {
        tc_ld32(s_addr + 64, v[0]);
        tc_ld32(s_addr + 96, v[1]);
        tc_wait_ld();
        log_window(v[0], 2);
        log_window(v[1], 3);
      }
      };
      if (valid < 128) sweep(std::true_type{}); else sweep(std::false_type{});
      if (!ok) break;
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(bPFull + buf));
    }
    if (ok && active) {
      // a barrier that completes exactly once, after the last PV product: the per-tile PV barrier will
      // not do, a parity wait cannot tell phases two apart and this warp may be that far behind it
      ok = mbar_wait_warp(bar(bFinal + qt), 0, abort_flag, status);
    }
    if (ok && active) {
      tc_fence_after();
      const float inv = 1.f / l;
      const int qi = q_first + qt * 128 + row;
      // The normalised rows go to the query tile's shared memory (no product reads it any more) in the layout
      // of a TMA box - two halves of 64 columns, rows of 128 bytes, 128-byte swizzle - and one thread sends the
      // tile out with two bulk tensor stores: a row written by its own thread straight to global memory costs a
      // 128-byte line per lane and store instruction.  The tensor map clips the rows beyond n_k.
      const uint32_t stage = base + kOffQ + qt * kTileBytes + row * 128;
      float o[2][32];
      tc_ld32(o_addr, o[0]);
#pragma unroll
      for (int cc = 0; cc < kChunks; ++cc) {
        tc_wait_ld();
        if (cc + 1 < kChunks) tc_ld32(o_addr + (cc + 1) * 32, o[(cc + 1) & 1]);
        const float *oc = o[cc & 1];
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          const uint32_t wx = pack_bf16(oc[8 * v4 + 0] * inv, oc[8 * v4 + 1] * inv);
          const uint32_t wy = pack_bf16(oc[8 * v4 + 2] * inv, oc[8 * v4 + 3] * inv);
          const uint32_t wz = pack_bf16(oc[8 * v4 + 4] * inv, oc[8 * v4 + 5] * inv);
          const uint32_t ww = pack_bf16(oc[8 * v4 + 6] * inv, oc[8 * v4 + 7] * inv);
          const uint32_t addr = stage + (uint32_t)(cc >> 1) * kHalfBytes + ((uint32_t)(((cc & 1) * 4 + v4) ^ (row & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(wx), "r"(wy), "r"(wz), "r"(ww) : "memory");
        }
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(bOut + qt));
      if (quarter == 0) {
        // one warp waits until all rows of the tile are staged; one of its lanes issues the stores
        ok = mbar_wait_warp(bar(bOut + qt), 0, abort_flag, status);
        if (ok && elect_one()) {
          const uint32_t src = base + kOffQ + qt * kTileBytes;
          tma_store_4d(&tmO, src, 0, q_first + qt * 128, h, b);
          tma_store_4d(&tmO, src + kHalfBytes, 64, q_first + qt * 128, h, b);
          tma_store_commit();
        }
        __syncwarp();
      }
      if (prm.lse != nullptr && qi < n_k) prm.lse[(size_t)slice * n_k + qi] = (m + log2f(l)) * 0.6931471805599453f;
      if (kWindow && wrank >= 0) prm.win_lse[(size_t)slice * prm.w + wrank] = m + log2f(l);
    }
    if (quarter == 0) tma_store_wait_read();   // (a lane that issued nothing has nothing to wait for)
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace tc

// Host side: tensor maps over the K and V pools (built once) and over Q (per call), launch.
struct AttendTc {
  using EncodeFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  EncodeFn encode = nullptr;
  CUtensorMap tmK, tmV;
  bool on = false;
  int box_rows = 128;

  bool init(int dtype, int head_dim, void *k_pool, void *v_pool, long long n_pages, int page_tokens, std::string &err) {
    on = false;
    if (dtype != 0 || head_dim != 128) return true;   // f32 x 64 is served by the FMA kernel
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) {
      err = "cuTensorMapEncodeTiled not available";
      return false;
    }
    encode = reinterpret_cast<EncodeFn>(fn);
    box_rows = page_tokens < 128 ? page_tokens : 128;
    const cuuint64_t dims[2] = {128, (cuuint64_t)n_pages * (cuuint64_t)page_tokens};
    const cuuint64_t strides[1] = {256};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    for (int i = 0; i < 2; ++i) {
      CUresult r = encode(i == 0 ? &tmK : &tmV, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, i == 0 ? k_pool : v_pool, dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) { err = "cuTensorMapEncodeTiled(pool) failed with code " + std::to_string((int)r); return false; }
    }
    if (cudaFuncSetAttribute(tc::attend_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(tc::attend_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes) != cudaSuccess) {
      err = "cannot raise the dynamic shared memory limit";
      return false;
    }
    on = true;
    return true;
  }
  bool enabled() const { return on; }

  // [B][H][n_k][128] bf16 view -> 4-D tensor map with boxes of 128 rows x 64 columns
  bool map_rows(CUtensorMap *tm, const TensorView &X, int n_k, int n_heads, int B, const char *what, std::string &err) {
    const cuuint64_t dims[4] = {128, (cuuint64_t)n_k, (cuuint64_t)n_heads, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)X.st * 2, (cuuint64_t)X.sh * 2, (cuuint64_t)X.sb * 2};
    const cuuint32_t box[4] = {64, 128, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<char *>(X.ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { err = std::string("cuTensorMapEncodeTiled(") + what + ") failed with code " + std::to_string((int)r); return false; }
    return true;
  }

  // Kc / Vc: the current map's K and V when they have not been copied into the store yet (the kernel
  // reads them there and copies them in), else nullptr.
  // win_logits / win_pos / w: where to record the window rows' logits (nullptr: do not).
  bool launch(const LayerView &lv, const TensorView &Q, const TensorView &O, float *lse, int n_k, const TensorView *Kc,
              const TensorView *Vc, bool copy_in, int n_prev, float scale, float *win_logits, float *win_lse, int ld_l, const int *win_pos, int w,
              cudaStream_t stream, std::string &err) {
    CUtensorMap tmQ, tmKc, tmVc, tmO;
    const int B = lv.n_slices / lv.n_heads;
    if (!map_rows(&tmQ, Q, n_k, lv.n_heads, B, "Q", err)) return false;
    if (!map_rows(&tmO, O, n_k, lv.n_heads, B, "O", err)) return false;
    const bool fused = Kc != nullptr && Vc != nullptr;
    if (fused) {
      if (!map_rows(&tmKc, *Kc, n_k, lv.n_heads, B, "K", err) || !map_rows(&tmVc, *Vc, n_k, lv.n_heads, B, "V", err)) return false;
    } else {
      tmKc = tmQ;
      tmVc = tmQ;
    }
    tc::Params prm;
    prm.lv = lv; prm.O = O; prm.lse = lse; prm.n_k = n_k;
    prm.scale_log2e = scale * 1.4426950408889634f;
    prm.box_rows = box_rows;
    prm.fused_append = fused ? 1 : 0;
    prm.copy_in = (fused && copy_in) ? 1 : 0;
    prm.n_prev = n_prev;
    prm.win_logits = win_logits;
    prm.win_lse = win_lse;
    prm.ld_l = ld_l;
    prm.w = win_logits ? w : 0;
    for (int e = 0; e < kMaxWindow; ++e) prm.win_pos[e] = (win_logits && e < w) ? win_pos[e] : -1;
    dim3 grid((n_k + 255) / 256, lv.n_slices);
    // programmatic stream serialisation: the kernel's set-up may overlap the end of the kernel before it in the stream
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(tc::kThreads);
    cfg.dynamicSmemBytes = tc::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t launched = win_logits ? cudaLaunchKernelEx(&cfg, tc::attend_tc_kernel<true>, tmQ, tmK, tmV, tmKc, tmVc, tmO, prm)
                                            : cudaLaunchKernelEx(&cfg, tc::attend_tc_kernel<false>, tmQ, tmK, tmV, tmKc, tmVc, tmO, prm);
    if (launched != cudaSuccess) {
      err = "attend: kernel launch failed";
      return false;
    }
    return true;
  }
};

}  // namespace scalekv
