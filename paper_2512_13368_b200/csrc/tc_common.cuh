// Blackwell (sm_100a) building blocks of the tensor-core kernels: mbarrier, TMA tile loads,
// tcgen05 MMA / TMEM access, shared-memory matrix descriptors and column-mask helpers.
//
// Every wait is bounded: a wait that does not complete within kTimeoutCycles sets a sticky
// per-CTA abort flag, after which all further waits of the CTA return at once, the kernel runs
// to its normal end (all loops are bounded, barrier counts do not depend on wait results),
// frees its TMEM and reports BLOSSOM_ERR_TIMEOUT through the workspace status word.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace blossom {
namespace tc {

constexpr long long kTimeoutCycles = 400000000LL;  // ~0.2 s at 1.9 GHz

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier ---------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// named barrier among `count` threads (ids 1..15; 0 is __syncthreads)
__device__ __forceinline__ void named_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// One probe of the barrier.  try_wait lets the hardware park the thread for a short,
// implementation-defined time until the phase completes instead of returning at once, so a
// waiting warp does not compete for issue slots with the warps doing the arithmetic.  (An explicit
// suspend-time hint made every hand-off about 50 cycles slower.)
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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
// `site` (non-zero) names the wait in the kernel's source; the first wait of a CTA that runs out
// leaves it in the abort flag, from where it reaches word 1 of the workspace status.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          int site = 1) {
  if (mbar_try_wait(bar, parity)) return;
  if (*abort_flag) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag) return;
    if (clock64() - t0 > kTimeoutCycles) {
      *abort_flag = site;
      return;
    }
  }
}

// Move registers between the warpgroups of a CTA (every thread of a warpgroup executes it).
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// True in exactly one lane of a converged warp.  The single-thread roles keep their whole warp
// converged (every lane waits on the barriers and computes the uniform addresses) and put only the
// asynchronous instructions under this predicate, so that descriptors and addresses can live in
// uniform registers.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---- TMA: 4-D tiled load global -> shared, completion on an mbarrier ----------------------
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// 4-D tiled store shared -> global (rows past the tensor's extent are not written); the caller
// commits and waits for the bulk group before the shared memory is reused or the CTA exits.
__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2,
                                             int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
          reinterpret_cast<uint64_t>(map)),
      "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_store_commit_and_wait() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
// 1-D bulk copy global -> shared (both 16-byte aligned, size a multiple of 16), completion on an
// mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
      : "memory");
}
// generic-proxy shared-memory writes -> visible to the async proxy (TMA / tcgen05 operands)
__device__ __forceinline__ void fence_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---- TMEM + tcgen05 -----------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate; issued by ONE thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: A is a bf16 matrix held in tensor memory, row m in lane m, two
// consecutive K elements per 32-bit column (the lower K index in the low half), 8 columns per
// K = 16 step.
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc,
                                             uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the mbarrier once every MMA this thread issued so far has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_st() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets TMEM lane (warp%4)*32 + i.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float *v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
      "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
      "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
      "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
      "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])),
      "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])),
      "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
      "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])),
      "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])),
      "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}

// 16-column variants (thread i of the warp <-> TMEM lane (warp%4)*32 + i)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float *v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
      "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
      "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
      "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
      "r"(__float_as_uint(v[15]))
      : "memory");
}
// packed words (two bf16 per 32-bit column) -> tensor memory
__device__ __forceinline__ void tmem_st32u(uint32_t taddr, const uint32_t *v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
      "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
      "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
      "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16u(uint32_t taddr, const uint32_t *v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
      "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st8u(uint32_t taddr, const uint32_t *v) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr),
               "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
// two fp32 lanes per instruction (packed in a 64-bit register pair)
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;"
      : "=l"(d)
      : "l"(*reinterpret_cast<uint64_t *>(&a)), "l"(*reinterpret_cast<uint64_t *>(&b)),
        "l"(*reinterpret_cast<uint64_t *>(&c)));
  return *reinterpret_cast<float2 *>(&d);
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;"
      : "=l"(d)
      : "l"(*reinterpret_cast<uint64_t *>(&a)), "l"(*reinterpret_cast<uint64_t *>(&b)));
  return *reinterpret_cast<float2 *>(&d);
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;"
      : "=l"(d)
      : "l"(*reinterpret_cast<uint64_t *>(&a)), "l"(*reinterpret_cast<uint64_t *>(&b)));
  return *reinterpret_cast<float2 *>(&d);
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float *v) {
  static_assert(N == 16 || N == 32, "16 or 32 columns");
  if constexpr (N == 32) tmem_ld32(taddr, v); else tmem_ld16(taddr, v);
}
template <int N>
__device__ __forceinline__ void tmem_st(uint32_t taddr, const float *v) {
  static_assert(N == 16 || N == 32, "16 or 32 columns");
  if constexpr (N == 32) tmem_st32(taddr, v); else tmem_st16(taddr, v);
}

// ---- descriptors --------------------------------------------------------------------------
// Shared-memory matrix descriptor (64-bit): start address, leading / stride byte offsets
// (all >> 4), descriptor version 1, swizzle mode in bits 61..63 (2 = 128-byte, 4 = 64-byte).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                              uint32_t swizzle_mode) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= static_cast<uint64_t>(swizzle_mode) << 61;
  return d;
}
// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, majors (0 = K-major,
// 1 = MN-major), N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn_major) << 15) |
         (static_cast<uint32_t>(b_mn_major) << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// ---- 64-column masks ----------------------------------------------------------------------
__device__ __forceinline__ uint64_t cols_ge(int lo) {  // columns c >= lo
  return lo <= 0 ? ~0ull : (lo >= 64 ? 0ull : (~0ull << lo));
}
__device__ __forceinline__ uint64_t cols_le(int hi) {  // columns c <= hi
  return hi < 0 ? 0ull : (hi >= 63 ? ~0ull : ((2ull << hi) - 1ull));
}
// bit i of `bits` covers columns [i*bk, (i+1)*bk) of a 64-column tile
__device__ __forceinline__ uint64_t expand_block_bits(uint32_t bits, int bk) {
  if (bk == 64) return (bits & 1u) ? ~0ull : 0ull;
  if (bk == 32)
    return ((bits & 1u) ? 0x00000000FFFFFFFFull : 0ull) | ((bits & 2u) ? 0xFFFFFFFF00000000ull : 0ull);
  uint64_t m = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (bits & (1u << i)) m |= 0xFFFFull << (16 * i);
  return m;
}

// the smallest power of two >= x (1 for x <= 1)
__device__ __forceinline__ int pow2_at_least(int x) { return x <= 1 ? 1 : 1 << (32 - __clz(x - 1)); }

// Short-term mask of Eq. 15 over the 64 keys p0 ... p0 + 63 for query t, without the causal and
// the padding condition (the caller ANDs those): the window, and with the power-law mask the key
// blocks at power-of-two block distances and the last block.  `causal` is the caller's (often
// compile-time) copy of s.causal.
__device__ __forceinline__ uint64_t st_key_cols(const Shape &s, int t, int p0, bool causal) {
  uint64_t m = cols_ge(t - s.window + 1 - p0);
  if (!causal) m &= cols_le(t + s.window - 1 - p0);  // (without the causal mask the window has two sides)
  if (s.stis_mode) {
    m |= cols_ge(s.L - s.stis_blk - p0);
    const int bq = t / s.stis_blk;
    // key block bq - d, d a power of two: later d lie further left.  The walk starts at the first d
    // that can reach the tile from the right, the smallest power of two >= bq - (last block of the
    // tile), instead of at 1: a far tile then costs one or two steps, not log2 of its distance.
    const int dmin = bq - (p0 + 63) / s.stis_blk;
    for (int d = pow2_at_least(dmin); d <= bq; d <<= 1) {
      const int a = (bq - d) * s.stis_blk;
      if (a + s.stis_blk - 1 < p0) break;
      if (a <= p0 + 63) m |= cols_ge(a - p0) & cols_le(a + s.stis_blk - 1 - p0);
    }
    if (!causal) {
      for (int d = pow2_at_least(p0 / s.stis_blk - bq);; d <<= 1) {  // and key block bq + d: later d lie further right
        const int a = (bq + d) * s.stis_blk;
        if (a > p0 + 63 || a >= s.L) break;
        if (a + s.stis_blk - 1 >= p0) m |= cols_ge(a - p0) & cols_le(a + s.stis_blk - 1 - p0);
      }
    }
  }
  return m;
}
// The same mask seen from key p over the 64 queries t0 ... t0 + 63 (again without causality and
// padding).
__device__ __forceinline__ uint64_t st_query_cols(const Shape &s, int p, int t0, bool causal) {
  uint64_t m = cols_le(p + s.window - 1 - t0);
  if (!causal) m &= cols_ge(p - s.window + 1 - t0);
  if (s.stis_mode) {
    if (p >= s.L - s.stis_blk) return ~0ull;
    const int bk = p / s.stis_blk;
    for (int d = pow2_at_least(t0 / s.stis_blk - bk);; d <<= 1) {  // query block bk + d: later d lie further right
      const int a = (bk + d) * s.stis_blk;
      if (a > t0 + 63 || a >= s.L) break;
      if (a + s.stis_blk - 1 >= t0) m |= cols_ge(a - t0) & cols_le(a + s.stis_blk - 1 - t0);
    }
    if (!causal) {
      for (int d = pow2_at_least(bk - (t0 + 63) / s.stis_blk); d <= bk; d <<= 1) {  // and query block bk - d
        const int a = (bk - d) * s.stis_blk;
        if (a + s.stis_blk - 1 < t0) break;
        if (a <= t0 + 63) m |= cols_ge(a - t0) & cols_le(a + s.stis_blk - 1 - t0);
      }
    }
  }
  return m;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t *>(&h);
}

// Store one 64-column bf16 row (row r of a [rows][64] tile with 128-byte rows, 128-byte swizzle:
// 16-byte chunk ch lands at chunk position ch ^ (r & 7)).  `tile` must be 1024-byte aligned.
__device__ __forceinline__ void store_row_sw128(uint8_t *tile, int r, int ch, uint4 v) {
  *reinterpret_cast<uint4 *>(tile + r * 128 + ((ch ^ (r & 7)) << 4)) = v;
}

// ---- pieces shared by the forward and backward kernels ------------------------------------
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D>
struct Cfg {
  static constexpr int kRowBytes = D * 2;
  static constexpr int kBigBytes = 128 * kRowBytes;   // resident 128-row tile
  static constexpr int kSmallBytes = 64 * kRowBytes;  // streamed 64-row tile
  static constexpr int kAtomBytes = 8 * kRowBytes;    // 8-row swizzle atom of a D-wide tile
  static constexpr uint32_t kSwizzle = (D == 64) ? 2u : 4u;  // 128-byte / 64-byte swizzle
  static constexpr int kKStep = (16 * kRowBytes) >> 4;       // descriptor advance of 16 rows
};

// Per-CTA tile bookkeeping, built once per call by tc_meta_kernel and brought into shared memory
// by one bulk copy: [8][nT] selection bytes, nT list entries, nT flags, (forward) 2 nT per-phase
// items with 4 class bytes each, (dQ kernel) 16 class bytes per listed tile, and the counts {tiles
// on the list, long-term items, short-term items}.  Offsets in bytes; every part starts on a
// 16-byte boundary where a copy needs it.
// With a selection per query position (pq) an area of 128 nT bytes follows: in a query-major
// image [128 rows][nT] bytes, bit c of byte (r, jt): row r of the CTA selected key block
// jt * (64 / Bk) + c (the [8][nT] bytes at the start are then the union over a query block's
// rows); in a key-major image [8][nT] 64-bit words, bit i of word (g, qt): query position
// 64 qt + i selected key block g of the CTA.
struct MetaLayout {
  int list, flags, items, icls, jcls, counts, rows, bytes;
};
__host__ __device__ inline MetaLayout meta_layout(int nT, int pq = 0) {
  MetaLayout m;
  m.list = ((8 * nT + 15) / 16) * 16;
  m.flags = m.list + 2 * nT;
  m.items = ((m.flags + nT + 15) / 16) * 16;
  m.icls = m.items + 4 * nT;
  m.jcls = ((m.icls + 8 * nT + 15) / 16) * 16;
  m.counts = m.jcls + 16 * nT;
  m.rows = m.counts + 16;
  m.bytes = m.rows + (pq ? 128 * nT : 0);
  return m;
}
__host__ __device__ inline int meta_bytes(int nT, int pq = 0) { return meta_layout(nT, pq).bytes; }

// one arrival per warp, after all its lanes are done
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}

// common kernel end: everyone is done with tensor memory -> free it; report a timed-out wait
__device__ __forceinline__ void finish(int warp, uint32_t tmem_base, uint32_t ncols, int *abort_flag,
                                       int32_t *status) {
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, ncols);
  if (threadIdx.x == 0 && *abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}  // grace period for copies still in flight
    if (atomicCAS(status, 0, (int32_t)BLOSSOM_ERR_TIMEOUT) == 0) {  // first reporter: where it happened
      status[1] = *abort_flag;
      status[2] = (int32_t)blockIdx.x;
    }
  }
}

__device__ __forceinline__ float gate_alpha(const float *gate, int h) {
  return 1.f / (1.f + __expf(-(gate[h * 2 + 0] - gate[h * 2 + 1])));
}

// Store 16-byte chunk ch of row r of a D-wide bf16 tile laid out as TMA expects it (128-byte
// swizzle for D = 64, 64-byte swizzle for D = 32).  `tile` must be 1024-byte aligned.
template <int D>
__device__ __forceinline__ void store_row_chunk(uint8_t *tile, int r, int ch, uint4 v) {
  if constexpr (D == 64) *reinterpret_cast<uint4 *>(tile + r * 128 + ((ch ^ (r & 7)) << 4)) = v;
  else *reinterpret_cast<uint4 *>(tile + r * 64 + ((ch ^ ((r >> 1) & 3)) << 4)) = v;
}

// ---- host: TMA descriptor of a q-shaped bf16 tensor, box = (D, rows, 1, 1) -----------------
int make_tensor_map(CUtensorMap *map, const void *base, const Shape &s, int box_rows, bool kv = false,
                    int box_heads = 1);

// Builds the bookkeeping of every query-major CTA (forward, dQ) into qmeta and, if kmeta is not
// null, of every key-major CTA (dK/dV) into kmeta: meta_bytes(nT) bytes per CTA, CTA-major.
// branches: bit 0 long-term, bit 1 short-term: tiles that only the other branch needs are left out.
// with_fwd: 1 = the query-major images carry the forward's items, 0 = not, -1 = only when no
// key-major images are asked for (a forward call builds the forward's part, a backward call the
// rest; a training forward may build everything at once for a backward that reuses it).
int launch_tc_meta(const Shape &s, const int32_t *seq_lens, const int32_t *idx, uint8_t *qmeta,
                   uint8_t *kmeta, cudaStream_t st, int branches = 3, int with_fwd = -1);

// per-file launchers behind launch_fwd_tc / launch_bwd_tc
template <int D>
int launch_fwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt,
                    void *out_st, float *lse, const Workspace &ws, cudaStream_t st);
template <int D>
int launch_bwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, const void *out_lt,
                    const void *out_st, const float *lse, const void *dout, void *dq, void *dk,
                    void *dv, const Workspace &ws, cudaStream_t st, int branches, const float4 *records);

}  // namespace tc
}  // namespace blossom
