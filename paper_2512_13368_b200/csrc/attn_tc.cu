// Tensor-core kernels of the fused two-branch attention (bf16 storage, fp32 accumulate):
// forward, backward dQ, backward dK/dV.  All three share one warp-specialised pipeline.
//
// CTA = 288 threads: warp 8 is the producer (one lane issues every TMA load and every
// tcgen05.mma), warps 0..7 compute.  A CTA owns a resident 128-row tile (rows = TMEM lanes) and
// streams 64-row tiles past it.  Row r of the 128 is shared by two compute threads: warp w and
// warp w + 4 both address TMEM lane quarter w % 4; the first takes columns 0..31 of a 64-column
// tile, the second columns 32..63.  Per streamed tile i:
//
//   producer : wait TMA(i), wait "tile i-1 loaded into registers" -> issue the first-stage MMAs
//              of tile i (S = Q K^T, in the backward also dP = dO V^T) -> commit s_full
//              then wait "bf16 tile i-1 written" -> issue the second-stage MMAs of tile i-1
//              (P V / dS K / W^T dO, dS^T Q) -> commit mma_done -> refill that TMA stage
//   compute  : wait s_full(i) -> tcgen05.ld its 32 columns -> arrive s_empty -> masks + softmax /
//              gradient arithmetic in registers -> wait mma_done(i-1) -> write bf16 tile to
//              128-byte-swizzled shared memory -> arrive t_full
//
// so the first-stage MMAs of tile i+1 and the second-stage MMAs of tile i-1 run while the
// compute warps work on tile i, and nothing in the loop is a block-wide barrier.
//
//  forward      resident Q (128 queries), streams K,V 64-key tiles of the union of the tiles its
//               128/Bk query blocks selected (Eq. 14, 16) or reach through the window (Eq. 15, 17);
//               two online softmaxes with a lazily raised maximum (raised, and the TMEM
//               accumulator rescaled, only when a tile's maximum exceeds it by > 2^8); the two
//               threads of a row exchange their half-row maxima through shared memory;
//               epilogue: normalise, gate mix (Eq. 19), store out / out_lt / out_st / lse.
//  dQ           same walk; S and dP from TMEM, probabilities from the saved log-sum-exps,
//               dS = P_lt (alpha dP - delta_lt) + P_st (beta dP - delta_st) (one tile for both
//               branches, they share K), dQ += dS K.  Prologue: delta = rowsum(G_branch o O_branch)
//               (stored for the dK/dV kernel).  d alpha = sum (P_lt - P_st) dP in fp32.
//  dK/dV        transposed: resident K,V of 128 keys, streams Q,dO 64-query tiles that selected
//               one of its key blocks or whose window reaches them; S^T = K Q^T, dP^T = V dO^T;
//               thread = key row; per-query lse / delta come from shared memory;
//               W^T = alpha P_lt + beta P_st, dS^T; dV += W^T dO, dK += dS^T Q.
//
// Deterministic: no atomics on any gradient.  Every wait is bounded (tc_common.cuh).
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kThreads = 288;
constexpr int kComputeWarps = 8;

template <int D>
struct Cfg {
  static constexpr int kRowBytes = D * 2;
  static constexpr int kBigBytes = 128 * kRowBytes;   // resident 128-row tile
  static constexpr int kSmallBytes = 64 * kRowBytes;  // streamed 64-row tile
  static constexpr int kPBytes = 128 * 128;           // [128][64] bf16 tile, 128-byte rows
  static constexpr int kAtomBytes = 8 * kRowBytes;    // 8-row swizzle atom of a D-wide tile
  static constexpr uint32_t kSwizzle = (D == 64) ? 2u : 4u;  // 128-byte / 64-byte swizzle
  static constexpr int kKStep = (16 * kRowBytes) >> 4;       // descriptor advance of 16 rows
  static constexpr int OC = D / 2;                            // accumulator columns per thread
};

__host__ __device__ inline int meta_bytes(int nT) { return ((11 * nT + 15) / 16) * 16 + 16; }

struct Pipe {
  uint32_t full0, res, s_full, s_empty, t_full, mma_done;
};

template <int STAGES>
__device__ __forceinline__ Pipe pipe_setup(uint64_t *bars, int tid) {
  Pipe p;
  p.full0 = smem_u32(&bars[0]);
  p.res = smem_u32(&bars[STAGES]);
  p.s_full = smem_u32(&bars[STAGES + 1]);
  p.s_empty = smem_u32(&bars[STAGES + 2]);
  p.t_full = smem_u32(&bars[STAGES + 3]);
  p.mma_done = smem_u32(&bars[STAGES + 4]);
  if (tid == 0) {
    for (int i = 0; i < STAGES; ++i) mbar_init(p.full0 + 8 * i, 1);
    mbar_init(p.res, 1);
    mbar_init(p.s_full, 1);
    mbar_init(p.s_empty, kComputeWarps);
    mbar_init(p.t_full, kComputeWarps);
    mbar_init(p.mma_done, 1);
    mbar_fence_init();
  }
  return p;
}

// one arrival per compute warp, after all its lanes are done
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}

__device__ __forceinline__ void finish(int warp, uint32_t tmem_base, int *abort_flag, int32_t *status) {
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 256);
  if (threadIdx.x == 0 && *abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}  // grace period for copies still in flight
    atomicExch(status, (int32_t)BLOSSOM_ERR_TIMEOUT);
  }
}

__device__ __forceinline__ float gate_alpha(const float *gate, int h) {
  return 1.f / (1.f + __expf(-(gate[h * 2 + 0] - gate[h * 2 + 1])));
}

// Query-major tile list (forward and dQ): per 64-key tile, which key blocks each of the CTA's
// query blocks selected (selb[g * nT + tile]), and the ascending list of tiles to visit with
// flags (bit 0: some selected block lies in the tile, bit 1: the window of some row reaches it).
__device__ __forceinline__ void build_query_major_list(const Shape &s, const int32_t *idx, int u, int st,
                                                       int pad0, int nT, uint32_t *selw, uint8_t *selb,
                                                       uint16_t *list, uint8_t *lflags, int *nvis_out) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = 128 / s.Bk, nb = 64 / s.Bk;
  const int row0 = st * 128, row_last = min(s.L - 1, row0 + 127);
  for (int i = tid; i < (8 * nT + 3) / 4; i += kThreads) selw[i] = 0u;
  __syncthreads();
  for (int i = tid; i < G * s.topk; i += kThreads) {
    const int g = i / s.topk, slot = i % s.topk, qb = st * G + g;
    if (qb < s.M) {
      const int blk = idx[((int64_t)u * s.M + qb) * s.topk + slot];
      if (blk >= 0 && blk <= qb) {
        const int a = g * nT + blk / nb;
        atomicOr(&selw[a >> 2], (1u << (blk % nb)) << ((a & 3) * 8));
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    const int jt_max = row_last >> 6;
    int count = 0;
    for (int base = 0; base <= jt_max; base += 32) {
      const int jt = base + lane;
      int f = 0;
      if (jt <= jt_max && row_last >= pad0 && jt * 64 + 63 >= pad0) {
        for (int g = 0; g < G; ++g) f |= selb[g * nT + jt] ? 1 : 0;
        if (jt * 64 + 63 >= row0 - s.window + 1) f |= 2;
      }
      const unsigned bal = __ballot_sync(0xffffffffu, f != 0);
      if (f) {
        const int pos = count + __popc(bal & ((1u << lane) - 1u));
        list[pos] = (uint16_t)jt;
        lflags[pos] = (uint8_t)f;
      }
      count += __popc(bal);
    }
    if (lane == 0) *nvis_out = count;
  }
}

// ------------------------------------------------------------------------------- forward
template <int D>
__global__ void __launch_bounds__(kThreads, 2) fwd_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, Shape s, const float *__restrict__ gate,
    const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ idx,
    __nv_bfloat16 *__restrict__ out, __nv_bfloat16 *__restrict__ out_lt,
    __nv_bfloat16 *__restrict__ out_st, float *__restrict__ lse, int32_t *__restrict__ status,
    int nT) {
  using C = Cfg<D>;
  constexpr int STAGES = 3;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[STAGES + 5];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int nvis_s;
  __shared__ float2 xch[2][2][128];  // [tile parity][column half][row]: half-row maxima (lt, st)
  __shared__ float2 xl[2][128];      // [column half][row]: half-row sums for the epilogue

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nST = (s.L + 127) >> 7;
  const int st = nST - 1 - (int)(blockIdx.x % nST);  // long rows first
  const int u = blockIdx.x / nST, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int row0 = st * 128;

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *q_tile = tiles;
  uint8_t *kv_tiles = q_tile + C::kBigBytes;  // [stage][K, V]
  uint8_t *pl_tile = kv_tiles + STAGES * 2 * C::kSmallBytes;
  uint8_t *ps_tile = pl_tile + C::kPBytes;
  uint8_t *meta = ps_tile + C::kPBytes;
  uint32_t *selw = reinterpret_cast<uint32_t *>(meta);
  uint8_t *selb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ((8 * nT + 15) / 16) * 16);
  uint8_t *lflags = reinterpret_cast<uint8_t *>(list + nT);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;  // an earlier CTA timed out: do not wait again
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
  }
  const Pipe pb = pipe_setup<STAGES>(bars, tid);
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), 256);
    tmem_relinquish();
  }
  build_query_major_list(s, idx, u, st, pad0, nT, selw, selb, list, lflags, &nvis_s);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const int nvis = nvis_s;
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_ol = tmem_base + 64, tmem_os = tmem_base + 128;

  if (warp == kComputeWarps) {
    // ================================ producer ================================
    if (lane == 0 && nvis > 0) {
      constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
      constexpr uint32_t idesc_pv = instr_desc(128, D, 0, 1);
      auto load_stage = [&](int j) {
        const int sj = j % STAGES;
        const uint32_t bar = pb.full0 + 8 * sj;
        uint8_t *kt = kv_tiles + sj * 2 * C::kSmallBytes;
        mbar_expect_tx(bar, 2 * C::kSmallBytes);
        tma_load_4d(smem_u32(kt), &tmk, bar, 0, (int)list[j] * 64, h, n);
        tma_load_4d(smem_u32(kt + C::kSmallBytes), &tmv, bar, 0, (int)list[j] * 64, h, n);
      };
      auto second_stage = [&](int j, int &accL, int &accS) {  // O += P V of tile j
        const int f = lflags[j];
        uint8_t *v_tile = kv_tiles + (j % STAGES) * 2 * C::kSmallBytes + C::kSmallBytes;
        const uint64_t dv = smem_desc(smem_u32(v_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
        if (f & 1) {
          const uint64_t dp = smem_desc(smem_u32(pl_tile), 16, 1024, 2u);
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_bf16(tmem_ol, dp + 2 * k, dv + k * C::kKStep, idesc_pv, (accL | k) != 0);
          accL = 1;
        }
        if (f & 2) {
          const uint64_t dp = smem_desc(smem_u32(ps_tile), 16, 1024, 2u);
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_bf16(tmem_os, dp + 2 * k, dv + k * C::kKStep, idesc_pv, (accS | k) != 0);
          accS = 1;
        }
        umma_commit(pb.mma_done);
      };
      mbar_expect_tx(pb.res, C::kBigBytes);
      tma_load_4d(smem_u32(q_tile), &tmq, pb.res, 0, row0, h, n);
      for (int j = 0; j < min(STAGES, nvis); ++j) load_stage(j);
      int accL = 0, accS = 0;
      const uint64_t dq = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      for (int i = 0; i < nvis; ++i) {
        if (i == 0) mbar_wait(pb.res, 0, &abort_flag);
        mbar_wait(pb.full0 + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag);
        if (i >= 1) mbar_wait(pb.s_empty, (i - 1) & 1, &abort_flag);
        tc_fence_after();
        uint8_t *k_tile = kv_tiles + (i % STAGES) * 2 * C::kSmallBytes;
        const uint64_t dk = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_s, dq + 2 * k, dk + 2 * k, idesc_s, k > 0);
        umma_commit(pb.s_full);
        if (i >= 1) {
          mbar_wait(pb.t_full, (i - 1) & 1, &abort_flag);
          tc_fence_after();
          second_stage(i - 1, accL, accS);
          mbar_wait(pb.mma_done, (i - 1) & 1, &abort_flag);
          if (i - 1 + STAGES < nvis) load_stage(i - 1 + STAGES);
        }
      }
      mbar_wait(pb.t_full, (nvis - 1) & 1, &abort_flag);
      tc_fence_after();
      second_stage(nvis - 1, accL, accS);
    }
  } else {
    // ================================ compute =================================
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane, t = row0 + r, g = r / s.Bk;
    const bool row_ok = t < s.L;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    float mL = -INFINITY, lL = 0.f, mS = -INFINITY, lS = 0.f;
    bool zeroL = false, zeroS = false;
    int accL = 0, accS = 0;
    const float sc2 = s.scale * kLog2e;

    for (int i = 0; i < nvis; ++i) {
      const int jt = list[i], f = lflags[i], p0 = jt * 64;
      uint64_t maskL = 0ull, maskS = 0ull;
      if (row_ok) {
        const uint64_t mc = cols_le(t - p0) & cols_ge(pad0 - p0);
        if (f & 1) maskL = mc & expand_block_bits(selb[g * nT + jt], s.Bk);
        if (f & 2) maskS = mc & cols_ge(t - s.window + 1 - p0);
      }
      // identical in the two warps that share these 32 rows
      const bool pair_any = __any_sync(0xffffffffu, (maskL | maskS) != 0ull);
      const uint32_t hL = (uint32_t)(maskL >> (half * 32)), hS = (uint32_t)(maskS >> (half * 32));

      mbar_wait(pb.s_full, i & 1, &abort_flag);
      __syncwarp();
      tc_fence_after();
      float sv[32];
      if (pair_any) {
        tmem_ld32(tmem_s + lane_off + half * 32, sv);
        tmem_wait_ld();
      }
      tc_fence_before();
      warp_arrive(pb.s_empty, lane);

      uint32_t pL[16], pS[16];
      float facL = 1.f, facS = 1.f;
      bool needL = false, needS = false;
      if (pair_any) {
        float mtL = -INFINITY, mtS = -INFINITY;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          if ((hL >> c) & 1u) mtL = fmaxf(mtL, sv[c]);
          if ((hS >> c) & 1u) mtS = fmaxf(mtS, sv[c]);
        }
        xch[i & 1][half][r] = make_float2(mtL, mtS);
        named_bar_sync(1 + quarter, 64);
        const float2 o = xch[i & 1][half ^ 1][r];
        mtL = fmaxf(mtL, o.x) * sc2;
        mtS = fmaxf(mtS, o.y) * sc2;
        needL = mtL > mL + kRescaleThreshold;  // also true on the row's first keys
        needS = mtS > mS + kRescaleThreshold;
        if (needL) { facL = exp2f(mL - mtL); lL *= facL; mL = mtL; }
        if (needS) { facS = exp2f(mS - mtS); lS *= facS; mS = mtS; }
        if ((f & 1) && __any_sync(0xffffffffu, hL != 0u)) {
          const float nm = -mL;
          float acc = 0.f;
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float a = ((hL >> c) & 1u) ? exp2f(fmaf(sv[c], sc2, nm)) : 0.f;
            const float b = ((hL >> (c + 1)) & 1u) ? exp2f(fmaf(sv[c + 1], sc2, nm)) : 0.f;
            acc += a + b;
            pL[c >> 1] = pack_bf16(a, b);
          }
          lL += acc;
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) pL[c] = 0u;
        }
        if ((f & 2) && __any_sync(0xffffffffu, hS != 0u)) {
          const float nm = -mS;
          float acc = 0.f;
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float a = ((hS >> c) & 1u) ? exp2f(fmaf(sv[c], sc2, nm)) : 0.f;
            const float b = ((hS >> (c + 1)) & 1u) ? exp2f(fmaf(sv[c + 1], sc2, nm)) : 0.f;
            acc += a + b;
            pS[c >> 1] = pack_bf16(a, b);
          }
          lS += acc;
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) pS[c] = 0u;
        }
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c) { pL[c] = 0u; pS[c] = 0u; }
      }

      // the P tiles and the accumulators are free once the MMAs of tile i-1 have completed
      if (i >= 1) {
        mbar_wait(pb.mma_done, (i - 1) & 1, &abort_flag);
        __syncwarp();
        tc_fence_after();
      }
      if (pair_any) {
        if (accL && __any_sync(0xffffffffu, needL)) {
          float o[C::OC];
          tmem_ld<C::OC>(tmem_ol + lane_off + half * C::OC, o);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < C::OC; ++c) o[c] *= facL;
          tmem_st<C::OC>(tmem_ol + lane_off + half * C::OC, o);
          tmem_wait_st();
        }
        if (accS && __any_sync(0xffffffffu, needS)) {
          float o[C::OC];
          tmem_ld<C::OC>(tmem_os + lane_off + half * C::OC, o);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < C::OC; ++c) o[c] *= facS;
          tmem_st<C::OC>(tmem_os + lane_off + half * C::OC, o);
          tmem_wait_st();
        }
      }
      if ((f & 1) && (hL != 0u || !zeroL)) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
          store_row_sw128(pl_tile, r, half * 4 + ch,
                          make_uint4(pL[ch * 4], pL[ch * 4 + 1], pL[ch * 4 + 2], pL[ch * 4 + 3]));
        zeroL = hL == 0u;
      }
      if ((f & 2) && (hS != 0u || !zeroS)) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
          store_row_sw128(ps_tile, r, half * 4 + ch,
                          make_uint4(pS[ch * 4], pS[ch * 4 + 1], pS[ch * 4 + 2], pS[ch * 4 + 3]));
        zeroS = hS == 0u;
      }
      fence_async_smem();
      tc_fence_before();
      warp_arrive(pb.t_full, lane);
      accL |= (f & 1);
      accS |= (f & 2);
    }

    // ---- epilogue ----
    if (nvis > 0) {
      mbar_wait(pb.mma_done, (nvis - 1) & 1, &abort_flag);
      __syncwarp();
      tc_fence_after();
    }
    xl[half][r] = make_float2(lL, lS);
    named_bar_sync(1 + quarter, 64);
    {
      const float2 o = xl[half ^ 1][r];
      lL += o.x;
      lS += o.y;
    }
    const float alpha = gate_alpha(gate, h), beta = 1.f - alpha;
    const float iL = lL > 0.f ? 1.f / lL : 0.f, iS = lS > 0.f ? 1.f / lS : 0.f;
    const bool haveL = accL && lL > 0.f, haveS = accS && lS > 0.f;
    const int64_t ro = row_offset(s, n, h, row_ok ? t : 0) + half * C::OC;
    float oL[C::OC], oS[C::OC];
    if (accL) tmem_ld<C::OC>(tmem_ol + lane_off + half * C::OC, oL);  // accL / accS are CTA-uniform
    if (accS) tmem_ld<C::OC>(tmem_os + lane_off + half * C::OC, oS);
    tmem_wait_ld();
    if (row_ok) {
#pragma unroll
      for (int ch = 0; ch < C::OC / 8; ++ch) {
        uint32_t wo[4], wl[4], ws[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          const float a0 = haveL ? oL[c] * iL : 0.f, a1 = haveL ? oL[c + 1] * iL : 0.f;
          const float b0 = haveS ? oS[c] * iS : 0.f, b1 = haveS ? oS[c + 1] * iS : 0.f;
          wl[e] = pack_bf16(a0, a1);
          ws[e] = pack_bf16(b0, b1);
          wo[e] = pack_bf16(alpha * a0 + beta * b0, alpha * a1 + beta * b1);
        }
        const int64_t off = ro + ch * 8;
        *reinterpret_cast<uint4 *>(out + off) = make_uint4(wo[0], wo[1], wo[2], wo[3]);
        if (out_lt) *reinterpret_cast<uint4 *>(out_lt + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
        if (out_st) *reinterpret_cast<uint4 *>(out_st + off) = make_uint4(ws[0], ws[1], ws[2], ws[3]);
      }
      if (half == 0 && lse) {
        const int64_t BHL = (int64_t)s.B * s.H * s.L;
        lse[(int64_t)u * s.L + t] = lL > 0.f ? (mL + log2f(lL)) * kLn2 : 0.f;
        lse[BHL + (int64_t)u * s.L + t] = lS > 0.f ? (mS + log2f(lS)) * kLn2 : 0.f;
      }
    }
  }
  finish(warp, tmem_base, &abort_flag, status);
}

// ---------------------------------------------------------------------------- backward dQ
template <int D>
__global__ void __launch_bounds__(kThreads, 2) bwd_dq_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmg, Shape s,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, const __nv_bfloat16 *__restrict__ out_lt,
    const __nv_bfloat16 *__restrict__ out_st, const float *__restrict__ lse,
    const __nv_bfloat16 *__restrict__ dout, __nv_bfloat16 *__restrict__ dq,
    float *__restrict__ delta, double *__restrict__ dalpha_part, int32_t *__restrict__ status,
    int nT) {
  using C = Cfg<D>;
  constexpr int STAGES = 3;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[STAGES + 5];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int nvis_s;
  __shared__ double red[256];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nST = (s.L + 127) >> 7;
  const int st = nST - 1 - (int)(blockIdx.x % nST);
  const int u = blockIdx.x / nST, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int row0 = st * 128;
  const int G = 128 / s.Bk;

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *q_tile = tiles;
  uint8_t *g_tile = q_tile + C::kBigBytes;
  uint8_t *kv_tiles = g_tile + C::kBigBytes;
  uint8_t *ds_tile = kv_tiles + STAGES * 2 * C::kSmallBytes;
  uint8_t *meta = ds_tile + C::kPBytes;
  uint32_t *selw = reinterpret_cast<uint32_t *>(meta);
  uint8_t *selb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ((8 * nT + 15) / 16) * 16);
  uint8_t *lflags = reinterpret_cast<uint8_t *>(list + nT);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
    tma_prefetch_desc(&tmg);
  }
  const Pipe pb = pipe_setup<STAGES>(bars, tid);
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), 256);
    tmem_relinquish();
  }
  build_query_major_list(s, idx, u, st, pad0, nT, selw, selb, list, lflags, &nvis_s);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const int nvis = nvis_s;
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_dp = tmem_base + 64, tmem_dq = tmem_base + 128;

  if (warp == kComputeWarps) {
    if (lane == 0 && nvis > 0) {
      constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
      constexpr uint32_t idesc_dq = instr_desc(128, D, 0, 1);
      auto load_stage = [&](int j) {
        const int sj = j % STAGES;
        const uint32_t bar = pb.full0 + 8 * sj;
        uint8_t *kt = kv_tiles + sj * 2 * C::kSmallBytes;
        mbar_expect_tx(bar, 2 * C::kSmallBytes);
        tma_load_4d(smem_u32(kt), &tmk, bar, 0, (int)list[j] * 64, h, n);
        tma_load_4d(smem_u32(kt + C::kSmallBytes), &tmv, bar, 0, (int)list[j] * 64, h, n);
      };
      int acc = 0;
      auto second_stage = [&](int j) {  // dQ += dS K of tile j (K read MN-major)
        uint8_t *k_tile = kv_tiles + (j % STAGES) * 2 * C::kSmallBytes;
        const uint64_t dsd = smem_desc(smem_u32(ds_tile), 16, 1024, 2u);
        const uint64_t dkm = smem_desc(smem_u32(k_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_bf16(tmem_dq, dsd + 2 * k, dkm + k * C::kKStep, idesc_dq, (acc | k) != 0);
        acc = 1;
        umma_commit(pb.mma_done);
      };
      mbar_expect_tx(pb.res, 2 * C::kBigBytes);
      tma_load_4d(smem_u32(q_tile), &tmq, pb.res, 0, row0, h, n);
      tma_load_4d(smem_u32(g_tile), &tmg, pb.res, 0, row0, h, n);
      for (int j = 0; j < min(STAGES, nvis); ++j) load_stage(j);
      const uint64_t dqd = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dgd = smem_desc(smem_u32(g_tile), 16, C::kAtomBytes, C::kSwizzle);
      for (int i = 0; i < nvis; ++i) {
        if (i == 0) mbar_wait(pb.res, 0, &abort_flag);
        mbar_wait(pb.full0 + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag);
        if (i >= 1) mbar_wait(pb.s_empty, (i - 1) & 1, &abort_flag);
        tc_fence_after();
        uint8_t *k_tile = kv_tiles + (i % STAGES) * 2 * C::kSmallBytes, *v_tile = k_tile + C::kSmallBytes;
        const uint64_t dkd = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
        const uint64_t dvd = smem_desc(smem_u32(v_tile), 16, C::kAtomBytes, C::kSwizzle);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_s, dqd + 2 * k, dkd + 2 * k, idesc_s, k > 0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_dp, dgd + 2 * k, dvd + 2 * k, idesc_s, k > 0);
        umma_commit(pb.s_full);
        if (i >= 1) {
          mbar_wait(pb.t_full, (i - 1) & 1, &abort_flag);
          tc_fence_after();
          second_stage(i - 1);
          mbar_wait(pb.mma_done, (i - 1) & 1, &abort_flag);
          if (i - 1 + STAGES < nvis) load_stage(i - 1 + STAGES);
        }
      }
      mbar_wait(pb.t_full, (nvis - 1) & 1, &abort_flag);
      tc_fence_after();
      second_stage(nvis - 1);
    }
  } else {
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane, t = row0 + r, g = r / s.Bk;
    const bool row_ok = t < s.L, row_valid = row_ok && t >= pad0;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float alpha = gate_alpha(gate, h), beta = 1.f - alpha;
    const int64_t BHL = (int64_t)s.B * s.H * s.L;
    const int64_t ro = row_offset(s, n, h, row_ok ? t : 0);
    // delta of both branches and the saved log-sum-exps of this row (both threads of the row)
    float deltaL = 0.f, deltaS = 0.f, lseL2 = 0.f, lseS2 = 0.f;
    if (row_valid) {
      float aL = 0.f, aS = 0.f;
#pragma unroll
      for (int c = 0; c < D; c += 8) {
        const uint4 gv = *reinterpret_cast<const uint4 *>(dout + ro + c);
        const uint4 lv = *reinterpret_cast<const uint4 *>(out_lt + ro + c);
        const uint4 sv4 = *reinterpret_cast<const uint4 *>(out_st + ro + c);
        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, lw[4] = {lv.x, lv.y, lv.z, lv.w},
                       sw[4] = {sv4.x, sv4.y, sv4.z, sv4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float g0 = __uint_as_float(gw[e] << 16), g1 = __uint_as_float(gw[e] & 0xffff0000u);
          aL = fmaf(g0, __uint_as_float(lw[e] << 16), aL);
          aL = fmaf(g1, __uint_as_float(lw[e] & 0xffff0000u), aL);
          aS = fmaf(g0, __uint_as_float(sw[e] << 16), aS);
          aS = fmaf(g1, __uint_as_float(sw[e] & 0xffff0000u), aS);
        }
      }
      deltaL = alpha * aL;
      deltaS = beta * aS;
      lseL2 = lse[(int64_t)u * s.L + t] * kLog2e;
      lseS2 = lse[BHL + (int64_t)u * s.L + t] * kLog2e;
    }
    if (row_ok && half == 0) {
      delta[(int64_t)u * s.L + t] = deltaL;
      delta[BHL + (int64_t)u * s.L + t] = deltaS;
    }
    float dal = 0.f;
    bool ds_zero = false;
    const float sc2 = s.scale * kLog2e;

    for (int i = 0; i < nvis; ++i) {
      const int jt = list[i], f = lflags[i], p0 = jt * 64;
      uint64_t maskL = 0ull, maskS = 0ull;
      if (row_valid) {
        const uint64_t mc = cols_le(t - p0) & cols_ge(pad0 - p0);
        if (f & 1) maskL = mc & expand_block_bits(selb[g * nT + jt], s.Bk);
        if (f & 2) maskS = mc & cols_ge(t - s.window + 1 - p0);
      }
      const uint32_t hL = (uint32_t)(maskL >> (half * 32)), hS = (uint32_t)(maskS >> (half * 32));
      const bool anyL = __any_sync(0xffffffffu, hL != 0u), anyS = __any_sync(0xffffffffu, hS != 0u);

      mbar_wait(pb.s_full, i & 1, &abort_flag);
      __syncwarp();
      tc_fence_after();
      float sv[32], dp[32];
      if (anyL || anyS) {
        tmem_ld32(tmem_s + lane_off + half * 32, sv);
        tmem_ld32(tmem_dp + lane_off + half * 32, dp);
        tmem_wait_ld();
      }
      tc_fence_before();
      warp_arrive(pb.s_empty, lane);

      uint32_t dw[16];
      if (anyL || anyS) {
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float d[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float x = sv[c + e] * sc2, dpv = dp[c + e];
            float acc = 0.f;
            if (anyL) {
              const float pLv = ((hL >> (c + e)) & 1u) ? exp2f(x - lseL2) : 0.f;
              acc = pLv * fmaf(alpha, dpv, -deltaL);
              dal = fmaf(pLv, dpv, dal);
            }
            if (anyS) {
              const float pSv = ((hS >> (c + e)) & 1u) ? exp2f(x - lseS2) : 0.f;
              acc = fmaf(pSv, fmaf(beta, dpv, -deltaS), acc);
              dal = fmaf(-pSv, dpv, dal);
            }
            d[e] = acc;
          }
          dw[c >> 1] = pack_bf16(d[0], d[1]);
        }
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c) dw[c] = 0u;
      }
      if (i >= 1) {
        mbar_wait(pb.mma_done, (i - 1) & 1, &abort_flag);
        __syncwarp();
      }
      const bool mine = (hL | hS) != 0u;
      if (mine || !ds_zero) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
          store_row_sw128(ds_tile, r, half * 4 + ch,
                          make_uint4(dw[ch * 4], dw[ch * 4 + 1], dw[ch * 4 + 2], dw[ch * 4 + 3]));
        ds_zero = !mine;
      }
      fence_async_smem();
      warp_arrive(pb.t_full, lane);
    }

    if (nvis > 0) {
      mbar_wait(pb.mma_done, (nvis - 1) & 1, &abort_flag);
      __syncwarp();
      tc_fence_after();
    }
    float o[C::OC];
    if (nvis > 0) {
      tmem_ld<C::OC>(tmem_dq + lane_off + half * C::OC, o);
      tmem_wait_ld();
    }
    if (row_ok) {
      const bool live = nvis > 0 && row_valid;
#pragma unroll
      for (int ch = 0; ch < C::OC / 8; ++ch) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          w[e] = live ? pack_bf16(o[c] * s.scale, o[c + 1] * s.scale) : 0u;
        }
        *reinterpret_cast<uint4 *>(dq + ro + half * C::OC + ch * 8) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
    red[tid] = row_valid ? (double)dal : 0.0;
  }
  tc_fence_before();
  __syncthreads();
  // d alpha partial of this CTA -> first query-block slot of the super-tile, zeros in the rest
  if (tid == 0) {
    double a = 0.0;
    for (int i = 0; i < 256; ++i) a += red[i];  // fixed order
    for (int gq = 0; gq < G; ++gq)
      if (st * G + gq < s.M) dalpha_part[(int64_t)u * s.M + st * G + gq] = gq == 0 ? a : 0.0;
  }
  finish(warp, tmem_base, &abort_flag, status);
}

// ------------------------------------------------------------------------- backward dK, dV
template <int D>
__global__ void __launch_bounds__(kThreads, 2) bwd_dkdv_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmg, Shape s,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, const float *__restrict__ lse,
    const float *__restrict__ delta, __nv_bfloat16 *__restrict__ dk, __nv_bfloat16 *__restrict__ dv,
    int32_t *__restrict__ status, int nT) {
  using C = Cfg<D>;
  constexpr int STAGES = 2;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[STAGES + 5];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int nvis_s;
  // per query column of the current tile: lse_lt*log2e, lse_st*log2e, delta_lt, delta_st
  __shared__ __align__(16) float stats[2][64][4];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nKT = (s.L + 127) >> 7;
  const int kt = (int)(blockIdx.x % nKT);  // early keys have the most visitors: first
  const int u = blockIdx.x / nKT, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int key0 = kt * 128, key_last = min(s.L - 1, key0 + 127);
  const int G = 128 / s.Bk, nb = 64 / s.Bk;

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *k_tile = tiles;
  uint8_t *v_tile = k_tile + C::kBigBytes;
  uint8_t *qg_tiles = v_tile + C::kBigBytes;  // [stage][Q, dO]
  uint8_t *w_tile = qg_tiles + STAGES * 2 * C::kSmallBytes;
  uint8_t *ds_tile = w_tile + C::kPBytes;
  uint8_t *meta = ds_tile + C::kPBytes;
  uint32_t *invw = reinterpret_cast<uint32_t *>(meta);  // [8][nT] bytes: per key block, per query tile
  uint8_t *invb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ((8 * nT + 15) / 16) * 16);
  uint8_t *lflags = reinterpret_cast<uint8_t *>(list + nT);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
    tma_prefetch_desc(&tmg);
  }
  const Pipe pb = pipe_setup<STAGES>(bars, tid);
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), 256);
    tmem_relinquish();
  }
  for (int i = tid; i < (8 * nT + 3) / 4; i += kThreads) invw[i] = 0u;
  __syncthreads();
  {  // which query blocks selected each of this CTA's key blocks, per 64-query tile
    const int qb0 = kt * G, nq = s.M - qb0;
    for (int i = tid; i < nq * s.topk; i += kThreads) {
      const int qb = qb0 + i / s.topk;
      const int blk = idx[((int64_t)u * s.M + qb) * s.topk + (i % s.topk)];
      if (blk >= qb0 && blk < qb0 + G && blk <= qb) {
        const int a = (blk - qb0) * nT + qb / nb;
        atomicOr(&invw[a >> 2], (1u << (qb % nb)) << ((a & 3) * 8));
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    const int qt_min = key0 >> 6, qt_max = (s.L - 1) >> 6;
    int count = 0;
    for (int base = qt_min; base <= qt_max; base += 32) {
      const int qt = base + lane;
      int f = 0;
      if (qt <= qt_max && key_last >= pad0) {
        for (int g = 0; g < G; ++g) f |= invb[g * nT + qt] ? 1 : 0;
        if (qt * 64 <= key_last + s.window - 1) f |= 2;
      }
      const unsigned bal = __ballot_sync(0xffffffffu, f != 0);
      if (f) {
        const int pos = count + __popc(bal & ((1u << lane) - 1u));
        list[pos] = (uint16_t)qt;
        lflags[pos] = (uint8_t)f;
      }
      count += __popc(bal);
    }
    if (lane == 0) nvis_s = count;
  }
  __syncthreads();
  const int nvis = nvis_s;
  const int64_t BHL = (int64_t)s.B * s.H * s.L;
  // one statistic per compute thread: column tid & 63, kind tid >> 6
  auto load_stat = [&](int qt) -> float {
    const int tq = qt * 64 + (tid & 63), kind = tid >> 6;
    if (tq >= s.L) return 0.f;
    if (kind == 0) return lse[(int64_t)u * s.L + tq] * kLog2e;
    if (kind == 1) return lse[BHL + (int64_t)u * s.L + tq] * kLog2e;
    if (kind == 2) return delta[(int64_t)u * s.L + tq];
    return delta[BHL + (int64_t)u * s.L + tq];
  };
  if (tid < 256 && nvis > 0) stats[0][tid & 63][tid >> 6] = load_stat(list[0]);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_dp = tmem_base + 64, tmem_dv = tmem_base + 128,
                 tmem_dk = tmem_base + 192;

  if (warp == kComputeWarps) {
    if (lane == 0 && nvis > 0) {
      constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
      constexpr uint32_t idesc_o = instr_desc(128, D, 0, 1);
      auto load_stage = [&](int j) {
        const int sj = j % STAGES;
        const uint32_t bar = pb.full0 + 8 * sj;
        uint8_t *qt_ = qg_tiles + sj * 2 * C::kSmallBytes;
        mbar_expect_tx(bar, 2 * C::kSmallBytes);
        tma_load_4d(smem_u32(qt_), &tmq, bar, 0, (int)list[j] * 64, h, n);
        tma_load_4d(smem_u32(qt_ + C::kSmallBytes), &tmg, bar, 0, (int)list[j] * 64, h, n);
      };
      int acc = 0;
      auto second_stage = [&](int j) {  // dV += W^T dO, dK += dS^T Q of tile j
        uint8_t *q_tile = qg_tiles + (j % STAGES) * 2 * C::kSmallBytes, *g_tile = q_tile + C::kSmallBytes;
        const uint64_t dwd = smem_desc(smem_u32(w_tile), 16, 1024, 2u);
        const uint64_t dsd = smem_desc(smem_u32(ds_tile), 16, 1024, 2u);
        const uint64_t dgm = smem_desc(smem_u32(g_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
        const uint64_t dqm = smem_desc(smem_u32(q_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_bf16(tmem_dv, dwd + 2 * k, dgm + k * C::kKStep, idesc_o, (acc | k) != 0);
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_bf16(tmem_dk, dsd + 2 * k, dqm + k * C::kKStep, idesc_o, (acc | k) != 0);
        acc = 1;
        umma_commit(pb.mma_done);
      };
      mbar_expect_tx(pb.res, 2 * C::kBigBytes);
      tma_load_4d(smem_u32(k_tile), &tmk, pb.res, 0, key0, h, n);
      tma_load_4d(smem_u32(v_tile), &tmv, pb.res, 0, key0, h, n);
      for (int j = 0; j < min(STAGES, nvis); ++j) load_stage(j);
      const uint64_t dkd = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dvd = smem_desc(smem_u32(v_tile), 16, C::kAtomBytes, C::kSwizzle);
      for (int i = 0; i < nvis; ++i) {
        if (i == 0) mbar_wait(pb.res, 0, &abort_flag);
        mbar_wait(pb.full0 + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag);
        if (i >= 1) mbar_wait(pb.s_empty, (i - 1) & 1, &abort_flag);
        tc_fence_after();
        uint8_t *q_tile = qg_tiles + (i % STAGES) * 2 * C::kSmallBytes, *g_tile = q_tile + C::kSmallBytes;
        const uint64_t dqd = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
        const uint64_t dgd = smem_desc(smem_u32(g_tile), 16, C::kAtomBytes, C::kSwizzle);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_s, dkd + 2 * k, dqd + 2 * k, idesc_s, k > 0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_dp, dvd + 2 * k, dgd + 2 * k, idesc_s, k > 0);
        umma_commit(pb.s_full);
        if (i >= 1) {
          mbar_wait(pb.t_full, (i - 1) & 1, &abort_flag);
          tc_fence_after();
          second_stage(i - 1);
          mbar_wait(pb.mma_done, (i - 1) & 1, &abort_flag);
          if (i - 1 + STAGES < nvis) load_stage(i - 1 + STAGES);
        }
      }
      mbar_wait(pb.t_full, (nvis - 1) & 1, &abort_flag);
      tc_fence_after();
      second_stage(nvis - 1);
    }
  } else {
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane, p = key0 + r, g = r / s.Bk;
    const bool row_ok = p < s.L, row_valid = row_ok && p >= pad0;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float alpha = gate_alpha(gate, h), beta = 1.f - alpha;
    bool w_zero = false;
    const float sc2 = s.scale * kLog2e;

    for (int i = 0; i < nvis; ++i) {
      const int qt = list[i], f = lflags[i], t0 = qt * 64;
      uint64_t maskL = 0ull, maskS = 0ull;
      if (row_valid) {
        const uint64_t mc = cols_ge(p - t0) & cols_le(s.L - 1 - t0);
        if (f & 1) maskL = mc & expand_block_bits(invb[g * nT + qt], s.Bk);
        if (f & 2) maskS = mc & cols_le(p + s.window - 1 - t0);
      }
      const uint32_t hL = (uint32_t)(maskL >> (half * 32)), hS = (uint32_t)(maskS >> (half * 32));
      const bool anyL = __any_sync(0xffffffffu, hL != 0u), anyS = __any_sync(0xffffffffu, hS != 0u);

      // every compute warp has finished tile i-1 (incl. its reads of stats and its stores of the
      // next statistics) once t_full(i-1) completes
      if (i >= 1) mbar_wait(pb.t_full, (i - 1) & 1, &abort_flag);
      mbar_wait(pb.s_full, i & 1, &abort_flag);
      __syncwarp();
      tc_fence_after();
      float sv[32], dp[32];
      if (anyL || anyS) {
        tmem_ld32(tmem_s + lane_off + half * 32, sv);
        tmem_ld32(tmem_dp + lane_off + half * 32, dp);
        tmem_wait_ld();
      }
      tc_fence_before();
      warp_arrive(pb.s_empty, lane);
      const bool have_next = i + 1 < nvis;
      float next_stat = 0.f;
      if (have_next) next_stat = load_stat(list[i + 1]);

      uint32_t ww[16], dw[16];
      if (anyL || anyS) {
        const float4 *stt = reinterpret_cast<const float4 *>(&stats[i & 1][half * 32][0]);
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float wv[2], d[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float4 q4 = stt[c + e];
            const float x = sv[c + e] * sc2, dpv = dp[c + e];
            float wa = 0.f, da = 0.f;
            if (anyL) {
              const float pLv = ((hL >> (c + e)) & 1u) ? exp2f(x - q4.x) : 0.f;
              wa = alpha * pLv;
              da = pLv * fmaf(alpha, dpv, -q4.z);
            }
            if (anyS) {
              const float pSv = ((hS >> (c + e)) & 1u) ? exp2f(x - q4.y) : 0.f;
              wa = fmaf(beta, pSv, wa);
              da = fmaf(pSv, fmaf(beta, dpv, -q4.w), da);
            }
            wv[e] = wa;
            d[e] = da;
          }
          ww[c >> 1] = pack_bf16(wv[0], wv[1]);
          dw[c >> 1] = pack_bf16(d[0], d[1]);
        }
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c) { ww[c] = 0u; dw[c] = 0u; }
      }
      if (i >= 1) {
        mbar_wait(pb.mma_done, (i - 1) & 1, &abort_flag);
        __syncwarp();
      }
      const bool mine = (hL | hS) != 0u;
      if (mine || !w_zero) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          store_row_sw128(w_tile, r, half * 4 + ch,
                          make_uint4(ww[ch * 4], ww[ch * 4 + 1], ww[ch * 4 + 2], ww[ch * 4 + 3]));
          store_row_sw128(ds_tile, r, half * 4 + ch,
                          make_uint4(dw[ch * 4], dw[ch * 4 + 1], dw[ch * 4 + 2], dw[ch * 4 + 3]));
        }
        w_zero = !mine;
      }
      if (have_next) stats[(i + 1) & 1][tid & 63][tid >> 6] = next_stat;
      fence_async_smem();
      warp_arrive(pb.t_full, lane);
    }

    if (nvis > 0) {
      mbar_wait(pb.mma_done, (nvis - 1) & 1, &abort_flag);
      __syncwarp();
      tc_fence_after();
    }
    float ov[C::OC], okk[C::OC];
    if (nvis > 0) {
      tmem_ld<C::OC>(tmem_dv + lane_off + half * C::OC, ov);
      tmem_ld<C::OC>(tmem_dk + lane_off + half * C::OC, okk);
      tmem_wait_ld();
    }
    if (row_ok) {
      const bool live = nvis > 0 && row_valid;
      const int64_t ro = row_offset(s, n, h, p) + half * C::OC;
#pragma unroll
      for (int ch = 0; ch < C::OC / 8; ++ch) {
        uint32_t wv[4], wk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          wv[e] = live ? pack_bf16(ov[c], ov[c + 1]) : 0u;
          wk[e] = live ? pack_bf16(okk[c] * s.scale, okk[c + 1] * s.scale) : 0u;
        }
        *reinterpret_cast<uint4 *>(dv + ro + ch * 8) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        *reinterpret_cast<uint4 *>(dk + ro + ch * 8) = make_uint4(wk[0], wk[1], wk[2], wk[3]);
      }
    }
  }
  finish(warp, tmem_base, &abort_flag, status);
}

// ------------------------------------------------------------------------------- launchers
template <int D>
int launch_fwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt,
                    void *out_st, float *lse, const Workspace &ws, cudaStream_t st) {
  using C = Cfg<D>;
  CUtensorMap tq, tk, tv;
  if (make_tensor_map(&tq, q, s, 128) || make_tensor_map(&tk, k, s, 64) || make_tensor_map(&tv, v, s, 64))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const size_t smem = 1024 + C::kBigBytes + 3 * 2 * C::kSmallBytes + 2 * C::kPBytes + meta_bytes(nT);
  if (cudaFuncSetAttribute(fwd_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  const unsigned grid = (unsigned)nST * (unsigned)(s.B * s.H);
  {
    LaunchScope ls(K_FWD_TC, st);
    fwd_tc_kernel<D><<<grid, kThreads, smem, st>>>(tq, tk, tv, s, gate, seq_lens, idx, (__nv_bfloat16 *)out,
                                                  (__nv_bfloat16 *)out_lt, (__nv_bfloat16 *)out_st, lse,
                                                  ws.status, nT);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

template <int D>
int launch_bwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, const void *out_lt,
                    const void *out_st, const float *lse, const void *dout, void *dq, void *dk,
                    void *dv, const Workspace &ws, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  using C = Cfg<D>;
  CUtensorMap q128, k64, v64, g128, q64, k128, v128, g64;
  if (make_tensor_map(&q128, q, s, 128) || make_tensor_map(&k64, k, s, 64) ||
      make_tensor_map(&v64, v, s, 64) || make_tensor_map(&g128, dout, s, 128) ||
      make_tensor_map(&q64, q, s, 64) || make_tensor_map(&k128, k, s, 128) ||
      make_tensor_map(&v128, v, s, 128) || make_tensor_map(&g64, dout, s, 64))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const unsigned grid = (unsigned)nST * (unsigned)(s.B * s.H);
  const size_t smem_dq = 1024 + 2 * C::kBigBytes + 3 * 2 * C::kSmallBytes + C::kPBytes + meta_bytes(nT);
  const size_t smem_kv = 1024 + 2 * C::kBigBytes + 2 * 2 * C::kSmallBytes + 2 * C::kPBytes + meta_bytes(nT);
  if (cudaFuncSetAttribute(bwd_dq_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_dq) != cudaSuccess ||
      cudaFuncSetAttribute(bwd_dkdv_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kv) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    LaunchScope ls(K_BWD_DQ_TC, st);
    bwd_dq_tc_kernel<D><<<grid, kThreads, smem_dq, st>>>(q128, k64, v64, g128, s, gate, seq_lens, idx,
                                                        (const bf *)out_lt, (const bf *)out_st, lse,
                                                        (const bf *)dout, (bf *)dq, ws.delta, ws.dalpha,
                                                        ws.status, nT);
  }
  {
    LaunchScope ls(K_BWD_DKDV_TC, st);
    bwd_dkdv_tc_kernel<D><<<grid, kThreads, smem_kv, st>>>(q64, k128, v128, g64, s, gate, seq_lens, idx,
                                                          lse, ws.delta, (bf *)dk, (bf *)dv, ws.status, nT);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

// ---- host: TMA descriptor of a q-shaped bf16 tensor, box = (D, rows, 1, 1) -----------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

int make_tensor_map(CUtensorMap *map, const void *base, const Shape &s, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return 1;
  const cuuint64_t dims[4] = {(cuuint64_t)s.D, (cuuint64_t)s.L, (cuuint64_t)s.H, (cuuint64_t)s.B};
  const cuuint64_t strides[3] = {(cuuint64_t)s.sl * 2, (cuuint64_t)s.sh * 2, (cuuint64_t)s.sb * 2};
  const cuuint32_t box[4] = {(cuuint32_t)s.D, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUtensorMapSwizzle sw = s.D == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
  CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? 0 : 1;
}

bool fwd_tc_supported(const Shape &s, int dtype) {
  return dtype == BLOSSOM_DTYPE_BF16 && (s.D == 32 || s.D == 64) &&
         (s.Bk == 16 || s.Bk == 32 || s.Bk == 64) && (s.L + 63) / 64 <= 1024;
}

int launch_fwd_tc(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                  const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt, void *out_st,
                  float *lse, const Workspace &ws, cudaStream_t st) {
  if (s.D == 32) return launch_fwd_tc_t<32>(s, q, k, v, gate, seq_lens, idx, out, out_lt, out_st, lse, ws, st);
  return launch_fwd_tc_t<64>(s, q, k, v, gate, seq_lens, idx, out, out_lt, out_st, lse, ws, st);
}

int launch_bwd_tc(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                  const int32_t *seq_lens, const int32_t *idx, const void *out_lt, const void *out_st,
                  const float *lse, const void *dout, void *dq, void *dk, void *dv,
                  const Workspace &ws, cudaStream_t st) {
  if (s.D == 32)
    return launch_bwd_tc_t<32>(s, q, k, v, gate, seq_lens, idx, out_lt, out_st, lse, dout, dq, dk, dv, ws, st);
  return launch_bwd_tc_t<64>(s, q, k, v, gate, seq_lens, idx, out_lt, out_st, lse, dout, dq, dk, dv, ws, st);
}

}  // namespace tc
}  // namespace blossom
