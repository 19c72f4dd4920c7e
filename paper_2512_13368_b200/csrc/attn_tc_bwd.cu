// Tensor-core backward of the fused two-branch attention (bf16 storage, fp32 accumulate).
//
// Two kernels, both deterministic (no atomics on the gradients):
//
//  bwd_dq_tc    query-major, the forward's walk: a CTA owns 128 query rows and visits the same
//               64-key tiles.  Per tile S = Q K^T and dP = dO V^T go to TMEM (M = 128, N = 64);
//               thread = query row recomputes both branches' probabilities from the saved
//               log-sum-exps, forms dS = P_lt (alpha dP - delta_lt) + P_st (beta dP - delta_st)
//               (the branches share K, so one dS tile serves both), writes it as bf16 to swizzled
//               shared memory, and dQ += dS K accumulates in TMEM.  The prologue computes
//               delta = rowsum(G_branch o O_branch) for its rows (also stored for the second
//               kernel); d alpha is accumulated as sum (P_lt - P_st) dP in fp32.
//
//  bwd_dkdv_tc  key-major and transposed: a CTA owns 128 keys and visits the 64-query tiles that
//               selected one of its key blocks or whose window reaches them.  S^T = K Q^T and
//               dP^T = V dO^T (M = 128 keys, N = 64 queries); thread = key row; the per-query
//               statistics (lse, delta) come from shared memory; W^T = alpha P_lt + beta P_st and
//               dS^T are written as bf16 tiles, and dV += W^T dO, dK += dS^T Q accumulate in TMEM.
//
// Gradient formulas: softmax-attention chain rule applied to Eq. 16 / 17 / 19 (see blossom.h).
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct Cfg {
  static constexpr int kRowBytes = D * 2;
  static constexpr int kBigBytes = 128 * kRowBytes;   // resident 128-row tile
  static constexpr int kSmallBytes = 64 * kRowBytes;  // streamed 64-row tile
  static constexpr int kPBytes = 128 * 128;           // [128][64] bf16 tile
  static constexpr int kAtomBytes = 8 * kRowBytes;
  static constexpr uint32_t kSwizzle = (D == 64) ? 2u : 4u;
};

constexpr int kDqStages = 3;
constexpr int kKvStages = 2;

__host__ __device__ inline int meta_bytes(int nT) { return ((11 * nT + 15) / 16) * 16 + 16; }

__device__ __forceinline__ float sigmoid_gate(const float *gate, int h) {
  return 1.f / (1.f + __expf(-(gate[h * 2 + 0] - gate[h * 2 + 1])));
}

// ------------------------------------------------------------------------------ dQ kernel
template <int D>
__global__ void __launch_bounds__(128, 2) bwd_dq_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmg, Shape s,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, const __nv_bfloat16 *__restrict__ out_lt,
    const __nv_bfloat16 *__restrict__ out_st, const float *__restrict__ lse,
    const __nv_bfloat16 *__restrict__ dout, __nv_bfloat16 *__restrict__ dq,
    float *__restrict__ delta, double *__restrict__ dalpha_part, int32_t *__restrict__ status,
    int nT) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[kDqStages + 2];  // full[stages], qg, mma
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int nvis_s;
  __shared__ double red[128];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nST = (s.L + 127) >> 7;
  const int st = nST - 1 - (int)(blockIdx.x % nST);
  const int u = blockIdx.x / nST, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int row0 = st * 128, row_last = min(s.L - 1, row0 + 127);
  const int G = 128 / s.Bk, nb = 64 / s.Bk;

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *q_tile = tiles;
  uint8_t *g_tile = q_tile + C::kBigBytes;
  uint8_t *kv_tiles = g_tile + C::kBigBytes;
  uint8_t *ds_tile = kv_tiles + kDqStages * 2 * C::kSmallBytes;
  uint8_t *meta = ds_tile + C::kPBytes;
  uint32_t *selw = reinterpret_cast<uint32_t *>(meta);
  uint8_t *selb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ((8 * nT + 15) / 16) * 16);
  uint8_t *lflags = reinterpret_cast<uint8_t *>(list + nT);

  const uint32_t bar_full0 = smem_u32(&bars[0]);
  const uint32_t bar_qg = smem_u32(&bars[kDqStages]);
  const uint32_t bar_mma = smem_u32(&bars[kDqStages + 1]);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;
    for (int i = 0; i < kDqStages; ++i) mbar_init(bar_full0 + 8 * i, 1);
    mbar_init(bar_qg, 1);
    mbar_init(bar_mma, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
    tma_prefetch_desc(&tmg);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), 256);
    tmem_relinquish();
  }
  for (int i = tid; i < (8 * nT + 3) / 4; i += 128) selw[i] = 0u;
  __syncthreads();
  for (int i = tid; i < G * s.topk; i += 128) {
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
    if (lane == 0) nvis_s = count;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const int nvis = nvis_s;
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_dp = tmem_base + 64, tmem_dq = tmem_base + 128;
  const uint32_t lane_off = (uint32_t)(warp * 32) << 16;

  if (tid == 0 && nvis > 0) {
    mbar_expect_tx(bar_qg, 2 * C::kBigBytes);
    tma_load_4d(smem_u32(q_tile), &tmq, bar_qg, 0, row0, h, n);
    tma_load_4d(smem_u32(g_tile), &tmg, bar_qg, 0, row0, h, n);
    for (int i = 0; i < min(kDqStages, nvis); ++i) {
      const uint32_t bar = bar_full0 + 8 * i;
      uint8_t *kt = kv_tiles + i * 2 * C::kSmallBytes;
      mbar_expect_tx(bar, 2 * C::kSmallBytes);
      tma_load_4d(smem_u32(kt), &tmk, bar, 0, (int)list[i] * 64, h, n);
      tma_load_4d(smem_u32(kt + C::kSmallBytes), &tmv, bar, 0, (int)list[i] * 64, h, n);
    }
  }
  __syncwarp();

  // ---- per-row statistics: delta of both branches, saved log-sum-exps ----
  const int r = tid, t = row0 + r, g = r / s.Bk;
  const bool row_ok = t < s.L, row_valid = row_ok && t >= pad0;
  const float alpha = sigmoid_gate(gate, h), beta = 1.f - alpha;
  const int64_t BHL = (int64_t)s.B * s.H * s.L;
  const int64_t ro = row_offset(s, n, h, row_ok ? t : 0);
  float deltaL = 0.f, deltaS = 0.f, lseL2 = 0.f, lseS2 = 0.f;
  if (row_valid) {
    float aL = 0.f, aS = 0.f;
#pragma unroll
    for (int c = 0; c < D; c += 8) {
      const uint4 gv = *reinterpret_cast<const uint4 *>(dout + ro + c);
      const uint4 lv = *reinterpret_cast<const uint4 *>(out_lt + ro + c);
      const uint4 sv = *reinterpret_cast<const uint4 *>(out_st + ro + c);
      const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, lw[4] = {lv.x, lv.y, lv.z, lv.w},
                     sw[4] = {sv.x, sv.y, sv.z, sv.w};
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
  if (row_ok) {
    delta[(int64_t)u * s.L + t] = deltaL;
    delta[BHL + (int64_t)u * s.L + t] = deltaS;
  }

  float dal = 0.f;
  bool ds_zero = false;
  int acc = 0;
  const float sc2 = s.scale * kLog2e;
  constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
  constexpr uint32_t idesc_dq = instr_desc(128, D, 0, 1);
  uint32_t mma_phase = 0;

  for (int i = 0; i < nvis; ++i) {
    const int stage = i % kDqStages;
    const int jt = list[i], f = lflags[i], p0 = jt * 64;
    uint8_t *k_tile = kv_tiles + stage * 2 * C::kSmallBytes, *v_tile = k_tile + C::kSmallBytes;
    if (tid == 0) {
      if (i == 0) mbar_wait(bar_qg, 0, &abort_flag);
      mbar_wait(bar_full0 + 8 * stage, (i / kDqStages) & 1, &abort_flag);
      tc_fence_after();
      const uint64_t dqd = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dgd = smem_desc(smem_u32(g_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dkd = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dvd = smem_desc(smem_u32(v_tile), 16, C::kAtomBytes, C::kSwizzle);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_s, dqd + 2 * k, dkd + 2 * k, idesc_s, k > 0);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_dp, dgd + 2 * k, dvd + 2 * k, idesc_s, k > 0);
      umma_commit(bar_mma);
    }
    __syncwarp();
    mbar_wait(bar_mma, mma_phase, &abort_flag);
    __syncwarp();
    mma_phase ^= 1u;
    tc_fence_after();
    if (tid == 0 && i >= 1 && i - 1 + kDqStages < nvis) {
      const int j = i - 1 + kDqStages, sj = (i - 1) % kDqStages;
      const uint32_t bar = bar_full0 + 8 * sj;
      uint8_t *kt = kv_tiles + sj * 2 * C::kSmallBytes;
      mbar_expect_tx(bar, 2 * C::kSmallBytes);
      tma_load_4d(smem_u32(kt), &tmk, bar, 0, (int)list[j] * 64, h, n);
      tma_load_4d(smem_u32(kt + C::kSmallBytes), &tmv, bar, 0, (int)list[j] * 64, h, n);
    }
    __syncwarp();

    uint64_t maskL = 0ull, maskS = 0ull;
    if (row_valid) {
      const uint64_t mc = cols_le(t - p0) & cols_ge(pad0 - p0);
      if (f & 1) maskL = mc & expand_block_bits(selb[g * nT + jt], s.Bk);
      if (f & 2) maskS = mc & cols_ge(t - s.window + 1 - p0);
    }
    if (__any_sync(0xffffffffu, (maskL | maskS) != 0ull)) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        float sv[32], dp[32];
        tmem_ld32(tmem_s + lane_off + hh * 32, sv);
        tmem_ld32(tmem_dp + lane_off + hh * 32, dp);
        tmem_wait_ld();
        const uint32_t mLh = (uint32_t)(maskL >> (hh * 32)), mSh = (uint32_t)(maskS >> (hh * 32));
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          float d[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int c = ch * 8 + e;
            const float x = sv[c] * sc2;
            const float pL = ((mLh >> c) & 1u) ? exp2f(x - lseL2) : 0.f;
            const float pS = ((mSh >> c) & 1u) ? exp2f(x - lseS2) : 0.f;
            d[e] = fmaf(pL, fmaf(alpha, dp[c], -deltaL), pS * fmaf(beta, dp[c], -deltaS));
            dal = fmaf(pL - pS, dp[c], dal);
          }
          store_row_sw128(ds_tile, r, hh * 4 + ch,
                          make_uint4(pack_bf16(d[0], d[1]), pack_bf16(d[2], d[3]),
                                     pack_bf16(d[4], d[5]), pack_bf16(d[6], d[7])));
        }
      }
      ds_zero = false;
    } else if (!ds_zero) {
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) store_row_sw128(ds_tile, r, ch, make_uint4(0u, 0u, 0u, 0u));
      ds_zero = true;
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint64_t dsd = smem_desc(smem_u32(ds_tile), 16, 1024, 2u);
      const uint64_t dkm = smem_desc(smem_u32(k_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        umma_bf16(tmem_dq, dsd + 2 * k, dkm + k * (16 * C::kRowBytes >> 4), idesc_dq, (acc | k) != 0);
    }
    acc = 1;
  }

  if (nvis > 0) {
    if (tid == 0) umma_commit(bar_mma);
    __syncwarp();
    mbar_wait(bar_mma, mma_phase, &abort_flag);
    __syncwarp();
    tc_fence_after();
  }
#pragma unroll
  for (int hh = 0; hh < D / 32; ++hh) {
    float o[32];
    if (acc) {
      tmem_ld32(tmem_dq + lane_off + hh * 32, o);
      tmem_wait_ld();
    }
    if (row_ok) {
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          w[e] = (acc && row_valid) ? pack_bf16(o[c] * s.scale, o[c + 1] * s.scale) : 0u;
        }
        *reinterpret_cast<uint4 *>(dq + ro + hh * 32 + ch * 8) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
  // d alpha partial of this CTA -> first query-block slot of the super-tile, zeros in the rest
  red[tid] = row_valid ? (double)dal : 0.0;
  tc_fence_before();
  __syncthreads();
  if (tid == 0) {
    double a = 0.0;
    for (int i = 0; i < 128; ++i) a += red[i];
    for (int gq = 0; gq < G; ++gq)
      if (st * G + gq < s.M) dalpha_part[(int64_t)u * s.M + st * G + gq] = gq == 0 ? a : 0.0;
  }
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc(tmem_base, 256);
  }
  if (tid == 0 && abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}
    atomicExch(status, (int32_t)BLOSSOM_ERR_TIMEOUT);
  }
}

// --------------------------------------------------------------------------- dK, dV kernel
template <int D>
__global__ void __launch_bounds__(128, 2) bwd_dkdv_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmg, Shape s,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, const float *__restrict__ lse,
    const float *__restrict__ delta, __nv_bfloat16 *__restrict__ dk, __nv_bfloat16 *__restrict__ dv,
    int32_t *__restrict__ status, int nT) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[kKvStages + 2];  // full[stages], kv, mma
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int nvis_s;
  __shared__ __align__(16) float4 stats[2][64];  // per query column: lse_lt*log2e, lse_st*log2e, delta_lt, delta_st

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
  uint8_t *w_tile = qg_tiles + kKvStages * 2 * C::kSmallBytes;
  uint8_t *ds_tile = w_tile + C::kPBytes;
  uint8_t *meta = ds_tile + C::kPBytes;
  uint32_t *invw = reinterpret_cast<uint32_t *>(meta);  // [8][nT] bytes: per key block, per query tile
  uint8_t *invb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ((8 * nT + 15) / 16) * 16);
  uint8_t *lflags = reinterpret_cast<uint8_t *>(list + nT);

  const uint32_t bar_full0 = smem_u32(&bars[0]);
  const uint32_t bar_kv = smem_u32(&bars[kKvStages]);
  const uint32_t bar_mma = smem_u32(&bars[kKvStages + 1]);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;
    for (int i = 0; i < kKvStages; ++i) mbar_init(bar_full0 + 8 * i, 1);
    mbar_init(bar_kv, 1);
    mbar_init(bar_mma, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
    tma_prefetch_desc(&tmg);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), 256);
    tmem_relinquish();
  }
  for (int i = tid; i < (8 * nT + 3) / 4; i += 128) invw[i] = 0u;
  __syncthreads();
  // which query blocks selected each of this CTA's key blocks, per 64-query tile
  {
    const int qb0 = kt * G, nq = s.M - qb0;
    for (int i = tid; i < nq * s.topk; i += 128) {
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
        if (qt * 64 <= key_last + s.window - 1) f |= 2;  // qt*64+63 >= key0 holds for qt >= qt_min
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
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const int nvis = nvis_s;
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_dp = tmem_base + 64, tmem_dv = tmem_base + 128,
                 tmem_dk = tmem_base + 192;
  const uint32_t lane_off = (uint32_t)(warp * 32) << 16;

  if (tid == 0 && nvis > 0) {
    mbar_expect_tx(bar_kv, 2 * C::kBigBytes);
    tma_load_4d(smem_u32(k_tile), &tmk, bar_kv, 0, key0, h, n);
    tma_load_4d(smem_u32(v_tile), &tmv, bar_kv, 0, key0, h, n);
    for (int i = 0; i < min(kKvStages, nvis); ++i) {
      const uint32_t bar = bar_full0 + 8 * i;
      uint8_t *qt_ = qg_tiles + i * 2 * C::kSmallBytes;
      mbar_expect_tx(bar, 2 * C::kSmallBytes);
      tma_load_4d(smem_u32(qt_), &tmq, bar, 0, (int)list[i] * 64, h, n);
      tma_load_4d(smem_u32(qt_ + C::kSmallBytes), &tmg, bar, 0, (int)list[i] * 64, h, n);
    }
  }
  __syncwarp();

  const int64_t BHL = (int64_t)s.B * s.H * s.L;
  // per-query statistics of a tile: thread -> (column c, which half of the float4)
  auto load_stats = [&](int qt, float &a, float &b) {
    const int c = tid & 63, tq = qt * 64 + c;
    a = 0.f;
    b = 0.f;
    if (tq < s.L) {
      if (tid < 64) {
        a = lse[(int64_t)u * s.L + tq] * kLog2e;
        b = lse[BHL + (int64_t)u * s.L + tq] * kLog2e;
      } else {
        a = delta[(int64_t)u * s.L + tq];
        b = delta[BHL + (int64_t)u * s.L + tq];
      }
    }
  };
  auto store_stats = [&](int buf, float a, float b) {
    float *p = reinterpret_cast<float *>(&stats[buf][tid & 63]) + (tid < 64 ? 0 : 2);
    p[0] = a;
    p[1] = b;
  };
  if (nvis > 0) {
    float a, b;
    load_stats(list[0], a, b);
    store_stats(0, a, b);
  }
  __syncthreads();

  const int r = tid, p = key0 + r, g = r / s.Bk;
  const bool row_ok = p < s.L, row_valid = row_ok && p >= pad0;
  const float alpha = sigmoid_gate(gate, h), beta = 1.f - alpha;
  bool w_zero = false;
  int acc = 0;
  const float sc2 = s.scale * kLog2e;
  constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
  constexpr uint32_t idesc_o = instr_desc(128, D, 0, 1);
  uint32_t mma_phase = 0;

  for (int i = 0; i < nvis; ++i) {
    const int stage = i % kKvStages;
    const int qt = list[i], f = lflags[i], t0 = qt * 64;
    uint8_t *q_tile = qg_tiles + stage * 2 * C::kSmallBytes, *g_tile = q_tile + C::kSmallBytes;
    if (tid == 0) {
      if (i == 0) mbar_wait(bar_kv, 0, &abort_flag);
      mbar_wait(bar_full0 + 8 * stage, (i / kKvStages) & 1, &abort_flag);
      tc_fence_after();
      const uint64_t dkd = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dvd = smem_desc(smem_u32(v_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dqd = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dgd = smem_desc(smem_u32(g_tile), 16, C::kAtomBytes, C::kSwizzle);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_s, dkd + 2 * k, dqd + 2 * k, idesc_s, k > 0);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_dp, dvd + 2 * k, dgd + 2 * k, idesc_s, k > 0);
      umma_commit(bar_mma);
    }
    __syncwarp();
    // statistics of the next tile travel through registers while the MMAs run
    float na = 0.f, nbv = 0.f;
    const bool have_next = i + 1 < nvis;
    if (have_next) load_stats(list[i + 1], na, nbv);
    mbar_wait(bar_mma, mma_phase, &abort_flag);
    __syncwarp();
    mma_phase ^= 1u;
    tc_fence_after();
    if (tid == 0 && i >= 1 && i - 1 + kKvStages < nvis) {
      const int j = i - 1 + kKvStages, sj = (i - 1) % kKvStages;
      const uint32_t bar = bar_full0 + 8 * sj;
      uint8_t *qt_ = qg_tiles + sj * 2 * C::kSmallBytes;
      mbar_expect_tx(bar, 2 * C::kSmallBytes);
      tma_load_4d(smem_u32(qt_), &tmq, bar, 0, (int)list[j] * 64, h, n);
      tma_load_4d(smem_u32(qt_ + C::kSmallBytes), &tmg, bar, 0, (int)list[j] * 64, h, n);
    }
    __syncwarp();

    uint64_t maskL = 0ull, maskS = 0ull;
    if (row_valid) {
      const uint64_t mc = cols_ge(p - t0) & cols_le(s.L - 1 - t0);
      if (f & 1) maskL = mc & expand_block_bits(invb[g * nT + qt], s.Bk);
      if (f & 2) maskS = mc & cols_le(p + s.window - 1 - t0);
    }
    if (__any_sync(0xffffffffu, (maskL | maskS) != 0ull)) {
      const float4 *stt = stats[i & 1];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        float sv[32], dp[32];
        tmem_ld32(tmem_s + lane_off + hh * 32, sv);
        tmem_ld32(tmem_dp + lane_off + hh * 32, dp);
        tmem_wait_ld();
        const uint32_t mLh = (uint32_t)(maskL >> (hh * 32)), mSh = (uint32_t)(maskS >> (hh * 32));
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          float wv[8], d[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int c = ch * 8 + e;
            const float4 q4 = stt[hh * 32 + c];
            const float x = sv[c] * sc2;
            const float pL = ((mLh >> c) & 1u) ? exp2f(x - q4.x) : 0.f;
            const float pS = ((mSh >> c) & 1u) ? exp2f(x - q4.y) : 0.f;
            wv[e] = fmaf(alpha, pL, beta * pS);
            d[e] = fmaf(pL, fmaf(alpha, dp[c], -q4.z), pS * fmaf(beta, dp[c], -q4.w));
          }
          store_row_sw128(w_tile, r, hh * 4 + ch,
                          make_uint4(pack_bf16(wv[0], wv[1]), pack_bf16(wv[2], wv[3]),
                                     pack_bf16(wv[4], wv[5]), pack_bf16(wv[6], wv[7])));
          store_row_sw128(ds_tile, r, hh * 4 + ch,
                          make_uint4(pack_bf16(d[0], d[1]), pack_bf16(d[2], d[3]),
                                     pack_bf16(d[4], d[5]), pack_bf16(d[6], d[7])));
        }
      }
      w_zero = false;
    } else if (!w_zero) {
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        store_row_sw128(w_tile, r, ch, make_uint4(0u, 0u, 0u, 0u));
        store_row_sw128(ds_tile, r, ch, make_uint4(0u, 0u, 0u, 0u));
      }
      w_zero = true;
    }
    if (have_next) store_stats((i + 1) & 1, na, nbv);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint64_t dwd = smem_desc(smem_u32(w_tile), 16, 1024, 2u);
      const uint64_t dsd = smem_desc(smem_u32(ds_tile), 16, 1024, 2u);
      const uint64_t dgm = smem_desc(smem_u32(g_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
      const uint64_t dqm = smem_desc(smem_u32(q_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        umma_bf16(tmem_dv, dwd + 2 * k, dgm + k * (16 * C::kRowBytes >> 4), idesc_o, (acc | k) != 0);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        umma_bf16(tmem_dk, dsd + 2 * k, dqm + k * (16 * C::kRowBytes >> 4), idesc_o, (acc | k) != 0);
    }
    acc = 1;
  }

  if (nvis > 0) {
    if (tid == 0) umma_commit(bar_mma);
    __syncwarp();
    mbar_wait(bar_mma, mma_phase, &abort_flag);
    __syncwarp();
    tc_fence_after();
  }
  const int64_t ro = row_offset(s, n, h, row_ok ? p : 0);
#pragma unroll
  for (int hh = 0; hh < D / 32; ++hh) {
    float ov[32], ok[32];
    if (acc) {
      tmem_ld32(tmem_dv + lane_off + hh * 32, ov);
      tmem_ld32(tmem_dk + lane_off + hh * 32, ok);
      tmem_wait_ld();
    }
    if (row_ok) {
      const bool live = acc && row_valid;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t wv[4], wk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          wv[e] = live ? pack_bf16(ov[c], ov[c + 1]) : 0u;
          wk[e] = live ? pack_bf16(ok[c] * s.scale, ok[c + 1] * s.scale) : 0u;
        }
        *reinterpret_cast<uint4 *>(dv + ro + hh * 32 + ch * 8) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        *reinterpret_cast<uint4 *>(dk + ro + hh * 32 + ch * 8) = make_uint4(wk[0], wk[1], wk[2], wk[3]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 256);
  if (tid == 0 && abort_flag) {
    const long long t0c = clock64();
    while (clock64() - t0c < 2000000LL) {}
    atomicExch(status, (int32_t)BLOSSOM_ERR_TIMEOUT);
  }
}

template <int D>
int launch_bwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, const void *out_lt,
                    const void *out_st, const float *lse, const void *dout, void *dq, void *dk,
                    void *dv, const Workspace &ws, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  CUtensorMap q128, k64, v64, g128, q64, k128, v128, g64;
  if (make_tensor_map(&q128, q, s, 128) || make_tensor_map(&k64, k, s, 64) ||
      make_tensor_map(&v64, v, s, 64) || make_tensor_map(&g128, dout, s, 128) ||
      make_tensor_map(&q64, q, s, 64) || make_tensor_map(&k128, k, s, 128) ||
      make_tensor_map(&v128, v, s, 128) || make_tensor_map(&g64, dout, s, 64))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const unsigned grid = (unsigned)nST * (unsigned)(s.B * s.H);
  using C = Cfg<D>;
  const size_t smem_dq = 1024 + 2 * C::kBigBytes + kDqStages * 2 * C::kSmallBytes + C::kPBytes + meta_bytes(nT);
  const size_t smem_kv = 1024 + 2 * C::kBigBytes + kKvStages * 2 * C::kSmallBytes + 2 * C::kPBytes + meta_bytes(nT);
  if (cudaFuncSetAttribute(bwd_dq_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_dq) != cudaSuccess ||
      cudaFuncSetAttribute(bwd_dkdv_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kv) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    LaunchScope ls(K_BWD_DQ_TC, st);
    bwd_dq_tc_kernel<D><<<grid, 128, smem_dq, st>>>(q128, k64, v64, g128, s, gate, seq_lens, idx,
                                                   (const bf *)out_lt, (const bf *)out_st, lse,
                                                   (const bf *)dout, (bf *)dq, ws.delta, ws.dalpha,
                                                   ws.status, nT);
  }
  {
    LaunchScope ls(K_BWD_DKDV_TC, st);
    bwd_dkdv_tc_kernel<D><<<grid, 128, smem_kv, st>>>(q64, k128, v128, g64, s, gate, seq_lens, idx, lse,
                                                     ws.delta, (bf *)dk, (bf *)dv, ws.status, nT);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

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
