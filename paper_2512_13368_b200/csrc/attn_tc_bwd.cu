// Tensor-core backward of the fused two-branch attention (bf16 storage, fp32 accumulate): a small
// pre-pass and two main kernels, all deterministic (no atomics on any gradient); the main kernels
// recompute the probabilities from the saved log-sum-exps.
//
//  pre-pass  Delta_x = rowsum(dO o O_x) of both branches from coalesced reads, and the per-row
//            records the main kernels read: per pair of rows {nl_lt(2), -Delta_lt(2)}
//            {nl_st(2), -Delta_st(2)}, nl = -(lse*log2e - log2 weight): the branch weights alpha,
//            beta ride in the exponent, alpha P_lt = exp2(s*log2e + nl_lt).
//
// Main kernels: CTA = 384 threads.  Warps 0..7 compute; warps 8, 9, 10 stay converged and one
// elected lane of each issues the TMA loads, the first-stage MMAs and the second-stage MMAs;
// registers move from those warps to the compute warps (setmaxnreg).  A CTA owns a resident
// 128-row tile (rows = TMEM lanes) and streams 64-row tiles past it.  Row r of the 128 is shared by
// two compute threads: warp w and warp w + 4 both address TMEM lane quarter w % 4; the first takes
// columns 0..31 of a 64-column tile, the second columns 32..63.  The tile arithmetic runs in
// 16-column passes, two columns per FMA / ADD / MUL (packed f32x2); outputs are staged in shared
// memory and written with whole-line TMA stores.
//
//  dQ     resident Q, dO (128 queries: 128 positions of a head, or with grouped heads 64 positions
//         of two heads of a group, as in the forward); streams K, V 64-key tiles (same walk as the forward) and
//         works through them in half tiles of 32 keys.  Tensor memory: two buffers of 64
//         columns (half tile x uses buffer x % 2: S in its first 32 columns, dP in the other 32),
//         Q and dO as first operands of the first-stage products [128,128+D/2), [160,160+D/2)
//         (read from shared memory they cost 4 KB per product, more than the data pipe delivers
//         in the product's run time), and dQ [192,192+D).  S = Q K^T, dP = dO V^T; P'_x = weight_x exp(S - lse_x);
//         dS = P'_lt (dP - Delta_lt) + P'_st (dP - Delta_st) (one tile for both branches, they share
//         K).  A thread owns 16 of the 32 columns and writes its dS (bf16 pairs) over the first 8
//         of its own S columns, from where dQ += dS K reads it: the compute warps wait for one
//         thing per half tile (its S and dP), and the first stage of the next two half tiles runs
//         meanwhile.  d alpha = sum (P_lt - P_st) dP from the fp32 probabilities.
//  dK/dV  transposed: resident K, V of 128 keys, streams Q, dO 64-query tiles (and their row
//         records, by bulk copy) that selected one of its key blocks or whose window reaches them.
//         It works through them in half tiles of 32 queries.  Tensor memory: two buffers of 64
//         columns (half tile x uses buffer x % 2: S^T in its first 32 columns, dP^T in the other
//         32), dV [128,128+D), dK [192,192+D).  S^T = K Q^T, dP^T = V dO^T; thread = key row and
//         16 of the 32 query columns; it writes W^T = P'_lt + P'_st and dS^T (bf16 pairs) over the
//         first 8 of its own S^T / dP^T columns, from where dV += W^T dO and dK += dS^T Q read
//         their first operand: nothing of a tile's arithmetic goes through shared memory, whose
//         data pipe (operand reads of the products, row records) is the busiest unit of this
//         kernel, and the first stage of the next half tile runs during the arithmetic of this one.
// Every wait is bounded (tc_common.cuh).
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

// warps 0..7 compute; 8 loader, 9 first-stage issuer, 10 second-stage issuer, 11 spare
constexpr int kKvThreads = 384;
constexpr int kProducerRegs = 64, kKvComputeRegs = 88;  // 256 * 88 + 128 * 64 = 384 * 80 (measured: the issuing warps spill below 48)
constexpr int kComputeWarps = 8;
constexpr int kDqStages = 4;
constexpr int kKvStages = 4;
constexpr uint32_t kBwdTmemCols = 256;
constexpr int kStatBytes = 64 * 16;  // one 64-query tile of row records

__device__ __forceinline__ bool bit(uint32_t w, int c) { return (w >> c) & 1u; }

// ------------------------------------------------------------------ backward pre-pass
// Delta_x = rowsum(dO o O_x) of both branches and the per-row records both backward kernels read:
// per pair of rows {nl_lt(2), -Delta_lt(2)} {nl_st(2), -Delta_st(2)} with
// nl = -(lse * log2e - log2 weight), the branch weight (alpha, beta) riding in the exponent;
// zeros for padded rows and for the rows that pad L to a multiple of 64.
// D / 8 lanes share a row (one 16-byte load per tensor each): fully coalesced reads.
template <int D>
__global__ void __launch_bounds__(256) bwd_prep_kernel(Shape s, const float *__restrict__ gate,
                                                       const int32_t *__restrict__ seq_lens,
                                                       const __nv_bfloat16 *__restrict__ out_lt,
                                                       const __nv_bfloat16 *__restrict__ out_st,
                                                       const float *__restrict__ lse,
                                                       const __nv_bfloat16 *__restrict__ dout,
                                                       float4 *__restrict__ qstats, int Lpad) {
  grid_chain_enter();
  constexpr int LPR = D / 8;         // lanes per row
  constexpr int RPB = 256 / LPR;     // rows per block
  const int blocks_per_unit = (Lpad + RPB - 1) / RPB;
  const int u = blockIdx.x / blocks_per_unit, n = u / s.H, h = u % s.H;
  const int t = (blockIdx.x % blocks_per_unit) * RPB + threadIdx.x / LPR, ch = threadIdx.x % LPR;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const bool row_valid = t < s.L && t >= s.L - len;
  float aL = 0.f, aS = 0.f;
  if (row_valid) {
    const int64_t off = row_offset(s, n, h, t) + ch * 8;
    const uint4 gv = *reinterpret_cast<const uint4 *>(dout + off);
    const uint4 lv = *reinterpret_cast<const uint4 *>(out_lt + off);
    const uint4 sv4 = *reinterpret_cast<const uint4 *>(out_st + off);
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
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) {  // fixed-shape tree over the row's lanes
    aL += __shfl_xor_sync(0xffffffffu, aL, o);
    aS += __shfl_xor_sync(0xffffffffu, aS, o);
  }
  if (ch == 0 && t < Lpad) {
    float r0 = 0.f, r2 = 0.f, r4 = 0.f, r6 = 0.f;
    if (row_valid) {
      const float alpha = gate_alpha(gate, h), beta = 1.f - alpha;
      const int64_t BHL = (int64_t)s.B * s.H * s.L;
      r0 = -(lse[(int64_t)u * s.L + t] * kLog2e - log2f(alpha));
      r4 = -(lse[BHL + (int64_t)u * s.L + t] * kLog2e - log2f(beta));
      r2 = -aL;
      r6 = -aS;
    }
    float *rec = reinterpret_cast<float *>(qstats) + ((int64_t)u * Lpad + (t & ~1)) * 4 + (t & 1);
    rec[0] = r0;
    rec[2] = r2;
    rec[4] = r4;
    rec[6] = r6;
  }
}

// ---------------------------------------------------------------------------- backward dQ
// 16 columns of one tile for one row: dS packed to bf16 pairs, partial sums of P' dP.
// nlL / nlS = -(lse * log2e - log2 alpha) resp. beta: the branch weight rides in the exponent, so
// P' = alpha P_lt (beta P_st) comes straight out of the exponential; nDL / nDS = -Delta.
// Two columns per FMA / ADD / MUL instruction.
template <bool HAS_L, bool HAS_S, bool FULL>
__device__ __forceinline__ void dq_tile(const float (&sv)[16], const float (&dp)[16], uint32_t hL,
                                        uint32_t hS, float sc2, float nlL, float nlS, float nDL,
                                        float nDS, float2 &dalL, float2 &dalS, uint32_t (&dw)[8]) {
  const float2 sc = make_float2(sc2, sc2);
#pragma unroll
  for (int c = 0; c < 16; c += 2) {
    const float2 s2 = make_float2(sv[c], sv[c + 1]), dp2 = make_float2(dp[c], dp[c + 1]);
    float2 acc = make_float2(0.f, 0.f);
    if (HAS_L) {
      const float2 x = ffma2(s2, sc, make_float2(nlL, nlL));
      float2 p = make_float2(exp2f(x.x), exp2f(x.y));
      if (!FULL) {
        p.x = bit(hL, c) ? p.x : 0.f;
        p.y = bit(hL, c + 1) ? p.y : 0.f;
      }
      dalL = ffma2(p, dp2, dalL);
      acc = fmul2(p, fadd2(dp2, make_float2(nDL, nDL)));
    }
    if (HAS_S) {
      const float2 x = ffma2(s2, sc, make_float2(nlS, nlS));
      float2 p = make_float2(exp2f(x.x), exp2f(x.y));
      if (!FULL) {
        p.x = bit(hS, c) ? p.x : 0.f;
        p.y = bit(hS, c + 1) ? p.y : 0.f;
      }
      dalS = ffma2(p, dp2, dalS);
      acc = ffma2(p, fadd2(dp2, make_float2(nDS, nDS)), acc);
    }
    dw[c >> 1] = pack_bf16(acc.x, acc.y);
  }
}

// PLAIN (both kernels below): the causal mask and one selection per query block (the measured
// path): the other modes' tests fold away at compile time.
// PACK (dQ kernel): rows 0..63 and 64..127 of the CTA are the same 64 positions of two query heads
// with a common key/value head, as in the forward kernel.
template <int D, bool PLAIN, bool PACK>
__global__ void __launch_bounds__(kKvThreads, 2) bwd_dq_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmg, Shape s,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const uint8_t *__restrict__ qmeta, const __grid_constant__ CUtensorMap tmdq,
    const float4 *__restrict__ qstats, double *__restrict__ dalpha_part, int32_t *__restrict__ status,
    int nT) {
  grid_chain_enter();
  using C = Cfg<D>;
  constexpr int STAGES = kDqStages;
  constexpr int OC = D / 2;  // accumulator columns per thread
  extern __shared__ uint8_t smem_raw[];
  // barriers: full[STAGES], empty[STAGES], res, meta, a_ready, then one per buffer: s_full[2],
  // t_full[2], mma_done[2]
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 9];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ double red[kComputeWarps];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nST = (s.L + 127) >> 7;
  // long rows first, tile-major: every unit's last tile, then every unit's last but one, ...
  // (PACK: a unit is a pair of heads, a tile 64 positions; h = the pair's first head)
  const int nU = PACK ? s.B * (s.H / 2) : s.B * s.H, nQT = PACK ? nT : nST;
  const int st = nQT - 1 - (int)(blockIdx.x / nU);
  const int u = (int)(blockIdx.x % nU);
  const int n = PACK ? u / (s.H / 2) : u / s.H, h = PACK ? 2 * (u % (s.H / 2)) : u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int row0 = PACK ? st * 64 : st * 128;
  const int Lpad = nT * 64;

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *q_tile = tiles;
  uint8_t *g_tile = q_tile + C::kBigBytes;
  uint8_t *kv_tiles = g_tile + C::kBigBytes;
  uint8_t *meta = kv_tiles + STAGES * 2 * C::kSmallBytes;  // image built by tc_meta_kernel
  const bool causal = PLAIN || s.causal;
  const int pq = PLAIN ? 0 : s.pq;
  const MetaLayout ml = meta_layout(nT, pq);
  const uint8_t *selb = meta;
  const uint8_t *rowb = meta + ml.rows;  // (selection per query position) [128 rows][nT]
  const uint16_t *list = reinterpret_cast<const uint16_t *>(meta + ml.list);
  const uint8_t *lflags = meta + ml.flags;
  const uint8_t *jcls = meta + ml.jcls;  // [tile][half tile][compute warp]

  const uint32_t b_full = smem_u32(&bars[0]), b_empty = smem_u32(&bars[STAGES]);
  const uint32_t b_res = smem_u32(&bars[2 * STAGES]), b_meta = smem_u32(&bars[2 * STAGES + 1]);
  const uint32_t b_aready = smem_u32(&bars[2 * STAGES + 2]);
  const uint32_t b_sfull = smem_u32(&bars[2 * STAGES + 3]), b_tfull = smem_u32(&bars[2 * STAGES + 5]);
  const uint32_t b_done = smem_u32(&bars[2 * STAGES + 7]);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
    tma_prefetch_desc(&tmg);
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(b_full + 8 * i, 1);
      mbar_init(b_empty + 8 * i, 1);
    }
    mbar_init(b_res, 1);
    mbar_init(b_aready, kComputeWarps);
    for (int i = 0; i < 2; ++i) {
      mbar_init(b_sfull + 8 * i, 1);
      mbar_init(b_tfull + 8 * i, kComputeWarps);
      mbar_init(b_done + 8 * i, 1);
    }
    mbar_init(b_meta, 1);
    mbar_fence_init();
    // the CTA's tile lists and its resident tiles
    mbar_expect_tx(b_meta, (uint32_t)ml.bytes);
    bulk_load(smem_u32(meta), qmeta + ((size_t)u * nQT + (nQT - 1 - st)) * ml.bytes, (uint32_t)ml.bytes, b_meta);
    mbar_expect_tx(b_res, 2 * C::kBigBytes);
    tma_load_4d(smem_u32(q_tile), &tmq, b_res, 0, row0, h, n);
    tma_load_4d(smem_u32(g_tile), &tmg, b_res, 0, row0, h, n);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), kBwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  mbar_wait(b_meta, 0, &abort_flag, 223);
  const int nvis = *reinterpret_cast<const int *>(meta + ml.counts);
  const uint32_t tmem_base = tmem_slot;
  // buffers at tmem_base + 64 * (half tile % 2); Q and dO as first operands (bf16 pairs, D / 2
  // columns each) at 128 and 160; the dQ accumulator at 192
  const uint32_t tmem_qa = tmem_base + 128, tmem_ga = tmem_base + 160, tmem_dq = tmem_base + 192;

  if (warp >= kComputeWarps) {
    // ============ three single-thread roles, one converged warp each ============
    setmaxnreg_dec<kProducerRegs>();
    if (warp == kComputeWarps && nvis > 0) {
      // ---- loader: Q, dO once; K/V tiles up to STAGES ahead of their consumers ----
      for (int j = 0; j < nvis; ++j) {
        const int sj = j % STAGES;
        if (j >= STAGES) mbar_wait(b_empty + 8 * sj, ((j - STAGES) / STAGES) & 1, &abort_flag, 205);
        const uint32_t bar = b_full + 8 * sj;
        const uint32_t kt = smem_u32(kv_tiles + sj * 2 * C::kSmallBytes);
        const int row = (int)list[j] * 64;
        if (elect_one()) {
          mbar_expect_tx(bar, 2 * C::kSmallBytes);
          tma_load_4d(kt, &tmk, bar, 0, row, h / s.G, n);  // the key/value head of this query head
          tma_load_4d(kt + C::kSmallBytes, &tmv, bar, 0, row, h / s.G, n);
        }
        __syncwarp();
      }
    } else if (warp == kComputeWarps + 1 && nvis > 0) {
      // ---- S = Q K^T and dP = dO V^T of a half tile (32 keys) into buffer x % 2 once
      // dQ += dS K of half tile x-2 has read that buffer.  Q and dO are read from tensor memory
      // (the compute warps copied the resident tiles there), so a product fetches only its 32
      // keys from shared memory instead of 128 rows of Q or dO as well ----
      constexpr uint32_t idesc_s = instr_desc(128, 32, 0, 0);
      mbar_wait(b_aready, 0, &abort_flag, 201);
      tc_fence_after();
      for (int i = 0, x = 0, b = 0, ph = 0; i < nvis; ++i) {  // x = 2 i + hh, b = x % 2, ph = (x / 2) & 1
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 202);
        for (int hh = 0; hh < 2; ++hh, ++x) {
          if (x >= 2) mbar_wait(b_done + 8 * b, ph ^ 1, &abort_flag, 203);
          tc_fence_after();
          const uint32_t kt = smem_u32(kv_tiles + (i % STAGES) * 2 * C::kSmallBytes) + hh * 32 * C::kRowBytes;
          const uint64_t dkd = smem_desc(kt, 16, C::kAtomBytes, C::kSwizzle);
          const uint64_t dvd = smem_desc(kt + C::kSmallBytes, 16, C::kAtomBytes, C::kSwizzle);
          const uint32_t ts = tmem_base + 64 * b;
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) umma_bf16_ts(ts, tmem_qa + 8 * k, dkd + 2 * k, idesc_s, k > 0);
#pragma unroll
            for (int k = 0; k < D / 16; ++k) umma_bf16_ts(ts + 32, tmem_ga + 8 * k, dvd + 2 * k, idesc_s, k > 0);
            umma_commit(b_sfull + 8 * b);
          }
          __syncwarp();
          if (++b == 2) {
            b = 0;
            ph ^= 1;
          }
        }
      }
    } else if (warp == kComputeWarps + 2 && nvis > 0) {
      // ---- dQ += dS K of a half tile (dS from tensor memory, K MN-major) ----
      constexpr uint32_t idesc_dq = instr_desc(128, D, 0, 1);
      for (int i = 0, b = 0, ph = 0; i < nvis; ++i) {
        const uint64_t dkm = smem_desc(smem_u32(kv_tiles + (i % STAGES) * 2 * C::kSmallBytes), C::kSmallBytes,
                                       C::kAtomBytes, C::kSwizzle);
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 206);
        for (int hh = 0; hh < 2; ++hh) {
          mbar_wait(b_tfull + 8 * b, ph, &abort_flag, 204);
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 2; ++kk)
              umma_bf16_ts(tmem_dq, tmem_base + 64 * b + 16 * kk, dkm + (2 * hh + kk) * C::kKStep, idesc_dq,
                           (i | hh | kk) != 0);
            umma_commit(b_done + 8 * b);
            if (hh == 1) umma_commit(b_empty + 8 * (i % STAGES));  // every product on this stage has completed
          }
          __syncwarp();
          if (++b == 2) {
            b = 0;
            ph ^= 1;
          }
        }
      }
    }
  } else {
    setmaxnreg_inc<kKvComputeRegs>();
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane, t = PACK ? row0 + (r & 63) : row0 + r, g = r / s.Bk;
    const int hr = PACK ? h + (r >> 6) : h;  // this row's head
    const bool row_ok = t < s.L, row_valid = row_ok && t >= pad0;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float alpha = gate_alpha(gate, hr), beta = 1.f - alpha;
    // this row's record from the pre-pass: nl = -(lse * log2e - log2 weight), nD = -Delta
    float nlL = 0.f, nlS = 0.f, nDL = 0.f, nDS = 0.f;
    if (row_valid) {
      const float *rec =
          reinterpret_cast<const float *>(qstats) + (((int64_t)n * s.H + hr) * Lpad + (t & ~1)) * 4 + (t & 1);
      nlL = rec[0];
      nDL = rec[2];
      nlS = rec[4];
      nDS = rec[6];
    }
    float2 dalL = make_float2(0.f, 0.f), dalS = make_float2(0.f, 0.f);  // sums of P' dP per branch
    const float sc2 = s.scale * kLog2e;
    int b = 0, ph = 0;  // buffer x % 2 of half tile x = 2 i + hh and the parity (x / 2) & 1
    if (nvis > 0) {
      // The resident tiles become first operands in tensor memory: row r of Q (warps 0..3) or of dO
      // (warps 4..7) goes to lane r as it is stored, two bf16 per 32-bit column.
      mbar_wait(b_res, 0, &abort_flag, 208);
      const uint8_t *src = (half ? g_tile : q_tile) + r * C::kRowBytes;
      uint32_t wr[D / 2];
#pragma unroll
      for (int ch = 0; ch < D / 8; ++ch) {
        const int pos = D == 64 ? (ch ^ (r & 7)) : (ch ^ ((r >> 1) & 3));  // the TMA swizzle of the tile
        const uint4 v4 = *reinterpret_cast<const uint4 *>(src + (pos << 4));
        wr[4 * ch] = v4.x; wr[4 * ch + 1] = v4.y; wr[4 * ch + 2] = v4.z; wr[4 * ch + 3] = v4.w;
      }
      const uint32_t ta = (half ? tmem_ga : tmem_qa) + lane_off;
      if constexpr (D == 64) tmem_st32u(ta, wr); else tmem_st16u(ta, wr);
      tmem_wait_st();
      tc_fence_before();
      warp_arrive(b_aready, lane);
    }

    int cls_n = nvis > 0 ? jcls[warp] : 0;
    for (int x = 0; x < 2 * nvis; ++x) {  // half tile x: keys 32 (x % 2) ... of tile list[x / 2]
      const int cls = cls_n;
      if (x + 1 < 2 * nvis) cls_n = jcls[(x + 1) * kComputeWarps + warp];  // ahead of its use
      uint32_t hL = 0u, hS = 0u;  // this thread's 16 keys: keys 32 (x % 2) + 16 half ... of the tile
      bool anyL = cls & 1, anyS = cls & 2, full = true;
      if (cls & 8) {  // mixed: per-lane column masks
        const int i = x >> 1, jt = list[i], f = lflags[i], p0 = jt * 64;
        uint64_t maskL = 0ull, maskS = 0ull;
        if (row_valid) {
          const uint64_t mc = cols_le((causal ? t : s.L - 1) - p0) & cols_ge(pad0 - p0);
          if (f & 1) maskL = mc & expand_block_bits(pq ? rowb[r * nT + jt] : selb[g * nT + jt], s.Bk);
          if (f & 2) maskS = mc & st_key_cols(s, t, p0, causal);
        }
        hL = (uint32_t)(maskL >> (32 * (x & 1) + 16 * half)) & 0xffffu;
        hS = (uint32_t)(maskS >> (32 * (x & 1) + 16 * half)) & 0xffffu;
        anyL = __any_sync(0xffffffffu, hL != 0u);
        anyS = __any_sync(0xffffffffu, hS != 0u);
        full = __all_sync(0xffffffffu, (!anyL || hL == 0xffffu) && (!anyS || hS == 0xffffu));
      }
      const uint32_t tb = tmem_base + 64 * b + lane_off + 16 * half;  // S; dP 32 columns further

      mbar_wait(b_sfull + 8 * b, ph, &abort_flag, 207);
      __syncwarp();
      tc_fence_after();
      uint32_t dw[8];
      if (anyL || anyS) {
        float sv[16], dp[16];
        tmem_ld16(tb, sv);
        tmem_ld16(tb + 32, dp);
        tmem_wait_ld();
        if (!full) dq_tile<true, true, false>(sv, dp, hL, hS, sc2, nlL, nlS, nDL, nDS, dalL, dalS, dw);
        else if (anyL && anyS) dq_tile<true, true, true>(sv, dp, hL, hS, sc2, nlL, nlS, nDL, nDS, dalL, dalS, dw);
        else if (anyL) dq_tile<true, false, true>(sv, dp, hL, hS, sc2, nlL, nlS, nDL, nDS, dalL, dalS, dw);
        else dq_tile<false, true, true>(sv, dp, hL, hS, sc2, nlL, nlS, nDL, nDS, dalL, dalS, dw);
      } else {
#pragma unroll
        for (int c = 0; c < 8; ++c) dw[c] = 0u;
      }
      tmem_st8u(tb, dw);  // dS (bf16 pairs) over the first 8 of this thread's own 16 S columns
      tmem_wait_st();
      tc_fence_before();
      warp_arrive(b_tfull + 8 * b, lane);
      if (++b == 2) {
        b = 0;
        ph ^= 1;
      }
    }

    if (nvis > 0) {
      mbar_wait(b_done + 8, (nvis - 1) & 1, &abort_flag, 209);  // the last half tile used buffer 1
      __syncwarp();
      tc_fence_after();
    }
    float o[OC];
    if (nvis > 0) {
      tmem_ld<OC>(tmem_dq + lane_off + half * OC, o);
      tmem_wait_ld();
    }
    {
      // The rows go to shared memory in the layout a TMA store expects (the K/V stages are free:
      // every load has landed and every MMA has completed); one bulk store then writes whole lines,
      // clipped at L by the hardware.  Padded rows are written as zeros.
      const bool live = nvis > 0 && row_valid;
#pragma unroll
      for (int ch = 0; ch < OC / 8; ++ch) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          w[e] = live ? pack_bf16(o[c] * s.scale, o[c + 1] * s.scale) : 0u;
        }
        store_row_chunk<D>(kv_tiles, r, half * (OC / 8) + ch, make_uint4(w[0], w[1], w[2], w[3]));
      }
      fence_async_smem();
      named_bar_sync(5, kComputeWarps * 32);
      if (tid == 0) {
        tma_store_4d(&tmdq, smem_u32(kv_tiles), 0, row0, h, n);
        tma_store_commit_and_wait();
      }
    }
    // d alpha = sum (P_lt - P_st) dP; a weight of exactly 0 makes its branch's sum 0 and the gate
    // gradient alpha (1 - alpha) d alpha 0 whatever d alpha is
    const float dal = (alpha > 0.f ? (dalL.x + dalL.y) / alpha : 0.f) - (beta > 0.f ? (dalS.x + dalS.y) / beta : 0.f);
    double a = row_valid ? (double)dal : 0.0;  // fixed-shape tree over the warp, then over the warps
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) red[warp] = a;
  }
  tc_fence_before();
  __syncthreads();
  // d alpha partial of this CTA -> first query-block slot of its rows, zeros in the rest
  // (PACK: one partial per head, from the warps of that head's 64 rows)
  if (tid == 0) {
    if (PACK) {
      const int nb = 64 / s.Bk;
      for (int hh = 0; hh < 2; ++hh) {
        double a = 0.0;
        for (int i = 0; i < kComputeWarps; ++i)
          if (((i & 3) >> 1) == hh) a += red[i];  // fixed order
        for (int gq = 0; gq < nb; ++gq)
          if (st * nb + gq < s.M) dalpha_part[((int64_t)n * s.H + h + hh) * s.M + st * nb + gq] = gq == 0 ? a : 0.0;
      }
    } else {
      const int G = 128 / s.Bk;
      double a = 0.0;
      for (int i = 0; i < kComputeWarps; ++i) a += red[i];  // fixed order
      for (int gq = 0; gq < G; ++gq)
        if (st * G + gq < s.M) dalpha_part[(int64_t)u * s.M + st * G + gq] = gq == 0 ? a : 0.0;
    }
  }
  if (nvis == 0 && tid == 0) mbar_wait(b_res, 0, &abort_flag, 221);  // no load may outlive the CTA
  finish(warp, tmem_base, kBwdTmemCols, &abort_flag, status);
}

// ------------------------------------------------------------------------- backward dK, dV
// 16 query columns of one tile for one key row: W^T and dS^T packed to bf16 pairs.  st points at
// the records of these 8 query pairs: {nl_lt(2), -Delta_lt(2)} {nl_st(2), -Delta_st(2)} per pair
// (nl = -(lse * log2e - log2 weight): the branch weight rides in the exponent).  Two columns per
// FMA / ADD / MUL instruction.
template <bool HAS_L, bool HAS_S, bool FULL>
__device__ __forceinline__ void dkdv_tile(const float (&sv)[16], const float (&dp)[16], uint32_t hL,
                                          uint32_t hS, float sc2, const float4 *st, uint32_t (&ww)[8],
                                          uint32_t (&dw)[8]) {
  const float2 sc = make_float2(sc2, sc2);
#pragma unroll
  for (int c = 0; c < 16; c += 2) {
    const float2 s2 = make_float2(sv[c], sv[c + 1]), dp2 = make_float2(dp[c], dp[c + 1]);
    float2 w = make_float2(0.f, 0.f), d = make_float2(0.f, 0.f);
    if (HAS_L) {
      const float4 r = st[c];  // pair c / 2, long-term half of the record
      const float2 x = ffma2(s2, sc, make_float2(r.x, r.y));
      float2 p = make_float2(exp2f(x.x), exp2f(x.y));
      if (!FULL) {
        p.x = bit(hL, c) ? p.x : 0.f;
        p.y = bit(hL, c + 1) ? p.y : 0.f;
      }
      w = p;
      d = fmul2(p, fadd2(dp2, make_float2(r.z, r.w)));
    }
    if (HAS_S) {
      const float4 r = st[c + 1];  // short-term half
      const float2 x = ffma2(s2, sc, make_float2(r.x, r.y));
      float2 p = make_float2(exp2f(x.x), exp2f(x.y));
      if (!FULL) {
        p.x = bit(hS, c) ? p.x : 0.f;
        p.y = bit(hS, c + 1) ? p.y : 0.f;
      }
      w = HAS_L ? fadd2(w, p) : p;
      d = ffma2(p, fadd2(dp2, make_float2(r.z, r.w)), d);
    }
    ww[c >> 1] = pack_bf16(w.x, w.y);
    dw[c >> 1] = pack_bf16(d.x, d.y);
  }
}

template <int D, bool PLAIN>
__global__ void __launch_bounds__(kKvThreads, 2) bwd_dkdv_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmg, Shape s,
    const int32_t *__restrict__ seq_lens, const uint8_t *__restrict__ kmeta,
    const float4 *__restrict__ qstats, const __grid_constant__ CUtensorMap tmdk,
    const __grid_constant__ CUtensorMap tmdv, int32_t *__restrict__ status, int nT) {
  grid_chain_enter();
  using C = Cfg<D>;
  constexpr int STAGES = kKvStages;
  constexpr int OC = D / 2;
  constexpr int kStageBytes = 2 * C::kSmallBytes + kStatBytes;  // Q, dO, row records
  extern __shared__ uint8_t smem_raw[];
  // barriers: full[STAGES], empty[STAGES], res, meta, and per buffer s_full[2], t_full[2], done[2]
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 8];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nKT = (s.L + 127) >> 7;
  // A CTA owns 128 keys of one (batch, key/value head) and collects from every query head of the
  // group.  Early keys have the most visitors, so the grid runs tile-major: every unit's first
  // tile, then every unit's second, ... and the light tiles fill the tail.
  const int nU = s.B * s.Hkv;
  const int kt = (int)(blockIdx.x / nU), uk = (int)(blockIdx.x % nU), n = uk / s.Hkv, hk = uk % s.Hkv;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int key0 = kt * 128, key_last = min(s.L - 1, key0 + 127);
  const int Lpad = nT * 64;

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *k_tile = tiles;
  uint8_t *v_tile = k_tile + C::kBigBytes;
  uint8_t *qg_tiles = v_tile + C::kBigBytes;  // [stage][Q, dO, row records]
  uint8_t *meta = qg_tiles + STAGES * kStageBytes;  // image built by tc_meta_kernel
  const bool causal = PLAIN || s.causal;
  const int pq = PLAIN ? 0 : s.pq;
  const MetaLayout ml = meta_layout(nT, pq);
  const uint64_t *inv64 = reinterpret_cast<const uint64_t *>(meta + ml.rows);  // (selection per query position) [8][nT]
  const uint8_t *invb = meta;                           // [8][nT] bytes: per key block, per query tile
  const uint16_t *list = reinterpret_cast<const uint16_t *>(meta + ml.list);
  const uint8_t *lflags = meta + ml.flags;
  const uint8_t *kcls = meta + ml.jcls;                 // [listed tile][compute warp]

  const uint32_t b_full = smem_u32(&bars[0]), b_empty = smem_u32(&bars[STAGES]);
  const uint32_t b_res = smem_u32(&bars[2 * STAGES]), b_meta = smem_u32(&bars[2 * STAGES + 1]);
  const uint32_t b_sfull = smem_u32(&bars[2 * STAGES + 2]), b_tfull = smem_u32(&bars[2 * STAGES + 4]);
  const uint32_t b_done = smem_u32(&bars[2 * STAGES + 6]);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
    tma_prefetch_desc(&tmg);
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(b_full + 8 * i, 1);
      mbar_init(b_empty + 8 * i, 1);
    }
    mbar_init(b_res, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(b_sfull + 8 * i, 1);
      mbar_init(b_tfull + 8 * i, kComputeWarps);
      mbar_init(b_done + 8 * i, 1);
    }
    mbar_init(b_meta, 1);
    mbar_fence_init();
    // the CTA's tile lists and its resident tiles
    mbar_expect_tx(b_meta, (uint32_t)ml.bytes);
    bulk_load(smem_u32(meta), kmeta + ((size_t)uk * nKT + kt) * ml.bytes, (uint32_t)ml.bytes, b_meta);
    mbar_expect_tx(b_res, 2 * C::kBigBytes);
    tma_load_4d(smem_u32(k_tile), &tmk, b_res, 0, key0, hk, n);
    tma_load_4d(smem_u32(v_tile), &tmv, b_res, 0, key0, hk, n);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), kBwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  mbar_wait(b_meta, 0, &abort_flag, 224);
  // The tile list is the same for every query head of the group (one selection per group): the
  // kernel walks it once per head, item x = (head x / nlist, tile list[x % nlist]).
  const int nlist = *reinterpret_cast<const int *>(meta + ml.counts);
  const int nvis = nlist * s.G;
  const uint32_t tmem_base = tmem_slot;
  // half tile x uses buffer x % 2 at column 64 (x % 2): S^T in its first 32 columns, dP^T behind
  const uint32_t tmem_dv = tmem_base + 128, tmem_dk = tmem_base + 192;

  if (warp >= kComputeWarps) {
    // ===================== three single-thread roles, one warp each =====================
    setmaxnreg_dec<kProducerRegs>();
    if (warp == kComputeWarps && nvis > 0) {
      // ---- loader: K, V once; Q, dO tiles and their row records up to STAGES ahead ----
      int lj = 0, h = hk * s.G;
      for (int j = 0; j < nvis; ++j) {
        const int sj = j % STAGES;
        if (j >= STAGES) mbar_wait(b_empty + 8 * sj, ((j - STAGES) / STAGES) & 1, &abort_flag, 214);
        const uint32_t bar = b_full + 8 * sj;
        const uint32_t qt_ = smem_u32(qg_tiles + sj * kStageBytes);
        if (lj == nlist) { lj = 0; ++h; }  // the next query head of the group walks the same list
        const int row = (int)list[lj++] * 64;
        if (elect_one()) {
          mbar_expect_tx(bar, kStageBytes);
          tma_load_4d(qt_, &tmq, bar, 0, row, h, n);
          tma_load_4d(qt_ + C::kSmallBytes, &tmg, bar, 0, row, h, n);
          bulk_load(qt_ + 2 * C::kSmallBytes, qstats + ((int64_t)n * s.H + h) * Lpad + row, kStatBytes, bar);
        }
        __syncwarp();
      }
    } else if (warp == kComputeWarps + 1 && nvis > 0) {
      // ---- S^T = K Q^T, dP^T = V dO^T of half tile x into buffer x % 2 once the products of half
      // tile x - 2 have read that buffer ----
      constexpr uint32_t idesc_s = instr_desc(128, 32, 0, 0);
      const uint64_t dkd = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dvd = smem_desc(smem_u32(v_tile), 16, C::kAtomBytes, C::kSwizzle);
      mbar_wait(b_res, 0, &abort_flag, 210);
      for (int i = 0, x = 0; i < nvis; ++i) {
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 213);
        for (int hh = 0; hh < 2; ++hh, ++x) {
          const int b = x & 1, ph = (x >> 1) & 1;
          if (x >= 2) mbar_wait(b_done + 8 * b, ph ^ 1, &abort_flag, 212);
          tc_fence_after();
          const uint32_t qt_ = smem_u32(qg_tiles + (i % STAGES) * kStageBytes) + hh * 32 * C::kRowBytes;
          const uint64_t dqd = smem_desc(qt_, 16, C::kAtomBytes, C::kSwizzle);
          const uint64_t dgd = smem_desc(qt_ + C::kSmallBytes, 16, C::kAtomBytes, C::kSwizzle);
          const uint32_t ts = tmem_base + 64 * b;
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) umma_bf16(ts, dkd + 2 * k, dqd + 2 * k, idesc_s, k > 0);
#pragma unroll
            for (int k = 0; k < D / 16; ++k) umma_bf16(ts + 32, dvd + 2 * k, dgd + 2 * k, idesc_s, k > 0);
            umma_commit(b_sfull + 8 * b);
          }
          __syncwarp();
        }
      }
    } else if (warp == kComputeWarps + 2 && nvis > 0) {
      // ---- dV += W^T dO, dK += dS^T Q of a half tile; W^T and dS^T are read from tensor memory,
      // where the compute warps wrote them over the half tile's logits ----
      constexpr uint32_t idesc_o = instr_desc(128, D, 0, 1);
      for (int i = 0, x = 0; i < nvis; ++i) {
        uint8_t *q_tile = qg_tiles + (i % STAGES) * kStageBytes, *g_tile = q_tile + C::kSmallBytes;
        const uint64_t dgm = smem_desc(smem_u32(g_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
        const uint64_t dqm = smem_desc(smem_u32(q_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 215);
        for (int hh = 0; hh < 2; ++hh, ++x) {
          const int b = x & 1, ph = (x >> 1) & 1;
          mbar_wait(b_tfull + 8 * b, ph, &abort_flag, 211);
          tc_fence_after();
          const uint32_t tb = tmem_base + 64 * b;
          if (elect_one()) {
            // 16 queries per step: the bf16 pairs of the warps of column half kk, 8 columns
#pragma unroll
            for (int kk = 0; kk < 2; ++kk)
              umma_bf16_ts(tmem_dv, tb + 16 * kk, dgm + (2 * hh + kk) * C::kKStep, idesc_o, (x | kk) != 0);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk)
              umma_bf16_ts(tmem_dk, tb + 32 + 16 * kk, dqm + (2 * hh + kk) * C::kKStep, idesc_o, (x | kk) != 0);
            umma_commit(b_done + 8 * b);
            if (hh == 1) umma_commit(b_empty + 8 * (i % STAGES));  // every product on this stage has completed
          }
          __syncwarp();
        }
      }
    }
  } else {
    setmaxnreg_inc<kKvComputeRegs>();
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane, p = key0 + r, g = r / s.Bk;
    const bool row_ok = p < s.L, row_valid = row_ok && p >= pad0;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float sc2 = s.scale * kLog2e;

    int li = 0;
    for (int i = 0, x = 0; i < nvis; ++i) {
      if (li == nlist) li = 0;
      const int qt = list[li], f = lflags[li], t0 = qt * 64;
      const uint8_t *cls2 = kcls + li * 16 + warp;  // classes of the tile's two half tiles for this warp
      ++li;
      uint64_t maskL = 0ull, maskS = 0ull;
      if (cls2[0] == 8 || cls2[8] == 8) {  // a mixed half tile: per-lane column masks
        if (row_valid) {
          const uint64_t mc = cols_ge((causal ? p : pad0) - t0) & cols_le(s.L - 1 - t0);
          if (f & 1) maskL = mc & (pq ? inv64[g * nT + qt] : expand_block_bits(invb[g * nT + qt], s.Bk));
          if (f & 2) maskS = mc & st_query_cols(s, p, t0, causal);
        }
      }
      mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 216);  // the row records have landed
      const float4 *stt = reinterpret_cast<const float4 *>(qg_tiles + (i % STAGES) * kStageBytes + 2 * C::kSmallBytes);
      // A half tile = 32 queries; this thread's 16 columns of it are queries 32 hh + 16 half ...
      // W^T and dS^T go, as bf16 pairs, over the first 8 of the thread's own 16 columns of S^T / dP^T.
#pragma unroll
      for (int hh = 0; hh < 2; ++hh, ++x) {
        const int b = x & 1, ph = (x >> 1) & 1, c0 = 32 * hh + 16 * half;
        const int cls = cls2[8 * hh];
        uint32_t hL = 0u, hS = 0u;
        bool anyL = (cls & 1) != 0, anyS = (cls & 2) != 0, full = true;
        if (cls == 8) {
          hL = (uint32_t)(maskL >> c0) & 0xffffu;
          hS = (uint32_t)(maskS >> c0) & 0xffffu;
          anyL = __any_sync(0xffffffffu, hL != 0u);
          anyS = __any_sync(0xffffffffu, hS != 0u);
          full = __all_sync(0xffffffffu, (!anyL || hL == 0xffffu) && (!anyS || hS == 0xffffu));
        }
        const uint32_t tb = tmem_base + 64 * b + lane_off + 16 * half;
        mbar_wait(b_sfull + 8 * b, ph, &abort_flag, 217);
        __syncwarp();
        tc_fence_after();
        uint32_t ww[8], dw[8];
        if (anyL || anyS) {
          float sv[16], dp[16];
          tmem_ld16(tb, sv);
          tmem_ld16(tb + 32, dp);
          tmem_wait_ld();
          const float4 *sq = stt + c0;  // 8 pairs x 2 float4
          if (!full) dkdv_tile<true, true, false>(sv, dp, hL, hS, sc2, sq, ww, dw);
          else if (anyL && anyS) dkdv_tile<true, true, true>(sv, dp, hL, hS, sc2, sq, ww, dw);
          else if (anyL) dkdv_tile<true, false, true>(sv, dp, hL, hS, sc2, sq, ww, dw);
          else dkdv_tile<false, true, true>(sv, dp, hL, hS, sc2, sq, ww, dw);
        } else {
#pragma unroll
          for (int c = 0; c < 8; ++c) { ww[c] = 0u; dw[c] = 0u; }
        }
        tmem_st8u(tb, ww);
        tmem_st8u(tb + 32, dw);
        tmem_wait_st();
        tc_fence_before();
        warp_arrive(b_tfull + 8 * b, lane);
      }
    }

    if (nvis > 0) {
      mbar_wait(b_done + 8, (nvis - 1) & 1, &abort_flag, 218);  // the last half tile used buffer 1
      __syncwarp();
      tc_fence_after();
    }
    float ov[OC], okk[OC];
    if (nvis > 0) {
      tmem_ld<OC>(tmem_dv + lane_off + half * OC, ov);
      tmem_ld<OC>(tmem_dk + lane_off + half * OC, okk);
      tmem_wait_ld();
    }
    {
      // staged in the (now free) Q/dO stages, then two whole-line bulk stores clipped at L
      const bool live = nvis > 0 && row_valid;
      uint8_t *sv_t = qg_tiles, *sk_t = qg_tiles + C::kBigBytes;
#pragma unroll
      for (int ch = 0; ch < OC / 8; ++ch) {
        uint32_t wv[4], wk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          wv[e] = live ? pack_bf16(ov[c], ov[c + 1]) : 0u;
          wk[e] = live ? pack_bf16(okk[c] * s.scale, okk[c + 1] * s.scale) : 0u;
        }
        store_row_chunk<D>(sv_t, r, half * (OC / 8) + ch, make_uint4(wv[0], wv[1], wv[2], wv[3]));
        store_row_chunk<D>(sk_t, r, half * (OC / 8) + ch, make_uint4(wk[0], wk[1], wk[2], wk[3]));
      }
      fence_async_smem();
      named_bar_sync(5, kComputeWarps * 32);
      if (tid == 0) {
        tma_store_4d(&tmdv, smem_u32(sv_t), 0, key0, hk, n);
        tma_store_4d(&tmdk, smem_u32(sk_t), 0, key0, hk, n);
        tma_store_commit_and_wait();
      }
    }
  }
  if (nvis == 0 && tid == 0) mbar_wait(b_res, 0, &abort_flag, 222);  // no load may outlive the CTA
  finish(warp, tmem_base, kBwdTmemCols, &abort_flag, status);
}

}  // namespace

template <int D>
int launch_bwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, const void *out_lt,
                    const void *out_st, const float *lse, const void *dout, void *dq, void *dk,
                    void *dv, const Workspace &ws, cudaStream_t st, int branches, const float4 *records) {
  typedef __nv_bfloat16 bf;
  using C = Cfg<D>;
  CUtensorMap q128, k64, v64, g128, q64, k128, v128, g64, tdq, tdk, tdv;
  // (head-packed dQ kernel: a query-side box is 64 positions of two heads)
  const int qrows = s.pack ? 64 : 128, qheads = s.pack ? 2 : 1;
  if (make_tensor_map(&q128, q, s, qrows, false, qheads) || make_tensor_map(&k64, k, s, 64, true) ||
      make_tensor_map(&v64, v, s, 64, true) || make_tensor_map(&g128, dout, s, qrows, false, qheads) ||
      make_tensor_map(&q64, q, s, 64) || make_tensor_map(&k128, k, s, 128, true) ||
      make_tensor_map(&v128, v, s, 128, true) || make_tensor_map(&g64, dout, s, 64) ||
      make_tensor_map(&tdq, dq, s, qrows, false, qheads) || make_tensor_map(&tdk, dk, s, 128, true) ||
      make_tensor_map(&tdv, dv, s, 128, true))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const unsigned grid = (unsigned)nST * (unsigned)(s.B * s.H);
  const size_t smem_dq = 1024 + 2 * C::kBigBytes + kDqStages * 2 * C::kSmallBytes + meta_bytes(nT, s.pq);
  const size_t smem_kv =
      1024 + 2 * C::kBigBytes + kKvStages * (2 * C::kSmallBytes + kStatBytes) + meta_bytes(nT, s.pq);
  const bool plain = s.causal && !s.pq;
  auto kern_dq = s.pack ? (plain ? bwd_dq_tc_kernel<D, true, true> : bwd_dq_tc_kernel<D, false, true>)
                        : (plain ? bwd_dq_tc_kernel<D, true, false> : bwd_dq_tc_kernel<D, false, false>);
  auto kern_kv = plain ? bwd_dkdv_tc_kernel<D, true> : bwd_dkdv_tc_kernel<D, false>;
  if (cudaFuncSetAttribute(kern_dq, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_dq) != cudaSuccess ||
      cudaFuncSetAttribute(kern_kv, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kv) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  if (!(s.reuse_lists && branches == 3 && !records))  // (the passes of the input-dependent gate build their own)
    if (int rc = launch_tc_meta(s, seq_lens, idx, ws.qmeta, ws.kmeta, st, branches)) return rc;
  const float4 *rec = records ? records : ws.qstats;
  if (!records) {
    LaunchScope ls(K_BWD_PREP, st);
    const int Lpad = nT * 64, rpb = 256 / (D / 8);
    const unsigned gp = (unsigned)(s.B * s.H) * (unsigned)((Lpad + rpb - 1) / rpb);
    launch_chained(bwd_prep_kernel<D>, dim3(gp), dim3(256), 0, st, s, gate, seq_lens, (const bf *)out_lt,
                   (const bf *)out_st, lse, (const bf *)dout, ws.qstats, Lpad);
  }
  {
    LaunchScope ls(K_BWD_DQ_TC, st);
    const unsigned grid_q = s.pack ? (unsigned)nT * (unsigned)(s.B * (s.H / 2)) : grid;
    launch_chained(kern_dq, dim3(grid_q), dim3(kKvThreads), smem_dq, st, q128, k64, v64, g128, s, gate, seq_lens,
                   (const uint8_t *)ws.qmeta, tdq, rec, ws.dalpha, ws.status_bwd, nT);
  }
  {
    LaunchScope ls(K_BWD_DKDV_TC, st);
    const unsigned grid_k = (unsigned)nST * (unsigned)(s.B * s.Hkv);
    launch_chained(kern_kv, dim3(grid_k), dim3(kKvThreads), smem_kv, st, q64, k128, v128, g64, s, seq_lens,
                   (const uint8_t *)ws.kmeta, rec, tdk, tdv, ws.status_bwd, nT);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

template int launch_bwd_tc_t<32>(const Shape &, const void *, const void *, const void *, const float *,
                                 const int32_t *, const int32_t *, const void *, const void *,
                                 const float *, const void *, void *, void *, void *, const Workspace &,
                                 cudaStream_t, int, const float4 *);
template int launch_bwd_tc_t<64>(const Shape &, const void *, const void *, const void *, const float *,
                                 const int32_t *, const int32_t *, const void *, const void *,
                                 const float *, const void *, void *, void *, void *, const Workspace &,
                                 cudaStream_t, int, const float4 *);

}  // namespace tc
}  // namespace blossom
