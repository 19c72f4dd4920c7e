// Tensor-core forward of the fused two-branch attention (bf16 storage, fp32 accumulate).
//
// A CTA owns 128 query rows (128 / Bk query blocks) and walks a list of items, one 64-key tile of
// one branch each: first the tiles any of its query blocks selected (Eq. 14, 16), then the tiles
// its rows reach through the window (Eq. 15, 17).  One accumulator serves both phases: when the
// long-term phase ends its rows are parked in shared memory and the short-term phase starts the
// accumulator afresh.  A tile that belongs to both branches is visited once per phase.
//
// CTA = 384 threads.  Warps 0..7 are softmax warps: warp w owns TMEM lane quarter w % 4 (32 query
// rows) and column half w / 4 (32 of the 64 keys of a tile); both threads of a row look at all 64
// logits for the row maximum, so they keep identical running maxima without talking to each
// other, and each keeps the partial sum of its own columns.  Warp 8 lane 0 loads K/V tiles (TMA),
// warp 9 lane 0 issues S = Q K^T, warp 10 lane 0 issues O += P V with P read from tensor memory.
// Registers move from the three single-thread warps to the softmax warps (setmaxnreg).
//
// Tensor memory (256 columns): S buffers [0,64) [64,128), probability buffers (bf16 pairs)
// [128,160) [160,192), accumulator [192,192+D).  Item i uses S buffer and probability buffer
// i % 2, so that S(i+1) is computed and O += P(i-1) V runs while the softmax warps work on item i:
//
//   loader   : stage j <- K, V of item j once O += P V of item j - STAGES has completed
//   S issuer : wait K(i) and "S(i-2) is in registers" -> S(i) -> commit s_full[i%2]
//   softmax  : wait s_full -> tcgen05.ld 64 logits -> arrive s_empty -> online softmax of the row
//              (maximum raised, and the accumulator rescaled, only when it grows by > 2^8)
//              -> wait "O += P(i-2) V done" -> tcgen05.st P -> arrive t_full[i%2]
//   PV issuer: wait t_full -> O += P(i) V -> commit done[i%2], release the stage
//
// Every barrier that counts warp arrivals exists once per item parity: a warp can be one item
// ahead of the slowest warp, never two.  Rows whose query block does not need a tile skip its
// exponentials (warp-uniform) and contribute zero rows to P.
// Epilogue: normalise, gate mix (Eq. 19), store out / out_lt / out_st / lse.
// Every wait is bounded (tc_common.cuh).
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

constexpr float kRescaleThreshold = 8.0f;  // log2 units
// warps 0..7 softmax (warp w: TMEM lane quarter w % 4, column half w / 4); 8 loader, 9 S issuer,
// 10 PV issuer, 11 spare
constexpr int kFwdThreads = 384;
constexpr int kSoftmaxWarps = 8;
constexpr int kProducerRegs = 32, kSoftmaxRegs = 104;  // 256 * 104 + 128 * 32 = 384 * 80
constexpr int kFwdStages = 3;
constexpr uint32_t kFwdTmemCols = 256;

__device__ __forceinline__ bool bit(uint32_t w, int c) { return (w >> c) & 1u; }

// maximum of 32 logits (those whose bit is set, all of them when FULL)
template <bool FULL>
__device__ __forceinline__ float half_max(const float (&v)[32], uint32_t bits) {
  float a0 = -INFINITY, a1 = -INFINITY;
#pragma unroll
  for (int c = 0; c < 32; c += 4) {
    float x[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) x[e] = (FULL || bit(bits, c + e)) ? v[c + e] : -INFINITY;
    a0 = max3(a0, x[0], x[1]);
    a1 = max3(a1, x[2], x[3]);
  }
  return fmaxf(a0, a1);
}

// probabilities of 32 logits relative to the running maximum (nm = -m, log2 units), packed as
// bf16 pairs; their sum is added to l
template <bool FULL>
__device__ __forceinline__ void half_probs(const float (&sv)[32], uint32_t bits, float sc2, float nm,
                                           float &l, uint32_t (&pk)[16]) {
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int c = 0; c < 32; c += 2) {
    float a = exp2f(fmaf(sv[c], sc2, nm)), b = exp2f(fmaf(sv[c + 1], sc2, nm));
    if (!FULL) {
      a = bit(bits, c) ? a : 0.f;
      b = bit(bits, c + 1) ? b : 0.f;
    }
    s0 += a;
    s1 += b;
    pk[c >> 1] = pack_bf16(a, b);
  }
  l += s0 + s1;
}

// multiply this thread's N accumulator columns by fac (all lanes of the warp take part)
template <int N>
__device__ __forceinline__ void rescale_acc(uint32_t taddr, float fac) {
  float o[N];
  tmem_ld<N>(taddr, o);
  tmem_wait_ld();
#pragma unroll
  for (int c = 0; c < N; ++c) o[c] *= fac;
  tmem_st<N>(taddr, o);
  tmem_wait_st();
}

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 2) fwd_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, Shape s, const float *__restrict__ gate,
    const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ idx,
    __nv_bfloat16 *__restrict__ out, __nv_bfloat16 *__restrict__ out_lt,
    __nv_bfloat16 *__restrict__ out_st, float *__restrict__ lse, int32_t *__restrict__ status,
    int nT) {
  using C = Cfg<D>;
  constexpr int STAGES = kFwdStages;
  constexpr int OC = D / 2;  // accumulator columns per thread
  extern __shared__ uint8_t smem_raw[];
  // barriers: full[STAGES], empty[STAGES], res, then pairs by item parity: s_full, s_empty,
  // t_full, done
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 9];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int nvis_s, nL_s, nS_s;
  __shared__ float2 xl[2][128];  // [column half][row]: partial sums (lt, st) for the epilogue

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
  float *park = reinterpret_cast<float *>(kv_tiles + STAGES * 2 * C::kSmallBytes);  // [D][128]
  uint8_t *meta = reinterpret_cast<uint8_t *>(park + D * 128);
  uint32_t *selw = reinterpret_cast<uint32_t *>(meta);
  uint8_t *selb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ((8 * nT + 15) / 16) * 16);
  uint8_t *lflags = reinterpret_cast<uint8_t *>(list + nT);
  uint16_t *items = reinterpret_cast<uint16_t *>(meta + ((11 * nT + 15) / 16) * 16);  // [2 nT]

  const uint32_t b_full = smem_u32(&bars[0]), b_empty = smem_u32(&bars[STAGES]);
  const uint32_t b_res = smem_u32(&bars[2 * STAGES]);
  const uint32_t b_sfull = smem_u32(&bars[2 * STAGES + 1]), b_sempty = smem_u32(&bars[2 * STAGES + 3]);
  const uint32_t b_tfull = smem_u32(&bars[2 * STAGES + 5]), b_done = smem_u32(&bars[2 * STAGES + 7]);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;  // an earlier CTA timed out: do not wait again
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(b_full + 8 * i, 1);
      mbar_init(b_empty + 8 * i, 1);
    }
    mbar_init(b_res, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(b_sfull + 8 * i, 1);
      mbar_init(b_sempty + 8 * i, kSoftmaxWarps);
      mbar_init(b_tfull + 8 * i, kSoftmaxWarps);
      mbar_init(b_done + 8 * i, 1);
    }
    mbar_fence_init();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), kFwdTmemCols);
    tmem_relinquish();
  }
  build_query_major_list(s, idx, u, st, pad0, nT, selw, selb, list, lflags, &nvis_s);
  __syncthreads();
  if (warp == 0) {  // items: the tiles of the long-term phase, then those of the short-term phase
    const int nv = nvis_s;
    int count = 0, nl = 0;
    for (int ph = 1; ph <= 2; ++ph) {
      for (int base = 0; base < nv; base += 32) {
        const int j = base + lane;
        const bool on = j < nv && (lflags[j] & ph);
        const unsigned bal = __ballot_sync(0xffffffffu, on);
        if (on) items[count + __popc(bal & ((1u << lane) - 1u))] = list[j];
        count += __popc(bal);
      }
      if (ph == 1) nl = count;
    }
    if (lane == 0) {
      nL_s = nl;
      nS_s = count - nl;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const int nL = nL_s, nS = nS_s, nI = nL + nS;
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_p = tmem_base + 128, tmem_o = tmem_base + 192;

  if (warp >= kSoftmaxWarps) {
    // ===================== three single-thread roles, one warp each =====================
    setmaxnreg_dec<kProducerRegs>();
    if (warp == kSoftmaxWarps && lane == 0 && nI > 0) {
      // ---- loader: K/V tiles, up to STAGES ahead of their consumers ----
      mbar_expect_tx(b_res, C::kBigBytes);
      tma_load_4d(smem_u32(q_tile), &tmq, b_res, 0, row0, h, n);
      for (int j = 0; j < nI; ++j) {
        const int sj = j % STAGES;
        if (j >= STAGES) mbar_wait(b_empty + 8 * sj, ((j - STAGES) / STAGES) & 1, &abort_flag, 105);
        const uint32_t bar = b_full + 8 * sj;
        uint8_t *kt = kv_tiles + sj * 2 * C::kSmallBytes;
        mbar_expect_tx(bar, 2 * C::kSmallBytes);
        tma_load_4d(smem_u32(kt), &tmk, bar, 0, (int)items[j] * 64, h, n);
        tma_load_4d(smem_u32(kt + C::kSmallBytes), &tmv, bar, 0, (int)items[j] * 64, h, n);
      }
    } else if (warp == kSoftmaxWarps + 1 && lane == 0 && nI > 0) {
      // ---- S(i) = Q K^T into S buffer i % 2 once the softmax warps hold S(i-2) in registers ----
      constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
      const uint64_t dq = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      mbar_wait(b_res, 0, &abort_flag, 101);
      for (int i = 0; i < nI; ++i) {
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 102);
        if (i >= 2) mbar_wait(b_sempty + 8 * (i & 1), ((i - 2) >> 1) & 1, &abort_flag, 103);
        tc_fence_after();
        uint8_t *k_tile = kv_tiles + (i % STAGES) * 2 * C::kSmallBytes;
        const uint64_t dk = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
        const uint32_t ts = tmem_s + 64 * (i & 1);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) umma_bf16(ts, dq + 2 * k, dk + 2 * k, idesc_s, k > 0);
        umma_commit(b_sfull + 8 * (i & 1));
      }
    } else if (warp == kSoftmaxWarps + 2 && lane == 0 && nI > 0) {
      // ---- O += P(i) V once the probabilities of item i are in tensor memory ----
      constexpr uint32_t idesc_pv = instr_desc(128, D, 0, 1);
      for (int i = 0; i < nI; ++i) {
        uint8_t *v_tile = kv_tiles + (i % STAGES) * 2 * C::kSmallBytes + C::kSmallBytes;
        const uint64_t dv = smem_desc(smem_u32(v_tile), C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
        const uint32_t tp = tmem_p + 32 * (i & 1);
        const int first = (i == 0 || i == nL) ? 0 : 1;  // a phase starts the accumulator afresh
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 106);
        mbar_wait(b_tfull + 8 * (i & 1), (i >> 1) & 1, &abort_flag, 104);
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_bf16_ts(tmem_o, tp + 8 * k, dv + k * C::kKStep, idesc_pv, (first | k) != 0);
        umma_commit(b_done + 8 * (i & 1));
        umma_commit(b_empty + 8 * (i % STAGES));  // S(i) completed before the softmax warps read it
      }
    }
  } else {
    // ================================ softmax =================================
    setmaxnreg_inc<kSoftmaxRegs>();
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane, t = row0 + r, g = r / s.Bk;
    const bool row_ok = t < s.L;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    // Both threads of a row keep the same running maximum (each looks at all 64 logits of a tile)
    // and the partial sum of their own 32 columns.
    float m = -INFINITY, l = 0.f, mL = -INFINITY, lL = 0.f;
    bool zeroA = false, zeroB = false;  // this thread's columns of probability buffer 0 / 1 hold zeros
    int acc = 0;                        // the current phase has written the accumulator
    const float sc2 = s.scale * kLog2e;
    const int t_lo = row0 + quarter * 32;            // first row of this warp
    const bool uni = s.Bk >= 32;                     // the warp's rows share one query block
    const int gw = (quarter * 32) / s.Bk;
    const uint32_t allbits = (1u << (64 / s.Bk)) - 1u;
    const bool rows_all = t_lo >= pad0 && t_lo + 31 < s.L;

    for (int i = 0; i < nI; ++i) {
      const bool isL = i < nL;
      const int jt = items[i], p0 = jt * 64, par = i & 1;
      // Classify the tile for this warp with warp-uniform integer tests (0 = no row needs it,
      // 1 = every row sees all 64 keys, 2 = mixed); per-lane column masks only for mixed tiles.
      const bool some = p0 <= t_lo + 31 && p0 + 63 >= pad0 && t_lo + 31 >= pad0 && t_lo < s.L;
      const bool inner = rows_all && p0 >= pad0 && p0 + 63 <= t_lo;  // valid and causal for every row
      int cls = 0;
      if (some) {
        if (isL) {
          if (!uni) cls = 2;
          else {
            const uint32_t bits = selb[gw * nT + jt];
            cls = bits == 0u ? 0 : ((inner && bits == allbits) ? 1 : 2);
          }
        } else if (p0 + 63 >= t_lo - s.window + 1) {
          cls = (inner && p0 >= t_lo + 31 - s.window + 1) ? 1 : 2;
        }
      }
      uint64_t mask = 0ull;
      bool doB = cls == 1, fullB = cls == 1;
      if (cls == 2) {
        if (row_ok) {
          mask = cols_le(t - p0) & cols_ge(pad0 - p0);
          mask &= isL ? expand_block_bits(selb[g * nT + jt], s.Bk) : cols_ge(t - s.window + 1 - p0);
        }
        doB = __any_sync(0xffffffffu, mask != 0ull);
        fullB = __all_sync(0xffffffffu, mask == ~0ull);
      }

      mbar_wait(b_sfull + 8 * par, (i >> 1) & 1, &abort_flag, 107);
      __syncwarp();
      tc_fence_after();
      float sv[32];         // this thread's 32 logits
      float ox = -INFINITY; // maximum of the other 32 logits of the row
      if (doB) {
        float ov[32];
        tmem_ld32(tmem_s + 64 * par + lane_off + half * 32, sv);
        tmem_ld32(tmem_s + 64 * par + lane_off + (half ^ 1) * 32, ov);
        tmem_wait_ld();
        ox = fullB ? half_max<true>(ov, 0u) : half_max<false>(ov, (uint32_t)(mask >> ((half ^ 1) * 32)));
      }
      tc_fence_before();
      warp_arrive(b_sempty + 8 * par, lane);

      bool waited_prev = i == 0;  // the MMAs of item i-1 have completed
      if (i == nL && nL > 0) {
        // End of the long-term phase: park its accumulator rows and statistics; the first P V
        // product of the short-term phase overwrites the accumulator.
        mbar_wait(b_done + 8 * ((i - 1) & 1), ((i - 1) >> 1) & 1, &abort_flag, 111);
        __syncwarp();
        tc_fence_after();
        waited_prev = true;
        float o[OC];
        tmem_ld<OC>(tmem_o + lane_off + half * OC, o);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < OC; ++c) park[(half * OC + c) * 128 + r] = o[c];
        mL = m;
        lL = l;
        m = -INFINITY;
        l = 0.f;
        acc = 0;
      }

      const uint32_t bits = (uint32_t)(mask >> (half * 32));
      uint32_t pk[16];
      float fac = 1.f;
      bool need = false;
      if (doB) {
        const float own = fullB ? half_max<true>(sv, 0u) : half_max<false>(sv, bits);
        const float mt = fmaxf(own, ox) * sc2;
        need = mt > m + kRescaleThreshold;  // also true on the row's first keys
        if (need) {
          fac = exp2f(m - mt);
          l *= fac;
          m = mt;
        }
        if (fullB) half_probs<true>(sv, 0u, sc2, -m, l, pk);
        else half_probs<false>(sv, bits, sc2, -m, l, pk);
      }
      // Probability buffer i % 2 was last read by the MMAs of item i-2; rescaling the accumulator
      // needs those of item i-1.
      const bool rescale = doB && acc && __any_sync(0xffffffffu, need);
      if (rescale && !waited_prev) {
        mbar_wait(b_done + 8 * ((i - 1) & 1), ((i - 1) >> 1) & 1, &abort_flag, 108);
      } else if (i >= 2) {
        mbar_wait(b_done + 8 * par, ((i - 2) >> 1) & 1, &abort_flag, 109);
      }
      __syncwarp();
      tc_fence_after();
      const uint32_t t_p = tmem_p + 32 * par + lane_off + half * 16;
      const bool zero = par ? zeroB : zeroA;
      if (doB) {
        if (rescale) rescale_acc<OC>(tmem_o + lane_off + half * OC, fac);
        tmem_st16u(t_p, pk);
      } else if (!zero) {
#pragma unroll
        for (int c = 0; c < 16; ++c) pk[c] = 0u;
        tmem_st16u(t_p, pk);
      }
      if (par) zeroB = !doB; else zeroA = !doB;
      tmem_wait_st();
      tc_fence_before();
      warp_arrive(b_tfull + 8 * par, lane);
      acc = 1;
    }

    // ---- epilogue ----
    if (nI > 0) {
      mbar_wait(b_done + 8 * ((nI - 1) & 1), ((nI - 1) >> 1) & 1, &abort_flag, 110);
      __syncwarp();
      tc_fence_after();
    }
    float mS = -INFINITY, lS = 0.f;
    if (nS > 0) { mS = m; lS = l; } else { mL = m; lL = l; }
    xl[half][r] = make_float2(lL, lS);
    named_bar_sync(1 + quarter, 64);
    {
      const float2 a = xl[0][r], b = xl[1][r];  // fixed order: both threads get the same sums
      lL = a.x + b.x;
      lS = a.y + b.y;
    }
    const float alpha = gate_alpha(gate, h), beta = 1.f - alpha;
    const float iL = lL > 0.f ? 1.f / lL : 0.f, iS = lS > 0.f ? 1.f / lS : 0.f;
    const bool haveL = nL > 0 && lL > 0.f, haveS = nS > 0 && lS > 0.f;
    const bool parked = nL > 0 && nS > 0;  // long-term rows in shared memory, short-term in TMEM
    const int64_t ro = row_offset(s, n, h, row_ok ? t : 0) + half * OC;
    float o[OC];
    if (nI > 0) {
      tmem_ld<OC>(tmem_o + lane_off + half * OC, o);
      tmem_wait_ld();
    }
    if (row_ok) {
#pragma unroll
      for (int ch = 0; ch < OC / 8; ++ch) {
        uint32_t wo[4], wl[4], ws[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
          if (haveL) {
            a0 = (parked ? park[(half * OC + c) * 128 + r] : o[c]) * iL;
            a1 = (parked ? park[(half * OC + c + 1) * 128 + r] : o[c + 1]) * iL;
          }
          if (haveS) {
            b0 = o[c] * iS;
            b1 = o[c + 1] * iS;
          }
          wl[e] = pack_bf16(a0, a1);
          ws[e] = pack_bf16(b0, b1);
          wo[e] = pack_bf16(alpha * a0 + beta * b0, alpha * a1 + beta * b1);
        }
        const int64_t off = ro + ch * 8;
        *reinterpret_cast<uint4 *>(out + off) = make_uint4(wo[0], wo[1], wo[2], wo[3]);
        if (out_lt) *reinterpret_cast<uint4 *>(out_lt + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
        if (out_st) *reinterpret_cast<uint4 *>(out_st + off) = make_uint4(ws[0], ws[1], ws[2], ws[3]);
      }
    }
    if (row_ok && lse && half == 0) {
      const int64_t BHL = (int64_t)s.B * s.H * s.L;
      lse[(int64_t)u * s.L + t] = lL > 0.f ? (mL + log2f(lL)) * kLn2 : 0.f;
      lse[BHL + (int64_t)u * s.L + t] = lS > 0.f ? (mS + log2f(lS)) * kLn2 : 0.f;
    }
  }
  finish(warp, tmem_base, kFwdTmemCols, &abort_flag, status);
}

}  // namespace

template <int D>
int launch_fwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt,
                    void *out_st, float *lse, const Workspace &ws, cudaStream_t st) {
  using C = Cfg<D>;
  CUtensorMap tq, tk, tv;
  if (make_tensor_map(&tq, q, s, 128) || make_tensor_map(&tk, k, s, 64) || make_tensor_map(&tv, v, s, 64))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const size_t smem = 1024 + C::kBigBytes + kFwdStages * 2 * C::kSmallBytes + (size_t)s.D * 128 * sizeof(float) + meta_bytes(nT);
  if (cudaFuncSetAttribute(fwd_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  const unsigned grid = (unsigned)nST * (unsigned)(s.B * s.H);
  {
    LaunchScope ls(K_FWD_TC, st);
    fwd_tc_kernel<D><<<grid, kFwdThreads, smem, st>>>(tq, tk, tv, s, gate, seq_lens, idx,
                                                     (__nv_bfloat16 *)out, (__nv_bfloat16 *)out_lt,
                                                     (__nv_bfloat16 *)out_st, lse, ws.status, nT);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

template int launch_fwd_tc_t<32>(const Shape &, const void *, const void *, const void *, const float *,
                                 const int32_t *, const int32_t *, void *, void *, void *, float *,
                                 const Workspace &, cudaStream_t);
template int launch_fwd_tc_t<64>(const Shape &, const void *, const void *, const void *, const float *,
                                 const int32_t *, const int32_t *, void *, void *, void *, float *,
                                 const Workspace &, cudaStream_t);

}  // namespace tc
}  // namespace blossom
