// Tensor-core forward of the fused two-branch attention (bf16 storage, fp32 accumulate).
//
// A CTA owns 128 query rows (128 / Bk query blocks) and walks a list of items, one 64-key tile of
// one branch each: first the tiles any of its query blocks selected (Eq. 14, 16), then the tiles
// its rows reach through the window (Eq. 15, 17).  One accumulator serves both phases: when the
// long-term phase ends each thread parks its row in registers and the short-term phase starts the
// accumulator afresh.  A tile that belongs to both branches is visited once per phase.
//
// CTA = 256 threads.  Warps 0..3 are softmax warps (thread = query row = TMEM lane: no exchange
// between threads in the loop).  Warps 4, 5, 6 stay converged and one elected lane of each loads
// K/V tiles (TMA), issues S = Q K^T, and issues O += P V with P read from tensor memory.
// Registers move from those warps to the softmax warps (setmaxnreg).
//
// Tensor memory (256 columns): three logits / probability buffers [0,64) [64,128) [128,192) and
// the accumulator [192,192+D).  Item i uses buffer i % 3: S(i) = Q K^T lands there as fp32, each
// softmax thread reads its row and writes the row's probabilities (bf16 pairs) over the first 32
// columns of the same buffer, and O += P(i) V reads them from there.  A row's probabilities only
// replace that row's own logits, so the softmax warps wait for one thing per item:
//
//   loader   : stage j <- K, V of item j once O += P V of item j - STAGES has completed
//   S issuer : wait K(i) and "O += P(i-3) V done" (the buffer is free) -> S(i) -> commit s_full[i%3]
//   softmax  : wait s_full -> tcgen05.ld 64 logits -> online softmax of the row (maximum raised,
//              and the accumulator rescaled, only when it grows by > 2^8) -> tcgen05.st P over the
//              logits -> arrive t_full[i%3]
//   PV issuer: wait t_full -> O += P(i) V -> commit done[i%3], release the stage
//
// so S(i+1) and S(i+2) are computed, and O += P(i-1) V runs, while the softmax warps work on item
// i.  A softmax warp cannot pass s_full(i+3) before every warp has arrived on t_full(i), so a
// barrier never collects two arrivals of one warp in one phase.  Rows whose query block does not
// need a tile skip its exponentials (warp-uniform) and write zero rows.
// Epilogue: normalise, gate mix (Eq. 19), stage the rows in shared memory and write out / out_lt /
// out_st with whole-line TMA stores; lse directly.
// Every wait is bounded (tc_common.cuh).
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kFwdThreads = 256;  // warps 0..3 softmax; 4 loader, 5 S issuer, 6 PV issuer, 7 spare
constexpr int kSoftmaxWarps = 4;
constexpr int kProducerRegs = 40, kSoftmaxRegs = 216;  // (128 - 40) * 128 = (216 - 128) * 128
constexpr int kFwdStages = 5;
constexpr uint32_t kFwdTmemCols = 256;

// maximum of a row's 64 logits (those whose mask bit is set, all of them when FULL)
template <bool FULL>
__device__ __forceinline__ float row_max(const float (&v)[64], uint64_t mask) {
  const uint32_t mlo = (uint32_t)mask, mhi = (uint32_t)(mask >> 32);
  float a[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) a[e] = -INFINITY;
#pragma unroll
  for (int c = 0; c < 64; c += 16) {
    float x[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const int cc = c + e;
      x[e] = (FULL || (((cc < 32 ? mlo : mhi) >> (cc & 31)) & 1u)) ? v[cc] : -INFINITY;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = max3(a[e], x[2 * e], x[2 * e + 1]);
  }
  return fmaxf(max3(a[0], a[1], a[2]), max3(max3(a[3], a[4], a[5]), a[6], a[7]));
}

// probabilities of a row's 64 logits relative to the running maximum (nm = -m, log2 units),
// packed as bf16 pairs; their sum is added to l.  Two logits per FMA / ADD instruction.
template <bool FULL>
__device__ __forceinline__ void row_probs(const float (&sv)[64], uint64_t mask, float sc2, float nm,
                                          float &l, uint32_t (&pk)[32]) {
  const uint32_t mlo = (uint32_t)mask, mhi = (uint32_t)(mask >> 32);
  const float2 sc = make_float2(sc2, sc2), nn = make_float2(nm, nm);
  float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
#pragma unroll
  for (int c = 0; c < 64; c += 4) {
    const float2 x0 = ffma2(make_float2(sv[c], sv[c + 1]), sc, nn);
    const float2 x1 = ffma2(make_float2(sv[c + 2], sv[c + 3]), sc, nn);
    float2 e0 = make_float2(exp2f(x0.x), exp2f(x0.y)), e1 = make_float2(exp2f(x1.x), exp2f(x1.y));
    if (!FULL) {
      const uint32_t w = (c < 32 ? mlo : mhi) >> (c & 31);
      e0.x = (w & 1u) ? e0.x : 0.f;
      e0.y = (w & 2u) ? e0.y : 0.f;
      e1.x = (w & 4u) ? e1.x : 0.f;
      e1.y = (w & 8u) ? e1.y : 0.f;
    }
    s0 = fadd2(s0, e0);
    s1 = fadd2(s1, e1);
    pk[c >> 1] = pack_bf16(e0.x, e0.y);
    pk[(c >> 1) + 1] = pack_bf16(e1.x, e1.y);
  }
  l += (s0.x + s0.y) + (s1.x + s1.y);
}

// multiply the row's accumulator by fac (all lanes of the warp take part)
template <int D>
__device__ __forceinline__ void rescale_acc(uint32_t taddr, float fac) {
#pragma unroll
  for (int c0 = 0; c0 < D; c0 += 32) {
    float o[32];
    tmem_ld32(taddr + c0, o);
    tmem_wait_ld();
#pragma unroll
    for (int c = 0; c < 32; ++c) o[c] *= fac;
    tmem_st32(taddr + c0, o);
  }
  tmem_wait_st();
}

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 2) fwd_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmo,
    const __grid_constant__ CUtensorMap tmol, const __grid_constant__ CUtensorMap tmos, Shape s,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const uint8_t *__restrict__ qmeta, int training, float *__restrict__ lse,
    int32_t *__restrict__ status, int nT) {
  using C = Cfg<D>;
  constexpr int STAGES = kFwdStages;
  extern __shared__ uint8_t smem_raw[];
  // barriers: full[STAGES], empty[STAGES], res, one per buffer: s_full[3], t_full[3], done[3], meta
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 11];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nST = (s.L + 127) >> 7;
  // long rows first, tile-major: every unit's last tile, then every unit's last but one, ...
  const int nU = s.B * s.H;
  const int st = nST - 1 - (int)(blockIdx.x / nU);
  const int u = (int)(blockIdx.x % nU), n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int row0 = st * 128;

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *q_tile = tiles;
  uint8_t *kv_tiles = q_tile + C::kBigBytes;  // [stage][K, V]
  uint8_t *meta = kv_tiles + STAGES * 2 * C::kSmallBytes;  // image built by tc_meta_kernel
  const MetaLayout ml = meta_layout(nT);
  const uint8_t *selb = meta;
  const uint16_t *items = reinterpret_cast<const uint16_t *>(meta + ml.items);  // [2 nT]
  const uint8_t *icls = meta + ml.icls;                                         // [2 nT][4]
  const int *counts = reinterpret_cast<const int *>(meta + ml.counts);

  const uint32_t b_full = smem_u32(&bars[0]), b_empty = smem_u32(&bars[STAGES]);
  const uint32_t b_res = smem_u32(&bars[2 * STAGES]);
  const uint32_t b_sfull = smem_u32(&bars[2 * STAGES + 1]), b_tfull = smem_u32(&bars[2 * STAGES + 4]);
  const uint32_t b_done = smem_u32(&bars[2 * STAGES + 7]), b_meta = smem_u32(&bars[2 * STAGES + 10]);

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
    for (int i = 0; i < 3; ++i) {
      mbar_init(b_sfull + 8 * i, 1);
      mbar_init(b_tfull + 8 * i, kSoftmaxWarps);
      mbar_init(b_done + 8 * i, 1);
    }
    mbar_init(b_meta, 1);
    mbar_fence_init();
    // the CTA's tile lists and its query tile
    mbar_expect_tx(b_meta, (uint32_t)ml.bytes);
    bulk_load(smem_u32(meta), qmeta + ((size_t)u * nST + (nST - 1 - st)) * ml.bytes, (uint32_t)ml.bytes, b_meta);
    mbar_expect_tx(b_res, C::kBigBytes);
    tma_load_4d(smem_u32(q_tile), &tmq, b_res, 0, row0, h, n);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), kFwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  mbar_wait(b_meta, 0, &abort_flag, 113);
  const int nL = counts[1], nS = counts[2], nI = nL + nS;
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_o = tmem_base + 192;  // buffers at tmem_base + 64 * (item % 3)

  if (warp >= kSoftmaxWarps) {
    // ===================== three single-thread roles, one warp each =====================
    setmaxnreg_dec<kProducerRegs>();
    if (warp == kSoftmaxWarps && nI > 0) {
      // ---- loader: K/V tiles, up to STAGES ahead of their consumers ----
      for (int j = 0; j < nI; ++j) {
        const int sj = j % STAGES;
        if (j >= STAGES) mbar_wait(b_empty + 8 * sj, ((j - STAGES) / STAGES) & 1, &abort_flag, 105);
        const uint32_t bar = b_full + 8 * sj;
        const uint32_t kt = smem_u32(kv_tiles + sj * 2 * C::kSmallBytes);
        const int row = (int)items[j] * 64;
        if (elect_one()) {
          mbar_expect_tx(bar, 2 * C::kSmallBytes);
          tma_load_4d(kt, &tmk, bar, 0, row, h / s.G, n);  // the key/value head of this query head
          tma_load_4d(kt + C::kSmallBytes, &tmv, bar, 0, row, h / s.G, n);
        }
        __syncwarp();
      }
    } else if (warp == kSoftmaxWarps + 1 && nI > 0) {
      // ---- S(i) = Q K^T into buffer i % 3 once O += P(i-3) V has read that buffer ----
      constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
      const uint64_t dq = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      mbar_wait(b_res, 0, &abort_flag, 101);
      for (int i = 0, b = 0, ph = 0; i < nI; ++i) {  // b = i % 3, ph = (i / 3) & 1
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 102);
        if (i >= 3) mbar_wait(b_done + 8 * b, ph ^ 1, &abort_flag, 103);
        tc_fence_after();
        const uint64_t dk =
            smem_desc(smem_u32(kv_tiles + (i % STAGES) * 2 * C::kSmallBytes), 16, C::kAtomBytes, C::kSwizzle);
        const uint32_t ts = tmem_base + 64 * b;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) umma_bf16(ts, dq + 2 * k, dk + 2 * k, idesc_s, k > 0);
          umma_commit(b_sfull + 8 * b);
        }
        __syncwarp();
        if (++b == 3) {
          b = 0;
          ph ^= 1;
        }
      }
    } else if (warp == kSoftmaxWarps + 2 && nI > 0) {
      // ---- O += P(i) V once the probabilities of item i are in tensor memory ----
      constexpr uint32_t idesc_pv = instr_desc(128, D, 0, 1);
      for (int i = 0, b = 0, ph = 0; i < nI; ++i) {
        const uint64_t dv = smem_desc(smem_u32(kv_tiles + (i % STAGES) * 2 * C::kSmallBytes + C::kSmallBytes),
                                      C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
        const uint32_t tp = tmem_base + 64 * b;
        const uint32_t first = (i == 0 || i == nL) ? 0u : 1u;  // a phase starts the accumulator afresh
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 106);
        mbar_wait(b_tfull + 8 * b, ph, &abort_flag, 104);
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_bf16_ts(tmem_o, tp + 8 * k, dv + k * C::kKStep, idesc_pv, (first | (uint32_t)k) != 0u);
          umma_commit(b_done + 8 * b);
          umma_commit(b_empty + 8 * (i % STAGES));  // S(i) completed before the softmax warps read it
        }
        __syncwarp();
        if (++b == 3) {
          b = 0;
          ph ^= 1;
        }
      }
    }
  } else {
    // ================================ softmax =================================
    setmaxnreg_inc<kSoftmaxRegs>();
    const int r = warp * 32 + lane, t = row0 + r, g = r / s.Bk;
    const bool row_ok = t < s.L;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    float m = -INFINITY, l = 0.f, mL = -INFINITY, lL = 0.f;
    float park[D];  // the row's long-term accumulator while the short-term phase runs
    int acc = 0;    // the current phase has written the accumulator
    const float sc2 = s.scale * kLog2e;
    int b = 0, ph = 0;  // buffer i % 3 and the parity (i / 3) & 1 of its barriers
    int jt_n = nI > 0 ? items[0] : 0, cls_n = nI > 0 ? icls[warp] : 0;

    for (int i = 0; i < nI; ++i) {
      const bool isL = i < nL;
      const int jt = jt_n, cls = cls_n, p0 = jt * 64;
      if (i + 1 < nI) {  // the next item's tile and class, ahead of their use
        jt_n = items[i + 1];
        cls_n = icls[(i + 1) * kSoftmaxWarps + warp];
      }
      uint64_t mask = 0ull;
      bool doB = cls == 1, fullB = cls == 1;
      if (cls == 2) {
        if (row_ok) {
          mask = cols_le(t - p0) & cols_ge(pad0 - p0);
          mask &= isL ? expand_block_bits(selb[g * nT + jt], s.Bk) : st_key_cols(s, t, p0);
        }
        doB = __any_sync(0xffffffffu, mask != 0ull);
        fullB = __all_sync(0xffffffffu, mask == ~0ull);
      }
      const uint32_t t_b = tmem_base + 64 * b + lane_off;
      const uint32_t b_prev = b_done + 8 * (b == 0 ? 2 : b - 1), ph_prev = b == 0 ? ph ^ 1 : ph;  // item i-1

      mbar_wait(b_sfull + 8 * b, ph, &abort_flag, 107);
      __syncwarp();
      tc_fence_after();
      float sv[64];
      if (doB) {
        tmem_ld32(t_b, sv);
        tmem_ld32(t_b + 32, sv + 32);
        tmem_wait_ld();
      }

      bool waited_prev = false;  // the MMAs of item i-1 have completed
      if (i == nL && nL > 0) {
        // End of the long-term phase: park its accumulator rows and statistics; the first P V
        // product of the short-term phase overwrites the accumulator.
        mbar_wait(b_prev, ph_prev, &abort_flag, 111);
        __syncwarp();
        tc_fence_after();
        waited_prev = true;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) tmem_ld32(tmem_o + lane_off + c0, park + c0);
        tmem_wait_ld();
        mL = m;
        lL = l;
        m = -INFINITY;
        l = 0.f;
        acc = 0;
      }

      uint32_t pk[32];
      if (doB) {
        float fac = 1.f;
        bool need = false;
        const float mt = (fullB ? row_max<true>(sv, 0ull) : row_max<false>(sv, mask)) * sc2;
        need = mt > m + kRescaleThreshold;  // also true on the row's first keys
        if (need) {
          fac = exp2f(m - mt);
          l *= fac;
          m = mt;
        }
        if (fullB) row_probs<true>(sv, 0ull, sc2, -m, l, pk);
        else row_probs<false>(sv, mask, sc2, -m, l, pk);
        if (acc && __any_sync(0xffffffffu, need)) {  // rescaling needs the MMAs of item i-1
          if (!waited_prev) {
            mbar_wait(b_prev, ph_prev, &abort_flag, 108);
            __syncwarp();
            tc_fence_after();
          }
          rescale_acc<D>(tmem_o + lane_off, fac);
        }
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) pk[c] = 0u;
      }
      tmem_st32u(t_b, pk);  // the row's probabilities replace its logits
      tmem_wait_st();
      tc_fence_before();
      warp_arrive(b_tfull + 8 * b, lane);  // the stores have completed (wait::st)
      acc = 1;
      if (++b == 3) {
        b = 0;
        ph ^= 1;
      }
    }

    // ---- epilogue ----
    if (nI > 0) {
      mbar_wait(b_done + 8 * ((nI - 1) % 3), ((nI - 1) / 3) & 1, &abort_flag, 110);
      __syncwarp();
      tc_fence_after();
    }
    float mS = -INFINITY, lS = 0.f;
    if (nS > 0) { mS = m; lS = l; } else { mL = m; lL = l; }
    const float alpha = gate_alpha(gate, h), beta = 1.f - alpha;
    const float iL = lL > 0.f ? 1.f / lL : 0.f, iS = lS > 0.f ? 1.f / lS : 0.f;
    const bool haveL = nL > 0 && lL > 0.f, haveS = nS > 0 && lS > 0.f;
    const bool parked = nL > 0 && nS > 0;  // long-term rows in registers, short-term in TMEM
    // Rows go to shared memory in the layout TMA stores expect (the K/V stages are free: every
    // load has landed and every MMA has completed), then three bulk stores write whole lines;
    // rows past L are clipped by the hardware, padded rows are written as zeros.
    uint8_t *so = kv_tiles, *sl = so + C::kBigBytes, *ss = sl + C::kBigBytes;
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 32) {
      float o[32];
      if (nI > 0) {
        tmem_ld32(tmem_o + lane_off + c0, o);
        tmem_wait_ld();
      }
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t wo[4], wl[4], ws[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = ch * 8 + e * 2;
          float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
          if (haveL) {
            a0 = (parked ? park[c0 + c] : o[c]) * iL;
            a1 = (parked ? park[c0 + c + 1] : o[c + 1]) * iL;
          }
          if (haveS) {
            b0 = o[c] * iS;
            b1 = o[c + 1] * iS;
          }
          wl[e] = pack_bf16(a0, a1);
          ws[e] = pack_bf16(b0, b1);
          wo[e] = pack_bf16(alpha * a0 + beta * b0, alpha * a1 + beta * b1);
        }
        const int chunk = c0 / 8 + ch;
        store_row_chunk<D>(so, r, chunk, make_uint4(wo[0], wo[1], wo[2], wo[3]));
        if (training) {
          store_row_chunk<D>(sl, r, chunk, make_uint4(wl[0], wl[1], wl[2], wl[3]));
          store_row_chunk<D>(ss, r, chunk, make_uint4(ws[0], ws[1], ws[2], ws[3]));
        }
      }
    }
    fence_async_smem();
    named_bar_sync(1, kSoftmaxWarps * 32);
    if (tid == 0) {
      tma_store_4d(&tmo, smem_u32(so), 0, row0, h, n);
      if (training) {
        tma_store_4d(&tmol, smem_u32(sl), 0, row0, h, n);
        tma_store_4d(&tmos, smem_u32(ss), 0, row0, h, n);
      }
      tma_store_commit_and_wait();
    }
    if (row_ok && lse) {
      const int64_t BHL = (int64_t)s.B * s.H * s.L;
      lse[(int64_t)u * s.L + t] = lL > 0.f ? (mL + log2f(lL)) * kLn2 : 0.f;
      lse[BHL + (int64_t)u * s.L + t] = lS > 0.f ? (mS + log2f(lS)) * kLn2 : 0.f;
    }
  }
  if (nI == 0 && tid == 0) mbar_wait(b_res, 0, &abort_flag, 112);  // no load may outlive the CTA
  finish(warp, tmem_base, kFwdTmemCols, &abort_flag, status);
}

}  // namespace

template <int D>
int launch_fwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt,
                    void *out_st, float *lse, const Workspace &ws, cudaStream_t st) {
  using C = Cfg<D>;
  CUtensorMap tq, tk, tv, to, tol, tos;
  const int training = out_lt != nullptr;
  if (make_tensor_map(&tq, q, s, 128) || make_tensor_map(&tk, k, s, 64, true) ||
      make_tensor_map(&tv, v, s, 64, true) ||
      make_tensor_map(&to, out, s, 128) || make_tensor_map(&tol, training ? out_lt : out, s, 128) ||
      make_tensor_map(&tos, training ? out_st : out, s, 128))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const size_t smem = 1024 + C::kBigBytes + kFwdStages * 2 * C::kSmallBytes + meta_bytes(nT);
  if (cudaFuncSetAttribute(fwd_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  const unsigned grid = (unsigned)nST * (unsigned)(s.B * s.H);
  if (int rc = launch_tc_meta(s, seq_lens, idx, ws.qmeta, nullptr, st)) return rc;
  {
    LaunchScope ls(K_FWD_TC, st);
    fwd_tc_kernel<D><<<grid, kFwdThreads, smem, st>>>(tq, tk, tv, to, tol, tos, s, gate, seq_lens, ws.qmeta,
                                                     training, lse, ws.status, nT);
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
