// Tensor-core forward of the fused two-branch attention (bf16 storage, fp32 accumulate).
//
// A CTA owns 128 query rows (128 / Bk query blocks) and walks a list of items, one 64-key tile of
// one branch each: first the tiles any of its query blocks selected (Eq. 14, 16), then the tiles
// its rows reach through the window (Eq. 15, 17).  A tile that belongs to both branches is visited
// once per phase.  With grouped heads (an even number per key/value head) the 128 rows are instead
// the same 64 positions of two heads of a group, which share their selection (Eq. 12), their window
// tiles and their K/V: every tile on the list then has work for every row (template flag PACK).
//
// CTA = 384 threads.  Warps 0..7 are softmax warps: a query row (= TMEM lane) is shared by two
// threads, warp w and warp w + 4, which split the KEYS of every tile: group 0 (warps 0..3) takes
// keys 0..31, group 1 keys 32..63.  Each group keeps its own running maximum and sum and its own
// accumulator (O_A += P[:, 0:32] V[0:32], O_B += P[:, 32:64] V[32:64]), so the two threads of a row
// never exchange anything inside the loop; the two partial results are merged, exactly as two
// halves of an online softmax, when a phase ends.  Sixteen softmax warps per SM instead of eight
// hide the latency of a thread's dependent chain (load, maximum, exponentials, store).
// Warps 8, 9, 10 stay converged and one elected lane of each loads K/V tiles (TMA), issues
// S = Q K^T, and issues the two O += P V products with P read from tensor memory.
//
// Tensor memory (256 columns): two logits / probability buffers [0,64) [64,128), O_A [128,128+D),
// O_B [192,192+D).  Item i uses buffer i % 2: S(i) lands there as fp32, a softmax thread reads its
// 32 logits and writes their probabilities (bf16 pairs) over the first 16 of them, from where the
// products read their first operand:
//
//   loader   : stage j <- K, V of item j once the products of item j - STAGES have completed
//   S issuer : wait K(i) and "products of item i-2 done" (the buffer is free) -> S(i) -> s_full[i%2]
//   softmax  : wait s_full -> tcgen05.ld 32 logits -> online softmax of the half row (maximum
//              raised, and the group's accumulator rescaled, only when it grows by > 2^8) ->
//              tcgen05.st P -> arrive t_full[group][i%2]
//   PV issuer: wait t_full[0] -> O_A += P_A V[0:32]; wait t_full[1] -> O_B += P_B V[32:64] ->
//              commit done[i%2], release the stage
//
// When the long-term phase ends the merged, normalised rows go (as bf16) to a staging tile in
// shared memory, from where they are stored and read back for the gate mix of the epilogue
// (Eq. 19); the short-term phase then starts both accumulators afresh.
// Epilogue: merge, normalise, gate mix, stage the rows in shared memory and write out / out_lt /
// out_st with whole-line TMA stores; lse directly.  Every wait is bounded (tc_common.cuh).
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kFwdThreads = 384;  // warps 0..7 softmax; 8 loader, 9 S issuer, 10 PV issuer, 11 spare
constexpr int kSoftmaxWarps = 8;
// The kernel is compiled for 80 registers per thread (two CTAs of 384 threads per SM): the pool of
// a CTA is 384 * 80 = 30720, and the two register counts must fit in it or the increase would
// wait for registers that never come: 256 * 96 + 128 * 40 = 29696.
constexpr int kProducerRegs = 40, kSoftmaxRegs = 96;
static_assert(256 * kSoftmaxRegs + 128 * kProducerRegs <= kFwdThreads * 80, "register pool of a CTA");
constexpr int kFwdStages = 4;
constexpr uint32_t kFwdTmemCols = 256;

// maximum of 32 logits (those whose mask bit is set, all of them when FULL)
template <bool FULL>
__device__ __forceinline__ float half_row_max(const float (&v)[32], uint32_t mask) {
  float a[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) a[e] = -INFINITY;
#pragma unroll
  for (int c = 0; c < 32; c += 8) {
    float x[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) x[e] = (FULL || ((mask >> (c + e)) & 1u)) ? v[c + e] : -INFINITY;
#pragma unroll
    for (int e = 0; e < 4; ++e) a[e] = max3(a[e], x[2 * e], x[2 * e + 1]);
  }
  return fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
}

// probabilities of 32 logits relative to the running maximum (nm = -m, log2 units), packed as
// bf16 pairs; their sum is added to l.  Two logits per FMA / ADD instruction.
template <bool FULL>
__device__ __forceinline__ void half_row_probs(const float (&sv)[32], uint32_t mask, float sc2, float nm,
                                               float &l, uint32_t (&pk)[16]) {
  const float2 sc = make_float2(sc2, sc2), nn = make_float2(nm, nm);
  float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
#pragma unroll
  for (int c = 0; c < 32; c += 4) {
    const float2 x0 = ffma2(make_float2(sv[c], sv[c + 1]), sc, nn);
    const float2 x1 = ffma2(make_float2(sv[c + 2], sv[c + 3]), sc, nn);
    float2 e0 = make_float2(exp2f(x0.x), exp2f(x0.y)), e1 = make_float2(exp2f(x1.x), exp2f(x1.y));
    if (!FULL) {
      const uint32_t w = mask >> c;
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

// 16-byte chunk ch of row r of a staged D-wide bf16 tile (the layout of store_row_chunk)
template <int D>
__device__ __forceinline__ uint4 load_row_chunk(const uint8_t *tile, int r, int ch) {
  if constexpr (D == 64) return *reinterpret_cast<const uint4 *>(tile + r * 128 + ((ch ^ (r & 7)) << 4));
  else return *reinterpret_cast<const uint4 *>(tile + r * 64 + ((ch ^ ((r >> 1) & 3)) << 4));
}

// PLAIN: the causal mask and one selection per query block (the measured path): the other modes'
// tests fold away at compile time.
// PACK: rows 0..63 and 64..127 of the CTA are the same 64 positions of two query heads with a common
// key/value head: by Eq. 12 they selected the same blocks and their windows reach the same tiles,
// so every tile the CTA loads has work for all its rows.
template <int D, bool PLAIN, bool PACK>
__global__ void __launch_bounds__(kFwdThreads, 2) fwd_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmo,
    const __grid_constant__ CUtensorMap tmol, const __grid_constant__ CUtensorMap tmos, Shape s,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const uint8_t *__restrict__ qmeta, int training, float *__restrict__ lse,
    int32_t *__restrict__ status, int nT) {
  grid_chain_enter();
  using C = Cfg<D>;
  constexpr int STAGES = kFwdStages;
  constexpr int DC = D / 2;  // output columns a softmax thread merges and stages
  extern __shared__ uint8_t smem_raw[];
  // barriers: full[STAGES], empty[STAGES], res, meta, then per buffer: s_full[2], t_full[group][2], done[2]
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 10];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ float2 stat[2][128];  // (maximum, sum) of each group's half of every row, exchanged at a phase end

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

  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t *tiles = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  uint8_t *q_tile = tiles;
  uint8_t *kv_tiles = q_tile + C::kBigBytes;                  // [stage][K, V]
  uint8_t *sl = kv_tiles + STAGES * 2 * C::kSmallBytes;       // the long-term rows, staged when their phase ends
  uint8_t *meta = sl + C::kBigBytes;                          // image built by tc_meta_kernel
  const bool causal = PLAIN || s.causal;
  const int pq = PLAIN ? 0 : s.pq;
  const MetaLayout ml = meta_layout(nT, pq);
  const uint8_t *selb = meta;
  const uint8_t *rowb = meta + ml.rows;  // (selection per query position) [128 rows][nT]
  const uint16_t *items = reinterpret_cast<const uint16_t *>(meta + ml.items);  // [2 nT]
  const uint8_t *icls = meta + ml.icls;                                         // [2 nT][4]
  const int *counts = reinterpret_cast<const int *>(meta + ml.counts);

  const uint32_t b_full = smem_u32(&bars[0]), b_empty = smem_u32(&bars[STAGES]);
  const uint32_t b_res = smem_u32(&bars[2 * STAGES]), b_meta = smem_u32(&bars[2 * STAGES + 1]);
  const uint32_t b_sfull = smem_u32(&bars[2 * STAGES + 2]), b_tfull = smem_u32(&bars[2 * STAGES + 4]);  // [group][buffer]
  const uint32_t b_done = smem_u32(&bars[2 * STAGES + 8]);

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
    mbar_init(b_meta, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(b_sfull + 8 * i, 1);
      mbar_init(b_tfull + 8 * i, kSoftmaxWarps / 2);        // group 0
      mbar_init(b_tfull + 8 * (2 + i), kSoftmaxWarps / 2);  // group 1
      mbar_init(b_done + 8 * i, 1);
    }
    mbar_fence_init();
    // the CTA's tile lists and its query tile
    mbar_expect_tx(b_meta, (uint32_t)ml.bytes);
    bulk_load(smem_u32(meta), qmeta + ((size_t)u * nQT + (nQT - 1 - st)) * ml.bytes, (uint32_t)ml.bytes, b_meta);
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
  const uint32_t tmem_oa = tmem_base + 128, tmem_ob = tmem_base + 192;  // buffers at tmem_base + 64 * (item % 2)

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
      // ---- S(i) = Q K^T into buffer i % 2 once the products of item i - 2 have read that buffer ----
      constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
      const uint64_t dq = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      mbar_wait(b_res, 0, &abort_flag, 101);
      for (int i = 0; i < nI; ++i) {
        const int b = i & 1, ph = (i >> 1) & 1;
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 102);
        if (i >= 2) mbar_wait(b_done + 8 * b, ph ^ 1, &abort_flag, 103);
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
      }
    } else if (warp == kSoftmaxWarps + 2 && nI > 0) {
      // ---- O_A += P(i)[:, 0:32] V[0:32], O_B += P(i)[:, 32:64] V[32:64] once that group's
      // probabilities of item i are in tensor memory ----
      constexpr uint32_t idesc_pv = instr_desc(128, D, 0, 1);
      for (int i = 0; i < nI; ++i) {
        const int b = i & 1, ph = (i >> 1) & 1;
        const uint64_t dv = smem_desc(smem_u32(kv_tiles + (i % STAGES) * 2 * C::kSmallBytes + C::kSmallBytes),
                                      C::kSmallBytes, C::kAtomBytes, C::kSwizzle);
        const uint32_t tp = tmem_base + 64 * b;
        const uint32_t first = (i == 0 || i == nL) ? 0u : 1u;  // a phase starts the accumulators afresh
        mbar_wait(b_full + 8 * (i % STAGES), (i / STAGES) & 1, &abort_flag, 106);
        mbar_wait(b_tfull + 8 * b, ph, &abort_flag, 104);
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 2; ++k)
            umma_bf16_ts(tmem_oa, tp + 8 * k, dv + k * C::kKStep, idesc_pv, (first | (uint32_t)k) != 0u);
        }
        __syncwarp();
        mbar_wait(b_tfull + 8 * (2 + b), ph, &abort_flag, 109);
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 2; ++k)
            umma_bf16_ts(tmem_ob, tp + 32 + 8 * k, dv + (2 + k) * C::kKStep, idesc_pv, (first | (uint32_t)k) != 0u);
          umma_commit(b_done + 8 * b);
          umma_commit(b_empty + 8 * (i % STAGES));  // S(i) completed before the softmax warps read it
        }
        __syncwarp();
      }
    }
  } else {
    // ================================ softmax =================================
    setmaxnreg_inc<kSoftmaxRegs>();
    const int quarter = warp & 3, grp = warp >> 2;  // TMEM lane quarter; key half of every tile
    const int r = quarter * 32 + lane, t = PACK ? row0 + (r & 63) : row0 + r, g = r / s.Bk;
    const int hr = PACK ? h + (r >> 6) : h;  // this row's head
    const bool row_ok = t < s.L;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const uint32_t acc_own = (grp ? tmem_ob : tmem_oa) + lane_off;
    float m = -INFINITY, l = 0.f;  // this group's running maximum (log2 units) and sum of the row
    float lseL = 0.f, lseS = 0.f;
    bool haveL = false, haveS = false;
    int acc = 0;  // the current phase has written the accumulators
    const float sc2 = s.scale * kLog2e;
    const float alpha = gate_alpha(gate, hr), beta = 1.f - alpha;
    int jt_n = nI > 0 ? items[0] : 0, cls_n = nI > 0 ? icls[quarter] : 0;
    uint8_t *so = kv_tiles, *ss = so + C::kBigBytes;  // staging of out / out_st (the K/V stages, free by then)

    // End of a phase: the two groups' halves of every row are merged (maxima, sums, accumulators),
    // normalised, and this thread's DC columns are staged: the long-term rows into sl; at the very
    // end the short-term rows and the gate mix (Eq. 19) into ss and so, the long-term rows being
    // read back from sl.  The caller has waited for the phase's last products.
    auto merge = [&](bool long_term, bool final_phase) {
      stat[grp][r] = make_float2(m, l);
      named_bar_sync(1, kSoftmaxWarps * 32);
      const float2 oth = stat[grp ^ 1][r];
      const float mt = fmaxf(m, oth.x);
      const float fo = l > 0.f ? exp2f(m - mt) : 0.f, fp = oth.y > 0.f ? exp2f(oth.x - mt) : 0.f;
      const float lt = l * fo + oth.y * fp;
      const float inv = (lt > 0.f && row_ok && t >= pad0) ? 1.f / lt : 0.f;
      const float fa = (grp ? fp : fo) * inv, fb = (grp ? fo : fp) * inv;
      const float lse_v = lt > 0.f ? (mt + log2f(lt)) * kLn2 : 0.f;
      if (long_term) { lseL = lse_v; haveL = lt > 0.f; } else { lseS = lse_v; haveS = lt > 0.f; }
#pragma unroll
      for (int c0 = 0; c0 < DC; c0 += 16) {
        float a[16], b[16];
        tmem_ld16(tmem_oa + lane_off + DC * grp + c0, a);
        tmem_ld16(tmem_ob + lane_off + DC * grp + c0, b);
        tmem_wait_ld();
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          const int chunk = (DC * grp + c0) / 8 + ch;
          float o[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) o[e] = inv > 0.f ? a[ch * 8 + e] * fa + b[ch * 8 + e] * fb : 0.f;
          if (long_term || nL == 0) {  // (no long-term phase at all: its rows are zeros)
            store_row_chunk<D>(sl, r, chunk, make_uint4(pack_bf16(o[0], o[1]), pack_bf16(o[2], o[3]),
                                                         pack_bf16(o[4], o[5]), pack_bf16(o[6], o[7])));
          }
          if (final_phase) {
            float oL[8], oS[8];
            if (long_term) {  // (no short-term items at all: the long-term rows are the last phase)
#pragma unroll
              for (int e = 0; e < 8; ++e) { oL[e] = o[e]; oS[e] = 0.f; }
            } else {
              const uint4 w = nL > 0 ? load_row_chunk<D>(sl, r, chunk) : make_uint4(0u, 0u, 0u, 0u);
              const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                oL[2 * e] = __uint_as_float(ww[e] << 16);
                oL[2 * e + 1] = __uint_as_float(ww[e] & 0xffff0000u);
                oS[2 * e] = o[2 * e];
                oS[2 * e + 1] = o[2 * e + 1];
              }
            }
            uint32_t wo[4], ws[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              wo[e] = pack_bf16(alpha * oL[2 * e] + beta * oS[2 * e], alpha * oL[2 * e + 1] + beta * oS[2 * e + 1]);
              ws[e] = pack_bf16(oS[2 * e], oS[2 * e + 1]);
            }
            store_row_chunk<D>(so, r, chunk, make_uint4(wo[0], wo[1], wo[2], wo[3]));
            store_row_chunk<D>(ss, r, chunk, make_uint4(ws[0], ws[1], ws[2], ws[3]));
          }
        }
      }
    };

    for (int i = 0; i < nI; ++i) {
      const bool isL = i < nL;
      const int jt = jt_n, cls = cls_n, p0 = jt * 64;
      if (i + 1 < nI) {  // the next item's tile and class, ahead of their use
        jt_n = items[i + 1];
        cls_n = icls[(i + 1) * 4 + quarter];
      }
      const int b = i & 1, ph = (i >> 1) & 1;
      const uint32_t b_prev = b_done + 8 * (b ^ 1), ph_prev = ((i - 1) >> 1) & 1;  // item i-1
      if (i == nL && nL > 0) {
        // End of the long-term phase: merge and stage its rows; the first products of the
        // short-term phase overwrite the accumulators.
        mbar_wait(b_prev, ph_prev, &abort_flag, 111);
        __syncwarp();
        tc_fence_after();
        merge(true, false);
        tc_fence_before();
        // Both groups read both accumulators in the merge, and the first product of the next phase
        // overwrites an accumulator as soon as ITS group has stored the next probabilities: no
        // warp may go on before every warp has read.
        named_bar_sync(3, kSoftmaxWarps * 32);
        m = -INFINITY;
        l = 0.f;
        acc = 0;
      }
      uint32_t hm = 0u;  // this thread's 32 keys of the tile that the row sees
      bool doB = cls == 1, fullB = cls == 1;
      if (cls == 2) {
        if (row_ok && (causal || t >= pad0)) {  // (a padded row sees nothing; under the causal mask the bounds below say so)
          uint64_t mask = cols_le((causal ? t : s.L - 1) - p0) & cols_ge(pad0 - p0);
          mask &= isL ? expand_block_bits(pq ? rowb[r * nT + jt] : selb[g * nT + jt], s.Bk) : st_key_cols(s, t, p0, causal);
          hm = (uint32_t)(mask >> (32 * grp));
        }
        doB = __any_sync(0xffffffffu, hm != 0u);
        fullB = __all_sync(0xffffffffu, hm == 0xffffffffu);
      }
      const uint32_t t_b = tmem_base + 64 * b + lane_off + 32 * grp;

      mbar_wait(b_sfull + 8 * b, ph, &abort_flag, 107);
      __syncwarp();
      tc_fence_after();
      uint32_t pk[16];
      if (doB) {
        float sv[32];
        tmem_ld32(t_b, sv);
        tmem_wait_ld();
        float fac = 1.f;
        const float mt = (fullB ? half_row_max<true>(sv, 0u) : half_row_max<false>(sv, hm)) * sc2;
        const bool need = mt > m + kRescaleThreshold;  // also true on the row's first keys
        if (need) {
          fac = exp2f(m - mt);
          l *= fac;
          m = mt;
        }
        if (fullB) half_row_probs<true>(sv, 0u, sc2, -m, l, pk);
        else half_row_probs<false>(sv, hm, sc2, -m, l, pk);
        if (acc && __any_sync(0xffffffffu, need)) {  // rescaling needs the products of item i-1
          mbar_wait(b_prev, ph_prev, &abort_flag, 108);
          __syncwarp();
          tc_fence_after();
          rescale_acc<D>(acc_own, fac);
        }
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c) pk[c] = 0u;
      }
      tmem_st16u(t_b, pk);  // the probabilities replace this thread's logits
      tmem_wait_st();
      tc_fence_before();
      warp_arrive(b_tfull + 8 * (2 * grp + b), lane);  // the stores have completed (wait::st)
      acc = 1;
    }

    // ---- epilogue ----
    if (nI > 0) {
      mbar_wait(b_done + 8 * ((nI - 1) & 1), ((nI - 1) >> 1) & 1, &abort_flag, 110);
      __syncwarp();
      tc_fence_after();
      merge(nS == 0, true);
    } else {
#pragma unroll
      for (int ch = 0; ch < DC / 8; ++ch) {
        const int chunk = DC * grp / 8 + ch;
        store_row_chunk<D>(so, r, chunk, make_uint4(0u, 0u, 0u, 0u));
        store_row_chunk<D>(sl, r, chunk, make_uint4(0u, 0u, 0u, 0u));
        store_row_chunk<D>(ss, r, chunk, make_uint4(0u, 0u, 0u, 0u));
      }
    }
    // Whole-line bulk stores of the staged rows; rows past L are clipped by the hardware, padded
    // rows were staged as zeros.
    fence_async_smem();
    named_bar_sync(2, kSoftmaxWarps * 32);
    if (tid == 0) {
      tma_store_4d(&tmo, smem_u32(so), 0, row0, h, n);
      if (training) {
        tma_store_4d(&tmol, smem_u32(sl), 0, row0, h, n);
        tma_store_4d(&tmos, smem_u32(ss), 0, row0, h, n);
      }
      tma_store_commit_and_wait();
    }
    if (grp == 0 && row_ok && lse) {
      const int64_t BHL = (int64_t)s.B * s.H * s.L;
      const int64_t row = ((int64_t)n * s.H + hr) * s.L + t;
      lse[row] = haveL ? lseL : 0.f;
      lse[BHL + row] = haveS ? lseS : 0.f;
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
  // (head-packed: a query-side box is 64 positions of two heads)
  const int qrows = s.pack ? 64 : 128, qheads = s.pack ? 2 : 1;
  if (make_tensor_map(&tq, q, s, qrows, false, qheads) || make_tensor_map(&tk, k, s, 64, true) ||
      make_tensor_map(&tv, v, s, 64, true) || make_tensor_map(&to, out, s, qrows, false, qheads) ||
      make_tensor_map(&tol, training ? out_lt : out, s, qrows, false, qheads) ||
      make_tensor_map(&tos, training ? out_st : out, s, qrows, false, qheads))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const size_t smem = 1024 + 2 * C::kBigBytes + kFwdStages * 2 * C::kSmallBytes + meta_bytes(nT, s.pq);
  const bool plain = s.causal && !s.pq;
  auto kern = s.pack ? (plain ? fwd_tc_kernel<D, true, true> : fwd_tc_kernel<D, false, true>)
                     : (plain ? fwd_tc_kernel<D, true, false> : fwd_tc_kernel<D, false, false>);
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  const unsigned grid = s.pack ? (unsigned)nT * (unsigned)(s.B * (s.H / 2)) : (unsigned)nST * (unsigned)(s.B * s.H);
  // A training call also builds the backward's tile lists (the same launch: one warp per image):
  // a backward call told to reuse them (blossom_params::reuse_tile_lists) then builds none.
  if (int rc = launch_tc_meta(s, seq_lens, idx, ws.qmeta, training ? ws.kmeta : nullptr, st, 3, 1)) return rc;
  {
    LaunchScope ls(K_FWD_TC, st);
    launch_chained(kern, dim3(grid), dim3(kFwdThreads), smem, st, tq, tk, tv, to, tol, tos, s, gate, seq_lens,
                   (const uint8_t *)ws.qmeta, training, lse, ws.status, nT);
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
