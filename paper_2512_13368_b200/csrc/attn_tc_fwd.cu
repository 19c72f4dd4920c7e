// Tensor-core forward of the fused two-branch attention (bf16 storage, fp32 accumulate).
//
// One CTA owns 128 consecutive query rows of one (batch, head) unit (= 128 / Bk query blocks)
// and walks the 64-key tiles that any of its rows needs: the union of the tiles holding a
// selected key block of one of its query blocks (long-term branch, Eq. 14 + 16) and of the tiles
// the causal window reaches (short-term branch, Eq. 15 first case + 17).  Per tile:
//   TMA (128-byte swizzle) stages K and V; one thread issues S = Q K^T as tcgen05.mma
//   (M = 128, N = 64) into TMEM; each of the 128 threads owns one query row (= one TMEM lane),
//   reads its 64 scores, applies the two branch masks and the online softmax of both branches in
//   fp32, writes the two probability tiles as bf16 into swizzled shared memory, and one thread
//   issues O_lt += P_lt V and O_st += P_st V (M = 128, N = D) with both accumulators in TMEM.
// The running maximum is lazy: it is only raised (and the TMEM accumulator rescaled) when a tile's
// maximum exceeds it by more than 2^8, which keeps probabilities <= 256 and rescales rare.
// Epilogue: normalise, mix the branches with the gate (Eq. 19), store out / out_lt / out_st / lse.
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kStages = 3;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct Cfg {
  static constexpr int kRowBytes = D * 2;
  static constexpr int kQBytes = 128 * kRowBytes;
  static constexpr int kKVBytes = 64 * kRowBytes;
  static constexpr int kPBytes = 128 * 128;
  static constexpr int kAtomBytes = 8 * kRowBytes;           // 8-row swizzle atom of a D-wide tile
  static constexpr uint32_t kSwizzle = (D == 64) ? 2u : 4u;  // 128-byte / 64-byte swizzle
  static constexpr int kTileBytes = kQBytes + kStages * 2 * kKVBytes + 2 * kPBytes;
};

__host__ __device__ inline int meta_bytes(int nT) { return ((2 * nT + nT + 8 * nT + 15) / 16) * 16 + 16; }

// One branch of the online softmax for the calling thread's row.  Returns nothing; updates the
// running state and writes the probability row (bf16) into the swizzled tile.
template <int D>
__device__ __forceinline__ void softmax_branch(const float (&sreg)[64], uint64_t mask, float sc2,
                                               float &m_used, float &l, bool acc_started,
                                               uint32_t tmem_o, uint8_t *ptile, int r, bool &row_zero) {
  const bool warp_any = __any_sync(0xffffffffu, mask != 0ull);
  if (!warp_any) {
    if (!row_zero) {
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) store_row_sw128(ptile, r, ch, make_uint4(0u, 0u, 0u, 0u));
      row_zero = true;
    }
    return;
  }
  const bool full = __all_sync(0xffffffffu, mask == ~0ull);
  float mt = -INFINITY;
  if (full) {
#pragma unroll
    for (int c = 0; c < 64; ++c) mt = fmaxf(mt, sreg[c]);
  } else {
#pragma unroll
    for (int c = 0; c < 64; ++c)
      if ((mask >> c) & 1ull) mt = fmaxf(mt, sreg[c]);
  }
  mt *= sc2;
  const bool need = mt > m_used + kRescaleThreshold;  // also true on the row's first keys
  float factor = 1.f;
  if (need) {
    factor = exp2f(m_used - mt);  // 0 when m_used = -inf
    l *= factor;
    m_used = mt;
  }
  if (acc_started && __any_sync(0xffffffffu, need)) {
    float o[32];
#pragma unroll
    for (int h = 0; h < D / 32; ++h) {
      tmem_ld32(tmem_o + h * 32, o);
      tmem_wait_ld();
#pragma unroll
      for (int c = 0; c < 32; ++c) o[c] *= factor;
      tmem_st32(tmem_o + h * 32, o);
    }
    tmem_wait_st();
  }
  const float neg_m = -m_used;  // finite whenever a column of this row is on
  float lsum = 0.f;
#pragma unroll
  for (int ch = 0; ch < 8; ++ch) {
    float p[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int c = ch * 8 + e;
      const float x = exp2f(fmaf(sreg[c], sc2, neg_m));
      p[e] = (full || ((mask >> c) & 1ull)) ? x : 0.f;
      lsum += p[e];
    }
    store_row_sw128(ptile, r, ch,
                    make_uint4(pack_bf16(p[0], p[1]), pack_bf16(p[2], p[3]), pack_bf16(p[4], p[5]),
                               pack_bf16(p[6], p[7])));
  }
  l += lsum;
  row_zero = false;
}

template <int D>
__global__ void __launch_bounds__(128, 2) fwd_tc_kernel(
    const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
    const __grid_constant__ CUtensorMap tmv, Shape s, const float *__restrict__ gate,
    const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ idx,
    __nv_bfloat16 *__restrict__ out, __nv_bfloat16 *__restrict__ out_lt,
    __nv_bfloat16 *__restrict__ out_st, float *__restrict__ lse, int32_t *__restrict__ status,
    int nT) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[kStages + 2];  // full[kStages], q, mma
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int nvis_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nST = (s.L + 127) >> 7;
  const int st = nST - 1 - (int)(blockIdx.x % nST);  // long rows first
  const int u = blockIdx.x / nST, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int row0 = st * 128, row_last = min(s.L - 1, row0 + 127);
  const int G = 128 / s.Bk, nb = 64 / s.Bk;

  // ---- shared-memory carve-up (tiles 1024-byte aligned) ----
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
  uint8_t *tiles = smem_raw + pad;
  uint8_t *q_tile = tiles;
  uint8_t *kv_tiles = q_tile + C::kQBytes;                 // [stage][K, V]
  uint8_t *pl_tile = kv_tiles + kStages * 2 * C::kKVBytes;
  uint8_t *ps_tile = pl_tile + C::kPBytes;
  uint8_t *meta = ps_tile + C::kPBytes;
  uint32_t *selw = reinterpret_cast<uint32_t *>(meta);              // [8][nT] bytes, word access
  uint8_t *selb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ((8 * nT + 15) / 16) * 16);
  uint8_t *lflags = reinterpret_cast<uint8_t *>(list + nT);

  const uint32_t bar_full0 = smem_u32(&bars[0]);
  const uint32_t bar_q = smem_u32(&bars[kStages]);
  const uint32_t bar_mma = smem_u32(&bars[kStages + 1]);

  if (tid == 0) {
    abort_flag = (*status != 0) ? 1 : 0;  // a previous CTA timed out: do not wait again
    for (int i = 0; i < kStages; ++i) mbar_init(bar_full0 + 8 * i, 1);
    mbar_init(bar_q, 1);
    mbar_init(bar_mma, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmq);
    tma_prefetch_desc(&tmk);
    tma_prefetch_desc(&tmv);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), 256);
    tmem_relinquish();
  }
  for (int i = tid; i < (8 * nT + 3) / 4; i += 128) selw[i] = 0u;
  __syncthreads();

  // ---- which key blocks did each of this CTA's query blocks select, per 64-key tile ----
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
  const uint32_t tmem_s = tmem_base;            // S: columns [0, 64)
  const uint32_t tmem_ol = tmem_base + 64;      // O_lt: [64, 64 + D)
  const uint32_t tmem_os = tmem_base + 128;     // O_st: [128, 128 + D)
  const uint32_t lane_off = (uint32_t)(warp * 32) << 16;

  // ---- producer prologue: Q and the first tiles ----
  if (tid == 0 && nvis > 0) {
    mbar_expect_tx(bar_q, C::kQBytes);
    tma_load_4d(smem_u32(q_tile), &tmq, bar_q, 0, row0, h, n);
    for (int i = 0; i < min(kStages, nvis); ++i) {
      const uint32_t bar = bar_full0 + 8 * i;
      uint8_t *kt = kv_tiles + i * 2 * C::kKVBytes;
      mbar_expect_tx(bar, 2 * C::kKVBytes);
      tma_load_4d(smem_u32(kt), &tmk, bar, 0, (int)list[i] * 64, h, n);
      tma_load_4d(smem_u32(kt + C::kKVBytes), &tmv, bar, 0, (int)list[i] * 64, h, n);
    }
  }

  // ---- per-row state ----
  const int r = tid, t = row0 + r, g = r / s.Bk;
  const bool row_ok = t < s.L;
  float mL = -INFINITY, lL = 0.f, mS = -INFINITY, lS = 0.f;
  bool zeroL = false, zeroS = false;
  int accL = 0, accS = 0;  // CTA-uniform: has the accumulator been written yet
  const float sc2 = s.scale * kLog2e;
  constexpr uint32_t idesc_s = instr_desc(128, 64, 0, 0);
  constexpr uint32_t idesc_pv = instr_desc(128, D, 0, 1);
  uint32_t mma_phase = 0;

  for (int i = 0; i < nvis; ++i) {
    const int stage = i % kStages;
    const int jt = list[i], f = lflags[i], p0 = jt * 64;
    uint8_t *k_tile = kv_tiles + stage * 2 * C::kKVBytes, *v_tile = k_tile + C::kKVBytes;
    if (tid == 0) {
      if (i == 0) mbar_wait(bar_q, 0, &abort_flag);
      mbar_wait(bar_full0 + 8 * stage, (i / kStages) & 1, &abort_flag);
      tc_fence_after();
      const uint64_t dq = smem_desc(smem_u32(q_tile), 16, C::kAtomBytes, C::kSwizzle);
      const uint64_t dk = smem_desc(smem_u32(k_tile), 16, C::kAtomBytes, C::kSwizzle);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) umma_bf16(tmem_s, dq + 2 * k, dk + 2 * k, idesc_s, k > 0);
      umma_commit(bar_mma);
    }
    __syncwarp();
    mbar_wait(bar_mma, mma_phase, &abort_flag);
    __syncwarp();
    mma_phase ^= 1u;
    tc_fence_after();
    // S(i) complete => every earlier MMA is complete: the stage of tile i-1 is free again
    if (tid == 0 && i >= 1 && i - 1 + kStages < nvis) {
      const int j = i - 1 + kStages, sj = (i - 1) % kStages;
      const uint32_t bar = bar_full0 + 8 * sj;
      uint8_t *kt = kv_tiles + sj * 2 * C::kKVBytes;
      mbar_expect_tx(bar, 2 * C::kKVBytes);
      tma_load_4d(smem_u32(kt), &tmk, bar, 0, (int)list[j] * 64, h, n);
      tma_load_4d(smem_u32(kt + C::kKVBytes), &tmv, bar, 0, (int)list[j] * 64, h, n);
    }
    __syncwarp();

    // ---- masks of this row for this tile ----
    uint64_t maskL = 0ull, maskS = 0ull;
    if (row_ok) {
      const uint64_t mc = cols_le(t - p0) & cols_ge(pad0 - p0);
      if (f & 1) maskL = mc & expand_block_bits(selb[g * nT + jt], s.Bk);
      if (f & 2) maskS = mc & cols_ge(t - s.window + 1 - p0);
    }
    float sreg[64];
    if (__any_sync(0xffffffffu, (maskL | maskS) != 0ull)) {
      tmem_ld32(tmem_s + lane_off, sreg);
      tmem_ld32(tmem_s + lane_off + 32, sreg + 32);
      tmem_wait_ld();
    } else {
#pragma unroll
      for (int c = 0; c < 64; ++c) sreg[c] = 0.f;
    }
    if (f & 1) softmax_branch<D>(sreg, maskL, sc2, mL, lL, accL != 0, tmem_ol + lane_off, pl_tile, r, zeroL);
    if (f & 2) softmax_branch<D>(sreg, maskS, sc2, mS, lS, accS != 0, tmem_os + lane_off, ps_tile, r, zeroS);

    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint64_t dv = smem_desc(smem_u32(v_tile), C::kKVBytes, C::kAtomBytes, C::kSwizzle);
      if (f & 1) {
        const uint64_t dp = smem_desc(smem_u32(pl_tile), 16, 1024, 2u);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(tmem_ol, dp + 2 * k, dv + k * (16 * C::kRowBytes >> 4), idesc_pv, (accL | k) != 0);
      }
      if (f & 2) {
        const uint64_t dp = smem_desc(smem_u32(ps_tile), 16, 1024, 2u);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(tmem_os, dp + 2 * k, dv + k * (16 * C::kRowBytes >> 4), idesc_pv, (accS | k) != 0);
      }
    }
    accL |= (f & 1);
    accS |= (f & 2);
  }

  // ---- epilogue ----
  if (nvis > 0) {
    if (tid == 0) umma_commit(bar_mma);
    __syncwarp();
    mbar_wait(bar_mma, mma_phase, &abort_flag);
    __syncwarp();
    tc_fence_after();
  }
  const float alpha = 1.f / (1.f + __expf(-(gate[h * 2 + 0] - gate[h * 2 + 1]))), beta = 1.f - alpha;
  const float iL = lL > 0.f ? 1.f / lL : 0.f, iS = lS > 0.f ? 1.f / lS : 0.f;
  const bool haveL = accL && lL > 0.f, haveS = accS && lS > 0.f;
  const int64_t ro = row_offset(s, n, h, row_ok ? t : 0);
#pragma unroll
  for (int hh = 0; hh < D / 32; ++hh) {
    float oL[32], oS[32];
    if (accL) tmem_ld32(tmem_ol + lane_off + hh * 32, oL);   // accL / accS are CTA-uniform
    if (accS) tmem_ld32(tmem_os + lane_off + hh * 32, oS);
    tmem_wait_ld();
    if (row_ok) {
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
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
        const int64_t off = ro + hh * 32 + ch * 8;
        *reinterpret_cast<uint4 *>(out + off) = make_uint4(wo[0], wo[1], wo[2], wo[3]);
        if (out_lt) *reinterpret_cast<uint4 *>(out_lt + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
        if (out_st) *reinterpret_cast<uint4 *>(out_st + off) = make_uint4(ws[0], ws[1], ws[2], ws[3]);
      }
    }
  }
  if (row_ok && lse) {
    const int64_t BHL = (int64_t)s.B * s.H * s.L;
    lse[(int64_t)u * s.L + t] = lL > 0.f ? (mL + log2f(lL)) * kLn2 : 0.f;
    lse[BHL + (int64_t)u * s.L + t] = lS > 0.f ? (mS + log2f(lS)) * kLn2 : 0.f;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 256);
  if (tid == 0 && abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}  // grace period for copies still in flight
    atomicExch(status, (int32_t)BLOSSOM_ERR_TIMEOUT);
  }
}

template <int D>
int launch_fwd_tc_t(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                    const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt,
                    void *out_st, float *lse, const Workspace &ws, cudaStream_t st) {
  CUtensorMap tq, tk, tv;
  if (make_tensor_map(&tq, q, s, 128) || make_tensor_map(&tk, k, s, 64) || make_tensor_map(&tv, v, s, 64))
    return BLOSSOM_ERR_CUDA;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const size_t smem = 1024 + Cfg<D>::kTileBytes + meta_bytes(nT);
  if (cudaFuncSetAttribute(fwd_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  const unsigned grid = (unsigned)nST * (unsigned)(s.B * s.H);
  {
    LaunchScope ls(K_FWD_TC, st);
    fwd_tc_kernel<D><<<grid, 128, smem, st>>>(tq, tk, tv, s, gate, seq_lens, idx, (__nv_bfloat16 *)out,
                                             (__nv_bfloat16 *)out_lt, (__nv_bfloat16 *)out_st, lse,
                                             ws.status, nT);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

// ---- host: TMA descriptor ----
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

}  // namespace tc
}  // namespace blossom
