// Block summary, importance scoring and top-k selection (paper Eq. 8-13).
//
// One code path serves the plain selection (compression size = stride = selection size = Bk, the
// ragged last block kept) and the selection through overlapping compression blocks (Eq. 8 with
// length l and stride s, only whole blocks, and the score remap of Eq. 11), for one head per
// key/value head or for groups of heads that share one selection (Eq. 12: the probabilities of the
// group's heads are summed).  The "scored blocks" below are the compression blocks: positions
// [s c, s c + l), summarised by the mean of their valid keys (Eq. 9 with the summary = mean).
// Query block b scores the scored blocks that end before it starts (candidates c < nc(b)), every
// valid query taking a softmax over the live candidates (Eq. 10), the probabilities being summed
// over the block's queries and the group's heads; Eq. 11 maps those sums onto the selection blocks
// j < b (the identity in the plain mode); the own block plus the top_k - 1 best selectable past
// blocks are kept, ties to the lower index (Eq. 13).
//
// The selection is a discrete decision taken from floating-point sums whose neighbours differ by
// ~1e-3 relative on Gaussian inputs, and the library promises the choice a double-precision
// evaluation makes (ties below ~1e-12 relative excepted).  Two stages deliver it:
//   1. every query block is scored in single precision together with a rigorous bound on the
//      distance of each score from its exact value; if the last kept and the first dropped
//      selection block are further apart than the bound allows them to move, the choice is certain
//      and is written out;
//   2. the (few per cent of) query blocks whose choice is not certain are appended to a work
//      list and re-scored in double precision by a second kernel.
// With left padding a block is live exactly when it reaches past the padding, so liveness is a
// comparison of indices (cmin, jmin below); the counts of valid keys are kept for callers that
// want them.
#include "common.cuh"

#include <cooperative_groups.h>

namespace blossom {

namespace cg = cooperative_groups;

namespace {

// Geometry of the scored blocks.
struct SelGeom {
  int n;       // scored blocks per (batch, key/value head): Mc, or M in the plain mode
  int l, s;    // their length and stride in positions
  int rs, rl;  // Bk / s and l / s, the two sums of Eq. 11 (1, 1 in the plain mode)
  int plain;
};

SelGeom sel_geom(const Shape &sh) {
  SelGeom g;
  if (sh.cmp_l > 0) {
    g.n = sh.Mc; g.l = sh.cmp_l; g.s = sh.cmp_s; g.rs = sh.Bk / sh.cmp_s; g.rl = sh.cmp_l / sh.cmp_s;
    g.plain = 0;
  } else {
    g.n = sh.M; g.l = sh.Bk; g.s = sh.Bk; g.rs = 1; g.rl = 1; g.plain = 1;
  }
  return g;
}

// scored blocks 0 .. nc - 1 end before query block b starts
__device__ __forceinline__ int n_candidates(const Shape &sh, const SelGeom &g, int b) {
  if (g.plain) return b;
  const int start = b * sh.Bk;
  return start >= g.l ? min(g.n, (start - g.l) / g.s + 1) : 0;
}
// the first scored block that holds a valid key (pad0 = number of padded positions)
__device__ __forceinline__ int first_live_scored(const SelGeom &g, int pad0) {
  return pad0 < g.l ? 0 : (pad0 - g.l) / g.s + 1;
}

// Eight consecutive elements as loaded (16 bytes of bf16, 32 of fp32), unpacked to floats on use.
template <typename T>
struct Raw8;
template <>
struct Raw8<__nv_bfloat16> {
  uint4 r;
  __device__ __forceinline__ void load(const __nv_bfloat16 *p) { r = *reinterpret_cast<const uint4 *>(p); }
  __device__ __forceinline__ void zero() { r = make_uint4(0u, 0u, 0u, 0u); }
  __device__ __forceinline__ void unpack(float (&x)[8]) const {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      x[2 * e] = __uint_as_float(w[e] << 16);
      x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
  }
};
template <>
struct Raw8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float *p) {
    a = *reinterpret_cast<const float4 *>(p);
    b = *reinterpret_cast<const float4 *>(p + 4);
  }
  __device__ __forceinline__ void zero() { a = b = make_float4(0.f, 0.f, 0.f, 0.f); }
  __device__ __forceinline__ void unpack(float (&x)[8]) const {
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  }
};

// ---- Eq. 8 + 9: mean of the valid keys of every scored block (fp64) ------------------------
// One warp per scored block, 8 blocks per CTA.  A lane owns eight columns (one 16-byte load of
// bf16, two of fp32) of every (32 / (D / 8))-th row and sums them in a fixed order with eight rows
// in flight (kept as loaded until they are added); the lanes that share columns are combined by
// shuffles in a fixed tree.
template <typename T, int D, bool PHI>
__global__ void __launch_bounds__(256, PHI ? 2 : 4) summary_kernel(Shape sh, SelGeom g, const T *__restrict__ k,
                                                         const int32_t *__restrict__ seq_lens,
                                                         double *__restrict__ mean,
                                                         int32_t *__restrict__ live,
                                                         float *__restrict__ mean32,
                                                         float *__restrict__ norm,
                                                         int32_t *__restrict__ sel_count) {
  grid_chain_enter();
  constexpr int LPR = D / 8;     // lanes per row
  constexpr int RPI = 32 / LPR;  // rows per warp iteration
  constexpr int NF = sizeof(T) == 2 ? 8 : 2;  // rows in flight per lane
  if (blockIdx.x == 0 && threadIdx.x == 0) *sel_count = 0;  // work list of the scoring kernel
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t blk = (int64_t)blockIdx.x * 8 + warp;  // (batch, key/value head, scored block)
  if (blk >= (int64_t)sh.B * sh.Hkv * g.n) return;
  const int c = (int)(blk % g.n), u = (int)(blk / g.n), n = u / sh.Hkv, hk = u % sh.Hkv;
  int len = seq_lens ? seq_lens[n] : sh.L;
  len = min(max(len, 0), sh.L);
  const int pad0 = sh.L - len;
  const int lo = max(c * g.s, pad0), hi = min(c * g.s + g.l, sh.L);
  const int sub = lane / LPR, col = (lane % LPR) * 8;
  const T *base = k + row_offset_kv(sh, n, hk, 0) + col;
  double a[8], wsum = 0.0;  // weighted column sums and the sum of the weights (Eq. 9)
#pragma unroll
  for (int e = 0; e < 8; ++e) a[e] = 0.0;
  for (int p = lo + sub; p < hi; p += NF * RPI) {
    Raw8<T> x[NF];
#pragma unroll
    for (int r = 0; r < NF; ++r) {
      const int pp = p + r * RPI;
      if (pp < hi) x[r].load(base + (int64_t)pp * sh.ksl);
      else x[r].zero();
    }
    if (PHI) {  // learnable summary: weight exp(phi[i]) for position i of the block
#pragma unroll
      for (int r = 0; r < NF; ++r) {
        const int pp = p + r * RPI;
        const double w = pp < hi ? exp((double)sh.phi[pp - c * g.s]) : 0.0;
        float f[8];
        x[r].unpack(f);
#pragma unroll
        for (int e = 0; e < 8; ++e) a[e] = fma(w, (double)f[e], a[e]);
        wsum += w;
      }
    } else {
#pragma unroll
      for (int r = 0; r < NF; ++r) {
        float f[8];
        x[r].unpack(f);
#pragma unroll
        for (int e = 0; e < 8; ++e) a[e] += (double)f[e];
      }
    }
  }
#pragma unroll
  for (int o = LPR; o < 32; o <<= 1)  // the lanes that took other rows of the same columns
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] += __shfl_xor_sync(0xffffffffu, a[e], o);
  const int cnt = max(hi - lo, 0);
  if (PHI) {
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
  } else {
    wsum = (double)cnt;
  }
  float sq = 0.f;
  if (sub == 0) {
    double m[8];
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      m[e] = cnt > 0 ? a[e] / wsum : 0.0;
      f[e] = (float)m[e];
      sq = fmaf(f[e], f[e], sq);
    }
    double2 *md = reinterpret_cast<double2 *>(mean + blk * D + col);
    md[0] = make_double2(m[0], m[1]); md[1] = make_double2(m[2], m[3]);
    md[2] = make_double2(m[4], m[5]); md[3] = make_double2(m[6], m[7]);
    float4 *mf = reinterpret_cast<float4 *>(mean32 + blk * D + col);
    mf[0] = make_float4(f[0], f[1], f[2], f[3]);
    mf[1] = make_float4(f[4], f[5], f[6], f[7]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  if (lane == 0) {
    live[blk] = cnt;
    norm[blk] = sqrtf(sq) * 1.0001f;  // an upper bound of the fp32 mean's norm
  }
}

// ---- Eq. 11 for one query block: scores of the selection blocks j in [jmin, b) -------------
// Sc[c], c in [cmin, nc): summed probabilities of the live candidates (anything outside counts as
// zero).  One warp.
template <typename F>
__device__ __forceinline__ void map_scores(const SelGeom &g, const F *Sc, int cmin, int nc, int jmin, int b,
                                           F *S, int lane) {
  for (int j = jmin + lane; j < b; j += 32) {
    F acc = (F)0;
    for (int m = 0; m < g.rs; ++m)
      for (int n = 0; n < g.rl; ++n) {
        const int i = g.rs * j - m - n;
        if (i >= cmin && i < nc) acc += Sc[i];
      }
    S[j] = acc;
  }
}

// Eq. 13 by rank: block j in [jmin, b) is kept iff fewer than `want` selectable blocks beat it
// (larger score, or equal score and lower index).  One warp; `bound` receives the smallest kept
// and the largest dropped score.
template <typename F>
__device__ __forceinline__ void rank_select(const F *S, int jmin, int b, int want, uint8_t *taken, F *bound,
                                            int lane) {
  for (int j = jmin + lane; j < b; j += 32) {
    const F sj = S[j];
    int rank = 0;
    for (int i = jmin; i < b; ++i) {
      const F si = S[i];
      rank += (si > sj || (si == sj && i < j)) ? 1 : 0;
    }
    taken[j] = rank < want ? 1 : 0;
    if (rank == want - 1) bound[0] = sj;  // the smallest kept score
    if (rank == want) bound[1] = sj;      // the largest dropped score
  }
}

// ascending: the flagged blocks of [jmin, b), then the own block, then -1
__device__ __forceinline__ void emit_row(int32_t *row, const uint8_t *taken, int jmin, int b, int topk, int lane) {
  int pos = 0;
  for (int base = jmin; base < b; base += 32) {
    const int j = base + lane;
    const bool f = j < b && taken[j];
    const unsigned m = __ballot_sync(0xffffffffu, f);
    if (f) row[pos + __popc(m & ((1u << lane) - 1u))] = j;
    pos += __popc(m);
  }
  if (lane == 0) row[pos] = b;
  for (int i = pos + 1 + lane; i < topk; i += 32) row[i] = -1;
}

// Partial column sums of the probabilities p[a][e] of a thread's rows ty + 16 a: first over GA
// consecutive a (rows of one query block when Bk >= 16 GA), then over the four lanes ty of the
// warp (rows 4 warp .. 4 warp + 3 of each 16-row group), in that fixed order.  part[warp][group][64].
template <int GA>
__device__ __forceinline__ void row_group_sums(const float (&p)[8][8], float *part, int warp, int lane) {
#pragma unroll
  for (int gi = 0; gi < 8 / GA; ++gi)
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float v = p[gi * GA][e];
#pragma unroll
      for (int a = 1; a < GA; ++a) v += p[gi * GA + a][e];
      v += __shfl_xor_sync(0xffffffffu, v, 8);
      v += __shfl_xor_sync(0xffffffffu, v, 16);
      if (lane < 8) part[(warp * 8 + gi) * 64 + lane + 8 * e] = v;
    }
}

// ascending: the flagged blocks of [lo, hi), then -1
__device__ __forceinline__ void emit_flags(int32_t *row, const uint8_t *taken, int lo, int hi, int topk, int lane) {
  int pos = 0;
  for (int base = lo; base < hi; base += 32) {
    const int j = base + lane;
    const bool f = j < hi && taken[j];
    const unsigned m = __ballot_sync(0xffffffffu, f);
    if (f) row[pos + __popc(m & ((1u << lane) - 1u))] = j;
    pos += __popc(m);
  }
  for (int i = pos + lane; i < topk; i += 32) row[i] = -1;
}

// ---- stage 1: single-precision scoring with an error bound ----------------------------------
// A CTA of 128 threads takes 128 consecutive positions of one (batch, key/value head): 128 / Bk
// query blocks.  Logits against 64 candidate means at a time come from a register-blocked fp32
// product out of shared memory: thread (ty, tx) owns rows ty + 16 a and candidates tx + 8 e
// (a, e < 8), so a row's 64 logits sit in the eight lanes tx = 0..7 and the softmax of a row needs
// three shuffles.  The candidates e = 2 e2 and 2 e2 + 1 of a thread sit interleaved in shared
// memory, so one 16-byte load brings two dimensions of both and one packed instruction does two of
// the thread's multiply-adds (each accumulator still adds its D products one after the other).  Probabilities are summed over groups of four rows by shuffles and over a query
// block's groups in a fixed order through shared memory.
//
// Error bound.  With u = 2^-24: every logit is within E = (D + 4) u scale max|q_t| max|mean_c| of
// its exact value (D roundings of the accumulation, the rounding of the mean to fp32, the scale),
// so every exact probability lies within a factor exp(+-2E) of the exact softmax of the computed
// logits; evaluating that softmax and the sums in fp32 adds 2^-21 (exp2 approximation and
// division), 2^-22 per unit of logit range, and one u per addition: 16 per candidate chunk for
// the normaliser, 2 + Bk / 4 for the column sum, one per head of the group, one per term of
// Eq. 11, and a margin of 40.  R is the total, relative; two scores a > b are in certain order
// when a - b > R (a + b).
constexpr int kFastThreads = 128;

// d = a * b + c on two packed fp32 values: two IEEE fused multiply-adds in one instruction (the
// same rounding, and the same flush of denormals, as the scalar fmaf of this build)
__device__ __forceinline__ float2 fma_pair(float2 a, float2 b, float2 c) {
  uint64_t d;
  asm("fma.rn.ftz.f32x2 %0, %1, %2, %3;"
      : "=l"(d)
      : "l"(*reinterpret_cast<uint64_t *>(&a)), "l"(*reinterpret_cast<uint64_t *>(&b)),
        "l"(*reinterpret_cast<uint64_t *>(&c)));
  return *reinterpret_cast<float2 *>(&d);
}
constexpr int kRowTile = 128;  // positions per CTA
constexpr int kChunk = 64;     // candidates per product

template <typename T, int D>
__global__ void __launch_bounds__(kFastThreads, 3) score_fast_kernel(
    Shape sh, SelGeom g, const T *__restrict__ q, const float *__restrict__ mean32,
    const float *__restrict__ norm, const int32_t *__restrict__ seq_lens, int32_t *__restrict__ idx,
    int32_t *__restrict__ worklist, int32_t *__restrict__ work_count, int sc_pitch) {
  grid_chain_enter();
  constexpr int P = D + 4;  // row pitch of the query tile (floats): conflict-free 128-bit reads
  constexpr int PK = D + 2;  // row pitch of the interleaved means (pairs of floats): the same
  extern __shared__ float fsm[];
  __shared__ float rn[kRowTile];  // norm bound of every query row (largest over the group's heads)
  __shared__ float bound_s[16][2];
  __shared__ int kn_bits;
  const int M = sh.M, Bk = sh.Bk;
  const int nqb_full = kRowTile / Bk;
  float *qs = fsm;                                      // [128][P]  the tile's queries of one head
  float *ks = qs + kRowTile * P;                        // [4 e2][8 tx][PK][2] a chunk of candidate means: candidates
                                                        // tx + 16 e2 and tx + 16 e2 + 8 interleaved per dimension
  float *part = ks + kChunk * P;                        // [4 warps][8][64] sums over groups of four rows
  float *Sc = part + 4 * 8 * 64;                        // [nqb][sc_pitch] summed probabilities per candidate
  float *Ssel = Sc + nqb_full * sc_pitch;               // [nqb][M] selection-block scores (overlapping mode)
  uint8_t *taken = reinterpret_cast<uint8_t *>(Ssel + (g.plain ? 0 : nqb_full * M));  // [nqb][M]

  const int ntiles = (sh.L + kRowTile - 1) / kRowTile, nU = sh.B * sh.Hkv;
  // late tiles have the most candidates: they go first (tile-major)
  const int tile = ntiles - 1 - (int)(blockIdx.x / nU), u = (int)(blockIdx.x % nU), n = u / sh.Hkv, hk = u % sh.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ty = tid >> 3, tx = tid & 7;
  int len = seq_lens ? seq_lens[n] : sh.L;
  len = min(max(len, 0), sh.L);
  const int pad0 = sh.L - len;
  const int row0 = tile * kRowTile;
  const int qb0 = row0 / Bk, nqb = min(nqb_full, M - qb0);
  const int cmin = first_live_scored(g, pad0);  // live candidates: c >= cmin
  const int jmin = pad0 / Bk;                   // selectable selection blocks: j >= jmin
  const int nc_max = n_candidates(sh, g, qb0 + nqb - 1);

  // Does any query block of the tile have a real choice to make from non-zero scores?
  bool need = false;
  for (int i = 0; i < nqb; ++i) {
    const int b = qb0 + i;
    const bool valid = max(b * Bk, pad0) < min((b + 1) * Bk, sh.L);
    const int nsel = max(0, b - jmin), want = min(sh.topk - 1, nsel);
    const int ncand = max(0, n_candidates(sh, g, b) - cmin);
    need |= valid && nsel > want && want > 0 && ncand > 0;
  }
  if (tid == 0) kn_bits = 0;
  rn[tid] = 0.f;
  __syncthreads();

  if (need) {
    {  // the largest norm among the live candidates of the tile
      float km = 0.f;
      for (int c = cmin + tid; c < nc_max; c += kFastThreads) km = fmaxf(km, norm[(int64_t)u * g.n + c]);
      if (km > 0.f) atomicMax(&kn_bits, __float_as_int(km));  // positive floats order like ints
    }
    const int ch_lo = cmin / kChunk, ch_hi = (nc_max + kChunk - 1) / kChunk;  // chunks that hold live candidates
    const int npass = ch_hi - ch_lo > 1 ? 2 : 1;
    // candidate limit of each of this thread's rows (the block of row ty + 16 a)
    int nc_row[8];
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      const int t = row0 + ty + 16 * a;
      nc_row[a] = (t >= pad0 && t < sh.L) ? n_candidates(sh, g, t / Bk) : 0;
    }
    const float *kbase = mean32 + (int64_t)u * g.n * D;

#pragma unroll 1
    for (int hg = 0; hg < sh.G; ++hg) {  // the heads of the group take turns (Eq. 12)
      const int h = hk * sh.G + hg;
      __syncthreads();  // the previous head's tiles are no longer read
      // The tile's queries (fp32 in shared memory, invalid rows zero) and the first chunk of
      // candidate means: every global load of the thread is in flight before the first store.
      {
        constexpr int CPR = D / 8, NQ = kRowTile * CPR / kFastThreads;  // 8-element chunks per row; loads per thread
        constexpr int NK = kChunk * (D / 4) / kFastThreads;
        Raw8<T> x[NQ];
        float4 v[NK];
        const int c0 = ch_lo * kChunk, nb = min(kChunk, nc_max - c0);
#pragma unroll
        for (int it = 0; it < NQ; ++it) {
          const int i = tid + it * kFastThreads, lt = i / CPR, c = (i % CPR) * 8, t = row0 + lt;
          if (t >= pad0 && t < sh.L) x[it].load(q + row_offset(sh, n, h, t) + c);
          else x[it].zero();
        }
#pragma unroll
        for (int it = 0; it < NK; ++it) {
          const int i = tid + it * kFastThreads, lj = i / (D / 4), c = (i % (D / 4)) * 4;
          v[it] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (lj < nb && c0 + lj >= cmin) v[it] = *reinterpret_cast<const float4 *>(kbase + (int64_t)(c0 + lj) * D + c);
        }
#pragma unroll
        for (int it = 0; it < NQ; ++it) {
          const int i = tid + it * kFastThreads, lt = i / CPR, c = (i % CPR) * 8;
          float f[8];
          x[it].unpack(f);
          *reinterpret_cast<float4 *>(qs + lt * P + c) = make_float4(f[0], f[1], f[2], f[3]);
          *reinterpret_cast<float4 *>(qs + lt * P + c + 4) = make_float4(f[4], f[5], f[6], f[7]);
        }
#pragma unroll
        for (int it = 0; it < NK; ++it) {
          const int i = tid + it * kFastThreads, lj = i / (D / 4), c = (i % (D / 4)) * 4;
          float *dst = ks + ((((lj >> 4) * 8 + (lj & 7)) * PK + c) << 1) + ((lj >> 3) & 1);
          dst[0] = v[it].x; dst[2] = v[it].y; dst[4] = v[it].z; dst[6] = v[it].w;
        }
      }
      __syncthreads();
      {  // norm bound of row tid (128 rows, 128 threads)
        float a = 0.f;
#pragma unroll 8
        for (int c = 0; c < D; ++c) a = fmaf(qs[tid * P + c], qs[tid * P + c], a);
        rn[tid] = fmaxf(rn[tid], sqrtf(a) * 1.0001f);
      }
      float mx[8], den[8];  // online softmax statistics of this thread's rows
#pragma unroll
      for (int a = 0; a < 8; ++a) {
        mx[a] = -INFINITY;
        den[a] = 0.f;
      }
#pragma unroll 1
      for (int pass = 0; pass < npass; ++pass) {
#pragma unroll 1
        for (int ch = ch_lo; ch < ch_hi; ++ch) {
          const int c0 = ch * kChunk, nb = min(kChunk, nc_max - c0);
          if (pass > 0 || ch > ch_lo) {  // (the head's first chunk is in place already)
            constexpr int NK = kChunk * (D / 4) / kFastThreads;
            float4 v[NK];
            __syncthreads();  // previous users of ks and part are done
#pragma unroll
            for (int it = 0; it < NK; ++it) {
              const int i = tid + it * kFastThreads, lj = i / (D / 4), c = (i % (D / 4)) * 4;
              v[it] = make_float4(0.f, 0.f, 0.f, 0.f);
              if (lj < nb && c0 + lj >= cmin) v[it] = *reinterpret_cast<const float4 *>(kbase + (int64_t)(c0 + lj) * D + c);
            }
#pragma unroll
            for (int it = 0; it < NK; ++it) {
              const int i = tid + it * kFastThreads, lj = i / (D / 4), c = (i % (D / 4)) * 4;
              float *dst = ks + ((((lj >> 4) * 8 + (lj & 7)) * PK + c) << 1) + ((lj >> 3) & 1);
              dst[0] = v[it].x; dst[2] = v[it].y; dst[4] = v[it].z; dst[6] = v[it].w;
            }
            __syncthreads();
          }
          float2 acc2[8][4];  // (row a; candidates e = 2 e2, 2 e2 + 1)
#pragma unroll
          for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2) acc2[a][e2] = make_float2(0.f, 0.f);
          const int ne = (nb + 7) >> 3;  // groups of 8 candidates that hold any (block-uniform)
          const int ne2 = (ne + 1) >> 1;  // (the odd group's partner holds zeros)
#pragma unroll 2
          for (int c = 0; c < D; c += 4) {
            float4 qa[8], kb[4][2];  // kb[e2][h]: dimensions c + 2 h, c + 2 h + 1 of the two candidates
#pragma unroll
            for (int a = 0; a < 8; ++a) qa[a] = *reinterpret_cast<const float4 *>(qs + (ty + 16 * a) * P + c);
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2)
              if (e2 < ne2) {
                const float *src = ks + (((e2 * 8 + tx) * PK + c) << 1);
                kb[e2][0] = *reinterpret_cast<const float4 *>(src);
                kb[e2][1] = *reinterpret_cast<const float4 *>(src + 4);
              }
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2)
              if (e2 < ne2) {
#pragma unroll
                for (int a = 0; a < 8; ++a) {
                  float2 r = acc2[a][e2];
                  r = fma_pair(make_float2(qa[a].x, qa[a].x), make_float2(kb[e2][0].x, kb[e2][0].y), r);
                  r = fma_pair(make_float2(qa[a].y, qa[a].y), make_float2(kb[e2][0].z, kb[e2][0].w), r);
                  r = fma_pair(make_float2(qa[a].z, qa[a].z), make_float2(kb[e2][1].x, kb[e2][1].y), r);
                  r = fma_pair(make_float2(qa[a].w, qa[a].w), make_float2(kb[e2][1].z, kb[e2][1].w), r);
                  acc2[a][e2] = r;
                }
              }
          }
          float acc[8][8];
#pragma unroll
          for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2) {
              acc[a][2 * e2] = acc2[a][e2].x;
              acc[a][2 * e2 + 1] = acc2[a][e2].y;
            }
          // logits; pairs that do not take part (dead candidates, candidates not before the row's
          // block, invalid rows) become -inf and drop out of every sum below
#pragma unroll
          for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int c = c0 + tx + 8 * e;
              acc[a][e] = (e < ne && c >= cmin && c < nc_row[a]) ? acc[a][e] * sh.scale : -INFINITY;
            }
          if (pass == 0) {  // fold the chunk into (mx, den) of every row
#pragma unroll
            for (int a = 0; a < 8; ++a) {
              float cm = acc[a][0];
#pragma unroll
              for (int e = 1; e < 8; ++e) cm = fmaxf(cm, acc[a][e]);
              cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
              cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
              cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 4));
              const float nm = fmaxf(mx[a], cm), ref = nm > -INFINITY ? nm : 0.f;
              float es = 0.f;
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float ex = __expf(acc[a][e] - ref);  // exp(-inf) = 0
                es += ex;
                if (npass == 1) acc[a][e] = ex;  // one chunk: these are the numerators
              }
              es += __shfl_xor_sync(0xffffffffu, es, 1);
              es += __shfl_xor_sync(0xffffffffu, es, 2);
              es += __shfl_xor_sync(0xffffffffu, es, 4);
              den[a] = (mx[a] > -INFINITY ? den[a] * __expf(mx[a] - nm) : 0.f) + es;
              mx[a] = nm;
            }
          }
          if (pass == npass - 1) {  // probabilities, summed over the thread's rows of one query block
                                    // (rows 16 a + ty: Bk / 16 consecutive a) and over groups of four rows
#pragma unroll
            for (int a = 0; a < 8; ++a) {
              const float inv = den[a] > 0.f ? 1.f / den[a] : 0.f, ref = mx[a] > -INFINITY ? mx[a] : 0.f;
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[a][e] = (npass == 1 ? acc[a][e] : __expf(acc[a][e] - ref)) * inv;
            }
            if (Bk >= 64) row_group_sums<4>(acc, part, warp, lane);
            else if (Bk >= 32) row_group_sums<2>(acc, part, warp, lane);
            else row_group_sums<1>(acc, part, warp, lane);
            __syncthreads();
            // a query block's column sums: the partial sums of its rows in a fixed order
            const int ga = Bk >= 64 ? 4 : (Bk >= 32 ? 2 : 1);  // rows of a thread per partial sum
            for (int o = tid; o < nqb * kChunk; o += kFastThreads) {
              const int i = o / kChunk, col = o % kChunk;
              if (col < nb) {
                // block i: rows [i Bk, (i + 1) Bk) = partial sums (warp w, group gi) with 16 ga gi + 4 w inside
                float a = 0.f;
                for (int r4 = i * Bk / 4; r4 < (i + 1) * Bk / 4; ++r4)
                  if ((r4 >> 2) % ga == 0) a += part[((r4 & 3) * 8 + (r4 >> 2) / ga) * 64 + col];
                float *dst = Sc + i * sc_pitch + c0 + col;
                *dst = hg == 0 ? a : *dst + a;  // heads in ascending order
              }
            }
          }
        }
      }
    }
  }
  __syncthreads();

  // Eq. 11, Eq. 13 and the certificate: one warp per query block
  for (int i = warp; i < nqb; i += kFastThreads / 32) {
    const int b = qb0 + i;
    int32_t *row = idx + ((int64_t)u * M + b) * sh.topk;
    if (max(b * Bk, pad0) >= min((b + 1) * Bk, sh.L)) {  // the query block holds only padding
      for (int x = lane; x < sh.topk; x += 32) row[x] = -1;
      continue;
    }
    const int nc = n_candidates(sh, g, b), ncand = max(0, nc - cmin);
    const int nsel = max(0, b - jmin), want = min(sh.topk - 1, nsel);
    const bool choose = nsel > want && want > 0;
    uint8_t *tk = taken + i * M;
    bool certain = true;
    if (!choose) {
      for (int j = jmin + lane; j < b; j += 32) tk[j] = want > 0 ? 1 : 0;
    } else if (ncand == 0) {  // every score is zero in any precision: the lowest blocks win the ties
      for (int j = jmin + lane; j < b; j += 32) tk[j] = j - jmin < want ? 1 : 0;
    } else {
      float *S = Sc + i * sc_pitch;
      if (!g.plain) {
        S = Ssel + i * M;
        map_scores<float>(g, Sc + i * sc_pitch, cmin, nc, jmin, b, S, lane);
        __syncwarp();
      }
      rank_select<float>(S, jmin, b, want, tk, bound_s[i], lane);
      __syncwarp();
      // Certain iff the gap between the last kept and the first dropped score exceeds what the
      // errors can bridge.
      float qn = 0.f;
      for (int x = lane; x < Bk; x += 32) qn = fmaxf(qn, rn[i * Bk + x]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) qn = fmaxf(qn, __shfl_xor_sync(0xffffffffu, qn, o));
      const float kn = __int_as_float(kn_bits);
      const float uu = 5.9604645e-8f;          // 2^-24
      const float bound = sh.scale * qn * kn;  // >= every |logit|
      const float E = (float)(D + 4) * uu * bound * 1.01f;
      const float nchunks = (float)((nc + kChunk - 1) / kChunk);
      const float R = 2.f * E + 4.77e-7f + 2.f * bound * 2.39e-7f +
                      (16.f * nchunks + (float)(Bk / 4) + 2.f + (float)sh.G + (float)(g.rs * g.rl) + 40.f) * uu;
      const float smin = bound_s[i][0], umax = bound_s[i][1];
      certain = (smin - umax) > R * (smin + umax) * 1.001f;
    }
    __syncwarp();
    if (certain) emit_row(row, tk, jmin, b, sh.topk, lane);
    else if (lane == 0) worklist[atomicAdd(work_count, 1)] = u * M + b;  // re-scored in double precision
  }
}

// ---- stage 2: the same scores in double precision ------------------------------------------
// One CTA of 256 threads per query block of the work list (every query block when worklist ==
// nullptr).  64 query rows at a time (the block's queries of the group's heads, head-major)
// against 64 candidate means at a time: thread (row tid / 4, part tid % 4) forms the 16 logits of
// candidates part + 4 k, so sixteen independent accumulation chains are in flight; softmax per row
// by 4 lanes; the probabilities go through a shared tile for the column sums (fixed order).
// Launched in thread-block clusters when a query block has more than 64 rows (grouped heads): CTA
// r of a cluster takes the row chunks r, r + cluster size, ..., and CTA 0 adds the other CTAs'
// column sums to its own in rank order out of their shared memory, which with one chunk per CTA
// is the order a single CTA adds them in.  The work of a query block is otherwise serial, and the
// work list is short (a few per cent of the query blocks), so without the split the kernel's time
// is that of one CTA walking G * Bk rows.
template <typename T, int D, int NZ>  // NZ: chunks of 64 candidates whose logits a thread may keep in registers
__global__ void __launch_bounds__(256, 2) score_exact_kernel(
    Shape sh, SelGeom g, const T *__restrict__ q, const double *__restrict__ mean,
    const int32_t *__restrict__ seq_lens, int32_t *__restrict__ idx, const int32_t *__restrict__ worklist,
    const int32_t *__restrict__ work_count, int sc_len) {
  grid_chain_enter();
  constexpr int PD = D + 1;
  extern __shared__ double dsm[];
  __shared__ double bound_d[2];
  double *qd = dsm;             // [64][PD] query rows
  double *kd = qd + 64 * PD;    // [64] candidate means (pitch PD), then the probability tile (pitch 65)
  double *csum = kd + 64 * 65;  // [256]
  double *Sc = csum + 256;      // [sc_len] summed probabilities per candidate
  double *S = Sc + sc_len;      // [M] scores of the selection blocks
  uint8_t *taken = reinterpret_cast<uint8_t *>(S + sh.M);  // [M]

  const int M = sh.M, Bk = sh.Bk;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rt = tid >> 2, part = tid & 3;
  const int total = worklist ? *work_count : M * sh.B * sh.Hkv;
  cg::cluster_group cluster = cg::this_cluster();
  const int nrank = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  // (every CTA of a cluster walks the same query blocks, so the cluster barriers below match up)
  for (int wi = blockIdx.x / nrank; wi < total; wi += gridDim.x / nrank) {
    const int row_id = worklist ? worklist[wi] : wi;
    const int b = row_id % M, u = row_id / M, n = u / sh.Hkv, hk = u % sh.Hkv;
    int len = seq_lens ? seq_lens[n] : sh.L;
    len = min(max(len, 0), sh.L);
    const int pad0 = sh.L - len;
    const int qlo = max(b * Bk, pad0), qhi = min((b + 1) * Bk, sh.L);
    int32_t *row = idx + ((int64_t)u * M + b) * sh.topk;
    __syncthreads();  // shared memory is reused from the previous query block
    if (qlo >= qhi) {  // the query block holds only padding
      if (rank == 0)
        for (int i = tid; i < sh.topk; i += 256) row[i] = -1;
      continue;
    }
    const int cmin = first_live_scored(g, pad0), jmin = pad0 / Bk;
    // without the causal mask (plain selection only) every other live block is a candidate
    const int hi = sh.causal ? b : M;
    const int nc = sh.causal ? n_candidates(sh, g, b) : g.n;
    const int ncand = max(0, nc - cmin - (sh.causal ? 0 : 1));
    const int nsel = max(0, hi - jmin - (sh.causal ? 0 : 1)), want = min(sh.topk - 1, nsel);
    const bool choose = nsel > want && want > 0;

    if (choose && ncand > 0) {
      for (int c = cmin + tid; c < nc; c += 256) Sc[c] = 0.0;
      const int nq = qhi - qlo, nrows = nq * sh.G;  // rows: head r / nq of the group, query qlo + r % nq
      const int ch_lo = cmin / 64, ch_hi = (nc + 63) / 64;
      const double *kbase = mean + (int64_t)u * g.n * D;
      for (int r0 = 64 * rank; r0 < nrows; r0 += 64 * nrank) {
        const int nr = min(64, nrows - r0);
        __syncthreads();
        for (int i = tid; i < 64 * (D / 4); i += 256) {  // 64 query rows as doubles, missing rows zero
          const int lr = i / (D / 4), c = (i % (D / 4)) * 4;
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (lr < nr) {
            const int r = r0 + lr;
            v = ld4(q + row_offset(sh, n, hk * sh.G + r / nq, qlo + r % nq) + c);
          }
          double *d = qd + lr * PD + c;
          d[0] = (double)v.x; d[1] = (double)v.y; d[2] = (double)v.z; d[3] = (double)v.w;
        }
        const bool row_on = rt < nr;
        const double *qr = qd + rt * PD;
        // logits of this thread's row against the 16 candidates part + 4 k of chunk ch, and which
        // of them count
        auto logits = [&](int ch, double (&z)[16], uint32_t &on) {
          const int c0 = ch * 64, nb = min(64, nc - c0);
          __syncthreads();  // previous users of kd are done
          for (int i = tid; i < 64 * (D / 2); i += 256) {
            const int lj = i / (D / 2), c = (i % (D / 2)) * 2;
            double2 v = make_double2(0.0, 0.0);
            if (lj < nb && c0 + lj >= cmin) v = *reinterpret_cast<const double2 *>(kbase + (int64_t)(c0 + lj) * D + c);
            kd[lj * PD + c] = v.x;
            kd[lj * PD + c + 1] = v.y;
          }
          __syncthreads();
#pragma unroll
          for (int k = 0; k < 16; ++k) z[k] = 0.0;
#pragma unroll 2
          for (int c = 0; c < D; ++c) {
            const double qv = qr[c];
#pragma unroll
            for (int k = 0; k < 16; ++k) z[k] = fma(qv, kd[(part + 4 * k) * PD + c], z[k]);
          }
          on = 0u;
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            z[k] *= sh.scale_d;
            const int c = c0 + part + 4 * k;
            if (row_on && part + 4 * k < nb && c >= cmin && (sh.causal || c != b)) on |= 1u << k;
          }
        };
        // running maximum and normaliser of the row over the chunks seen so far
        auto fold = [&](const double (&z)[16], uint32_t on, double &mx, double &den) {
          double cm = -INFINITY;
#pragma unroll
          for (int k = 0; k < 16; ++k)
            if ((on >> k) & 1u) cm = fmax(cm, z[k]);
          cm = fmax(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
          cm = fmax(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
          const double nm = fmax(mx, cm);
          double es = 0.0;
          if (nm > -INFINITY) {
#pragma unroll
            for (int k = 0; k < 16; ++k)
              if ((on >> k) & 1u) es += exp(z[k] - nm);
          }
          es += __shfl_xor_sync(0xffffffffu, es, 1);
          es += __shfl_xor_sync(0xffffffffu, es, 2);
          den = (mx > -INFINITY ? den * exp(mx - nm) : 0.0) + es;
          mx = nm;
        };
        // probabilities of chunk ch and their column sums, added to Sc
        auto columns = [&](int ch, const double (&z)[16], uint32_t on, double mx, double den) {
          const int c0 = ch * 64, nb = min(64, nc - c0);
          __syncthreads();  // everyone has read kd: it becomes the probability tile
#pragma unroll
          for (int k = 0; k < 16; ++k)
            kd[rt * 65 + part + 4 * k] = ((on >> k) & 1u) ? exp(z[k] - mx) / den : 0.0;
          __syncthreads();
          {  // column sums in a fixed order: four partial sums of 16 rows, then their tree
            const int j = tid & 63, quarter = tid >> 6;
            double a = 0.0;
#pragma unroll
            for (int t = 0; t < 16; ++t) a += kd[(quarter * 16 + t) * 65 + j];
            csum[tid] = a;
          }
          __syncthreads();
          if (tid < nb) Sc[c0 + tid] += (csum[tid] + csum[64 + tid]) + (csum[128 + tid] + csum[192 + tid]);
        };
        double mx = -INFINITY, den = 0.0;
        if (ch_hi - ch_lo <= NZ) {
          // the logits of all (one or two) chunks stay in registers
          double za[16], zb[NZ > 1 ? 16 : 1];
          uint32_t ona = 0u, onb = 0u;
          const bool two = NZ > 1 && ch_hi - ch_lo == 2;
          logits(ch_lo, za, ona);
          fold(za, ona, mx, den);
          if constexpr (NZ > 1) {
            if (two) {
              logits(ch_lo + 1, zb, onb);
              fold(zb, onb, mx, den);
            }
          }
          columns(ch_lo, za, ona, mx, den);
          if constexpr (NZ > 1) {
            if (two) columns(ch_lo + 1, zb, onb, mx, den);
          }
        } else {
          // more: one pass for the maxima and normalisers, a second one for the probabilities
          double z[16];
          uint32_t on;
          for (int ch = ch_lo; ch < ch_hi; ++ch) {
            logits(ch, z, on);
            fold(z, on, mx, den);
          }
          for (int ch = ch_lo; ch < ch_hi; ++ch) {
            logits(ch, z, on);
            columns(ch, z, on, mx, den);
          }
        }
      }
    }
    if (nrank > 1) {
      cluster.sync();  // every CTA's column sums are complete
      if (rank == 0 && choose && ncand > 0) {
        for (int c = cmin + tid; c < nc; c += 256) {
          double a = Sc[c];
          for (int r = 1; r < nrank; ++r) a += cluster.map_shared_rank(Sc, r)[c];
          Sc[c] = a;
        }
      }
      cluster.sync();  // the other CTAs' sums have been read: they may go on (or exit)
      if (rank != 0) continue;
    }
    __syncthreads();
    if (warp == 0) {
      if (!choose) {
        for (int j = jmin + lane; j < hi; j += 32) taken[j] = want > 0 ? 1 : 0;
      } else if (ncand == 0) {
        for (int j = jmin + lane; j < hi; j += 32) taken[j] = j - jmin < want ? 1 : 0;
      } else {
        map_scores<double>(g, Sc, cmin, nc, jmin, hi, S, lane);
        __syncwarp();
        if (!sh.causal && lane == 0) S[b] = -INFINITY;  // the own block is not ranked: it is kept anyway
        __syncwarp();
        rank_select<double>(S, jmin, hi, want, taken, bound_d, lane);
      }
      __syncwarp();
      if (sh.causal) {
        emit_row(row, taken, jmin, b, sh.topk, lane);
      } else {  // the own block takes its place in the ascending row
        if (lane == 0) taken[b] = 1;
        __syncwarp();
        emit_flags(row, taken, jmin, hi, sh.topk, lane);
      }
    }
  }
}

// ---- selection per query position (Eq. 13 as printed), double precision -------------------
// One warp per (batch, key/value head, position t): the softmax of Eq. 10 over the live blocks
// before t's block for every head of the group, the probabilities summed over the heads (Eq. 12),
// the top_k - 1 largest kept together with t's own block, ties to the lower index.  block_idx is
// [B][Hkv][L][top_k].  Lanes stride over the candidate blocks; the means come from global memory
// (they are shared by the neighbouring positions and stay in L2).
template <typename T, int D>
__global__ void __launch_bounds__(256) score_per_query_kernel(
    Shape sh, const T *__restrict__ q, const double *__restrict__ mean,
    const int32_t *__restrict__ seq_lens, int32_t *__restrict__ idx) {
  grid_chain_enter();
  extern __shared__ double dsm[];
  __shared__ double bound_d[8][2];
  const int M = sh.M, Bk = sh.Bk;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  double *P = dsm + (size_t)warp * (2 * M + D);  // [M] summed probabilities of this warp's position
  double *Z = P + M;                             // [M] logits of the current head
  double *qrow = Z + M;                          // [D]
  uint8_t *taken = reinterpret_cast<uint8_t *>(dsm + (size_t)8 * (2 * M + D)) + (size_t)warp * M;
  const int64_t pos = (int64_t)blockIdx.x * 8 + warp;
  if (pos >= (int64_t)sh.B * sh.Hkv * sh.L) return;
  const int t = (int)(pos % sh.L), u = (int)(pos / sh.L), n = u / sh.Hkv, hk = u % sh.Hkv;
  int len = seq_lens ? seq_lens[n] : sh.L;
  len = min(max(len, 0), sh.L);
  const int pad0 = sh.L - len;
  int32_t *row = idx + pos * sh.topk;
  if (t < pad0) {
    for (int i = lane; i < sh.topk; i += 32) row[i] = -1;
    return;
  }
  const int b = t / Bk, jmin = pad0 / Bk;  // live blocks before the own one: jmin .. b - 1
  const int nsel = max(0, b - jmin), want = min(sh.topk - 1, nsel);
  if (nsel > want && want > 0) {
    for (int j = jmin + lane; j < b; j += 32) P[j] = 0.0;
    const double *kbase = mean + (int64_t)u * M * D;
    for (int hg = 0; hg < sh.G; ++hg) {
      __syncwarp();
      const T *qp = q + row_offset(sh, n, hk * sh.G + hg, t);
      for (int c = lane; c < D; c += 32) qrow[c] = (double)ld1(qp + c);
      __syncwarp();
      double mx = -INFINITY;
      for (int j = jmin + lane; j < b; j += 32) {
        const double *kj = kbase + (int64_t)j * D;
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
#pragma unroll 4
        for (int c = 0; c < D; c += 4) {
          a0 = fma(qrow[c], kj[c], a0);
          a1 = fma(qrow[c + 1], kj[c + 1], a1);
          a2 = fma(qrow[c + 2], kj[c + 2], a2);
          a3 = fma(qrow[c + 3], kj[c + 3], a3);
        }
        const double z = sh.scale_d * ((a0 + a1) + (a2 + a3));
        Z[j] = z;
        mx = fmax(mx, z);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      double den = 0.0;
      for (int j = jmin + lane; j < b; j += 32) {
        const double e = exp(Z[j] - mx);
        Z[j] = e;
        den += e;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
      for (int j = jmin + lane; j < b; j += 32) P[j] += Z[j] / den;  // heads in ascending order
    }
    __syncwarp();
    rank_select<double>(P, jmin, b, want, taken, bound_d[warp], lane);
  } else {
    for (int j = jmin + lane; j < b; j += 32) taken[j] = want > 0 ? 1 : 0;
  }
  __syncwarp();
  emit_row(row, taken, jmin, b, sh.topk, lane);
}

// The same selection, tiled: one CTA of 256 threads per 64 consecutive positions of a (batch,
// key/value head), for up to 64 NZ scored blocks (the selection blocks themselves, or overlapping
// compression blocks whose probabilities Eq. 11 maps onto the selection blocks, row by row).  The 64 query rows of one head at a time and
// 64 candidate means at a time sit in shared memory as doubles; thread (row tid / 4, part tid % 4)
// forms the 16 logits of candidates part + 4 k per chunk (sixteen independent accumulation
// chains) and keeps the logits of all chunks in registers; the row's softmax takes 4 lanes; the
// probabilities are added, head after head, into a [64 rows][64 NZ] table in shared memory, from
// which one warp per row ranks and emits.  The means are read once per tile and head instead of
// once per position and head.
template <typename T, int D, int NZ>
__global__ void __launch_bounds__(256, NZ == 1 ? 2 : 1) score_per_query_tile_kernel(
    Shape sh, SelGeom g, const T *__restrict__ q, const double *__restrict__ mean,
    const int32_t *__restrict__ seq_lens, int32_t *__restrict__ idx) {
  grid_chain_enter();
  constexpr int PD = D + 1, MP = 64 * NZ;
  extern __shared__ double dsm[];
  __shared__ double bound_d[8][2];
  double *qd = dsm;                // [64][PD] query rows of the current head
  double *kd = qd + 64 * PD;       // [64][PD] a chunk of candidate means
  double *P = kd + 64 * PD;        // [64][MP] probabilities summed over the group's heads
  double *Smap = P + 64 * MP;      // [8 warps][MP] a row's scores of the selection blocks (Eq. 11; overlapping mode)
  uint8_t *taken_all = reinterpret_cast<uint8_t *>(Smap + (g.plain ? 0 : 8 * MP));  // [8 warps][MP]
  const int M = sh.M, Bk = sh.Bk;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rt = tid >> 2, part = tid & 3;
  const int ntile = (sh.L + 63) / 64;
  const int u = (int)(blockIdx.x / ntile), tile = (int)(blockIdx.x % ntile), n = u / sh.Hkv, hk = u % sh.Hkv;
  int len = seq_lens ? seq_lens[n] : sh.L;
  len = min(max(len, 0), sh.L);
  const int pad0 = sh.L - len;
  const int t0 = tile * 64, t_last = min(t0 + 63, sh.L - 1);
  const int jmin = pad0 / Bk;                    // selectable selection blocks: j >= jmin
  const int cmin = first_live_scored(g, pad0);   // live scored blocks: c >= cmin
  // candidates of the tile's rows: scored blocks cmin .. nc - 1 (row t: those that end before block t / Bk)
  const int nc = n_candidates(sh, g, t_last / Bk);
  const int t = t0 + rt;
  const bool row_on = t >= pad0 && t < sh.L;
  const int nc_row = row_on ? n_candidates(sh, g, t / Bk) : 0;

  if (t_last >= pad0 && nc > cmin) {
    for (int i = tid; i < 64 * MP; i += 256) P[i] = 0.0;
    const int ch_lo = cmin / 64, ch_hi = (nc + 63) / 64;  // at most NZ chunks apart (host-checked: blocks <= 64 NZ)
    const double *kbase = mean + (int64_t)u * g.n * D;
    for (int hg = 0; hg < sh.G; ++hg) {
      __syncthreads();  // the previous head's rows are no longer read
      for (int i = tid; i < 64 * (D / 4); i += 256) {
        const int lr = i / (D / 4), c = (i % (D / 4)) * 4, tt = t0 + lr;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (tt >= pad0 && tt < sh.L) v = ld4(q + row_offset(sh, n, hk * sh.G + hg, tt) + c);
        double *d = qd + lr * PD + c;
        d[0] = (double)v.x; d[1] = (double)v.y; d[2] = (double)v.z; d[3] = (double)v.w;
      }
      const double *qr = qd + rt * PD;
      double z[NZ][16];
      uint32_t on[NZ];
      double mx = -INFINITY;
#pragma unroll
      for (int ci = 0; ci < NZ; ++ci) {
        on[ci] = 0u;
        const int ch = ch_lo + ci;
        if (ch < ch_hi) {  // (block-uniform)
          const int c0 = ch * 64, nb = min(64, nc - c0);
          __syncthreads();  // previous users of kd are done (and qd is complete)
          for (int i = tid; i < 64 * (D / 2); i += 256) {
            const int lj = i / (D / 2), c = (i % (D / 2)) * 2;
            double2 v = make_double2(0.0, 0.0);
            if (lj < nb && c0 + lj >= cmin) v = *reinterpret_cast<const double2 *>(kbase + (int64_t)(c0 + lj) * D + c);
            kd[lj * PD + c] = v.x;
            kd[lj * PD + c + 1] = v.y;
          }
          __syncthreads();
#pragma unroll
          for (int k = 0; k < 16; ++k) z[ci][k] = 0.0;
#pragma unroll 2
          for (int c = 0; c < D; ++c) {
            const double qv = qr[c];
#pragma unroll
            for (int k = 0; k < 16; ++k) z[ci][k] = fma(qv, kd[(part + 4 * k) * PD + c], z[ci][k]);
          }
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            z[ci][k] *= sh.scale_d;
            const int c = c0 + part + 4 * k;
            if (row_on && c >= cmin && c < nc_row) {
              on[ci] |= 1u << k;
              mx = fmax(mx, z[ci][k]);
            }
          }
        }
      }
      mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      double den = 0.0;
#pragma unroll
      for (int ci = 0; ci < NZ; ++ci)
#pragma unroll
        for (int k = 0; k < 16; ++k)
          if ((on[ci] >> k) & 1u) {
            z[ci][k] = exp(z[ci][k] - mx);
            den += z[ci][k];
          }
      den += __shfl_xor_sync(0xffffffffu, den, 1);
      den += __shfl_xor_sync(0xffffffffu, den, 2);
#pragma unroll
      for (int ci = 0; ci < NZ; ++ci)
#pragma unroll
        for (int k = 0; k < 16; ++k)
          if ((on[ci] >> k) & 1u) P[rt * MP + (ch_lo + ci) * 64 - ch_lo * 64 + part + 4 * k] += z[ci][k] / den;  // heads in ascending order
    }
  }
  __syncthreads();
  // one warp per row: Eq. 11 and Eq. 13 from the row's summed probabilities (table column =
  // scored block - 64 ch_lo)
  const int col0 = (cmin / 64) * 64;
  uint8_t *taken = taken_all + warp * MP;
  double *Srow = Smap + warp * MP;
  for (int lr = warp; lr < 64; lr += 8) {
    const int tt = t0 + lr;
    if (tt >= sh.L) break;
    int32_t *row = idx + ((int64_t)u * sh.L + tt) * sh.topk;
    if (tt < pad0) {
      for (int i = lane; i < sh.topk; i += 32) row[i] = -1;
      continue;
    }
    const int b = tt / Bk, nsel = max(0, b - jmin), want = min(sh.topk - 1, nsel);
    __syncwarp();
    if (nsel > want && want > 0) {
      if (g.plain) {
        rank_select<double>(P + lr * MP - col0, jmin, b, want, taken, bound_d[warp], lane);
      } else if (n_candidates(sh, g, b) > cmin) {
        map_scores<double>(g, P + lr * MP - col0, cmin, n_candidates(sh, g, b), jmin, b, Srow, lane);
        __syncwarp();
        rank_select<double>(Srow, jmin, b, want, taken, bound_d[warp], lane);
      } else {  // no compression block lies in the past yet: all scores are zero, the lowest blocks win the ties
        for (int j = jmin + lane; j < b; j += 32) taken[j] = j - jmin < want ? 1 : 0;
      }
    } else {
      for (int j = jmin + lane; j < b; j += 32) taken[j] = want > 0 ? 1 : 0;
    }
    __syncwarp();
    emit_row(row, taken, jmin, b, sh.topk, lane);
  }
}

// The arrays the selection kernels work in (the caller's workspace or the built-in scratch).
struct SelBuffers {
  double *mean;
  int32_t *live;
  float *mean32, *norm;
  int32_t *list, *count;
};

// Dynamic shared memory of the two scoring kernels; 0 = the single-precision stage does not take
// this shape (more score slots per CTA than it keeps) and every query block goes to stage 2.
size_t fast_smem_bytes(const Shape &sh, const SelGeom &g, int D, int *sc_pitch) {
  const int nqb = kRowTile / sh.Bk;
  *sc_pitch = ((g.n + kChunk - 1) / kChunk) * kChunk;
  const size_t slots = (size_t)nqb * *sc_pitch + (g.plain ? 0 : (size_t)nqb * sh.M);
  if (slots > 20480) return 0;
  return ((size_t)(kRowTile + kChunk) * (D + 4) + 4 * 8 * 64 + slots) * sizeof(float) + (size_t)nqb * sh.M + 16;
}
size_t exact_smem_bytes(const Shape &sh, const SelGeom &g, int D, int *sc_len) {
  *sc_len = ((g.n + 63) / 64) * 64;
  return ((size_t)64 * (D + 1) + 64 * 65 + 256 + *sc_len + sh.M) * sizeof(double) + (size_t)sh.M + 16;
}

template <typename T, int D>
int launch_select_t(const Shape &sh, const T *q, const T *k, const int32_t *seq_lens, int32_t *idx,
                    const SelBuffers &w, cudaStream_t st) {
  const SelGeom g = sel_geom(sh);
  const int64_t units = (int64_t)sh.B * sh.Hkv;
  if (g.n > 0) {
    LaunchScope ls(K_SUMMARY, st);
    auto summary = sh.phi ? summary_kernel<T, D, true> : summary_kernel<T, D, false>;
    summary<<<(unsigned)((units * g.n + 7) / 8), 256, 0, st>>>(sh, g, k, seq_lens, w.mean, w.live, w.mean32, w.norm,
                                                               w.count);
  } else if (cudaMemsetAsync(w.count, 0, sizeof(int32_t), st) != cudaSuccess) {
    return BLOSSOM_ERR_CUDA;
  }
  if (sh.pq) {  // one selection per query position: block_idx is [B][Hkv][L][top_k]
    if (g.n <= 128 && sh.M <= 128) {  // the tiled kernel keeps the logits of up to two chunks of 64 blocks in registers
      const int nz = (g.n <= 64 && sh.M <= 64) ? 1 : 2;
      const size_t tsm = ((size_t)2 * 64 * (D + 1) + (size_t)64 * 64 * nz + (g.plain ? 0 : (size_t)8 * 64 * nz)) * sizeof(double) +
                         (size_t)8 * 64 * nz + 16;
      auto kern = nz == 1 ? score_per_query_tile_kernel<T, D, 1> : score_per_query_tile_kernel<T, D, 2>;
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tsm) != cudaSuccess)
        return BLOSSOM_ERR_CUDA;
      LaunchScope ls(K_SCORE_SELECT, st);
      launch_chained(kern, dim3((unsigned)(units * ((sh.L + 63) / 64))), dim3(256), tsm, st, sh, g, q,
                     (const double *)w.mean, seq_lens, idx);
      return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
    }
    if (!g.plain) return BLOSSOM_ERR_UNSUPPORTED;  // (more than 128 blocks: the per-warp kernel scores selection blocks only)
    const size_t psm = (size_t)8 * (2 * sh.M + D) * sizeof(double) + (size_t)8 * sh.M + 16;
    if (psm > 48 * 1024 && cudaFuncSetAttribute(score_per_query_kernel<T, D>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)psm) != cudaSuccess)
      return BLOSSOM_ERR_CUDA;
    LaunchScope ls(K_SCORE_SELECT, st);
    launch_chained(score_per_query_kernel<T, D>, dim3((unsigned)((units * sh.L + 7) / 8)), dim3(256), psm, st, sh, q,
                   (const double *)w.mean, seq_lens, idx);
    return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
  }
  int sc_pitch = 0, sc_len = 0;
  const size_t fsm = fast_smem_bytes(sh, g, D, &sc_pitch);
  // (without the causal mask the candidates are not a prefix of the blocks: double precision only)
  const bool exact_only = exact_select_only() || fsm == 0 || !sh.causal;
  if (!exact_only) {
    if (fsm > 48 * 1024 && cudaFuncSetAttribute(score_fast_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)fsm) != cudaSuccess)
      return BLOSSOM_ERR_CUDA;
    const unsigned ntiles = (unsigned)((sh.L + kRowTile - 1) / kRowTile);
    LaunchScope ls(K_SCORE_FAST, st);
    launch_chained(score_fast_kernel<T, D>, dim3(ntiles * (unsigned)units), dim3(kFastThreads), fsm, st, sh, g, q,
                   (const float *)w.mean32, (const float *)w.norm, seq_lens, idx, w.list, w.count, sc_pitch);
  }
  const size_t esm = exact_smem_bytes(sh, g, D, &sc_len);
  auto exact = g.n > 64 ? score_exact_kernel<T, D, 2> : score_exact_kernel<T, D, 1>;
  if (esm > 48 * 1024 &&
      cudaFuncSetAttribute(exact, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)esm) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    // double precision: every query block (exact_only) or the work list of the kernel above
    LaunchScope ls(K_SCORE_SELECT, st);
    const int64_t rows = units * sh.M;
    const int chunks = (sh.G * sh.Bk + 63) / 64;  // 64-row chunks of a query block
    const unsigned cl = chunks >= 8 ? 8u : chunks >= 4 ? 4u : chunks >= 2 ? 2u : 1u;
    const int64_t max_clusters = 592 / cl;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(rows < max_clusters ? rows : max_clusters) * cl);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = esm;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // chained behind the kernel before it
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained_launches() ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, exact, sh, g, q, (const double *)w.mean, seq_lens, idx,
                           (const int32_t *)(exact_only ? nullptr : w.list), (const int32_t *)w.count,
                           sc_len) != cudaSuccess)
      return BLOSSOM_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

int launch_select_buffers(const Shape &s, int dtype, const void *q, const void *k, const int32_t *seq_lens,
                          int32_t *idx, const SelBuffers &w, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == BLOSSOM_DTYPE_FP32) {
    if (s.D == 32) return launch_select_t<float, 32>(s, (const float *)q, (const float *)k, seq_lens, idx, w, st);
    return launch_select_t<float, 64>(s, (const float *)q, (const float *)k, seq_lens, idx, w, st);
  }
  if (s.D == 32) return launch_select_t<bf, 32>(s, (const bf *)q, (const bf *)k, seq_lens, idx, w, st);
  return launch_select_t<bf, 64>(s, (const bf *)q, (const bf *)k, seq_lens, idx, w, st);
}

}  // namespace

int launch_select(const Shape &s, int dtype, const void *q, const void *k, const int32_t *seq_lens,
                  int32_t *idx, const Workspace &ws, cudaStream_t st) {
  SelBuffers w;
  if (s.cmp_l > 0) {  // the means of the overlapping compression blocks have arrays of their own
    w.mean = ws.cmean; w.live = ws.clive; w.mean32 = ws.cmean32; w.norm = ws.cnorm;
  } else {
    w.mean = ws.kmean; w.live = ws.klive; w.mean32 = ws.kmean32; w.norm = ws.knorm;
  }
  w.list = ws.sel_list;
  w.count = ws.sel_count;
  return launch_select_buffers(s, dtype, q, k, seq_lens, idx, w, st);
}

// ---- selection with built-in scratch (no allocation anywhere on the call path) -------------
// The block means and live counts that blossom_select_blocks keeps in the caller's workspace
// live here in one array that is part of the loaded module.  Every launch overwrites each entry
// it later reads, so nothing has to start at zero and stale contents of earlier calls are
// harmless; two calls in flight at once on one device would overwrite each other's means.
constexpr size_t kStaticMeanElems = 524288;  // doubles: batch * kv_heads * M * head_dim may not exceed this
constexpr size_t kStaticBlocks = 8192;       // int32:   batch * kv_heads * M may not exceed this
// doubles (means) | floats (fp32 means) | int32 live counts | float norms | int32 work list | counter
constexpr size_t kStaticOffMean32 = kStaticMeanElems * sizeof(double);
constexpr size_t kStaticOffLive = kStaticOffMean32 + kStaticMeanElems * sizeof(float);
constexpr size_t kStaticOffNorm = kStaticOffLive + kStaticBlocks * sizeof(int32_t);
constexpr size_t kStaticOffList = kStaticOffNorm + kStaticBlocks * sizeof(float);
constexpr size_t kStaticOffCount = kStaticOffList + kStaticBlocks * sizeof(int32_t);
constexpr size_t kStaticBytes = kStaticOffCount + 256;
static __device__ __align__(256) unsigned char g_select_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
static void *g_scratch_addr[kMaxDevices] = {nullptr};  // device address of the array, per device

size_t select_static_capacity_bytes() { return kStaticBytes; }

int launch_select_static(const Shape &s, int dtype, const void *q, const void *k,
                         const int32_t *seq_lens, int32_t *idx, cudaStream_t st) {
  // the built-in scratch serves the plain selection (and has no room for rotated copies of q and k)
  if (s.cmp_l > 0 || s.pq || s.rope_theta > 0) return BLOSSOM_ERR_UNSUPPORTED;
  const size_t blocks = (size_t)s.B * s.Hkv * s.M;  // every scratch array is per key/value head
  if (blocks > kStaticBlocks || blocks * (size_t)s.D > kStaticMeanElems) return BLOSSOM_ERR_TOO_LARGE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BLOSSOM_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    // In host code the array's name is only a handle: ask the runtime for its device address on
    // the current device (once per device) and hand that to the kernels.
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || !p) return BLOSSOM_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  unsigned char *base = static_cast<unsigned char *>(g_scratch_addr[dev]);
  SelBuffers w;
  w.mean = reinterpret_cast<double *>(base);
  w.mean32 = reinterpret_cast<float *>(base + kStaticOffMean32);
  w.live = reinterpret_cast<int32_t *>(base + kStaticOffLive);
  w.norm = reinterpret_cast<float *>(base + kStaticOffNorm);
  w.list = reinterpret_cast<int32_t *>(base + kStaticOffList);
  w.count = reinterpret_cast<int32_t *>(base + kStaticOffCount);
  return launch_select_buffers(s, dtype, q, k, seq_lens, idx, w, st);
}

}  // namespace blossom
