// Block selection with overlapping compression blocks (paper Eq. 8-11 and 13).
//
// Compression blocks K_i = positions [s i, s i + l), i < Mc = floor((L - l) / s) + 1, are
// summarised by the mean of their valid keys (Eq. 9 with the summary = mean).  A query block
// (selection blocks of Bk positions) scores the live compression blocks that end before it starts
// (Eq. 10 per query, summed over the block's valid queries), Eq. 11 maps those scores onto the past
// selection blocks, S[j] = sum_{m < Bk/s} sum_{n < l/s} Sc[(Bk/s) j - m - n] (terms out of range or
// not scored are zero), and the own block plus the top_k - 1 best past blocks are kept, ties to
// the lower index (Eq. 13).  As in the plain selection the choice is the one a double-precision
// evaluation makes: a single-precision stage with a rigorous error bound decides the query blocks
// whose choice is certain, a double-precision kernel the rest.
// This path serves cmp_block / cmp_stride different from block_size; the plain selection
// (select.cu) stays as it is.
#include "common.cuh"

namespace blossom {
namespace {

constexpr int kCmpThreads = 256;
constexpr int kCmpWarps = kCmpThreads / 32;

// grid Mc * B * H (unit-major), 256 threads: mean of the valid keys of one compression block
template <typename T, int D>
__global__ void __launch_bounds__(256) cmp_summary_kernel(Shape s, const T *__restrict__ k,
                                                          const int32_t *__restrict__ seq_lens,
                                                          double *__restrict__ cmean,
                                                          int32_t *__restrict__ clive,
                                                          float *__restrict__ cmean32,
                                                          float *__restrict__ cnorm,
                                                          int32_t *__restrict__ sel_count) {
  constexpr int CH = D / 4, RG = 256 / CH;
  __shared__ double part[RG][D];
  __shared__ float sq[D];
  if (blockIdx.x == 0 && threadIdx.x == 0) *sel_count = 0;  // work list of the scoring kernel
  const int i = blockIdx.x % s.Mc, u = blockIdx.x / s.Mc, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int lo = max(i * s.cmp_s, pad0), hi = i * s.cmp_s + s.cmp_l;  // hi <= L by the count Mc
  const int ch = threadIdx.x % CH, rg = threadIdx.x / CH;
  double a0 = 0, a1 = 0, a2 = 0, a3 = 0;
  for (int p = lo + rg; p < hi; p += RG) {
    const float4 x = ld4(k + row_offset(s, n, h, p) + ch * 4);
    a0 += (double)x.x; a1 += (double)x.y; a2 += (double)x.z; a3 += (double)x.w;
  }
  part[rg][ch * 4 + 0] = a0; part[rg][ch * 4 + 1] = a1;
  part[rg][ch * 4 + 2] = a2; part[rg][ch * 4 + 3] = a3;
  __syncthreads();
  const int cnt = max(hi - lo, 0);
  if (threadIdx.x < D) {
    double acc = 0;
    for (int r = 0; r < RG; ++r) acc += part[r][threadIdx.x];  // fixed order
    const double mean = cnt > 0 ? acc / (double)cnt : 0.0;
    cmean[((int64_t)u * s.Mc + i) * D + threadIdx.x] = mean;
    const float m32 = (float)mean;
    cmean32[((int64_t)u * s.Mc + i) * D + threadIdx.x] = m32;
    sq[threadIdx.x] = m32 * m32;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    clive[(int64_t)u * s.Mc + i] = cnt;
    float a = 0.f;
    for (int c = 0; c < D; ++c) a += sq[c];
    cnorm[(int64_t)u * s.Mc + i] = sqrtf(a) * 1.0001f;  // an upper bound of the fp32 mean's norm
  }
}

// grid M * B * H (unit-major), 256 threads: one query block.  One warp per query row, lanes over
// the candidate compression blocks; per-warp partial sums, fixed-order combine, Eq. 11, rank
// selection.  Shared memory (doubles): zbuf[8][Mc], sp[8][Mc], qrow[8][D], Sc[Mc], S[M];
// ints: livec[Mc], taken[M].
template <typename T, int D>
__global__ void __launch_bounds__(kCmpThreads) cmp_score_select_kernel(
    Shape s, const T *__restrict__ q, const double *__restrict__ cmean,
    const int32_t *__restrict__ clive, const int32_t *__restrict__ seq_lens,
    int32_t *__restrict__ idx, int means_in_smem, const int32_t *__restrict__ worklist,
    const int32_t *__restrict__ work_count) {
  extern __shared__ double smd[];
  // every query block, or (worklist != nullptr) the ones the single-precision stage left open
  const int total = worklist ? *work_count : s.M * s.B * s.H;
  for (int wi = blockIdx.x; wi < total; wi += gridDim.x) {
  const int row_id = worklist ? worklist[wi] : wi;
  __syncthreads();  // shared memory is reused from the previous row
  const int M = s.M, Mc = max(s.Mc, 1);
  double *zbuf = smd, *sp = zbuf + kCmpWarps * Mc, *qrow = sp + kCmpWarps * Mc;
  double *Sc = qrow + kCmpWarps * D, *S = Sc + Mc;
  int *livec = reinterpret_cast<int *>(S + M), *taken = livec + Mc;
  // the candidates' means, row pitch D + 1 doubles (conflict-free when lanes read different rows)
  double *kt_s = reinterpret_cast<double *>(taken + M + ((Mc + M) & 1));
  const int b = row_id % M, u = row_id / M, n = u / s.H, h = u % s.H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int qlo = max(b * s.Bk, pad0), qhi = min((b + 1) * s.Bk, s.L);
  int32_t *row = idx + ((int64_t)u * M + b) * s.topk;
  if (qlo >= qhi) {  // the query block holds only padding
    for (int i = tid; i < s.topk; i += kCmpThreads) row[i] = -1;
    continue;
  }
  // candidates: compression blocks 0 .. nc-1 end before the query block starts
  const int nc = b * s.Bk >= s.cmp_l ? min(s.Mc, (b * s.Bk - s.cmp_l) / s.cmp_s + 1) : 0;
  const double *kt = cmean + (int64_t)u * s.Mc * D;
  int kpitch = D;
  if (means_in_smem) {
    for (int i = tid; i < nc * D; i += kCmpThreads) kt_s[(i / D) * (D + 1) + (i % D)] = kt[i];
    kt = kt_s;
    kpitch = D + 1;
  }
  for (int i = tid; i < nc; i += kCmpThreads) livec[i] = clive[(int64_t)u * s.Mc + i] > 0;
  for (int i = tid; i < kCmpWarps * Mc; i += kCmpThreads) sp[i] = 0.0;
  __syncthreads();
  int ncand = 0;
  for (int base = 0; base < nc; base += kCmpThreads)
    ncand += __syncthreads_count(base + tid < nc && livec[base + tid]);

  if (ncand > 0) {  // Eq. 10 per query, summed over the block's valid queries
    double *zw = zbuf + warp * Mc, *spw = sp + warp * Mc, *qw = qrow + warp * D;
    for (int t = qlo + warp; t < qhi; t += kCmpWarps) {
      const T *qp = q + row_offset(s, n, h, t);
      for (int c = lane; c < D; c += 32) qw[c] = (double)ld1(qp + c);
      __syncwarp();
      double mx = -INFINITY;
      for (int i = lane; i < nc; i += 32) {
        if (!livec[i]) continue;
        const double *ki = kt + (int64_t)i * kpitch;
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
#pragma unroll 4
        for (int c = 0; c < D; c += 4) {
          a0 = fma(qw[c], ki[c], a0);
          a1 = fma(qw[c + 1], ki[c + 1], a1);
          a2 = fma(qw[c + 2], ki[c + 2], a2);
          a3 = fma(qw[c + 3], ki[c + 3], a3);
        }
        const double z = s.scale_d * ((a0 + a1) + (a2 + a3));
        zw[i] = z;
        mx = fmax(mx, z);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      double den = 0.0;
      for (int i = lane; i < nc; i += 32)
        if (livec[i]) {
          const double e = exp(zw[i] - mx);
          zw[i] = e;
          den += e;
        }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
      for (int i = lane; i < nc; i += 32)
        if (livec[i]) spw[i] += zw[i] / den;
      __syncwarp();
    }
  }
  __syncthreads();
  for (int i = tid; i < nc; i += kCmpThreads) {
    double acc = 0.0;
    for (int w = 0; w < kCmpWarps; ++w) acc += sp[w * Mc + i];  // fixed order
    Sc[i] = livec[i] ? acc : 0.0;
  }
  __syncthreads();
  // Eq. 11 and which past selection blocks hold a valid key (taken: 2 = not selectable)
  const int rs = s.Bk / s.cmp_s, rl = s.cmp_l / s.cmp_s;
  int nlive = 0;
  for (int base = 0; base < b; base += kCmpThreads) {
    const int j = base + tid;
    bool lv = false;
    if (j < b) {
      double acc = 0.0;
      for (int m = 0; m < rs; ++m)
        for (int e = 0; e < rl; ++e) {
          const int i = rs * j - m - e;
          if (i >= 0 && i < nc) acc += Sc[i];
        }
      S[j] = acc;
      lv = min((j + 1) * s.Bk, s.L) > max(j * s.Bk, pad0);
      taken[j] = lv ? 0 : 2;
    }
    nlive += __syncthreads_count(lv);
  }
  __syncthreads();
  // Eq. 13 by rank: a live block is kept iff fewer than `want` live blocks beat it (larger score,
  // or equal score and lower index)
  const int want = min(s.topk - 1, nlive);
  for (int j = tid; j < b; j += kCmpThreads) {
    if (taken[j] == 2) continue;
    const double sj = S[j];
    int rank = 0;
    for (int i = 0; i < b; ++i)
      if (taken[i] != 2) {
        const double si = S[i];
        rank += (si > sj || (si == sj && i < j)) ? 1 : 0;
      }
    if (rank < want) taken[j] = 1;  // (other threads only test for 2: no race on the value read)
  }
  __syncthreads();
  if (warp == 0) {  // emit ascending, then the own block
    int pos = 0;
    for (int base = 0; base < b; base += 32) {
      const int j = base + lane;
      const bool f = j < b && taken[j] == 1;
      const unsigned mk = __ballot_sync(0xffffffffu, f);
      if (f) row[pos + __popc(mk & ((1u << lane) - 1u))] = j;
      pos += __popc(mk);
    }
    if (lane == 0) row[pos] = b;
    for (int i = pos + 1 + lane; i < s.topk; i += 32) row[i] = -1;
  }
  }  // rows
}

// ---- single-precision first stage with an error bound -------------------------------------
// One query block per CTA, as in the plain selection: fp32 logits of the block's (up to 64) queries
// against 64 candidate means at a time (thread = 4 queries x 4 candidates, out of shared memory),
// softmax per query row by 4 lanes (two passes over the candidate chunks: statistics, then
// probabilities), fixed-order column sums Sc, Eq. 11 in fp32, rank selection.
// Error bound: with u = 2^-24 every logit is within E = (D + 4) u scale max|q_t| max|mean_i| of
// exact, so every probability is within a factor exp(+-2E); the fp32 softmax and column sums add
// 2^-21 + 2^-22 per unit of logit range + (nc/4 + 80 + 8 chunks) u, and Eq. 11 one rounding per
// added term.  Two selection scores a > b are in certain order when a - b > R (a + b); query blocks
// whose last kept and first dropped block are closer go on the work list for the fp64 kernel.
template <typename T, int D>
__global__ void __launch_bounds__(256, 4) cmp_score_select_fast_kernel(
    Shape s, const T *__restrict__ q, const float *__restrict__ cmean32, const float *__restrict__ cnorm,
    const int32_t *__restrict__ clive, const int32_t *__restrict__ seq_lens, int32_t *__restrict__ idx,
    int32_t *__restrict__ worklist, int32_t *__restrict__ work_count) {
  constexpr int P = D + 4, ZP = 68, NT = 256;
  extern __shared__ float fsm[];
  __shared__ float rn[64];
  __shared__ float csum[256];
  __shared__ float bound_s[2];
  __shared__ int kn_bits;
  const int M = s.M, Mc = max(s.Mc, 1);
  float *qs = fsm;                           // [64][P]  the block's queries
  float *ks = qs + 64 * P;                   // [64][P]  a chunk of candidate means; reused as zs [64][ZP]
  float *zs = ks;
  float *Sc = ks + 64 * (P > ZP ? P : ZP);   // [Mc] compression scores
  float *S = Sc + Mc;                        // [M]  selection scores (Eq. 11)
  int *livec = reinterpret_cast<int *>(S + M);  // [Mc]
  int *taken = livec + Mc;                      // [M]  0 selectable, 1 kept, 2 not selectable

  const int b = blockIdx.x % M, u = blockIdx.x / M, n = u / s.H, h = u % s.H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int qlo = max(b * s.Bk, pad0), qhi = min((b + 1) * s.Bk, s.L);
  int32_t *row = idx + ((int64_t)u * M + b) * s.topk;
  if (qlo >= qhi) {  // the query block holds only padding
    for (int i = tid; i < s.topk; i += NT) row[i] = -1;
    return;
  }
  const int nc = b * s.Bk >= s.cmp_l ? min(s.Mc, (b * s.Bk - s.cmp_l) / s.cmp_s + 1) : 0;
  if (tid == 0) kn_bits = 0;
  for (int i = tid; i < nc; i += NT) {
    livec[i] = clive[(int64_t)u * s.Mc + i] > 0;
    Sc[i] = 0.f;
  }
  __syncthreads();
  int ncand = 0, nlive = 0;
  for (int base = 0; base < nc; base += NT) ncand += __syncthreads_count(base + tid < nc && livec[base + tid]);
  for (int base = 0; base < b; base += NT) {
    const int j = base + tid;
    const bool lv = j < b && min((j + 1) * s.Bk, s.L) > max(j * s.Bk, pad0);
    if (j < b) taken[j] = lv ? 0 : 2;
    nlive += __syncthreads_count(lv);
  }
  const int want = min(s.topk - 1, nlive);
  const bool choose = nlive > want && want > 0 && ncand > 0;  // a real choice that needs scores

  if (choose) {
    for (int i = tid; i < 64 * (D / 4); i += NT) {  // the query block, fp32, invalid rows zero
      const int lt = i / (D / 4), c = (i % (D / 4)) * 4, t = b * s.Bk + lt;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lt < s.Bk && t >= qlo && t < qhi) v = ld4(q + row_offset(s, n, h, t) + c);
      *reinterpret_cast<float4 *>(qs + lt * P + c) = v;
    }
    {
      float km = 0.f;
      for (int i = tid; i < nc; i += NT)
        if (livec[i]) km = fmaxf(km, cnorm[(int64_t)u * s.Mc + i]);
      if (km > 0.f) atomicMax(&kn_bits, __float_as_int(km));  // positive floats order like ints
    }
    __syncthreads();
    if (tid < 64) {
      float a = 0.f;
      for (int c = 0; c < D; ++c) a = fmaf(qs[tid * P + c], qs[tid * P + c], a);
      rn[tid] = sqrtf(a) * 1.0001f;
    }
    const int ty = tid >> 4, tx = tid & 15;  // product: queries ty + 16 a, candidates tx + 16 e
    const int rt = tid >> 2, part = tid & 3;  // softmax: row rt, candidates part, part + 4, ...
    const bool row_valid = rt < s.Bk && b * s.Bk + rt >= qlo && b * s.Bk + rt < qhi;
    const int nchunks = (nc + 63) / 64;
    const float *kbase = cmean32 + (int64_t)u * s.Mc * D;
    float mx = -INFINITY, den = 0.f;  // online softmax statistics of row rt

    for (int pass = 0; pass < 2; ++pass) {
      for (int ch = 0; ch < nchunks; ++ch) {
        const int j0 = ch * 64, nb = min(64, nc - j0), ne = (nb + 15) >> 4;
        __syncthreads();  // previous users of ks / zs are done
        for (int i = tid; i < 64 * (D / 4); i += NT) {
          const int lj = i / (D / 4), c = (i % (D / 4)) * 4;
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (lj < nb && livec[j0 + lj]) v = *reinterpret_cast<const float4 *>(kbase + (int64_t)(j0 + lj) * D + c);
          *reinterpret_cast<float4 *>(ks + lj * P + c) = v;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[a][e] = 0.f;
#pragma unroll 4
        for (int c = 0; c < D; c += 4) {
          float4 qa[4], kb[4];
#pragma unroll
          for (int a = 0; a < 4; ++a) {
            qa[a] = *reinterpret_cast<const float4 *>(qs + (ty + 16 * a) * P + c);
            if (a < ne) kb[a] = *reinterpret_cast<const float4 *>(ks + (tx + 16 * a) * P + c);
          }
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (e < ne) {
#pragma unroll
              for (int a = 0; a < 4; ++a) {
                acc[a][e] = fmaf(qa[a].x, kb[e].x, acc[a][e]);
                acc[a][e] = fmaf(qa[a].y, kb[e].y, acc[a][e]);
                acc[a][e] = fmaf(qa[a].z, kb[e].z, acc[a][e]);
                acc[a][e] = fmaf(qa[a].w, kb[e].w, acc[a][e]);
              }
            }
        }
        __syncthreads();  // everyone has read ks: it becomes zs
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int e = 0; e < 4; ++e) zs[(ty + 16 * a) * ZP + tx + 16 * e] = s.scale * acc[a][e];
        __syncthreads();
        if (pass == 0) {  // fold the chunk into (mx, den) of row rt
          float cm = -INFINITY;
          for (int j = part; j < nb; j += 4)
            if (livec[j0 + j]) cm = fmaxf(cm, zs[rt * ZP + j]);
          cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
          cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
          const float nm = fmaxf(mx, cm);
          float e = 0.f;
          if (nm > -INFINITY)
            for (int j = part; j < nb; j += 4)
              if (livec[j0 + j]) e += __expf(zs[rt * ZP + j] - nm);
          e += __shfl_xor_sync(0xffffffffu, e, 1);
          e += __shfl_xor_sync(0xffffffffu, e, 2);
          den = (mx > -INFINITY ? den * __expf(mx - nm) : 0.f) + e;
          mx = nm;
        } else {  // probabilities in place, then their column sums
          const float inv = den > 0.f ? 1.f / den : 0.f;
          for (int j = part; j < nb; j += 4) {
            const bool on = row_valid && livec[j0 + j];
            zs[rt * ZP + j] = on ? __expf(zs[rt * ZP + j] - mx) * inv : 0.f;
          }
          __syncthreads();
          {  // column sums in a fixed order: four partial sums of 16 rows each, then their tree
            const int j = tid & 63, quarter = tid >> 6;
            float a = 0.f;
            if (j < nb) {
#pragma unroll
              for (int t = 0; t < 16; ++t) a += zs[(quarter * 16 + t) * ZP + j];
            }
            csum[tid] = a;
          }
          __syncthreads();
          if (tid < nb) Sc[j0 + tid] = (csum[tid] + csum[64 + tid]) + (csum[128 + tid] + csum[192 + tid]);
        }
      }
    }
    __syncthreads();
  }

  // Eq. 11 in fp32 (all terms non-negative), then selection by rank among the selectable blocks
  const int rs = s.Bk / s.cmp_s, rl = s.cmp_l / s.cmp_s;
  for (int j = tid; j < b; j += NT) {
    float acc = 0.f;
    if (choose)
      for (int m = 0; m < rs; ++m)
        for (int e = 0; e < rl; ++e) {
          const int i = rs * j - m - e;
          if (i >= 0 && i < nc && livec[i]) acc += Sc[i];
        }
    S[j] = acc;
  }
  __syncthreads();
  for (int j = tid; j < b; j += NT) {
    if (taken[j] == 2) continue;
    const float sj = S[j];
    int rank = 0;
    for (int i = 0; i < b; ++i)
      if (taken[i] != 2) {
        const float si = S[i];
        rank += (si > sj || (si == sj && i < j)) ? 1 : 0;
      }
    if (rank < want) taken[j] = 1;
    if (rank == want - 1) bound_s[0] = sj;  // the smallest kept score
    if (rank == want) bound_s[1] = sj;      // the largest dropped score
  }
  __syncthreads();

  if (warp == 0) {
    bool certain = true;  // without a real choice (or without any score: all zero) the rank rule is exact
    if (choose) {
      float qn = fmaxf(rn[lane], rn[lane + 32]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) qn = fmaxf(qn, __shfl_xor_sync(0xffffffffu, qn, o));
      const float kn = __int_as_float(kn_bits);
      const float uu = 5.9604645e-8f;  // 2^-24
      const float bound = s.scale * qn * kn;  // >= every |logit|
      const float E = (float)(D + 4) * uu * bound * 1.01f;
      const float R = 2.f * E + 4.77e-7f + 2.f * bound * 2.39e-7f +
                      ((float)nc * 0.25f + 80.f + 8.f * (float)((nc + 63) / 64) + (float)(rs * rl)) * uu;
      const float smin = bound_s[0], umax = bound_s[1];
      certain = (smin - umax) > R * (smin + umax) * 1.001f;
    }
    if (certain) {
      int pos = 0;
      for (int base = 0; base < b; base += 32) {
        const int j = base + lane;
        const bool f = j < b && taken[j] == 1;
        const unsigned mk = __ballot_sync(0xffffffffu, f);
        if (f) row[pos + __popc(mk & ((1u << lane) - 1u))] = j;
        pos += __popc(mk);
      }
      if (lane == 0) row[pos] = b;
      for (int i = pos + 1 + lane; i < s.topk; i += 32) row[i] = -1;
    } else if (lane == 0) {
      worklist[atomicAdd(work_count, 1)] = blockIdx.x;  // re-scored in double precision
    }
  }
}

size_t cmp_fast_smem_bytes(const Shape &s, int D) {
  const int P = D + 4, ZP = 68;
  const size_t Mc = s.Mc > 0 ? s.Mc : 1;
  return (size_t)(64 * P + 64 * (P > ZP ? P : ZP)) * sizeof(float) + (Mc + s.M) * (sizeof(float) + sizeof(int));
}

size_t cmp_smem_bytes(const Shape &s, int D, bool means_in_smem) {
  const size_t Mc = s.Mc > 0 ? s.Mc : 1;
  return (2 * (size_t)kCmpWarps * Mc + (size_t)kCmpWarps * D + Mc + s.M) * sizeof(double) +
         (Mc + s.M + ((Mc + s.M) & 1)) * sizeof(int) +
         (means_in_smem ? Mc * (size_t)(D + 1) * sizeof(double) : 0);
}

template <typename T, int D>
int launch_select_cmp_t(const Shape &s, const T *q, const T *k, const int32_t *seq_lens, int32_t *idx,
                        const Workspace &ws, cudaStream_t st) {
  const unsigned units = (unsigned)(s.B * s.H), rows = (unsigned)s.M * units;
  if (s.Mc > 0) {
    LaunchScope ls(K_SUMMARY, st);
    cmp_summary_kernel<T, D><<<(unsigned)s.Mc * units, 256, 0, st>>>(s, k, seq_lens, ws.cmean, ws.clive,
                                                                     ws.cmean32, ws.cnorm, ws.sel_count);
  } else if (cudaMemsetAsync(ws.sel_count, 0, sizeof(int32_t), st) != cudaSuccess) {
    return BLOSSOM_ERR_CUDA;
  }
  const bool exact_only = exact_select_only();
  if (!exact_only) {
    const size_t fsm = cmp_fast_smem_bytes(s, D);
    if (fsm > 100 * 1024) return BLOSSOM_ERR_UNSUPPORTED;
    if (fsm > 48 * 1024 &&
        cudaFuncSetAttribute(cmp_score_select_fast_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)fsm) != cudaSuccess)
      return BLOSSOM_ERR_CUDA;
    LaunchScope ls(K_SCORE_FAST, st);
    cmp_score_select_fast_kernel<T, D><<<rows, 256, fsm, st>>>(s, q, ws.cmean32, ws.cnorm, ws.clive, seq_lens,
                                                              idx, ws.sel_list, ws.sel_count);
  }
  const bool in_smem = cmp_smem_bytes(s, D, true) <= 160 * 1024;
  const size_t smem = cmp_smem_bytes(s, D, in_smem);
  if (smem > 200 * 1024) return BLOSSOM_ERR_UNSUPPORTED;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(cmp_score_select_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    // double precision: every query block (exact_only) or the work list of the kernel above
    LaunchScope ls(K_SCORE_SELECT, st);
    const unsigned g2 = exact_only ? rows : (rows < 592u ? rows : 592u);
    cmp_score_select_kernel<T, D><<<g2, kCmpThreads, smem, st>>>(s, q, ws.cmean, ws.clive, seq_lens, idx,
                                                                in_smem ? 1 : 0,
                                                                exact_only ? nullptr : ws.sel_list, ws.sel_count);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

int launch_select_cmp(const Shape &s, int dtype, const void *q, const void *k, const int32_t *seq_lens,
                      int32_t *idx, const Workspace &ws, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == BLOSSOM_DTYPE_FP32) {
    if (s.D == 32) return launch_select_cmp_t<float, 32>(s, (const float *)q, (const float *)k, seq_lens, idx, ws, st);
    return launch_select_cmp_t<float, 64>(s, (const float *)q, (const float *)k, seq_lens, idx, ws, st);
  }
  if (s.D == 32) return launch_select_cmp_t<bf, 32>(s, (const bf *)q, (const bf *)k, seq_lens, idx, ws, st);
  return launch_select_cmp_t<bf, 64>(s, (const bf *)q, (const bf *)k, seq_lens, idx, ws, st);
}

}  // namespace blossom
