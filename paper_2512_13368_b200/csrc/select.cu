// Block summary, importance scoring and top-k selection (paper Eq. 8-10, 12, 13 with
// compression size = stride = selection size = Bk and the summary = mean of a block's valid keys).
//
// The selection is a discrete decision taken from floating-point sums whose neighbours differ by
// ~1e-3 relative on Gaussian inputs, and the library promises the choice a double-precision
// evaluation makes (ties below ~1e-12 relative excepted).  Two stages deliver it:
//   1. every query block is scored in single precision together with a rigorous bound on the
//      distance of each score from its exact value; if the last kept and the first dropped
//      candidate are further apart than the bound allows them to move, the choice is certain and
//      is written out;
//   2. the (few per cent of) query blocks whose choice is not certain are appended to a work
//      list and re-scored in double precision by a second kernel.
#include "common.cuh"

namespace blossom {

namespace {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;

// ---- Eq. 8 + 9: per key block, mean of the valid keys (fp64) ------------------------------
// grid M*B*H (unit-major), 256 threads: thread = (row group, 4-element column chunk); 128-bit/64-bit loads.
template <typename T, int D>
__global__ void __launch_bounds__(256) summary_kernel(Shape s, const T *__restrict__ k,
                                                      const int32_t *__restrict__ seq_lens,
                                                      double *__restrict__ kmean,
                                                      int32_t *__restrict__ klive,
                                                      float *__restrict__ kmean32,
                                                      float *__restrict__ knorm,
                                                      int32_t *__restrict__ sel_count) {
  constexpr int CH = D / 4;        // chunks per row
  constexpr int RG = 256 / CH;     // row groups
  __shared__ double part[RG][D];
  __shared__ float sq[D];
  if (blockIdx.x == 0 && threadIdx.x == 0) *sel_count = 0;  // work list of the scoring kernel
  // u counts (batch, key/value head) pairs
  const int j = blockIdx.x % s.M, u = blockIdx.x / s.M, n = u / s.Hkv, hk = u % s.Hkv;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int lo = max(j * s.Bk, pad0), hi = min((j + 1) * s.Bk, s.L);
  const int ch = threadIdx.x % CH, rg = threadIdx.x / CH;
  double a0 = 0, a1 = 0, a2 = 0, a3 = 0;
  for (int p = lo + rg; p < hi; p += RG) {
    float4 x = ld4(k + row_offset_kv(s, n, hk, p) + ch * 4);
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
    kmean[((int64_t)u * s.M + j) * D + threadIdx.x] = mean;
    const float m32 = (float)mean;
    kmean32[((int64_t)u * s.M + j) * D + threadIdx.x] = m32;
    sq[threadIdx.x] = m32 * m32;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    klive[(int64_t)u * s.M + j] = cnt;
    float a = 0.f;
    for (int c = 0; c < D; ++c) a += sq[c];
    knorm[(int64_t)u * s.M + j] = sqrtf(a) * 1.0001f;  // an upper bound of the fp32 mean's norm
  }
}

// ---- Eq. 10 + 12 + 13: scores of one query block and its top-k --------------------------
// grid M*B*H (unit-major), 256 threads.  One warp per query row: lanes stride over the candidate blocks,
// softmax over the candidates, per-warp partial sums, fixed-order combine, then a candidate is
// kept iff fewer than top_k - 1 live candidates beat it (value desc, index asc).
template <typename T, int D>
__device__ __forceinline__ void score_select_row(
    const Shape &s, const T *__restrict__ q, const double *__restrict__ kmean,
    const int32_t *__restrict__ klive, const int32_t *__restrict__ seq_lens,
    int32_t *__restrict__ idx, int kt_in_smem, int row_id, double *sm) {
  // u counts (batch, key/value head) pairs; the queries of all G heads of the group are scored
  // and their probabilities summed (Eq. 12)
  const int b = row_id % s.M, u = row_id / s.M, n = u / s.Hkv, hk = u % s.Hkv;
  const int M = s.M;
  const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int qlo = max(b * s.Bk, pad0), qhi = min((b + 1) * s.Bk, s.L);
  int32_t *row = idx + ((int64_t)u * M + b) * s.topk;

  if (qlo >= qhi) {  // the query block holds only padding
    for (int i = tid; i < s.topk; i += kSelThreads) row[i] = -1;
    return;
  }

  double *zbuf = sm;                          // [warps][M]
  double *sp = zbuf + kSelWarps * M;          // [warps][M]
  double *qrow = sp + kSelWarps * M;          // [warps][D]
  double *S = qrow + kSelWarps * D;           // [M]
  int *live = reinterpret_cast<int *>(S + M);  // [M]
  int *taken = live + M;                      // [M]
  double *kt_s = reinterpret_cast<double *>(taken + M);  // [b][D+1] if it fits (2M ints keep 8-byte alignment)

  const double *kt = kmean + (int64_t)u * M * D;
  int kstride = D;
  for (int j = tid; j < b; j += kSelThreads) {
    live[j] = klive[(int64_t)u * M + j] > 0;
    taken[j] = 0;
  }
  for (int i = tid; i < kSelWarps * M; i += kSelThreads) sp[i] = 0.0;
  if (kt_in_smem) {
    for (int i = tid; i < b * D; i += kSelThreads) kt_s[(i / D) * (D + 1) + (i % D)] = kt[i];
    kt = kt_s;
    kstride = D + 1;
  }
  __syncthreads();

  int ncand = 0;
  for (int j = 0; j < b; ++j) ncand += live[j];  // uniform

  if (ncand > 0 && s.topk > 1) {
    double *zw = zbuf + warp * M, *spw = sp + warp * M, *qw = qrow + warp * D;
    constexpr int QPL = (D + 31) / 32;  // query elements per lane
    double qreg[QPL];                   // the next row, loaded while the current one is scored
    const int nq = qhi - qlo, nrows = nq * s.G;  // rows of the group: head g, query qlo + r % nq
    if (warp < nrows) {
      const T *qp = q + row_offset(s, n, hk * s.G + warp / nq, qlo + warp % nq);
#pragma unroll
      for (int e = 0; e < QPL; ++e)
        if (lane + 32 * e < D) qreg[e] = (double)ld1(qp + lane + 32 * e);
    }
    for (int r = warp; r < nrows; r += kSelWarps) {
#pragma unroll
      for (int e = 0; e < QPL; ++e)
        if (lane + 32 * e < D) qw[lane + 32 * e] = qreg[e];
      __syncwarp();
      if (r + kSelWarps < nrows) {
        const int r2 = r + kSelWarps;
        const T *qp = q + row_offset(s, n, hk * s.G + r2 / nq, qlo + r2 % nq);
#pragma unroll
        for (int e = 0; e < QPL; ++e)
          if (lane + 32 * e < D) qreg[e] = (double)ld1(qp + lane + 32 * e);
      }
      double mx = -INFINITY;
      for (int j = lane; j < b; j += 32) {
        if (!live[j]) continue;
        const double *kj = kt + (int64_t)j * kstride;
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;  // four chains: the FMA latency overlaps
#pragma unroll 4
        for (int c = 0; c < D; c += 4) {
          a0 = fma(qw[c], kj[c], a0);
          a1 = fma(qw[c + 1], kj[c + 1], a1);
          a2 = fma(qw[c + 2], kj[c + 2], a2);
          a3 = fma(qw[c + 3], kj[c + 3], a3);
        }
        const double z = s.scale_d * ((a0 + a1) + (a2 + a3));
        zw[j] = z;
        mx = fmax(mx, z);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      double den = 0.0;
      for (int j = lane; j < b; j += 32)
        if (live[j]) {
          const double e = exp(zw[j] - mx);
          zw[j] = e;
          den += e;
        }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
      for (int j = lane; j < b; j += 32)
        if (live[j]) spw[j] += zw[j] / den;
      __syncwarp();
    }
  }
  __syncthreads();
  for (int j = tid; j < b; j += kSelThreads) {
    double acc = 0.0;
    for (int w = 0; w < kSelWarps; ++w) acc += sp[w * M + j];  // fixed order
    S[j] = acc;
  }
  __syncthreads();

  {
    // Selection by rank: candidate j is kept iff fewer than `want` live candidates beat it (larger
    // score, or equal score and lower index).
    const int want = min(s.topk - 1, ncand);
    for (int j = tid; j < b; j += kSelThreads) {
      int rank = 0;
      if (live[j]) {
        const double sj = S[j];
        for (int i = 0; i < b; ++i)
          if (live[i]) {
            const double si = S[i];
            rank += (si > sj || (si == sj && i < j)) ? 1 : 0;
          }
      }
      taken[j] = live[j] && rank < want;
    }
  }
  __syncthreads();
  if (warp == 0) {
    // emit ascending: ballot over 32-wide chunks of the flags, then the own block
    int pos = 0;
    for (int base = 0; base < b; base += 32) {
      const int j = base + lane;
      const bool f = j < b && taken[j];
      const unsigned m = __ballot_sync(0xffffffffu, f);
      if (f) row[pos + __popc(m & ((1u << lane) - 1u))] = j;
      pos += __popc(m);
    }
    if (lane == 0) row[pos] = b;
    for (int i = pos + 1 + lane; i < s.topk; i += 32) row[i] = -1;
  }
}

// The double-precision scoring of the query blocks on the work list (all of them when
// worklist == nullptr).  grid: any; each CTA takes rows blockIdx.x, blockIdx.x + gridDim.x, ...
template <typename T, int D>
__global__ void __launch_bounds__(kSelThreads) score_select_kernel(
    Shape s, const T *__restrict__ q, const double *__restrict__ kmean,
    const int32_t *__restrict__ klive, const int32_t *__restrict__ seq_lens,
    int32_t *__restrict__ idx, int kt_in_smem, const int32_t *__restrict__ worklist,
    const int32_t *__restrict__ work_count) {
  extern __shared__ double sm[];
  const int total = worklist ? *work_count : s.M * s.B * s.Hkv;
  for (int w = blockIdx.x; w < total; w += gridDim.x) {
    score_select_row<T, D>(s, q, kmean, klive, seq_lens, idx, kt_in_smem, worklist ? worklist[w] : w, sm);
    __syncthreads();  // shared memory is reused by the next row
  }
}

// ---- stage 1: single-precision scoring with an error bound ----------------------------------
// grid M*B*Hkv (unit-major), 256 threads, one query block of one head group per CTA.  Logits z[t][j] of the block's
// (up to 64) queries against 64 candidate means at a time come from a register-blocked fp32
// product out of shared memory (thread = 4 queries x 4 candidates); softmax per query row by 4
// lanes; column sums in fixed order; warp 0 runs the top_k - 1 arg-max passes.
//
// Error bound.  With u = 2^-24: every logit is within E = (D + 4) u scale max|q_t| max|mean_j| of
// its exact value (D roundings of the accumulation, the rounding of the mean to fp32, the scale),
// so every exact probability lies within a factor exp(+-2E) of the exact softmax of the computed
// logits; evaluating that softmax and the column sum in fp32 adds 2^-21 (exp2 approximation and
// division), 2^-22 per unit of logit range, and (b/4 + 80 + 8 chunks) u for the sums.  R is the
// total, relative; two scores a > b are in certain order when a - b > R (a + b).
constexpr int kFastThreads = 256;

// GROUPED: several query heads per key/value head (their number is a run-time value; the
// one-head kernel keeps its loop-free body and its four CTAs per SM; the grouped one needs more registers).
template <typename T, int D, bool GROUPED>
__global__ void __launch_bounds__(kFastThreads, GROUPED ? 2 : 4) score_select_fast_kernel(
    Shape s, const T *__restrict__ q, const float *__restrict__ kmean32,
    const float *__restrict__ knorm, const int32_t *__restrict__ klive,
    const int32_t *__restrict__ seq_lens, int32_t *__restrict__ idx, int32_t *__restrict__ worklist,
    int32_t *__restrict__ work_count) {
  constexpr int P = D + 4;   // row pitch of the operand tiles (floats): conflict-free 128-bit reads
  constexpr int ZP = 68;     // row pitch of the logit tile (4 mod 32: the softmax reads hit 32 banks)
  extern __shared__ float fsm[];
  __shared__ float rn[64];
  __shared__ float csum[kFastThreads];
  __shared__ float bound_s[2];
  __shared__ int kn_bits;
  const int M = s.M;
  float *qs = fsm;                 // [64][P]   the block's queries
  float *ks = qs + 64 * P;         // [64][P]   a chunk of candidate means; reused as zs [64][ZP]
  float *zs = ks;
  float *S = ks + 64 * (P > ZP ? P : ZP);  // [M]
  int *live = reinterpret_cast<int *>(S + M);  // [M]
  int *taken = live + M;                       // [M]

  const int b = blockIdx.x % M, u = blockIdx.x / M, n = u / s.Hkv, hk = u % s.Hkv;  // u: (batch, key/value head)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int qlo = max(b * s.Bk, pad0), qhi = min((b + 1) * s.Bk, s.L);
  int32_t *row = idx + ((int64_t)u * M + b) * s.topk;
  if (qlo >= qhi) {  // the query block holds only padding
    for (int i = tid; i < s.topk; i += kFastThreads) row[i] = -1;
    return;
  }
  if (tid == 0) kn_bits = 0;
  int mine = 0;
  for (int j = tid; j < b; j += kFastThreads) {
    const int lv = klive[(int64_t)u * M + j] > 0;
    live[j] = lv;
    taken[j] = 0;
    mine += lv;
  }
  int ncand = 0;
  for (int base = 0; base < b; base += kFastThreads * 1) {  // one round unless b > 256
    ncand += __syncthreads_count(base + tid < b && live[base + tid]);
  }
  (void)mine;
  const int want = min(s.topk - 1, ncand);
  const bool choose = ncand > want && want > 0;  // a real choice: score the candidates
  bool certain = true;

  // The heads of the group take turns (Eq. 12): each adds its column sums to S.
  const int G = GROUPED ? s.G : 1;
  if (choose)
#pragma unroll 1
  for (int g = 0; g < G; ++g) {
    const int h = hk * G + g;
    // the query block, fp32, invalid rows zero
    for (int i = tid; i < 64 * (D / 4); i += kFastThreads) {
      const int lt = i / (D / 4), c = (i % (D / 4)) * 4, t = b * s.Bk + lt;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lt < s.Bk && t >= qlo && t < qhi) v = ld4(q + row_offset(s, n, h, t) + c);
      *reinterpret_cast<float4 *>(qs + lt * P + c) = v;
    }
    if (g == 0) {
      float km = 0.f;
      for (int j = tid; j < b; j += kFastThreads)
        if (live[j]) km = fmaxf(km, knorm[(int64_t)u * M + j]);
      if (km > 0.f) atomicMax(&kn_bits, __float_as_int(km));  // positive floats order like ints
    }
    __syncthreads();
    if (tid < 64) {
      float a = 0.f;
      for (int c = 0; c < D; ++c) a = fmaf(qs[tid * P + c], qs[tid * P + c], a);
      const float r = sqrtf(a) * 1.0001f;
      rn[tid] = g == 0 ? r : fmaxf(rn[tid], r);  // the bound below takes the largest query of the group
    }
    const int ty = tid >> 4, tx = tid & 15;          // product: queries ty + 16 a, candidates tx + 16 c
    const int rt = tid >> 2, part = tid & 3;          // softmax: row rt, candidates part, part + 4, ...
    const bool row_valid = rt < s.Bk && b * s.Bk + rt >= qlo && b * s.Bk + rt < qhi;
    const int nchunks = (b + 63) / 64;
    const float *kbase = kmean32 + (int64_t)u * M * D;
    float mx = -INFINITY, den = 0.f;  // online softmax statistics of row rt (passes > 1 chunk)

    auto logits_of_chunk = [&](int j0) {  // zs[t][j] = scale <q_t, mean_{j0+j}>
      const int nb = min(64, b - j0);
      __syncthreads();  // previous users of ks / zs are done
      for (int i = tid; i < 64 * (D / 4); i += kFastThreads) {
        const int lj = i / (D / 4), c = (i % (D / 4)) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lj < nb && live[j0 + lj]) v = *reinterpret_cast<const float4 *>(kbase + (int64_t)(j0 + lj) * D + c);
        *reinterpret_cast<float4 *>(ks + lj * P + c) = v;
      }
      __syncthreads();
      float acc[4][4];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c] = 0.f;
      const int ne = (nb + 15) >> 4;  // groups of 16 candidates that hold any (block-uniform)
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
    };
    // probabilities of the chunk in place (zs[t][j] = p_t[j0 + j], 0 where there is none), then
    // their column sums
    auto probabilities_and_sums = [&](int j0) {
      const int nb = min(64, b - j0);
      const float inv = den > 0.f ? 1.f / den : 0.f;
      for (int j = part; j < nb; j += 4) {
        const bool on = row_valid && live[j0 + j];
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
      if (tid < nb) {
        const float a = (csum[tid] + csum[64 + tid]) + (csum[128 + tid] + csum[192 + tid]);
        S[j0 + tid] = g == 0 ? a : S[j0 + tid] + a;  // heads in ascending order
      }
    };
    auto row_statistics = [&](int j0) {  // fold the chunk into (mx, den) of row rt
      const int nb = min(64, b - j0);
      float cm = -INFINITY;
      for (int j = part; j < nb; j += 4)
        if (live[j0 + j]) cm = fmaxf(cm, zs[rt * ZP + j]);
      cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
      cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
      const float nm = fmaxf(mx, cm);
      float e = 0.f;
      if (nm > -INFINITY) {
        for (int j = part; j < nb; j += 4)
          if (live[j0 + j]) e += __expf(zs[rt * ZP + j] - nm);
      }
      e += __shfl_xor_sync(0xffffffffu, e, 1);
      e += __shfl_xor_sync(0xffffffffu, e, 2);
      den = (mx > -INFINITY ? den * __expf(mx - nm) : 0.f) + e;
      mx = nm;
    };

    if (nchunks == 1) {
      logits_of_chunk(0);
      row_statistics(0);
      probabilities_and_sums(0);
    } else {
      for (int ch = 0; ch < nchunks; ++ch) {
        logits_of_chunk(ch * 64);
        row_statistics(ch * 64);
      }
      for (int ch = 0; ch < nchunks; ++ch) {
        logits_of_chunk(ch * 64);
        probabilities_and_sums(ch * 64);
      }
    }
    __syncthreads();
  }

  // Selection by rank: candidate j is kept iff fewer than `want` live candidates beat it
  // (larger score, or equal score and lower index).  4 lanes share a candidate.
  if (choose) {
    for (int j0 = 0; j0 < b; j0 += kFastThreads / 4) {
      const int j = j0 + (tid >> 2), part = tid & 3;
      int rank = 0;
      if (j < b && live[j]) {
        const float sj = S[j];
        for (int i = part; i < b; i += 4)
          if (live[i]) {
            const float si = S[i];
            rank += (si > sj || (si == sj && i < j)) ? 1 : 0;
          }
      }
      rank += __shfl_xor_sync(0xffffffffu, rank, 1);
      rank += __shfl_xor_sync(0xffffffffu, rank, 2);
      if (part == 0 && j < b && live[j]) {
        taken[j] = rank < want;
        if (rank == want - 1) bound_s[0] = S[j];  // the smallest kept score
        if (rank == want) bound_s[1] = S[j];      // the largest dropped score
      }
    }
  } else {
    for (int j = tid; j < b; j += kFastThreads) taken[j] = want > 0 ? live[j] : 0;
  }
  __syncthreads();

  if (warp == 0) {
    if (choose) {
      // Certain iff the gap between the last kept and the first dropped score exceeds what the
      // errors can bridge.
      float qn = fmaxf(rn[lane], rn[lane + 32]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) qn = fmaxf(qn, __shfl_xor_sync(0xffffffffu, qn, o));
      const float kn = __int_as_float(kn_bits);
      const float uu = 5.9604645e-8f;  // 2^-24
      const float bound = s.scale * qn * kn;  // >= every |logit|
      const float E = (float)(D + 4) * uu * bound * 1.01f;
      // a sum of G non-negative head scores, each within R of its exact value, is within R of the
      // exact sum, plus one rounding per addition
      const float R = 2.f * E + 4.77e-7f + 2.f * bound * 2.39e-7f +
                      ((float)b * 0.25f + 80.f + 8.f * (float)((b + 63) / 64) + (float)G) * uu;
      const float smin = bound_s[0], umax = bound_s[1];
      certain = (smin - umax) > R * (smin + umax) * 1.001f;
    }
    if (certain) {
      // emit ascending: ballot over 32-wide chunks of the flags, then the own block
      int pos = 0;
      for (int base = 0; base < b; base += 32) {
        const int j = base + lane;
        const bool f = j < b && taken[j];
        const unsigned m = __ballot_sync(0xffffffffu, f);
        if (f) row[pos + __popc(m & ((1u << lane) - 1u))] = j;
        pos += __popc(m);
      }
      if (lane == 0) row[pos] = b;
      for (int i = pos + 1 + lane; i < s.topk; i += 32) row[i] = -1;
    } else if (lane == 0) {
      worklist[atomicAdd(work_count, 1)] = blockIdx.x;  // re-scored in double precision
    }
  }
}

// ---- stage 1 for short sequences with small blocks ------------------------------------------
// With blocks of 16 or 32 positions a CTA of the kernel above fills a quarter or half of its 64
// query rows, and with few blocks per sequence its run time is all fixed cost (three rounds of
// global loads, a dozen block-wide barriers).  This kernel takes NBLK = 64 / Bk consecutive query
// blocks per CTA: the 64 rows are 64 consecutive positions, every row is scored against the
// candidates of the CTA's last block in one chunk (M <= 64) and keeps those before its own block;
// the column sums of a block are the sums of its 16-row quarters.  Same arithmetic per score and
// the same error bound as above (with the largest query norm of the block and the largest
// candidate norm of the CTA, both upper bounds).
template <typename T, int D, int NBLK>
__global__ void __launch_bounds__(kFastThreads, 4) score_select_fast_packed_kernel(
    Shape s, const T *__restrict__ q, const float *__restrict__ kmean32,
    const float *__restrict__ knorm, const int32_t *__restrict__ klive,
    const int32_t *__restrict__ seq_lens, int32_t *__restrict__ idx, int32_t *__restrict__ worklist,
    int32_t *__restrict__ work_count) {
  constexpr int P = D + 4, ZP = 68, BK = 64 / NBLK, QPB = 4 / NBLK;  // quarters (16 rows) per block
  extern __shared__ float fsm[];
  __shared__ float rn[64];
  __shared__ float csum[kFastThreads];
  __shared__ float S[NBLK][64];
  __shared__ float bound_s[NBLK][2];
  __shared__ int live[64], taken[NBLK][64];
  __shared__ int kn_bits;
  const int M = s.M, MC = (M + NBLK - 1) / NBLK;
  float *qs = fsm;          // [64][P]  the CTA's 64 query positions
  float *ks = qs + 64 * P;  // [64][P]  the candidate means; reused as zs [64][ZP]
  float *zs = ks;

  const int c = blockIdx.x % MC, u = blockIdx.x / MC, n = u / s.H, h = u % s.H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int b0 = c * NBLK;                      // first query block of the CTA
  const int nbk = min(NBLK, M - b0);            // its query blocks
  const int bmax = b0 + nbk - 1;                // candidates of the last one: blocks 0 .. bmax - 1
  if (tid == 0) kn_bits = 0;
  if (tid < 64) live[tid] = (tid < bmax && klive[(int64_t)u * M + tid] > 0) ? 1 : 0;
  __syncthreads();
  // per block: valid, number of live candidates, how many to keep, whether that is a real choice
  int want[NBLK];
  bool valid[NBLK], choose[NBLK], any_choose = false;
#pragma unroll
  for (int i = 0; i < NBLK; ++i) {
    const int b = b0 + i;
    valid[i] = i < nbk && max(b * BK, pad0) < min((b + 1) * BK, s.L);
    int nc = 0;
    for (int j = 0; j < b && i < nbk; ++j) nc += live[j];
    want[i] = min(s.topk - 1, nc);
    choose[i] = valid[i] && nc > want[i] && want[i] > 0;
    any_choose |= choose[i];
  }

  if (any_choose) {
    for (int i = tid; i < 64 * (D / 4); i += kFastThreads) {  // the 64 positions, fp32, invalid rows zero
      const int lt = i / (D / 4), cc = (i % (D / 4)) * 4, t = b0 * BK + lt;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (t >= pad0 && t < s.L) v = ld4(q + row_offset(s, n, h, t) + cc);
      *reinterpret_cast<float4 *>(qs + lt * P + cc) = v;
    }
    for (int i = tid; i < 64 * (D / 4); i += kFastThreads) {  // the candidate means
      const int lj = i / (D / 4), cc = (i % (D / 4)) * 4;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lj < bmax && live[lj])
        v = *reinterpret_cast<const float4 *>(kmean32 + ((int64_t)u * M + lj) * D + cc);
      *reinterpret_cast<float4 *>(ks + lj * P + cc) = v;
    }
    if (tid < bmax && live[tid]) {
      const float km = knorm[(int64_t)u * M + tid];
      if (km > 0.f) atomicMax(&kn_bits, __float_as_int(km));  // positive floats order like ints
    }
    __syncthreads();
    if (tid < 64) {
      float a = 0.f;
      for (int cc = 0; cc < D; ++cc) a = fmaf(qs[tid * P + cc], qs[tid * P + cc], a);
      rn[tid] = sqrtf(a) * 1.0001f;
    }
    const int ty = tid >> 4, tx = tid & 15;  // product: rows ty + 16 a, candidates tx + 16 e
    const int ne = (bmax + 15) >> 4;         // groups of 16 candidates that hold any
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][e] = 0.f;
#pragma unroll 4
    for (int cc = 0; cc < D; cc += 4) {
      float4 qa[4], kb[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        qa[a] = *reinterpret_cast<const float4 *>(qs + (ty + 16 * a) * P + cc);
        if (a < ne) kb[a] = *reinterpret_cast<const float4 *>(ks + (tx + 16 * a) * P + cc);
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
    {  // softmax of row rt over the live candidates before its own block, by 4 lanes, in registers
      const int rt = tid >> 2, part = tid & 3, t = b0 * BK + rt, brow = b0 + rt / BK;
      const bool row_valid = t >= pad0 && t < s.L;
      float z[16], e[16];
      unsigned lm = 0u;
      float cm = -INFINITY;
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const int j = part + 4 * k;
        const bool v = j < brow && live[j];
        lm |= (v ? 1u : 0u) << k;
        z[k] = v ? zs[rt * ZP + j] : -INFINITY;
        cm = fmaxf(cm, z[k]);
      }
      cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
      cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
      float sum = 0.f;
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        e[k] = 0.f;
        if (cm > -INFINITY && ((lm >> k) & 1u)) {
          e[k] = __expf(z[k] - cm);
          sum += e[k];
        }
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      const float inv = sum > 0.f ? 1.f / sum : 0.f;
#pragma unroll
      for (int k = 0; k < 16; ++k)
        zs[rt * ZP + part + 4 * k] = (row_valid && ((lm >> k) & 1u)) ? e[k] * inv : 0.f;
    }
    __syncthreads();
    {  // column sums of every 16-row quarter in a fixed order, then the blocks' sums of quarters
      const int j = tid & 63, quarter = tid >> 6;
      float a = 0.f;
#pragma unroll
      for (int t = 0; t < 16; ++t) a += zs[(quarter * 16 + t) * ZP + j];
      csum[tid] = a;
    }
    __syncthreads();
    for (int e = tid; e < NBLK * 64; e += kFastThreads) {
      const int i = e >> 6, j = e & 63;
      float a = csum[(i * QPB) * 64 + j];
#pragma unroll
      for (int qq = 1; qq < QPB; ++qq) a += csum[(i * QPB + qq) * 64 + j];
      S[i][j] = a;
    }
    __syncthreads();
  }

  // Selection by rank within each block, 4 lanes per (block, candidate)
  for (int e0 = 0; e0 < NBLK * 64; e0 += kFastThreads / 4) {
    const int e = e0 + (tid >> 2), part = tid & 3, i = e >> 6, j = e & 63, b = b0 + i;
    int rank = 0;
    const bool cand = i < nbk && j < b && live[j];
    bool ch = false;
    int wt = 0;
#pragma unroll
    for (int ii = 0; ii < NBLK; ++ii)
      if (ii == i) { ch = choose[ii]; wt = want[ii]; }
    if (cand && ch) {
      const float sj = S[i][j];
      for (int x = part; x < b; x += 4)
        if (live[x]) {
          const float sx = S[i][x];
          rank += (sx > sj || (sx == sj && x < j)) ? 1 : 0;
        }
    }
    rank += __shfl_xor_sync(0xffffffffu, rank, 1);
    rank += __shfl_xor_sync(0xffffffffu, rank, 2);
    if (part == 0 && i < nbk) {
      if (ch) {
        if (cand) {
          taken[i][j] = rank < wt;
          if (rank == wt - 1) bound_s[i][0] = S[i][j];  // the smallest kept score
          if (rank == wt) bound_s[i][1] = S[i][j];      // the largest dropped score
        } else {
          taken[i][j] = 0;
        }
      } else {
        taken[i][j] = (wt > 0 && cand) ? 1 : 0;
      }
    }
  }
  __syncthreads();

  if (warp < nbk) {  // warp i finishes block b0 + i
    const int i = warp, b = b0 + i;
    bool ch = false, vd = false;
#pragma unroll
    for (int ii = 0; ii < NBLK; ++ii)
      if (ii == i) { ch = choose[ii]; vd = valid[ii]; }
    int32_t *row = idx + ((int64_t)u * M + b) * s.topk;
    if (!vd) {  // the query block holds only padding
      for (int x = lane; x < s.topk; x += 32) row[x] = -1;
      return;
    }
    bool certain = true;
    if (ch) {
      float qn = 0.f;
      for (int x = lane; x < BK; x += 32) qn = fmaxf(qn, rn[i * BK + x]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) qn = fmaxf(qn, __shfl_xor_sync(0xffffffffu, qn, o));
      const float kn = __int_as_float(kn_bits);
      const float uu = 5.9604645e-8f;  // 2^-24
      const float bound = s.scale * qn * kn;  // >= every |logit|
      const float E = (float)(D + 4) * uu * bound * 1.01f;
      const float R = 2.f * E + 4.77e-7f + 2.f * bound * 2.39e-7f + ((float)b * 0.25f + 80.f + 8.f + 1.f) * uu;
      const float smin = bound_s[i][0], umax = bound_s[i][1];
      certain = (smin - umax) > R * (smin + umax) * 1.001f;
    }
    if (certain) {
      int pos = 0;
      for (int base = 0; base < b; base += 32) {
        const int j = base + lane;
        const bool f = j < b && taken[i][j];
        const unsigned mm = __ballot_sync(0xffffffffu, f);
        if (f) row[pos + __popc(mm & ((1u << lane) - 1u))] = j;
        pos += __popc(mm);
      }
      if (lane == 0) row[pos] = b;
      for (int x = pos + 1 + lane; x < s.topk; x += 32) row[x] = -1;
    } else if (lane == 0) {
      worklist[atomicAdd(work_count, 1)] = u * M + b;  // re-scored in double precision
    }
  }
}

size_t select_fast_smem_bytes(int M, int D) {
  const int P = D + 4, ZP = 68;
  return (size_t)(64 * P + 64 * (P > ZP ? P : ZP)) * sizeof(float) + (size_t)M * (sizeof(float) + 2 * sizeof(int));
}

size_t select_smem_bytes(int M, int D, bool kt_in_smem) {
  size_t dbl = (size_t)kSelWarps * M * 2 + (size_t)kSelWarps * D + M;
  size_t ints = 2 * (size_t)M;
  size_t kt = kt_in_smem ? (size_t)M * (D + 1) : 0;
  return (dbl + kt) * sizeof(double) + ints * sizeof(int);
}

template <typename T, int D>
int launch_select_t(const Shape &s, const T *q, const T *k, const int32_t *seq_lens, int32_t *idx,
                    const Workspace &ws, cudaStream_t st) {
  // block = (unit, query block), unit-major; a unit is a (batch, key/value head) pair
  const unsigned grid = (unsigned)s.M * (unsigned)(s.B * s.Hkv);
  {
    LaunchScope ls(K_SUMMARY, st);
    summary_kernel<T, D><<<grid, 256, 0, st>>>(s, k, seq_lens, ws.kmean, ws.klive, ws.kmean32, ws.knorm,
                                               ws.sel_count);
  }
  const bool exact_only = exact_select_only();
  if (!exact_only) {
    if (s.G == 1 && s.M <= 64 && (s.Bk == 16 || s.Bk == 32)) {
      // short sequences of small blocks: 64 / Bk query blocks per CTA
      const int nblk = 64 / s.Bk;
      const size_t psm = (size_t)(64 * (D + 4) + 64 * 68) * sizeof(float);
      auto packed = nblk == 2 ? score_select_fast_packed_kernel<T, D, 2> : score_select_fast_packed_kernel<T, D, 4>;
      const unsigned gpk = (unsigned)((s.M + nblk - 1) / nblk) * (unsigned)(s.B * s.Hkv);
      LaunchScope ls(K_SCORE_FAST, st);
      packed<<<gpk, kFastThreads, psm, st>>>(s, q, ws.kmean32, ws.knorm, ws.klive, seq_lens, idx, ws.sel_list,
                                             ws.sel_count);
    } else {
    const size_t fsm = select_fast_smem_bytes(s.M, D);
    auto fast = s.G > 1 ? score_select_fast_kernel<T, D, true> : score_select_fast_kernel<T, D, false>;
    if (fsm > 48 * 1024 &&
        cudaFuncSetAttribute(fast, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fsm) != cudaSuccess)
      return BLOSSOM_ERR_CUDA;
    LaunchScope ls(K_SCORE_FAST, st);
    fast<<<grid, kFastThreads, fsm, st>>>(s, q, ws.kmean32, ws.knorm, ws.klive, seq_lens, idx, ws.sel_list,
                                          ws.sel_count);
    }
  }
  bool in_smem = select_smem_bytes(s.M, D, true) <= 160 * 1024;
  size_t smem = select_smem_bytes(s.M, D, in_smem);
  if (smem > 48 * 1024) {
    if (cudaFuncSetAttribute(score_select_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return BLOSSOM_ERR_CUDA;
  }
  {
    // double precision: every query block (exact_only) or the work list of the kernel above
    LaunchScope ls(K_SCORE_SELECT, st);
    const unsigned g2 = exact_only ? grid : (grid < 592u ? grid : 592u);
    score_select_kernel<T, D><<<g2, kSelThreads, smem, st>>>(s, q, ws.kmean, ws.klive, seq_lens, idx,
                                                            in_smem ? 1 : 0, exact_only ? nullptr : ws.sel_list,
                                                            ws.sel_count);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

int launch_select(const Shape &s, int dtype, const void *q, const void *k, const int32_t *seq_lens,
                  int32_t *idx, const Workspace &ws, cudaStream_t st) {
  if (s.cmp_l > 0) return launch_select_cmp(s, dtype, q, k, seq_lens, idx, ws, st);  // Eq. 8-11
  if (dtype == BLOSSOM_DTYPE_FP32) {
    if (s.D == 32) return launch_select_t<float, 32>(s, (const float *)q, (const float *)k, seq_lens, idx, ws, st);
    return launch_select_t<float, 64>(s, (const float *)q, (const float *)k, seq_lens, idx, ws, st);
  }
  if (s.D == 32)
    return launch_select_t<__nv_bfloat16, 32>(s, (const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, seq_lens, idx, ws, st);
  return launch_select_t<__nv_bfloat16, 64>(s, (const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, seq_lens, idx, ws, st);
}

// ---- selection with built-in scratch (no allocation anywhere on the call path) -------------
// The block means and live counts that blossom_select_blocks keeps in the caller's workspace
// live here in one array that is part of the loaded module.  Every launch overwrites each entry
// it later reads, so nothing has to start at zero and stale contents of earlier calls are
// harmless; two calls in flight at once on one device would overwrite each other's means.
constexpr size_t kStaticMeanElems = 524288;  // doubles: batch * heads * M * head_dim may not exceed this
constexpr size_t kStaticBlocks = 8192;       // int32:   batch * heads * M may not exceed this
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
  if (s.cmp_l > 0) return BLOSSOM_ERR_UNSUPPORTED;  // the built-in scratch has no room for that mode
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
  Workspace ws = {};
  ws.kmean = reinterpret_cast<double *>(base);
  ws.kmean32 = reinterpret_cast<float *>(base + kStaticOffMean32);
  ws.klive = reinterpret_cast<int32_t *>(base + kStaticOffLive);
  ws.knorm = reinterpret_cast<float *>(base + kStaticOffNorm);
  ws.sel_list = reinterpret_cast<int32_t *>(base + kStaticOffList);
  ws.sel_count = reinterpret_cast<int32_t *>(base + kStaticOffCount);
  return launch_select(s, dtype, q, k, seq_lens, idx, ws, st);
}

}  // namespace blossom
