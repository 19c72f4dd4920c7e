// Block selection with overlapping compression blocks (paper Eq. 8-11 and 13).
//
// Compression blocks K_i = positions [s i, s i + l), i < Mc = floor((L - l) / s) + 1, are
// summarised by the mean of their valid keys (Eq. 9 with the summary = mean).  A query block
// (selection blocks of Bk positions) scores the live compression blocks that end before it starts
// (Eq. 10 per query, summed over the block's valid queries), Eq. 11 maps those scores onto the past
// selection blocks, S[j] = sum_{m < Bk/s} sum_{n < l/s} Sc[(Bk/s) j - m - n] (terms out of range or
// not scored are zero), and the own block plus the top_k - 1 best past blocks are kept, ties to
// the lower index (Eq. 13).  Everything is evaluated in double precision: the choice is discrete.
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
                                                          int32_t *__restrict__ clive) {
  constexpr int CH = D / 4, RG = 256 / CH;
  __shared__ double part[RG][D];
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
    cmean[((int64_t)u * s.Mc + i) * D + threadIdx.x] = cnt > 0 ? acc / (double)cnt : 0.0;
  }
  if (threadIdx.x == 0) clive[(int64_t)u * s.Mc + i] = cnt;
}

// grid M * B * H (unit-major), 256 threads: one query block.  One warp per query row, lanes over
// the candidate compression blocks; per-warp partial sums, fixed-order combine, Eq. 11, rank
// selection.  Shared memory (doubles): zbuf[8][Mc], sp[8][Mc], qrow[8][D], Sc[Mc], S[M];
// ints: livec[Mc], taken[M].
template <typename T, int D>
__global__ void __launch_bounds__(kCmpThreads) cmp_score_select_kernel(
    Shape s, const T *__restrict__ q, const double *__restrict__ cmean,
    const int32_t *__restrict__ clive, const int32_t *__restrict__ seq_lens,
    int32_t *__restrict__ idx, int means_in_smem) {
  extern __shared__ double smd[];
  const int M = s.M, Mc = max(s.Mc, 1);
  double *zbuf = smd, *sp = zbuf + kCmpWarps * Mc, *qrow = sp + kCmpWarps * Mc;
  double *Sc = qrow + kCmpWarps * D, *S = Sc + Mc;
  int *livec = reinterpret_cast<int *>(S + M), *taken = livec + Mc;
  // the candidates' means, row pitch D + 1 doubles (conflict-free when lanes read different rows)
  double *kt_s = reinterpret_cast<double *>(taken + M + ((Mc + M) & 1));
  const int b = blockIdx.x % M, u = blockIdx.x / M, n = u / s.H, h = u % s.H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int qlo = max(b * s.Bk, pad0), qhi = min((b + 1) * s.Bk, s.L);
  int32_t *row = idx + ((int64_t)u * M + b) * s.topk;
  if (qlo >= qhi) {  // the query block holds only padding
    for (int i = tid; i < s.topk; i += kCmpThreads) row[i] = -1;
    return;
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
  const unsigned units = (unsigned)(s.B * s.H);
  if (s.Mc > 0) {
    LaunchScope ls(K_SUMMARY, st);
    cmp_summary_kernel<T, D><<<(unsigned)s.Mc * units, 256, 0, st>>>(s, k, seq_lens, ws.cmean, ws.clive);
  }
  const bool in_smem = cmp_smem_bytes(s, D, true) <= 160 * 1024;
  const size_t smem = cmp_smem_bytes(s, D, in_smem);
  if (smem > 200 * 1024) return BLOSSOM_ERR_UNSUPPORTED;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(cmp_score_select_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    LaunchScope ls(K_SCORE_SELECT, st);
    cmp_score_select_kernel<T, D><<<(unsigned)s.M * units, kCmpThreads, smem, st>>>(s, q, ws.cmean, ws.clive,
                                                                                   seq_lens, idx, in_smem ? 1 : 0);
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
