// Block summary, importance scoring and top-k selection (paper Eq. 8-10, 12, 13 with
// compression size = stride = selection size = Bk and the summary = mean of a block's valid keys).
//
// Scores are evaluated in double precision: the selection is a discrete decision taken from
// floating-point sums whose neighbours differ by ~1e-3 relative on Gaussian inputs, and the
// library promises the fp64 choice (ties below ~1e-12 relative excepted).
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
                                                      int32_t *__restrict__ klive) {
  constexpr int CH = D / 4;        // chunks per row
  constexpr int RG = 256 / CH;     // row groups
  __shared__ double part[RG][D];
  const int j = blockIdx.x % s.M, u = blockIdx.x / s.M, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int lo = max(j * s.Bk, pad0), hi = min((j + 1) * s.Bk, s.L);
  const int ch = threadIdx.x % CH, rg = threadIdx.x / CH;
  double a0 = 0, a1 = 0, a2 = 0, a3 = 0;
  for (int p = lo + rg; p < hi; p += RG) {
    float4 x = ld4(k + row_offset(s, n, h, p) + ch * 4);
    a0 += (double)x.x; a1 += (double)x.y; a2 += (double)x.z; a3 += (double)x.w;
  }
  part[rg][ch * 4 + 0] = a0; part[rg][ch * 4 + 1] = a1;
  part[rg][ch * 4 + 2] = a2; part[rg][ch * 4 + 3] = a3;
  __syncthreads();
  const int cnt = max(hi - lo, 0);
  if (threadIdx.x < D) {
    double acc = 0;
    for (int r = 0; r < RG; ++r) acc += part[r][threadIdx.x];  // fixed order
    kmean[((int64_t)u * s.M + j) * D + threadIdx.x] = cnt > 0 ? acc / (double)cnt : 0.0;
  }
  if (threadIdx.x == 0) klive[(int64_t)u * s.M + j] = cnt;
}

// ---- Eq. 10 + 12 + 13: scores of one query block and its top-k --------------------------
// grid M*B*H (unit-major), 256 threads.  One warp per query row: lanes stride over the candidate blocks,
// softmax over the candidates, per-warp partial sums, fixed-order combine, then warp 0 runs
// top_k - 1 arg-max passes (value desc, index asc).
template <typename T, int D>
__global__ void __launch_bounds__(kSelThreads) score_select_kernel(
    Shape s, const T *__restrict__ q, const double *__restrict__ kmean,
    const int32_t *__restrict__ klive, const int32_t *__restrict__ seq_lens,
    int32_t *__restrict__ idx, int kt_in_smem) {
  extern __shared__ double sm[];
  const int b = blockIdx.x % s.M, u = blockIdx.x / s.M, n = u / s.H, h = u % s.H;
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
    for (int t = qlo + warp; t < qhi; t += kSelWarps) {
      const T *qp = q + row_offset(s, n, h, t);
      for (int c = lane; c < D; c += 32) qw[c] = (double)ld1(qp + c);
      __syncwarp();
      double mx = -INFINITY;
      for (int j = lane; j < b; j += 32) {
        if (!live[j]) continue;
        const double *kj = kt + (int64_t)j * kstride;
        double acc = 0.0;
#pragma unroll 8
        for (int c = 0; c < D; ++c) acc += qw[c] * kj[c];
        const double z = s.scale_d * acc;
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

  if (warp == 0) {
    const int want = min(s.topk - 1, ncand);
    for (int r = 0; r < want; ++r) {
      double bv = -INFINITY;
      int bj = 0x7fffffff;
      for (int j = lane; j < b; j += 32) {
        if (!live[j] || taken[j]) continue;
        const double vj = S[j];
        if (bj == 0x7fffffff || vj > bv) { bv = vj; bj = j; }  // ascending j: strict > keeps lower
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
        if (oj != 0x7fffffff && (bj == 0x7fffffff || ov > bv || (ov == bv && oj < bj))) {
          bv = ov;
          bj = oj;
        }
      }
      if (lane == 0) taken[bj] = 1;
      __syncwarp();
    }
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

size_t select_smem_bytes(int M, int D, bool kt_in_smem) {
  size_t dbl = (size_t)kSelWarps * M * 2 + (size_t)kSelWarps * D + M;
  size_t ints = 2 * (size_t)M;
  size_t kt = kt_in_smem ? (size_t)M * (D + 1) : 0;
  return (dbl + kt) * sizeof(double) + ints * sizeof(int);
}

template <typename T, int D>
int launch_select_t(const Shape &s, const T *q, const T *k, const int32_t *seq_lens, int32_t *idx,
                    const Workspace &ws, cudaStream_t st) {
  const unsigned grid = (unsigned)s.M * (unsigned)(s.B * s.H);  // block = (unit, query block), unit-major
  {
    LaunchScope ls(K_SUMMARY, st);
    summary_kernel<T, D><<<grid, 256, 0, st>>>(s, k, seq_lens, ws.kmean, ws.klive);
  }
  bool in_smem = select_smem_bytes(s.M, D, true) <= 160 * 1024;
  size_t smem = select_smem_bytes(s.M, D, in_smem);
  if (smem > 48 * 1024) {
    if (cudaFuncSetAttribute(score_select_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return BLOSSOM_ERR_CUDA;
  }
  {
    LaunchScope ls(K_SCORE_SELECT, st);
    score_select_kernel<T, D><<<grid, kSelThreads, smem, st>>>(s, q, ws.kmean, ws.klive, seq_lens,
                                                               idx, in_smem ? 1 : 0);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

int launch_select(const Shape &s, int dtype, const void *q, const void *k, const int32_t *seq_lens,
                  int32_t *idx, const Workspace &ws, cudaStream_t st) {
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
constexpr size_t kStaticBytes = kStaticMeanElems * sizeof(double) + kStaticBlocks * sizeof(int32_t);
static __device__ __align__(256) unsigned char g_select_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
static void *g_scratch_addr[kMaxDevices] = {nullptr};  // device address of the array, per device

size_t select_static_capacity_bytes() { return kStaticBytes; }

int launch_select_static(const Shape &s, int dtype, const void *q, const void *k,
                         const int32_t *seq_lens, int32_t *idx, cudaStream_t st) {
  const size_t blocks = (size_t)s.B * s.H * s.M;
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
  ws.klive = reinterpret_cast<int32_t *>(base + kStaticMeanElems * sizeof(double));
  return launch_select(s, dtype, q, k, seq_lens, idx, ws, st);
}

}  // namespace blossom
