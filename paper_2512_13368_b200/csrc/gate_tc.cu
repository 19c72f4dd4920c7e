// Input-dependent gate (paper Eq. 18 with a one-layer F_o) on the tensor-core attention kernels.
//
// alpha_t = sigmoid(<w_lt, O_lt,t> + <w_st, O_st,t> + b), O_t = alpha_t O_lt,t + (1 - alpha_t) O_st,t.
// The attention kernels themselves know a gate weight per row only through the per-row records of
// the backward pre-pass; everything else the gate needs is row-local or can be put into the
// tensors those kernels read:
//   forward   the attention kernel produces O_lt, O_st (and the log-sum-exps) as in training mode;
//             a row-wise kernel here forms alpha_t from them and writes O.
//   backward  with c_t = alpha_t (1 - alpha_t) <G_t, O_lt,t - O_st,t> the upstream gradients of the
//             two branches are alpha_t (G_t + kL_t w_lt) and (1 - alpha_t) (G_t + kS_t w_st) with
//             kL_t = c_t / alpha_t, kS_t = c_t / (1 - alpha_t).  They differ by more than a factor,
//             so the backward kernels run once per branch: pass 1 with the tensor G + kL w_lt in
//             place of dO, tile lists of the long-term branch only and records that carry alpha_t
//             in the exponent and switch the short-term branch off; pass 2 likewise for the
//             short-term branch into scratch tensors; a third kernel adds the two results.  The
//             gradient of F_o's parameters is row-local (dw_lt = sum_t c_t O_lt,t, dw_st likewise,
//             db = sum_t c_t) and is accumulated here in double precision, per query block, for the
//             fixed-order reduction of gate_param_grad_kernel.
// The branch outputs entering F_o are the stored (bf16) rows.
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

typedef __nv_bfloat16 bf;

__device__ __forceinline__ void unpack8(const uint4 &v, float (&x)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    x[2 * e] = __uint_as_float(w[e] << 16);
    x[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint4 pack8(const float (&x)[8]) {
  return make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
}
// sum over the LPR lanes that share a row (LPR a power of two, rows aligned in the warp)
template <int LPR>
__device__ __forceinline__ float row_sum(float a) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  return a;
}
// F_o's parameters of head h are 2 D + 1 floats: an odd count, so rows of it are not 16-byte aligned
__device__ __forceinline__ void load_w8(const float *p, float (&w)[8]) {
#pragma unroll
  for (int e = 0; e < 8; ++e) w[e] = p[e];
}
__device__ __forceinline__ void gate_of_row(float a, float &alpha, float &beta) {
  // both from the same exponential, so that alpha + beta = 1 to rounding and neither underflows first
  const float e = __expf(-fabsf(a));
  const float big = 1.f / (1.f + e), small = e / (1.f + e);
  alpha = a >= 0.f ? big : small;
  beta = a >= 0.f ? small : big;
}

// ---- forward: O = alpha_t O_lt + (1 - alpha_t) O_st -------------------------------------------
// D / 8 lanes per row, one 16-byte chunk each.  Padded rows hold zeros in both branches.
template <int D>
__global__ void __launch_bounds__(256) gate_mix_kernel(Shape s, const float *__restrict__ gate,
                                                       const bf *__restrict__ out_lt, const bf *__restrict__ out_st,
                                                       bf *__restrict__ out) {
  constexpr int LPR = D / 8, RPB = 256 / LPR;
  const int blocks_per_unit = (s.L + RPB - 1) / RPB;
  const int u = blockIdx.x / blocks_per_unit, n = u / s.H, h = u % s.H;
  const int t = (blockIdx.x % blocks_per_unit) * RPB + threadIdx.x / LPR, ch = threadIdx.x % LPR;
  const float *gw = gate + (int64_t)h * (2 * D + 1);
  float wl[8], wsv[8], ol[8] = {0, 0, 0, 0, 0, 0, 0, 0}, os[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  load_w8(gw + ch * 8, wl);
  load_w8(gw + D + ch * 8, wsv);
  const bool row = t < s.L;
  const int64_t off = row ? row_offset(s, n, h, t) + ch * 8 : 0;
  if (row) {
    unpack8(*reinterpret_cast<const uint4 *>(out_lt + off), ol);
    unpack8(*reinterpret_cast<const uint4 *>(out_st + off), os);
  }
  float a = 0.f;
#pragma unroll
  for (int e = 0; e < 8; ++e) a = fmaf(wl[e], ol[e], fmaf(wsv[e], os[e], a));
  a = row_sum<LPR>(a) + gw[2 * D];
  float alpha, beta;
  gate_of_row(a, alpha, beta);
  if (row) {
    float o[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) o[e] = alpha * ol[e] + beta * os[e];
    *reinterpret_cast<uint4 *>(out + off) = pack8(o);
  }
}

// ---- backward pre-pass --------------------------------------------------------------------------
// One CTA per (batch, head, query block).  Per row: alpha_t, c_t, the two upstream tensors (bf16,
// zeros in padded rows: the attention kernels multiply them by exact zeros, which must stay
// zeros), the records of the two passes (layout of bwd_prep_kernel; Delta of a pass is taken with
// the rounded tensor the pass multiplies with, and the branch a pass leaves out gets the exponent
// offset -1e30, i.e. probability 0), and the partial sums of the parameter gradient.
template <int D>
__global__ void __launch_bounds__(256) gate_prep_kernel(Shape s, const float *__restrict__ gate,
                                                        const int32_t *__restrict__ seq_lens,
                                                        const bf *__restrict__ out_lt, const bf *__restrict__ out_st,
                                                        const float *__restrict__ lse, const bf *__restrict__ dout,
                                                        bf *__restrict__ g_lt, bf *__restrict__ g_st,
                                                        float4 *__restrict__ rec_lt, float4 *__restrict__ rec_st,
                                                        double *__restrict__ dgate_part, int Lpad) {
  constexpr int LPR = D / 8, RPB = 256 / LPR, GW = 2 * D + 1;
  __shared__ double red[RPB][GW];
  const int u = blockIdx.x / s.M, qb = blockIdx.x % s.M, n = u / s.H, h = u % s.H;
  const int lr = threadIdx.x / LPR, ch = threadIdx.x % LPR;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const float *gw = gate + (int64_t)h * GW;
  float wl[8], wsv[8];
  load_w8(gw + ch * 8, wl);
  load_w8(gw + D + ch * 8, wsv);
  const float bias = gw[2 * D];
  const int64_t BHL = (int64_t)s.B * s.H * s.L;
  double accL[8], accS[8], accB = 0.0;
#pragma unroll
  for (int e = 0; e < 8; ++e) accL[e] = accS[e] = 0.0;
  // the last query block also writes the (zero) records of the rows that pad L to a multiple of 64
  const int t_end = qb == s.M - 1 ? Lpad : min((qb + 1) * s.Bk, s.L);
  for (int t0 = qb * s.Bk; t0 < t_end; t0 += RPB) {
    const int t = t0 + lr;
    const bool in_rec = t < t_end, row = in_rec && t < s.L, valid = row && t >= pad0;
    const int64_t off = row ? row_offset(s, n, h, t) + ch * 8 : 0;
    float g[8], ol[8], os[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) g[e] = ol[e] = os[e] = 0.f;
    if (valid) {
      unpack8(*reinterpret_cast<const uint4 *>(dout + off), g);
      unpack8(*reinterpret_cast<const uint4 *>(out_lt + off), ol);
      unpack8(*reinterpret_cast<const uint4 *>(out_st + off), os);
    }
    float aL = 0.f, aS = 0.f, woL = 0.f, woS = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      aL = fmaf(g[e], ol[e], aL);
      aS = fmaf(g[e], os[e], aS);
      woL = fmaf(wl[e], ol[e], woL);
      woS = fmaf(wsv[e], os[e], woS);
    }
    aL = row_sum<LPR>(aL);
    aS = row_sum<LPR>(aS);
    woL = row_sum<LPR>(woL);
    woS = row_sum<LPR>(woS);
    float alpha, beta;
    gate_of_row(woL + woS + bias, alpha, beta);
    const float diff = aL - aS, c = alpha * beta * diff, kL = beta * diff, kS = alpha * diff;
    float gl[8], gs[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      gl[e] = valid ? fmaf(kL, wl[e], g[e]) : 0.f;
      gs[e] = valid ? fmaf(kS, wsv[e], g[e]) : 0.f;
    }
    const uint4 pl = pack8(gl), ps = pack8(gs);
    if (row) {
      *reinterpret_cast<uint4 *>(g_lt + off) = pl;
      *reinterpret_cast<uint4 *>(g_st + off) = ps;
    }
    unpack8(pl, gl);  // as the attention kernels will read them
    unpack8(ps, gs);
    float dL = 0.f, dS = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      dL = fmaf(gl[e], ol[e], dL);
      dS = fmaf(gs[e], os[e], dS);
    }
    dL = row_sum<LPR>(dL);
    dS = row_sum<LPR>(dS);
    if (ch == 0 && in_rec) {
      float l0 = 0.f, l2 = 0.f, l4 = 0.f, s0 = 0.f, s4 = 0.f, s6 = 0.f;
      if (valid) {
        l0 = -(lse[(int64_t)u * s.L + t] * kLog2e - log2f(fmaxf(alpha, 1e-37f)));
        l2 = -dL;
        l4 = -1e30f;
        s0 = -1e30f;
        s4 = -(lse[BHL + (int64_t)u * s.L + t] * kLog2e - log2f(fmaxf(beta, 1e-37f)));
        s6 = -dS;
      }
      const int64_t ro = ((int64_t)u * Lpad + (t & ~1)) * 4 + (t & 1);
      float *rl = reinterpret_cast<float *>(rec_lt) + ro, *rs = reinterpret_cast<float *>(rec_st) + ro;
      rl[0] = l0; rl[2] = l2; rl[4] = l4; rl[6] = 0.f;
      rs[0] = s0; rs[2] = 0.f; rs[4] = s4; rs[6] = s6;
    }
    if (valid) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        accL[e] += (double)c * (double)ol[e];
        accS[e] += (double)c * (double)os[e];
      }
      if (ch == 0) accB += (double)c;
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    red[lr][ch * 8 + e] = accL[e];
    red[lr][D + ch * 8 + e] = accS[e];
  }
  if (ch == 0) red[lr][2 * D] = accB;
  __syncthreads();
  for (int d = threadIdx.x; d < GW; d += 256) {
    double a = 0.0;
    for (int r = 0; r < RPB; ++r) a += red[r][d];  // fixed order
    dgate_part[((int64_t)u * s.M + qb) * GW + d] = a;
  }
}

// ---- dst += src over a q-shaped (or k-shaped) bf16 tensor, one rounding --------------------------
__global__ void __launch_bounds__(256) grad_add_kernel(int B, int heads, int L, int D, int64_t sb, int64_t sh,
                                                       int64_t sl, bf *__restrict__ dst, const bf *__restrict__ src) {
  const int cpr = D / 8;
  const int64_t total = (int64_t)B * heads * L * cpr;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int ch = (int)(e % cpr);
    const int64_t row = e / cpr;
    const int t = (int)(row % L), h = (int)((row / L) % heads), n = (int)(row / ((int64_t)L * heads));
    const int64_t off = (int64_t)n * sb + (int64_t)h * sh + (int64_t)t * sl + ch * 8;
    float a[8], b[8];
    unpack8(*reinterpret_cast<const uint4 *>(dst + off), a);
    unpack8(*reinterpret_cast<const uint4 *>(src + off), b);
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] += b[i];
    *reinterpret_cast<uint4 *>(dst + off) = pack8(a);
  }
}

int add_into(const Shape &s, bool kv, void *dst, const void *src, cudaStream_t st) {
  const int heads = kv ? s.Hkv : s.H;
  const int64_t total = (int64_t)s.B * heads * s.L * (s.D / 8);
  const unsigned grid = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
  LaunchScope ls(K_GATE_GRAD, st);
  grad_add_kernel<<<grid, 256, 0, st>>>(s.B, heads, s.L, s.D, kv ? s.ksb : s.sb, kv ? s.ksh : s.sh,
                                        kv ? s.ksl : s.sl, (bf *)dst, (const bf *)src);
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

int launch_fwd_tc_gate(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                       const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt, void *out_st,
                       float *lse, const Workspace &ws, cudaStream_t st) {
  void *olt = out_lt ? out_lt : ws.gate_olt, *ost = out_st ? out_st : ws.gate_ost;
  // (the attention kernel also writes `out`, mixed with a per-head weight it reads from the first
  // floats of F_o's parameters: finite numbers, overwritten below)
  if (int rc = launch_fwd_tc(s, q, k, v, gate, seq_lens, idx, out, olt, ost, lse, ws, st)) return rc;
  const int rpb = 256 / (s.D / 8);
  const unsigned grid = (unsigned)(s.B * s.H) * (unsigned)((s.L + rpb - 1) / rpb);
  LaunchScope ls(K_GATE_GRAD, st);
  if (s.D == 32) gate_mix_kernel<32><<<grid, 256, 0, st>>>(s, gate, (const bf *)olt, (const bf *)ost, (bf *)out);
  else gate_mix_kernel<64><<<grid, 256, 0, st>>>(s, gate, (const bf *)olt, (const bf *)ost, (bf *)out);
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

int launch_bwd_tc_gate(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                       const int32_t *seq_lens, const int32_t *idx, const void *out_lt, const void *out_st,
                       const float *lse, const void *dout, void *dq, void *dk, void *dv, float *dgate,
                       const Workspace &ws, cudaStream_t st) {
  const int Lpad = (s.L + 63) / 64 * 64;
  {
    LaunchScope ls(K_BWD_PREP, st);
    const unsigned grid = (unsigned)(s.B * s.H) * (unsigned)s.M;
    if (s.D == 32)
      gate_prep_kernel<32><<<grid, 256, 0, st>>>(s, gate, seq_lens, (const bf *)out_lt, (const bf *)out_st, lse,
                                                 (const bf *)dout, (bf *)ws.gate_glt, (bf *)ws.gate_gst, ws.qstats,
                                                 ws.qstats2, ws.dgate_part, Lpad);
    else
      gate_prep_kernel<64><<<grid, 256, 0, st>>>(s, gate, seq_lens, (const bf *)out_lt, (const bf *)out_st, lse,
                                                 (const bf *)dout, (bf *)ws.gate_glt, (bf *)ws.gate_gst, ws.qstats,
                                                 ws.qstats2, ws.dgate_part, Lpad);
    if (cudaGetLastError() != cudaSuccess) return BLOSSOM_ERR_CUDA;
  }
  int rc = launch_bwd_tc(s, q, k, v, gate, seq_lens, idx, out_lt, out_st, lse, ws.gate_glt, dq, dk, dv, ws, st, 1,
                         ws.qstats);
  if (rc) return rc;
  rc = launch_bwd_tc(s, q, k, v, gate, seq_lens, idx, out_lt, out_st, lse, ws.gate_gst, ws.gate_dq, ws.gate_dk,
                     ws.gate_dv, ws, st, 2, ws.qstats2);
  if (rc) return rc;
  if ((rc = add_into(s, false, dq, ws.gate_dq, st))) return rc;
  if ((rc = add_into(s, true, dk, ws.gate_dk, st))) return rc;
  if ((rc = add_into(s, true, dv, ws.gate_dv, st))) return rc;
  return launch_gate_param_grad(s, ws, dgate, st);
}

}  // namespace tc
}  // namespace blossom
