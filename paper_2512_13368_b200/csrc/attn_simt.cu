// fp32 CUDA-core path of the fused two-branch attention (forward + backward).
//
// It serves fp32 inputs (whose 1e-4 tolerance rules out reduced-precision tensor-core products)
// and every shape the tensor-core path does not take.  One CTA per (unit, query block) for the
// forward and dQ kernels, one CTA per (unit, key block) for dK/dV; a query (or key) row is owned
// by 4 adjacent lanes, each holding D/4 columns as interleaved float4 chunks, so dot products
// finish with two shuffles and shared-memory reads are conflict-free 128-bit loads.
//
// Paper: selected-block attention Eq. 14 + 16, window attention Eq. 15 (first case, causal) + 17,
// both instances of the masked softmax attention of Eq. 1; gate combine Eq. 19.
#include "common.cuh"

namespace blossom {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float group_sum(float x, unsigned gmask) {
  x += __shfl_xor_sync(gmask, x, 1);
  x += __shfl_xor_sync(gmask, x, 2);
  return x;
}
__device__ __forceinline__ float dot4(const float4 a, const float4 b, float acc) {
  acc = fmaf(a.x, b.x, acc);
  acc = fmaf(a.y, b.y, acc);
  acc = fmaf(a.z, b.z, acc);
  return fmaf(a.w, b.w, acc);
}
__device__ __forceinline__ void axpy4(float4 &y, float a, const float4 x) {
  y.x = fmaf(a, x.x, y.x); y.y = fmaf(a, x.y, y.y); y.z = fmaf(a, x.z, y.z); y.w = fmaf(a, x.w, y.w);
}
__device__ __forceinline__ void scale_axpy4(float4 &y, float c, float a, const float4 x) {
  y.x = fmaf(a, x.x, y.x * c); y.y = fmaf(a, x.y, y.y * c);
  y.z = fmaf(a, x.z, y.z * c); y.w = fmaf(a, x.w, y.w * c);
}
// four consecutive floats from an address that is only 4-byte aligned (the rows of F_o's
// parameters are 2 D + 1 floats long)
__device__ __forceinline__ float4 ldw4(const float *p) { return make_float4(p[0], p[1], p[2], p[3]); }
__device__ __forceinline__ float4 zero4() { return make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + __expf(-x)); }

// Stage rows [row0, row0 + Bk) of a q-shaped tensor into shared memory as fp32 (zero past L).
// `head0` = element offset of row 0 of the (batch, head) the tile belongs to, `sl` = row stride.
template <typename T, int D>
__device__ __forceinline__ void stage_tile(const Shape &s, const T *base, int64_t head0, int64_t sl,
                                           int row0, float *dst) {
  constexpr int CH = D / 4;
  for (int i = threadIdx.x; i < s.Bk * CH; i += blockDim.x) {
    const int pr = i / CH, ch = i % CH, p = row0 + pr;
    float4 x = zero4();
    if (p < s.L) x = ld4(base + head0 + (int64_t)p * sl + ch * 4);
    reinterpret_cast<float4 *>(dst)[i] = x;
  }
}

// flags[blk], blk <= qb: bit 0 = blk is one of the query block's selected blocks,
// bit 1 = the short-term branch of some query of the block may reach into blk.
__device__ __forceinline__ void build_visit_flags(const Shape &s, const int32_t *idxrow, int qb,
                                                  int *flags) {
  const int t0 = qb * s.Bk, t1 = min(s.L, t0 + s.Bk) - 1;
  const int last = s.causal ? qb : s.M - 1;  // without the causal mask later blocks are visited too
  for (int blk = threadIdx.x; blk <= last; blk += blockDim.x) {
    int f = st_ranges_touch(s, t0, t1, blk * s.Bk, min(s.L, blk * s.Bk + s.Bk) - 1) ? 2 : 0;
    for (int i = 0; i < s.topk; ++i) f |= (idxrow[i] == blk) ? 1 : 0;
    flags[blk] = f;
  }
}

// Selection per query position (block_idx [B][Hkv][L][top_k]): every row of the query block has a
// list of its own.  rowsel[r][w] = bit set of the blocks row r selected; flags[blk] bit 0 = some
// row selected blk, bit 1 as above.  `active` rows only (thread (r, sub) takes every fourth entry).
__device__ __forceinline__ void build_row_selections(const Shape &s, const int32_t *idxrow, int qb, int r,
                                                     int sub, bool active, int *flags, uint32_t *rowsel) {
  const int MW = (s.M + 31) >> 5;
  const int t0 = qb * s.Bk, t1 = min(s.L, t0 + s.Bk) - 1;
  for (int blk = threadIdx.x; blk <= qb; blk += blockDim.x)
    flags[blk] = st_ranges_touch(s, t0, t1, blk * s.Bk, min(s.L, blk * s.Bk + s.Bk) - 1) ? 2 : 0;
  for (int i = threadIdx.x; i < s.Bk * MW; i += blockDim.x) rowsel[i] = 0u;
  __syncthreads();
  if (active)
    for (int i = sub; i < s.topk; i += 4) {
      const int j = idxrow[i];
      if (j >= 0 && j <= qb) {
        atomicOr(&rowsel[r * MW + (j >> 5)], 1u << (j & 31));
        atomicOr(&flags[j], 1);
      }
    }
}

// ------------------------------------------------------------------------------- forward
template <typename T, int D>
__global__ void __launch_bounds__(256) fwd_simt_kernel(
    Shape s, const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, T *__restrict__ out, T *__restrict__ out_lt,
    T *__restrict__ out_st, float *__restrict__ lse) {
  constexpr int NV = D / 16, CH = D / 4;
  extern __shared__ float smf[];
  float *Ks = smf, *Vs = Ks + s.Bk * D;
  int *flags = reinterpret_cast<int *>(Vs + s.Bk * D);
  const int qb = blockIdx.x % s.M, u = blockIdx.x / s.M, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int tid = threadIdx.x, r = tid >> 2, sub = tid & 3;
  const unsigned gmask = 0xFu << ((tid & 31) & ~3);
  const int t = qb * s.Bk + r;
  const bool inrange = t < s.L, active = inrange && t >= pad0;

  const int hk = h / s.G;  // key/value head of this query head; its group shares one selection
  uint32_t *rowsel = reinterpret_cast<uint32_t *>(flags + s.M);  // [Bk][ceil(M / 32)], per-position selection only
  const int MW = (s.M + 31) >> 5;
  if (s.pq)
    build_row_selections(s, idx + (((int64_t)n * s.Hkv + hk) * s.L + (inrange ? t : 0)) * s.topk, qb, r, sub, active,
                         flags, rowsel);
  else
    build_visit_flags(s, idx + (((int64_t)n * s.Hkv + hk) * s.M + qb) * s.topk, qb, flags);

  float4 qv[NV], aL[NV], aS[NV];
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    qv[c] = active ? ld4(q + row_offset(s, n, h, t) + (c * 4 + sub) * 4) : zero4();
    aL[c] = zero4();
    aS[c] = zero4();
  }
  float mL = -INFINITY, lL = 0.f, mS = -INFINITY, lS = 0.f;
  const float sc2 = s.scale * kLog2e;
  const bool block_live = min((qb + 1) * s.Bk, s.L) > pad0;
  __syncthreads();

  if (block_live) {
    for (int blk = 0; blk <= (s.causal ? qb : s.M - 1); ++blk) {
      const int f = flags[blk];
      if (!f) continue;
      __syncthreads();
      stage_tile<T, D>(s, k, row_offset_kv(s, n, hk, 0), s.ksl, blk * s.Bk, Ks);
      stage_tile<T, D>(s, v, row_offset_kv(s, n, hk, 0), s.ksl, blk * s.Bk, Vs);
      __syncthreads();
      if (!active) continue;
      const int p0 = blk * s.Bk;
      const int pbeg = max(0, pad0 - p0), pend = min(min(s.Bk, s.L - p0), s.causal ? t - p0 + 1 : s.Bk);
      const bool selb = s.pq ? (rowsel[r * MW + (blk >> 5)] >> (blk & 31)) & 1u : f & 1;
      for (int pi = pbeg; pi < pend; ++pi) {
        const bool inS = st_visible(s, t, p0 + pi);
        if (!selb && !inS) continue;
        const float4 *kr = reinterpret_cast<const float4 *>(Ks) + pi * CH;
        const float4 *vr = reinterpret_cast<const float4 *>(Vs) + pi * CH;
        float part = 0.f;
#pragma unroll
        for (int c = 0; c < NV; ++c) part = dot4(qv[c], kr[c * 4 + sub], part);
        const float sv = group_sum(part, gmask) * sc2;
        if (selb) {
          const float mn = fmaxf(mL, sv), corr = exp2f(mL - mn), pe = exp2f(sv - mn);
          lL = fmaf(lL, corr, pe);
#pragma unroll
          for (int c = 0; c < NV; ++c) scale_axpy4(aL[c], corr, pe, vr[c * 4 + sub]);
          mL = mn;
        }
        if (inS) {
          const float mn = fmaxf(mS, sv), corr = exp2f(mS - mn), pe = exp2f(sv - mn);
          lS = fmaf(lS, corr, pe);
#pragma unroll
          for (int c = 0; c < NV; ++c) scale_axpy4(aS[c], corr, pe, vr[c * 4 + sub]);
          mS = mn;
        }
      }
    }
  }

  if (!inrange) return;
  const float iL = lL > 0.f ? 1.f / lL : 0.f, iS = lS > 0.f ? 1.f / lS : 0.f;
  const int64_t ro = row_offset(s, n, h, t);
  float4 oL[NV], oS[NV];
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    oL[c] = make_float4(aL[c].x * iL, aL[c].y * iL, aL[c].z * iL, aL[c].w * iL);
    oS[c] = make_float4(aS[c].x * iS, aS[c].y * iS, aS[c].z * iS, aS[c].w * iS);
  }
  float alpha;
  if (s.gate_mode) {  // Eq. 18: alpha_t = sigmoid(<w_lt, O_lt,t> + <w_st, O_st,t> + b)
    const float *gw = gate + (int64_t)h * (2 * D + 1);
    float a = 0.f;
#pragma unroll
    for (int c = 0; c < NV; ++c) {
      a = dot4(ldw4(gw + (c * 4 + sub) * 4), oL[c], a);
      a = dot4(ldw4(gw + D + (c * 4 + sub) * 4), oS[c], a);
    }
    alpha = sigmoidf_(group_sum(a, gmask) + gw[2 * D]);
  } else {
    alpha = sigmoidf_(gate[h * 2 + 0] - gate[h * 2 + 1]);
  }
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    const float be = 1.f - alpha;
    const float4 o = make_float4(alpha * oL[c].x + be * oS[c].x, alpha * oL[c].y + be * oS[c].y,
                                 alpha * oL[c].z + be * oS[c].z, alpha * oL[c].w + be * oS[c].w);
    const int64_t off = ro + (c * 4 + sub) * 4;
    st4(out + off, o);
    if (out_lt) st4(out_lt + off, oL[c]);
    if (out_st) st4(out_st + off, oS[c]);
  }
  if (sub == 0 && lse) {
    const int64_t BHL = (int64_t)s.B * s.H * s.L;
    lse[(int64_t)u * s.L + t] = lL > 0.f ? mL * kLn2 + __logf(lL) : 0.f;
    lse[BHL + (int64_t)u * s.L + t] = lS > 0.f ? mS * kLn2 + __logf(lS) : 0.f;
  }
}

// ------------------------------------------------------------------------- backward: dQ
// Also produces delta[2][B][H][L] and the per-query-block partial of d alpha for the later kernels.
template <typename T, int D>
__global__ void __launch_bounds__(256) bwd_dq_simt_kernel(
    Shape s, const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, const T *__restrict__ out_lt, const T *__restrict__ out_st,
    const float *__restrict__ lse, const T *__restrict__ dout, T *__restrict__ dq,
    float *__restrict__ delta, double *__restrict__ dalpha_part, float *__restrict__ gate_ac,
    double *__restrict__ dgate_part) {
  constexpr int NV = D / 16, CH = D / 4;
  extern __shared__ float smf[];
  float *Ks = smf, *Vs = Ks + s.Bk * D;
  int *flags = reinterpret_cast<int *>(Vs + s.Bk * D);
  double *red = reinterpret_cast<double *>(flags + s.M + (s.M & 1));  // [Bk]
  uint32_t *rowsel = reinterpret_cast<uint32_t *>(red + s.Bk);  // [Bk][ceil(M / 32)], per-position selection only
  const int MW = (s.M + 31) >> 5;
  const int qb = blockIdx.x % s.M, u = blockIdx.x / s.M, n = u / s.H, h = u % s.H;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int tid = threadIdx.x, r = tid >> 2, sub = tid & 3;
  const unsigned gmask = 0xFu << ((tid & 31) & ~3);
  const int t = qb * s.Bk + r;
  const bool inrange = t < s.L, active = inrange && t >= pad0;
  const int64_t BHL = (int64_t)s.B * s.H * s.L;
  // scalar gate: one alpha per head; input-dependent gate (Eq. 18): one per row, and the row's
  // upstream gradients of the two branches gain c w_lt, c w_st with c = alpha (1 - alpha) <G, O_lt - O_st>
  float alpha = s.gate_mode ? 0.f : sigmoidf_(gate[h * 2 + 0] - gate[h * 2 + 1]), beta = 1.f - alpha;
  const float *gw = gate + (int64_t)h * (2 * D + 1);

  const int hk = h / s.G;  // key/value head of this query head; its group shares one selection
  if (s.pq)
    build_row_selections(s, idx + (((int64_t)n * s.Hkv + hk) * s.L + (inrange ? t : 0)) * s.topk, qb, r, sub, active,
                         flags, rowsel);
  else
    build_visit_flags(s, idx + (((int64_t)n * s.Hkv + hk) * s.M + qb) * s.topk, qb, flags);

  float4 qv[NV], gv[NV], acc[NV], wL[NV], wS[NV];
  float dL = 0.f, dS = 0.f, woL = 0.f, woS = 0.f;
  const int64_t ro = row_offset(s, n, h, inrange ? t : 0);
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    const int64_t off = ro + (c * 4 + sub) * 4;
    qv[c] = active ? ld4(q + off) : zero4();
    gv[c] = active ? ld4(dout + off) : zero4();
    acc[c] = zero4();
    wL[c] = s.gate_mode ? ldw4(gw + (c * 4 + sub) * 4) : zero4();
    wS[c] = s.gate_mode ? ldw4(gw + D + (c * 4 + sub) * 4) : zero4();
    if (active) {
      const float4 ol = ld4(out_lt + off), os = ld4(out_st + off);
      dL = dot4(gv[c], ol, dL);
      dS = dot4(gv[c], os, dS);
      woL = dot4(wL[c], ol, woL);
      woS = dot4(wS[c], os, woS);
    }
  }
  dL = group_sum(dL, gmask);
  dS = group_sum(dS, gmask);
  float cpre = 0.f;
  if (s.gate_mode) {
    woL = group_sum(woL, gmask);
    woS = group_sum(woS, gmask);
    alpha = sigmoidf_(woL + woS + gw[2 * D]);
    beta = 1.f - alpha;
    cpre = active ? alpha * beta * (dL - dS) : 0.f;
    if (inrange && sub == 0) {
      gate_ac[(int64_t)u * s.L + t] = alpha;
      gate_ac[(int64_t)s.B * s.H * s.L + (int64_t)u * s.L + t] = cpre;
    }
  }
  const float deltaL = alpha * dL + cpre * woL, deltaS = beta * dS + cpre * woS;
  float lseL2 = 0.f, lseS2 = 0.f;
  if (active) {
    lseL2 = lse[(int64_t)u * s.L + t] * kLog2e;
    lseS2 = lse[BHL + (int64_t)u * s.L + t] * kLog2e;
  }
  if (inrange && sub == 0) {
    delta[(int64_t)u * s.L + t] = deltaL;
    delta[BHL + (int64_t)u * s.L + t] = deltaS;
  }
  const float sc2 = s.scale * kLog2e;
  const bool block_live = min((qb + 1) * s.Bk, s.L) > pad0;
  // d alpha of the row = <G, O_lt - O_st> = sum_p (P_lt - P_st) dP, accumulated from the fp32
  // probabilities below rather than from the stored (rounded) branch outputs
  float dal = 0.f;
  __syncthreads();

  if (block_live) {
    for (int blk = 0; blk <= (s.causal ? qb : s.M - 1); ++blk) {
      const int f = flags[blk];
      if (!f) continue;
      __syncthreads();
      stage_tile<T, D>(s, k, row_offset_kv(s, n, hk, 0), s.ksl, blk * s.Bk, Ks);
      stage_tile<T, D>(s, v, row_offset_kv(s, n, hk, 0), s.ksl, blk * s.Bk, Vs);
      __syncthreads();
      if (!active) continue;
      const int p0 = blk * s.Bk;
      const int pbeg = max(0, pad0 - p0), pend = min(min(s.Bk, s.L - p0), s.causal ? t - p0 + 1 : s.Bk);
      const bool selb = s.pq ? (rowsel[r * MW + (blk >> 5)] >> (blk & 31)) & 1u : f & 1;
      for (int pi = pbeg; pi < pend; ++pi) {
        const bool inS = st_visible(s, t, p0 + pi);
        if (!selb && !inS) continue;
        const float4 *kr = reinterpret_cast<const float4 *>(Ks) + pi * CH;
        const float4 *vr = reinterpret_cast<const float4 *>(Vs) + pi * CH;
        float part = 0.f, dpart = 0.f, uL = 0.f, uS = 0.f;
#pragma unroll
        for (int c = 0; c < NV; ++c) {
          part = dot4(qv[c], kr[c * 4 + sub], part);
          dpart = dot4(gv[c], vr[c * 4 + sub], dpart);
        }
        if (s.gate_mode) {  // <w_lt, v_p>, <w_st, v_p>: the part of dP that comes through alpha
#pragma unroll
          for (int c = 0; c < NV; ++c) {
            uL = dot4(wL[c], vr[c * 4 + sub], uL);
            uS = dot4(wS[c], vr[c * 4 + sub], uS);
          }
          uL = cpre * group_sum(uL, gmask);
          uS = cpre * group_sum(uS, gmask);
        }
        const float sv = group_sum(part, gmask) * sc2;
        const float dP = group_sum(dpart, gmask);
        float dSsum = 0.f;
        if (selb) {
          const float P = exp2f(sv - lseL2);
          dSsum = P * (alpha * dP + uL - deltaL);
          dal = fmaf(P, dP, dal);
        }
        if (inS) {
          const float P = exp2f(sv - lseS2);
          dSsum = fmaf(P, beta * dP + uS - deltaS, dSsum);
          dal = fmaf(-P, dP, dal);
        }
        const float w = s.scale * dSsum;
#pragma unroll
        for (int c = 0; c < NV; ++c) axpy4(acc[c], w, kr[c * 4 + sub]);
      }
    }
  }
  if (sub == 0) red[r] = active ? (double)dal : 0.0;
  __syncthreads();
  if (tid == 0) {
    double a = 0.0;
    for (int i = 0; i < s.Bk; ++i) a += red[i];  // fixed order
    dalpha_part[(int64_t)u * s.M + qb] = a;
  }
  if (s.gate_mode) {
    // gradient of F_o's parameters from this query block: sum_t c_t O_lt,t, sum_t c_t O_st,t, sum_t c_t
    // (rows staged in the K / V tiles, which nobody reads any more; fixed order over the rows)
    __syncthreads();
#pragma unroll
    for (int c = 0; c < NV; ++c) {
      const int64_t off = ro + (c * 4 + sub) * 4;
      const float4 ol = active ? ld4(out_lt + off) : zero4(), os = active ? ld4(out_st + off) : zero4();
      reinterpret_cast<float4 *>(Ks)[r * CH + c * 4 + sub] = make_float4(cpre * ol.x, cpre * ol.y, cpre * ol.z, cpre * ol.w);
      reinterpret_cast<float4 *>(Vs)[r * CH + c * 4 + sub] = make_float4(cpre * os.x, cpre * os.y, cpre * os.z, cpre * os.w);
    }
    if (sub == 0) red[r] = (double)cpre;
    __syncthreads();
    for (int d = tid; d < 2 * D + 1; d += blockDim.x) {
      double a = 0.0;
      for (int i = 0; i < s.Bk; ++i)
        a += d < D ? (double)Ks[i * D + d] : (d < 2 * D ? (double)Vs[i * D + d - D] : red[i]);
      dgate_part[((int64_t)u * s.M + qb) * (2 * D + 1) + d] = a;
    }
  }
  if (!inrange) return;
#pragma unroll
  for (int c = 0; c < NV; ++c) st4(dq + ro + (c * 4 + sub) * 4, acc[c]);
}

// -------------------------------------------------------------------- backward: dK, dV
template <typename T, int D>
__global__ void __launch_bounds__(256) bwd_dkdv_simt_kernel(
    Shape s, const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
    const float *__restrict__ gate, const int32_t *__restrict__ seq_lens,
    const int32_t *__restrict__ idx, const float *__restrict__ lse,
    const float *__restrict__ delta, const T *__restrict__ dout, T *__restrict__ dk,
    T *__restrict__ dv, const float *__restrict__ gate_ac) {
  constexpr int NV = D / 16, CH = D / 4;
  extern __shared__ float smf[];
  float *Qs = smf, *Gs = Qs + s.Bk * D;
  float *lLs = Gs + s.Bk * D, *lSs = lLs + s.Bk, *dLs = lSs + s.Bk, *dSs = dLs + s.Bk;
  int *flags = reinterpret_cast<int *>(dSs + s.Bk);
  int *rsel = flags + s.M;  // [Bk] per-position selection only: which queries of the staged block selected this key block
  float *als = reinterpret_cast<float *>(rsel + s.Bk), *cs = als + s.Bk;  // [Bk] each: alpha_t, c_t (input-dependent gate)
  // uk counts (batch, key/value head) pairs: the key block collects from every query head of its group
  const int j = blockIdx.x % s.M, uk = blockIdx.x / s.M, n = uk / s.Hkv, hk = uk % s.Hkv;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  const int tid = threadIdx.x, r = tid >> 2, sub = tid & 3;
  const unsigned gmask = 0xFu << ((tid & 31) & ~3);
  const int p = j * s.Bk + r;
  const bool inrange = p < s.L, active = inrange && p >= pad0;
  const int64_t BHL = (int64_t)s.B * s.H * s.L;

  // which query blocks visit this key block: bit 0 = selected it, bit 1 = their short-term branch
  // may reach it
  const int q0 = s.causal ? j : 0, nqv = s.M - q0;  // the query blocks that may visit this key block
  for (int qb = q0 + tid; qb < s.M; qb += blockDim.x) {
    const int32_t *row = idx + ((int64_t)uk * s.M + qb) * s.topk;  // (read only when the selection is per block)
    int f = st_ranges_touch(s, qb * s.Bk, min(s.L, qb * s.Bk + s.Bk) - 1, j * s.Bk,
                            min(s.L, j * s.Bk + s.Bk) - 1) ? 2 : 0;
    if (!s.pq)
      for (int i = 0; i < s.topk; ++i) f |= (row[i] == j) ? 1 : 0;
    flags[qb] = f;
  }

  float4 kv[NV], vv[NV], dka[NV], dva[NV];
  const int64_t ro = row_offset_kv(s, n, hk, inrange ? p : 0);
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    const int64_t off = ro + (c * 4 + sub) * 4;
    kv[c] = active ? ld4(k + off) : zero4();
    vv[c] = active ? ld4(v + off) : zero4();
    dka[c] = zero4();
    dva[c] = zero4();
  }
  const float sc2 = s.scale * kLog2e;
  const bool block_live = min((j + 1) * s.Bk, s.L) > pad0;
  __syncthreads();

  if (block_live) {
    for (int x = 0; x < s.G * nqv; ++x) {  // every query head of the group, every query block that may visit
      const int h = hk * s.G + x / nqv, qb = q0 + x % nqv;
      const int64_t u = (int64_t)n * s.H + h;
      const float alpha_h = s.gate_mode ? 0.f : sigmoidf_(gate[h * 2 + 0] - gate[h * 2 + 1]);
      int f = flags[qb];
      if (s.pq) {  // every query position has a list of its own
        __syncthreads();
        int any = 0;
        for (int i = tid; i < s.Bk; i += blockDim.x) {
          const int t = qb * s.Bk + i;
          int sel = 0;
          if (t < s.L && t >= pad0) {
            const int32_t *row = idx + ((int64_t)uk * s.L + t) * s.topk;
            for (int e = 0; e < s.topk; ++e) sel |= (row[e] == j) ? 1 : 0;
          }
          rsel[i] = sel;
          any |= sel;
        }
        f |= __syncthreads_or(any) ? 1 : 0;
      }
      if (!f) continue;
      __syncthreads();
      stage_tile<T, D>(s, q, row_offset(s, n, h, 0), s.sl, qb * s.Bk, Qs);
      stage_tile<T, D>(s, dout, row_offset(s, n, h, 0), s.sl, qb * s.Bk, Gs);
      for (int i = tid; i < s.Bk; i += blockDim.x) {
        const int t = qb * s.Bk + i;
        const bool ok = t < s.L;
        lLs[i] = ok ? lse[u * s.L + t] * kLog2e : 0.f;
        lSs[i] = ok ? lse[BHL + u * s.L + t] * kLog2e : 0.f;
        dLs[i] = ok ? delta[u * s.L + t] : 0.f;
        dSs[i] = ok ? delta[BHL + u * s.L + t] : 0.f;
        als[i] = s.gate_mode ? (ok ? gate_ac[u * s.L + t] : 0.f) : alpha_h;
        cs[i] = (s.gate_mode && ok) ? gate_ac[BHL + u * s.L + t] : 0.f;
      }
      __syncthreads();
      if (!active) continue;
      // input-dependent gate: <w_lt, v_p>, <w_st, v_p> of this thread's key row and the weights' chunks
      float4 wL[NV], wS[NV];
      float uL = 0.f, uS = 0.f;
      if (s.gate_mode) {
        const float *gw = gate + (int64_t)h * (2 * D + 1);
#pragma unroll
        for (int c = 0; c < NV; ++c) {
          wL[c] = ldw4(gw + (c * 4 + sub) * 4);
          wS[c] = ldw4(gw + D + (c * 4 + sub) * 4);
          uL = dot4(wL[c], vv[c], uL);
          uS = dot4(wS[c], vv[c], uS);
        }
        uL = group_sum(uL, gmask);
        uS = group_sum(uS, gmask);
      }
      const int t0 = qb * s.Bk;
      const int tbeg = s.causal ? max(0, p - t0) : max(0, pad0 - t0), tend = min(s.Bk, s.L - t0);  // valid t (>= p if causal)
      const bool sel_all = f & 1;
      for (int ti = tbeg; ti < tend; ++ti) {
        const bool selb = s.pq ? rsel[ti] != 0 : sel_all;
        const bool inS = st_visible(s, t0 + ti, p);
        if (!selb && !inS) continue;
        const float4 *qr = reinterpret_cast<const float4 *>(Qs) + ti * CH;
        const float4 *gr = reinterpret_cast<const float4 *>(Gs) + ti * CH;
        float part = 0.f, dpart = 0.f;
#pragma unroll
        for (int c = 0; c < NV; ++c) {
          part = dot4(qr[c * 4 + sub], kv[c], part);
          dpart = dot4(gr[c * 4 + sub], vv[c], dpart);
        }
        const float sv = group_sum(part, gmask) * sc2;
        const float dP = group_sum(dpart, gmask);
        const float alpha = als[ti], beta = 1.f - alpha, ct = cs[ti];
        float wv = 0.f, dSsum = 0.f, cwL = 0.f, cwS = 0.f;
        if (selb) {
          const float P = exp2f(sv - lLs[ti]);
          wv = alpha * P;
          cwL = ct * P;
          dSsum = P * (alpha * dP + ct * uL - dLs[ti]);
        }
        if (inS) {
          const float P = exp2f(sv - lSs[ti]);
          wv = fmaf(beta, P, wv);
          cwS = ct * P;
          dSsum = fmaf(P, beta * dP + ct * uS - dSs[ti], dSsum);
        }
        const float wk = s.scale * dSsum;
#pragma unroll
        for (int c = 0; c < NV; ++c) {
          axpy4(dva[c], wv, gr[c * 4 + sub]);
          axpy4(dka[c], wk, qr[c * 4 + sub]);
        }
        if (s.gate_mode) {  // dV_p += P_lt c_t w_lt + P_st c_t w_st
#pragma unroll
          for (int c = 0; c < NV; ++c) {
            axpy4(dva[c], cwL, wL[c]);
            axpy4(dva[c], cwS, wS[c]);
          }
        }
      }
    }
  }
  if (!inrange) return;
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    st4(dk + ro + (c * 4 + sub) * 4, dka[c]);
    st4(dv + ro + (c * 4 + sub) * 4, dva[c]);
  }
}

}  // namespace

// d alpha partials -> dgate[H][2]; one block per head, fixed reduction shape (deterministic).
__global__ void __launch_bounds__(256) gate_grad_kernel(Shape s, const float *__restrict__ gate,
                                                        const double *__restrict__ dalpha_part,
                                                        float *__restrict__ dgate) {
  grid_chain_enter();
  __shared__ double red[256];
  const int h = blockIdx.x;
  double a = 0.0;
  const int per = s.M, total = s.B * per;
  for (int i = threadIdx.x; i < total; i += 256) {
    const int n = i / per, qb = i % per;
    a += dalpha_part[((int64_t)n * s.H + h) * s.M + qb];
  }
  red[threadIdx.x] = a;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double al = 1.0 / (1.0 + exp(-((double)gate[h * 2 + 0] - (double)gate[h * 2 + 1])));
    const double g0 = al * (1.0 - al) * red[0];
    dgate[h * 2 + 0] = (float)g0;
    dgate[h * 2 + 1] = (float)(-g0);
  }
}

// Gradient of F_o's parameters (input-dependent gate): the per-query-block partial sums added
// over batch entries and query blocks in a fixed order.  One warp per (head, parameter): lane i
// adds the entries i, i + 32, ... in ascending order, then a fixed shuffle tree joins the lanes.
__global__ void __launch_bounds__(256) gate_param_grad_kernel(Shape s, const double *__restrict__ part,
                                                              float *__restrict__ dgate) {
  const int GW = 2 * s.D + 1;
  const int w = (int)blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (w >= s.H * GW) return;
  const int h = w / GW, d = w % GW, n_entries = s.B * s.M;
  double a = 0.0;
  for (int e = lane; e < n_entries; e += 32) {
    const int n = e / s.M, qb = e % s.M;
    a += part[(((int64_t)n * s.H + h) * s.M + qb) * GW + d];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  if (lane == 0) dgate[(int64_t)h * GW + d] = (float)a;
}

namespace {

template <typename T, int D>
int launch_fwd_t(const Shape &s, const T *q, const T *k, const T *v, const float *gate,
                 const int32_t *seq_lens, const int32_t *idx, T *out, T *out_lt, T *out_st,
                 float *lse, cudaStream_t st) {
  const unsigned grid = (unsigned)s.M * (unsigned)(s.B * s.H);
  const size_t rowsel = s.pq ? (size_t)s.Bk * ((s.M + 31) / 32) * sizeof(uint32_t) : 0;
  const size_t smem = (size_t)2 * s.Bk * D * sizeof(float) + (size_t)s.M * sizeof(int) + rowsel;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(fwd_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    LaunchScope ls(K_FWD_SIMT, st);
    fwd_simt_kernel<T, D><<<grid, s.Bk * 4, smem, st>>>(s, q, k, v, gate, seq_lens, idx, out, out_lt,
                                                        out_st, lse);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

template <typename T, int D>
int launch_bwd_t(const Shape &s, const T *q, const T *k, const T *v, const float *gate,
                 const int32_t *seq_lens, const int32_t *idx, const T *out_lt, const T *out_st,
                 const float *lse, const T *dout, T *dq, T *dk, T *dv, float *dgate,
                 const Workspace &ws, cudaStream_t st) {
  const unsigned grid = (unsigned)s.M * (unsigned)(s.B * s.H);
  const size_t rowsel = s.pq ? (size_t)s.Bk * ((s.M + 31) / 32) * sizeof(uint32_t) : 0;
  const size_t smem_q = (size_t)2 * s.Bk * D * sizeof(float) +
                        (size_t)(s.M + (s.M & 1)) * sizeof(int) + (size_t)s.Bk * sizeof(double) + rowsel;
  if (smem_q > 48 * 1024 &&
      cudaFuncSetAttribute(bwd_dq_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem_q) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    LaunchScope ls(K_BWD_DQ_SIMT, st);
    bwd_dq_simt_kernel<T, D><<<grid, s.Bk * 4, smem_q, st>>>(s, q, k, v, gate, seq_lens, idx, out_lt,
                                                             out_st, lse, dout, dq, ws.delta,
                                                             ws.dalpha, ws.gate_ac, ws.dgate_part);
  }
  const size_t smem_k = (size_t)(2 * s.Bk * D + 6 * s.Bk) * sizeof(float) + (size_t)(s.M + s.Bk) * sizeof(int);
  if (smem_k > 48 * 1024 &&
      cudaFuncSetAttribute(bwd_dkdv_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem_k) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  {
    LaunchScope ls(K_BWD_DKDV_SIMT, st);
    const unsigned grid_k = (unsigned)s.M * (unsigned)(s.B * s.Hkv);
    bwd_dkdv_simt_kernel<T, D><<<grid_k, s.Bk * 4, smem_k, st>>>(s, q, k, v, gate, seq_lens, idx, lse,
                                                               ws.delta, dout, dk, dv, ws.gate_ac);
  }
  if (s.gate_mode) {
    LaunchScope ls(K_GATE_GRAD, st);
    gate_param_grad_kernel<<<(unsigned)((s.H * (2 * s.D + 1) + 7) / 8), 256, 0, st>>>(s, ws.dgate_part, dgate);
    return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
  }
  return launch_gate_grad(s, gate, ws, dgate, st);
}

}  // namespace

int launch_gate_param_grad(const Shape &s, const Workspace &ws, float *dgate, cudaStream_t st) {
  {
    LaunchScope ls(K_GATE_GRAD, st);
    gate_param_grad_kernel<<<(unsigned)((s.H * (2 * s.D + 1) + 7) / 8), 256, 0, st>>>(s, ws.dgate_part, dgate);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

int launch_gate_grad(const Shape &s, const float *gate, const Workspace &ws, float *dgate,
                     cudaStream_t st) {
  {
    LaunchScope ls(K_GATE_GRAD, st);
    launch_chained(gate_grad_kernel, dim3(s.H), dim3(256), 0, st, s, gate, (const double *)ws.dalpha, dgate);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

int launch_fwd_simt(const Shape &s, int dtype, const void *q, const void *k, const void *v,
                    const float *gate, const int32_t *seq_lens, const int32_t *idx, void *out,
                    void *out_lt, void *out_st, float *lse, const Workspace &, cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == BLOSSOM_DTYPE_FP32) {
    if (s.D == 32)
      return launch_fwd_t<float, 32>(s, (const float *)q, (const float *)k, (const float *)v, gate, seq_lens, idx, (float *)out, (float *)out_lt, (float *)out_st, lse, st);
    return launch_fwd_t<float, 64>(s, (const float *)q, (const float *)k, (const float *)v, gate, seq_lens, idx, (float *)out, (float *)out_lt, (float *)out_st, lse, st);
  }
  if (s.D == 32)
    return launch_fwd_t<bf, 32>(s, (const bf *)q, (const bf *)k, (const bf *)v, gate, seq_lens, idx, (bf *)out, (bf *)out_lt, (bf *)out_st, lse, st);
  return launch_fwd_t<bf, 64>(s, (const bf *)q, (const bf *)k, (const bf *)v, gate, seq_lens, idx, (bf *)out, (bf *)out_lt, (bf *)out_st, lse, st);
}

int launch_bwd_simt(const Shape &s, int dtype, const void *q, const void *k, const void *v,
                    const float *gate, const int32_t *seq_lens, const int32_t *idx,
                    const void *out_lt, const void *out_st, const float *lse, const void *dout,
                    void *dq, void *dk, void *dv, float *dgate, const Workspace &ws,
                    cudaStream_t st) {
  typedef __nv_bfloat16 bf;
  if (dtype == BLOSSOM_DTYPE_FP32) {
    if (s.D == 32)
      return launch_bwd_t<float, 32>(s, (const float *)q, (const float *)k, (const float *)v, gate, seq_lens, idx, (const float *)out_lt, (const float *)out_st, lse, (const float *)dout, (float *)dq, (float *)dk, (float *)dv, dgate, ws, st);
    return launch_bwd_t<float, 64>(s, (const float *)q, (const float *)k, (const float *)v, gate, seq_lens, idx, (const float *)out_lt, (const float *)out_st, lse, (const float *)dout, (float *)dq, (float *)dk, (float *)dv, dgate, ws, st);
  }
  if (s.D == 32)
    return launch_bwd_t<bf, 32>(s, (const bf *)q, (const bf *)k, (const bf *)v, gate, seq_lens, idx, (const bf *)out_lt, (const bf *)out_st, lse, (const bf *)dout, (bf *)dq, (bf *)dk, (bf *)dv, dgate, ws, st);
  return launch_bwd_t<bf, 64>(s, (const bf *)q, (const bf *)k, (const bf *)v, gate, seq_lens, idx, (const bf *)out_lt, (const bf *)out_st, lse, (const bf *)dout, (bf *)dq, (bf *)dk, (bf *)dv, dgate, ws, st);
}

}  // namespace blossom
