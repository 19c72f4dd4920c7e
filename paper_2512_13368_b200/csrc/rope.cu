// Rotary position embedding of q and k inside the library (paper: "RoPE is applied to Q and K to
// encode relative positional information" before both branches).
//
// With rope_theta > 0 every entry point first writes rotated copies of q and k into the workspace
// (same strides as the originals) and runs on those; the backward afterwards turns the gradients
// of the rotated tensors back (the rotation is orthogonal: its transpose).  Pairs are the
// interleaved ones of the original formulation, (x[2i], x[2i+1]), rotated by the angle
// t * theta^(-2i / D) at array position t.  The rotation is evaluated in double precision and
// rounded once to the storage type, so that it is the storage-type rounding of the exact rotation.
#include "common.cuh"

namespace blossom {
namespace {

__device__ __forceinline__ void store_pair(float *p, double a, double b) {
  *reinterpret_cast<float2 *>(p) = make_float2((float)a, (float)b);
}
__device__ __forceinline__ void store_pair(__nv_bfloat16 *p, double a, double b) {
  __nv_bfloat162 h;
  h.x = __double2bfloat16(a);
  h.y = __double2bfloat16(b);
  *reinterpret_cast<__nv_bfloat162 *>(p) = h;
}
__device__ __forceinline__ double2 load_pair(const float *p) {
  const float2 v = *reinterpret_cast<const float2 *>(p);
  return make_double2((double)v.x, (double)v.y);
}
__device__ __forceinline__ double2 load_pair(const __nv_bfloat16 *p) {
  const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162 *>(p);
  return make_double2((double)__bfloat162float(v.x), (double)__bfloat162float(v.y));
}

// One thread per (position t, pair i) and slice of the (batch, head) rows: the angle, its sine and
// cosine are evaluated once and applied to that pair of every row of the slice, so the
// double-precision transcendental work is shared by all rows that sit at the same position.  A
// warp's 32 pairs are 32 consecutive pairs of one row: whole 128-byte (bf16) lines.  heads /
// strides describe the tensor ([B][heads][L][D]); dir = +1 rotates by the position's angle, -1 by
// its negative (the transpose).  src may equal dst.
template <typename T>
__global__ void __launch_bounds__(256) rope_kernel(int B, int heads, int L, int D, int64_t sb, int64_t sh,
                                                   int64_t sl, double theta, int dir, const T *__restrict__ src,
                                                   T *__restrict__ dst) {
  const int half = D / 2;
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (int64_t)L * half) return;
  const int i = (int)(e % half), t = (int)(e / half);
  const double ang = (double)t * pow(theta, -2.0 * (double)i / (double)D) * (double)dir;
  double sn, cs;
  sincos(ang, &sn, &cs);
  const int rows = B * heads;
  const int64_t base = (int64_t)t * sl + 2 * i;
  for (int r0 = (int)blockIdx.y * 4; r0 < rows; r0 += (int)gridDim.y * 4) {
    double2 x[4];
    int64_t off[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {  // four rows in flight
      const int r = r0 + j;
      off[j] = base + (int64_t)(r / heads) * sb + (int64_t)(r % heads) * sh;
      if (r < rows) x[j] = load_pair(src + off[j]);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (r0 + j < rows) store_pair(dst + off[j], x[j].x * cs - x[j].y * sn, x[j].x * sn + x[j].y * cs);
  }
}

template <typename T>
int launch_rope_t(int B, int heads, int L, int D, int64_t sb, int64_t sh, int64_t sl, double theta, int dir,
                  const T *src, T *dst, cudaStream_t st) {
  const int64_t per_row = (int64_t)L * (D / 2);
  const unsigned gx = (unsigned)((per_row + 255) / 256);
  // enough slices of the rows to fill the GPU about eight CTAs deep, each of at least four rows
  const int64_t want = (148 * 8 + gx - 1) / gx, most = ((int64_t)B * heads + 3) / 4;
  int64_t gy = want < 1 ? 1 : (want > most ? most : want);
  if (gy > 65535) gy = 65535;
  {
    LaunchScope ls(K_ROPE, st);
    rope_kernel<T><<<dim3(gx, (unsigned)gy), 256, 0, st>>>(B, heads, L, D, sb, sh, sl, theta, dir, src, dst);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace

// kv = false: a q-shaped tensor (query heads, q strides); true: a k-shaped one.
int launch_rope(const Shape &s, int dtype, bool kv, int dir, const void *src, void *dst, cudaStream_t st) {
  const int heads = kv ? s.Hkv : s.H;
  const int64_t sb = kv ? s.ksb : s.sb, sh = kv ? s.ksh : s.sh, sl = kv ? s.ksl : s.sl;
  if (dtype == BLOSSOM_DTYPE_FP32)
    return launch_rope_t<float>(s.B, heads, s.L, s.D, sb, sh, sl, s.rope_theta, dir, (const float *)src, (float *)dst, st);
  return launch_rope_t<__nv_bfloat16>(s.B, heads, s.L, s.D, sb, sh, sl, s.rope_theta, dir,
                                      (const __nv_bfloat16 *)src, (__nv_bfloat16 *)dst, st);
}

}  // namespace blossom
