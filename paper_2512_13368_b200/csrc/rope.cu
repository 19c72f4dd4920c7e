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

// One thread per (row, pair).  heads / strides describe the tensor ([B][heads][L][D]); dir = +1
// rotates by the position's angle, -1 by its negative (the transpose).  src may equal dst.
template <typename T>
__global__ void __launch_bounds__(256) rope_kernel(int B, int heads, int L, int D, int64_t sb, int64_t sh,
                                                   int64_t sl, double theta, int dir, const T *__restrict__ src,
                                                   T *__restrict__ dst) {
  const int half = D / 2;
  const int64_t total = (int64_t)B * heads * L * half;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int i = (int)(e % half);
    const int64_t row = e / half;
    const int t = (int)(row % L);
    const int h = (int)((row / L) % heads), n = (int)(row / ((int64_t)L * heads));
    const int64_t off = (int64_t)n * sb + (int64_t)h * sh + (int64_t)t * sl + 2 * i;
    const double ang = (double)t * pow(theta, -2.0 * (double)i / (double)D) * (double)dir;
    double sn, cs;
    sincos(ang, &sn, &cs);
    const double2 x = load_pair(src + off);
    store_pair(dst + off, x.x * cs - x.y * sn, x.x * sn + x.y * cs);
  }
}

template <typename T>
int launch_rope_t(int B, int heads, int L, int D, int64_t sb, int64_t sh, int64_t sl, double theta, int dir,
                  const T *src, T *dst, cudaStream_t st) {
  const int64_t total = (int64_t)B * heads * L * (D / 2);
  const unsigned grid = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
  {
    LaunchScope ls(K_ROPE, st);
    rope_kernel<T><<<grid, 256, 0, st>>>(B, heads, L, D, sb, sh, sl, theta, dir, src, dst);
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
