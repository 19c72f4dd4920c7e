// Host side of the tensor-core path: TMA descriptors and dispatch on the head dimension.
#include "tc_common.cuh"

namespace blossom {
namespace tc {

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

// q-shaped bf16 tensor [B][H][L][D] with the caller's strides, box = (D, box_rows, box_heads, 1)
// (the box's heads follow one another in shared memory, box_rows rows each); rows past L read as zeros.  The swizzle matches the shared-memory descriptors of the kernels.
int make_tensor_map(CUtensorMap *map, const void *base, const Shape &s, int box_rows, bool kv, int box_heads) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return 1;
  // kv: a key/value-shaped tensor [B][Hkv][L][D] with its own strides
  const cuuint64_t dims[4] = {(cuuint64_t)s.D, (cuuint64_t)s.L, (cuuint64_t)(kv ? s.Hkv : s.H), (cuuint64_t)s.B};
  const cuuint64_t strides[3] = {(cuuint64_t)(kv ? s.ksl : s.sl) * 2, (cuuint64_t)(kv ? s.ksh : s.sh) * 2,
                                 (cuuint64_t)(kv ? s.ksb : s.sb) * 2};
  const cuuint32_t box[4] = {(cuuint32_t)s.D, (cuuint32_t)box_rows, (cuuint32_t)box_heads, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUtensorMapSwizzle sw = s.D == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
  CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? 0 : 1;
}

// Diagnostic kernel: the bounded-wait machinery of the attention kernels on a wait that cannot
// complete.  One CTA allocates tensor memory like the attention kernels, initialises an mbarrier
// that expects an arrival nobody makes, and every warp waits on it: the waits run out after the
// common limit, the first one records its site, later ones return at once, and the common kernel
// end frees the tensor memory and reports BLOSSOM_ERR_TIMEOUT, the site and the CTA through the
// status words.  Nothing faults and nothing spins without bound.
__global__ void __launch_bounds__(128) wait_selftest_kernel(int32_t *status) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_slot), 32);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  mbar_wait(smem_u32(&bar), 0, &abort_flag, 900 + warp);  // phase 0 never completes
  finish(warp, tmem_slot, 32, &abort_flag, status);
}

int launch_wait_selftest(int32_t *status, cudaStream_t st) {
  if (cudaMemsetAsync(status, 0, 32, st) != cudaSuccess) return BLOSSOM_ERR_CUDA;
  wait_selftest_kernel<<<1, 128, 0, st>>>(status);
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

bool fwd_tc_supported(const Shape &s, int dtype) {
  // (a selection per query position adds 128 bytes per tile to a CTA's bookkeeping in shared
  // memory: up to 64 tiles, i.e. L <= 4096; longer sequences take the CUDA-core kernels)
  // (the input-dependent gate goes through launch_fwd_tc_gate / launch_bwd_tc_gate)
  return (!s.pq || (s.L + 63) / 64 <= 64) && dtype == BLOSSOM_DTYPE_BF16 && (s.D == 32 || s.D == 64) &&
         (s.Bk == 16 || s.Bk == 32 || s.Bk == 64) && (s.L + 63) / 64 <= 1024;
}

size_t tc_meta_bytes(const Shape &s) {
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  return ((size_t)s.B * s.H * nST * (size_t)meta_bytes(nT, s.pq) + 255) / 256 * 256;
}

// Selection per query position: one bit per (batch, key/value head, key block, position) = that
// position selected that block; written while the query-major images are built, read by the
// key-major ones.  It lies behind the key-major images in the workspace.
size_t tc_inv_bits_bytes(const Shape &s) {
  return s.pq ? (size_t)s.B * s.Hkv * s.M * (size_t)((s.L + 31) / 32) * sizeof(uint32_t) : 0;
}

int launch_fwd_tc(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                  const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt, void *out_st,
                  float *lse, const Workspace &ws, cudaStream_t st) {
  if (s.D == 32) return launch_fwd_tc_t<32>(s, q, k, v, gate, seq_lens, idx, out, out_lt, out_st, lse, ws, st);
  return launch_fwd_tc_t<64>(s, q, k, v, gate, seq_lens, idx, out, out_lt, out_st, lse, ws, st);
}

int launch_bwd_tc(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                  const int32_t *seq_lens, const int32_t *idx, const void *out_lt, const void *out_st,
                  const float *lse, const void *dout, void *dq, void *dk, void *dv,
                  const Workspace &ws, cudaStream_t st, int branches, const float4 *records) {
  if (s.D == 32)
    return launch_bwd_tc_t<32>(s, q, k, v, gate, seq_lens, idx, out_lt, out_st, lse, dout, dq, dk, dv, ws, st,
                               branches, records);
  return launch_bwd_tc_t<64>(s, q, k, v, gate, seq_lens, idx, out_lt, out_st, lse, dout, dq, dk, dv, ws, st,
                             branches, records);
}

}  // namespace tc
}  // namespace blossom
