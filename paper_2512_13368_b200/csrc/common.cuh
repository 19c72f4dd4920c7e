// Shared device/host declarations of the blossom CUDA library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "../../include/blossom.h"

namespace blossom {

// Problem shape handed to every kernel by value.
struct Shape {
  int B, H, L, D, Bk, topk, window, M;
  int stis_mode, stis_blk;  // short-term mask: 0 = window, 1 = power-law (Eq. 15) with block stis_blk
  int cmp_l, cmp_s, Mc;     // overlapping compression blocks (Eq. 8, 11): length, stride, count;
                            // cmp_l == 0: the compression blocks are the selection blocks
  float scale;     // attention logit scale (fp32 arithmetic of the attention kernels)
  double scale_d;  // the same scale in double for the fp64 block scoring
  int64_t sb, sh, sl;  // element strides of q-shaped tensors
  int Hkv, G;             // key/value heads and query heads per key/value head (H = Hkv * G)
  int pq;                 // 1: one selection per query position (block_idx is [B][Hkv][L][top_k])
  double rope_theta;      // > 0: q and k are rotated by position inside the library (base of the angles)
  int esz;                // bytes per element of the q-shaped tensors (2 or 4)
  int causal;             // 1: causal mask (default); 0: bidirectional (CUDA-core kernels)
  int gate_mode;          // 0: one gate weight per head from two logits; 1: Eq. 18's input-dependent gate
  const float *phi;       // logits of the learnable block summary (Eq. 9) or nullptr = the mean
  int reuse_lists;        // backward: the tile lists of the preceding training forward are in the workspace
  int pack;               // tensor-core forward and dQ kernel: a CTA's 128 rows are the same 64 positions of
                          // two query heads that share a key/value head (they select the same blocks,
                          // Eq. 12, and their windows reach the same tiles), not 128 positions of one head;
                          // set whenever the heads per key/value head are even
  int64_t ksb, ksh, ksl;  // element strides of k, v, dk, dv ([B][Hkv][L][D])
};

// Device scratch carved out of the caller's workspace.
struct Workspace {
  int32_t *status;   // [4] word 0: device status (0 = ok) of the selection / forward kernels
  int32_t *status_bwd;  // [4] the same for the backward kernels (status + 4)
  double *kmean;     // [B][H][M][D]  mean of each block's valid keys (Eq. 9 summary)
  int32_t *klive;    // [B][H][M]     number of valid keys in the block
  float *kmean32;    // [B][H][M][D]  the means rounded to fp32 (single-precision scoring stage)
  float *knorm;      // [B][H][M]     upper bound of the Euclidean norm of each fp32 mean
  int32_t *sel_list; // [B][H][M]     query blocks whose choice the fp32 stage could not certify
  int32_t *sel_count;// [1]           length of that list
  float *delta;      // [2][B][H][L]  rowsum(G_branch o O_branch) for the backward
  double *dalpha;    // [B][H][M]     per query block partial of d alpha
  float4 *qstats;    // [B][H][ceil(L/64)*64]  16 bytes per query row, laid out per pair of rows as
                     //   {nl_lt(2), -Delta_lt(2)} {nl_st(2), -Delta_st(2)} for the dK/dV kernel
  double *cmean;     // [B][H][Mc][D]  means of the overlapping compression blocks (cmp_l > 0)
  int32_t *clive;    // [B][H][Mc]     their numbers of valid keys
  float *cmean32;    // [B][H][Mc][D]  the means rounded to fp32
  float *cnorm;      // [B][H][Mc]     upper bounds of the norms of the fp32 means
  void *q_rot, *k_rot;  // rotated copies of q and k (rope_theta > 0), laid out with the originals' strides
  float *gate_ac;    // [2][B][H][L]  input-dependent gate: alpha_t and c_t of every row (backward)
  double *dgate_part;// [B][H][M][2 D + 1]  per query block partial of the gradient of F_o's parameters
  // input-dependent gate on the tensor-core kernels (bf16 only): the two branches' upstream
  // tensors, the second pass's gradients (added to the first pass's afterwards), its records, and
  // the branch outputs of a forward call that does not return them; q-shaped ones laid out with
  // q's strides, k-shaped ones with k's
  void *gate_glt, *gate_gst, *gate_dq, *gate_dk, *gate_dv, *gate_olt, *gate_ost;
  float4 *qstats2;
  uint8_t *qmeta;    // per query-major CTA of the tensor-core kernels: tile lists (tc_meta_kernel)
  uint8_t *kmeta;    // per key-major CTA (dK/dV kernel): tile lists
  size_t bytes;
};

Workspace carve_workspace(const Shape &s, void *base);

extern unsigned long long g_launches;  // host-side launch counter

// Kernel identifiers reported by the optional per-launch event profile.
enum KernelId {
  K_SUMMARY = 0, K_SCORE_SELECT, K_FWD_SIMT, K_BWD_DQ_SIMT, K_BWD_DKDV_SIMT, K_GATE_GRAD,
  K_FWD_TC, K_BWD_DQ_TC, K_BWD_DKDV_TC, K_SCORE_FAST, K_BWD_PREP, K_TC_META, K_ROPE, K_COUNT
};
void prof_mark(int id, int phase, cudaStream_t st);  // no-op unless a profile is running

// Wrap every kernel launch: counts it and, when a profile is running, brackets it with events.
struct LaunchScope {
  int id;
  cudaStream_t st;
  LaunchScope(int id_, cudaStream_t st_) : id(id_), st(st_) { ++g_launches; prof_mark(id, 0, st); }
  ~LaunchScope() { prof_mark(id, 1, st); }
};

// ---- chained launches ---------------------------------------------------------------------
// The kernels of a call follow one another on the caller's stream, each reading what the one before
// wrote.  A kernel launched with launch_chained() may become resident while its predecessor's last
// CTAs still run (programmatic dependent launch), which hides the launch latency and part of the
// predecessor's tail; such a kernel calls grid_chain_enter() as its first statement, in every
// thread: it lets the kernel behind it do the same and then waits until the kernel before it has
// completed and its writes are visible.  Nothing before that call may touch global memory.  Behind
// anything but a kernel (a memset, an event) and with the switch off (chained_launches()) the
// launch is an ordinary one and the call returns at once.
__device__ __forceinline__ void grid_chain_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
bool chained_launches();  // blossom_debug_switch(2, ...) / BLOSSOM_SERIAL_LAUNCH

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chained_launches() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// ---- element access: 4 consecutive elements as float4 ------------------------------------
__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 ld4(const __nv_bfloat16 *p) {
  uint2 r = *reinterpret_cast<const uint2 *>(p);
  float4 o;
  o.x = __uint_as_float(r.x << 16);
  o.y = __uint_as_float(r.x & 0xffff0000u);
  o.z = __uint_as_float(r.y << 16);
  o.w = __uint_as_float(r.y & 0xffff0000u);
  return o;
}
__device__ __forceinline__ void st4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void st4(__nv_bfloat16 *p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);  // round to nearest even, once
  __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
  uint2 r;
  r.x = *reinterpret_cast<uint32_t *>(&a);
  r.y = *reinterpret_cast<uint32_t *>(&b);
  *reinterpret_cast<uint2 *>(p) = r;
}
__device__ __forceinline__ float ld1(const float *p) { return *p; }
__device__ __forceinline__ float ld1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

__device__ __forceinline__ int64_t row_offset(const Shape &s, int n, int h, int t) {
  return (int64_t)n * s.sb + (int64_t)h * s.sh + (int64_t)t * s.sl;
}
// row p of key/value head hk in k, v, dk, dv
__device__ __forceinline__ int64_t row_offset_kv(const Shape &s, int n, int hk, int p) {
  return (int64_t)n * s.ksb + (int64_t)hk * s.ksh + (int64_t)p * s.ksl;
}

// ---- the short-term mask (Eq. 15), shared by the CUDA-core and the tensor-core kernels ----
// Eq. 15: may query t attend to key p in the short-term branch?  (Under the causal mask callers
// only ask for p <= t.)  Mode 0: the window alone, |t - p| < w.  Mode 1 (power-law mask): the
// window, or the block-index distance |floor(t / blk) - floor(p / blk)| is a power of two, or p is
// one of the last blk positions.
__device__ __forceinline__ bool st_visible(const Shape &s, int t, int p) {
  if (abs(t - p) < s.window) return true;
  if (s.stis_mode == 0) return false;
  const int bd = abs(t / s.stis_blk - p / s.stis_blk);
  return (bd >= 1 && (bd & (bd - 1)) == 0) || p >= s.L - s.stis_blk;
}
// May some query in [t0, t1] see some key in [p0, p1] (p0 <= t1 under the causal mask) through the short-term branch?
// Exact for the window; for the power-law mask a superset (any power of two inside the range of
// block distances counts), which only costs a visit: st_visible decides every pair.
__device__ __forceinline__ bool st_ranges_touch(const Shape &s, int t0, int t1, int p0, int p1) {
  if (!s.causal) {  // keys on both sides of the queries
    if (t0 - p1 < s.window && p0 - t1 < s.window) return true;
    if (s.stis_mode == 0) return false;
    if (p1 >= s.L - s.stis_blk) return true;
    // is a power of two among the block distances of keys before the queries, or of keys after?
    const int bq0 = t0 / s.stis_blk, bq1 = t1 / s.stis_blk, bk0 = p0 / s.stis_blk, bk1 = p1 / s.stis_blk;
    const int lmax = bq1 - bk0, lmin = max(1, bq0 - bk1), rmax = bk1 - bq0, rmin = max(1, bk0 - bq1);
    return (lmax >= lmin && (1 << (31 - __clz(lmax))) >= lmin) || (rmax >= rmin && (1 << (31 - __clz(rmax))) >= rmin);
  }
  if (t0 - p1 < s.window) return true;
  if (s.stis_mode == 0) return false;
  if (p1 >= s.L - s.stis_blk) return true;
  const int dmax = t1 / s.stis_blk - p0 / s.stis_blk;
  const int dmin = max(1, t0 / s.stis_blk - p1 / s.stis_blk);
  return dmax >= dmin && (1 << (31 - __clz(dmax))) >= dmin;  // largest power of two <= dmax
}

// launchers (one translation unit each)
int launch_select(const Shape &s, int dtype, const void *q, const void *k, const int32_t *seq_lens,
                  int32_t *idx, const Workspace &ws, cudaStream_t st);
int launch_fwd_simt(const Shape &s, int dtype, const void *q, const void *k, const void *v,
                    const float *gate, const int32_t *seq_lens, const int32_t *idx, void *out,
                    void *out_lt, void *out_st, float *lse, const Workspace &ws, cudaStream_t st);
int launch_bwd_simt(const Shape &s, int dtype, const void *q, const void *k, const void *v,
                    const float *gate, const int32_t *seq_lens, const int32_t *idx,
                    const void *out_lt, const void *out_st, const float *lse, const void *dout,
                    void *dq, void *dk, void *dv, float *dgate, const Workspace &ws,
                    cudaStream_t st);

int launch_select_static(const Shape &s, int dtype, const void *q, const void *k,
                         const int32_t *seq_lens, int32_t *idx, cudaStream_t st);
size_t select_static_capacity_bytes();
int launch_gate_grad(const Shape &s, const float *gate, const Workspace &ws, float *dgate,
                     cudaStream_t st);
// input-dependent gate: fixed-order reduction of ws.dgate_part into dgate [H][2 D + 1]
int launch_gate_param_grad(const Shape &s, const Workspace &ws, float *dgate, cudaStream_t st);
int launch_rope(const Shape &s, int dtype, bool kv, int dir, const void *src, void *dst, cudaStream_t st);

namespace tc {
int launch_wait_selftest(int32_t *status, cudaStream_t st);
bool fwd_tc_supported(const Shape &s, int dtype);
size_t tc_meta_bytes(const Shape &s);  // bytes of one of the two tile-list areas of the workspace
size_t tc_inv_bits_bytes(const Shape &s);  // (selection per position) bytes of the bit table behind the second
// branches: bit 0 long-term, bit 1 short-term branch: the tile lists hold only the tiles those
// branches need.  records: null = computed from out_lt, out_st, lse, dout and the per-head gate by
// the pre-pass; otherwise the caller's per-row records (layout of Workspace::qstats) are used as
// they are.
int launch_bwd_tc(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                  const int32_t *seq_lens, const int32_t *idx, const void *out_lt, const void *out_st,
                  const float *lse, const void *dout, void *dq, void *dk, void *dv,
                  const Workspace &ws, cudaStream_t st, int branches = 3, const float4 *records = nullptr);
// the same two calls with the input-dependent gate (gate = F_o's parameters [H][2 D + 1])
int launch_fwd_tc_gate(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                       const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt, void *out_st,
                       float *lse, const Workspace &ws, cudaStream_t st);
int launch_bwd_tc_gate(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                       const int32_t *seq_lens, const int32_t *idx, const void *out_lt, const void *out_st,
                       const float *lse, const void *dout, void *dq, void *dk, void *dv, float *dgate,
                       const Workspace &ws, cudaStream_t st);
int launch_fwd_tc(const Shape &s, const void *q, const void *k, const void *v, const float *gate,
                  const int32_t *seq_lens, const int32_t *idx, void *out, void *out_lt, void *out_st,
                  float *lse, const Workspace &ws, cudaStream_t st);
}  // namespace tc

// BLOSSOM_FORCE_SIMT=1 in the environment routes every call to the fp32 CUDA-core kernels.
bool force_simt();
// BLOSSOM_EXACT_SELECT=1 scores every query block in double precision (skips the fp32 stage).
bool exact_select_only();

}  // namespace blossom
