// C ABI of the blossom library: argument validation, workspace carving and dispatch.
// Every check happens on the host before anything is launched.
#include <math.h>
#include <stdlib.h>

#include "common.cuh"

namespace blossom {

unsigned long long g_launches = 0;

// ---- optional per-launch event profile (process-wide, off by default) ---------------------
static cudaEvent_t *g_prof_events = nullptr;  // [2 * cap]: before / after each launch
static int *g_prof_ids = nullptr;
static int *g_prof_start = nullptr;           // index of the event a record's time starts at
static int g_prof_cap = 0, g_prof_n = 0;
static cudaStream_t g_prof_chain_stream = nullptr;
static bool g_prof_chain = false;  // the last thing put on g_prof_chain_stream was a record's end event
static int g_prof_every = 1;       // blossom_profile_every: every n-th launch of each kernel is bracketed
static unsigned g_prof_seen[K_COUNT];
static bool g_prof_skip = false;   // the launch in progress is not bracketed

void prof_mark(int id, int phase, cudaStream_t st) {
  if (!g_prof_events) return;
  if (phase == 0) {
    g_prof_skip = (g_prof_seen[id]++ % (unsigned)g_prof_every) != 0;
    if (g_prof_skip) {
      g_prof_chain = false;  // the next bracketed launch records its own start
      return;
    }
    if (g_prof_n >= g_prof_cap) return;
    g_prof_ids[g_prof_n] = id;
    // back-to-back launches of one call share an event: the end of one is the start of the next
    if (g_prof_chain && g_prof_chain_stream == st && g_prof_n > 0) {
      g_prof_start[g_prof_n] = 2 * (g_prof_n - 1) + 1;
    } else {
      g_prof_start[g_prof_n] = 2 * g_prof_n;
      cudaEventRecord(g_prof_events[2 * g_prof_n], st);
    }
  } else {
    if (g_prof_skip || g_prof_n >= g_prof_cap) return;
    cudaEventRecord(g_prof_events[2 * g_prof_n + 1], st);
    g_prof_chain = true;
    g_prof_chain_stream = st;
    ++g_prof_n;
  }
}

// Called on entry of every launching API call: whatever the caller put on the stream since the
// last call must not be charged to this call's first kernel.
void prof_break() { g_prof_chain = false; }

// The environment switches are read once, when the library is loaded.
static bool env_flag(const char *name) {
  const char *e = getenv(name);
  return e && e[0] && e[0] != '0';
}
static const bool g_force_simt = env_flag("BLOSSOM_FORCE_SIMT");
static const bool g_exact_select = env_flag("BLOSSOM_EXACT_SELECT");
static const bool g_serial_launch = env_flag("BLOSSOM_SERIAL_LAUNCH");
static int g_force_simt_override = -1, g_exact_select_override = -1, g_serial_launch_override = -1;  // blossom_debug_switch

bool force_simt() { return g_force_simt_override >= 0 ? g_force_simt_override != 0 : g_force_simt; }

bool chained_launches() {
  return !(g_serial_launch_override >= 0 ? g_serial_launch_override != 0 : g_serial_launch);
}

bool exact_select_only() {
  return g_exact_select_override >= 0 ? g_exact_select_override != 0 : g_exact_select;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

Workspace carve_workspace(const Shape &s, void *base) {
  Workspace w;
  char *p = static_cast<char *>(base);
  size_t off = 0;
  const size_t units = (size_t)s.B * s.H;
  auto take = [&](size_t bytes) {
    char *r = p ? p + off : nullptr;
    off += align_up(bytes, 256);
    return r;
  };
  w.status = reinterpret_cast<int32_t *>(take(256));
  w.status_bwd = w.status ? w.status + 4 : nullptr;
  w.kmean = reinterpret_cast<double *>(take(units * s.M * s.D * sizeof(double)));
  w.klive = reinterpret_cast<int32_t *>(take(units * s.M * sizeof(int32_t)));
  w.kmean32 = reinterpret_cast<float *>(take(units * s.M * s.D * sizeof(float)));
  w.knorm = reinterpret_cast<float *>(take(units * s.M * sizeof(float)));
  w.sel_list = reinterpret_cast<int32_t *>(take(units * s.M * sizeof(int32_t)));
  w.sel_count = reinterpret_cast<int32_t *>(take(256));
  w.delta = reinterpret_cast<float *>(take(2 * units * s.L * sizeof(float)));
  w.dalpha = reinterpret_cast<double *>(take(units * s.M * sizeof(double)));
  w.qstats = reinterpret_cast<float4 *>(take(units * (size_t)((s.L + 63) / 64 * 64) * sizeof(float4)));
  w.cmean = reinterpret_cast<double *>(take(units * (size_t)s.Mc * s.D * sizeof(double)));
  w.clive = reinterpret_cast<int32_t *>(take(units * (size_t)s.Mc * sizeof(int32_t)));
  w.cmean32 = reinterpret_cast<float *>(take(units * (size_t)s.Mc * s.D * sizeof(float)));
  w.cnorm = reinterpret_cast<float *>(take(units * (size_t)s.Mc * sizeof(float)));
  {
    // rotated copies of q and k span what the originals span (same strides)
    const size_t qspan = (size_t)((s.B - 1) * s.sb + (s.H - 1) * s.sh + (int64_t)(s.L - 1) * s.sl + s.D);
    const size_t kspan = (size_t)((s.B - 1) * s.ksb + (s.Hkv - 1) * s.ksh + (int64_t)(s.L - 1) * s.ksl + s.D);
    w.q_rot = take(s.rope_theta > 0 ? qspan * s.esz : 0);
    w.k_rot = take(s.rope_theta > 0 ? kspan * s.esz : 0);
  }
  w.gate_ac = reinterpret_cast<float *>(take(s.gate_mode ? 2 * units * s.L * sizeof(float) : 0));
  w.dgate_part = reinterpret_cast<double *>(take(s.gate_mode ? units * s.M * (2 * s.D + 1) * sizeof(double) : 0));
  {
    // input-dependent gate on the tensor-core kernels (bf16): scratch tensors of the two passes
    const bool on = s.gate_mode && s.esz == 2;
    const size_t qspan = (size_t)((s.B - 1) * s.sb + (s.H - 1) * s.sh + (int64_t)(s.L - 1) * s.sl + s.D);
    const size_t kspan = (size_t)((s.B - 1) * s.ksb + (s.Hkv - 1) * s.ksh + (int64_t)(s.L - 1) * s.ksl + s.D);
    w.gate_glt = take(on ? qspan * 2 : 0);
    w.gate_gst = take(on ? qspan * 2 : 0);
    w.gate_dq = take(on ? qspan * 2 : 0);
    w.gate_olt = take(on ? qspan * 2 : 0);
    w.gate_ost = take(on ? qspan * 2 : 0);
    w.gate_dk = take(on ? kspan * 2 : 0);
    w.gate_dv = take(on ? kspan * 2 : 0);
    w.qstats2 = reinterpret_cast<float4 *>(take(on ? units * (size_t)((s.L + 63) / 64 * 64) * sizeof(float4) : 0));
  }
  w.qmeta = reinterpret_cast<uint8_t *>(take(tc::tc_meta_bytes(s)));
  w.kmeta = reinterpret_cast<uint8_t *>(take(tc::tc_meta_bytes(s) + tc::tc_inv_bits_bytes(s)));
  w.bytes = off;
  return w;
}

// Returns BLOSSOM_OK and fills the shape, or the status describing what is wrong.
static int make_shape(const blossom_params *p, Shape *out) {
  if (!p) return BLOSSOM_ERR_INVALID_ARG;
  if (p->batch < 1 || p->heads < 1 || p->seq_len < 1 || p->head_dim < 1 || p->block_size < 1 ||
      p->top_k < 1 || p->window < 1)
    return BLOSSOM_ERR_INVALID_ARG;
  if (!(p->sm_scale >= 0.f) || isinf(p->sm_scale)) return BLOSSOM_ERR_INVALID_ARG;
  if (p->dtype != BLOSSOM_DTYPE_FP32 && p->dtype != BLOSSOM_DTYPE_BF16)
    return BLOSSOM_ERR_INVALID_ARG;
  if (p->stride_l < p->head_dim || p->stride_h < 1 || p->stride_b < 1) return BLOSSOM_ERR_INVALID_ARG;
  if (p->stride_l % 8 || p->stride_h % 8 || p->stride_b % 8) return BLOSSOM_ERR_INVALID_ARG;
  if (p->kv_heads < 1 || p->heads % p->kv_heads) return BLOSSOM_ERR_INVALID_ARG;
  const bool kv_given = p->kv_stride_b || p->kv_stride_h || p->kv_stride_l;
  if (kv_given && (p->kv_stride_l < p->head_dim || p->kv_stride_h < 1 || p->kv_stride_b < 1 ||
                   p->kv_stride_l % 8 || p->kv_stride_h % 8 || p->kv_stride_b % 8))
    return BLOSSOM_ERR_INVALID_ARG;
  if (p->select_mode < 0 || p->select_mode > 1) return BLOSSOM_ERR_INVALID_ARG;
  if (p->causal != 0 && p->causal != 1) return BLOSSOM_ERR_INVALID_ARG;
  if (p->stis_mode < 0 || p->stis_mode > 1 || p->stis_block < 0) return BLOSSOM_ERR_INVALID_ARG;
  if (p->head_dim != 32 && p->head_dim != 64) return BLOSSOM_ERR_UNSUPPORTED;
  if (p->block_size != 8 && p->block_size != 16 && p->block_size != 32 && p->block_size != 64)
    return BLOSSOM_ERR_UNSUPPORTED;
  if (p->top_k > 64) return BLOSSOM_ERR_UNSUPPORTED;
  const int64_t M = ((int64_t)p->seq_len + p->block_size - 1) / p->block_size;
  if (M > 1024) return BLOSSOM_ERR_UNSUPPORTED;
  if ((int64_t)p->batch * p->heads * M > 0x7fffffffLL) return BLOSSOM_ERR_UNSUPPORTED;
  Shape s;
  s.B = p->batch; s.H = p->heads; s.L = p->seq_len; s.D = p->head_dim; s.Bk = p->block_size;
  s.topk = p->top_k; s.window = p->window; s.M = (int)M;
  s.stis_mode = p->stis_mode; s.stis_blk = p->stis_block > 0 ? p->stis_block : 1;
  s.cmp_l = s.cmp_s = s.Mc = 0;
  if (p->cmp_block < 0 || p->cmp_stride < 0) return BLOSSOM_ERR_INVALID_ARG;
  if (p->cmp_block > 0 || p->cmp_stride > 0) {
    const int l = p->cmp_block > 0 ? p->cmp_block : p->block_size;
    const int st = p->cmp_stride > 0 ? p->cmp_stride : p->block_size;
    if (l % st || p->block_size % st) return BLOSSOM_ERR_INVALID_ARG;
    if (l != p->block_size || st != p->block_size) {
      const int64_t mc = p->seq_len >= l ? ((int64_t)p->seq_len - l) / st + 1 : 0;
      if (mc > 4096) return BLOSSOM_ERR_UNSUPPORTED;
      s.cmp_l = l; s.cmp_s = st; s.Mc = (int)mc;
    }
  }
  s.scale_d = p->sm_scale > 0.f ? (double)p->sm_scale : 1.0 / sqrt((double)p->head_dim);
  s.scale = (float)s.scale_d;
  s.sb = p->stride_b; s.sh = p->stride_h; s.sl = p->stride_l;
  s.Hkv = p->kv_heads; s.G = p->heads / p->kv_heads;
  if (p->gate_mode < 0 || p->gate_mode > 1) return BLOSSOM_ERR_INVALID_ARG;
  s.gate_mode = p->gate_mode;
  if (!(p->rope_theta >= 0.f) || isinf(p->rope_theta) || (p->rope_theta > 0.f && p->rope_theta < 1.f))
    return BLOSSOM_ERR_INVALID_ARG;
  s.rope_theta = (double)p->rope_theta;
  if (p->reuse_tile_lists < 0 || p->reuse_tile_lists > 1) return BLOSSOM_ERR_INVALID_ARG;
  s.reuse_lists = p->reuse_tile_lists;
  s.esz = p->dtype == BLOSSOM_DTYPE_BF16 ? 2 : 4;
  s.pq = p->select_mode;
  s.causal = p->causal;
  s.pack = s.G % 2 == 0 ? 1 : 0;
  if (!s.causal && (s.pq || s.cmp_l > 0)) return BLOSSOM_ERR_UNSUPPORTED;  // bidirectional: plain per-block selection
  s.phi = p->phi_logits;
  if (reinterpret_cast<uintptr_t>(s.phi) % 4) return BLOSSOM_ERR_INVALID_ARG;
  // per-position selection through compression blocks: the tiled kernel only (up to 128 blocks of either kind)
  if (s.pq && s.cmp_l > 0 && (s.Mc > 128 || s.M > 128)) return BLOSSOM_ERR_UNSUPPORTED;
  if (kv_given) {
    s.ksb = p->kv_stride_b; s.ksh = p->kv_stride_h; s.ksl = p->kv_stride_l;
  } else if (s.G == 1) {
    s.ksb = s.sb; s.ksh = s.sh; s.ksl = s.sl;
  } else {
    s.ksl = s.D; s.ksh = (int64_t)s.L * s.D; s.ksb = (int64_t)s.Hkv * s.L * s.D;
  }
  *out = s;
  return BLOSSOM_OK;
}

// With rope_theta > 0: rotated copies of q and k go to the workspace and *q, *k point at them.
// reuse: the copies of the preceding forward on this workspace are still there (the backward's
// reuse_tile_lists promise).
static int rotate_inputs(const Shape &s, int dtype, const Workspace &ws, const void **q, const void **k,
                         cudaStream_t st, bool reuse = false) {
  if (s.rope_theta <= 0) return BLOSSOM_OK;
  if (!reuse) {
    int rc = launch_rope(s, dtype, false, +1, *q, ws.q_rot, st);
    if (rc) return rc;
    rc = launch_rope(s, dtype, true, +1, *k, ws.k_rot, st);
    if (rc) return rc;
  }
  *q = ws.q_rot;
  *k = ws.k_rot;
  return BLOSSOM_OK;
}

static bool misaligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

// Validates the workspace and clears status words on the stream (a memset, not a kernel).  The
// forward (and the selection) report in words 0..3, the backward in words 4..7.  A forward or a
// selection clears both sets (a new step begins), a backward only its own, so a wait that ran out
// in the forward is still on record after the backward that follows it on the same workspace.
static int check_workspace(const Shape &s, void *ws, size_t bytes, cudaStream_t st, Workspace *out,
                           bool backward = false) {
  if (!ws || misaligned(ws, 256)) return BLOSSOM_ERR_WORKSPACE;
  *out = carve_workspace(s, ws);
  if (bytes < out->bytes) return BLOSSOM_ERR_WORKSPACE;
  if (cudaMemsetAsync(backward ? out->status_bwd : out->status, 0, backward ? 16 : 32, st) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  return BLOSSOM_OK;
}

}  // namespace blossom

using namespace blossom;

extern "C" {

size_t blossom_workspace_bytes(const blossom_params *params) {
  Shape s;
  if (make_shape(params, &s) != BLOSSOM_OK) return 0;
  return carve_workspace(s, nullptr).bytes;
}

int blossom_select_blocks(const blossom_params *params, const void *q, const void *k,
                          const int32_t *seq_lens, int32_t *block_idx, void *workspace,
                          size_t workspace_bytes, blossom_stream_t stream) {
  prof_break();
  Shape s;
  int rc = make_shape(params, &s);
  if (rc) return rc;
  if (!q || !k || !block_idx) return BLOSSOM_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(block_idx, 4) || misaligned(seq_lens, 4))
    return BLOSSOM_ERR_INVALID_ARG;
  Workspace ws;
  rc = check_workspace(s, workspace, workspace_bytes, (cudaStream_t)stream, &ws);
  if (rc) return rc;
  rc = rotate_inputs(s, params->dtype, ws, &q, &k, (cudaStream_t)stream);
  if (rc) return rc;
  return launch_select(s, params->dtype, q, k, seq_lens, block_idx, ws, (cudaStream_t)stream);
}

int blossom_select_blocks_static(const blossom_params *params, const void *q, const void *k,
                                 const int32_t *seq_lens, int32_t *block_idx,
                                 blossom_stream_t stream) {
  prof_break();
  Shape s;
  int rc = make_shape(params, &s);
  if (rc) return rc;
  if (!q || !k || !block_idx) return BLOSSOM_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(block_idx, 4) || misaligned(seq_lens, 4))
    return BLOSSOM_ERR_INVALID_ARG;
  return launch_select_static(s, params->dtype, q, k, seq_lens, block_idx, (cudaStream_t)stream);
}

int blossom_attn_fwd(const blossom_params *params, const void *q, const void *k, const void *v,
                     const float *gate_logits, const int32_t *seq_lens, int32_t *block_idx,
                     int32_t idx_is_input, void *out, void *out_lt, void *out_st, float *lse,
                     void *workspace, size_t workspace_bytes, blossom_stream_t stream) {
  prof_break();
  Shape s;
  int rc = make_shape(params, &s);
  if (rc) return rc;
  if (!q || !k || !v || !gate_logits || !block_idx || !out) return BLOSSOM_ERR_INVALID_ARG;
  if ((out_lt == nullptr) != (out_st == nullptr)) return BLOSSOM_ERR_INVALID_ARG;
  if (out_lt && !lse) return BLOSSOM_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(out, 16) ||
      misaligned(out_lt, 16) || misaligned(out_st, 16) || misaligned(lse, 4) ||
      misaligned(gate_logits, 4) || misaligned(block_idx, 4) || misaligned(seq_lens, 4))
    return BLOSSOM_ERR_INVALID_ARG;
  Workspace ws;
  rc = check_workspace(s, workspace, workspace_bytes, (cudaStream_t)stream, &ws);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  rc = rotate_inputs(s, params->dtype, ws, &q, &k, st);
  if (rc) return rc;
  if (!idx_is_input) {
    rc = launch_select(s, params->dtype, q, k, seq_lens, block_idx, ws, st);
    if (rc) return rc;
  }
  if (!force_simt() && tc::fwd_tc_supported(s, params->dtype)) {
    if (s.gate_mode)
      return tc::launch_fwd_tc_gate(s, q, k, v, gate_logits, seq_lens, block_idx, out, out_lt, out_st, lse,
                                    ws, st);
    return tc::launch_fwd_tc(s, q, k, v, gate_logits, seq_lens, block_idx, out, out_lt, out_st, lse, ws,
                             st);
  }
  return launch_fwd_simt(s, params->dtype, q, k, v, gate_logits, seq_lens, block_idx, out, out_lt,
                         out_st, lse, ws, st);
}

int blossom_attn_bwd(const blossom_params *params, const void *q, const void *k, const void *v,
                     const float *gate_logits, const int32_t *seq_lens, const int32_t *block_idx,
                     const void *out_lt, const void *out_st, const float *lse, const void *dout,
                     void *dq, void *dk, void *dv, float *dgate, void *workspace,
                     size_t workspace_bytes, blossom_stream_t stream) {
  prof_break();
  Shape s;
  int rc = make_shape(params, &s);
  if (rc) return rc;
  if (!q || !k || !v || !gate_logits || !block_idx || !out_lt || !out_st || !lse || !dout || !dq ||
      !dk || !dv || !dgate)
    return BLOSSOM_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(out_lt, 16) ||
      misaligned(out_st, 16) || misaligned(dout, 16) || misaligned(dq, 16) || misaligned(dk, 16) ||
      misaligned(dv, 16) || misaligned(lse, 4) || misaligned(dgate, 4) ||
      misaligned(gate_logits, 4) || misaligned(block_idx, 4) || misaligned(seq_lens, 4))
    return BLOSSOM_ERR_INVALID_ARG;
  Workspace ws;
  rc = check_workspace(s, workspace, workspace_bytes, (cudaStream_t)stream, &ws, true);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  rc = rotate_inputs(s, params->dtype, ws, &q, &k, st, s.reuse_lists != 0);
  if (rc) return rc;
  if (!force_simt() && tc::fwd_tc_supported(s, params->dtype)) {
    if (s.gate_mode) {
      rc = tc::launch_bwd_tc_gate(s, q, k, v, gate_logits, seq_lens, block_idx, out_lt, out_st, lse, dout,
                                  dq, dk, dv, dgate, ws, st);
    } else {
      rc = tc::launch_bwd_tc(s, q, k, v, gate_logits, seq_lens, block_idx, out_lt, out_st, lse, dout, dq,
                             dk, dv, ws, st);
      if (!rc) rc = launch_gate_grad(s, gate_logits, ws, dgate, st);
    }
  } else {
    rc = launch_bwd_simt(s, params->dtype, q, k, v, gate_logits, seq_lens, block_idx, out_lt,
                         out_st, lse, dout, dq, dk, dv, dgate, ws, st);
  }
  if (rc || s.rope_theta <= 0) return rc;
  // dq, dk hold the gradients of the rotated tensors: turn them back (the transpose), in place
  rc = launch_rope(s, params->dtype, false, -1, dq, dq, st);
  if (rc) return rc;
  return launch_rope(s, params->dtype, true, -1, dk, dk, st);
}

int blossom_device_status(const void *workspace, blossom_stream_t stream, int32_t *host_out) {
  if (!workspace || !host_out) return BLOSSOM_ERR_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BLOSSOM_ERR_CUDA;
  int32_t words[8];
  if (cudaMemcpy(words, workspace, sizeof(words), cudaMemcpyDeviceToHost) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  *host_out = words[0] ? words[0] : words[4];  // the forward's word, else the backward's
  return BLOSSOM_OK;
}

int blossom_selftest_wait_timeout(void *workspace, size_t workspace_bytes, blossom_stream_t stream) {
  if (!workspace || misaligned(workspace, 256) || workspace_bytes < 256) return BLOSSOM_ERR_WORKSPACE;
  ++g_launches;
  return tc::launch_wait_selftest(static_cast<int32_t *>(workspace), (cudaStream_t)stream);
}

int blossom_debug_switch(int which, int value) {
  if (value < -1 || value > 1) return BLOSSOM_ERR_INVALID_ARG;
  if (which == 0) g_force_simt_override = value;
  else if (which == 1) g_exact_select_override = value;
  else if (which == 2) g_serial_launch_override = value;
  else return BLOSSOM_ERR_INVALID_ARG;
  return BLOSSOM_OK;
}

const char *blossom_status_string(int status) {
  switch (status) {
    case BLOSSOM_OK: return "ok";
    case BLOSSOM_ERR_INVALID_ARG: return "invalid argument";
    case BLOSSOM_ERR_UNSUPPORTED: return "unsupported configuration";
    case BLOSSOM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case BLOSSOM_ERR_CUDA: return "CUDA error";
    case BLOSSOM_ERR_TIMEOUT: return "device-side wait timed out";
    case BLOSSOM_ERR_TOO_LARGE: return "problem exceeds the built-in scratch capacity";
    default: return "unknown status";
  }
}

int blossom_version(void) { return 100; }

int blossom_profile_start(int max_launches) {
  if (max_launches < 1 || g_prof_events) return BLOSSOM_ERR_INVALID_ARG;
  cudaEvent_t *ev = new cudaEvent_t[2 * (size_t)max_launches];
  for (int i = 0; i < 2 * max_launches; ++i)
    if (cudaEventCreate(&ev[i]) != cudaSuccess) {
      for (int j = 0; j < i; ++j) cudaEventDestroy(ev[j]);
      delete[] ev;
      return BLOSSOM_ERR_CUDA;
    }
  g_prof_ids = new int[max_launches];
  g_prof_start = new int[max_launches];
  for (int i = 0; i < K_COUNT; ++i) g_prof_seen[i] = 0;
  g_prof_skip = false;
  g_prof_chain = false;
  g_prof_cap = max_launches;
  g_prof_n = 0;
  g_prof_events = ev;
  return BLOSSOM_OK;
}

int blossom_profile_every(int n) {
  if (n < 1 || g_prof_events) return BLOSSOM_ERR_INVALID_ARG;
  g_prof_every = n;
  return BLOSSOM_OK;
}

int blossom_profile_stop(int32_t *kernel_ids, float *ms, int capacity) {
  if (!g_prof_events) return -1;
  cudaEvent_t *ev = g_prof_events;
  g_prof_events = nullptr;  // stop recording
  int n = g_prof_n < capacity ? g_prof_n : capacity, bad = 0;
  for (int i = 0; i < n; ++i) {
    if (cudaEventSynchronize(ev[2 * i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&ms[i], ev[g_prof_start[i]], ev[2 * i + 1]) != cudaSuccess)
      bad = 1;
    kernel_ids[i] = g_prof_ids[i];
  }
  for (int i = 0; i < 2 * g_prof_cap; ++i) cudaEventDestroy(ev[i]);
  delete[] ev;
  delete[] g_prof_ids;
  delete[] g_prof_start;
  g_prof_ids = nullptr;
  g_prof_start = nullptr;
  g_prof_cap = g_prof_n = 0;
  return bad ? -1 : n;
}

const char *blossom_kernel_name(int id) {
  static const char *names[K_COUNT] = {
      "summary", "score_select", "fwd_simt", "bwd_dq_simt", "bwd_dkdv_simt", "gate_grad",
      "fwd_tc", "bwd_dq_tc", "bwd_dkdv_tc", "score_fast", "bwd_prep", "tc_meta", "rope"};
  return (id >= 0 && id < K_COUNT) ? names[id] : "unknown";
}

uint64_t blossom_launch_count(void) { return g_launches; }

}  // extern "C"
