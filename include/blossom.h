/*
 * blossom.h -- C ABI of the B200 (sm_100a) BlossomRec block-sparse attention library.
 *
 * One operation, forward and backward: for every (batch, head) the long-term branch scores
 * key-block summaries, keeps the top-k key blocks per query block and attends over them; the
 * short-term branch attends over a causal sliding window; a per-head gate mixes the two.
 *
 * General conventions (all entry points)
 *   - Every pointer is DEVICE memory unless a comment says "host".  The caller owns every
 *     buffer; except where an entry point says otherwise the library allocates nothing,
 *     launches only on the given stream and never synchronises.  State kept between calls: none
 *     that a result depends on; process-wide there are a launch counter, the optional event
 *     profile below, and the debugging switches (blossom_debug_switch).
 *   - q-shaped tensors (q, k, v, out, out_lt, out_st, dout, dq, dk, dv) are [B][H][L][D] with
 *     element strides (stride_b, stride_h, stride_l, 1) shared by all of them; the element type
 *     is params.dtype.  Base pointers must be 16-byte aligned and the three strides multiples
 *     of 8 elements.
 *   - seq_lens[B] (int32, may be NULL = every position valid) is the number of valid,
 *     right-aligned positions of a left-padded sequence.  Padded keys never take part; padded
 *     query rows produce 0 in out / out_lt / out_st / lse and in every gradient.
 *   - block_idx is int32 [B][H][M][top_k], M = ceil(seq_len / block_size): for each query block
 *     the selected key blocks in ascending order, -1 padded.  The query block's own block is
 *     always one of them.  (select_mode 1: a row per query position, [B][H][L][top_k].)
 *   - lse is float [2][B][H][L]: plane 0 long-term branch, plane 1 short-term branch; natural log
 *     of the sum over the branch's visible keys of exp(sm_scale * <q, k>).
 *   - gate_logits is float [H][2]: column 0 long-term, column 1 short-term logit;
 *     alpha_h = sigmoid(g[h][0] - g[h][1]) and out = alpha_h * out_lt + (1 - alpha_h) * out_st.
 *   - Outputs are overwritten, never accumulated into; they need no zeroing.
 *   - Return value: a blossom_status.  Arguments are checked on the host before any launch
 *     (BLOSSOM_ERR_INVALID_ARG / _UNSUPPORTED / _WORKSPACE, nothing launched); a failed launch
 *     gives BLOSSOM_ERR_CUDA.  Device-side bounded waits report through the status word read by
 *     blossom_device_status.
 *   - Calls on different streams are independent as long as their workspaces are distinct.
 */
#ifndef BLOSSOM_H_
#define BLOSSOM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BLOSSOM_OK = 0,
  BLOSSOM_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, non-positive size, bad stride      */
  BLOSSOM_ERR_UNSUPPORTED = 2, /* a legal request this version does not implement               */
  BLOSSOM_ERR_WORKSPACE = 3,   /* workspace NULL, misaligned (256 B) or smaller than required   */
  BLOSSOM_ERR_CUDA = 4,        /* a CUDA launch or runtime call failed                          */
  BLOSSOM_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (see blossom_device_status)*/
  BLOSSOM_ERR_TOO_LARGE = 6    /* problem exceeds the fixed capacity of a no-allocation entry   */
} blossom_status;

enum { BLOSSOM_DTYPE_FP32 = 0, BLOSSOM_DTYPE_BF16 = 1 };

/* CUDA stream handle (same object as cudaStream_t / CUstream); NULL = the default stream. */
typedef struct CUstream_st *blossom_stream_t;

typedef struct {
  int32_t batch, heads;
  int32_t kv_heads;    /* key/value heads: heads must be a multiple; query head h uses key/value
                        * head h / (heads / kv_heads) and a group has ONE selection, made from
                        * the summed scores of its heads (Eq. 12): k, v, dk, dv are
                        * [B][kv_heads][L][D] and block_idx is [B][kv_heads][M][top_k]            */
  int32_t seq_len;     /* L >= 1, ceil(L / block_size) <= 1024                                   */
  int32_t head_dim;    /* D in {32, 64}                                                          */
  int32_t block_size;  /* key block = query block size Bk in {8, 16, 32, 64}                     */
  int32_t top_k;       /* 1 <= top_k <= 64 blocks per query block, the own block included        */
  int32_t window;      /* w >= 1: query t sees keys t - w < p <= t in the short-term branch (and
                        * more with stis_mode 1)                                                 */
  int32_t causal;      /* 1 = causal mask: key p <= query t everywhere, the selection scores the
                        * blocks before the query block.  0 = none (bidirectional encoders): a
                        * query block scores every other live block, a query sees every valid key of
                        * its selected blocks, and Eq. 15 is taken as printed (symmetric); not
                        * combined with select_mode 1 or cmp_block / cmp_stride                    */
  int32_t select_mode; /* 0 = one selection per query block, from the probabilities summed over the
                        * block's queries (tensor-core kernels for bf16); 1 = one selection per
                        * query position (Eq. 13 as printed): block_idx is then
                        * [B][kv_heads][L][top_k], a row per position (tensor-core kernels for
                        * bf16 up to 4096 positions, CUDA-core kernels beyond).  With cmp_block /
                        * cmp_stride a position scores the compression blocks that end before its
                        * selection block starts (up to 128 selection and 128 compression blocks,
                        * else BLOSSOM_ERR_UNSUPPORTED)                                            */
  int32_t dtype;       /* BLOSSOM_DTYPE_FP32 or BLOSSOM_DTYPE_BF16                               */
  float sm_scale;      /* 0 -> 1/sqrt(head_dim); scales block scores and attention logits alike  */
  int64_t stride_b, stride_h, stride_l; /* element strides of every q-shaped tensor              */
  int32_t stis_mode;   /* short-term branch: 0 = causal window only; 1 = the power-law mask of
                        * Eq. 15: window, or block-index distance floor(t/blk) - floor(p/blk) a
                        * power of two, or p among the last blk positions (all with p <= t)      */
  int32_t stis_block;  /* blk >= 1 of the power-law mask (0 reads as 1); ignored in mode 0       */
  int32_t cmp_block;   /* l: length of the compression blocks the selection scores (Eq. 8); 0 =
                        * block_size.  With cmp_stride it allows overlapping blocks whose scores
                        * Eq. 11 maps onto the selection blocks of block_size positions          */
  int32_t cmp_stride;  /* s: their stride; 0 = block_size; must divide cmp_block and block_size  */
  int64_t kv_stride_b, kv_stride_h, kv_stride_l; /* element strides of k, v, dk, dv; all 0 = the
                        * strides above if kv_heads == heads, else contiguous [B][kv_heads][L][D] */
  const float *phi_logits; /* DEVICE pointer or NULL.  Eq. 9's learnable block summary, in the
                        * one-layer form this library takes: a softmax pooling over the positions
                        * of a scored block, summary = sum_i w_i k_i / sum_i w_i over the block's
                        * valid keys, w_i = exp(phi_logits[i]), i the position inside the block;
                        * float [cmp_block] (or [block_size] without compression blocks).  NULL =
                        * the mean.  Only the selection reads it, and no gradient reaches it (the
                        * top-k is piecewise constant), so it has no entry in the backward.       */
  int32_t gate_mode;   /* 0: gate_logits is float [H][2] and alpha_h = sigmoid(g[h][0] - g[h][1]);
                        * 1: the input-dependent gate of Eq. 18 with a one-layer F_o: gate_logits
                        * (and dgate) are float [H][2 D + 1] = (w_lt[D], w_st[D], b) per head and
                        * alpha = sigmoid(<w_lt, out_lt> + <w_st, out_st> + b) per query row,
                        * broadcast over the head's channels in Eq. 19.  The out_lt, out_st that
                        * enter F_o are the rows as stored (bf16 roundings for bf16 tensors on
                        * the tensor-core kernels, which then run the backward once per branch
                        * and need about seven q-sized scratch tensors in the workspace)          */
  float rope_theta;    /* 0 = q and k are used as given.  > 0 (>= 1, e.g. 10000): rotary position
                        * embedding inside the library: q and k are rotated by position before the
                        * selection and both branches (pairs (x[2i], x[2i+1]), angle
                        * t * rope_theta^(-2i / D) at array position t, evaluated in double precision
                        * and rounded once to the storage type; the copies live in the workspace),
                        * and blossom_attn_bwd returns dq, dk with respect to the unrotated inputs  */
  int32_t reuse_tile_lists; /* read by blossom_attn_bwd only.  0: the call builds the tile lists its
                        * kernels walk from block_idx (one more launch).  1: the caller promises that
                        * the last call on this workspace was a blossom_attn_fwd in training mode
                        * (out_lt, out_st given) with the same params, seq_lens and block_idx contents:
                        * that call has left the backward's lists in the workspace and they are used
                        * as they are.  A broken promise gives wrong gradients, not a fault (lists of
                        * another shape are never read: the shape is part of the promise).  The lists
                        * are ignored on the CUDA-core path and with gate_mode 1.  With rope_theta > 0
                        * the promise extends to q and k: the rotated copies that forward left in the
                        * workspace are used instead of being formed again (every path)             */
} blossom_params;

/* Bytes of device scratch the calls below need for these params (one size serves all three);
 * 0 if the params are invalid or unsupported.  The workspace must be 256-byte aligned.  Its
 * contents carry nothing from one call to the next, except that blossom_attn_bwd reads nothing
 * from it that blossom_attn_fwd wrote (the saved tensors are the caller's).  Host function. */
size_t blossom_workspace_bytes(const blossom_params *params /* host */);

/*
 * Block summary, importance scoring and top-k selection (paper: LTIS "Block Splitting",
 * "Block Compression", "Importance Scoring", "Top-k Selection"; Eq. 8-10, 12, 13 with
 * compression size = stride = selection size = block_size and the summary = mean of a block's
 * valid keys).  For each query block b: every valid query of the block takes a softmax of
 * sm_scale * <q, mean-key_j> over the live blocks j < b; the probabilities are summed over the
 * block's queries; the top_k - 1 largest sums (ties to the lower j) plus b itself are written
 * ascending to block_idx.  The choice is the one a double-precision evaluation makes (ties below
 * 1e-12 relative excepted): query blocks are first scored in single precision with an error
 * bound, and only those whose choice the bound cannot certify are re-scored in double precision.
 *   q, k        in   q-shaped
 *   seq_lens    in   [B] or NULL
 *   block_idx   out  [B][H][M][top_k]
 */
int blossom_select_blocks(const blossom_params *params /* host */, const void *q, const void *k,
                          const int32_t *seq_lens, int32_t *block_idx, void *workspace,
                          size_t workspace_bytes, blossom_stream_t stream);

/*
 * blossom_select_blocks for callers that cannot provide a workspace.  (The paper has no
 * counterpart: this is a packaging variant of the selection above, same inputs, same result.)
 *
 * Who needs it: code that runs where device memory can no longer be requested -- inside a
 * serving process whose memory pool was handed out in full at start-up, in a plug-in that is
 * given tensors but no allocator, or on a thread that must not take the allocator's lock.  Such a
 * caller cannot size and allocate the workspace the other entry points ask for, so here the
 * scratch (per-block key means, live counts and the list of query blocks that need the
 * double-precision pass) is a fixed array inside the library image.
 *
 *   - Nothing on this call path allocates or frees memory: no cudaMalloc / cudaFree, no library
 *     allocator.  The array (6 MiB + 96.25 KiB) is resident on every GPU that loads the library,
 *     from load to exit, whether or not this function is ever called.
 *   - Capacity: batch * heads * M <= 8192 and batch * heads * M * head_dim <= 524288
 *     (M = ceil(seq_len / block_size)); larger problems return BLOSSOM_ERR_TOO_LARGE before
 *     anything is launched.  Overlapping compression blocks (cmp_block / cmp_stride other than
 *     block_size) are not taken: BLOSSOM_ERR_UNSUPPORTED.  All other argument rules are those of
 *     blossom_select_blocks (grouped heads included: the capacity then counts kv_heads).
 *   - The first call on each device looks up the array's device address (a runtime query, done
 *     once per device with that device current).  Make that first call outside any stream
 *     capture; later calls only launch kernels on `stream`.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left in it;
 *     each call overwrites every entry before reading it and its first kernel resets the one
 *     counter that must start at zero, so the caller clears nothing.  Two calls
 *     whose kernels may run at the same time on one device (different streams, or different
 *     host threads) race on it and must be serialised by the caller.
 */
int blossom_select_blocks_static(const blossom_params *params /* host */, const void *q,
                                 const void *k, const int32_t *seq_lens, int32_t *block_idx,
                                 blossom_stream_t stream);

/*
 * Forward (paper: Eq. 14 and 16 for the selected-block branch, Eq. 15 under the causal mask
 * (its first case alone with stis_mode 0, all three with stis_mode 1) and Eq. 17 for the
 * short-term branch, Eq. 19 for the gate, each branch being the masked softmax attention of
 * Eq. 1 with online softmax in fp32).
 *   q, k, v      in   q-shaped
 *   gate_logits  in   [H][2]
 *   seq_lens     in   [B] or NULL
 *   block_idx    in/out [B][H][M][top_k]; idx_is_input = 0: selection is computed (as by
 *                blossom_select_blocks) and written here; != 0: used as given (entries outside
 *                [0, M) are ignored; blocks after the query block contribute nothing)
 *   out          out  q-shaped, the gated mix
 *   out_lt,out_st out q-shaped per-branch outputs, needed by the backward; both may be NULL
 *                (inference: nothing is saved), else both non-NULL
 *   lse          out  [2][B][H][L]; may be NULL only when out_lt and out_st are NULL
 */
int blossom_attn_fwd(const blossom_params *params /* host */, const void *q, const void *k,
                     const void *v, const float *gate_logits, const int32_t *seq_lens,
                     int32_t *block_idx, int32_t idx_is_input, void *out, void *out_lt,
                     void *out_st, float *lse, void *workspace, size_t workspace_bytes,
                     blossom_stream_t stream);

/*
 * Backward of blossom_attn_fwd for upstream gradient dout = dLoss/d out, with the selection
 * frozen (top-k is piecewise constant, no gradient flows through the scores).  Chain rule through
 * Eq. 19 (gate), Eq. 16 / 17 and the softmax of Eq. 1, recomputing the probabilities from the
 * saved log-sum-exps: P = exp(sm_scale <q,k> - lse), dV += P^T G, dP = G V^T,
 * dS = P o (dP - rowsum(G o O)), dQ += sm_scale dS K, dK += sm_scale dS^T Q per branch with
 * G_lt = alpha G, G_st = (1 - alpha) G; d alpha_h = sum G o (out_lt - out_st),
 * dgate[h][0] = alpha (1 - alpha) d alpha = -dgate[h][1].
 *   q, k, v, gate_logits, seq_lens, block_idx   in   as given to / produced by the forward
 *   out_lt, out_st, lse                          in   saved by the forward
 *   dout                                         in   q-shaped
 *   dq, dk, dv                                   out  q-shaped
 *   dgate                                        out  float [H][2]
 */
int blossom_attn_bwd(const blossom_params *params /* host */, const void *q, const void *k,
                     const void *v, const float *gate_logits, const int32_t *seq_lens,
                     const int32_t *block_idx, const void *out_lt, const void *out_st,
                     const float *lse, const void *dout, void *dq, void *dk, void *dv,
                     float *dgate, void *workspace, size_t workspace_bytes,
                     blossom_stream_t stream);

/* Synchronises the stream and copies the workspace's device status to *host_out (host): 0 = no
 * device-side error, else a blossom_status.  The workspace holds one status word for the forward
 * (blossom_select_blocks and blossom_attn_fwd clear both words when they start: a new step) and
 * one for the backward (blossom_attn_bwd clears only that one), so a read after a forward + backward pair on one
 * workspace reports a wait that ran out in either; the forward's word wins if both are set.
 * Returns BLOSSOM_ERR_CUDA if the synchronise or the copy fails. */
int blossom_device_status(const void *workspace, blossom_stream_t stream, int32_t *host_out);

/* Diagnostic (no counterpart in the paper): shows that a device-side wait that cannot complete
 * ends in a report, not in a hang.  Launches one tiny kernel on `stream` that sets up tensor
 * memory and an mbarrier like the attention kernels and then waits for an arrival nobody makes:
 * the wait gives up after the library's limit (about 0.2 s of GPU time), the kernel runs to its
 * normal end, frees its tensor memory and records BLOSSOM_ERR_TIMEOUT in the status words at the
 * start of `workspace` (>= 256 bytes, 256-byte aligned), where blossom_device_status finds it.
 * The context stays usable.  Returns BLOSSOM_OK if the kernel was launched. */
int blossom_selftest_wait_timeout(void *workspace, size_t workspace_bytes, blossom_stream_t stream);

/* Debugging switches (no counterpart in the paper), process-wide, host only, not thread-safe.
 * which = 0: route every call to the fp32 CUDA-core kernels instead of the tensor-core ones;
 * which = 1: score every query block in double precision (skip the certified fp32 stage);
 * which = 2: launch every kernel fully serialised behind its predecessor (by default the kernels
 * of a call are chained by programmatic dependent launches: a kernel may become resident while
 * the last CTAs of the one before it still run, and waits for that kernel's completion before it
 * touches global memory; results do not depend on the switch).
 * value 1 = on, 0 = off, -1 = back to the default, which is the environment variable
 * BLOSSOM_FORCE_SIMT, BLOSSOM_EXACT_SELECT resp. BLOSSOM_SERIAL_LAUNCH as it stood when the
 * library was loaded (unset or "0" = off).  Returns BLOSSOM_ERR_INVALID_ARG for other arguments. */
int blossom_debug_switch(int which, int value);

/* Human-readable name of a blossom_status (host string, static storage). */
const char *blossom_status_string(int status);

/* Library version: major * 10000 + minor * 100 + patch. */
int blossom_version(void);

/* Number of kernels the library launched from this process since it was loaded (all streams);
 * a host-side counter for benchmarks. */
uint64_t blossom_launch_count(void);

/*
 * Measurement aid (no counterpart in the paper): per-launch device times of the library's own
 * kernels.  blossom_profile_start creates 2 * max_launches CUDA events; from then on every
 * kernel the library launches (any stream) is bracketed by two event records until
 * blossom_profile_stop, which waits for the recorded events, writes for launch i its kernel id
 * and its device time in milliseconds to kernel_ids[i] / ms[i] (host arrays of `capacity`
 * entries), destroys the events and returns the number of launches written (-1 on error or if
 * no profile is running).  Process-wide and not thread-safe; off by default; launches beyond
 * max_launches are not recorded.  blossom_kernel_name maps an id to a static host string.
 * An event record between two kernels keeps the second from becoming resident before the first
 * has completed (see blossom_debug_switch, which = 2) and costs a few microseconds itself;
 * blossom_profile_every(n), called while no profile is running, makes the following profiles
 * bracket only every n-th launch of each kernel (n >= 1, default 1; BLOSSOM_ERR_INVALID_ARG
 * otherwise), so that a timed loop of several steps is disturbed in one step out of n.
 */
int blossom_profile_start(int max_launches);
int blossom_profile_every(int n);
int blossom_profile_stop(int32_t *kernel_ids /* host */, float *ms /* host */, int capacity);
const char *blossom_kernel_name(int kernel_id);

#ifdef __cplusplus
}
#endif
#endif /* BLOSSOM_H_ */
