/*
 * libgswa: Group Shifted Window Attention (GSWA) for NVIDIA B200 (sm_100a).
 *
 * One attention layer of AgileIR (arXiv 2409.06206), Sec. "Group Shifted Window
 * Attention": the heads of a window-attention layer are split into groups; a
 * group with shift 0 attends inside plain non-overlapping M x M windows
 * (GW-MSA), a group with shift s > 0 attends after a cyclic shift of the
 * feature map under the shifted-window mask (GSW-MSA); every head adds a
 * learnable relative-position bias (Sec. "Learnable Relative Shifted Bias");
 * the heads are concatenated and projected (Eq. 6, Eq. 7).  Forward and the
 * training backward are provided; the backward recomputes the attention
 * weights per window and never stores an M^2 x M^2 matrix.
 *
 * Plain C ABI.  Unless a parameter says "host", every pointer is a DEVICE
 * pointer owned by the caller, 16-byte aligned, valid until the work enqueued
 * on `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream) has
 * finished.  Except where stated the library allocates no device memory and
 * keeps no tensor state between calls.  What it does keep, per device and
 * until the process exits: one internal non-blocking stream with three events
 * (created on the first gswa_backward of a bf16 tensor-core layer; that call
 * forks its two weight-gradient GEMMs onto it and joins it back into
 * `cuda_stream` before returning, on every exit path, so the caller only ever
 * orders against `cuda_stream`; concurrent gswa_backward calls on one device
 * take turns enqueueing on it), the cached multiprocessor count, and the
 * address of the built-in array of gswa_forward_static.  Every function returns
 * GSWA_OK (0) or a negative gswa_status; argument errors are reported before
 * anything is enqueued; nothing throws, traps or asserts on the device.
 *
 * Tensor conventions (the paper leaves them open):
 *   x, y, dy, dx      [B,H,W,C], C fastest.
 *   w_qkv             [3C, C] row-major (out, in); rows ordered q | k | v, head-major inside each.
 *                     With narrowed projections (qk_dim, v_dim below): [2*heads*qk_dim + heads*v_dim, C].
 *   b_qkv             [3C] (in general: one entry per row of w_qkv) or NULL (= zeros).
 *   w_proj, b_proj    [C, C] (out, in) (in general [C, heads*v_dim]), [C] or NULL.
 *   bias_table        [(2M-1)^2, num_heads]; row (a_p-a_q+M-1)(2M-1) + (c_p-c_q+M-1) for query slot
 *                     (a_p,c_p) and key slot (a_q,c_q) of a window.
 *   q k^T is scaled by qk_dim^-1/2 (= head_dim^-1/2 by default); softmax runs over keys; the mask removes pairs
 *   (weight exactly 0).
 *   cyclic shift by s: shifted[i',j'] = x[(i'+s) mod H, (j'+s) mod W].
 * All of x, y, dy, dx, weights, biases and the table have the element type
 * `dtype`; parameter gradients are always float32.
 */
#ifndef GSWA_H_
#define GSWA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gswa_status {
  GSWA_OK = 0,
  GSWA_ERR_NULL = -1,        /* a required pointer is NULL                                  */
  GSWA_ERR_SHAPE = -2,       /* inconsistent sizes (H or W not a multiple of M, bad groups) */
  GSWA_ERR_ALIGN = -3,       /* a device pointer is not 16-byte aligned                     */
  GSWA_ERR_UNSUPPORTED = -4, /* valid but not implemented (e.g. a window problem too large for one block) */
  GSWA_ERR_WORKSPACE = -5,   /* scratch / saved buffer too small                            */
  GSWA_ERR_CUDA = -6,        /* a CUDA runtime call or launch failed                        */
  GSWA_ERR_DEVICE = -7       /* a kernel gave up on a bounded internal wait (gswa_scratch_status) */
} gswa_status;

enum { GSWA_F32 = 0, GSWA_BF16 = 1 };

enum {
  GSWA_FLAG_ACCUMULATE = 1u, /* add into the parameter gradients instead of overwriting them */
  GSWA_FLAG_GENERIC = 2u,    /* force the shape-generic CUDA-core kernels (no tensor-core fast path) */
  /* (No flag asks for bitwise-reproducible reductions: the float32 parameter gradients are accumulated with
   *  atomics on every path, see gswa_backward.) */
  GSWA_FLAG_FUSED_FWD = 4u,  /* tensor-core path: one kernel for QKV projection + forward attention (slower at C = 180; kept as a measured alternative) */
  GSWA_FLAG_TCGEN05_ATTN = 8u, /* tensor-core path: attention backward on tcgen05 with TMEM accumulators instead of warp-level mma.sync (4 % slower at C = 180; kept as a measured alternative) */
  GSWA_FLAG_COPY_LOADERS = 16u /* tensor-core path: feed the window-order GEMMs with 8/16-byte asynchronous copies into a shared-memory operand (the path layers with odd shifts take anyway) instead of bulk copies + a TMEM A operand */
};

/* Layer description (host memory, read during the call only). */
typedef struct gswa_desc {
  int32_t B, H, W, C;         /* x is [B,H,W,C]                                               */
  int32_t num_heads;          /* C % num_heads == 0; head_dim = C / num_heads                 */
  int32_t window;             /* M; H % M == 0 and W % M == 0                                 */
  int32_t num_groups;         /* G >= 1                                                       */
  const int32_t* group_heads; /* host [G]; consecutive heads per group; sums to num_heads     */
  const int32_t* group_shift; /* host [G]; 0 <= s < M; 0 = plain windows, no mask             */
  int32_t dtype;              /* GSWA_F32 or GSWA_BF16                                        */
  int32_t qk_dim, v_dim;      /* per-head widths of q,k and of v (Sec. "Parameter Allocation": Q and K narrowed to
                                 16 or 32 channels); 0 = head_dim = C / num_heads.  Other widths (<= 64) run on the
                                 shape-generic kernels                                                            */
  uint32_t flags;             /* GSWA_FLAG_*                                                  */
} gswa_desc;

/* Buffer sizes for a layer description.
 *   saved_bytes          forward -> backward carry (projected q,k,v, attention output, row log-sum-exp).
 *   fwd_scratch_bytes    scratch of gswa_forward when `saved` is given.
 *   infer_scratch_bytes  scratch of gswa_forward when `saved` is NULL (the carry then lives in scratch): a
 *                        fourth size beside the three a training caller needs, so that an inference caller
 *                        allocates one buffer instead of two.
 *   bwd_scratch_bytes    scratch of gswa_backward.
 * Any output pointer may be NULL. */
int gswa_workspace_query(const gswa_desc* desc, size_t* saved_bytes, size_t* fwd_scratch_bytes,
                         size_t* infer_scratch_bytes, size_t* bwd_scratch_bytes);

/* Forward pass, Eq. 6 and Eq. 7 with the window mask and relative bias:
 *   y = Concat_h[ softmax(q_h k_h^T / sqrt(d) + B_h + mask) v_h ] W^P + b^P,  (q|k|v) = x W_qkv^T + b_qkv.
 * `saved` (saved_bytes) receives what gswa_backward needs, or is NULL for inference.
 * Contents of `scratch` are undefined afterwards.  Asynchronous on `cuda_stream`. */
int gswa_forward(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                 const void* b_proj, const void* bias_table, void* y, void* saved, void* scratch,
                 size_t scratch_bytes, void* cuda_stream);

/* Inference forward for callers that cannot allocate device memory (the paper has no counterpart).
 * Some hosts hand a library its input and output buffers and nothing else: a plug-in loaded into an
 * application that owns all device memory, a C program without an allocator for the GPU, a real-time
 * loop in which cudaMalloc (which may synchronise the whole device) is not acceptable.  gswa_forward
 * needs `infer_scratch_bytes` of scratch from such a caller; this variant takes none.  It computes
 * exactly what gswa_forward computes with saved == NULL, and keeps its intermediates (projected q,k,v
 * tiles, attention output, weight images) in one array that is part of the library's device image:
 * GSWA_STATIC_SCRATCH_BYTES bytes, held on every GPU that loads the library until the process exits.
 *   - A layer whose infer_scratch_bytes (gswa_workspace_query) exceeds GSWA_STATIC_SCRATCH_BYTES is
 *     rejected with GSWA_ERR_WORKSPACE before anything is enqueued; nothing is ever allocated or freed,
 *     by this call or by anything it calls.
 *   - The first call on a device looks the array's device address up (once per device, with the
 *     caller's current device); make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the last call's contents; what has to
 *     start from zero is cleared by each call.  Two calls whose work overlaps on the GPU (different
 *     streams, or different threads) race on it: serialise them.
 * x, the parameters and y are the caller's device buffers as for gswa_forward. */
#define GSWA_STATIC_SCRATCH_BYTES (16u << 20)
int gswa_forward_static(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv,
                        const void* w_proj, const void* b_proj, const void* bias_table, void* y, void* cuda_stream);

/* Device-side status of the last gswa_forward_static on the current device (the paper has no counterpart): what
 * gswa_scratch_status is for caller-owned scratch, for the built-in array whose address the caller cannot name.
 * Waits for `cuda_stream`; returns GSWA_OK or GSWA_ERR_DEVICE (y is then invalid).  Allocates nothing.  The
 * array's address is looked up once per device and cached for the life of the process: after a cudaDeviceReset the
 * cached address is stale, so a process that resets a device must not call the *_static functions on it again. */
int gswa_static_status(void* cuda_stream);

/* Backward pass (reverse mode of gswa_forward; the paper's stated target is the memory of
 * back-propagation).  `saved` is the buffer written by gswa_forward for the same desc and inputs; the weights must
 * be the ones that call was given (on the tensor-core path `saved` also carries the re-laid-out copies of them that
 * the backward GEMMs read, so that this call launches no preparation kernel).
 * Writes dx (element type `dtype`) and the float32 parameter gradients dw_qkv[3C,C], db_qkv[3C],
 * dw_proj[C,C], db_proj[C], dbias_table[(2M-1)^2, num_heads]; each gradient pointer may be NULL to
 * skip it (dx included).  Gradients are overwritten unless GSWA_FLAG_ACCUMULATE is set.  Float32
 * reductions use atomics: results are reproducible to rounding, not bitwise. */
int gswa_backward(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                  const void* bias_table, const void* saved, const void* dy, void* dx, float* dw_qkv,
                  float* db_qkv, float* dw_proj, float* db_proj, float* dbias_table, void* scratch,
                  size_t scratch_bytes, void* cuda_stream);

/* Index maps of group `group`, computed on the device by the routines the shape-generic kernels use
 * (Sec. "Patch Embedding" window partition; cyclic shift and window mask of GSW-MSA); gswa_debug_index_maps
 * below exposes the arithmetic of the tensor-core kernels.  All int32,
 * any pointer may be NULL:
 *   win[H*W], slot[H*W], region[H*W]   per ORIGINAL token (i,j): window number in the shifted frame,
 *                                      slot inside it (row-major M x M), mask label 3*r(i')+r(j')
 *                                      with r = 0 on [0,n-M), 1 on [n-M,n-s), 2 on [n-s,n);
 *   token_of[H*W]                      inverse map: token_of[win*M*M + slot] = i*W + j;
 *   rel_index[M^2 * M^2]               bias-table row for (query slot, key slot). */
int gswa_index_maps(const gswa_desc* desc, int32_t group, int32_t* win, int32_t* slot, int32_t* region,
                    int32_t* token_of, int32_t* rel_index, void* cuda_stream);

/* Index maps of group `group` over the whole batch, computed by the arithmetic of the kernels that will run the
 * layer: for a layer on the bf16 tensor-core path, by the window set-up and bias-row routines of its attention
 * kernels; otherwise by the routines of gswa_index_maps.  For
 * bit-exact comparison with the definition (Sec. "Patch Embedding"; shift and mask of GSW-MSA; Sec. "Learnable
 * Relative Shifted Bias").  All int32 device pointers, any of them may be NULL:
 *   win_id[B*H*W]        b * (H/M)(W/M) + window of every token in the shifted frame;
 *   slot[H*W], region[H*W], rel_index[M^2 * M^2]   as in gswa_index_maps. */
int gswa_debug_index_maps(const gswa_desc* desc, int32_t group, int32_t* win_id, int32_t* slot, int32_t* region,
                          int32_t* rel_index, void* cuda_stream);

/* Test hook for the device-side failure report (the paper has no counterpart): enqueues a one-block kernel that
 * waits on a barrier nobody arrives on, gives up after about two thousand polls (well under a millisecond), sets the
 * error word at the head of `scratch` exactly as a tensor-core kernel does when one of its bounded waits runs
 * out, and returns normally.  gswa_scratch_status(desc, scratch) then reports GSWA_ERR_DEVICE; the next
 * gswa_forward / gswa_backward on that scratch clears the word.  Nothing faults, traps or hangs.
 * GSWA_ERR_UNSUPPORTED for layers off the tensor-core path (they keep no error word). */
int gswa_debug_expire_wait(const gswa_desc* desc, void* scratch, void* cuda_stream);

/* ---- The layer around GSWA (Sec. "Agile Swin Transformer Block", Eq. 4 and Eq. 5):
 *        X1 = GSWA(LN(X)) + X,    X2 = MLP(LN(X1)) + X1.
 * LayerNorm is taken over the C channels of each token (biased variance, eps = 1e-5, learnable scale and shift);
 * the MLP is FC1 [mlp_hidden, C] -> GELU (exact Gaussian-CDF form) -> FC2 [C, mlp_hidden].  mlp_hidden == 0 stops
 * after Eq. 4 (the output is X1 and the second LayerNorm / MLP pointers are ignored).  All pointers of both
 * structures are DEVICE pointers; parameters have the element type `dtype`, gradients are float32 and every one of
 * them is required (overwritten unless GSWA_FLAG_ACCUMULATE).  `saved` / `scratch` follow gswa_forward /
 * gswa_backward: sizes from gswa_astl_workspace_query, `saved` NULL = inference (scratch of infer_scratch_bytes).
 * The device error word of the tensor-core attention kernels is at the head of `scratch` (gswa_scratch_status). */
typedef struct gswa_astl_params {
  const void *ln1_g, *ln1_b;                                    /* [C]                                   */
  const void *w_qkv, *b_qkv, *w_proj, *b_proj, *bias_table;     /* as for gswa_forward (b_* may be NULL) */
  const void *ln2_g, *ln2_b;                                    /* [C]                                   */
  const void *w_fc1, *b_fc1;                                    /* [mlp_hidden, C], [mlp_hidden]         */
  const void *w_fc2, *b_fc2;                                    /* [C, mlp_hidden], [C]                  */
} gswa_astl_params;
typedef struct gswa_astl_grads {
  float *dln1_g, *dln1_b, *dw_qkv, *db_qkv, *dw_proj, *db_proj, *dbias_table;
  float *dln2_g, *dln2_b, *dw_fc1, *db_fc1, *dw_fc2, *db_fc2;
} gswa_astl_grads;
int gswa_astl_workspace_query(const gswa_desc* desc, int32_t mlp_hidden, size_t* saved_bytes, size_t* fwd_scratch_bytes,
                              size_t* infer_scratch_bytes, size_t* bwd_scratch_bytes);
int gswa_astl_forward(const gswa_desc* desc, int32_t mlp_hidden, const void* x, const gswa_astl_params* params, void* y,
                      void* saved, void* scratch, size_t scratch_bytes, void* cuda_stream);
int gswa_astl_backward(const gswa_desc* desc, int32_t mlp_hidden, const void* x, const gswa_astl_params* params,
                       const void* saved, const void* dy, void* dx, const gswa_astl_grads* grads, void* scratch,
                       size_t scratch_bytes, void* cuda_stream);

/* One training step on HOST buffers: copies x, the parameters and dy to the device arena, runs
 * gswa_forward + gswa_backward, copies y, dx and the parameter gradients back, and waits for the
 * stream.  All tensor pointers are HOST pointers (pinned memory makes the copies asynchronous);
 * `arena` is a DEVICE buffer of at least *arena_bytes_needed bytes (call with arena == NULL to get
 * the size: returns GSWA_ERR_WORKSPACE and fills arena_bytes_needed). b_qkv / b_proj may be NULL. */
int gswa_step_host(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                   const void* b_proj, const void* bias_table, const void* dy, void* y, void* dx, float* dw_qkv,
                   float* db_qkv, float* dw_proj, float* db_proj, float* dbias_table, void* arena,
                   size_t arena_bytes, size_t* arena_bytes_needed, void* cuda_stream);

/* Device-side status of the last gswa_forward / gswa_backward that used `scratch` (the paper has no
 * counterpart).  The tensor-core kernels hand tiles between warps through barriers whose waits are
 * bounded; a wait that runs out makes the kernel return early and set a word at the start of
 * `scratch`.  This call waits for `cuda_stream`, reads the word and returns GSWA_OK or
 * GSWA_ERR_DEVICE (outputs are then invalid; the context stays usable). */
int gswa_scratch_status(const gswa_desc* desc, const void* scratch, void* cuda_stream);

/* Per-launch timing for benchmarks (the paper has no counterpart).  While enabled, every kernel the
 * library launches is bracketed by a CUDA event pair on its stream.  gswa_profile_read waits for the
 * recorded launches, writes up to max_records entries (names: max_records x 32 chars, NUL-terminated;
 * ms: milliseconds), stores the number written in *count and clears the list.  Host pointers. */
int gswa_profile_enable(int on);
int gswa_profile_read(int32_t max_records, char* names, float* ms, int32_t* count);

/* Number of kernels this library has launched in the calling process since load (monotonic). */
uint64_t gswa_launch_count(void);

/* Text for a gswa_status; for GSWA_ERR_CUDA the text of the last CUDA error seen by this thread. */
const char* gswa_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* GSWA_H_ */
