// Data layout of the bf16 tensor-core path (window 8x8, head dim <= 32) and the launch interfaces
// of its kernels.
//
// "Tiled" buffers hold one contiguous block per (group, window, head, kind): [64 slots][DP] bf16 with
// the head dim padded to DP (16 or 32).  Windows of one group are numbered b*nW + w.  The QKV
// projection writes q,k,v straight into this layout (cyclic shift + window partition happen in its
// epilogue addressing), so the attention kernels read contiguous, 16-byte aligned tiles:
//   qkv tiles of group g : base + qkv_off[g] + window*(gh*3*64*DP) + ((hl*3 + kind)*64 + slot)*DP + c
//   dO  tiles of group g : base + do_off[g]  + window*(gh*64*DP)   + (hl*64 + slot)*DP + c
//   L   tiles of group g : base + l_off[g]   + window*(gh*64)      +  hl*64 + slot            (float)
// Inside a [64][DP] block the 16-byte chunks of a row are permuted (tile_off below) so that the block
// is at the same time the shared-memory image the attention kernels read with ldmatrix: the GEMM
// epilogue builds the image in shared memory and ships it with one bulk copy, the attention kernels
// fetch it with plain linear copies.
// "Token-major" buffers hold rows in original token order with the head dim padded like the tiles:
// attention output A[T, Ap], Ap = heads * DP, and dqkv[T, 3*Ap] (q | k | v, head-major inside each);
// the attention epilogues undo partition and shift when they store into them.  Their row pitches are
// multiples of 16 bytes, so the GEMMs that consume them fetch 64-column x 128-row (or 64-row) boxes
// with TMA, which also applies the 128-byte swizzle the tensor core expects.  Pad columns hold zeros,
// except A[:, d] of head 0 (when d < DP), which holds ones: multiplied with dy it yields the bias
// gradient of the output projection for free.
#pragma once

#include <cuda.h>

#include "gswa_internal.h"

namespace gswa {

constexpr int kMaxUnits = 8;   // (group, head range) work units per launch

// Byte offset of 16-byte chunk `chunk` of row `row` inside a [64][DP] bf16 tile image: eight
// consecutive rows map to eight different 16-byte bank groups (ldmatrix and 16-byte stores of
// consecutive rows are conflict free).
template <int DP>
__host__ __device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  constexpr int CH = DP / 8;                // chunks per row (4 or 2)
  return (uint32_t)(row * (DP * 2) + ((chunk ^ ((row / (8 / CH)) % CH)) << 4));
}

struct FastGeom {
  int B, H, W, C, nh, d, dp, G;
  int nW, nWw, nWh;
  long long T, n_windows;          // n_windows = B*nW
  int gh[kMaxGroups], gs[kMaxGroups], gh0[kMaxGroups];
  long long qkv_off[kMaxGroups], do_off[kMaxGroups], l_off[kMaxGroups];   // element offsets
};

// ---- window GEMM: rows gathered in window order from a packed [T, lda] source, output to tiles
struct GWUnit {
  const __nv_bfloat16* A;      // source rows (x or dy), pitch lda elements, `kvalid` valid columns
  int lda, kvalid;
  int H, W, s, nW, nWw;
  long long n_windows;
  const unsigned char* Bimg;   // weight image: [KP/64 atoms][NT rows][128 B], rows swizzled
  const float* bias;           // [NT] or nullptr
  __nv_bfloat16* out;          // tile base of this unit (already offset to its first block)
  long long win_stride;        // elements between consecutive windows
  int nchunks, cw;             // NT = nchunks*cw accumulator columns; cw multiple of 16 and of DP
  int q_every3;                // 1: blocks with index % 3 == 0 are scaled by qscale
  float qscale;
  int a16;                     // 16-byte copies possible for: 0 no row, 1 rows of even tokens, 2 all rows of A (set by launch_gw)
  int ones_col;                // 1: the loaders put a one into K column `kvalid` (the weight image carries the bias in that row)
};
struct GWLaunch {
  GWUnit u[kMaxUnits];
  int* err;
  int nslots;                  // ring slots of 16 KB (set by launch_gw) / quarter-tile stages (set by launch_gwt)
  int cta0[kMaxUnits + 1];     // first CTA of every unit (set by launch_gw)
};

// ---- token GEMM: A rows in token order, fetched by TMA from a padded [rows, K] buffer; packed rows out
struct GTSplit {
  const unsigned char* Bimg;   // [KP/64 atoms][NB rows][128 B]
  const float* bias;           // [NB] or nullptr
  int col0, ncols;             // output columns [col0, col0+ncols) of each row
};
struct GTLaunch {
  CUtensorMap tmA;             // [rows, K] bf16, box 64 columns x 128 rows, 128-byte swizzle
  int natoms;                  // K atoms of 64 columns
  long long rows;
  __nv_bfloat16* out;
  int ldo;
  const __nv_bfloat16* resid;  // or nullptr: packed rows [rows, ldo] added to the result (skip connection)
  int NB;                      // accumulator columns per CTA (multiple of 32, <= 256)
  int nstages;
  int stream_b;                // 1: the weight image travels through the ring with the A atoms (see gt_kernel)
  GTSplit s[kMaxUnits];
  int* err;
};

// ---- reduction GEMM: out[m, n] += sum_t L[t, m] R[t, n].  One operand is a padded token-major buffer
// fetched by TMA (box 64 columns x 64 rows), the other a packed caller tensor fetched by 8-byte copies.
//   tma_is_L = 1 (dW_qkv): L = dqkv[T, 3*Ap], R = x[T, C] plus a column of ones at index C
//   tma_is_L = 0 (dW_proj): L = dy[T, C],      R = A[T, Ap] (whose column d holds ones when d < DP)
// Padded indices (kind, head, c) map to kind*C + head*d + c; c >= d is dropped.
struct GRLaunch {
  CUtensorMap tm;
  int tma_is_L;
  const __nv_bfloat16* P;      // the copy-fed operand, [rows, ldp] with pvalid valid columns
  int ldp, pvalid;
  int p16;                     // 16-byte copies possible for: 0 no row, 1 even rows, 2 all rows of P (set by launch_gr)
  int Ap, dp, d, C;
  int M;                       // extent of the M index space (3*Ap or C)
  long long rows;
  int NP;                      // accumulator columns (multiple of 64)
  int nsplit;                  // token splits
  int mbpc;                    // M blocks of 128 handled by one CTA (1 or 2)
  int nstages;                 // depth of the TMA ring (set by launch_gr)
  float* out;                  // float, accumulated with atomics: [3C, C] or [C, C]
  float* colsum;               // or nullptr: dB[m] = sum_t L[t, m]
  int* err;
};

int launch_gw(const GWLaunch& L, int nunits, int Cp, int dp, cudaStream_t st, const char* name);
// The same GEMM with the A operand in tensor memory (fast_gemm_tm.cu): rows arrive by bulk copies of whole window
// rows, which needs every piece of a window row to start and end on a 16-byte boundary (gwt_usable).
bool gwt_usable(const void* A, int lda, int H, int W, const int* shifts, int nshifts);
int gwt_heads_per_unit(int Cp, int dp, int C, int nb, int cap);   // nb = output blocks of dp columns per head (3: q,k,v; 1: dO)
int launch_gwt(const GWLaunch& L, int nunits, int Cp, int dp, cudaStream_t st, const char* name);

// ---- fused forward: QKV projection of a window pair on the tensor core, its q,k,v tiles handed to the
// attention warps of the same CTA through shared memory (and, for training, shipped to `qkv_out`).
struct FWUnit {
  const __nv_bfloat16* X;      // x, pitch lda elements, kvalid valid columns
  int lda, kvalid;
  int H, W, s, nW, nWw;
  long long n_windows;
  const unsigned char* Bimg;   // QKV weight image of this unit's heads: [KP/64 atoms][NT rows][128 B]
  const float* bias;           // [NT] or nullptr
  float qscale;                // d^-1/2 * log2(e), applied to the q blocks
  int h0, nheads;              // first head (global index), heads in this unit
  __nv_bfloat16* qkv_out;      // tile image of this unit's first block in window 0, or nullptr (inference)
  long long qkv_wstride;       // elements between consecutive windows
  float* lt;                   // row log-sum-exp tiles of this unit in window 0, or nullptr
  long long l_wstride;
};
struct FWLaunch {
  FWUnit u[kMaxUnits];
  FastGeom geo;
  const __nv_bfloat16* table;  // [(2M-1)^2, nh]
  __nv_bfloat16* A;            // [T, Ap] out
  int* err;
  int nslots;                  // ring slots of 16 KB (set by launch_fw)
};
// Shared memory the fused kernel needs for units of at most `maxheads` heads (0 if it cannot run).
size_t fw_smem_bytes(int Cp, int dp, int maxheads, int* nslots);
int launch_fw(const FWLaunch& L, int nunits, int Cp, int dp, cudaStream_t st);
int launch_gt(const GTLaunch& L, int nsplits, cudaStream_t st, const char* name);
int launch_gr(const GRLaunch& L, cudaStream_t st, const char* name);
// Tensor map of a padded token-major bf16 buffer [rows, cols]: box 64 columns x box_rows rows, 128-byte swizzle.
int make_tmap(CUtensorMap* tm, const void* base, long long rows, int cols, int box_rows);
// Tensor map of a padded token-major bf16 buffer [B*H image rows, W, cols] for stores of a block of
// box_h x box_w tokens x dp columns.  Shared-memory side: rows of dp elements in box order, either with
// the tile_off swizzle (8 x 8 boxes: the [64][dp] tile image) or unswizzled.
int make_tmap_window(CUtensorMap* tm, const void* base, long long img_rows, int W, int cols, int dp, int box_w, int box_h,
                     bool swizzled);

// Weight images (shared-memory images of the B operands, built once per call by a small kernel).
enum PrepMode { PREP_QKV = 0, PREP_PROJ_T = 1, PREP_PROJ = 2, PREP_QKV_T = 3 };
struct PrepJob {
  int mode;
  const __nv_bfloat16* W;      // source weight
  const __nv_bfloat16* b;      // source bias or nullptr
  unsigned char* img;
  float* bias_out;             // or nullptr
  int C, d, dp, h0, nheads;    // head range for the per-head modes
  int n0, NT, KP;              // first output row (PREP_PROJ / PREP_QKV_T), rows, padded K
  int Ap;                      // heads * dp: K of PREP_PROJ / PREP_QKV_T runs over padded (kind, head, c) indices
  int fold_bias;               // PREP_QKV: write the bias into image row k == C (needs C < KP) instead of bias_out
};
int launch_prep(const PrepJob* jobs, int njobs, cudaStream_t st, int* err_word = nullptr);   // err_word: 64 ints zeroed by the same launch

// ---- attention (mma.sync m16n8k16, softmax in registers)
struct AttnUnit {
  int g, h0, nheads;           // group, first head (global index), heads in this unit
  int s;
  long long qkv_off, do_off, l_off;      // element offsets of the unit's first block inside window 0
  long long qkv_wstride, do_wstride, l_wstride;
};
struct AttnLaunch {
  CUtensorMap tm_out;          // window-block stores into dqkv (tcgen05 backward only)
  CUtensorMap tm_wrap[4];      // the four pieces of a window that wraps around the image edge (shift wrap_s):
                               // [2 * (lower rows) + (right columns)], boxes of (8-s | s) x (8-s | s) tokens
  int wrap_s;                  // shift the pieces were cut for (an even shift of some unit), or 0
  FastGeom geo;
  AttnUnit u[kMaxUnits];
  int nunits;
  const __nv_bfloat16* qkv;    // tile base
  const __nv_bfloat16* table;  // [(2M-1)^2, nh]
  __nv_bfloat16* A;            // fwd: [T, Ap] out
  float* Lt;                   // L tiles (fwd: out or nullptr; bwd: in)
  const __nv_bfloat16* dO;     // bwd: dO tiles
  __nv_bfloat16* dqkv;         // bwd: [T, 3*Ap] out
  float* dtable;               // bwd: [(2M-1)^2, nh] float, atomics; or nullptr
  int* err;                    // device error word (set when a bounded wait gives up)
  float scale;
};
int launch_attn_fwd(const AttnLaunch& L, cudaStream_t st);
int launch_attn_bwd(const AttnLaunch& L, cudaStream_t st);
// Backward on tcgen05 (units of one head only; GSWA_ERR_UNSUPPORTED otherwise).
int launch_attn_bwd_tc(const AttnLaunch& L, cudaStream_t st);

// Index maps computed by the routines of the tensor-core attention kernels (window 8): win_id[B*H*W] window number
// b*nW + w of every token in the frame shifted by s, slot[H*W], region[H*W], rel[64*64]; any pointer may be null.
int launch_fast_index_maps(const FastGeom& g, int s, int32_t* win_id, int32_t* slot, int32_t* region, int32_t* rel,
                           cudaStream_t st);
int fast_index_maps(const Plan& p, int group, int32_t* win_id, int32_t* slot, int32_t* region, int32_t* rel, cudaStream_t st);

// ---- orchestration
bool fast_path_ok(const Plan& p);
void fast_plan_sizes(Plan* p);
int fast_forward(const Plan& p, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                 const void* b_proj, const void* table, void* y, void* saved, void* scratch, bool want_L,
                 cudaStream_t st, const void* resid = nullptr);   // resid [B,H,W,C] or nullptr: added to y
int fast_backward(const Plan& p, const void* x, const void* w_qkv, const void* w_proj, const void* table,
                  const void* saved, const void* dy, void* dx, float* dw_qkv, float* db_qkv, float* dw_proj,
                  float* db_proj, float* dtable, void* scratch, cudaStream_t st);

}  // namespace gswa
