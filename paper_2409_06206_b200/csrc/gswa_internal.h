// Internal declarations shared by the host planner and the kernel files of libgswa.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "gswa.h"

namespace gswa {

constexpr int kMaxGroups = 16;
constexpr int kMaxHeads = 64;

// Validated, flattened copy of a gswa_desc plus derived sizes.
struct Plan {
  int B, H, W, C, nh, d, M, N, G;
  int dqk, dv;                 // per-head widths of q,k and of v (d unless the descriptor narrows them)
  int Cq, Cv, Cqkv;            // heads*dqk, heads*dv, 2*Cq + Cv (rows of w_qkv)
  int nWh, nWw, nW;            // windows per image: rows, cols, total
  long long T;                 // tokens = B*H*W
  int dtype;
  uint32_t flags;
  int gh[kMaxGroups], gs[kMaxGroups], gh0[kMaxGroups];  // heads, shift, first head of each group
  int esize;                   // bytes per element of dtype
  int fast;                    // 1 = bf16 tensor-core path, 0 = generic CUDA-core path
  // fast-path geometry
  int dp;                      // head dim padded to an MMA-friendly width (16 or 32)
  int Cp;                      // C padded to a multiple of 64 (K of the GEMMs that read the caller's rows)
  int Ap;                      // heads * dp: row length of the padded attention output
  // byte offsets inside `saved`
  size_t off_qkv, off_A, off_L, off_bimg, saved_bytes;   // off_bimg: weight images of the backward GEMMs (built by the forward call)
  size_t fwd_scratch, infer_scratch, bwd_scratch;
};

// Per-head shift table passed by value to the attention kernels.
struct HeadShifts {
  int8_t s[kMaxHeads];
};

int make_plan(const gswa_desc* desc, Plan* plan);
// One GSWA forward / backward for a validated plan: pointer checks, then the tensor-core or the shape-generic path.
// `resid` ([B,H,W,C] or nullptr) is added to y in the output projection's epilogue (skip connection of Eq. 4).
int forward_impl(const Plan& p, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj, const void* b_proj,
                 const void* bias_table, void* y, void* saved, void* scratch, size_t scratch_bytes, cudaStream_t st,
                 const void* resid);
int backward_impl(const Plan& p, const void* x, const void* w_qkv, const void* w_proj, const void* bias_table,
                  const void* saved, const void* dy, void* dx, float* dw_qkv, float* db_qkv, float* dw_proj, float* db_proj,
                  float* dbias_table, void* scratch, size_t scratch_bytes, cudaStream_t st);
int check_launch();  // GSWA_OK or GSWA_ERR_CUDA (records the CUDA error text)
int launch_zero(float* const* ptrs, const long long* counts, int nbuf, cudaStream_t st);   // one launch zeroes them all
int device_sm_count();     // multiprocessors of the current device (148 if the query fails)
bool profiling_enabled();  // per-kernel event timing is on (kernels are then kept on one stream)

// Wraps one kernel launch: counts it and, while profiling is enabled, brackets it with a CUDA
// event pair on the launching stream.  Usage: { KernelScope k("name", st); kernel<<<...>>>(...); }
struct KernelScope {
  KernelScope(const char* name, cudaStream_t st);
  ~KernelScope();
  cudaStream_t st;
  int slot;
};

// ---- generic CUDA-core path (any shape the descriptor allows, f32 or bf16 storage, f32 arithmetic)
int generic_forward(const Plan& p, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                    const void* b_proj, const void* table, void* y, void* saved, cudaStream_t st,
                    const void* resid = nullptr);   // resid [B,H,W,C] or nullptr: added to y (skip connection)
int generic_backward(const Plan& p, const void* x, const void* w_qkv, const void* w_proj, const void* table,
                     const void* saved, const void* dy, void* dx, float* dw_qkv, float* db_qkv, float* dw_proj,
                     float* db_proj, float* dtable, void* scratch, cudaStream_t st);
size_t generic_attn_fwd_smem(const Plan& p);   // dynamic shared memory of the generic attention kernels
size_t generic_attn_bwd_smem(const Plan& p);
int launch_colsum_bf16(const __nv_bfloat16* G, long long rows, int cols, long long ld, float* out, cudaStream_t st);
int launch_index_maps(const Plan& p, int group, int32_t* win, int32_t* slot, int32_t* region, int32_t* token_of,
                      int32_t* rel, cudaStream_t st);
// win_id[B*H*W] = b*nW + window of every token (the per-image map of launch_index_maps repeated over the batch)
int launch_batch_window_ids(const Plan& p, int group, int32_t* win_id, cudaStream_t st);
// A one-block kernel that waits on a barrier nobody arrives on, gives up after a few thousand polls and sets the
// device error word at `err` (the path every bounded wait of the tensor-core kernels takes when it runs out).
int launch_wait_timeout(int* err, cudaStream_t st);

}  // namespace gswa
