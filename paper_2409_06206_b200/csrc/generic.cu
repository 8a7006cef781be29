// Shape-generic GSWA kernels on CUDA cores: f32 or bf16 storage, f32 arithmetic (plain FMA, no
// tensor-core rounding), any window size with M*M <= 144 and head dim <= 64.  This is the path
// for float32 layers and for shapes the bf16 tensor-core kernels do not cover.
//
//   forward : qkv = x W_qkv^T + b (q scaled)            gemm_generic            (Eq. 6 projections)
//             per (window, head) softmax attention      attn_fwd_generic        (Eq. 6 Attn, bias, mask)
//             y = A W_proj^T + b                        gemm_generic            (Eq. 7)
//   backward: dA = dy W_proj, dW_proj, db_proj          gemm_generic / colsum
//             recompute P, dq dk dv, d(table)           attn_bwd_generic
//             dx = dqkv W_qkv, dW_qkv, db_qkv           gemm_generic / colsum
#include "generic_core.cuh"

namespace gswa {
using namespace generic;
namespace {

__global__ void index_maps_kernel(int H, int W, int M, int s, int32_t* win, int32_t* slot, int32_t* region,
                                  int32_t* token_of, int32_t* rel) {
  const int N = M * M;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < H * W) {
    const int i = idx / W, j = idx % W;
    int w, t, r;
    token_to_slot(H, W, M, s, i, j, &w, &t, &r);
    if (win) win[idx] = w;
    if (slot) slot[idx] = t;
    if (region) region[idx] = r;
    if (token_of) {
      int ii, jj, rr;
      slot_to_token(H, W, M, s, idx / N, idx % N, &ii, &jj, &rr);
      token_of[idx] = ii * W + jj;
    }
  }
  if (rel && idx < N * N) rel[idx] = rel_row(M, idx / N, idx % N);
}

AttnGeom attn_geom(const Plan& p) {
  return AttnGeom{p.H, p.W, p.nh, p.dqk, p.dv, p.M, p.N, p.Cq, p.Cv, p.Cqkv};
}

template <typename T>
int forward_t(const Plan& p, const T* x, const T* w_qkv, const T* b_qkv, const T* w_proj, const T* b_proj,
              const T* table, T* y, char* saved, cudaStream_t st, const T* resid) {
  T* qkv = reinterpret_cast<T*>(saved + p.off_qkv);
  T* A = reinterpret_cast<T*>(saved + p.off_A);
  float* L = reinterpret_cast<float*>(saved + p.off_L);
  const int C = p.C;
  const float scale = 1.0f / sqrtf((float)p.dqk);
  const size_t smem = generic_attn_fwd_smem(p);
  if (cudaFuncSetAttribute(attn_fwd_generic<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  int rc = launch_gemm<T, T, T>(x, C, 1, w_qkv, 1, C, qkv, p.Cqkv, b_qkv, p.T, p.Cqkv, C, scale, p.Cq, st);
  if (rc) return rc;
  { KernelScope ks_("attn_fwd_generic", st); attn_fwd_generic<T><<<dim3(p.B * p.nW, p.nh), 128, smem, st>>>(attn_geom(p), head_shifts(p), qkv, table, A, L); }
  if ((rc = check_launch())) return rc;
  return launch_gemm<T, T, T>(A, p.Cv, 1, w_proj, 1, p.Cv, y, C, b_proj, p.T, C, p.Cv, 1.f, 0, st, 0, resid, C);
}

template <typename T>
int backward_t(const Plan& p, const T* x, const T* w_qkv, const T* w_proj, const T* table, const char* saved,
               const T* dy, T* dx, float* dw_qkv, float* db_qkv, float* dw_proj, float* db_proj, float* dtable,
               char* scratch, cudaStream_t st) {
  const T* qkv = reinterpret_cast<const T*>(saved + p.off_qkv);
  const T* A = reinterpret_cast<const T*>(saved + p.off_A);
  const float* L = reinterpret_cast<const float*>(saved + p.off_L);
  const int C = p.C, Cv = p.Cv, Q = p.Cqkv;
  T* dA = reinterpret_cast<T*>(scratch);
  T* dqkv = dA + p.T * Cv;
  const float scale = 1.0f / sqrtf((float)p.dqk);
  int rc;
  // every fallible host-side step comes before the first launch
  const size_t smem = generic_attn_bwd_smem(p);
  if (cudaFuncSetAttribute(attn_bwd_generic<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  // dA = dy W_proj
  if ((rc = launch_gemm<T, T, T>(dy, C, 1, w_proj, Cv, 1, dA, Cv, nullptr, p.T, Cv, C, 1.f, 0, st))) return rc;
  if (dw_proj && (rc = launch_gemm_tn<T, T>(dy, C, C, A, Cv, Cv, p.T, dw_proj, st))) return rc;
  if (db_proj && (rc = launch_colsum<T>(dy, p.T, C, C, db_proj, st))) return rc;
  { KernelScope ks_("attn_bwd_generic", st); attn_bwd_generic<T><<<dim3(p.B * p.nW, p.nh), 256, smem, st>>>(attn_geom(p), head_shifts(p), scale, qkv, table, A, L, dA, dqkv,
                                                                 dtable); }
  if ((rc = check_launch())) return rc;
  if (dx && (rc = launch_gemm<T, T, T>(dqkv, Q, 1, w_qkv, C, 1, dx, C, nullptr, p.T, C, Q, 1.f, 0, st)))
    return rc;
  if (dw_qkv && (rc = launch_gemm_tn<T, T>(dqkv, Q, Q, x, C, C, p.T, dw_qkv, st))) return rc;
  if (db_qkv && (rc = launch_colsum<T>(dqkv, p.T, Q, Q, db_qkv, st))) return rc;
  return GSWA_OK;
}

}  // namespace

size_t generic_attn_fwd_smem(const Plan& p) {
  return sizeof(float) * ((size_t)2 * p.N * (p.dqk + 1) + (size_t)p.N * (p.dv + 1) + (size_t)p.N * (p.N + 1)) + 8 * (size_t)p.N;
}
size_t generic_attn_bwd_smem(const Plan& p) {
  const size_t nrel = (size_t)(2 * p.M - 1) * (2 * p.M - 1);
  return sizeof(float) * ((size_t)2 * p.N * (p.dqk + 1) + (size_t)2 * p.N * (p.dv + 1) + (size_t)p.N * (p.N + 1) + 2 * p.N + nrel) +
         8 * (size_t)p.N;
}

int generic_forward(const Plan& p, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                    const void* b_proj, const void* table, void* y, void* saved, cudaStream_t st, const void* resid) {
  if (p.dtype == GSWA_F32)
    return forward_t<float>(p, (const float*)x, (const float*)w_qkv, (const float*)b_qkv, (const float*)w_proj,
                            (const float*)b_proj, (const float*)table, (float*)y, (char*)saved, st, (const float*)resid);
  using bf = __nv_bfloat16;
  return forward_t<bf>(p, (const bf*)x, (const bf*)w_qkv, (const bf*)b_qkv, (const bf*)w_proj, (const bf*)b_proj,
                       (const bf*)table, (bf*)y, (char*)saved, st, (const bf*)resid);
}

int generic_backward(const Plan& p, const void* x, const void* w_qkv, const void* w_proj, const void* table,
                     const void* saved, const void* dy, void* dx, float* dw_qkv, float* db_qkv, float* dw_proj,
                     float* db_proj, float* dtable, void* scratch, cudaStream_t st) {
  if (p.dtype == GSWA_F32)
    return backward_t<float>(p, (const float*)x, (const float*)w_qkv, (const float*)w_proj, (const float*)table,
                             (const char*)saved, (const float*)dy, (float*)dx, dw_qkv, db_qkv, dw_proj, db_proj,
                             dtable, (char*)scratch, st);
  using bf = __nv_bfloat16;
  return backward_t<bf>(p, (const bf*)x, (const bf*)w_qkv, (const bf*)w_proj, (const bf*)table, (const char*)saved,
                        (const bf*)dy, (bf*)dx, dw_qkv, db_qkv, dw_proj, db_proj, dtable, (char*)scratch, st);
}

// Zeroes up to six float buffers with one launch (the parameter gradients of a backward call: six separate
// memsets cost six stream operations in front of the first kernel).
struct ZeroJobs {
  float* p[6];
  long long n[6];
};
__global__ void zero_kernel(const __grid_constant__ ZeroJobs J) {
  float* p = J.p[blockIdx.y];
  const long long n = J.n[blockIdx.y];
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) p[i] = 0.f;
}
int launch_zero(float* const* ptrs, const long long* counts, int nbuf, cudaStream_t st) {
  ZeroJobs J{};
  int k = 0;
  for (int i = 0; i < nbuf && k < 6; ++i)
    if (ptrs[i] != nullptr && counts[i] > 0) { J.p[k] = ptrs[i]; J.n[k] = counts[i]; ++k; }
  if (k == 0) return GSWA_OK;
  { KernelScope ks_("zero_grads", st); zero_kernel<<<dim3(48, k), 256, 0, st>>>(J); }
  return check_launch();
}

int launch_colsum_bf16(const __nv_bfloat16* G, long long rows, int cols, long long ld, float* out, cudaStream_t st) {
  return launch_colsum<__nv_bfloat16>(G, rows, cols, ld, out, st);
}

__global__ void batch_window_ids_kernel(int B, int H, int W, int M, int s, int32_t* win_id) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)B * H * W) return;
  const int b = (int)(idx / (H * W)), rem = (int)(idx % (H * W));
  int w, t, r;
  token_to_slot(H, W, M, s, rem / W, rem % W, &w, &t, &r);
  win_id[idx] = b * (H / M) * (W / M) + w;
}

int launch_batch_window_ids(const Plan& p, int group, int32_t* win_id, cudaStream_t st) {
  if (p.T == 0) return GSWA_OK;
  { KernelScope ks_("batch_window_ids", st);
    batch_window_ids_kernel<<<(unsigned)((p.T + 255) / 256), 256, 0, st>>>(p.B, p.H, p.W, p.M, p.gs[group], win_id); }
  return check_launch();
}

// The give-up path of a bounded wait, on purpose: a barrier that expects one arrival and never gets it.  The poll
// limit is small, the kernel returns normally, and the only trace is the error word.
__global__ void wait_timeout_kernel(int* err) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"((uint32_t)__cvta_generic_to_shared(&bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bool done = false;
    for (int i = 0; i < 2000 && !done; ++i) {
      uint32_t ok;
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.b32 %0, 1, 0, p;\n\t}\n"
                   : "=r"(ok)
                   : "r"((uint32_t)__cvta_generic_to_shared(&bar))
                   : "memory");
      done = ok != 0;
      if (!done) __nanosleep(32);
    }
    if (!done) atomicExch(err, 1);
  }
}

int launch_wait_timeout(int* err, cudaStream_t st) {
  { KernelScope ks_("wait_timeout", st); wait_timeout_kernel<<<1, 32, 0, st>>>(err); }
  return check_launch();
}

int launch_index_maps(const Plan& p, int group, int32_t* win, int32_t* slot, int32_t* region, int32_t* token_of,
                      int32_t* rel, cudaStream_t st) {
  const int n = max(p.H * p.W, p.N * p.N);
  { KernelScope ks_("index_maps", st); index_maps_kernel<<<(n + 255) / 256, 256, 0, st>>>(p.H, p.W, p.M, p.gs[group], win, slot, region, token_of, rel); }
  return check_launch();
}

}  // namespace gswa
