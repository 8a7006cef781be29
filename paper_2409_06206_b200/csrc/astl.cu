// The layer around GSWA (Sec. "Agile Swin Transformer Block", Eq. 4 and Eq. 5):
//     X1 = GSWA(LN(X)) + X,      X2 = MLP(LN(X1)) + X1
// and the channel-sliced, cascaded form of the attention (Eq. 6 read literally, Eq. 8).
//
//   forward : LayerNorm (one warp per token row, statistics kept for the backward pass)
//             GSWA on the normalised rows, the skip connection added in the output projection's epilogue
//             LayerNorm, FC1 + GELU, FC2 + skip (CUDA-core GEMMs with fused epilogues)
//   backward: the reverse; each LayerNorm backward kernel also adds the gradient that arrives over the skip
//             connection and reduces the scale / shift gradients per block before its atomics.
// The attention itself runs on whichever GSWA path the layer description selects (tensor-core or shape-generic).
#include "generic_core.cuh"

namespace gswa {
using namespace generic;
namespace {

constexpr float kLnEps = 1e-5f;

// ------------------------------------------------------------------------------------------
// LayerNorm over the C channels of each token: y = (x - mean) * rstd * g + b; stats[row] = (mean, rstd).
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) ln_fwd_kernel(const T* __restrict__ x, const T* __restrict__ g, const T* __restrict__ b,
                                                     T* __restrict__ y, float2* __restrict__ stats, long long rows, int C) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (long long row = (long long)blockIdx.x * 8 + warp; row < rows; row += (long long)gridDim.x * 8) {
    const T* xr = x + row * C;
    float s = 0.f;
    for (int c = lane; c < C; c += 32) s += ldf(xr + c);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mean = s / (float)C;
    float v = 0.f;
    for (int c = lane; c < C; c += 32) {
      const float d = ldf(xr + c) - mean;
      v = fmaf(d, d, v);
    }
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const float rstd = rsqrtf(v / (float)C + kLnEps);
    for (int c = lane; c < C; c += 32) stf(y + row * C + c, (ldf(xr + c) - mean) * rstd * ldf(g + c) + ldf(b + c));
    if (lane == 0 && stats != nullptr) stats[row] = make_float2(mean, rstd);
  }
}

// Backward of the LayerNorm plus the skip connection:
//   dx = dskip + rstd * (dxhat - mean_c(dxhat) - xhat * mean_c(dxhat * xhat)),  dxhat = dy * g,
//   dg += sum_rows dy * xhat,  db += sum_rows dy      (per block in shared memory first, then one atomic per channel)
template <typename T>
__global__ void __launch_bounds__(256) ln_bwd_kernel(const T* __restrict__ x, const float2* __restrict__ stats,
                                                     const T* __restrict__ g, const T* __restrict__ dy,
                                                     const T* __restrict__ dskip, T* __restrict__ dx, float* __restrict__ dg,
                                                     float* __restrict__ db, long long rows, int C) {
  extern __shared__ float sm[];
  float* sdg = sm;
  float* sdb = sm + C;
  for (int c = threadIdx.x; c < 2 * C; c += blockDim.x) sm[c] = 0.f;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (long long row = (long long)blockIdx.x * 8 + warp; row < rows; row += (long long)gridDim.x * 8) {
    const float2 st = stats[row];
    const T* xr = x + row * C;
    const T* dyr = dy + row * C;
    float s1 = 0.f, s2 = 0.f;
    for (int c = lane; c < C; c += 32) {
      const float xh = (ldf(xr + c) - st.x) * st.y, d = ldf(dyr + c), dxh = d * ldf(g + c);
      s1 += dxh;
      s2 = fmaf(dxh, xh, s2);
      atomicAdd(sdg + c, d * xh);
      atomicAdd(sdb + c, d);
    }
    for (int o = 16; o; o >>= 1) {
      s1 += __shfl_xor_sync(0xffffffffu, s1, o);
      s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    const float m1 = s1 / (float)C, m2 = s2 / (float)C;
    for (int c = lane; c < C; c += 32) {
      const float xh = (ldf(xr + c) - st.x) * st.y, dxh = ldf(dyr + c) * ldf(g + c);
      float v = st.y * (dxh - m1 - xh * m2);
      if (dskip != nullptr) v += ldf(dskip + row * C + c);
      stf(dx + row * C + c, v);
    }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    atomicAdd(dg + c, sdg[c]);
    atomicAdd(db + c, sdb[c]);
  }
}

// a = GELU(h) and, in place, d = d * GELU'(h)   (exact Gaussian-CDF form)
template <typename T>
__global__ void __launch_bounds__(256) gelu_bwd_kernel(const T* __restrict__ h, T* __restrict__ d, T* __restrict__ a, long long n) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const float v = ldf(h + i);
    const float cdf = 0.5f * (1.f + erff(v * 0.70710678118654752f));
    stf(a + i, v * cdf);
    stf(d + i, ldf(d + i) * (cdf + v * 0.3989422804014327f * expf(-0.5f * v * v)));
  }
}

template <typename T>
int launch_ln_fwd(const T* x, const T* g, const T* b, T* y, float2* stats, long long rows, int C, cudaStream_t st) {
  { KernelScope ks_("ln_fwd", st); ln_fwd_kernel<T><<<grid_for(rows, 8), 256, 0, st>>>(x, g, b, y, stats, rows, C); }
  return check_launch();
}
template <typename T>
int launch_ln_bwd(const T* x, const float2* stats, const T* g, const T* dy, const T* dskip, T* dx, float* dg, float* db,
                  long long rows, int C, cudaStream_t st) {
  const int grid = grid_for(rows, 8 * 32);       // about 32 rows per warp: few atomics per block
  { KernelScope ks_("ln_bwd", st);
    ln_bwd_kernel<T><<<grid, 256, 2 * C * sizeof(float), st>>>(x, stats, g, dy, dskip, dx, dg, db, rows, C); }
  return check_launch();
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Byte offsets of the layer's buffers.  `saved` carries forward -> backward: the normalised input of the attention,
// the statistics of both LayerNorms, the attention's own carry and, with the MLP, X1 and the pre-activation of FC1.
struct AstlLayout {
  size_t s_xn, s_st1, s_attn, s_x1, s_st2, s_h, saved_total;
  size_t f_attn, f_xn2, fwd_total;
  size_t b_attn, b_dxn, b_dx1, b_xn2, b_a, b_dh, b_dxn2, bwd_total;
};

AstlLayout astl_layout(const Plan& p, int hidden) {
  AstlLayout l{};
  const size_t act = align_up((size_t)p.T * p.C * p.esize, 256), st = align_up((size_t)p.T * sizeof(float2), 256);
  const size_t hid = align_up((size_t)p.T * (size_t)hidden * p.esize, 256);
  size_t o = 0;
  l.s_xn = o; o += act;
  l.s_st1 = o; o += st;
  l.s_attn = o; o += align_up(p.saved_bytes, 256);
  if (hidden > 0) {
    l.s_x1 = o; o += act;
    l.s_st2 = o; o += st;
    l.s_h = o; o += hid;
  }
  l.saved_total = o;
  o = 0;
  l.f_attn = o; o += align_up(p.fwd_scratch, 256);        // first: the tensor-core path keeps its error word at the head
  if (hidden > 0) { l.f_xn2 = o; o += act; }
  l.fwd_total = o;
  o = 0;
  l.b_attn = o; o += align_up(p.bwd_scratch, 256);
  l.b_dxn = o; o += act;
  if (hidden > 0) {
    l.b_dx1 = o; o += act;
    l.b_xn2 = o; o += act;
    l.b_a = o; o += hid;
    l.b_dh = o; o += hid;
    l.b_dxn2 = o; o += act;
  }
  l.bwd_total = o;
  return l;
}

template <typename T>
int astl_forward_t(const Plan& p, int hidden, const T* x, const gswa_astl_params& q, T* y, char* saved, char* scratch,
                   cudaStream_t st) {
  const AstlLayout l = astl_layout(p, hidden);
  const int C = p.C;
  T* xn = reinterpret_cast<T*>(saved + l.s_xn);
  float2* st1 = reinterpret_cast<float2*>(saved + l.s_st1);
  int rc;
  if ((rc = launch_ln_fwd<T>(x, (const T*)q.ln1_g, (const T*)q.ln1_b, xn, st1, p.T, C, st))) return rc;
  // X1 = GSWA(LN(X)) + X: the skip connection is the output projection's epilogue
  T* x1 = hidden > 0 ? reinterpret_cast<T*>(saved + l.s_x1) : y;
  if ((rc = forward_impl(p, xn, q.w_qkv, q.b_qkv, q.w_proj, q.b_proj, q.bias_table, x1, saved + l.s_attn,
                         scratch + l.f_attn, p.fwd_scratch, st, x)))
    return rc;
  if (hidden <= 0) return GSWA_OK;
  T* xn2 = reinterpret_cast<T*>(scratch + l.f_xn2);
  float2* st2 = reinterpret_cast<float2*>(saved + l.s_st2);
  T* h = reinterpret_cast<T*>(saved + l.s_h);
  if ((rc = launch_ln_fwd<T>(x1, (const T*)q.ln2_g, (const T*)q.ln2_b, xn2, st2, p.T, C, st))) return rc;
  // h = xn2 W1^T + b1 (kept before the activation: the backward pass needs GELU'(h)); X2 = GELU(h) W2^T + b2 + X1
  if ((rc = launch_gemm<T, T, T>(xn2, C, 1, (const T*)q.w_fc1, 1, C, h, hidden, (const T*)q.b_fc1, p.T, hidden, C, 1.f, 0, st)))
    return rc;
  return launch_gemm<T, T, T>(h, hidden, 1, (const T*)q.w_fc2, 1, hidden, y, C, (const T*)q.b_fc2, p.T, C, hidden, 1.f, 0, st, 0,
                              x1, C, 1);
}

template <typename T>
int astl_backward_t(const Plan& p, int hidden, const T* x, const gswa_astl_params& q, const char* saved, const T* dy, T* dx,
                    const gswa_astl_grads& g, char* scratch, cudaStream_t st) {
  const AstlLayout l = astl_layout(p, hidden);
  const int C = p.C;
  const T* xn = reinterpret_cast<const T*>(saved + l.s_xn);
  const float2* st1 = reinterpret_cast<const float2*>(saved + l.s_st1);
  T* dxn = reinterpret_cast<T*>(scratch + l.b_dxn);
  int rc;
  {
    // the LayerNorm and MLP gradients accumulate with atomics: zero them first (the attention's own are zeroed by its call)
    const bool z = !(p.flags & GSWA_FLAG_ACCUMULATE);
    float* const a[6] = {z ? g.dln1_g : nullptr, z ? g.dln1_b : nullptr, z && hidden > 0 ? g.dln2_g : nullptr,
                         z && hidden > 0 ? g.dln2_b : nullptr, z && hidden > 0 ? g.db_fc1 : nullptr, z && hidden > 0 ? g.db_fc2 : nullptr};
    const long long na[6] = {C, C, C, C, hidden, C};
    if ((rc = launch_zero(a, na, 6, st))) return rc;
    float* const b[2] = {z && hidden > 0 ? g.dw_fc1 : nullptr, z && hidden > 0 ? g.dw_fc2 : nullptr};
    const long long nb[2] = {(long long)hidden * C, (long long)hidden * C};
    if ((rc = launch_zero(b, nb, 2, st))) return rc;
  }
  const T* dx1 = dy;                                      // gradient at X1
  if (hidden > 0) {
    const T* x1 = reinterpret_cast<const T*>(saved + l.s_x1);
    const float2* st2 = reinterpret_cast<const float2*>(saved + l.s_st2);
    const T* h = reinterpret_cast<const T*>(saved + l.s_h);
    T* dx1w = reinterpret_cast<T*>(scratch + l.b_dx1);
    T* xn2 = reinterpret_cast<T*>(scratch + l.b_xn2);
    T* a = reinterpret_cast<T*>(scratch + l.b_a);
    T* dh = reinterpret_cast<T*>(scratch + l.b_dh);
    T* dxn2 = reinterpret_cast<T*>(scratch + l.b_dxn2);
    // da = dy W2, then a = GELU(h) and dh = da * GELU'(h)
    if ((rc = launch_gemm<T, T, T>(dy, C, 1, (const T*)q.w_fc2, hidden, 1, dh, hidden, nullptr, p.T, hidden, C, 1.f, 0, st))) return rc;
    { KernelScope ks_("gelu_bwd", st);
      gelu_bwd_kernel<T><<<grid_for(p.T * hidden, 256 * 8), 256, 0, st>>>(h, dh, a, p.T * hidden); }
    if ((rc = check_launch())) return rc;
    if ((rc = launch_gemm_tn<T, T>(dy, C, C, a, hidden, hidden, p.T, g.dw_fc2, st))) return rc;        // dW2 = dy^T GELU(h)
    if ((rc = launch_colsum<T>(dy, p.T, C, C, g.db_fc2, st))) return rc;
    // xn2 is recomputed (one LayerNorm pass costs less than carrying another activation)
    if ((rc = launch_ln_fwd<T>(x1, (const T*)q.ln2_g, (const T*)q.ln2_b, xn2, nullptr, p.T, C, st))) return rc;
    if ((rc = launch_gemm_tn<T, T>(dh, hidden, hidden, xn2, C, C, p.T, g.dw_fc1, st))) return rc;      // dW1 = dh^T xn2
    if ((rc = launch_colsum<T>(dh, p.T, hidden, hidden, g.db_fc1, st))) return rc;
    if ((rc = launch_gemm<T, T, T>(dh, hidden, 1, (const T*)q.w_fc1, C, 1, dxn2, C, nullptr, p.T, C, hidden, 1.f, 0, st))) return rc;
    // dX1 = dy (skip of Eq. 5) + LayerNorm backward of dxn2
    if ((rc = launch_ln_bwd<T>(x1, st2, (const T*)q.ln2_g, dxn2, dy, dx1w, g.dln2_g, g.dln2_b, p.T, C, st))) return rc;
    dx1 = dx1w;
  }
  if ((rc = backward_impl(p, xn, q.w_qkv, q.w_proj, q.bias_table, saved + l.s_attn, dx1, dxn, g.dw_qkv, g.db_qkv, g.dw_proj,
                          g.db_proj, g.dbias_table, scratch + l.b_attn, p.bwd_scratch, st)))
    return rc;
  // dX = dX1 (skip of Eq. 4) + LayerNorm backward of the attention's input gradient
  return launch_ln_bwd<T>(x, st1, (const T*)q.ln1_g, dxn, dx1, dx, g.dln1_g, g.dln1_b, p.T, C, st);
}

bool bad16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) != 0; }

}  // namespace
}  // namespace gswa

using namespace gswa;

extern "C" {

int gswa_astl_workspace_query(const gswa_desc* desc, int32_t mlp_hidden, size_t* saved_bytes, size_t* fwd_scratch_bytes,
                              size_t* infer_scratch_bytes, size_t* bwd_scratch_bytes) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (mlp_hidden < 0) return GSWA_ERR_SHAPE;
  const AstlLayout l = astl_layout(p, mlp_hidden);
  if (saved_bytes) *saved_bytes = l.saved_total;
  if (fwd_scratch_bytes) *fwd_scratch_bytes = l.fwd_total;
  if (infer_scratch_bytes) *infer_scratch_bytes = l.fwd_total + l.saved_total;
  if (bwd_scratch_bytes) *bwd_scratch_bytes = l.bwd_total;
  return GSWA_OK;
}

int gswa_astl_forward(const gswa_desc* desc, int32_t mlp_hidden, const void* x, const gswa_astl_params* params, void* y,
                      void* saved, void* scratch, size_t scratch_bytes, void* cuda_stream) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (mlp_hidden < 0) return GSWA_ERR_SHAPE;
  if (!x || !y || !params || !scratch) return GSWA_ERR_NULL;
  const gswa_astl_params& q = *params;
  if (!q.ln1_g || !q.ln1_b || !q.w_qkv || !q.w_proj || !q.bias_table) return GSWA_ERR_NULL;
  if (mlp_hidden > 0 && (!q.ln2_g || !q.ln2_b || !q.w_fc1 || !q.b_fc1 || !q.w_fc2 || !q.b_fc2)) return GSWA_ERR_NULL;
  if (bad16(x) || bad16(y) || bad16(saved) || bad16(scratch)) return GSWA_ERR_ALIGN;
  const AstlLayout l = astl_layout(p, mlp_hidden);
  if (scratch_bytes < (saved ? l.fwd_total : l.fwd_total + l.saved_total)) return GSWA_ERR_WORKSPACE;
  if (p.T == 0) return GSWA_OK;
  char* sc = static_cast<char*>(scratch);
  char* sv = saved ? static_cast<char*>(saved) : sc + l.fwd_total;     // inference: the carry lives behind the scratch
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (p.dtype == GSWA_F32) return astl_forward_t<float>(p, mlp_hidden, (const float*)x, q, (float*)y, sv, sc, st);
  return astl_forward_t<__nv_bfloat16>(p, mlp_hidden, (const __nv_bfloat16*)x, q, (__nv_bfloat16*)y, sv, sc, st);
}

int gswa_astl_backward(const gswa_desc* desc, int32_t mlp_hidden, const void* x, const gswa_astl_params* params,
                       const void* saved, const void* dy, void* dx, const gswa_astl_grads* grads, void* scratch,
                       size_t scratch_bytes, void* cuda_stream) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (mlp_hidden < 0) return GSWA_ERR_SHAPE;
  if (!x || !dy || !dx || !params || !grads || !saved || !scratch) return GSWA_ERR_NULL;
  const gswa_astl_params& q = *params;
  const gswa_astl_grads& g = *grads;
  if (!q.ln1_g || !q.w_qkv || !q.w_proj || !q.bias_table || !g.dln1_g || !g.dln1_b || !g.dw_qkv || !g.db_qkv || !g.dw_proj ||
      !g.db_proj || !g.dbias_table)
    return GSWA_ERR_NULL;
  if (mlp_hidden > 0 && (!q.ln2_g || !q.ln2_b || !q.w_fc1 || !q.w_fc2 || !g.dln2_g || !g.dln2_b || !g.dw_fc1 || !g.db_fc1 || !g.dw_fc2 ||
                         !g.db_fc2))
    return GSWA_ERR_NULL;
  if (bad16(x) || bad16(dy) || bad16(dx) || bad16(saved) || bad16(scratch)) return GSWA_ERR_ALIGN;
  const AstlLayout l = astl_layout(p, mlp_hidden);
  if (scratch_bytes < l.bwd_total) return GSWA_ERR_WORKSPACE;
  if (p.T == 0) return GSWA_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (p.dtype == GSWA_F32)
    return astl_backward_t<float>(p, mlp_hidden, (const float*)x, q, (const char*)saved, (const float*)dy, (float*)dx, g,
                                  (char*)scratch, st);
  return astl_backward_t<__nv_bfloat16>(p, mlp_hidden, (const __nv_bfloat16*)x, q, (const char*)saved, (const __nv_bfloat16*)dy,
                                        (__nv_bfloat16*)dx, g, (char*)scratch, st);
}

}  // extern "C"
