// Channel-sliced heads with the cascade (Sec. "Group Shifted Window Attention", Eq. 6 read literally, and Eq. 8):
// head i projects only its own slice of ds = C / heads input channels (W_i: rows q | k | v, [2*dq + ds, ds]) and
// attends inside its group's (shifted) windows; with the cascade the input of head i >= 1 is its slice plus the
// output of head i-1, so the heads run one after the other.  The outputs are concatenated and projected (Eq. 7).
// Runs on the shape-generic CUDA-core kernels: one small projection GEMM and one attention launch per head.
//   saved   : per-head q|k|v [heads][T, 2*dq + ds] | attention output A [T, C] | row log-sum-exp L [T, heads]
#include "generic_core.cuh"

namespace gswa {
using namespace generic;
namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct SlicedLayout {
  int ds, dq, ld;                    // slice width, q/k width, row length of one head's q|k|v
  size_t s_qkv, qkv_head, s_A, s_L, saved_total;
  size_t f_xin, fwd_total;
  size_t b_dA, b_dqkv, b_xin, bwd_total;
};

int sliced_layout(const Plan& p, SlicedLayout* l) {
  if (p.dv != p.d) return GSWA_ERR_UNSUPPORTED;          // a head's output must have its slice's width (Eq. 8 adds them)
  l->ds = p.d; l->dq = p.dqk; l->ld = 2 * p.dqk + p.d;
  const size_t es = (size_t)p.esize, T = (size_t)p.T;
  size_t o = 0;
  l->qkv_head = align_up(T * l->ld * es, 256);
  l->s_qkv = o; o += l->qkv_head * p.nh;
  l->s_A = o; o += align_up(T * p.C * es, 256);
  l->s_L = o; o += align_up(T * p.nh * sizeof(float), 256);
  l->saved_total = o;
  l->f_xin = 0; l->fwd_total = align_up(T * l->ds * es, 256);
  o = 0;
  l->b_dA = o; o += align_up(T * p.C * es, 256);
  l->b_dqkv = o; o += align_up(T * l->ld * es, 256);
  l->b_xin = o; o += align_up(T * l->ds * es, 256);
  l->bwd_total = o;
  return GSWA_OK;
}

// Geometry of one head's attention launch: the head's own q|k|v buffer, its column of A / dA (row pitch C), and its
// column of the bias table and of L (the kernels index those with head 0 and pitch `nh`).
AttnGeom head_geom(const Plan& p, const SlicedLayout& l) {
  return AttnGeom{p.H, p.W, p.nh, l.dq, l.ds, p.M, p.N, l.dq, p.C, l.ld};
}

int head_shift(const Plan& p, int head) {
  for (int g = 0; g < p.G; ++g)
    if (head < p.gh0[g] + p.gh[g]) return p.gs[g];
  return 0;
}

size_t sliced_fwd_smem(const Plan& p, const SlicedLayout& l) {
  return sizeof(float) * ((size_t)2 * p.N * (l.dq + 1) + (size_t)p.N * (l.ds + 1) + (size_t)p.N * (p.N + 1)) + 8 * (size_t)p.N;
}
size_t sliced_bwd_smem(const Plan& p, const SlicedLayout& l) {
  const size_t nrel = (size_t)(2 * p.M - 1) * (2 * p.M - 1);
  return sizeof(float) * ((size_t)2 * p.N * (l.dq + 1) + (size_t)2 * p.N * (l.ds + 1) + (size_t)p.N * (p.N + 1) + 2 * p.N + nrel) +
         8 * (size_t)p.N;
}

template <typename T>
int sliced_forward_t(const Plan& p, const SlicedLayout& l, bool cascade, const T* x, const T* w_heads, const T* b_heads,
                     const T* w_proj, const T* b_proj, const T* table, T* y, char* saved, char* scratch, cudaStream_t st) {
  const int C = p.C, ds = l.ds, ld = l.ld;
  T* A = reinterpret_cast<T*>(saved + l.s_A);
  float* L = reinterpret_cast<float*>(saved + l.s_L);
  T* xin = reinterpret_cast<T*>(scratch + l.f_xin);
  const float scale = 1.0f / sqrtf((float)l.dq);
  const size_t smem = sliced_fwd_smem(p, l);
  if (cudaFuncSetAttribute(attn_fwd_generic<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  const AttnGeom g = head_geom(p, l);
  int rc;
  for (int i = 0; i < p.nh; ++i) {
    T* qkv = reinterpret_cast<T*>(saved + l.s_qkv + (size_t)i * l.qkv_head);
    const T* in = x + i * ds;
    long long ldin = C;
    if (cascade && i > 0) {                                // Eq. 8: the former head's output joins this head's input
      if ((rc = launch_add_cols<T>(x + i * ds, C, A + (i - 1) * ds, C, xin, ds, p.T, ds, st))) return rc;
      in = xin;
      ldin = ds;
    }
    const T* wi = w_heads + (size_t)i * ld * ds;
    if ((rc = launch_gemm<T, T, T>(in, ldin, 1, wi, 1, ds, qkv, ld, b_heads ? b_heads + (size_t)i * ld : nullptr, p.T, ld, ds,
                                   scale, l.dq, st)))
      return rc;
    HeadShifts hs{};
    hs.s[0] = (int8_t)head_shift(p, i);
    { KernelScope ks_("attn_fwd_generic", st);
      attn_fwd_generic<T><<<dim3(p.B * p.nW, 1), 128, smem, st>>>(g, hs, qkv, table + i, A + i * ds, L + i); }
    if ((rc = check_launch())) return rc;
  }
  return launch_gemm<T, T, T>(A, C, 1, w_proj, 1, C, y, C, b_proj, p.T, C, C, 1.f, 0, st);   // Eq. 7
}
