// Shape-generic CUDA-core building blocks (f32 or bf16 storage, f32 arithmetic, plain FMA): a strided GEMM with a
// bias / column-scale epilogue, column sums, and the per-(window, head) attention kernels.  Shared by the GSWA path
// for shapes off the tensor-core path (generic.cu) and by the layer around it (astl.cu).
#pragma once

#include "gswa_index.cuh"
#include "gswa_internal.h"

namespace gswa {
namespace generic {


__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// ------------------------------------------------------------------------------------------
// C(m,n) = [resid(m,n) +] act(scale_n * (sum_k A'(m,k) B(k,n) + bias[n])), A' = A or GELU(A),  A(m,k) = A[m*sam + k*sak], B(k,n) = B[k*sbk + n*sbn].
// grid.z splits K; with ATOMIC the partial sums are added into float C (which then must hold
// the running value), otherwise C is overwritten and grid.z must be 1.
// ------------------------------------------------------------------------------------------
constexpr int GB = 64, GK = 16;

template <typename TA, typename TB, typename TC, bool ATOMIC>
__global__ void __launch_bounds__(256) gemm_generic(const TA* __restrict__ A, long long sam, long long sak,
                                                    const TB* __restrict__ Bm, long long sbk, long long sbn,
                                                    TC* __restrict__ Cm, long long scm, const TB* __restrict__ bias,
                                                    int Mr, int Nc, long long K, long long kchunk, float scale,
                                                    int scale_cols, int gelu, const TC* __restrict__ resid,
                                                    long long srm, int gelu_a) {
  __shared__ float As[GK][GB + 4];
  __shared__ float Bs[GK][GB + 4];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.x * GB, n0 = blockIdx.y * GB;
  const long long kbeg = (long long)blockIdx.z * kchunk;
  const long long kend = min(K, kbeg + kchunk);
  const int ty = tid / 16, tx = tid % 16;
  float acc[4][4] = {};
  const bool a_kfast = (sak == 1), b_kfast = (sbk == 1);
  for (long long k0 = kbeg; k0 < kend; k0 += GK) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int e = tid + r * 256;
      int m, k;
      if (a_kfast) { k = e % GK; m = e / GK; } else { m = e % GB; k = e / GB; }
      float v = 0.f;
      if (m0 + m < Mr && k0 + k < kend) v = ldf(A + (long long)(m0 + m) * sam + (k0 + k) * sak);
      if (gelu_a) v = 0.5f * v * (1.f + erff(v * 0.70710678118654752f));   // the A operand is GELU(A) (FC2 reads FC1's pre-activation)
      As[k][m] = v;
      int n;
      if (b_kfast) { k = e % GK; n = e / GK; } else { n = e % GB; k = e / GB; }
      v = 0.f;
      if (n0 + n < Nc && k0 + k < kend) v = ldf(Bm + (k0 + k) * sbk + (long long)(n0 + n) * sbn);
      Bs[k][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < GK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= Mr) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= Nc) continue;
      float v = acc[i][j];
      if (bias != nullptr && blockIdx.z == 0) v += ldf(bias + n);
      if (n < scale_cols) v *= scale;
      if (gelu) v = 0.5f * v * (1.f + erff(v * 0.70710678118654752f));     // exact (Gaussian CDF) form
      if constexpr (ATOMIC) {
        atomicAdd(reinterpret_cast<float*>(Cm) + (long long)m * scm + n, v);
      } else {
        if (resid != nullptr) v += ldf(resid + (long long)m * srm + n);    // skip connection
        stf(Cm + (long long)m * scm + n, v);
      }
    }
  }
}

// out[n] += sum_t G[t*ld + n]
template <typename T>
__global__ void __launch_bounds__(256) colsum_generic(const T* __restrict__ G, long long rows, int cols, long long ld,
                                                      long long rchunk, float* __restrict__ out) {
  const int n = blockIdx.x * 32 + threadIdx.x % 32;
  const int lane_r = threadIdx.x / 32;
  const long long r0 = (long long)blockIdx.y * rchunk, r1 = min(rows, r0 + rchunk);
  float s = 0.f;
  if (n < cols)
    for (long long r = r0 + lane_r; r < r1; r += 8) s += ldf(G + r * ld + n);
  __shared__ float red[8][33];
  red[lane_r][threadIdx.x % 32] = s;
  __syncthreads();
  if (lane_r == 0 && n < cols) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) t += red[i][threadIdx.x];
    atomicAdd(out + n, t);
  }
}

// ------------------------------------------------------------------------------------------
// Attention of one (window, head) per block.  qkv is token-major [T, 2*Cq + Cv] (q | k | v, head-major inside
// each, q already scaled); q and k have dq columns per head, v and the output dv (Sec. "Parameter Allocation":
// the Q and K projections may be narrower than V).
// ------------------------------------------------------------------------------------------
struct AttnGeom {
  int H, W, nh, dq, dv, M, N;
  int Cq, Cv, ld;              // heads * dq, heads * dv, row length of qkv (2*Cq + Cv)
};

template <typename T>
__global__ void __launch_bounds__(128) attn_fwd_generic(AttnGeom g, HeadShifts hs, const T* __restrict__ qkv,
                                                        const T* __restrict__ table, T* __restrict__ A,
                                                        float* __restrict__ L) {
  extern __shared__ float sm[];
  const int N = g.N, dq = g.dq, dv = g.dv, dqp = dq + 1, dvp = dv + 1, Np = N + 1;
  float* qs = sm;
  float* ks = qs + N * dqp;
  float* vs = ks + N * dqp;
  float* S = vs + N * dvp;
  int* tok = reinterpret_cast<int*>(S + N * Np);
  int* reg = tok + N;
  const int h = blockIdx.y, s = hs.s[h];
  const int nW = (g.H / g.M) * (g.W / g.M);
  const int b = blockIdx.x / nW, w = blockIdx.x % nW;
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int t = tid; t < N; t += nt) {
    int i, j, r;
    slot_to_token(g.H, g.W, g.M, s, w, t, &i, &j, &r);
    tok[t] = (b * g.H + i) * g.W + j;
    reg[t] = r;
  }
  __syncthreads();
  for (int e = tid; e < N * dq; e += nt) {
    const int t = e / dq, c = e % dq;
    const T* row = qkv + (long long)tok[t] * g.ld + h * dq + c;
    qs[t * dqp + c] = ldf(row);
    ks[t * dqp + c] = ldf(row + g.Cq);
  }
  for (int e = tid; e < N * dv; e += nt) {
    const int t = e / dv, c = e % dv;
    vs[t * dvp + c] = ldf(qkv + (long long)tok[t] * g.ld + 2 * g.Cq + h * dv + c);
  }
  __syncthreads();
  for (int e = tid; e < N * N; e += nt) {
    const int p = e / N, q = e % N;
    float acc = 0.f;
    for (int c = 0; c < dq; ++c) acc = fmaf(qs[p * dqp + c], ks[q * dqp + c], acc);
    acc += ldf(table + rel_row(g.M, p, q) * g.nh + h);
    S[p * Np + q] = (reg[p] == reg[q]) ? acc : -INFINITY;
  }
  __syncthreads();
  const int lane = tid % 32, warp = tid / 32, nwarp = nt / 32;
  for (int p = warp; p < N; p += nwarp) {
    float mx = -INFINITY;
    for (int q = lane; q < N; q += 32) mx = fmaxf(mx, S[p * Np + q]);
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
    for (int q = lane; q < N; q += 32) {
      const float e = expf(S[p * Np + q] - mx);
      S[p * Np + q] = e;
      sum += e;
    }
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv = 1.f / sum;
    for (int q = lane; q < N; q += 32) S[p * Np + q] *= inv;
    if (lane == 0 && L != nullptr) L[(long long)tok[p] * g.nh + h] = mx + logf(sum);
  }
  __syncthreads();
  for (int e = tid; e < N * dv; e += nt) {
    const int p = e / dv, c = e % dv;
    float acc = 0.f;
    for (int q = 0; q < N; ++q) acc = fmaf(S[p * Np + q], vs[q * dvp + c], acc);
    stf(A + (long long)tok[p] * g.Cv + h * dv + c, acc);
  }
}

// Backward of one (window, head): recompute P from q, k and the saved row log-sum-exp.  One N x N buffer serves
// two passes (first P, for dV = P^T dO; then, in place, dS = P o (dP - D), for dQ and dK), so that a 12 x 12
// window with head dims up to 48 fits the shared memory of one block.
template <typename T>
__global__ void __launch_bounds__(256) attn_bwd_generic(AttnGeom g, HeadShifts hs, float scale,
                                                        const T* __restrict__ qkv, const T* __restrict__ table,
                                                        const T* __restrict__ A, const float* __restrict__ L,
                                                        const T* __restrict__ dA, T* __restrict__ dqkv,
                                                        float* __restrict__ dtable) {
  extern __shared__ float sm[];
  const int N = g.N, dq = g.dq, dv = g.dv, dqp = dq + 1, dvp = dv + 1, Np = N + 1, nrel = (2 * g.M - 1) * (2 * g.M - 1);
  float* qs = sm;
  float* ks = qs + N * dqp;
  float* vs = ks + N * dqp;
  float* dOs = vs + N * dvp;
  float* PS = dOs + N * dvp;                // P, then dS
  float* D = PS + N * Np;
  float* Ls = D + N;
  float* hist = Ls + N;
  int* tok = reinterpret_cast<int*>(hist + nrel);
  int* reg = tok + N;
  const int h = blockIdx.y, s = hs.s[h];
  const int nW = (g.H / g.M) * (g.W / g.M);
  const int b = blockIdx.x / nW, w = blockIdx.x % nW;
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int t = tid; t < N; t += nt) {
    int i, j, r;
    slot_to_token(g.H, g.W, g.M, s, w, t, &i, &j, &r);
    tok[t] = (b * g.H + i) * g.W + j;
    reg[t] = r;
    Ls[t] = L[(long long)tok[t] * g.nh + h];
  }
  for (int e = tid; e < nrel; e += nt) hist[e] = 0.f;
  __syncthreads();
  for (int e = tid; e < N * dq; e += nt) {
    const int t = e / dq, c = e % dq;
    const T* row = qkv + (long long)tok[t] * g.ld + h * dq + c;
    qs[t * dqp + c] = ldf(row);
    ks[t * dqp + c] = ldf(row + g.Cq);
  }
  for (int e = tid; e < N * dv; e += nt) {
    const int t = e / dv, c = e % dv;
    vs[t * dvp + c] = ldf(qkv + (long long)tok[t] * g.ld + 2 * g.Cq + h * dv + c);
    dOs[t * dvp + c] = ldf(dA + (long long)tok[t] * g.Cv + h * dv + c);
  }
  __syncthreads();
  // D_p = sum_c dO[p,c] O[p,c]
  for (int p = tid; p < N; p += nt) {
    float acc = 0.f;
    for (int c = 0; c < dv; ++c) acc = fmaf(dOs[p * dvp + c], ldf(A + (long long)tok[p] * g.Cv + h * dv + c), acc);
    D[p] = acc;
  }
  // pass 1: P
  for (int e = tid; e < N * N; e += nt) {
    const int p = e / N, q = e % N;
    float sc = 0.f;
    for (int c = 0; c < dq; ++c) sc = fmaf(qs[p * dqp + c], ks[q * dqp + c], sc);
    sc += ldf(table + rel_row(g.M, p, q) * g.nh + h);
    PS[p * Np + q] = (reg[p] == reg[q]) ? expf(sc - Ls[p]) : 0.f;
  }
  __syncthreads();
  for (int e = tid; e < N * dv; e += nt) {
    const int t = e / dv, c = e % dv;
    float av = 0.f;
    for (int u = 0; u < N; ++u) av = fmaf(PS[u * Np + t], dOs[u * dvp + c], av);
    stf(dqkv + (long long)tok[t] * g.ld + 2 * g.Cq + h * dv + c, av);
  }
  __syncthreads();
  // pass 2: dS in place
  for (int e = tid; e < N * N; e += nt) {
    const int p = e / N, q = e % N;
    const float pv = PS[p * Np + q];
    float dpv = 0.f;
    for (int c = 0; c < dv; ++c) dpv = fmaf(dOs[p * dvp + c], vs[q * dvp + c], dpv);
    const float ds = pv * (dpv - D[p]);
    PS[p * Np + q] = ds;
    if (dtable != nullptr && pv != 0.f) atomicAdd(hist + rel_row(g.M, p, q), ds);
  }
  __syncthreads();
  for (int e = tid; e < N * dq; e += nt) {
    const int t = e / dq, c = e % dq;
    float aq = 0.f, ak = 0.f;
    for (int u = 0; u < N; ++u) {
      aq = fmaf(PS[t * Np + u], ks[u * dqp + c], aq);
      ak = fmaf(PS[u * Np + t], qs[u * dqp + c], ak);
    }
    T* row = dqkv + (long long)tok[t] * g.ld + h * dq + c;
    stf(row, aq * scale);
    stf(row + g.Cq, ak);
  }
  if (dtable != nullptr)
    for (int e = tid; e < nrel; e += nt) atomicAdd(dtable + e * g.nh + h, hist[e]);
}

template <typename TA, typename TB, typename TC>
int launch_gemm(const TA* A, long long sam, long long sak, const TB* Bm, long long sbk, long long sbn, TC* Cm,
                long long scm, const TB* bias, long long Mr, int Nc, long long K, float scale, int scale_cols,
                cudaStream_t st, int gelu = 0, const TC* resid = nullptr, long long srm = 0, int gelu_a = 0) {
  dim3 grid((unsigned)((Mr + GB - 1) / GB), (Nc + GB - 1) / GB, 1);
  { KernelScope ks_("gemm_generic", st); gemm_generic<TA, TB, TC, false><<<grid, 256, 0, st>>>(A, sam, sak, Bm, sbk, sbn, Cm, scm, bias, (int)Mr, Nc, K, K,
                                                        scale, scale_cols, gelu, resid, srm, gelu_a); }
  return check_launch();
}

// Cm[n1,n2] += sum_t G[t,n1] X[t,n2], reduction split over blocks.
template <typename TA, typename TB>
int launch_gemm_tn(const TA* G, long long ldg, int n1, const TB* X, long long ldx, int n2, long long rows, float* Cm,
                   cudaStream_t st) {
  long long splits = (rows + 2047) / 2048;
  if (splits > 1024) splits = 1024;
  if (splits < 1) splits = 1;
  long long kchunk = ((rows + splits - 1) / splits + GK - 1) / GK * GK;
  splits = (rows + kchunk - 1) / kchunk;
  dim3 grid((n1 + GB - 1) / GB, (n2 + GB - 1) / GB, (unsigned)splits);
  { KernelScope ks_("gemm_tn_generic", st); gemm_generic<TA, TB, float, true><<<grid, 256, 0, st>>>(G, 1, ldg, X, ldx, 1, Cm, n2, nullptr, n1, n2, rows, kchunk,
                                                          1.f, 0, 0, nullptr, 0, 0); }
  return check_launch();
}

template <typename T>
int launch_colsum(const T* G, long long rows, int cols, long long ld, float* out, cudaStream_t st) {
  long long chunks = (rows + 4095) / 4096;
  if (chunks > 2048) chunks = 2048;
  const long long rchunk = (rows + chunks - 1) / chunks;
  dim3 grid((cols + 31) / 32, (unsigned)chunks);
  { KernelScope ks_("colsum_generic", st); colsum_generic<T><<<grid, 256, 0, st>>>(G, rows, cols, ld, rchunk, out); }
  return check_launch();
}

inline HeadShifts head_shifts(const Plan& p) {
  HeadShifts hs{};
  for (int g = 0; g < p.G; ++g)
    for (int h = 0; h < p.gh[g]; ++h) hs.s[p.gh0[g] + h] = (int8_t)p.gs[g];
  return hs;
}

// ------------------------------------------------------------------------------------------
// small element-wise helpers
// ------------------------------------------------------------------------------------------
// out[row, 0..w) = a[row*lda + 0..w) + b[row*ldb + 0..w)   (b may be null)
template <typename T>
__global__ void __launch_bounds__(256) add_cols_kernel(const T* __restrict__ a, long long lda, const T* __restrict__ b, long long ldb,
                                                       T* __restrict__ out, long long ldo, long long rows, int w) {
  const long long n = rows * w;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / w;
    const int c = (int)(i - r * w);
    float v = ldf(a + r * lda + c);
    if (b != nullptr) v += ldf(b + r * ldb + c);
    stf(out + r * ldo + c, v);
  }
}

inline int grid_for(long long work_items, int per_block) {
  long long g = (work_items + per_block - 1) / per_block;
  const long long cap = (long long)device_sm_count() * 8;
  if (g > cap) g = cap;
  return g < 1 ? 1 : (int)g;
}

template <typename T>
int launch_add_cols(const T* a, long long lda, const T* b, long long ldb, T* out, long long ldo, long long rows, int w,
                    cudaStream_t st) {
  { KernelScope ks_("add_cols", st);
    add_cols_kernel<T><<<grid_for(rows * w, 256 * 8), 256, 0, st>>>(a, lda, b, ldb, out, ldo, rows, w); }
  return check_launch();
}

}  // namespace generic
}  // namespace gswa
