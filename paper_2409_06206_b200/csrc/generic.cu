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
#include "gswa_index.cuh"
#include "gswa_internal.h"

namespace gswa {
namespace {

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// ------------------------------------------------------------------------------------------
// C(m,n) = scale_n * (sum_k A(m,k) B(k,n) + bias[n]),  A(m,k) = A[m*sam + k*sak], B(k,n) = B[k*sbk + n*sbn].
// grid.z splits K; with ATOMIC the partial sums are added into float C (which then must hold
// the running value), otherwise C is overwritten and grid.z must be 1.
// ------------------------------------------------------------------------------------------
constexpr int GB = 64, GK = 16;

template <typename TA, typename TB, typename TC, bool ATOMIC>
__global__ void __launch_bounds__(256) gemm_generic(const TA* __restrict__ A, long long sam, long long sak,
                                                    const TB* __restrict__ Bm, long long sbk, long long sbn,
                                                    TC* __restrict__ Cm, long long scm, const TB* __restrict__ bias,
                                                    int Mr, int Nc, long long K, long long kchunk, float scale,
                                                    int scale_cols) {
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
      if constexpr (ATOMIC) {
        atomicAdd(reinterpret_cast<float*>(Cm) + (long long)m * scm + n, v);
      } else {
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

template <typename TA, typename TB, typename TC>
int launch_gemm(const TA* A, long long sam, long long sak, const TB* Bm, long long sbk, long long sbn, TC* Cm,
                long long scm, const TB* bias, long long Mr, int Nc, long long K, float scale, int scale_cols,
                cudaStream_t st) {
  dim3 grid((unsigned)((Mr + GB - 1) / GB), (Nc + GB - 1) / GB, 1);
  { KernelScope ks_("gemm_generic", st); gemm_generic<TA, TB, TC, false><<<grid, 256, 0, st>>>(A, sam, sak, Bm, sbk, sbn, Cm, scm, bias, (int)Mr, Nc, K, K,
                                                        scale, scale_cols); }
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
                                                          1.f, 0); }
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

HeadShifts head_shifts(const Plan& p) {
  HeadShifts hs{};
  for (int g = 0; g < p.G; ++g)
    for (int h = 0; h < p.gh[g]; ++h) hs.s[p.gh0[g] + h] = (int8_t)p.gs[g];
  return hs;
}

AttnGeom attn_geom(const Plan& p) {
  return AttnGeom{p.H, p.W, p.nh, p.dqk, p.dv, p.M, p.N, p.Cq, p.Cv, p.Cqkv};
}

template <typename T>
int forward_t(const Plan& p, const T* x, const T* w_qkv, const T* b_qkv, const T* w_proj, const T* b_proj,
              const T* table, T* y, char* saved, cudaStream_t st) {
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
  return launch_gemm<T, T, T>(A, p.Cv, 1, w_proj, 1, p.Cv, y, C, b_proj, p.T, C, p.Cv, 1.f, 0, st);
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
                    const void* b_proj, const void* table, void* y, void* saved, cudaStream_t st) {
  if (p.dtype == GSWA_F32)
    return forward_t<float>(p, (const float*)x, (const float*)w_qkv, (const float*)b_qkv, (const float*)w_proj,
                            (const float*)b_proj, (const float*)table, (float*)y, (char*)saved, st);
  using bf = __nv_bfloat16;
  return forward_t<bf>(p, (const bf*)x, (const bf*)w_qkv, (const bf*)b_qkv, (const bf*)w_proj, (const bf*)b_proj,
                       (const bf*)table, (bf*)y, (char*)saved, st);
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
