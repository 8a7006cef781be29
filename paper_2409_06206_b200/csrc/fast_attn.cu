// Window attention of the bf16 path, forward and recompute-based backward (Eq. 6 `Attn`, with the
// relative-position bias and the shifted-window mask).  One 8x8 window is a 64 x 64 x d problem per
// head: far too small to feed a 128-row tcgen05 tile without packing unrelated windows, and its cost
// is dominated by the softmax and the index work, so these kernels use warp-level mma.sync
// m16n8k16 with the score tile, the softmax and the probability operand all kept in registers
// (row statistics by quad shuffles).  q, k, v arrive as contiguous per-(window, head) tiles; the
// mask is evaluated from per-slot region labels (never a [windows, 64, 64] tensor) and only in the
// windows of the last row / column of a shifted group; window reverse and reverse shift are the
// address arithmetic of the output stores.
//
// The backward pass keeps only the row log-sum-exp from the forward pass: P = exp(S - L) is rebuilt
// per window, D = rowsum(P * dP) replaces the usual dO.O term, and P / dS cross from the
// query-major phase (dQ) to the key-major phase (dK, dV) through shared memory.
#include "attn_core.cuh"

namespace gswa {
using namespace attn;
namespace {

// ------------------------------------------------------------------------------------------
// forward: persistent CTAs stride over the windows of a unit; 4 warps per head, 16 query rows per
// warp.  The q,k,v tiles of the next window are copied into the second buffer while the current
// window is being computed.
// ------------------------------------------------------------------------------------------
// HPU = heads per CTA the kernel is compiled for (1: one head per CTA, 128 threads, many CTAs per SM;
// 3: up to three heads per CTA).
template <int DP, int HPU>
__global__ void __launch_bounds__(128 * HPU, HPU == 1 ? 7 : 2) attn_fwd_kernel(const __grid_constant__ AttnLaunch L) {
  const AttnUnit& u = L.u[blockIdx.y];
  const FastGeom& g = L.geo;
  extern __shared__ __align__(128) unsigned char sm[];
  const int nh_u = u.nheads;
  const int tile_bytes = nh_u * 3 * 64 * DP * 2;
  float2* tab = reinterpret_cast<float2*>(sm + 2 * (size_t)tile_bytes);     // pair table, see bias_init
  int* tok2 = reinterpret_cast<int*>(tab + nh_u * 225);
  unsigned char* reg2 = reinterpret_cast<unsigned char*>(tok2 + 128);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* ostg = sm + 2 * (size_t)tile_bytes + (((size_t)nh_u * 225 * 8 + 128 * 4 + 128 + 15) & ~(size_t)15) +
                        (size_t)warp * 16 * DP * 2;                 // this warp's 16 x DP output staging block
  const int nt = nh_u * 128;
  __shared__ uint64_t ldbar[2];
  if (tid == 0) {
    umma::mbar_init(&ldbar[0], 1);
    umma::mbar_init(&ldbar[1], 1);
    umma::mbar_init_fence();
  }
  __syncthreads();
  if (tid >= nt) return;

  fill_pair_table(tab, L.table, g.nh, u.h0, nh_u, tid, nt);
  const int hl = warp >> 2, r0 = (warp & 3) * 16;
  const int h = u.h0 + hl;

  // Windows are visited from the last to the first: the kernel that produced the tiles wrote the last
  // windows last, so they are the ones still resident in L2.
  // One window's q,k,v tile images are contiguous in global memory and already laid out as the kernel
  // wants them: one bulk asynchronous copy per window, counted in bytes on a barrier per buffer.
  auto fetch = [&](long long w, int b) {
    if (tid == 0) {
      umma::fence_proxy_async();
      umma::mbar_arrive_expect_tx(&ldbar[b], (uint32_t)tile_bytes);
      umma::bulk_load(smem_u32(sm + (size_t)b * tile_bytes), L.qkv + u.qkv_off + w * u.qkv_wstride, (uint32_t)tile_bytes, &ldbar[b]);
    }
  };
  long long win = g.n_windows - 1 - blockIdx.x;
  if (win >= 0) fetch(win, 0);
  for (int buf = 0, it = 0; win >= 0; win -= gridDim.x, buf ^= 1, ++it) {
    int* tok = tok2 + buf * 64;
    unsigned char* reg = reg2 + buf * 64;
    const WinCtx wc = window_setup(g, u.s, win, tok, reg, tid);
    if (!umma::mbar_wait(&ldbar[buf], (it >> 1) & 1) && L.err != nullptr) atomicExch(L.err, 1);
    __syncthreads();   // this window's tiles and maps are complete; every warp has left the previous window,
                       // so the other buffer may be refilled
    const long long nxt = win - gridDim.x;
    if (nxt >= 0) fetch(nxt, buf ^ 1);

    unsigned char* tiles = sm + (size_t)buf * tile_bytes;
    const uint32_t q_base = smem_u32(tiles + (size_t)(hl * 3 + 0) * 64 * DP * 2);
    fwd_window<DP>(q_base, q_base + 64 * DP * 2, q_base + 2 * 64 * DP * 2, tab + hl * 225, tok, reg, wc.masked, r0, lane,
                   ostg, L.A, g.nh * DP, h, g.d,
                   L.Lt != nullptr ? L.Lt + u.l_off + win * u.l_wstride + hl * 64 : nullptr);
  }
}

// ------------------------------------------------------------------------------------------
// backward: persistent CTAs stride over the windows of a unit
// ------------------------------------------------------------------------------------------
template <int DP, int HPU>
__global__ void __launch_bounds__(128 * HPU, HPU == 1 ? 4 : 1) attn_bwd_kernel(const __grid_constant__ AttnLaunch L) {
  const AttnUnit& u = L.u[blockIdx.y];
  const FastGeom& g = L.geo;
  extern __shared__ __align__(128) unsigned char sm[];
  const int nh_u = u.nheads;
  constexpr int kTile = 64 * DP * 2;
  const int in_bytes = nh_u * 4 * kTile;                       // q,k,v per head then dO per head: one window
  unsigned char* Ps = sm + 2 * (size_t)in_bytes;               // [head][64][64] bf16
  unsigned char* dSs = Ps + (size_t)nh_u * 8192;
  float* Lrow2 = reinterpret_cast<float*>(dSs + (size_t)nh_u * 8192);   // [2][head][64], 16-byte aligned
  float2* tab = reinterpret_cast<float2*>(Lrow2 + 2 * nh_u * 64);          // pair table, see bias_init
  float* hist = reinterpret_cast<float*>(sm);                  // per-offset sums of dS: built after the last window, over the dead input tiles
  int* tok2 = reinterpret_cast<int*>(tab + nh_u * 225);        // [2][64]
  unsigned char* reg2 = reinterpret_cast<unsigned char*>(tok2 + 128);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* ostg = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(reg2 + 128) + 15) & ~(uintptr_t)15) +
                        (size_t)warp * 16 * DP * 2;              // this warp's 16 x DP output staging block
  const int nt = nh_u * 128;
  __shared__ uint64_t ldbar[2];
  if (tid == 0) {
    umma::mbar_init(&ldbar[0], 1);
    umma::mbar_init(&ldbar[1], 1);
    umma::mbar_init_fence();
  }
  __syncthreads();
  if (tid >= nt) return;

  fill_pair_table(tab, L.table, g.nh, u.h0, nh_u, tid, nt);
  const int hl = warp >> 2, r0 = (warp & 3) * 16, gq = lane >> 2, t = lane & 3;
  const int h = u.h0 + hl;
  const int Ap = g.nh * DP;                                    // row length of the padded token-major buffers
  unsigned char* Ph = Ps + (size_t)hl * 8192;
  unsigned char* dSh = dSs + (size_t)hl * 8192;
  const int p0 = r0 + gq;
  float dsum[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) dsum[j][0] = dsum[j][1] = dsum[j][2] = dsum[j][3] = 0.f;

  // One window's inputs (q,k,v tile images, dO tile images, row log-sum-exp) are three contiguous runs in
  // global memory: three bulk asynchronous copies per window, counted in bytes on a barrier per buffer.
  auto fetch = [&](long long w, int b) {
    if (tid == 0) {
      const uint32_t qb = (uint32_t)nh_u * 3 * kTile, ob = (uint32_t)nh_u * kTile, lb = (uint32_t)nh_u * 64 * 4;
      unsigned char* dst = sm + (size_t)b * in_bytes;
      umma::fence_proxy_async();
      umma::mbar_arrive_expect_tx(&ldbar[b], qb + ob + lb);
      umma::bulk_load(smem_u32(dst), L.qkv + u.qkv_off + w * u.qkv_wstride, qb, &ldbar[b]);
      umma::bulk_load(smem_u32(dst + qb), L.dO + u.do_off + w * u.do_wstride, ob, &ldbar[b]);
      umma::bulk_load(smem_u32(Lrow2 + b * nh_u * 64), L.Lt + u.l_off + w * u.l_wstride, lb, &ldbar[b]);
    }
  };

  // last window first: the dO tiles written last by the preceding GEMM are still in L2
  long long win = g.n_windows - 1 - blockIdx.x;
  if (win >= 0) fetch(win, 0);
  for (int buf = 0, it = 0; win >= 0; win -= gridDim.x, buf ^= 1, ++it) {
    int* tok = tok2 + buf * 64;
    unsigned char* reg = reg2 + buf * 64;
    const float* Lrow = Lrow2 + buf * nh_u * 64;
    const WinCtx wc = window_setup(g, u.s, win, tok, reg, tid);
    if (!umma::mbar_wait(&ldbar[buf], (it >> 1) & 1) && L.err != nullptr) atomicExch(L.err, 1);
    __syncthreads();   // this window's inputs are complete; every warp has left the previous window, so the
                       // other input buffer, P and dS may be overwritten
    const long long nxt = win - gridDim.x;
    if (nxt >= 0) fetch(nxt, buf ^ 1);
    unsigned char* tiles = sm + (size_t)buf * in_bytes;
    const uint32_t q_base = smem_u32(tiles + (size_t)(hl * 3) * kTile);
    const uint32_t k_base = q_base + kTile, v_base = k_base + kTile;
    const uint32_t do_base = smem_u32(tiles + (size_t)(nh_u * 3 + hl) * kTile);

    // ---- query-major phase: this warp owns query rows r0 .. r0+15 of head hl
    float s[8][4];
    bias_init(s, tab + hl * 225, p0, t);
    qk_scores<DP, false>(s, q_base, k_base, r0, lane);
    apply_mask(s, reg, wc.masked, p0, t);
    const float l0 = Lrow[hl * 64 + p0] * kLog2e, l1 = Lrow[hl * 64 + p0 + 8] * kLog2e;
    {
      const unsigned long long ll0 = pk2(l0, l0), ll1 = pk2(l1, l1);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        upk2(sub2(pk2(s[j][0], s[j][1]), ll0), s[j][0], s[j][1]);
        upk2(sub2(pk2(s[j][2], s[j][3]), ll1), s[j][2], s[j][3]);
        s[j][0] = ex2(s[j][0]);
        s[j][1] = ex2(s[j][1]);
        s[j][2] = ex2(s[j][2]);
        s[j][3] = ex2(s[j][3]);
      }
    }
    float dp[8][4];
    qk_scores<DP>(dp, do_base, v_base, r0, lane);          // dP = dO V^T
    float d0, d1;
    {
      unsigned long long a0 = pk2(0.f, 0.f), a1 = a0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        a0 = fma2(pk2(s[j][0], s[j][1]), pk2(dp[j][0], dp[j][1]), a0);
        a1 = fma2(pk2(s[j][2], s[j][3]), pk2(dp[j][2], dp[j][3]), a1);
      }
      float a, b;
      upk2(a0, a, b);
      d0 = a + b;
      upk2(a1, a, b);
      d1 = a + b;
    }
    d0 += __shfl_xor_sync(0xffffffffu, d0, 1);
    d0 += __shfl_xor_sync(0xffffffffu, d0, 2);
    d1 += __shfl_xor_sync(0xffffffffu, d1, 1);
    d1 += __shfl_xor_sync(0xffffffffu, d1, 2);
    {
      const unsigned long long dd0 = pk2(d0, d0), dd1 = pk2(d1, d1);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const unsigned long long e0 = mul2(pk2(s[j][0], s[j][1]), sub2(pk2(dp[j][0], dp[j][1]), dd0));
        const unsigned long long e1 = mul2(pk2(s[j][2], s[j][3]), sub2(pk2(dp[j][2], dp[j][3]), dd1));
        upk2(e0, dp[j][0], dp[j][1]);
        upk2(e1, dp[j][2], dp[j][3]);
        upk2(add2(pk2(dsum[j][0], dsum[j][1]), e0), dsum[j][0], dsum[j][1]);
        upk2(add2(pk2(dsum[j][2], dsum[j][3]), e1), dsum[j][2], dsum[j][3]);
      }
    }
    {
      // P and dS cross to the key-major phase through shared memory: four 8x8 blocks per stmatrix
      const int m = lane >> 3, srow = r0 + (m & 1) * 8 + (lane & 7);
      const uint32_t pa = smem_u32(Ph), da = smem_u32(dSh);
#pragma unroll
      for (int j = 0; j < 8; j += 2) {
        const uint32_t off = sq_off(srow, j + (m >> 1));
        stsm_x4(pa + off, pack2(s[j][0], s[j][1]), pack2(s[j][2], s[j][3]), pack2(s[j + 1][0], s[j + 1][1]),
                pack2(s[j + 1][2], s[j + 1][3]));
        stsm_x4(da + off, pack2(dp[j][0], dp[j][1]), pack2(dp[j][2], dp[j][3]), pack2(dp[j + 1][0], dp[j + 1][1]),
                pack2(dp[j + 1][2], dp[j + 1][3]));
      }
    }
    unsigned char* const drow0 = reinterpret_cast<unsigned char*>(L.dqkv + (long long)tok[p0] * 3 * Ap + h * DP);
    unsigned char* const drow1 = reinterpret_cast<unsigned char*>(L.dqkv + (long long)tok[p0 + 8] * 3 * Ap + h * DP);
    {
      float dq[DP / 8][4];
#pragma unroll
      for (int j = 0; j < DP / 8; ++j) dq[j][0] = dq[j][1] = dq[j][2] = dq[j][3] = 0.f;
      regs_times_tile<DP>(dq, dp, k_base, lane);             // dQ = dS K
      store_tile<DP>(ostg, dq, L.scale, L.scale, drow0, drow1, lane, -1);
    }
    __syncthreads();

    // ---- key-major phase: this warp owns keys r0 .. r0+15: dV = P^T dO, dK = dS^T Q
    float dv[DP / 8][4], dk[DP / 8][4];
#pragma unroll
    for (int j = 0; j < DP / 8; ++j)
      dv[j][0] = dv[j][1] = dv[j][2] = dv[j][3] = dk[j][0] = dk[j][1] = dk[j][2] = dk[j][3] = 0.f;
    const uint32_t p_addr = smem_u32(Ph), ds_addr = smem_u32(dSh);
    const int kc = (warp & 3) * 2;   // first 16-byte key chunk of this warp
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t ap[4], ad[4];
      const int qrow = 16 * kk + (lane & 7) + (((lane >> 4) & 1) << 3);
      const int chunk = kc + ((lane >> 3) & 1);
      ldsm_x4_t(ap, p_addr + sq_off(qrow, chunk));
      ldsm_x4_t(ad, ds_addr + sq_off(qrow, chunk));
#pragma unroll
      for (int jn = 0; jn < DP / 16; ++jn) {
        uint32_t b[4];
        const int brow = 16 * kk + (lane & 7) + (((lane >> 3) & 1) << 3);
        ldsm_x4_t(b, do_base + tile_off<DP>(brow, 2 * jn + (lane >> 4)));
        mma16816(dv[2 * jn], ap, b[0], b[1]);
        mma16816(dv[2 * jn + 1], ap, b[2], b[3]);
        ldsm_x4_t(b, q_base + tile_off<DP>(brow, 2 * jn + (lane >> 4)));
        mma16816(dk[2 * jn], ad, b[0], b[1]);
        mma16816(dk[2 * jn + 1], ad, b[2], b[3]);
      }
    }
    // q was stored scaled by log2(e) (the scores live in the log2 domain): dK = dS^T q takes it back out
    store_tile<DP>(ostg, dk, kLn2, kLn2, drow0 + Ap * 2, drow1 + Ap * 2, lane, -1);
    store_tile<DP, false>(ostg, dv, 1.f, 1.f, drow0 + Ap * 4, drow1 + Ap * 4, lane, -1);
  }

  // ---- gradient of the bias table: fold this CTA's summed dS through the relative-position map
  if (L.dtable != nullptr) {
    __syncthreads();                        // every warp has left the last window: its input tiles are dead
    for (int e = tid; e < nh_u * 225; e += nt) hist[e] = 0.f;
    __syncthreads();
    const int pa0 = p0 >> 3, pc0 = p0 & 7;
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int rel = (pa0 + (e >> 1) - j + 7) * 15 + (pc0 - (2 * t + (e & 1)) + 7);
        atomicAdd(hist + hl * 225 + rel, dsum[j][e]);
      }
    __syncthreads();
    for (int e = tid; e < nh_u * 225; e += nt) atomicAdd(L.dtable + (e % 225) * g.nh + u.h0 + e / 225, hist[e]);
  }
}

// Index maps as the tensor-core kernels compute them: one block per window of one group runs window_setup (window ->
// original tokens and mask labels) and the fragment-wise bias-row arithmetic of bias_init, and scatters the results
// into per-token maps, for a bit-exact comparison with the definition.
__global__ void __launch_bounds__(128) fast_index_maps_kernel(FastGeom g, int s, int32_t* win_id, int32_t* slot, int32_t* region,
                                                              int32_t* rel) {
  __shared__ int tok[64];
  __shared__ unsigned char reg[64];
  const int tid = threadIdx.x;
  window_setup(g, s, (long long)blockIdx.x, tok, reg, tid);
  __syncthreads();
  if (tid < 64) {
    const int token = tok[tid];
    if (win_id != nullptr) win_id[token] = (int)blockIdx.x;
    if (blockIdx.x < (unsigned)g.nW) {                       // first image: the per-image maps
      if (slot != nullptr) slot[token] = tid;
      if (region != nullptr) region[token] = reg[tid];
    }
  }
  if (rel != nullptr && blockIdx.x == 0) {
    // the four warps' fragments: thread (warp, lane) holds queries p0 and p0 + 8 against keys 8j + 2t, 8j + 2t + 1
    const int warp = tid >> 5, lane = tid & 31, p0 = warp * 16 + (lane >> 2), t = lane & 3;
    for (int j = 0; j < 8; ++j) {
      const int r = frag_bias_row(p0, t, j), q = 8 * j + 2 * t;
      rel[p0 * 64 + q] = r;
      rel[p0 * 64 + q + 1] = r - 1;
      rel[(p0 + 8) * 64 + q] = r + 15;
      rel[(p0 + 8) * 64 + q + 1] = r + 14;
    }
  }
}

template <int DP>
size_t fwd_smem(int nheads) {
  return (size_t)2 * nheads * 3 * 64 * DP * 2 + (size_t)nheads * 225 * 8 + 128 * 4 + 128 + 128 + (size_t)nheads * 4 * 16 * DP * 2;
}
template <int DP>
size_t bwd_smem(int nheads) {
  return (size_t)2 * nheads * 4 * 64 * DP * 2 + (size_t)nheads * 2 * 8192 + (size_t)nheads * (2 * 225 + 2 * 64) * 4 + 128 * 4 + 128 + 128 +
         (size_t)nheads * 4 * 16 * DP * 2;
}

// CTAs per SM the hardware will co-schedule for this kernel and launch shape.
template <typename K>
int blocks_per_sm(K kernel, int threads, size_t smem) {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess || n < 1) {
    (void)cudaGetLastError();
    n = 1;
  }
  return n;
}

template <int DP, int HPU>
int launch_fwd_t(const AttnLaunch& L, int maxh, cudaStream_t st) {
  const size_t smem = fwd_smem<DP>(maxh);
  if (cudaFuncSetAttribute(attn_fwd_kernel<DP, HPU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int per_sm = blocks_per_sm(attn_fwd_kernel<DP, HPU>, maxh * 128, smem);
  long long gx = (long long)sms * per_sm / L.nunits;
  if (gx < 1) gx = 1;
  if (gx > L.geo.n_windows) gx = L.geo.n_windows;
  { KernelScope ks_("attn_fwd", st);
    attn_fwd_kernel<DP, HPU><<<dim3((unsigned)gx, L.nunits), maxh * 128, smem, st>>>(L); }
  return check_launch();
}

template <int DP, int HPU>
int launch_bwd_t(const AttnLaunch& L, int maxh, cudaStream_t st) {
  const size_t smem = bwd_smem<DP>(maxh);
  if (cudaFuncSetAttribute(attn_bwd_kernel<DP, HPU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int per_sm = blocks_per_sm(attn_bwd_kernel<DP, HPU>, maxh * 128, smem);
  long long gx = (long long)sms * per_sm / L.nunits;
  if (gx < 1) gx = 1;
  if (gx > L.geo.n_windows) gx = L.geo.n_windows;
  { KernelScope ks_("attn_bwd", st);
    attn_bwd_kernel<DP, HPU><<<dim3((unsigned)gx, L.nunits), maxh * 128, smem, st>>>(L); }
  return check_launch();
}

int max_heads(const AttnLaunch& L) {
  int maxh = 0;
  for (int i = 0; i < L.nunits; ++i) maxh = L.u[i].nheads > maxh ? L.u[i].nheads : maxh;
  return maxh;
}

}  // namespace

int launch_fast_index_maps(const FastGeom& g, int s, int32_t* win_id, int32_t* slot, int32_t* region, int32_t* rel,
                           cudaStream_t st) {
  if (g.n_windows <= 0) return GSWA_OK;
  { KernelScope ks_("fast_index_maps", st);
    fast_index_maps_kernel<<<dim3((unsigned)g.n_windows), 128, 0, st>>>(g, s, win_id, slot, region, rel); }
  return check_launch();
}

int launch_attn_fwd(const AttnLaunch& L, cudaStream_t st) {
  const int maxh = max_heads(L);
  if (maxh == 1) return L.geo.dp == 32 ? launch_fwd_t<32, 1>(L, 1, st) : launch_fwd_t<16, 1>(L, 1, st);
  return L.geo.dp == 32 ? launch_fwd_t<32, 3>(L, maxh, st) : launch_fwd_t<16, 3>(L, maxh, st);
}
int launch_attn_bwd(const AttnLaunch& L, cudaStream_t st) {
  const int maxh = max_heads(L);
  if (maxh == 1) return L.geo.dp == 32 ? launch_bwd_t<32, 1>(L, 1, st) : launch_bwd_t<16, 1>(L, 1, st);
  return L.geo.dp == 32 ? launch_bwd_t<32, 3>(L, maxh, st) : launch_bwd_t<16, 3>(L, maxh, st);
}

}  // namespace gswa
