// Projection GEMMs of the bf16 path on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// TMEM).  Three persistent, warp-specialised kernels share one structure:
//     warps 0-3  epilogue   TMEM -> registers -> global        (one accumulator row per thread)
//     warp  4    MMA issue  one elected thread, tcgen05.mma + tcgen05.commit
//     warps 5-12 loaders    global -> registers -> swizzled shared memory (row pitches of C = 60/180
//                           elements are not 16-byte multiples, so the caller's tensors cannot be
//                           described to TMA; rows are fetched with 8-byte loads and K is zero-padded
//                           on the fly)
// Roles talk through mbarriers; every wait is bounded and reports through an error word.
//
//   gw_kernel  Eq. 6 projections (and dA = dy W^P): rows are gathered in WINDOW order of one head
//              group (cyclic shift + window partition as address arithmetic) and the epilogue writes
//              contiguous per-(window, head) tiles.
//   gt_kernel  Eq. 7 output projection (and dx = dqkv W_qkv): rows in token order, packed rows out.
//   gr_kernel  parameter gradients dW = sum_t L[t,:]^T R[t,:] with both operands MN-major, bias
//              gradients through a column of ones.
#include "fast.cuh"
#include "gswa_index.cuh"
#include "umma.cuh"

namespace gswa {
using namespace umma;
namespace {

constexpr int kEpiWarps = 4, kLoadWarps = 8;
constexpr int kThreads = 32 * (kEpiWarps + 1 + kLoadWarps);   // 416
constexpr int kLoadThreads = 32 * kLoadWarps;                 // 256
constexpr uint32_t kSpinLimit = 2000000u;

// Bounded wait shared by all roles.  On timeout raises the CTA-wide abort flag and the error word.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_s, int* err) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 127u) == 127u) {
      if (*abort_s) return false;
      __nanosleep(40);
    }
  }
  *abort_s = 1;
  if (err) atomicExch(err, 1);
  return false;
}
// All lanes of a warp take the same decision.
__device__ __forceinline__ bool wait_bar_warp(uint64_t* bar, uint32_t parity, volatile int* abort_s, int* err) {
  const bool ok = wait_bar(bar, parity, abort_s, err);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
  return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~(uintptr_t)1023);
}
__device__ __forceinline__ uint2 ldg8(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint2*>(p)); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__host__ __device__ inline uint32_t pow2_cols(int n) {
  uint32_t c = 32;
  while ((int)c < n) c <<= 1;
  return c;
}

// ==========================================================================================
// gw_kernel
// ==========================================================================================
template <int CP, int DP>
__global__ void __launch_bounds__(kThreads, 1) gw_kernel(const __grid_constant__ GWLaunch L) {
  const GWUnit& u = L.u[blockIdx.y];
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  constexpr int kStageBytes = 128 * CP * 2;
  constexpr int kAtomBytesA = 128 * 128;
  const int NT = u.nchunks * u.cw;
  unsigned char* sB = sm;
  unsigned char* sA0 = sB + (size_t)NT * CP * 2;
  float* sBias = reinterpret_cast<float*>(sA0 + 2 * kStageBytes);
  __shared__ uint64_t full[2], empty[2], tfull[8], tempty[8];
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < NT * CP * 2 / 16; i += kThreads)
    reinterpret_cast<uint4*>(sB)[i] = __ldg(reinterpret_cast<const uint4*>(u.Bimg) + i);
  for (int i = tid; i < NT; i += kThreads) sBias[i] = u.bias ? u.bias[i] : 0.f;
  fence_proxy_async();
  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 2; ++i) { mbar_init(&full[i], kLoadThreads); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 8; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], 128); }
    mbar_init_fence();
  }
  const uint32_t tcols = pow2_cols(NT);
  if (warp == kEpiWarps) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;
  const long long n_tiles = (u.n_windows + 1) / 2;

  if (warp > kEpiWarps) {
    // ---------------- loaders: warp lw owns window column lw of every window row
    const int lw = warp - kEpiWarps - 1;
    constexpr int NPC = (CP / 4 + 31) / 32;      // 8-byte pieces per lane per row
    int it = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      const int stage = it & 1;
      if (!wait_bar_warp(&empty[stage], ((it >> 1) & 1) ^ 1, &abort_s, L.err)) break;
      unsigned char* sA = sA0 + stage * kStageBytes;
#pragma unroll
      for (int kb = 0; kb < 16; kb += 4) {
        uint2 v[4][NPC];
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int k = kb + kk;
          const long long win = 2 * tile + (k >> 3);
          const __nv_bfloat16* src = nullptr;
          if (win < u.n_windows) {
            const int b = (int)(win / u.nW), w = (int)(win % u.nW);
            int i = (w / u.nWw) * 8 + (k & 7) + u.s, j = (w % u.nWw) * 8 + lw + u.s;
            if (i >= u.H) i -= u.H;
            if (j >= u.W) j -= u.W;
            src = u.A + ((long long)(b * u.H + i) * u.W + j) * u.lda;
          }
#pragma unroll
          for (int pi = 0; pi < NPC; ++pi) {
            const int col = (lane + 32 * pi) * 4;
            v[kk][pi] = make_uint2(0u, 0u);
            if (src != nullptr && col < u.kvalid) v[kk][pi] = ldg8(src + col);
          }
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int r = lw + 8 * (kb + kk);
#pragma unroll
          for (int pi = 0; pi < NPC; ++pi) {
            const int col = (lane + 32 * pi) * 4;
            if (col < CP)
              *reinterpret_cast<uint2*>(sA + (col >> 6) * kAtomBytesA + sw128_offset(r, col & 63)) = v[kk][pi];
          }
        }
      }
      fence_proxy_async();
      mbar_arrive(&full[stage]);
    }
  } else if (warp == kEpiWarps) {
    // ---------------- MMA issue
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, u.cw, 0, 0);
      const uint32_t bAddr = smem_u32(sB);
      int it = 0;
      bool ok = true;
      for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
        const int stage = it & 1;
        if (!wait_bar(&full[stage], (it >> 1) & 1, &abort_s, L.err)) break;
        fence_after_sync();
        const uint32_t aAddr = smem_u32(sA0 + stage * kStageBytes);
        for (int c = 0; c < u.nchunks; ++c) {
          if (!wait_bar(&tempty[c], (it & 1) ^ 1, &abort_s, L.err)) { ok = false; break; }
          fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < CP / 16; ++kk) {
            const uint64_t ad = make_desc(aAddr + (kk >> 2) * kAtomBytesA + (kk & 3) * 32, 16, 1024);
            const uint64_t bd = make_desc(bAddr + (kk >> 2) * (NT * 128) + c * u.cw * 128 + (kk & 3) * 32, 16, 1024);
            mma_bf16(tmem + c * u.cw, ad, bd, idesc, kk > 0);
          }
          commit(&tfull[c]);
        }
        commit(&empty[stage]);
      }
    }
  } else {
    // ---------------- epilogue: thread = accumulator row = (window of the pair, slot)
    const int r = tid;
    const int nblk = u.cw / DP;
    int it = 0;
    bool ok = true;
    for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
      const long long win = 2 * tile + (r >> 6);
      const bool valid = win < u.n_windows;
      __nv_bfloat16* orow = u.out + win * u.win_stride + (r & 63) * DP;
      for (int c = 0; c < u.nchunks; ++c) {
        if (!wait_bar_warp(&tfull[c], it & 1, &abort_s, L.err)) { ok = false; break; }
        fence_after_sync();
        for (int blk = 0; blk < nblk; ++blk) {
          uint32_t v[DP];
          const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + c * u.cw + blk * DP;
          if constexpr (DP == 32) tmem_ld32(taddr, v); else tmem_ld16(taddr, v);
          tmem_ld_wait();
          const int gb = c * nblk + blk, n0 = c * u.cw + blk * DP;
          const float sc = (u.q_every3 && gb % 3 == 0) ? u.qscale : 1.f;
          uint32_t o[DP / 2];
#pragma unroll
          for (int j = 0; j < DP / 2; ++j)
            o[j] = pack_bf16((__uint_as_float(v[2 * j]) + sBias[n0 + 2 * j]) * sc,
                             (__uint_as_float(v[2 * j + 1]) + sBias[n0 + 2 * j + 1]) * sc);
          if (valid) {
            uint4* dst = reinterpret_cast<uint4*>(orow + (long long)gb * 64 * DP);
#pragma unroll
            for (int j = 0; j < DP / 8; ++j) dst[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
          }
        }
        fence_before_sync();
        mbar_arrive(&tempty[c]);
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kEpiWarps) {
    __syncwarp();
    tmem_dealloc(tmem, tcols);
  }
}

// ==========================================================================================
// gt_kernel
// ==========================================================================================
constexpr int kAtomStage = 128 * 128;   // one K atom of a 128-row tile: 16 KB

__global__ void __launch_bounds__(kThreads, 1) gt_kernel(const __grid_constant__ GTLaunch L) {
  const GTSplit& sp = L.s[blockIdx.y];
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  const int NB = L.NB, natoms = L.natoms, S = L.nstages;
  unsigned char* sB = sm;
  unsigned char* ring = sB + (size_t)natoms * NB * 128;
  unsigned char* stg = ring + (size_t)S * kAtomStage;
  float* sBias = reinterpret_cast<float*>(stg + (size_t)128 * NB * 2);
  __shared__ uint64_t full[8], empty[8], tfull[2], tempty[2];
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < natoms * NB * 8; i += kThreads)
    reinterpret_cast<uint4*>(sB)[i] = __ldg(reinterpret_cast<const uint4*>(sp.Bimg) + i);
  for (int i = tid; i < NB; i += kThreads) sBias[i] = sp.bias ? sp.bias[i] : 0.f;
  fence_proxy_async();
  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 8; ++i) { mbar_init(&full[i], kLoadThreads); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], 128); }
    mbar_init_fence();
  }
  const uint32_t tcols = pow2_cols(2 * NB);
  if (warp == kEpiWarps) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;
  const long long n_tiles = (L.rows + 127) / 128;

  if (warp > kEpiWarps) {
    // ---------------- loaders: thread -> (8-byte piece of the atom, 8 rows)
    const int tl = tid - 32 * (kEpiWarps + 1);
    const int piece = tl & 15, row0 = tl >> 4;
    int st = 0, ph = 0;
    bool ok = true;
    for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      for (int atom = 0; atom < natoms; ++atom) {
        if (!wait_bar_warp(&empty[st], ph ^ 1, &abort_s, L.err)) { ok = false; break; }
        const int col = atom * 64 + piece * 4;
        uint2 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const long long t = tile * 128 + row0 + 16 * k;
          v[k] = make_uint2(0u, 0u);
          if (t < L.rows && col < L.kvalid) v[k] = ldg8(L.A + t * L.lda + col);
        }
        unsigned char* sA = ring + st * kAtomStage;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          *reinterpret_cast<uint2*>(sA + sw128_offset(row0 + 16 * k, piece * 4)) = v[k];
        fence_proxy_async();
        mbar_arrive(&full[st]);
        if (++st == S) { st = 0; ph ^= 1; }
      }
    }
  } else if (warp == kEpiWarps) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, NB, 0, 0);
      const uint32_t bAddr = smem_u32(sB), rAddr = smem_u32(ring);
      int st = 0, ph = 0, it = 0;
      bool ok = true;
      for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
        const int buf = it & 1;
        if (!wait_bar(&tempty[buf], ((it >> 1) & 1) ^ 1, &abort_s, L.err)) break;
        fence_after_sync();
        for (int atom = 0; atom < natoms; ++atom) {
          if (!wait_bar(&full[st], ph, &abort_s, L.err)) { ok = false; break; }
          fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t ad = make_desc(rAddr + st * kAtomStage + kk * 32, 16, 1024);
            const uint64_t bd = make_desc(bAddr + atom * (NB * 128) + kk * 32, 16, 1024);
            mma_bf16(tmem + buf * NB, ad, bd, idesc, (atom | kk) != 0);
          }
          commit(&empty[st]);
          if (++st == S) { st = 0; ph ^= 1; }
        }
        if (ok) commit(&tfull[buf]);
      }
    }
  } else {
    // ---------------- epilogue: stage the warp's 32 rows in shared memory, then store row pieces
    const int ncols = sp.ncols, n8 = ncols / 4;
    unsigned char* mystg = stg + (size_t)warp * 32 * ncols * 2;
    int it = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      const int buf = it & 1;
      if (!wait_bar_warp(&tfull[buf], (it >> 1) & 1, &abort_s, L.err)) break;
      fence_after_sync();
      for (int c0 = 0; c0 < ncols; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + buf * NB + c0, v);
        tmem_ld_wait();
        uint32_t* dst = reinterpret_cast<uint32_t*>(mystg + ((size_t)lane * ncols + c0) * 2);
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c0 + 2 * j < ncols)
            dst[j] = pack_bf16(__uint_as_float(v[2 * j]) + sBias[c0 + 2 * j],
                               __uint_as_float(v[2 * j + 1]) + sBias[c0 + 2 * j + 1]);
      }
      fence_before_sync();
      mbar_arrive(&tempty[buf]);
      __syncwarp();
      const long long trow0 = tile * 128 + warp * 32;
      for (int e = lane; e < 32 * n8; e += 32) {
        const int rr = e / n8, pc = e - rr * n8;
        const long long t = trow0 + rr;
        if (t < L.rows)
          *reinterpret_cast<uint2*>(L.out + t * L.ldo + sp.col0 + pc * 4) =
              *reinterpret_cast<const uint2*>(mystg + ((size_t)rr * ncols + pc * 4) * 2);
      }
      __syncwarp();
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kEpiWarps) {
    __syncwarp();
    tmem_dealloc(tmem, tcols);
  }
}

// ==========================================================================================
// gr_kernel
// ==========================================================================================
__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}

__global__ void __launch_bounds__(kThreads, 1) gr_kernel(const __grid_constant__ GRLaunch L) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  const int NP = L.NP, ratoms = NP / 64;
  const int stage_bytes = (2 + ratoms) * 8192;
  __shared__ uint64_t full[4], empty[4], done;
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;
  constexpr int S = 4;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mb = blockIdx.y;
  long long chunk = (L.rows + L.nsplit - 1) / L.nsplit;
  chunk = (chunk + 63) / 64 * 64;
  const long long t0 = (long long)blockIdx.x * chunk;
  const long long t1 = t0 + chunk < L.rows ? t0 + chunk : L.rows;
  if (t0 >= t1) return;
  const int nst = (int)((t1 - t0 + 63) / 64);

  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < S; ++i) { mbar_init(&full[i], kLoadThreads); mbar_init(&empty[i], 1); }
    mbar_init(&done, 1);
    mbar_init_fence();
  }
  const uint32_t tcols = pow2_cols(NP);
  if (warp == kEpiWarps) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;

  if (warp > kEpiWarps) {
    const int lw = warp - kEpiWarps - 1;
    const int lcol = mb * 128 + lane * 4;
    int st = 0, ph = 0;
    for (int s = 0; s < nst; ++s) {
      if (!wait_bar_warp(&empty[st], ph ^ 1, &abort_s, L.err)) break;
      unsigned char* sL = sm + (size_t)st * stage_bytes;
      unsigned char* sR = sL + 2 * 8192;
      const long long tb = t0 + (long long)s * 64;
#pragma unroll
      for (int kb = 0; kb < 8; kb += 4) {
        uint2 vl[4], vr[4][2];
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const long long t = tb + lw + 8 * (kb + kk);
          const bool tv = t < t1;
          vl[kk] = make_uint2(0u, 0u);
          if (tv && lcol < L.mvalid) vl[kk] = ldg8(L.L + t * L.ldl + lcol);
#pragma unroll
          for (int pi = 0; pi < 2; ++pi) {
            const int col = (lane + 32 * pi) * 4;
            vr[kk][pi] = make_uint2(0u, 0u);
            if (tv) {
              if (col < L.nvalid) vr[kk][pi] = ldg8(L.R + t * L.ldr + col);
              else if (col == L.nvalid) vr[kk][pi] = make_uint2(0x3F80u, 0u);   // bf16 1.0: the ones column
            }
          }
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int r = lw + 8 * (kb + kk);
          *reinterpret_cast<uint2*>(sL + (lane >> 4) * 8192 + sw128_offset(r, (lane & 15) * 4)) = vl[kk];
#pragma unroll
          for (int pi = 0; pi < 2; ++pi) {
            const int col = (lane + 32 * pi) * 4;
            if (col < NP) *reinterpret_cast<uint2*>(sR + (col >> 6) * 8192 + sw128_offset(r, col & 63)) = vr[kk][pi];
          }
        }
      }
      fence_proxy_async();
      mbar_arrive(&full[st]);
      if (++st == S) { st = 0; ph ^= 1; }
    }
  } else if (warp == kEpiWarps) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, NP, 1, 1);
      int st = 0, ph = 0;
      bool ok = true;
      for (int s = 0; s < nst; ++s) {
        if (!wait_bar(&full[st], ph, &abort_s, L.err)) { ok = false; break; }
        fence_after_sync();
        const uint32_t lAddr = smem_u32(sm + (size_t)st * stage_bytes), rAddr = lAddr + 2 * 8192;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const uint64_t ad = make_desc(lAddr + kk * 2048, 8192, 1024);
          const uint64_t bd = make_desc(rAddr + kk * 2048, 8192, 1024);
          mma_bf16(tmem, ad, bd, idesc, (s | kk) != 0);
        }
        commit(&empty[st]);
        if (++st == S) { st = 0; ph ^= 1; }
      }
      if (ok) commit(&done);
    }
  } else {
    if (wait_bar_warp(&done, 0, &abort_s, L.err)) {
      fence_after_sync();
      const int m = mb * 128 + tid;
      for (int c0 = 0; c0 < NP; c0 += 32) {
        if (c0 > L.nvalid) break;
        uint32_t v[32];
        tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + c0, v);
        tmem_ld_wait();
        if (m < L.mvalid) {
          float* orow = L.out + (long long)m * L.nvalid;
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const int n = c0 + j;
            if (n + 3 < L.nvalid) {
              red_add_v4(orow + n, __uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                         __uint_as_float(v[j + 3]));
            } else if (n == L.nvalid && L.colsum != nullptr) {
              atomicAdd(L.colsum + m, __uint_as_float(v[j]));
            }
          }
        }
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kEpiWarps) {
    __syncwarp();
    tmem_dealloc(tmem, tcols);
  }
}

// ==========================================================================================
// weight images
// ==========================================================================================
struct PrepJobs {
  PrepJob j[16];
};

__global__ void prep_kernel(const __grid_constant__ PrepJobs J) {
  const PrepJob& p = J.j[blockIdx.y];
  const int total = p.NT * p.KP;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
    const int n = e / p.KP, k = e % p.KP;
    float val = 0.f;
    const int C = p.C;
    if (p.mode == PREP_QKV) {            // row n = (head, q|k|v, c) of W_qkv; k = input channel
      const int blk = n / p.dp, c = n % p.dp, h = p.h0 + blk / 3, kind = blk % 3;
      if (c < p.d && k < C) val = __bfloat162float(p.W[(long long)(kind * C + h * p.d + c) * C + k]);
    } else if (p.mode == PREP_PROJ_T) {  // row n = (head, c) -> input channel of W_proj; k = output channel
      const int h = p.h0 + n / p.dp, c = n % p.dp;
      if (c < p.d && k < C) val = __bfloat162float(p.W[(long long)k * C + h * p.d + c]);
    } else if (p.mode == PREP_PROJ) {    // row n = output channel n0+n of W_proj; k = input channel
      if (p.n0 + n < C && k < C) val = __bfloat162float(p.W[(long long)(p.n0 + n) * C + k]);
    } else {                             // PREP_QKV_T: row n = input channel n0+n; k = row of W_qkv
      if (p.n0 + n < C && k < 3 * C) val = __bfloat162float(p.W[(long long)k * C + p.n0 + n]);
    }
    *reinterpret_cast<__nv_bfloat16*>(p.img + (size_t)(k >> 6) * p.NT * 128 + sw128_offset(n, k & 63)) =
        __float2bfloat16_rn(val);
    if (k == 0 && p.bias_out != nullptr) {
      float bv = 0.f;
      if (p.b != nullptr) {
        if (p.mode == PREP_QKV) {
          const int blk = n / p.dp, c = n % p.dp, h = p.h0 + blk / 3, kind = blk % 3;
          if (c < p.d) bv = __bfloat162float(p.b[kind * C + h * p.d + c]);
        } else if (p.mode == PREP_PROJ) {
          if (p.n0 + n < C) bv = __bfloat162float(p.b[p.n0 + n]);
        }
      }
      p.bias_out[n] = bv;
    }
  }
}

}  // namespace

int launch_prep(const PrepJob* jobs, int njobs, cudaStream_t st) {
  if (njobs <= 0) return GSWA_OK;
  if (njobs > 16) return GSWA_ERR_UNSUPPORTED;
  PrepJobs J{};
  for (int i = 0; i < njobs; ++i) J.j[i] = jobs[i];
  { KernelScope ks_("prep_weights", st); prep_kernel<<<dim3(64, njobs), 256, 0, st>>>(J); }
  return check_launch();
}

static int num_sms() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  }
  return n;
}

template <int CP, int DP>
static int launch_gw_t(const GWLaunch& L, int nunits, cudaStream_t st, const char* name) {
  int maxNT = 0;
  long long max_tiles = 1;
  for (int i = 0; i < nunits; ++i) {
    const int NT = L.u[i].nchunks * L.u[i].cw;
    if (NT > maxNT) maxNT = NT;
    const long long t = (L.u[i].n_windows + 1) / 2;
    if (t > max_tiles) max_tiles = t;
  }
  const size_t smem = 1024 + (size_t)maxNT * CP * 2 + 2 * 128 * CP * 2 + (size_t)maxNT * 4 + 64;
  if (cudaFuncSetAttribute(gw_kernel<CP, DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  long long gx = num_sms() / nunits;
  if (gx < 1) gx = 1;
  if (gx > max_tiles) gx = max_tiles;
  { KernelScope ks_(name, st); gw_kernel<CP, DP><<<dim3((unsigned)gx, nunits), kThreads, smem, st>>>(L); }
  return check_launch();
}

int launch_gw(const GWLaunch& L, int nunits, int Cp, int dp, cudaStream_t st, const char* name) {
#define GW_CASE(CPV)                                                        \
  if (Cp == CPV) return dp == 32 ? launch_gw_t<CPV, 32>(L, nunits, st, name) : launch_gw_t<CPV, 16>(L, nunits, st, name);
  GW_CASE(64) GW_CASE(128) GW_CASE(192) GW_CASE(256)
#undef GW_CASE
  return GSWA_ERR_UNSUPPORTED;
}

size_t gt_smem_bytes(int natoms, int NB, int nstages) {
  return 1024 + (size_t)natoms * NB * 128 + (size_t)nstages * kAtomStage + (size_t)128 * NB * 2 + (size_t)NB * 4 + 64;
}

int launch_gt(const GTLaunch& L, int nsplits, cudaStream_t st, const char* name) {
  const size_t smem = gt_smem_bytes(L.natoms, L.NB, L.nstages);
  if (cudaFuncSetAttribute(gt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  const long long n_tiles = (L.rows + 127) / 128;
  long long gx = num_sms() / nsplits;
  if (gx < 1) gx = 1;
  if (gx > n_tiles) gx = n_tiles;
  { KernelScope ks_(name, st); gt_kernel<<<dim3((unsigned)gx, nsplits), kThreads, smem, st>>>(L); }
  return check_launch();
}

int launch_gr(const GRLaunch& L, cudaStream_t st, const char* name) {
  const size_t smem = 1024 + (size_t)4 * (2 + L.NP / 64) * 8192 + 64;
  if (cudaFuncSetAttribute(gr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  const int mblocks = (L.mvalid + 127) / 128;
  { KernelScope ks_(name, st); gr_kernel<<<dim3(L.nsplit, mblocks), kThreads, smem, st>>>(L); }
  return check_launch();
}

}  // namespace gswa
