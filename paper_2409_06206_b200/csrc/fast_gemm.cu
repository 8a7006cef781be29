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
// Warp-wide wait: one lane polls (32 lanes polling one barrier word only serialise on it), the
// outcome is broadcast, and the warp barrier orders the other lanes after the observation.
__device__ __forceinline__ bool wait_bar_warp(uint64_t* bar, uint32_t parity, volatile int* abort_s, int* err) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = wait_bar(bar, parity, abort_s, err) ? 1 : 0;
  ok = __shfl_sync(0xffffffffu, ok, 0);
  return ok != 0;
}

// A loader warp publishes a stage: every lane has waited for its own copies; the proxy fence makes
// them visible to the tensor core, the warp barrier orders the lanes, one lane arrives.
__device__ __forceinline__ void publish(uint64_t* bar, int lane) {
  fence_proxy_async();
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
  return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~(uintptr_t)1023);
}
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
    for (int i = 0; i < 2; ++i) { mbar_init(&full[i], kLoadWarps); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 8; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], kEpiWarps); }
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
    // ---------------- loaders: warp lw owns window column lw of every window row.  Asynchronous
    // 8-byte copies land directly in the swizzled operand image; a stage is published one tile
    // late (after its copies have completed), so two tiles of loads are in flight per SM.
    const int lw = warp - kEpiWarps - 1;
    constexpr int NPC = (CP / 4 + 31) / 32;      // 8-byte pieces per lane per row
    // Per-lane constants: tile row r = lw + 8*(8*half + a) has (r & 7) == lw, so the swizzled
    // destination of a piece is a fixed offset plus 1024 bytes per row step.
    uint32_t dst0[NPC];
    int colb[NPC];                                // byte offset of the piece inside a source row, -1 = padding
#pragma unroll
    for (int pi = 0; pi < NPC; ++pi) {
      const int col = (lane + 32 * pi) * 4;
      dst0[pi] = (uint32_t)((col >> 6) * kAtomBytesA) + sw128_offset(lw, col & 63);
      colb[pi] = col < u.kvalid ? col * 2 : -1;
    }
    const char* const srcA = reinterpret_cast<const char*>(u.A);
    const long long row_bytes = (long long)u.lda * 2;
    int it = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      const int stage = it & 1;
      if (!wait_bar_warp(&empty[stage], ((it >> 1) & 1) ^ 1, &abort_s, L.err)) break;
      const uint32_t sA = smem_u32(sA0 + stage * kStageBytes);
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        // one window of the pair: cyclic shift + partition are this address arithmetic
        const int win = 2 * (int)tile + half;
        const bool wv = win < (int)u.n_windows;
        const int b = win / u.nW, w = win - b * u.nW;
        const int wi = w / u.nWw, wj = w - wi * u.nWw;
        int j = wj * 8 + lw + u.s;
        if (j >= u.W) j -= u.W;
        const int i0 = wi * 8 + u.s;
        const char* col0 = srcA + ((long long)b * u.H * u.W + j) * row_bytes;
        const long long line_bytes = (long long)u.W * row_bytes;
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          int i = i0 + a;
          if (i >= u.H) i -= u.H;
          const char* src = col0 + i * line_bytes;
#pragma unroll
          for (int pi = 0; pi < NPC; ++pi) {
            if ((lane + 32 * pi) * 4 < CP) {
              const bool v = wv && colb[pi] >= 0;
              cp_async8(sA + dst0[pi] + (8 * half + a) * 1024, v ? src + colb[pi] : srcA, v);
            }
          }
        }
      }
      cp_async_commit();
      if (it > 0) {
        cp_async_wait(1);
        publish(&full[(it - 1) & 1], lane);
      }
    }
    cp_async_wait(0);
    if (it > 0 && __all_sync(0xffffffffu, abort_s == 0)) publish(&full[(it - 1) & 1], lane);
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
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty[c]);
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
    for (int i = 0; i < 8; ++i) { mbar_init(&full[i], kLoadWarps); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], kEpiWarps); }
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
    // ---------------- loaders: thread -> (8-byte piece of the atom, 8 rows), asynchronous copies;
    // a ring stage is published `lag` steps after it was issued, once its copies have landed.
    const int tl = tid - 32 * (kEpiWarps + 1);
    const int piece = tl & 15, row0 = tl >> 4;
    const int lag = S - 1 < 3 ? S - 1 : 3;
    const uint32_t ringA = smem_u32(ring);
    // rows row0 + 16k share (row & 7), so a piece's swizzled destination is dst0 + 2048 k
    const uint32_t dst0 = sw128_offset(row0, piece * 4);
    const char* const srcA = reinterpret_cast<const char*>(L.A);
    const long long row_bytes = (long long)L.lda * 2;
    int st = 0, ph = 0, n = 0, pub = 0;          // pub: ring stage of the oldest unpublished step
    bool ok = true;
    for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      const long long trow = tile * 128 + row0;
      const char* const src_t = srcA + trow * row_bytes + piece * 8;
      const bool full_tile = (tile + 1) * 128 <= L.rows;
      for (int atom = 0; atom < natoms; ++atom) {
        if (!wait_bar_warp(&empty[st], ph ^ 1, &abort_s, L.err)) { ok = false; break; }
        const bool cv = atom * 64 + piece * 4 < L.kvalid;
        const uint32_t sA = ringA + st * kAtomStage + dst0;
        const char* src = src_t + atom * 128;
        if (full_tile) {
#pragma unroll
          for (int k = 0; k < 8; ++k) cp_async8(sA + k * 2048, cv ? src + k * 16 * row_bytes : srcA, cv);
        } else {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const bool v = cv && trow + 16 * k < L.rows;
            cp_async8(sA + k * 2048, v ? src + k * 16 * row_bytes : srcA, v);
          }
        }
        cp_async_commit();
        if (++st == S) { st = 0; ph ^= 1; }
        if (++n > lag) {
          cp_async_wait(lag);
          publish(&full[pub], lane);
          if (++pub == S) pub = 0;
        }
      }
    }
    {
      int left = n < lag ? n : lag;              // steps issued but not yet published
      while (left > 0) {
        cp_async_wait(left - 1);
        if (ok) publish(&full[pub], lane);
        if (++pub == S) pub = 0;
        --left;
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
        // the lane's row of the staging tile; rows are 2*ncols bytes apart (a multiple of 8, and an
        // odd multiple for C = 180, so these 8-byte stores do not collide on banks)
        uint2* dst = reinterpret_cast<uint2*>(mystg + ((size_t)lane * ncols + c0) * 2);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c0 + 4 * j < ncols)
            dst[j] = make_uint2(pack_bf16(__uint_as_float(v[4 * j]) + sBias[c0 + 4 * j],
                                          __uint_as_float(v[4 * j + 1]) + sBias[c0 + 4 * j + 1]),
                                pack_bf16(__uint_as_float(v[4 * j + 2]) + sBias[c0 + 4 * j + 2],
                                          __uint_as_float(v[4 * j + 3]) + sBias[c0 + 4 * j + 3]));
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[buf]);
      // copy-out: lane = 8-byte piece of a row (two pieces per lane cover up to 256 columns)
      const long long trow0 = tile * 128 + warp * 32;
      const int nrows = L.rows - trow0 < 32 ? (int)(L.rows - trow0) : 32;
      char* const obase = reinterpret_cast<char*>(L.out + trow0 * L.ldo + sp.col0) + lane * 8;
      const long long obytes = (long long)L.ldo * 2;
      const unsigned char* sbase = mystg + lane * 8;
      const bool p0 = lane < n8, p1 = lane + 32 < n8;
#pragma unroll 4
      for (int rr = 0; rr < nrows; ++rr) {
        if (p0) *reinterpret_cast<uint2*>(obase + rr * obytes) = *reinterpret_cast<const uint2*>(sbase + rr * ncols * 2);
        if (p1)
          *reinterpret_cast<uint2*>(obase + rr * obytes + 256) =
              *reinterpret_cast<const uint2*>(sbase + rr * ncols * 2 + 256);
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
    for (int i = 0; i < S; ++i) { mbar_init(&full[i], kLoadWarps); mbar_init(&empty[i], 1); }
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
    constexpr int lag = 2;
    // Stage row r = lw + 8k has (r & 7) == lw: every piece's swizzled destination is a per-lane
    // constant plus 1024 bytes per k.  Pieces that never change (K/M padding, the ones column that
    // turns the GEMM into a column sum of L) are written once per stage buffer, before the loop.
    const uint32_t dL = (uint32_t)((lane >> 4) * 8192) + sw128_offset(lw, (lane & 15) * 4);
    const bool lvalid = lcol < L.mvalid;
    uint32_t dR[2];
    int rkind[2];                                 // 0 = data, 1 = ones column, 2 = zero padding, 3 = outside the stage
#pragma unroll
    for (int pi = 0; pi < 2; ++pi) {
      const int col = (lane + 32 * pi) * 4;
      dR[pi] = (uint32_t)(2 * 8192 + (col >> 6) * 8192) + sw128_offset(lw, col & 63);
      rkind[pi] = col >= NP ? 3 : (col < L.nvalid ? 0 : (col == L.nvalid ? 1 : 2));
    }
    for (int sgi = 0; sgi < S; ++sgi) {
      unsigned char* base = sm + (size_t)sgi * stage_bytes;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (!lvalid) *reinterpret_cast<uint2*>(base + dL + k * 1024) = make_uint2(0u, 0u);
#pragma unroll
        for (int pi = 0; pi < 2; ++pi)
          if (rkind[pi] == 1 || rkind[pi] == 2)
            *reinterpret_cast<uint2*>(base + dR[pi] + k * 1024) = make_uint2(rkind[pi] == 1 ? 0x3F80u : 0u, 0u);
      }
    }
    const char* const srcL = reinterpret_cast<const char*>(L.L);
    const char* const srcR = reinterpret_cast<const char*>(L.R);
    const long long lrow = (long long)L.ldl * 2, rrow = (long long)L.ldr * 2;
    int st = 0, ph = 0, n = 0, pub = 0;
    bool ok = true;
    for (int s = 0; s < nst; ++s) {
      if (!wait_bar_warp(&empty[st], ph ^ 1, &abort_s, L.err)) { ok = false; break; }
      const uint32_t sS = smem_u32(sm + (size_t)st * stage_bytes);
      const long long tb = t0 + (long long)s * 64 + lw;
      const char* pl = srcL + tb * lrow + lcol * 2;
      const char* pr = srcR + tb * rrow + lane * 8;
      if (tb - lw + 64 <= t1) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (lvalid) cp_async8(sS + dL + k * 1024, pl + k * 8 * lrow, true);
          if (rkind[0] == 0) cp_async8(sS + dR[0] + k * 1024, pr + k * 8 * rrow, true);
          if (rkind[1] == 0) cp_async8(sS + dR[1] + k * 1024, pr + k * 8 * rrow + 256, true);
        }
      } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const bool tv = tb + 8 * k < t1;
          if (lvalid) cp_async8(sS + dL + k * 1024, tv ? pl + k * 8 * lrow : srcL, tv);
          if (rkind[0] == 0) cp_async8(sS + dR[0] + k * 1024, tv ? pr + k * 8 * rrow : srcR, tv);
          if (rkind[1] == 0) cp_async8(sS + dR[1] + k * 1024, tv ? pr + k * 8 * rrow + 256 : srcR, tv);
        }
      }
      cp_async_commit();
      if (++st == S) { st = 0; ph ^= 1; }
      if (++n > lag) {
        cp_async_wait(lag);
        publish(&full[pub], lane);
        if (++pub == S) pub = 0;
      }
    }
    {
      int left = n < lag ? n : lag;
      while (left > 0) {
        cp_async_wait(left - 1);
        if (ok) publish(&full[pub], lane);
        if (++pub == S) pub = 0;
        --left;
      }
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
