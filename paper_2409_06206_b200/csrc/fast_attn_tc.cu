// Backward of the windowed attention (gradients of Eq. 6 `Attn` with relative-position bias and window
// mask) on the 5th-generation tensor cores.  One CTA works on one head and walks over PAIRS of windows:
// the 2 x 64 query rows of a pair fill the 128 rows of a tcgen05.mma, accumulators live in TMEM.
//
//   warps 0-7    softmax group 0   two threads per query row (TMEM lane), 32 keys each; steps 0, 2, 4, ...
//   warps 8-15   softmax group 1   steps 1, 3, 5, ...
//   warp  16     MMA issue         one elected thread
//   warp  17     loader            one elected thread, bulk asynchronous copies of the tile images
//
// Per step (window pair w0, w1; rows 0-63 belong to w0, rows 64-127 to w1), products on the tensor core:
//   S   = Q K^T      [128 x 128]  the two diagonal 64 x 64 blocks are the windows' scores
//   dP  = dO V^T     [128 x 128]  likewise
//   dV_x = [P_w0 | P_w1]^T dO_wx   x = 0,1   [128 keys x DP]; rows of window x are dV of that window
//   dK_x = [dS_w0 | dS_w1]^T Q_wx            likewise
//   dQ_x = [dS rows] K_wx                    [128 queries x DP]; rows of window x are dQ of that window
// The off-diagonal halves are computed and dropped: a 64-row product does not fill the tensor core's
// 128 rows, and the arithmetic is free next to the memory traffic.  The [64][DP] tile images that the
// projection GEMMs wrote are at the same time canonical swizzled operands (64-byte rows for DP = 32,
// 32-byte rows for DP = 16), K-major for S and dP and MN-major for dV, dK and dQ, so they are used as
// they arrive.  Between the two rounds of products the softmax threads turn S and dP into P and dS
// (exp2 of the recomputed scores minus the saved row log-sum-exp; dS = P (dP - rowsum(P dP))) and write
// them as bf16 into 128-byte swizzled [64][64] blocks.  The two groups alternate, so one group's
// arithmetic overlaps the other's products.  Every wait is bounded and reports through an error word.
#include "attn_core.cuh"
#include "gemm_core.cuh"
#include "gswa_index.cuh"

namespace gswa {
namespace {
using namespace gemm;
using attn::ex2;
using attn::kLn2;
using attn::kLog2e;

constexpr int kTcThreads = 576;        // 16 softmax warps, MMA warp, loader warp
constexpr int kTcMmaWarp = 16, kTcLoadWarp = 17;
constexpr int kTcStages = 4;          // input ring: window pairs in flight
constexpr int kTabPitch = 24;         // row pitch of the bias table in shared memory: the 32 lanes of a warp
                                      // (4 window rows x 8 window columns of queries) hit 32 different banks

// Bounded waits of this kernel: a non-blocking test followed by a short sleep.  A sleeping warp takes no issue
// slots and no shared-memory bandwidth from the warps that work, and it notices the phase change within
// the sleep time (a blocking try_wait was seen to come back several hundred nanoseconds late).
__device__ __forceinline__ bool tc_wait(uint64_t* bar, uint32_t parity, volatile int* abort_s, int* err) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_test_wait(bar, parity)) return true;
    __nanosleep(64);
    if ((i & 63u) == 63u && *abort_s) return false;
  }
  *abort_s = 1;
  if (err) atomicExch(err, 1);
  return false;
}
__device__ __forceinline__ bool tc_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_s, int* err) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = tc_wait(bar, parity, abort_s, err) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

template <int DP>
struct TcCfg {
  static constexpr int kRB = DP * 2;                 // bytes per tile row
  static constexpr int kTile = 64 * kRB;             // one [64][DP] tile image
  static constexpr int kStage = 8 * kTile;           // Q, K, V, dO of two windows
  static constexpr uint32_t kSw = DP == 32 ? 4u : 6u;   // swizzle code of the tile images
  static constexpr int kPS = 4 * 8192;               // P_w0, dS_w0, P_w1, dS_w1 of one group
  static constexpr size_t kSmem = 1024 + (size_t)kTcStages * kStage + 2 * kPS + (size_t)kTcStages * 128 * 4 +
                                  (15 * kTabPitch + 228 + 512) * 4 + 64;
};

__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t* v) {
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Barrier `id` over `nthreads` threads that also ANDs a predicate: all of them go on or give up together.
__device__ __forceinline__ bool bar_vote(int id, int nthreads, bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %3, 0;\n\tbar.red.and.pred p, %1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(r)
      : "r"(id), "r"(nthreads), "r"((uint32_t)ok)
      : "memory");
  return r != 0;
}

// DP/2 accumulator columns of this thread's TMEM lane, scaled, as bf16 pairs.
template <int DP>
__device__ __forceinline__ void load_half(uint32_t taddr, float scale, uint32_t* w) {
  uint32_t v[DP / 2];
  if constexpr (DP == 32) tmem_ld16(taddr, v); else tmem_ld8(taddr, v);
  tmem_ld_wait();
#pragma unroll
  if (scale == 1.f) {       // resolved at compile time where the caller passes the literal
#pragma unroll
    for (int e = 0; e < DP / 4; ++e) w[e] = pack_bf16(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
    return;
  }
#pragma unroll
  for (int e = 0; e < DP / 4; ++e) w[e] = pack_bf16(__uint_as_float(v[2 * e]) * scale, __uint_as_float(v[2 * e + 1]) * scale);
}
// ... stored to DP/2 consecutive elements of a padded token-major row,
template <int DP>
__device__ __forceinline__ void store_half(uint32_t taddr, float scale, unsigned char* dst) {
  uint32_t w[DP / 4];
  load_half<DP>(taddr, scale, w);
#pragma unroll
  for (int c = 0; c < DP / 16; ++c) *reinterpret_cast<uint4*>(dst + c * 16) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
}
// ... or to half `half` of row `row` of a [64][DP] tile image in shared memory.
template <int DP>
__device__ __forceinline__ void stage_half(uint32_t taddr, float scale, unsigned char* tile, int row, int half) {
  uint32_t w[DP / 4];
  load_half<DP>(taddr, scale, w);
  const uint32_t base = smem_u32(tile);
#pragma unroll
  for (int c = 0; c < DP / 16; ++c)
    st_shared_v4(base + tile_off<DP>(row, half * (DP / 16) + c), w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
}

// ... or to 2*(DP/2) consecutive bytes of shared memory.
template <int DP>
__device__ __forceinline__ void stage_half_linear(uint32_t taddr, float scale, unsigned char* dst) {
  uint32_t w[DP / 4];
  load_half<DP>(taddr, scale, w);
  const uint32_t base = smem_u32(dst);
#pragma unroll
  for (int c = 0; c < DP / 16; ++c) st_shared_v4(base + c * 16, w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
}

template <int DP>
__global__ void __maxnreg__(96) attn_bwd_tc_kernel(const __grid_constant__ AttnLaunch L) {
  using C = TcCfg<DP>;
  const AttnUnit& u = L.u[blockIdx.y];
  const FastGeom& g = L.geo;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  unsigned char* ring = sm;                                           // [stage][Q2 | K2 | V2 | dO2]
  unsigned char* ps = ring + (size_t)kTcStages * C::kStage;           // [group][P_w0 | dS_w0 | P_w1 | dS_w1]
  float* Ls = reinterpret_cast<float*>(ps + 2 * C::kPS);              // [stage][128]
  float* tab = Ls + kTcStages * 128;                                  // [15][kTabPitch]
  float* hist = tab + 15 * kTabPitch;                                 // [225]
  float* Dx = hist + 228;                                             // [group][half][128] partial row sums
  __shared__ uint64_t inFull[kTcStages], inEmpty[kTcStages], barS[2], barP1[2], barP[2], barO1[2], barO[2], barE[2], barFin;
  __shared__ uint32_t tmem_s;
  __shared__ volatile int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long npairs = (g.n_windows + 1) / 2;
  // pairs of this CTA: last first (the tiles written last by the preceding kernels are still in L2)
  const long long first = npairs - 1 - blockIdx.x;
  const int nsteps = first < 0 ? 0 : (int)(first / gridDim.x) + 1;

  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < kTcStages; ++i) { mbar_init(&inFull[i], 1); mbar_init(&inEmpty[i], 2); }
    for (int i = 0; i < 2; ++i) { mbar_init(&barS[i], 1); mbar_init(&barP1[i], 8); mbar_init(&barO1[i], 1); mbar_init(&barP[i], 8); mbar_init(&barO[i], 1); mbar_init(&barE[i], 2); }
    mbar_init(&barFin, 1);
    mbar_init_fence();
  }
  if (warp == kTcMmaWarp) tmem_alloc(&tmem_s, 512);
  for (int e = tid; e < 225; e += kTcThreads) {
    tab[(e / 15) * kTabPitch + e % 15] = __bfloat162float(L.table[e * g.nh + u.h0]) * kLog2e;
    hist[e] = 0.f;
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;

  if (warp == kTcLoadWarp) {
    // ---------------- loader: the tile images of a window pair, as far ahead as the ring allows
    if (lane == 0) {
      for (int i = 0; i < nsteps; ++i) {
        const int slot = i % kTcStages;
        if (i >= kTcStages && !tc_wait(&inEmpty[slot], ((i / kTcStages) - 1) & 1, &abort_s, L.err)) break;
        const long long w0 = 2 * (first - (long long)i * gridDim.x);
        const int nw = w0 + 1 < g.n_windows ? 2 : 1;
        unsigned char* st = ring + (size_t)slot * C::kStage;
        fence_proxy_async();
        mbar_arrive_expect_tx(&inFull[slot], (uint32_t)nw * (4u * C::kTile + 256u));
        for (int x = 0; x < nw; ++x) {
          const __nv_bfloat16* qsrc = L.qkv + u.qkv_off + (w0 + x) * u.qkv_wstride;      // q | k | v images of this head
          for (int kind = 0; kind < 3; ++kind)
            bulk_load(smem_u32(st + (2 * kind + x) * C::kTile), qsrc + kind * 64 * DP, C::kTile, &inFull[slot]);
          bulk_load(smem_u32(st + (6 + x) * C::kTile), L.dO + u.do_off + (w0 + x) * u.do_wstride, C::kTile, &inFull[slot]);
          bulk_load(smem_u32(Ls + slot * 128 + x * 64), L.Lt + u.l_off + (w0 + x) * u.l_wstride, 256u, &inFull[slot]);
        }
      }
    }
  } else if (warp == kTcMmaWarp) {
    // ---------------- MMA issue
    if (lane == 0) {
      const uint32_t idS = make_idesc(128, 128, 0, 0);        // K-major x K-major
      const uint32_t idT = make_idesc(128, 2 * DP, 1, 1);     // MN-major x MN-major
      const uint32_t idQ = make_idesc(128, 2 * DP, 0, 1);     // K-major x MN-major
      constexpr uint32_t kSbo = 8 * C::kRB;
      // descriptors without their address field (addresses are below 256 KB: adding address >> 4 cannot carry out of it)
      const uint64_t dK0 = make_desc_sw(0, 16, kSbo, C::kSw);           // tile image, K-major
      const uint64_t dM0 = make_desc_sw(0, C::kTile, kSbo, C::kSw);     // the two windows' tile images side by side, MN-major
      const uint64_t dP0 = make_desc(0, 8192, 1024);                    // [P_w0 | P_w1] or [dS_w0 | dS_w1], MN-major
      const uint64_t dQ0 = make_desc(0, 16, 1024);                      // dS_w0 over dS_w1 (128 rows), K-major
      constexpr int kStep = (16 * C::kRB) >> 4;                         // 16 rows of a tile
      // Work is issued in whatever order its inputs become ready: dV of a step as soon as its P is written
      // (while the softmax threads still compute dS), dK and dQ once dS is written, the first round of step si
      // as soon as its tiles have landed and the TMEM half of its group has been read out.  This one thread
      // polls without sleeping (it watches several barriers at a time).
      int si = 0, vj = 0, mj = 0;
      uint32_t idle = 0;
      while (mj < nsteps) {
        if (mj < vj && mbar_test_wait(&barP[mj & 1], (mj >> 1) & 1)) {
          // second round, part two, of step mj (dS is written, dP is read): dK and dQ of both windows
          fence_after_sync();
          const uint64_t sm0 = dM0 + (smem_u32(ring + (size_t)(mj % kTcStages) * C::kStage) >> 4);
          const uint64_t pb = smem_u32(ps + (size_t)(mj & 1) * C::kPS) >> 4;               // P_w0 | P_w1 | dS_w0 | dS_w1
          const uint32_t tO = tmem + (mj & 1) * 256;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)          // [dK_0 | dK_1] = [dS_w0 | dS_w1]^T [Q_w0 | Q_w1], 16 query rows per instruction
            mma_bf16(tO + 2 * DP, dP0 + pb + 1024 + kk * 128, sm0 + kk * kStep, idT, kk != 0);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)          // [dQ_0 | dQ_1] = [dS_w0 ; dS_w1] [K_w0 | K_w1], 16 keys per instruction
            mma_bf16(tO + 4 * DP, dQ0 + pb + 1024 + kk * 2, sm0 + ((2 * C::kTile) >> 4) + kk * kStep, idQ, kk != 0);
          commit(&barO[mj & 1]);
          ++mj;
          idle = 0;
        } else if (vj < si && mbar_test_wait(&barP1[vj & 1], (vj >> 1) & 1)) {
          // second round, part one, of step vj (P is written, S is read): dV of both windows over the scores' columns
          fence_after_sync();
          const uint64_t sm0 = dM0 + (smem_u32(ring + (size_t)(vj % kTcStages) * C::kStage) >> 4);
          const uint64_t pb = smem_u32(ps + (size_t)(vj & 1) * C::kPS) >> 4;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)          // [dV_0 | dV_1] = [P_w0 | P_w1]^T [dO_w0 | dO_w1]
            mma_bf16(tmem + (vj & 1) * 256, dP0 + pb + kk * 128, sm0 + ((6 * C::kTile) >> 4) + kk * kStep, idT, kk != 0);
          commit(&barO1[vj & 1]);
          ++vj;
          idle = 0;
        } else if (si < nsteps && mbar_test_wait(&inFull[si % kTcStages], (si / kTcStages) & 1) &&
                   (si < 2 || mbar_test_wait(&barE[si & 1], ((si >> 1) - 1) & 1))) {
          // first round of step si: scores and dP of the pair into the TMEM half of group si & 1
          fence_after_sync();
          const uint64_t qd = dK0 + (smem_u32(ring + (size_t)(si % kTcStages) * C::kStage) >> 4);
          const uint64_t kd = qd + ((2 * C::kTile) >> 4), vd = qd + ((4 * C::kTile) >> 4), od = qd + ((6 * C::kTile) >> 4);
          const uint32_t tS = tmem + (si & 1) * 256;
#pragma unroll
          for (int kk = 0; kk < DP / 16; ++kk) mma_bf16(tS, qd + kk * 2, kd + kk * 2, idS, kk != 0);
#pragma unroll
          for (int kk = 0; kk < DP / 16; ++kk) mma_bf16(tS + 128, od + kk * 2, vd + kk * 2, idS, kk != 0);
          commit(&barS[si & 1]);
          ++si;
          idle = 0;
        } else {
          if (++idle > kSpinLimit || abort_s) {
            if (!abort_s) { abort_s = 1; if (L.err) atomicExch(L.err, 1); }
            break;
          }
        }
      }
      // nothing may still be running on the tensor core when TMEM is given back
      commit(&barFin);
      tc_wait(&barFin, 0, &abort_s, L.err);
    }
  } else {
    // ---------------- softmax groups: two threads per query row of the pair (32 of the row's 64 keys each);
    // in the second round the same pair of threads owns one key row.
    const int grp = warp >> 3, wq = warp & 3, half = (warp >> 2) & 1;
    const int r = wq * 32 + lane, x = r >> 6, q = r & 63;      // x (window of the pair) is the same for a whole warp
    const int qa = q >> 3, qc = q & 7;
    const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
    // bias of key (ka, kc) = 32 half + j: tabq[-(j >> 3) * pitch - (j & 7)]
    const float* tabq = tab + (qa + 7 - 4 * half) * kTabPitch + qc + 7;
    // this thread's 64 bytes of row q of P_wx (dS_wx lies 16384 further: P_w0 | P_w1 | dS_w0 | dS_w1)
    const uint32_t prow = smem_u32(ps + (size_t)grp * C::kPS + x * 8192) + q * 128;
    const uint32_t swz = (uint32_t)(q & 7);
    const int Ap = g.nh * DP;
    const uint32_t tS = tmem + lane_base + grp * 256 + x * 64 + half * 32, tD = tS + 128;
    const uint32_t tO = tmem + lane_base + grp * 256 + half * (DP / 2);
    float* dpart = Dx + (grp * 2 + (half ^ 1)) * 128 + r;      // where the partner reads this thread's part of D
    const float* dpeer = Dx + (grp * 2 + half) * 128 + r;
    const int pair_id = 1 + grp * 4 + wq, win_id = 9 + grp * 2 + x;
    unsigned long long dsum2[16];                           // per-key sums of dS, two keys per packed f32x2 word
#pragma unroll
    for (int k = 0; k < 16; ++k) dsum2[k] = attn::pk2(0.f, 0.f);
    int pending = -1;                                      // input slot whose release waits for this thread's stores
    const float inv_nW = 1.0f / (float)g.nW, inv_nWw = 1.0f / (float)g.nWw;
    // Staging layout of a window that wraps around the image edge: its four pieces (upper/lower rows x
    // left/right columns, split after 8 - s positions) one after the other, each in box order, unswizzled.
    const bool wrap_tma = u.s > 0 && u.s == L.wrap_s;
    const int we = 8 - u.s;
    const int wri = qa >= we, wci = qc >= we;
    const int wrow = (wri ? 8 * we : 0) + (wci ? (wri ? u.s : we) * we : 0) + (qa - wri * we) * (wci ? u.s : we) + (qc - wci * we);

    for (int i = grp, n = 0; i < nsteps; i += 2, ++n) {
      const int slot = i % kTcStages;
      const int win = 2 * (int)(first - (long long)i * gridDim.x) + x;
      const bool valid = win < (int)g.n_windows;
      // (image, window row, window column) without integer division: float reciprocal, corrected by one step
      int b = (int)(((float)win + 0.5f) * inv_nW), wl = win - b * g.nW;
      if (wl < 0) { --b; wl += g.nW; } else if (wl >= g.nW) { ++b; wl -= g.nW; }
      int wi = (int)(((float)wl + 0.5f) * inv_nWw), wj = wl - wi * g.nWw;
      if (wj < 0) { --wi; wj += g.nWw; } else if (wj >= g.nWw) { ++wi; wj -= g.nWw; }
      // A window in the last row or column of a shifted frame wraps around the image edge and carries mask
      // labels; along such an axis the first 8 - s positions have one label, the rest another.  Bit j of
      // `msk` = this query may attend to key 32 half + j.
      const bool lastrow = u.s > 0 && wi == g.nWh - 1, lastcol = u.s > 0 && wj == g.nWw - 1;
      const bool wmasked = valid && (lastrow || lastcol);
      uint32_t msk = 0xFFFFFFFFu;
      if (wmasked) {
        const uint32_t low = (1u << (8 - u.s)) - 1u;
        const uint32_t rm = (!lastrow ? 0xFFu : (qa < 8 - u.s ? low : (0xFFu & ~low))) >> (4 * half);
        const uint32_t cm = !lastcol ? 0xFFu : (qc < 8 - u.s ? low : (0xFFu & ~low));
        msk = 0u;
#pragma unroll
        for (int ka = 0; ka < 4; ++ka)
          if ((rm >> ka) & 1u) msk |= cm << (8 * ka);
      }
      // A failed wait must not strand a partner warp at the barriers below: failures flow through their votes and
      // every warp leaves the loop only after the last barrier of an iteration.
      bool ok = tc_wait_warp(&inFull[slot], (i / kTcStages) & 1, &abort_s, L.err) &&
                tc_wait_warp(&barS[grp], n & 1, &abort_s, L.err);
      fence_after_sync();
      float D = 0.f;
      if (ok && valid) {
        const float l2 = Ls[slot * 128 + r] * kLog2e;
        const unsigned long long l22 = attn::pk2(l2, l2);
        unsigned long long D2 = attn::pk2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t sv[16], dv[16], pk[8];
          tmem_ld16(tS + c * 16, sv);
          tmem_ld16(tD + c * 16, dv);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const int k0 = c * 16 + j, k1 = k0 + 1;
            float p0, p1;
            attn::upk2(attn::sub2(attn::add2(attn::pk2(__uint_as_float(sv[j]), __uint_as_float(sv[j + 1])),
                                             attn::pk2(tabq[-(k0 >> 3) * kTabPitch - (k0 & 7)], tabq[-(k1 >> 3) * kTabPitch - (k1 & 7)])),
                                  l22),
                       p0, p1);
            p0 = ex2(p0);
            p1 = ex2(p1);
            if (wmasked) {
              if (!((msk >> k0) & 1u)) p0 = 0.f;
              if (!((msk >> k1) & 1u)) p1 = 0.f;
            }
            D2 = attn::fma2(attn::pk2(p0, p1), attn::pk2(__uint_as_float(dv[j]), __uint_as_float(dv[j + 1])), D2);
            pk[j >> 1] = pack_bf16(p0, p1);
          }
          // P goes to its block at once (16 keys = two 16-byte chunks of the row, 128-byte swizzle); the second
          // pass reads it back, which keeps it out of the registers in between
          st_shared_v4(prow + (((uint32_t)(4 * half + 2 * c) ^ swz) << 4), pk[0], pk[1], pk[2], pk[3]);
          st_shared_v4(prow + (((uint32_t)(4 * half + 2 * c + 1) ^ swz) << 4), pk[4], pk[5], pk[6], pk[7]);
        }
        {
          float da, db;
          attn::upk2(D2, da, db);
          D = da + db;
        }
        *dpart = D;
      }
      // P is written and S is read: dV may run (it overwrites the scores' first columns)
      fence_proxy_async();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&barP1[grp]);
      ok = bar_vote(pair_id, 64, ok);                      // the two warps that share these rows
      if (ok && valid) {
        D += *dpeer;
        const unsigned long long DD = attn::pk2(D, D);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t dv[16], dsw[8], pk[8];
          const uint32_t o0 = ((uint32_t)(4 * half + 2 * c) ^ swz) << 4, o1 = ((uint32_t)(4 * half + 2 * c + 1) ^ swz) << 4;
          tmem_ld16(tD + c * 16, dv);
          ld_shared_v4(prow + o0, pk);
          ld_shared_v4(prow + o1, pk + 4);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const int k0 = c * 16 + j;
            const uint32_t w = pk[j >> 1];
            const unsigned long long ds2 = attn::mul2(attn::pk2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u)),
                                                      attn::sub2(attn::pk2(__uint_as_float(dv[j]), __uint_as_float(dv[j + 1])), DD));
            dsum2[k0 >> 1] = attn::add2(dsum2[k0 >> 1], ds2);
            float ds0, ds1;
            attn::upk2(ds2, ds0, ds1);
            dsw[j >> 1] = pack_bf16(ds0, ds1);
          }
          st_shared_v4(prow + 16384 + o0, dsw[0], dsw[1], dsw[2], dsw[3]);
          st_shared_v4(prow + 16384 + o1, dsw[4], dsw[5], dsw[6], dsw[7]);
        }
      }
      if (pending >= 0) {                                  // the previous step's stores have long read their tiles
        bulk_group_wait_read();
        mbar_arrive(&inEmpty[pending]);
        pending = -1;
      }
      // dS is written and dP is read: dK and dQ may run (dQ overwrites dP)
      fence_proxy_async();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&barP[grp]);

      // The step's input tiles are dead by the time their products are done and serve as staging for the output
      // tiles (dQ over Q, dK over K, dV over V).  A window that lies inside the image is a box of the
      // token-major buffer: one tiled bulk store per tile.  A window that wraps around the image edge (exactly
      // the masked ones) goes out as four boxes (even shifts) or row by row.  Each thread moves half of its
      // row's DP columns.  dV is ready first (it only needed P) and is drained while dK and dQ still run.
      unsigned char* stg = ring + (size_t)slot * C::kStage + x * C::kTile;
      long long tokrow = 0;
      if (wmasked && !wrap_tma) {
        int ti = wi * 8 + qa + u.s, tj = wj * 8 + qc + u.s;            // undo the cyclic shift
        if (ti >= g.H) ti -= g.H;
        if (tj >= g.W) tj -= g.W;
        tokrow = ((long long)b * g.H + ti) * g.W + tj;
      }
      unsigned char* drow = reinterpret_cast<unsigned char*>(L.dqkv + tokrow * 3 * Ap + u.h0 * DP) + half * DP;
      ok = ok && tc_wait_warp(&barO1[grp], n & 1, &abort_s, L.err);
      fence_after_sync();
      if (ok && valid) {
        if (!wmasked) stage_half<DP>(tO + x * DP, 1.f, stg + 4 * C::kTile, q, half);
        else if (wrap_tma) stage_half_linear<DP>(tO + x * DP, 1.f, stg + 4 * C::kTile + wrow * C::kRB + half * DP);
        else store_half<DP>(tO + x * DP, 1.f, drow + Ap * 4);
      }
      ok = ok && tc_wait_warp(&barO[grp], n & 1, &abort_s, L.err);
      fence_after_sync();
      if (ok && valid) {
        // q was stored scaled by log2(e) (the scores live in the log2 domain): dK = dS^T q takes it back out
        if (!wmasked) {
          stage_half<DP>(tO + (4 + x) * DP, L.scale, stg, q, half);
          stage_half<DP>(tO + (2 + x) * DP, kLn2, stg + 2 * C::kTile, q, half);
        } else if (wrap_tma) {
          stage_half_linear<DP>(tO + (4 + x) * DP, L.scale, stg + wrow * C::kRB + half * DP);
          stage_half_linear<DP>(tO + (2 + x) * DP, kLn2, stg + 2 * C::kTile + wrow * C::kRB + half * DP);
        } else {
          store_half<DP>(tO + (4 + x) * DP, L.scale, drow);
          store_half<DP>(tO + (2 + x) * DP, kLn2, drow + Ap * 2);
        }
        fence_proxy_async();
      }
      fence_before_sync();
      if (!bar_vote(win_id, 128, ok)) break;               // the four warps of this window
      if (q == 0 && half == 0) {
        mbar_arrive(&barE[grp]);                           // the TMEM half has been read out
        if (valid && !wmasked) {
#pragma unroll
          for (int kind = 0; kind < 3; ++kind)
            tma_store_3d(&L.tm_out, smem_u32(stg + 2 * kind * C::kTile), kind * Ap + u.h0 * DP, wj * 8 + u.s, b * g.H + wi * 8 + u.s);
          bulk_group_commit();
          pending = slot;                                  // released to the loader once the stores have read it
        } else if (valid && wrap_tma) {
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) {
            const int ri = pc >> 1, ci = pc & 1;
            int r0 = wi * 8 + u.s + ri * we, c0 = wj * 8 + u.s + ci * we;      // first token of the piece, shift undone
            if (r0 >= g.H) r0 -= g.H;
            if (c0 >= g.W) c0 -= g.W;
            const int prow0 = (ri ? 8 * we : 0) + (ci ? (ri ? u.s : we) * we : 0);   // first staging row of the piece
#pragma unroll
            for (int kind = 0; kind < 3; ++kind)
              tma_store_3d(&L.tm_wrap[pc], smem_u32(stg + 2 * kind * C::kTile + prow0 * C::kRB), kind * Ap + u.h0 * DP, c0, b * g.H + r0);
          }
          bulk_group_commit();
          pending = slot;
        } else {
          mbar_arrive(&inEmpty[slot]);
        }
      }
    }
    if (pending >= 0) {
      bulk_group_wait_read();
      mbar_arrive(&inEmpty[pending]);
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // shared memory must outlive the stores that read it

    // ---- gradient of the bias table: fold the summed dS of all rows through the relative-position map
    if (L.dtable != nullptr) {
#pragma unroll
      for (int k = 0; k < 32; k += 2) {
        float e0, e1;
        attn::upk2(dsum2[k >> 1], e0, e1);
        atomicAdd(hist + (qa - 4 * half - (k >> 3) + 7) * 15 + (qc - (k & 7) + 7), e0);
        atomicAdd(hist + (qa - 4 * half - ((k + 1) >> 3) + 7) * 15 + (qc - ((k + 1) & 7) + 7), e1);
      }
    }
    asm volatile("bar.sync 13, 512;" ::: "memory");        // all softmax warps
    if (L.dtable != nullptr && tid < 225) atomicAdd(L.dtable + tid * g.nh + u.h0, hist[tid]);
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kTcMmaWarp) {
    __syncwarp();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

size_t attn_bwd_tc_smem(int dp) { return dp == 32 ? TcCfg<32>::kSmem : TcCfg<16>::kSmem; }

template <int DP>
static int launch_bwd_tc_t(const AttnLaunch& L, cudaStream_t st) {
  const size_t smem = TcCfg<DP>::kSmem;
  if (cudaFuncSetAttribute(attn_bwd_tc_kernel<DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const long long npairs = (L.geo.n_windows + 1) / 2;
  long long gx = sms / L.nunits;
  if (gx < 1) gx = 1;
  if (gx > npairs) gx = npairs;
  { KernelScope ks_("attn_bwd", st);
    attn_bwd_tc_kernel<DP><<<dim3((unsigned)gx, L.nunits), kTcThreads, smem, st>>>(L); }
  return check_launch();
}

// One head per unit only (the planner builds such units whenever the head count allows).
int launch_attn_bwd_tc(const AttnLaunch& L, cudaStream_t st) {
  for (int i = 0; i < L.nunits; ++i)
    if (L.u[i].nheads != 1) return GSWA_ERR_UNSUPPORTED;
  if (L.geo.n_windows <= 0) return GSWA_OK;
  return L.geo.dp == 32 ? launch_bwd_tc_t<32>(L, st) : launch_bwd_tc_t<16>(L, st);
}

}  // namespace gswa
