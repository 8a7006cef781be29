// Projection GEMMs of the bf16 path on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// TMEM).  Three persistent, warp-specialised kernels share one structure:
//     epilogue warps   TMEM -> registers -> shared-memory staging -> global (one accumulator row per thread;
//                      four in gr_kernel, eight in gw_kernel and gt_kernel: two per 32-lane TMEM quadrant)
//     one MMA warp     one elected thread, tcgen05.mma + tcgen05.commit
//     producers        padded token-major buffers (attention output, dqkv) come by TMA from one thread; the
//                      caller's tensors (x, dy) have row pitches of 2C bytes (360 at C = 180), which cannot be
//                      described to TMA: eight loader warps fetch their rows with asynchronous 8- and 16-byte
//                      copies straight into the swizzled operand image, K padded on the fly
// Roles talk through mbarriers; every wait is bounded and reports through an error word.
//
//   gw_kernel  Eq. 6 projections (and dA = dy W^P): rows are gathered in WINDOW order of one head
//              group (cyclic shift + window partition as address arithmetic) and the epilogue writes
//              contiguous per-(window, head) tiles.
//   gt_kernel  Eq. 7 output projection (and dx = dqkv W_qkv): rows in token order, packed rows out.
//   gr_kernel  parameter gradients dW = sum_t L[t,:]^T R[t,:] with both operands MN-major, bias
//              gradients through a column of ones.
#include "gemm_core.cuh"
#include "gswa_index.cuh"

namespace gswa {
using namespace umma;
using namespace gemm;
namespace {
// ==========================================================================================
// gw_kernel
// ==========================================================================================
template <int CP, int DP>
__global__ void __launch_bounds__(kThreads2, 1) gw_kernel(const __grid_constant__ GWLaunch L) {
  // CTAs cta0[i] .. cta0[i+1]-1 work on unit i (units get CTAs in proportion to their work)
  int ui = 0;
  while (ui + 1 < kMaxUnits && (int)blockIdx.x >= L.cta0[ui + 1]) ++ui;
  const GWUnit& u = L.u[ui];
  const int bx = (int)blockIdx.x - L.cta0[ui], gxu = L.cta0[ui + 1] - L.cta0[ui];
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  constexpr int NA = CP / 64;                  // K atoms per tile
  const int NT = u.nchunks * u.cw;
  const int S = L.nslots;
  unsigned char* sB = sm;
  unsigned char* ring = sB + (size_t)NT * CP * 2;
  constexpr int kPiece = 32 * DP * 2;                      // 32 rows of one output block: contiguous in global memory
  unsigned char* stg = ring + (size_t)S * kAtomBytes;      // two pieces per epilogue warp
  float* sBias = reinterpret_cast<float*>(stg + (size_t)kEpi2 * 2 * kPiece);
  __shared__ uint64_t full[8], empty[8], tfull[8], tempty[8];
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < NT * CP * 2 / 16; i += kThreads2)
    reinterpret_cast<uint4*>(sB)[i] = __ldg(reinterpret_cast<const uint4*>(u.Bimg) + i);
  for (int i = tid; i < NT; i += kThreads2) sBias[i] = u.bias ? u.bias[i] : 0.f;
  fence_proxy_async();
  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 8; ++i) { mbar_init(&full[i], 2); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 8; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], kEpi2); }
    mbar_init_fence();
  }
  // TMEM holds a ring of RC accumulator chunks of cw columns; a tile takes nchunks consecutive ring
  // positions, so the MMAs of the next tile start while this tile's chunks are still being drained.
  const int RC = 512 / u.cw < 8 ? 512 / u.cw : 8;
  const uint32_t tcols = pow2_cols(RC * u.cw);
  if (warp == kEpi2) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;
  const long long n_tiles = (u.n_windows + 1) / 2;

  if (warp > kEpi2) {
    // ---------------- loaders
    const int set = (warp - kEpi2 - 1) >> 1;
    LoaderLane ll;
    ll.init(((warp - kEpi2 - 1) & 1) * 32 + lane);
    const char* const srcA = reinterpret_cast<const char*>(u.A);
    const long long row_bytes = (long long)u.lda * 2, line_bytes = (long long)u.W * row_bytes;
    // Rows of this thread that start on 16-byte boundaries: all, or those of even tokens.  The token parity of tile
    // row (a, c) is that of shift + c (image width and height are even), and c = rq or rq + 4 for all rows of a thread.
    const bool row16 = u.a16 == 2 || (u.a16 == 1 && ((u.s + ll.rq) & 1) == 0);
    const uint32_t ringA = smem_u32(ring);
    RingPos rp;
    rp.init(set, S);
    int g = set;                                 // ring step = tile iteration * NA + atom
    int it = 0;
    for (long long tile = bx; tile < n_tiles; tile += gxu, ++it) {
      // the two windows of the pair: cyclic shift + partition are this address arithmetic.  Tile row
      // r = 64*half + 8*a + lw holds slot (a, lw) of window `half`; this thread owns lw = rq and rq + 4.
      const char* col0[2][2];
      int i0[2];
      bool wv[2];
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int win = 2 * (int)tile + half;
        wv[half] = win < (int)u.n_windows;
        const int b = win / u.nW, w = win - b * u.nW;
        const int wi = w / u.nWw, wj = w - wi * u.nWw;
        i0[half] = wi * 8 + u.s;
#pragma unroll
        for (int v = 0; v < 2; ++v) {
          int j = wj * 8 + ll.rq + 4 * v + u.s;
          if (j >= u.W) j -= u.W;
          col0[half][v] = srcA + ((long long)b * u.H * u.W + j) * row_bytes + ll.pc * 8;
        }
      }
      bool ok = true;
      for (; g < (it + 1) * NA; g += kSets) {
        const int atom = g - it * NA;
        if (!wait_bar_warp(&empty[rp.slot], rp.ph ^ 1, &abort_s, L.err)) { ok = false; break; }
        const uint32_t dst = ringA + rp.slot * kAtomBytes;
        const bool cv = atom * 128 + ll.pc * 8 < u.kvalid * 2;      // inside the valid columns of a source row
        // rows on 16-byte boundaries: the even piece's thread copies both pieces of a fully valid 16-byte chunk
        const bool c16 = row16 && atom * 128 + (ll.pc | 1) * 8 < u.kvalid * 2;
        if (c16) {
          if ((ll.pc & 1) == 0) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const bool v = wv[half];
#pragma unroll
              for (int a8 = 0; a8 < 8; ++a8) {
                int i = i0[half] + a8;
                if (i >= u.H) i -= u.H;
                const long long off = i * line_bytes + atom * 128;
                const int k = 16 * half + 2 * a8;
                cp_async16(dst + ll.dst(k), v ? col0[half][0] + off : srcA, v);
                cp_async16(dst + ll.dst(k + 1), v ? col0[half][1] + off : srcA, v);
              }
            }
          }
        } else if (cv) {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const bool v = wv[half];
#pragma unroll
            for (int a8 = 0; a8 < 8; ++a8) {
              int i = i0[half] + a8;
              if (i >= u.H) i -= u.H;
              const long long off = i * line_bytes + atom * 128;
              const int k = 16 * half + 2 * a8;
              cp_async8(dst + ll.dst(k), v ? col0[half][0] + off : srcA, v);
              cp_async8(dst + ll.dst(k + 1), v ? col0[half][1] + off : srcA, v);
            }
          }
        } else {
          // K padding: zeros, except a one in column kvalid when the bias rides in the weight image's row kvalid
          const uint32_t w0 = (u.ones_col && atom * 64 + ll.pc * 4 == u.kvalid) ? 0x3F80u : 0u;
#pragma unroll
          for (int k = 0; k < 32; ++k)
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(dst + ll.dst(k)), "r"(w0), "r"(0u) : "memory");
        }
        cp_async_commit();
        cp_async_wait(0);
        publish(&full[rp.slot], lane);
        rp.advance(kSets, S);
      }
      if (!ok) break;
    }
    cp_async_wait(0);
  } else if (warp == kEpi2) {
    // ---------------- MMA issue.  Descriptors advance by adding to their address field.  All K atoms
    // of a tile are consumed accumulator by accumulator (switching the accumulator between
    // consecutive MMAs costs about as much as two MMAs of this width).
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, u.cw, 0, 0);
      const uint64_t a0 = make_desc(smem_u32(ring), 16, 1024), b0 = make_desc(smem_u32(sB), 16, 1024);
      RingPos rp;
      rp.init(0, S);
      int q = 0, qph = 0, qlast = 0;                               // ring position of the next chunk and its phase
      bool ok = true;
      for (long long tile = bx; tile < n_tiles && ok; tile += gxu) {
        int slot_a[NA];
        for (int c = 0; c < u.nchunks && ok; ++c) {
          if (!wait_bar(&tempty[q], qph ^ 1, &abort_s, L.err)) { ok = false; break; }
          fence_after_sync();
#pragma unroll
          for (int atom = 0; atom < NA; ++atom) {
            if (c == 0) {
              if (!wait_bar(&full[rp.slot], rp.ph, &abort_s, L.err)) { ok = false; break; }
              fence_after_sync();
              slot_a[atom] = rp.slot;
              rp.advance(1, S);
            }
            const uint64_t ad = a0 + (uint64_t)((slot_a[atom] * kAtomBytes) >> 4);
            const uint64_t bd = b0 + (uint64_t)(((atom * NT + c * u.cw) * 128) >> 4);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) mma_bf16(tmem + q * u.cw, ad + 2 * kk, bd + 2 * kk, idesc, (atom | kk) != 0);
          }
          qlast = q;
          if (++q == RC) { q = 0; qph ^= 1; }
        }
        if (!ok) break;
#pragma unroll
        for (int atom = 0; atom < NA; ++atom) commit(&empty[slot_a[atom]]);
        commit(&tfull[qlast]);                     // one completion signal per tile, on its last chunk
      }
    }
  } else {
    // ---------------- epilogue: accumulator row = (window of the pair, slot).  A warp owns 32 rows; the
    // 32 rows of one output block are contiguous in the global tile image, so the warp builds that
    // piece in its private staging buffer and ships it with one bulk copy (two buffers alternate).
    const int quad = warp & 3, half = warp >> 2;
    const int row = (quad & 1) * 32 + lane;       // slot inside the window
    const int nblk = u.cw / DP;
    unsigned char* mystg = stg + (size_t)warp * 2 * kPiece;
    const uint32_t mystgA = smem_u32(mystg);
    int nst = 0, q = 0, qph = 0;                  // q, qph: ring position of the next chunk and its phase
    // A tile's completion is signalled on the ring position of its LAST chunk only.  The last positions of
    // successive tiles cycle with period RC / gcd(nchunks, RC) tiles and visit every position of the cycle once,
    // so the barrier at a tile's last position has flipped (tile iteration / period) times before.
    int gcd_ = u.nchunks, rem_ = RC;
    while (rem_) { const int t_ = gcd_ % rem_; gcd_ = rem_; rem_ = t_; }
    const int period = RC / gcd_;
    int it = 0;
    bool ok = true;
    for (long long tile = bx; tile < n_tiles && ok; tile += gxu, ++it) {
      const long long win = 2 * tile + (quad >> 1);
      const bool valid = win < u.n_windows;
      __nv_bfloat16* obase = u.out + win * u.win_stride + (quad & 1) * 32 * DP;
      {
        // the tile is complete when its last chunk is (MMAs finish in issue order)
        int ql = q + u.nchunks - 1;
        if (ql >= RC) ql -= RC;
        if (!wait_bar_warp(&tfull[ql], (it / period) & 1, &abort_s, L.err)) break;
      }
      for (int c = 0; c < u.nchunks; ++c) {
        fence_after_sync();
        for (int blk = 0; blk < nblk; ++blk) {
          const int gb = c * nblk + blk;
          if ((gb & 1) != half) continue;          // the two warps of a quadrant alternate blocks
          uint32_t v[DP];
          const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + q * u.cw + blk * DP;
          if constexpr (DP == 32) tmem_ld32(taddr, v); else tmem_ld16(taddr, v);
          const int buf = nst & 1;
          if (nst >= 2) {                          // the copy that last read this buffer has finished reading
            if (lane == 0) bulk_wait_read1();
            __syncwarp();
          }
          tmem_ld_wait();
          unsigned char* piece = mystg + buf * kPiece - (quad & 1) * kPiece;   // tile_off counts rows from the block start
          const bool scaled = u.q_every3 && gb % 3 == 0;
          if (u.bias != nullptr) {                 // bias added here (no spare K column to carry it)
            const float sc = scaled ? u.qscale : 1.f;
#pragma unroll
            for (int j = 0; j < DP / 8; ++j) {
              const float4 b0v = *reinterpret_cast<const float4*>(sBias + gb * DP + 8 * j);
              const float4 b1v = *reinterpret_cast<const float4*>(sBias + gb * DP + 8 * j + 4);
              uint4 o;
              o.x = pack_bf16((__uint_as_float(v[8 * j]) + b0v.x) * sc, (__uint_as_float(v[8 * j + 1]) + b0v.y) * sc);
              o.y = pack_bf16((__uint_as_float(v[8 * j + 2]) + b0v.z) * sc, (__uint_as_float(v[8 * j + 3]) + b0v.w) * sc);
              o.z = pack_bf16((__uint_as_float(v[8 * j + 4]) + b1v.x) * sc, (__uint_as_float(v[8 * j + 5]) + b1v.y) * sc);
              o.w = pack_bf16((__uint_as_float(v[8 * j + 6]) + b1v.z) * sc, (__uint_as_float(v[8 * j + 7]) + b1v.w) * sc);
              *reinterpret_cast<uint4*>(piece + tile_off<DP>(row, j)) = o;
            }
          } else if (scaled) {
            const float sc = u.qscale;
#pragma unroll
            for (int j = 0; j < DP / 8; ++j) {
              uint4 o;
              o.x = pack_bf16(__uint_as_float(v[8 * j]) * sc, __uint_as_float(v[8 * j + 1]) * sc);
              o.y = pack_bf16(__uint_as_float(v[8 * j + 2]) * sc, __uint_as_float(v[8 * j + 3]) * sc);
              o.z = pack_bf16(__uint_as_float(v[8 * j + 4]) * sc, __uint_as_float(v[8 * j + 5]) * sc);
              o.w = pack_bf16(__uint_as_float(v[8 * j + 6]) * sc, __uint_as_float(v[8 * j + 7]) * sc);
              *reinterpret_cast<uint4*>(piece + tile_off<DP>(row, j)) = o;
            }
          } else {
#pragma unroll
            for (int j = 0; j < DP / 8; ++j) {
              uint4 o;
              o.x = pack_bf16(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1]));
              o.y = pack_bf16(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
              o.z = pack_bf16(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
              o.w = pack_bf16(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
              *reinterpret_cast<uint4*>(piece + tile_off<DP>(row, j)) = o;
            }
          }
          fence_proxy_async();                     // the bulk copy reads these stores through the async proxy
          __syncwarp();
          if (lane == 0) {
            if (valid) bulk_store(obase + (long long)gb * 64 * DP, mystgA + buf * kPiece, kPiece);
            else bulk_commit();
          }
          ++nst;
        }
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty[q]);
        if (++q == RC) { q = 0; qph ^= 1; }
      }
    }
    if (lane == 0) bulk_wait_all();
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kEpi2) {
    __syncwarp();
    tmem_dealloc(tmem, tcols);
  }
}

// ==========================================================================================
// gt_kernel
// ==========================================================================================

// Four bf16 sums in float arithmetic.
__device__ __forceinline__ uint2 add_bf16x4(uint2 a, uint2 b) {
  const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.x)), a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.y));
  const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.x)), b1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.y));
  return make_uint2(pack_bf16(a0.x + b0.x, a0.y + b0.y), pack_bf16(a1.x + b1.x, a1.y + b1.y));
}

__global__ void __launch_bounds__(kThreads2, 1) gt_kernel(const __grid_constant__ GTLaunch L) {
  const GTSplit& sp = L.s[blockIdx.y];
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  const int NB = L.NB, natoms = L.natoms, S = L.nstages;
  // The B operand (weight image) either stays resident in shared memory, or - when all its K atoms do not
  // fit beside the ring - travels through the ring with the A atoms: the image is small and lives in L2,
  // so streaming it costs no HBM traffic, whereas splitting N over several CTAs would make every one of
  // them read all of A.
  const bool stream = L.stream_b != 0;
  const int stage_bytes = kAtomBytes + (stream ? NB * 128 : 0);
  unsigned char* sB = sm;
  unsigned char* ring = sB + (stream ? 0 : (size_t)natoms * NB * 128);
  unsigned char* stg = ring + (size_t)S * stage_bytes;
  float* sBias = reinterpret_cast<float*>(stg + (size_t)128 * NB * 2);
  __shared__ uint64_t full[8], empty[8], tfull[2], tempty[2];
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (!stream)
    for (int i = tid; i < natoms * NB * 8; i += kThreads2)
      reinterpret_cast<uint4*>(sB)[i] = __ldg(reinterpret_cast<const uint4*>(sp.Bimg) + i);
  for (int i = tid; i < NB; i += kThreads2) sBias[i] = sp.bias ? sp.bias[i] : 0.f;
  fence_proxy_async();
  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 8; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], kEpi2); }
    mbar_init_fence();
  }
  const uint32_t tcols = pow2_cols(2 * NB);
  if (warp == kEpi2) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;
  const long long n_tiles = (L.rows + 127) / 128;

  if (warp > kEpi2) {
    // ---------------- producer: one thread asks TMA for one K atom (64 columns x 128 rows, swizzled on
    // the way in) per ring step; rows past the end of the tensor arrive as zeros
    if (warp == kEpi2 + 1 && lane == 0) {
      const uint32_t ringA = smem_u32(ring);
      RingPos rp;
      rp.init(0, S);
      bool ok = true;
      for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        for (int atom = 0; atom < natoms; ++atom) {
          if (!wait_bar(&empty[rp.slot], rp.ph ^ 1, &abort_s, L.err)) { ok = false; break; }
          mbar_arrive_expect_tx(&full[rp.slot], (uint32_t)stage_bytes);
          tma_load_2d(ringA + rp.slot * stage_bytes, &L.tmA, atom * 64, (int)(tile * 128), &full[rp.slot]);
          if (stream)
            bulk_load(ringA + rp.slot * stage_bytes + kAtomBytes, sp.Bimg + (size_t)atom * NB * 128, (uint32_t)NB * 128u, &full[rp.slot]);
          rp.advance(1, S);
        }
      }
    }
  } else if (warp == kEpi2) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, NB, 0, 0);
      const uint64_t a0 = make_desc(smem_u32(ring), 16, 1024), b0 = make_desc(smem_u32(sB), 16, 1024);
      RingPos rp;
      rp.init(0, S);
      int it = 0;
      bool ok = true;
      for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
        const int buf = it & 1;
        if (!wait_bar(&tempty[buf], ((it >> 1) & 1) ^ 1, &abort_s, L.err)) break;
        fence_after_sync();
        for (int atom = 0; atom < natoms; ++atom) {
          if (!wait_bar(&full[rp.slot], rp.ph, &abort_s, L.err)) { ok = false; break; }
          fence_after_sync();
          const uint64_t ad = a0 + (uint64_t)((rp.slot * stage_bytes) >> 4);
          const uint64_t bd = stream ? ad + (kAtomBytes >> 4) : b0 + (uint64_t)((atom * NB * 128) >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) mma_bf16(tmem + buf * NB, ad + 2 * kk, bd + 2 * kk, idesc, (atom | kk) != 0);
          commit(&empty[rp.slot]);
          rp.advance(1, S);
        }
        if (ok) commit(&tfull[buf]);
      }
    }
  } else {
    // ---------------- epilogue: stage the warp's 32 rows in shared memory, then store row pieces
    const int ncols = sp.ncols, n8 = ncols / 4;
    const int quad = warp & 3, half = warp >> 2;
    unsigned char* mystg = stg + (size_t)quad * 32 * ncols * 2;
    int it = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      const int buf = it & 1;
      // the vote is also the barrier after which last tile's staging rows may be overwritten
      if (!pair_vote(quad, wait_bar_warp(&tfull[buf], (it >> 1) & 1, &abort_s, L.err))) break;
      fence_after_sync();
      for (int c0 = 32 * half; c0 < ncols; c0 += 64) {   // the two warps of a quadrant alternate column chunks
        uint32_t v[32];
        tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + buf * NB + c0, v);
        tmem_ld_wait();
        // the lane's row of the staging tile; rows are 2*ncols bytes apart (a multiple of 8, and an
        // odd multiple for C = 180, so these 8-byte stores do not collide on banks)
        uint2* dst = reinterpret_cast<uint2*>(mystg + ((size_t)lane * ncols + c0) * 2);
        if (sp.bias != nullptr) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (c0 + 4 * j < ncols) {
              const float4 bq = *reinterpret_cast<const float4*>(sBias + c0 + 4 * j);
              dst[j] = make_uint2(pack_bf16(__uint_as_float(v[4 * j]) + bq.x, __uint_as_float(v[4 * j + 1]) + bq.y),
                                  pack_bf16(__uint_as_float(v[4 * j + 2]) + bq.z, __uint_as_float(v[4 * j + 3]) + bq.w));
            }
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (c0 + 4 * j < ncols)
              dst[j] = make_uint2(pack_bf16(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1])),
                                  pack_bf16(__uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
        }
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[buf]);
      pair_sync(quad);                           // both halves of the staging rows are written
      // copy-out: lane = 8-byte piece of a row (two pieces per lane cover up to 256 columns); each
      // warp of the pair stores 16 of the quadrant's 32 rows
      const long long trow0 = tile * 128 + quad * 32;
      const int nrows = L.rows - trow0 < 32 ? (int)(L.rows - trow0) : 32;
      char* const obase = reinterpret_cast<char*>(L.out + trow0 * L.ldo + sp.col0) + lane * 8;
      const long long obytes = (long long)L.ldo * 2;
      const unsigned char* sbase = mystg + lane * 8;
      const bool p0 = lane < n8, p1 = lane + 32 < n8;
      const int rend = nrows < 16 * half + 16 ? nrows : 16 * half + 16;
      if (L.resid == nullptr) {
#pragma unroll 4
        for (int rr = 16 * half; rr < rend; ++rr) {
          if (p0) *reinterpret_cast<uint2*>(obase + rr * obytes) = *reinterpret_cast<const uint2*>(sbase + rr * ncols * 2);
          if (p1)
            *reinterpret_cast<uint2*>(obase + rr * obytes + 256) =
                *reinterpret_cast<const uint2*>(sbase + rr * ncols * 2 + 256);
        }
      } else {
        // skip connection: the residual rows have the layout of the output rows
        const char* const rbase = reinterpret_cast<const char*>(L.resid + trow0 * L.ldo + sp.col0) + lane * 8;
#pragma unroll 4
        for (int rr = 16 * half; rr < rend; ++rr) {
          if (p0)
            *reinterpret_cast<uint2*>(obase + rr * obytes) =
                add_bf16x4(*reinterpret_cast<const uint2*>(sbase + rr * ncols * 2), __ldg(reinterpret_cast<const uint2*>(rbase + rr * obytes)));
          if (p1)
            *reinterpret_cast<uint2*>(obase + rr * obytes + 256) =
                add_bf16x4(*reinterpret_cast<const uint2*>(sbase + rr * ncols * 2 + 256), __ldg(reinterpret_cast<const uint2*>(rbase + rr * obytes + 256)));
        }
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kEpi2) {
    __syncwarp();
    tmem_dealloc(tmem, tcols);
  }
}

// ==========================================================================================
// gr_kernel
// ==========================================================================================
__device__ __forceinline__ void red_add_f32(float* p, float a) {
  asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(p), "f"(a) : "memory");
}
__device__ __forceinline__ void red_add_v4(float* p, float4 v) {
  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void red_add_v2(float* p, float a, float b) {
  asm volatile("red.relaxed.gpu.global.add.v2.f32 [%0], {%1, %2};" ::"l"(p), "f"(a), "f"(b) : "memory");
}
// Padded index (kind, head, c) -> kind*C + head*d + c, or -1 for a pad column.
__device__ __forceinline__ int unpad_index(int idx, int Ap, int dp, int d, int C) {
  const int kind = idx / Ap, rem = idx - kind * Ap;
  const int h = rem / dp, c = rem - h * dp;
  return c < d ? kind * C + h * d + c : -1;
}

__global__ void __launch_bounds__(kThreadsR, 1) gr_kernel(const __grid_constant__ GRLaunch L) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  const int NP = L.NP, ratoms = NP / 64;
  const int MB = L.mbpc, latoms = 2 * MB;                  // M blocks of 128 per CTA: the other operand is fetched once for all of them
  // Two rings of 64-token stages: one for the padded operand that TMA fetches (deep, because those bytes
  // come from HBM with microseconds of latency), one for the caller's tensor that the loader sets copy.
  const int tma_atoms_all = L.tma_is_L ? latoms : ratoms;
  const int copy_atoms = L.tma_is_L ? ratoms : latoms;
  const int tbytes = tma_atoms_all * 8192, cbytes = copy_atoms * 8192;
  const int ST = L.nstages, SC = kSets;
  unsigned char* ringT = sm;
  unsigned char* ringC = sm + (size_t)ST * tbytes;
  __shared__ uint64_t fullT[8], emptyT[8], fullC[kSets], emptyC[kSets], done;
  __shared__ int rowmap[256], colmap[256];
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mb = blockIdx.y * MB;                          // first M block of this CTA
  long long chunk = (L.rows + L.nsplit - 1) / L.nsplit;
  chunk = (chunk + 63) / 64 * 64;
  const long long t0 = (long long)blockIdx.x * chunk;
  const long long t1 = t0 + chunk < L.rows ? t0 + chunk : L.rows;
  if (t0 >= t1) return;
  const int nst = (int)((t1 - t0 + 63) / 64);
  const int tma_cols = L.tma_is_L ? L.M - mb * 128 : L.Ap;                 // valid columns of the TMA-fed operand here
  const int tma_atoms = (tma_cols + 63) / 64 < tma_atoms_all ? (tma_cols + 63) / 64 : tma_atoms_all;

  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 8; ++i) { mbar_init(&fullT[i], 1); mbar_init(&emptyT[i], 1); }
    for (int i = 0; i < kSets; ++i) { mbar_init(&fullC[i], 2); mbar_init(&emptyC[i], 1); }
    mbar_init(&done, 1);
    mbar_init_fence();
  }
  const uint32_t tcols = pow2_cols(MB * NP);
  if (warp == kEpiWarps) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;

  if (warp == kEpiWarps + 1) {
    // ---------------- TMA producer: 64-token boxes of the padded operand, as far ahead as the ring allows.
    // Atoms that lie wholly outside the tensor are never requested: they are zeroed once.
    for (int sgi = 0; sgi < ST; ++sgi)
      for (int a = tma_atoms; a < tma_atoms_all; ++a) {
        unsigned char* at = ringT + (size_t)sgi * tbytes + a * 8192;
        for (int e = lane; e < 8192 / 16; e += 32) reinterpret_cast<uint4*>(at)[e] = make_uint4(0u, 0u, 0u, 0u);
      }
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      RingPos rp;
      rp.init(0, ST);
      for (int s = 0; s < nst; ++s) {
        if (!wait_bar_nap(&emptyT[rp.slot], rp.ph ^ 1, &abort_s, L.err)) break;
        const uint32_t dst = smem_u32(ringT + (size_t)rp.slot * tbytes);
        mbar_arrive_expect_tx(&fullT[rp.slot], (uint32_t)tma_atoms * 8192u);
        for (int a = 0; a < tma_atoms; ++a)
          tma_load_2d(dst + a * 8192, &L.tm, (L.tma_is_L ? mb * 128 : 0) + a * 64, (int)(t0 + (long long)s * 64), &fullT[rp.slot]);
        rp.advance(1, ST);
      }
    }
  } else if (warp > kEpiWarps + 1) {
    // ---------------- loader sets for the caller's tensor: set q fills copy-ring steps q, q+4, ... (slot q)
    const int set = (warp - kEpiWarps - 2) >> 1;
    const int ts = ((warp - kEpiWarps - 2) & 1) * 32 + lane;
    LoaderLane4 ll;
    ll.init(ts);
    const int copy_col0 = L.tma_is_L ? 0 : mb * 128;                       // first column of the copy-fed operand here
    unsigned char* base = ringC + (size_t)set * cbytes;
    // Pieces that never change (padding, the ones column) are written once, before the loop.
    for (int a = 0; a < copy_atoms; ++a)
      for (int half = 0; half < 2; ++half) {
        const int col = copy_col0 + a * 64 + ll.pp * 8 + half * 4;
        if (col < L.pvalid) continue;
        const uint2 val = make_uint2((L.tma_is_L && col == L.pvalid) ? 0x3F80u : 0u, 0u);
#pragma unroll
        for (int k = 0; k < 8; ++k) *reinterpret_cast<uint2*>(base + a * 8192 + ll.dst0 + k * 1024 + half * 8) = val;
      }
    const char* const srcP = reinterpret_cast<const char*>(L.P);
    const long long prow = (long long)L.ldp * 2;
    // rows of this thread that start on 16-byte boundaries: all of them, the even ones (its rows all have lw's parity), or none
    const bool row16 = L.p16 == 2 || (L.p16 == 1 && (ll.lw & 1) == 0);
    const uint32_t sS = smem_u32(base);
    int ph = 0;
    for (int s = set; s < nst; s += kSets, ph ^= 1) {
      if (!wait_bar_warp_nap(&emptyC[set], ph ^ 1, &abort_s, L.err)) break;
      const long long tb = t0 + (long long)s * 64;
      const char* pp = srcP + (tb + ll.lw) * prow + (copy_col0 + ll.pp * 8) * 2;
      const bool whole = tb + 64 <= t1;
      for (int a = 0; a < copy_atoms; ++a) {
        const int col = copy_col0 + a * 64 + ll.pp * 8;
        const bool v0 = col < L.pvalid, v1 = col + 4 < L.pvalid;
        if (!v0) break;
        const uint32_t dst = sS + a * 8192 + ll.dst0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const bool tv = whole || tb + ll.lw + 8 * k < t1;
          const char* src = pp + k * 8 * prow + a * 128;
          if (row16 && v1) {
            cp_async16(dst + k * 1024, tv ? src : srcP, tv);
          } else {
            cp_async8(dst + k * 1024, tv ? src : srcP, tv);
            if (v1) cp_async8(dst + k * 1024 + 8, tv ? src + 8 : srcP, tv);
          }
        }
      }
      cp_async_commit();
      cp_async_wait(0);
      publish(&fullC[set], lane);
    }
    cp_async_wait(0);
  } else if (warp == kEpiWarps) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, NP, 1, 1);
      RingPos rt;
      rt.init(0, ST);
      bool ok = true;
      for (int s = 0; s < nst; ++s) {
        const int sc = s & (kSets - 1), pc = (s / kSets) & 1;
        if (!wait_bar_nap(&fullT[rt.slot], rt.ph, &abort_s, L.err) || !wait_bar_nap(&fullC[sc], pc, &abort_s, L.err)) { ok = false; break; }
        fence_after_sync();
        const uint32_t tAddr = smem_u32(ringT + (size_t)rt.slot * tbytes), cAddr = smem_u32(ringC + (size_t)sc * cbytes);
        const uint32_t lAddr = L.tma_is_L ? tAddr : cAddr, rAddr = L.tma_is_L ? cAddr : tAddr;
        const uint64_t bd = make_desc(rAddr, 8192, 1024);
        for (int blk = 0; blk < MB; ++blk) {
          const uint64_t ad = make_desc(lAddr + blk * 2 * 8192, 8192, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) mma_bf16(tmem + blk * NP, ad + kk * 128, bd + kk * 128, idesc, (s | kk) != 0);
        }
        commit(&emptyT[rt.slot]);
        commit(&emptyC[sc]);
        rt.advance(1, ST);
      }
      if (ok) commit(&done);
    }
  } else {
    // caller indices of this CTA's accumulator rows and columns (-1: padding, -2: the ones column)
    {
      const int ones = L.tma_is_L ? L.pvalid : (L.d < L.dp ? L.d : -1);
      for (int i = tid; i < MB * 128; i += kEpiWarps * 32) {
        const int mi = mb * 128 + i;
        rowmap[i] = L.tma_is_L ? (mi < L.M ? unpad_index(mi, L.Ap, L.dp, L.d, L.C) : -1) : (mi < L.M ? mi : -1);
      }
      for (int ni = tid; ni < NP; ni += kEpiWarps * 32)
        colmap[ni] = ni == ones ? -2 : (L.tma_is_L ? (ni < L.C ? ni : -1) : (ni < L.Ap ? unpad_index(ni, L.Ap, L.dp, L.d, L.C) : -1));
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    if (wait_bar_warp_nap(&done, 0, &abort_s, L.err)) {
      fence_after_sync();
      {
        // Atomic accumulation into the caller's gradients.  The padded row and column indices were turned into
        // caller indices once, while the MMAs ran (rowmap, colmap); each 32 x 32 block goes through shared memory
        // so that eight lanes add the 32 consecutive columns of one row with 16-byte vector reductions (the L2
        // atomic units, not DRAM, bound this tail: every CTA adds its whole accumulator into the same addresses).
        float* tp = reinterpret_cast<float*>(sm) + warp * 32 * 36;
        const int l8 = lane & 7, r4 = lane >> 3;              // 8 lanes x 4 columns cover a row's 32 columns; 4 rows per instruction
        for (int blk = 0; blk < MB; ++blk)
          for (int c0 = 0; c0 < NP; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + blk * NP + c0, v);
            tmem_ld_wait();
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(tp + lane * 36 + j) =
                  make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
            __syncwarp();
            const int n0 = colmap[c0 + 4 * l8], n3 = colmap[c0 + 4 * l8 + 3];
            const bool run4 = n0 >= 0 && n3 == n0 + 3;                               // four consecutive targets
            const bool vec = run4 && ((L.C & 3) == 0) && ((n0 & 3) == 0);            // ... 16-byte aligned
            const bool pair = run4 && ((L.C & 1) == 0) && ((n0 & 1) == 0);           // ... or at least 8-byte aligned
#pragma unroll 4
            for (int rr = 0; rr < 32; rr += 4) {
              const int r = rr + r4;
              const int m = rowmap[blk * 128 + warp * 32 + r];
              if (m < 0) continue;
              const float4 val = *reinterpret_cast<const float4*>(tp + r * 36 + 4 * l8);
              float* o = L.out + (long long)m * L.C;
              if (vec) {
                red_add_v4(o + n0, val);
              } else if (pair) {
                red_add_v2(o + n0, val.x, val.y);
                red_add_v2(o + n0 + 2, val.z, val.w);
              } else {
                const float e[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const int n = colmap[c0 + 4 * l8 + k];
                  if (n >= 0) red_add_f32(o + n, e[k]);
                  else if (n == -2 && L.colsum != nullptr) atomicAdd(L.colsum + m, e[k]);
                }
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
  int* err_word;               // or nullptr: 64 ints zeroed by block (0, 0)
};

// Value of image element (row n, K index k) and of the bias that goes with row n.
__device__ __forceinline__ float prep_value(const PrepJob& p, int n, int k, int ldp, int dmask) {
  const int C = p.C;
  if (p.mode == PREP_QKV) {            // row n = (head, q|k|v, c) of W_qkv; k = input channel
    const int blk = n >> ldp, c = n & dmask, h = p.h0 + blk / 3, kind = blk % 3;
    if (c < p.d && k < C) return __bfloat162float(p.W[(long long)(kind * C + h * p.d + c) * C + k]);
    if (c < p.d && k == C && p.fold_bias && p.b != nullptr) return __bfloat162float(p.b[kind * C + h * p.d + c]);   // meets the ones column of the A operand
  } else if (p.mode == PREP_PROJ_T) {  // row n = (head, c) -> input channel of W_proj; k = output channel
    const int h = p.h0 + (n >> ldp), c = n & dmask;
    if (c < p.d && k < C) return __bfloat162float(p.W[(long long)k * C + h * p.d + c]);
  } else if (p.mode == PREP_PROJ) {    // row n = output channel n0+n of W_proj; k = padded (head, c) input index
    const int h = k >> ldp, c = k & dmask;
    if (p.n0 + n < C && k < p.Ap && c < p.d) return __bfloat162float(p.W[(long long)(p.n0 + n) * C + h * p.d + c]);
    if (p.n0 + n < C && k == p.d && p.fold_bias && p.b != nullptr) return __bfloat162float(p.b[p.n0 + n]);   // meets the ones in column d of head 0 of A
  } else {                             // PREP_QKV_T: row n = input channel n0+n; k = padded (kind, head, c) row of W_qkv
    const int kind = (k >= p.Ap) + (k >= 2 * p.Ap), rem = k - kind * p.Ap, h = rem >> ldp, c = rem & dmask;
    if (p.n0 + n < C && k < 3 * p.Ap && c < p.d) return __bfloat162float(p.W[(long long)(kind * C + h * p.d + c) * C + p.n0 + n]);
  }
  return 0.f;
}

// Threads run along the index that is contiguous in the source weight (k for the plain images, n for the
// transposed ones), blocks along the other; the padded head width is a power of two, so nothing divides per element.
__global__ void __launch_bounds__(256) prep_kernel(const __grid_constant__ PrepJobs J) {
  const PrepJob& p = J.j[blockIdx.y];
  if (J.err_word != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < 64) J.err_word[threadIdx.x] = 0;
  const int ldp = p.dp == 32 ? 5 : 4, dmask = p.dp - 1;
  const bool transposed = p.mode == PREP_PROJ_T || p.mode == PREP_QKV_T;
  const int nouter = transposed ? p.KP : p.NT, ninner = transposed ? p.NT : p.KP;
  for (int o = blockIdx.x; o < nouter; o += gridDim.x)
    for (int i = threadIdx.x; i < ninner; i += blockDim.x) {
      const int n = transposed ? i : o, k = transposed ? o : i;
      *reinterpret_cast<__nv_bfloat16*>(p.img + (size_t)(k >> 6) * p.NT * 128 + sw128_offset(n, k & 63)) =
          __float2bfloat16_rn(prep_value(p, n, k, ldp, dmask));
    }
  if (p.bias_out != nullptr)
    for (int n = blockIdx.x * blockDim.x + threadIdx.x; n < p.NT; n += gridDim.x * blockDim.x) {
      float bv = 0.f;
      if (p.b != nullptr && !p.fold_bias) {
        if (p.mode == PREP_QKV) {
          const int blk = n >> ldp, c = n & dmask, h = p.h0 + blk / 3, kind = blk % 3;
          if (c < p.d) bv = __bfloat162float(p.b[kind * p.C + h * p.d + c]);
        } else if (p.mode == PREP_PROJ) {
          if (p.n0 + n < p.C) bv = __bfloat162float(p.b[p.n0 + n]);
        }
      }
      p.bias_out[n] = bv;
    }
}

}  // namespace

int launch_prep(const PrepJob* jobs, int njobs, cudaStream_t st, int* err_word) {
  if (njobs <= 0) return GSWA_OK;
  if (njobs > 16) return GSWA_ERR_UNSUPPORTED;
  PrepJobs J{};
  for (int i = 0; i < njobs; ++i) J.j[i] = jobs[i];
  J.err_word = err_word;
  { KernelScope ks_("prep_weights", st); prep_kernel<<<dim3(96, njobs), 256, 0, st>>>(J); }
  return check_launch();
}

static int num_sms() { return device_sm_count(); }

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
  const size_t fixed = 1024 + (size_t)maxNT * CP * 2 + (size_t)kEpi2 * 2 * 32 * DP * 2 + (size_t)maxNT * 4 + 64;
  int nslots = (int)((215 * 1024 - fixed) / (128 * 128));
  if (nslots > 8) nslots = 8;
  if (nslots < CP / 64 + 1 || nslots < 4) return GSWA_ERR_UNSUPPORTED;
  const size_t smem = fixed + (size_t)nslots * 128 * 128;
  if (cudaFuncSetAttribute(gw_kernel<CP, DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  GWLaunch Lc = L;
  Lc.nslots = nslots;
  for (int i = 0; i < nunits; ++i) {      // 16-byte copies need 16-byte aligned sources (see the loaders)
    const GWUnit& un = L.u[i];
    Lc.u[i].a16 = (reinterpret_cast<uintptr_t>(un.A) & 15) != 0 || (un.W & 1) || (un.H & 1) ? 0 : ((un.lda * 2) % 16 == 0 ? 2 : ((un.lda * 2) % 16 == 8 ? 1 : 0));
  }
  // One CTA per SM; a unit's share of them follows its work per tile (the loads and MMA issue every unit pays,
  // plus an epilogue proportional to its columns), so that all units finish together.
  double wsum = 0, w[kMaxUnits];
  for (int i = 0; i < nunits; ++i) { w[i] = 160.0 + L.u[i].nchunks * L.u[i].cw; wsum += w[i]; }
  const int total = num_sms() < nunits ? nunits : num_sms();
  int given = 0;
  Lc.cta0[0] = 0;
  for (int i = 0; i < nunits; ++i) {
    int c = i + 1 == nunits ? total - given : (int)(total * w[i] / wsum + 0.5);
    const long long t = (L.u[i].n_windows + 1) / 2;
    if (c < 1) c = 1;
    if (c > t && t > 0) c = (int)t;
    given += c;
    Lc.cta0[i + 1] = given;
  }
  for (int i = nunits + 1; i <= kMaxUnits; ++i) Lc.cta0[i] = given;
  { KernelScope ks_(name, st); gw_kernel<CP, DP><<<dim3((unsigned)given), kThreads2, smem, st>>>(Lc); }
  return check_launch();
}

int launch_gw(const GWLaunch& L, int nunits, int Cp, int dp, cudaStream_t st, const char* name) {
#define GW_CASE(CPV)                                                        \
  if (Cp == CPV) return dp == 32 ? launch_gw_t<CPV, 32>(L, nunits, st, name) : launch_gw_t<CPV, 16>(L, nunits, st, name);
  GW_CASE(64) GW_CASE(128) GW_CASE(192) GW_CASE(256)
#undef GW_CASE
  return GSWA_ERR_UNSUPPORTED;
}

size_t gt_smem_bytes(int natoms, int NB, int nstages, int stream_b) {
  return 1024 + (stream_b ? 0 : (size_t)natoms * NB * 128) + (size_t)nstages * (kAtomBytes + (stream_b ? (size_t)NB * 128 : 0)) +
         (size_t)128 * NB * 2 + (size_t)NB * 4 + 64;
}

typedef CUresult (*TmapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static TmapEncodeFn tmap_encoder() {
  static TmapEncodeFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return nullptr;
    }
    fn = reinterpret_cast<TmapEncodeFn>(p);
  }
  return fn;
}

int make_tmap(CUtensorMap* tm, const void* base, long long rows, int cols, int box_rows) {
  const TmapEncodeFn fn = tmap_encoder();
  if (fn == nullptr) return GSWA_ERR_CUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t es[2] = {1u, 1u};
  const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? GSWA_OK : GSWA_ERR_CUDA;
}

int make_tmap_window(CUtensorMap* tm, const void* base, long long img_rows, int W, int cols, int dp, int box_w, int box_h,
                     bool swizzled) {
  const TmapEncodeFn fn = tmap_encoder();
  if (fn == nullptr) return GSWA_ERR_CUDA;
  const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)W, (cuuint64_t)img_rows};
  const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * (cuuint64_t)W};
  const cuuint32_t box[3] = {(cuuint32_t)dp, (cuuint32_t)box_w, (cuuint32_t)box_h};
  const cuuint32_t es[3] = {1u, 1u, 1u};
  const CUtensorMapSwizzle sw = !swizzled ? CU_TENSOR_MAP_SWIZZLE_NONE : (dp == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? GSWA_OK : GSWA_ERR_CUDA;
}

int launch_gt(const GTLaunch& L, int nsplits, cudaStream_t st, const char* name) {
  const size_t smem = gt_smem_bytes(L.natoms, L.NB, L.nstages, L.stream_b);
  if (cudaFuncSetAttribute(gt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  const long long n_tiles = (L.rows + 127) / 128;
  long long gx = num_sms() / nsplits;
  if (gx < 1) gx = 1;
  if (gx > n_tiles) gx = n_tiles;
  { KernelScope ks_(name, st); gt_kernel<<<dim3((unsigned)gx, nsplits), kThreads2, smem, st>>>(L); }
  return check_launch();
}

int launch_gr(const GRLaunch& L, cudaStream_t st, const char* name) {
  GRLaunch Lc = L;
  if (L.NP > 256 || L.NP % 64 != 0) return GSWA_ERR_UNSUPPORTED;      // N extent of one tcgen05.mma
  if (Lc.mbpc < 1 || Lc.mbpc * L.NP > 512) Lc.mbpc = 1;
  // 16-byte copies need 16-byte aligned sources: the base, and a row pitch of 0 (every row) or 8 (even rows) mod 16
  Lc.p16 = (reinterpret_cast<uintptr_t>(L.P) & 15) != 0 ? 0 : ((L.ldp * 2) % 16 == 0 ? 2 : ((L.ldp * 2) % 16 == 8 ? 1 : 0));
  const int latoms = 2 * Lc.mbpc, ratoms = L.NP / 64;
  const size_t tbytes = (size_t)(L.tma_is_L ? latoms : ratoms) * 8192, cbytes = (size_t)(L.tma_is_L ? ratoms : latoms) * 8192;
  const size_t budget = 215 * 1024;
  if (budget < 1024 + kSets * cbytes + 2 * tbytes) return GSWA_ERR_UNSUPPORTED;
  Lc.nstages = (int)((budget - 1024 - kSets * cbytes) / tbytes);      // TMA ring depth
  if (Lc.nstages > 8) Lc.nstages = 8;
  const size_t smem = 1024 + (size_t)Lc.nstages * tbytes + kSets * cbytes + 64;
  if (cudaFuncSetAttribute(gr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  const int mblocks = ((L.M + 127) / 128 + Lc.mbpc - 1) / Lc.mbpc;
  { KernelScope ks_(name, st); gr_kernel<<<dim3(L.nsplit, mblocks), kThreadsR, smem, st>>>(Lc); }
  return check_launch();
}

}  // namespace gswa
