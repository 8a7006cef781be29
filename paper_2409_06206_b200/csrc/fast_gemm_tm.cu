// Window-order projection GEMM with the A operand in tensor memory (Eq. 6 projections q|k|v = x W^T, and
// dO = dy W^P in the backward pass).
//
// The caller's activation rows are 2C bytes apart (360 at C = 180): no tensor map can describe them and no
// shared-memory operand layout of the tensor core matches a linear [token][C] image.  tcgen05.mma can, however,
// read its A operand from TMEM, where row i of A sits in lane i with its K elements packed two per column - which
// is exactly what a thread that owns one token row can write with tcgen05.st.  So:
//     producer (4 lanes)      bulk asynchronous copies of whole window rows (8 tokens = 16C contiguous bytes; a
//                             window that wraps round the image edge as two pieces) into a ring of quarter-tile
//                             stages in shared memory: cyclic shift + window partition are these source addresses
//     8 converter warps       one thread per token row: row -> registers -> TMEM (K padded with zeros, a one in
//                             column C when the bias rides in the weight image); the two groups of four warps
//                             alternate tiles and A buffers
//     MMA warp                one thread: A from TMEM, B (the resident weight image) from shared memory, one
//                             accumulator chunk per head, chunk ring in TMEM
//     16 epilogue warps       TMEM -> bf16 -> per-(window, head, kind) tile images, 16-byte stores from registers
// A unit is a whole head group (all its heads' columns, up to what TMEM holds), so x is fetched once per group.
// Needs every piece of a window row to start and end on 16-byte boundaries: 2C * shift a multiple of 16.
#include "gemm_core.cuh"
#include "gswa_index.cuh"

namespace gswa {
using namespace umma;
using namespace gemm;
namespace {

constexpr int kConvWarps = 8, kEpiW = 16;
constexpr int kMmaWarp = kConvWarps + kEpiW, kProdWarp = kMmaWarp + 1;
constexpr int kThreadsTM = 32 * (kProdWarp + 1);      // 832
// Every converter warp owns its quarter-tile stages (stage = warp + 8 k): a stage's uses are then waited for by
// one warp in order, and a parity wait can never be satisfied by the phase before the one it means.  (A ring shared
// between warps allows exactly that: the warp that waits for use n+1 of a stage may arrive while use n is still in
// flight, and the parity of the phase before use n equals that of use n+1.)
constexpr int kMaxStages = 16, kMinStages = 8;
constexpr size_t kTmSmemBudget = 227 * 1024 - 1024;     // dynamic shared memory: the block's limit less its static variables

template <int CP, int DP>
__global__ void __launch_bounds__(kThreadsTM, 1) gwt_kernel(const __grid_constant__ GWLaunch L) {
  int ui = 0;
  while (ui + 1 < kMaxUnits && (int)blockIdx.x >= L.cta0[ui + 1]) ++ui;
  const GWUnit& u = L.u[ui];
  const int bx = (int)blockIdx.x - L.cta0[ui], gxu = L.cta0[ui + 1] - L.cta0[ui];
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  constexpr int NA = CP / 64;                           // K atoms
  constexpr int AW = CP / 2;                            // TMEM columns of one A buffer
  const int NT = u.nchunks * u.cw;
  const int S = L.nslots;                               // quarter-tile stages: 8 or 16 (one or two per converter warp)
  const int KS = S >> 3;
  const int row_bytes = u.lda * 2, qbytes = 32 * row_bytes;
  unsigned char* sB = sm;                               // weight image [NA][NT][128 B]
  unsigned char* stage = sB + (size_t)NT * CP * 2;
  float* sBias = reinterpret_cast<float*>(stage + (((size_t)S * qbytes + 127) & ~(size_t)127));
  __shared__ uint64_t sfull[kMaxStages], sempty[kMaxStages], afull[2], aempty[2], tfull[8], tempty[8];
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < NT * CP * 2 / 16; i += kThreadsTM)
    reinterpret_cast<uint4*>(sB)[i] = __ldg(reinterpret_cast<const uint4*>(u.Bimg) + i);
  for (int i = tid; i < NT; i += kThreadsTM) sBias[i] = u.bias ? u.bias[i] : 0.f;
  fence_proxy_async();
  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < kMaxStages; ++i) { mbar_init(&sfull[i], 1); mbar_init(&sempty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&afull[i], kConvWarps / 2); mbar_init(&aempty[i], 1); }
    for (int i = 0; i < 8; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], kEpiW); }
    mbar_init_fence();
  }
  // TMEM: two A buffers of AW columns, then a ring of RC accumulator chunks of cw columns; a tile takes nchunks
  // consecutive ring positions, so the next tile's first chunks are computed while this tile's last are drained.
  int RC = (512 - CP) / u.cw;
  if (RC > 8) RC = 8;
  const uint32_t tcols = pow2_cols(CP + RC * u.cw);
  if (warp == kMmaWarp) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;
  const long long n_tiles = (u.n_windows + 1) / 2;

  if (warp < kConvWarps) {
    // ---------------- converters: group `grp` takes the tiles with the same parity of the iteration count and
    // A buffer `grp`; warp `quad` of the group owns tile rows 32*quad .. +31 = one quarter-tile stage
    const int grp = warp >> 2, quad = warp & 3;
    const int npieces = row_bytes >> 3;                   // 8-byte pieces of a source row
    const uint32_t ta = tmem + ((uint32_t)(quad * 32) << 16) + grp * AW;
    const uint32_t stageA = smem_u32(stage);
    int it = grp;
    for (long long tile = bx + (long long)grp * gxu; tile < n_tiles; tile += 2LL * gxu, it += 2) {
      const int use = it >> 1, st = warp + 8 * (use % KS);
      if (!wait_bar_warp_nap(&sfull[st], (use / KS) & 1, &abort_s, L.err)) break;
      if (!wait_bar_warp_nap(&aempty[grp], (use & 1) ^ 1, &abort_s, L.err)) break;
      fence_after_sync();
      const bool valid = 2 * tile + (quad >> 1) < u.n_windows;
      // the lane's row: 8-byte pieces (rows are 2C bytes apart: lanes 0-15 and 16-31 each cover all 32 banks)
      const uint32_t src = stageA + (uint32_t)st * (uint32_t)qbytes + (uint32_t)lane * (uint32_t)row_bytes;
      const int np = valid ? npieces : 0;
#pragma unroll
      for (int j = 0; j < NA; ++j) {
        uint32_t v[32];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int piece = j * 16 + k;
          uint32_t a, b;
          lds64(a, b, src + (piece < np ? piece : 0) * 8);              // (pieces past the row re-read its head and are dropped)
          v[2 * k] = piece < np ? a : ((piece == npieces && u.ones_col) ? 0x3F80u : 0u);   // (1.0, 0) meets the bias row of the weight image
          v[2 * k + 1] = piece < np ? b : 0u;
        }
        tmem_st32(ta + j * 32, v);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sempty[st]);            // the stage's bytes are in registers
      tmem_st_wait();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&afull[grp]);
    }
  } else if (warp == kProdWarp) {
    // ---------------- producer: one round per tile; lane = 4 * quarter + window row fetches that row (one bulk
    // copy, two where the window wraps round the image edge)
    const char* const srcA = reinterpret_cast<const char*>(u.A);
    const long long line_bytes = (long long)u.W * row_bytes;
    const int quad = (lane >> 2) & 3, r4 = lane & 3;
    const uint32_t stageA = smem_u32(stage);
    const int nwin = (int)u.n_windows;
    bool ok = true;
    int it = 0;
    for (int tile = bx; tile < (int)n_tiles && ok; tile += gxu, ++it) {
      const int use = it >> 1, st0 = (it & 1) * 4 + 8 * (use % KS);   // stages of converter warps 4*(it & 1) + 0..3
      const uint32_t par = (((uint32_t)(use / KS)) & 1u) ^ 1u;
      for (int qd = 0; qd < 4; ++qd)
        if (!wait_bar_warp_nap(&sempty[st0 + qd], par, &abort_s, L.err)) { ok = false; break; }
      if (!ok) break;
      const int win = 2 * tile + (quad >> 1);
      const bool valid = win < nwin;
      if (lane < 16 && r4 == 0) {
        if (valid) mbar_arrive_expect_tx(&sfull[st0 + quad], (uint32_t)qbytes);
        else mbar_arrive(&sfull[st0 + quad]);               // second window of the last pair of an odd count
      }
      __syncwarp();
      if (lane < 16 && valid) {
        const int b = win / u.nW, w = win - b * u.nW;
        const int wi = w / u.nWw, wj = w - wi * u.nWw;
        int i = wi * 8 + (quad & 1) * 4 + r4 + u.s;       // cyclic shift: the shifted frame reads from +s
        if (i >= u.H) i -= u.H;
        const int j0 = wj * 8 + u.s;                      // < W + 8
        const char* line = srcA + ((long long)b * u.H + i) * line_bytes;
        const uint32_t dst = stageA + (uint32_t)(st0 + quad) * (uint32_t)qbytes + (uint32_t)(r4 * 8 * row_bytes);
        const int n0 = j0 + 8 <= u.W ? 8 : u.W - j0;      // tokens before the image edge (>= 1)
        bulk_load(dst, line + (long long)j0 * row_bytes, (uint32_t)(n0 * row_bytes), &sfull[st0 + quad]);
        if (n0 < 8) bulk_load(dst + n0 * row_bytes, line, (uint32_t)((8 - n0) * row_bytes), &sfull[st0 + quad]);
      }
    }
  } else if (warp == kMmaWarp) {
    // ---------------- MMA issue: A from TMEM, B from the resident weight image; one chunk after the other
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, u.cw, 0, 0);
      const uint64_t b0 = make_desc(smem_u32(sB), 16, 1024);
      const uint32_t atom_step = (uint32_t)NT * 8u, chunk_step = (uint32_t)u.cw * 8u;   // descriptor address units of 16 bytes
      int q = 0, qph = 0, it = 0;
      bool ok = true;
      for (long long tile = bx; tile < n_tiles && ok; tile += gxu, ++it) {
        const int ab = it & 1, use = it >> 1;
        if (!wait_bar_nap(&afull[ab], use & 1, &abort_s, L.err)) break;
        fence_after_sync();
        const uint32_t ta = tmem + ab * AW;
        for (int c = 0; c < u.nchunks; ++c) {
          if (!wait_bar_nap(&tempty[q], qph ^ 1, &abort_s, L.err)) { ok = false; break; }
          fence_after_sync();
          const uint32_t td = tmem + CP + q * u.cw;
          const uint64_t bc = b0 + (uint64_t)(c * chunk_step);
#pragma unroll
          for (int atom = 0; atom < NA; ++atom) {
            const uint64_t bd = bc + (uint64_t)(atom * atom_step);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) mma_bf16_ts(td, ta + (atom * 4 + kk) * 8, bd + 2 * kk, idesc, (atom | kk) != 0);
          }
          commit(&tfull[q]);
          if (++q == RC) { q = 0; qph ^= 1; }
        }
        if (ok) commit(&aempty[ab]);                      // the A buffer may be overwritten once these MMAs are done
      }
    }
  } else {
    // ---------------- epilogue: accumulator row = (window of the pair, slot); a thread owns one row.  The 32 rows of
    // a warp are contiguous in the global tile image of each output block (2 * DP bytes per row, 16-byte chunks
    // permuted inside a row), so the DP/8 16-byte stores of a block cover one contiguous piece of 64 * DP bytes
    // between them.  Four warps per TMEM quadrant share the blocks round robin (block counter modulo 4, running over
    // chunks and tiles).  Every warp waits for and releases every chunk, with or without a block in it: a warp that
    // skipped uses of a ring position could find the position's barrier two phases on, which a parity wait cannot
    // tell from "not yet".
    const int ew = warp - kConvWarps, quad = ew & 3, sub = ew >> 2;
    const int row = (quad & 1) * 32 + lane;               // slot inside the window
    const int nblk = u.cw / DP;
    int q = 0, qph = 0;
    unsigned cc = 0;                                      // chunks seen so far
    bool ok = true;
    for (long long tile = bx; tile < n_tiles && ok; tile += gxu) {
      const long long win = 2 * tile + (quad >> 1);
      const bool valid = win < u.n_windows;
      unsigned char* orow = reinterpret_cast<unsigned char*>(u.out + win * u.win_stride);
      for (int c = 0; c < u.nchunks; ++c, ++cc) {
        const int first = (int)((sub - cc * nblk) & 3u);  // my first block of this chunk
        {
          if (!wait_bar_warp_nap(&tfull[q], qph, &abort_s, L.err)) { ok = false; break; }
          fence_after_sync();
          for (int blk = first; blk < nblk; blk += 4) {
            const int gb = c * nblk + blk;
            uint32_t v[DP];
            const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + CP + q * u.cw + blk * DP;
            if constexpr (DP == 32) tmem_ld32(taddr, v); else tmem_ld16(taddr, v);
            tmem_ld_wait();
            const bool scaled = u.q_every3 && gb % 3 == 0;
            unsigned char* dst = orow + (size_t)gb * 64 * DP * 2;
            if (u.bias == nullptr && !scaled) {           // the common case: convert and store
#pragma unroll
              for (int j = 0; j < DP / 8; ++j) {
                uint4 o;
                o.x = pack_bf16(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1]));
                o.y = pack_bf16(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
                o.z = pack_bf16(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
                o.w = pack_bf16(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
                if (valid) *reinterpret_cast<uint4*>(dst + tile_off<DP>(row, j)) = o;
              }
            } else {
              const float sc = scaled ? u.qscale : 1.f;
#pragma unroll
              for (int j = 0; j < DP / 8; ++j) {
                float4 b0v = make_float4(0.f, 0.f, 0.f, 0.f), b1v = b0v;
                if (u.bias != nullptr) {                  // bias added here (no spare K column to carry it)
                  b0v = *reinterpret_cast<const float4*>(sBias + gb * DP + 8 * j);
                  b1v = *reinterpret_cast<const float4*>(sBias + gb * DP + 8 * j + 4);
                }
                uint4 o;
                o.x = pack_bf16((__uint_as_float(v[8 * j]) + b0v.x) * sc, (__uint_as_float(v[8 * j + 1]) + b0v.y) * sc);
                o.y = pack_bf16((__uint_as_float(v[8 * j + 2]) + b0v.z) * sc, (__uint_as_float(v[8 * j + 3]) + b0v.w) * sc);
                o.z = pack_bf16((__uint_as_float(v[8 * j + 4]) + b1v.x) * sc, (__uint_as_float(v[8 * j + 5]) + b1v.y) * sc);
                o.w = pack_bf16((__uint_as_float(v[8 * j + 6]) + b1v.z) * sc, (__uint_as_float(v[8 * j + 7]) + b1v.w) * sc);
                if (valid) *reinterpret_cast<uint4*>(dst + tile_off<DP>(row, j)) = o;
              }
            }
          }
          fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty[q]);
        }
        if (++q == RC) { q = 0; qph ^= 1; }
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    __syncwarp();
    tmem_dealloc(tmem, tcols);
  }
}

struct TmShape {
  size_t smem;
  int stages;
};

// Shared memory of a launch whose largest unit has maxNT accumulator columns: 16 stages if they fit, else 8.
TmShape tm_shape(int CP, int maxNT, int row_bytes) {
  const size_t qbytes = (size_t)32 * row_bytes;
  for (int stages = 16; stages >= 8; stages -= 8) {
    const size_t smem = 1024 + (size_t)maxNT * CP * 2 + (((size_t)stages * qbytes + 127) & ~(size_t)127) + (size_t)maxNT * 4 + 64;
    if (smem <= kTmSmemBudget) return TmShape{smem, stages};
  }
  return TmShape{0, 0};
}

template <int CP, int DP>
int launch_gwt_t(const GWLaunch& L, int nunits, cudaStream_t st, const char* name) {
  int maxNT = 0;
  for (int i = 0; i < nunits; ++i) {
    const int NT = L.u[i].nchunks * L.u[i].cw;
    if (NT > maxNT) maxNT = NT;
    if (L.u[i].cw > 256 || L.u[i].cw % 16 != 0 || NT + CP > 512) return GSWA_ERR_UNSUPPORTED;
  }
  const TmShape ts = tm_shape(CP, maxNT, L.u[0].lda * 2);
  if (ts.stages < kMinStages) return GSWA_ERR_UNSUPPORTED;
  if (cudaFuncSetAttribute(gwt_kernel<CP, DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ts.smem) != cudaSuccess)
    return check_launch();
  GWLaunch Lc = L;
  Lc.nslots = ts.stages;
  // One CTA per SM; a unit's share of them follows its work per tile (loads and conversion every unit pays, plus
  // MMAs and an epilogue proportional to its columns), so that all units finish together.
  double wsum = 0, w[kMaxUnits];
  for (int i = 0; i < nunits; ++i) { w[i] = 96.0 + L.u[i].nchunks * L.u[i].cw; wsum += w[i]; }
  const int sms = device_sm_count();
  const int total = sms < nunits ? nunits : sms;
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
  { KernelScope ks_(name, st); gwt_kernel<CP, DP><<<dim3((unsigned)given), kThreadsTM, ts.smem, st>>>(Lc); }
  return check_launch();
}

}  // namespace

bool gwt_usable(const void* A, int lda, int H, int W, const int* shifts, int nshifts) {
  if ((reinterpret_cast<uintptr_t>(A) & 15) != 0 || (W & 7) || (H & 7) || (lda & 3)) return false;
  for (int i = 0; i < nshifts; ++i)
    if ((2 * lda * shifts[i]) % 16 != 0) return false;   // every piece of a window row starts and ends on 16 bytes
  return true;
}

// Largest number of heads per unit for which the weight image, at least eight stages and the accumulators fit.
int gwt_heads_per_unit(int Cp, int dp, int C, int nb, int cap) {
  int best = 0;
  for (int n = 1; n <= cap; ++n) {
    const int NT = n * nb * dp;
    if (NT + Cp > 512) break;
    if (tm_shape(Cp, NT, 2 * C).stages >= kMinStages) best = n;
  }
  return best;
}

int launch_gwt(const GWLaunch& L, int nunits, int Cp, int dp, cudaStream_t st, const char* name) {
#define GWT_CASE(CPV) \
  if (Cp == CPV) return dp == 32 ? launch_gwt_t<CPV, 32>(L, nunits, st, name) : launch_gwt_t<CPV, 16>(L, nunits, st, name);
  GWT_CASE(64) GWT_CASE(128) GWT_CASE(192) GWT_CASE(256)
#undef GWT_CASE
  return GSWA_ERR_UNSUPPORTED;
}

}  // namespace gswa
