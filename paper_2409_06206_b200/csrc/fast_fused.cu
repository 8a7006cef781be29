// Fused forward of Eq. 6: per window pair, the QKV projection runs on the tensor core (tcgen05.mma,
// accumulators in TMEM) and its result goes straight to the attention warps of the same CTA through
// shared memory -- q, k, v never make a round trip through HBM on the inference path, and on the
// training path they leave once, as the tile images the backward kernel reloads.
//
//   warps 0-11   attention: warp = 4*head + quadrant.  A warp first drains its TMEM quadrant
//                (32 rows of one window) for its head's q,k,v columns into the tile images, then
//                computes softmax attention for 16 query rows of each window (mma.sync, see attn_core.cuh)
//   warp  12     MMA issue
//   warps 13-18  loaders (three sets of two warps, see gemm_core.cuh)
#include "attn_core.cuh"
#include "gemm_core.cuh"

namespace gswa {
using namespace umma;
using namespace gemm;
using namespace attn;
namespace {

constexpr int kAttnWarps = 12;
constexpr int kSetsF = 3;                                       // loader sets (19 warps leave 96 registers per thread)
constexpr int kThreadsF = 32 * (kAttnWarps + 1 + 2 * kSetsF);   // 608

__device__ __forceinline__ void attn_sync(int nt) { asm volatile("bar.sync 1, %0;" ::"r"(nt) : "memory"); }
__device__ __forceinline__ bool attn_vote(int nt, bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %2, 0;\n\tbar.red.and.pred p, 1, %1, q;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(r)
      : "r"(nt), "r"((uint32_t)ok)
      : "memory");
  return r != 0;
}

template <int CP, int DP>
__global__ void __launch_bounds__(kThreadsF, 1) fw_kernel(const __grid_constant__ FWLaunch L) {
  const FWUnit& u = L.u[blockIdx.y];
  const FastGeom& g = L.geo;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = align1024(smem_raw);
  constexpr int NA = CP / 64;                  // K atoms per tile
  constexpr int kTile = 64 * DP * 2;           // one [64][DP] tile image
  const int nh_u = u.nheads;
  const int NT = nh_u * 3 * DP;
  const int S = L.nslots;
  unsigned char* sB = sm;
  unsigned char* ring = sB + (size_t)NT * CP * 2;
  unsigned char* tiles = ring + (size_t)S * kAtomBytes;          // q,k,v of one window: [head][kind][64][DP]
  float* sBias = reinterpret_cast<float*>(tiles + (size_t)nh_u * 3 * kTile);
  float2* tab = reinterpret_cast<float2*>(sBias + NT);        // pair table, see bias_init
  int* tok = reinterpret_cast<int*>(tab + nh_u * 225);
  unsigned char* reg = reinterpret_cast<unsigned char*>(tok + 64);
  unsigned char* ostg0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(reg + 64) + 15) & ~(uintptr_t)15);
  __shared__ uint64_t full[8], empty[8], tfull, tempty;
  __shared__ uint32_t tmem_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < NT * CP * 2 / 16; i += kThreadsF)
    reinterpret_cast<uint4*>(sB)[i] = __ldg(reinterpret_cast<const uint4*>(u.Bimg) + i);
  for (int i = tid; i < NT; i += kThreadsF) sBias[i] = u.bias ? u.bias[i] : 0.f;
  attn::fill_pair_table(tab, L.table, g.nh, u.h0, nh_u, tid, kThreadsF);
  fence_proxy_async();
  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 8; ++i) { mbar_init(&full[i], 2); mbar_init(&empty[i], 1); }
    mbar_init(&tfull, 1);
    mbar_init(&tempty, nh_u * 4);
    mbar_init_fence();
  }
  const uint32_t tcols = pow2_cols(NT);
  if (warp == kAttnWarps) tmem_alloc(&tmem_s, tcols);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = tmem_s;
  const long long n_tiles = (u.n_windows + 1) / 2;

  if (warp > kAttnWarps) {
    // ---------------- loaders: rows gathered in window order (cyclic shift + partition as addresses)
    const int set = (warp - kAttnWarps - 1) >> 1;
    LoaderLane ll;
    ll.init(((warp - kAttnWarps - 1) & 1) * 32 + lane);
    const char* const srcA = reinterpret_cast<const char*>(u.X);
    const long long row_bytes = (long long)u.lda * 2, line_bytes = (long long)u.W * row_bytes;
    const uint32_t ringA = smem_u32(ring);
    RingPos rp;
    rp.init(set, S);
    int g_step = set;                            // ring step = tile iteration * NA + atom
    int it = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
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
      for (; g_step < (it + 1) * NA; g_step += kSetsF) {
        const int atom = g_step - it * NA;
        if (!wait_bar_warp(&empty[rp.slot], rp.ph ^ 1, &abort_s, L.err)) { ok = false; break; }
        const uint32_t dst = ringA + rp.slot * kAtomBytes;
        const bool cv = atom * 128 + ll.pc * 8 < u.kvalid * 2;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const bool v = wv[half] && cv;
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
        cp_async_commit();
        cp_async_wait(0);
        publish(&full[rp.slot], lane);
        rp.advance(kSetsF, S);
      }
      if (!ok) break;
    }
    cp_async_wait(0);
  } else if (warp == kAttnWarps) {
    // ---------------- MMA issue: one accumulator chunk per head, all K atoms of a tile per chunk
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, 3 * DP, 0, 0);
      const uint64_t a0 = make_desc(smem_u32(ring), 16, 1024), b0 = make_desc(smem_u32(sB), 16, 1024);
      RingPos rp;
      rp.init(0, S);
      int it = 0;
      bool ok = true;
      for (long long tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
        if (!wait_bar(&tempty, (it & 1) ^ 1, &abort_s, L.err)) break;
        fence_after_sync();
        int slot_a[NA];
        for (int c = 0; c < nh_u && ok; ++c) {
#pragma unroll
          for (int atom = 0; atom < NA; ++atom) {
            if (c == 0) {
              if (!wait_bar(&full[rp.slot], rp.ph, &abort_s, L.err)) { ok = false; break; }
              fence_after_sync();
              slot_a[atom] = rp.slot;
              rp.advance(1, S);
            }
            const uint64_t ad = a0 + (uint64_t)((slot_a[atom] * kAtomBytes) >> 4);
            const uint64_t bd = b0 + (uint64_t)(((atom * NT + c * 3 * DP) * 128) >> 4);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) mma_bf16(tmem + c * 3 * DP, ad + 2 * kk, bd + 2 * kk, idesc, (atom | kk) != 0);
          }
        }
        if (!ok) break;
#pragma unroll
        for (int atom = 0; atom < NA; ++atom) commit(&empty[slot_a[atom]]);
        commit(&tfull);
      }
    }
  } else if (warp < nh_u * 4) {
    // ---------------- attention warps
    const int nt = nh_u * 128;
    const int hl = warp >> 2, quad = warp & 3, r0 = quad * 16;
    const int h = u.h0 + hl;
    const int row = (quad & 1) * 32 + lane;       // accumulator row of this lane inside its window
    unsigned char* ostg = ostg0 + (size_t)warp * 16 * DP * 2;
    const uint32_t q_base = smem_u32(tiles + (size_t)(hl * 3) * kTile);
    const uint32_t tilesA = smem_u32(tiles);
    int it = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      if (!attn_vote(nt, wait_bar_warp(&tfull, it & 1, &abort_s, L.err))) break;
      fence_after_sync();
#pragma unroll 1
      for (int w = 0; w < 2; ++w) {
        const long long win = 2 * tile + w;
        const bool valid = win < u.n_windows;
        if ((quad >> 1) == w) {
          // drain this warp's TMEM quadrant: q, k, v of head hl for 32 rows of window w
#pragma unroll 1
          for (int kind = 0; kind < 3; ++kind) {
            const int gb = hl * 3 + kind;
            uint32_t v[DP];
            const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + gb * DP;
            if constexpr (DP == 32) tmem_ld32(taddr, v); else tmem_ld16(taddr, v);
            tmem_ld_wait();
            const float sc = kind == 0 ? u.qscale : 1.f;
            unsigned char* blk = tiles + (size_t)gb * kTile;
#pragma unroll
            for (int j = 0; j < DP / 8; ++j) {
              const float4 b0v = *reinterpret_cast<const float4*>(sBias + gb * DP + 8 * j);
              const float4 b1v = *reinterpret_cast<const float4*>(sBias + gb * DP + 8 * j + 4);
              uint4 o;
              o.x = pack_bf16((__uint_as_float(v[8 * j]) + b0v.x) * sc, (__uint_as_float(v[8 * j + 1]) + b0v.y) * sc);
              o.y = pack_bf16((__uint_as_float(v[8 * j + 2]) + b0v.z) * sc, (__uint_as_float(v[8 * j + 3]) + b0v.w) * sc);
              o.z = pack_bf16((__uint_as_float(v[8 * j + 4]) + b1v.x) * sc, (__uint_as_float(v[8 * j + 5]) + b1v.y) * sc);
              o.w = pack_bf16((__uint_as_float(v[8 * j + 6]) + b1v.z) * sc, (__uint_as_float(v[8 * j + 7]) + b1v.w) * sc);
              *reinterpret_cast<uint4*>(blk + tile_off<DP>(row, j)) = o;
            }
          }
          fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty);
          if (u.qkv_out != nullptr) fence_proxy_async();   // the bulk copy reads the tiles through the async proxy
        }
        const WinCtx wc = window_setup(g, u.s, valid ? win : 0, tok, reg, tid);
        attn_sync(nt);                             // tiles, tok and reg of window w are complete
        if (valid) {
          if (u.qkv_out != nullptr && tid == 0) bulk_store(u.qkv_out + win * u.qkv_wstride, tilesA, (uint32_t)NT * 128);
          fwd_window<DP>(q_base, q_base + kTile, q_base + 2 * kTile, tab + hl * 225, tok, reg, wc.masked, r0, lane, ostg, L.A,
                         g.nh * DP, h, g.d, u.lt != nullptr ? u.lt + win * u.l_wstride + hl * 64 : nullptr);
          if (u.qkv_out != nullptr && tid == 0) bulk_wait_read();
        }
        attn_sync(nt);                             // the tiles may be overwritten
      }
    }
    if (tid == 0) bulk_wait_all();
  }
  fence_before_sync();
  __syncthreads();
  if (warp == kAttnWarps) {
    __syncwarp();
    tmem_dealloc(tmem, tcols);
  }
}

int fw_num_sms() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  }
  return n;
}

template <int CP, int DP>
int launch_fw_t(const FWLaunch& L, int nunits, cudaStream_t st) {
  int maxh = 0;
  long long max_tiles = 1;
  for (int i = 0; i < nunits; ++i) {
    if (L.u[i].nheads > maxh) maxh = L.u[i].nheads;
    const long long t = (L.u[i].n_windows + 1) / 2;
    if (t > max_tiles) max_tiles = t;
  }
  FWLaunch Lc = L;
  const size_t smem = fw_smem_bytes(CP, DP, maxh, &Lc.nslots);
  if (smem == 0) return GSWA_ERR_UNSUPPORTED;
  if (cudaFuncSetAttribute(fw_kernel<CP, DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return check_launch();
  long long gx = fw_num_sms() / nunits;
  if (gx < 1) gx = 1;
  if (gx > max_tiles) gx = max_tiles;
  { KernelScope ks_("qkv_attn_fwd", st); fw_kernel<CP, DP><<<dim3((unsigned)gx, nunits), kThreadsF, smem, st>>>(Lc); }
  return check_launch();
}

}  // namespace

size_t fw_smem_bytes(int Cp, int dp, int maxheads, int* nslots) {
  if (maxheads < 1 || maxheads > 3) return 0;
  const size_t NT = (size_t)maxheads * 3 * dp;
  const size_t fixed = 1024 + NT * Cp * 2 + (size_t)maxheads * 3 * 64 * dp * 2 + NT * 4 + (size_t)maxheads * 225 * 8 + 64 * 4 + 64 +
                       16 + (size_t)kAttnWarps * 16 * dp * 2 + 64;
  const size_t budget = 224 * 1024;
  const int need = Cp / 64 > kSetsF ? Cp / 64 : kSetsF;      // a tile's atoms must fit, and no more loader sets than slots
  if (fixed + (size_t)need * 16384 > budget) return 0;
  int s = (int)((budget - fixed) / 16384);
  if (s > 8) s = 8;
  if (nslots) *nslots = s;
  return fixed + (size_t)s * 16384;
}

int launch_fw(const FWLaunch& L, int nunits, int Cp, int dp, cudaStream_t st) {
#define FW_CASE(CPV) \
  if (Cp == CPV) return dp == 32 ? launch_fw_t<CPV, 32>(L, nunits, st) : launch_fw_t<CPV, 16>(L, nunits, st);
  FW_CASE(64) FW_CASE(128) FW_CASE(192) FW_CASE(256)
#undef FW_CASE
  return GSWA_ERR_UNSUPPORTED;
}

}  // namespace gswa
