// Warp-level building blocks of the window attention kernels (mma.sync m16n8k16, ldmatrix / stmatrix,
// softmax pieces, index helpers).  Shared by the stand-alone attention kernels and by the kernel that
// fuses the QKV projection with the forward attention.
#pragma once

#include "fast.cuh"
#include "gswa_index.cuh"
#include "umma.cuh"

namespace gswa {
namespace attn {
using umma::smem_u32;
using umma::cp_async_commit;


__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2(float x) {          // 2^x, one MUFU instruction; 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Two fp32 lanes per instruction (packed f32x2 arithmetic) and the three-input maximum: the softmax
// arithmetic of these kernels is bound by instruction issue, and each of these halves an instruction count.
__device__ __forceinline__ unsigned long long pk2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void upk2(unsigned long long r, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r));
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("add.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long sub2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("sub.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("mul.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ void stsm_x4(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
               : "memory");
}
__device__ __forceinline__ void stsm_x2(uint32_t addr, uint32_t r0, uint32_t r1) {
  asm volatile("stmatrix.sync.aligned.m8n8.x2.shared.b16 [%0], {%1,%2};" ::"r"(addr), "r"(r0), "r"(r1) : "memory");
}

// [64][64] bf16 matrices (P, dS): 128-byte rows, chunk ^= row & 7.
__device__ __forceinline__ uint32_t sq_off(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// Tiles arrive from global memory already in their shared-memory image (tile_off): a linear copy.
template <int DP>
__device__ __forceinline__ void load_tiles(unsigned char* dst, const __nv_bfloat16* src, int nblocks, int tid, int nt) {
  const int nchunks = nblocks * 64 * (DP / 8);
  const uint32_t d0 = smem_u32(dst);
  for (int ci = tid; ci < nchunks; ci += nt)
    cp_async16(d0 + ci * 16, reinterpret_cast<const unsigned char*>(src) + (size_t)ci * 16);
}

// S (16 rows x 64 keys) = Q K^T for the warp's rows; returns accumulators in s[8][4].
template <int DP, bool kZero = true>
__device__ __forceinline__ void qk_scores(float (*s)[4], uint32_t q_base, uint32_t k_base, int r0, int lane) {
  if constexpr (kZero) {
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
  }
#pragma unroll
  for (int kk = 0; kk < DP / 16; ++kk) {
    uint32_t a[4];
    ldsm_x4(a, q_base + tile_off<DP>(r0 + (lane & 15), 2 * kk + (lane >> 4)));
#pragma unroll
    for (int jp = 0; jp < 4; ++jp) {
      uint32_t b[4];
      ldsm_x4(b, k_base + tile_off<DP>(16 * jp + (lane & 7) + ((lane >> 4) << 3), 2 * kk + ((lane >> 3) & 1)));
      mma16816(s[2 * jp], a, b[0], b[1]);
      mma16816(s[2 * jp + 1], a, b[2], b[3]);
    }
  }
}

// acc (16 x DP) += A(16 x 64, from packed register fragments of `pf`) * B(64 x DP) with B read
// transposed from a [64][DP] tile (rows = contraction index).
template <int DP>
__device__ __forceinline__ void regs_times_tile(float (*acc)[4], const float (*pf)[4], uint32_t b_base, int lane) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    uint32_t a[4];
    a[0] = pack2(pf[2 * kk][0], pf[2 * kk][1]);
    a[1] = pack2(pf[2 * kk][2], pf[2 * kk][3]);
    a[2] = pack2(pf[2 * kk + 1][0], pf[2 * kk + 1][1]);
    a[3] = pack2(pf[2 * kk + 1][2], pf[2 * kk + 1][3]);
#pragma unroll
    for (int jn = 0; jn < DP / 16; ++jn) {
      uint32_t b[4];
      ldsm_x4_t(b, b_base + tile_off<DP>(16 * kk + (lane & 7) + (((lane >> 3) & 1) << 3), 2 * jn + (lane >> 4)));
      mma16816(acc[2 * jn], a, b[0], b[1]);
      mma16816(acc[2 * jn + 1], a, b[2], b[3]);
    }
  }
}

__device__ __forceinline__ void set_word(uint4& v, int i, uint32_t w) {
  if (i == 0) v.x = w; else if (i == 1) v.y = w; else if (i == 2) v.z = w; else v.w = w;
}

// Writes a warp's 16 x DP accumulator tile (rows gq, gq+8 of the mma fragment) to rows of a padded
// token-major buffer: the tile is first laid out in the warp's 16 x DP staging block (stmatrix), then
// every lane moves 16 bytes per row so that one store instruction covers whole 2*DP-byte row pieces.
// `row0` / `row1` are the global addresses of the lane's two rows (fragment rows gq and gq + 8).
// Fragment rows gq are multiplied by `scale0`, rows gq + 8 by `scale1` (kScaled = false: stored as they are).
template <int DP, bool kScaled = true>
__device__ __forceinline__ void store_tile(unsigned char* stg, const float (*acc)[4], float scale0, float scale1,
                                           unsigned char* row0, unsigned char* row1, int lane, int ones_col) {
  const uint32_t sa = smem_u32(stg);
  const int m = lane >> 3;
  const unsigned long long sc0 = pk2(scale0, scale0), sc1 = pk2(scale1, scale1);
#pragma unroll
  for (int jn = 0; jn < DP / 8; jn += 2) {
    const int row = (m & 1) * 8 + (lane & 7), chunk = jn + (m >> 1);
    float v[8];
    if constexpr (kScaled) {
      upk2(mul2(pk2(acc[jn][0], acc[jn][1]), sc0), v[0], v[1]);
      upk2(mul2(pk2(acc[jn][2], acc[jn][3]), sc1), v[2], v[3]);
      upk2(mul2(pk2(acc[jn + 1][0], acc[jn + 1][1]), sc0), v[4], v[5]);
      upk2(mul2(pk2(acc[jn + 1][2], acc[jn + 1][3]), sc1), v[6], v[7]);
    } else {
      v[0] = acc[jn][0]; v[1] = acc[jn][1]; v[2] = acc[jn][2]; v[3] = acc[jn][3];
      v[4] = acc[jn + 1][0]; v[5] = acc[jn + 1][1]; v[6] = acc[jn + 1][2]; v[7] = acc[jn + 1][3];
    }
    stsm_x4(sa + tile_off<DP>(row, chunk), pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
  }
  __syncwarp();
  if constexpr (DP == 32) {
    const int gq = lane >> 2, t = lane & 3;
    uint4 v0 = *reinterpret_cast<const uint4*>(stg + tile_off<DP>(gq, t));
    uint4 v1 = *reinterpret_cast<const uint4*>(stg + tile_off<DP>(gq + 8, t));
    if (ones_col >= 0 && (ones_col >> 3) == t) {
      set_word(v0, (ones_col & 7) >> 1, 0x00003F80u);        // (1.0, 0.0)
      set_word(v1, (ones_col & 7) >> 1, 0x00003F80u);
    }
    *reinterpret_cast<uint4*>(row0 + t * 16) = v0;
    *reinterpret_cast<uint4*>(row1 + t * 16) = v1;
  } else {
    // DP == 16: 16 rows x 2 chunks, one chunk per lane; the lane's row pointer comes from a neighbour
    const int r = lane >> 1, c = lane & 1;
    uint4 v = *reinterpret_cast<const uint4*>(stg + tile_off<DP>(r, c));
    if (ones_col >= 0 && (ones_col >> 3) == c) set_word(v, (ones_col & 7) >> 1, 0x00003F80u);
    // row pointers live in lanes with gq == r (rows 0..7: row0 of lane 4r) or gq == r - 8 (row1 of lane 4(r-8))
    const unsigned long long a0 = __shfl_sync(0xffffffffu, (unsigned long long)row0, (r & 7) * 4);
    const unsigned long long a1 = __shfl_sync(0xffffffffu, (unsigned long long)row1, (r & 7) * 4);
    *reinterpret_cast<uint4*>((r < 8 ? a0 : a1) + c * 16) = v;
  }
  __syncwarp();
}

struct WinCtx {
  int b, wi, wj;
  bool masked;
};

__device__ __forceinline__ WinCtx window_setup(const FastGeom& g, int s, long long win, int* tok, unsigned char* reg,
                                               int tid) {
  WinCtx c;
  // window -> (image, window row, window column) without integer division: quotient from a float reciprocal,
  // corrected by one step (window counts of this path stay far below 2^24)
  const int wn = (int)win;
  int b = (int)(((float)wn + 0.5f) * (1.0f / (float)g.nW));
  int w = wn - b * g.nW;
  if (w < 0) { --b; w += g.nW; } else if (w >= g.nW) { ++b; w -= g.nW; }
  int wi = (int)(((float)w + 0.5f) * (1.0f / (float)g.nWw));
  int wj = w - wi * g.nWw;
  if (wj < 0) { --wi; wj += g.nWw; } else if (wj >= g.nWw) { ++wi; wj -= g.nWw; }
  c.b = b;
  c.wi = wi;
  c.wj = wj;
  c.masked = s > 0 && (c.wi == g.nWh - 1 || c.wj == g.nWw - 1);
  if (tid < 64) {
    // slot tid of the window in the shifted frame -> original token and mask label (what slot_to_token computes)
    const int ip = wi * 8 + (tid >> 3), jp = wj * 8 + (tid & 7);
    int i = ip + s, j = jp + s;
    if (i >= g.H) i -= g.H;
    if (j >= g.W) j -= g.W;
    tok[tid] = (b * g.H + i) * g.W + j;
    reg[tid] = (unsigned char)(3 * axis_region(ip, g.H, 8, s) + axis_region(jp, g.W, 8, s));
  }
  return c;
}

// The scores start from the relative-position bias (the MMAs then accumulate q k^T on top of it: no separate
// addition); q and the table are already scaled by log2(e), the scores are in the log2 domain throughout.
// Bias-table row of query slot p0 against key slot 8*j + 2*t (the first of a thread's two key columns in key
// block j of the mma fragment).  Key 8*j + 2*t + 1 uses row - 1, query p0 + 8 (next window row) uses row + 15.
__device__ __forceinline__ int frag_bias_row(int p0, int t, int j) {
  const int pa0 = p0 >> 3, pc0 = p0 & 7;   // rows p0 and p0 + 8: same column in the window, next row
  return (pa0 - j + 7) * 15 + (pc0 - 2 * t + 7);
}
__device__ __forceinline__ void bias_init(float (*s)[4], const float2* tab2, int p0, int t) {
  // a thread's two columns of a key block are neighbours in the table: entry r of the pair table holds
  // (table[r], table[r - 1]), so one 8-byte load fills two accumulators
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int r = frag_bias_row(p0, t, j);
    const float2 a = tab2[r], b = tab2[r + 15];
    s[j][0] = a.x; s[j][1] = a.y; s[j][2] = b.x; s[j][3] = b.y;
  }
}
// Fills the pair table of `nheads` heads from the bf16 table [225][nh] (scaled by log2(e)).
__device__ __forceinline__ void fill_pair_table(float2* tab2, const __nv_bfloat16* table, int nh, int h0, int nheads, int tid, int nt) {
  for (int e = tid; e < nheads * 225; e += nt) {
    const int r = e % 225, hh = h0 + e / 225;
    tab2[e] = make_float2(__bfloat162float(table[r * nh + hh]) * kLog2e, r > 0 ? __bfloat162float(table[(r - 1) * nh + hh]) * kLog2e : 0.f);
  }
}
// Window mask: pairs whose slots carry different region labels are excluded.
__device__ __forceinline__ void apply_mask(float (*s)[4], const unsigned char* reg, bool masked, int p0, int t) {
  if (masked) {
    const unsigned char r0 = reg[p0], r1 = reg[p0 + 8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const unsigned char q0 = reg[8 * j + 2 * t], q1 = reg[8 * j + 2 * t + 1];
      if (q0 != r0) s[j][0] = -INFINITY;
      if (q1 != r0) s[j][1] = -INFINITY;
      if (q0 != r1) s[j][2] = -INFINITY;
      if (q1 != r1) s[j][3] = -INFINITY;
    }
  }
}


// Forward attention of one warp: 16 query rows (r0 .. r0+15) of one head against the 64 keys of its
// window (Eq. 6 `Attn` with relative-position bias and window mask).  q,k,v are [64][DP] tile images
// in shared memory (q and the table already carry the factor log2(e)).  Writes the 16 x DP output
// rows through the warp's staging block `ostg` to `A` (padded token-major, row length Ap) and, if
// `lt` is not null, the natural-log row log-sum-exp to lt[0..63] (this head's block of the L tile).
template <int DP>
__device__ __forceinline__ void fwd_window(uint32_t q_base, uint32_t k_base, uint32_t v_base, const float2* tab,
                                           const int* tok, const unsigned char* reg, bool masked, int r0, int lane,
                                           unsigned char* ostg, __nv_bfloat16* A, int Ap, int h, int d, float* lt) {
  const int gq = lane >> 2, t = lane & 3, p0 = r0 + gq;
  float s[8][4];
  bias_init(s, tab, p0, t);
  qk_scores<DP, false>(s, q_base, k_base, r0, lane);
  apply_mask(s, reg, masked, p0, t);

  float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    m0 = max3(m0, s[j][0], s[j][1]);
    m1 = max3(m1, s[j][2], s[j][3]);
  }
  m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
  m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
  m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
  m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
  float sum0, sum1;
  {
    const unsigned long long mm0 = pk2(m0, m0), mm1 = pk2(m1, m1);
    unsigned long long acc0 = pk2(0.f, 0.f), acc1 = acc0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      upk2(sub2(pk2(s[j][0], s[j][1]), mm0), s[j][0], s[j][1]);
      upk2(sub2(pk2(s[j][2], s[j][3]), mm1), s[j][2], s[j][3]);
      s[j][0] = ex2(s[j][0]);
      s[j][1] = ex2(s[j][1]);
      s[j][2] = ex2(s[j][2]);
      s[j][3] = ex2(s[j][3]);
      acc0 = add2(acc0, pk2(s[j][0], s[j][1]));
      acc1 = add2(acc1, pk2(s[j][2], s[j][3]));
    }
    float a, b;
    upk2(acc0, a, b);
    sum0 = a + b;
    upk2(acc1, a, b);
    sum1 = a + b;
  }
  sum0 += __shfl_xor_sync(0xffffffffu, sum0, 1);
  sum0 += __shfl_xor_sync(0xffffffffu, sum0, 2);
  sum1 += __shfl_xor_sync(0xffffffffu, sum1, 1);
  sum1 += __shfl_xor_sync(0xffffffffu, sum1, 2);

  float o[DP / 8][4];
#pragma unroll
  for (int j = 0; j < DP / 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
  regs_times_tile<DP>(o, s, v_base, lane);

  // rows of the padded attention output: DP columns per head, pad columns are exact zeros because
  // the pad columns of v are; column d of head 0 is set to one (bias-gradient column, see fast.cuh)
  const float inv0 = 1.f / sum0, inv1 = 1.f / sum1;
  store_tile<DP>(ostg, o, inv0, inv1, reinterpret_cast<unsigned char*>(A + (long long)tok[p0] * Ap + h * DP),
                 reinterpret_cast<unsigned char*>(A + (long long)tok[p0 + 8] * Ap + h * DP), lane,
                 (h == 0 && d < DP) ? d : -1);
  if (lt != nullptr && t == 0) {
    lt[p0] = m0 * kLn2 + logf(sum0);
    lt[p0 + 8] = m1 * kLn2 + logf(sum1);
  }
}

__device__ __forceinline__ void cp_async_wait_1() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

}  // namespace attn
}  // namespace gswa
