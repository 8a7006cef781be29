// Integer maps of GSWA: cyclic shift, window partition / reverse, window-mask labels and
// relative-position rows (Sec. "Patch Embedding"; shifted windows and masks of Sec. "Group
// Shifted Window Attention"; Sec. "Learnable Relative Shifted Bias").  Shift, partition and
// their inverses are never executed as copies: every kernel calls these functions to turn a
// (window, slot) pair into the address of the original token and back.
#pragma once

namespace gswa {

// Mask label along one axis of the shifted frame of length n: [0,n-M) -> 0, [n-M,n-s) -> 1, [n-s,n) -> 2.
__host__ __device__ __forceinline__ int axis_region(int u, int n, int M, int s) {
  if (s == 0) return 0;
  return u < n - M ? 0 : (u < n - s ? 1 : 2);
}

// Slot t of window w (numbered row-major over the shifted frame) -> original coordinates and mask label.
// shifted[i',j'] = x[(i'+s) mod H, (j'+s) mod W].
__host__ __device__ __forceinline__ void slot_to_token(int H, int W, int M, int s, int w, int t, int* i, int* j,
                                                       int* region) {
  const int nWw = W / M;
  const int ip = (w / nWw) * M + t / M;
  const int jp = (w % nWw) * M + t % M;
  int ii = ip + s, jj = jp + s;
  if (ii >= H) ii -= H;
  if (jj >= W) jj -= W;
  *i = ii;
  *j = jj;
  *region = 3 * axis_region(ip, H, M, s) + axis_region(jp, W, M, s);
}

// Original token (i,j) -> window, slot and mask label in the frame shifted by s.
__host__ __device__ __forceinline__ void token_to_slot(int H, int W, int M, int s, int i, int j, int* w, int* t,
                                                       int* region) {
  int ip = i - s, jp = j - s;
  if (ip < 0) ip += H;
  if (jp < 0) jp += W;
  *w = (ip / M) * (W / M) + jp / M;
  *t = (ip % M) * M + jp % M;
  *region = 3 * axis_region(ip, H, M, s) + axis_region(jp, W, M, s);
}

// Row of the bias table for query slot p and key slot q of an M x M window.
__host__ __device__ __forceinline__ int rel_row(int M, int p, int q) {
  return (p / M - q / M + M - 1) * (2 * M - 1) + (p % M - q % M + M - 1);
}

}  // namespace gswa
