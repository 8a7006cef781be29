// Planner and launch sequence of the bf16 tensor-core path.
//
//   forward : prep_weights -> qkv_gemm (gw) -> attn_fwd -> proj_gemm (gt)
//   backward: prep_weights -> dattn_gemm (gw: dO tiles = dy W^P per head group) -> dwproj_gemm (gr)
//             -> attn_bwd -> dx_gemm (gt) -> dwqkv_gemm (gr)
#include <cstring>

#include "fast.cuh"

#include <mutex>

namespace gswa {
namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr size_t kSmemBudget = 215 * 1024;

struct Unit {
  int g, h0, nheads;
};

struct TokenSplit {
  int nsplit, NB, nstages, natoms, stream_b;
};

// Largest number of heads per work unit such that the QKV weight image, two activation stages and
// the accumulators fit one SM.
int heads_per_unit(int Cp, int dp, int cap) {
  int best = 0;
  for (int n = 1; n <= cap; ++n) {
    const size_t NT = (size_t)n * 3 * dp;
    const int slots = Cp / 64 + 1 > 4 ? Cp / 64 + 1 : 4;
    const size_t smem = 1024 + NT * Cp * 2 + 8 * 2 * 32 * dp * 2 + (size_t)slots * 128 * 128 + NT * 4 + 64;   // weights, staging, ring
    if (smem <= kSmemBudget && NT <= 512) best = n;
  }
  return best;
}

// `cap` heads per unit at most: 2 for the QKV projection (two heads' 6*dp columns are one MMA and leave TMEM room for
// two tiles, so the MMAs of the next tile overlap this tile's epilogue), 3 for dO = dy W^P (dp columns per head).
int make_units(const Plan& p, Unit* units, int cap) {
  const int hpu = heads_per_unit(p.Cp, p.dp, cap);
  if (hpu == 0) return -1;
  int n = 0;
  for (int g = 0; g < p.G; ++g)
    for (int h = 0; h < p.gh[g]; h += hpu) {
      if (n == kMaxUnits) return -1;
      units[n++] = Unit{g, p.gh0[g] + h, p.gh[g] - h < hpu ? p.gh[g] - h : hpu};
    }
  return n;
}

// Units of the window GEMM with its A operand in tensor memory: whole head groups where the weight image, the
// accumulators and the row stages fit one SM, else the group cut into equal parts.  `nb` = output blocks per head.
int make_units_tm(const Plan& p, Unit* units, int nb, int cap) {
  int n = 0;
  for (int g = 0; g < p.G; ++g) {
    const int want = p.gh[g] < cap ? p.gh[g] : cap;
    const int hpu = gwt_heads_per_unit(p.Cp, p.dp, p.C, nb, want);
    if (hpu == 0) return -1;
    const int parts = (p.gh[g] + hpu - 1) / hpu;
    for (int i = 0, h = 0; i < parts; ++i) {
      const int take = (p.gh[g] - h + (parts - i) - 1) / (parts - i);
      if (n == kMaxUnits) return -1;
      units[n++] = Unit{g, p.gh0[g] + h, take};
      h += take;
    }
  }
  return n;
}

// Split of the output columns of a token GEMM with K = kvalid so that the resident weight image,
// the staging tile and at least three ring stages fit.
bool token_split(int C, int K, TokenSplit* ts) {
  const int natoms = (K + 63) / 64;
  {
    // all output columns in one CTA: with the weight image resident if it fits, else streamed through the ring
    const int NB = (int)align_up((size_t)C, 32);
    const size_t fixed = 1024 + (size_t)128 * NB * 2 + NB * 4 + 64;
    const size_t resident = (size_t)natoms * NB * 128, stage = 16384 + (size_t)NB * 128;
    if (NB <= 256 && fixed + resident + 4 * 16384 > kSmemBudget && fixed + 4 * stage <= kSmemBudget) {
      int S = (int)((kSmemBudget - fixed) / stage);
      if (S > 8) S = 8;
      *ts = TokenSplit{1, NB, S, natoms, 1};
      return true;
    }
  }
  for (int nsplit = 1; nsplit <= kMaxUnits; nsplit *= 2) {
    const int NB = (int)align_up((size_t)(C + nsplit - 1) / nsplit, 32);
    if (NB > 256) continue;
    const size_t fixed = 1024 + (size_t)natoms * NB * 128 + (size_t)128 * NB * 2 + NB * 4 + 64;
    if (fixed + 4 * 16384 > kSmemBudget) continue;
    int S = (int)((kSmemBudget - fixed) / 16384);
    if (S > 8) S = 8;
    *ts = TokenSplit{(C + NB - 1) / NB, NB, S, natoms, 0};
    return true;
  }
  return false;
}

FastGeom make_geom(const Plan& p) {
  FastGeom g{};
  g.B = p.B; g.H = p.H; g.W = p.W; g.C = p.C; g.nh = p.nh; g.d = p.d; g.dp = p.dp; g.G = p.G;
  g.nW = p.nW; g.nWw = p.nWw; g.nWh = p.nWh; g.T = p.T; g.n_windows = (long long)p.B * p.nW;
  long long qo = 0, dO = 0, lo = 0;
  for (int i = 0; i < p.G; ++i) {
    g.gh[i] = p.gh[i]; g.gs[i] = p.gs[i]; g.gh0[i] = p.gh0[i];
    g.qkv_off[i] = qo; g.do_off[i] = dO; g.l_off[i] = lo;
    qo += g.n_windows * p.gh[i] * 3 * 64 * p.dp;
    dO += g.n_windows * p.gh[i] * 64 * p.dp;
    lo += g.n_windows * p.gh[i] * 64;
  }
  return g;
}

// Scratch layouts (byte offsets).  The first 256 bytes of either scratch hold the device error word.
struct FwdScratch {
  size_t img[kMaxUnits], bias[kMaxUnits], pimg[kMaxUnits], pbias[kMaxUnits], total;
};
struct BwdScratch {
  size_t dO, dqkv, dummy, total;
};
// Weight images of the backward GEMMs (W^P transposed per unit, W_qkv transposed per column split).  A training
// forward call builds them next to its own images, into `saved`, so that the backward call launches no prep kernel.
struct BwdImages {
  size_t img[kMaxUnits], ximg[kMaxUnits], total;
};

int np_cols(int C) { return (int)align_up((size_t)C + 1, 64); }

// Extents of the two weight-gradient GEMM launches (dW_proj: which = 0, dW_qkv: which = 1).
struct GrShape {
  int M, NP, mbpc, nsplit;
};
GrShape gr_shape(const Plan& p, int which) {
  GrShape g{};
  g.M = which ? 3 * p.Ap : p.C;
  g.NP = which ? np_cols(p.C) : (int)align_up((size_t)p.Ap, 64);
  // dW_qkv: x is copied once for two M blocks of dqkv; dW_proj: two M blocks per CTA measured slower (fewer TMA stages)
  g.mbpc = which && 2 * g.NP <= 512 ? 2 : 1;
  const int mblocks = ((g.M + 127) / 128 + g.mbpc - 1) / g.mbpc;
  const long long ns = device_sm_count() / mblocks, cap = (p.T + 63) / 64;
  g.nsplit = (int)(ns < cap ? (ns < 1 ? 1 : ns) : cap);
  return g;
}

FwdScratch fwd_layout(const Plan& p, const Unit* units, int nu, const TokenSplit& ts) {
  FwdScratch s{};
  size_t off = 256;
  for (int i = 0; i < nu; ++i) {
    const size_t NT = (size_t)units[i].nheads * 3 * p.dp;
    s.img[i] = off; off += align_up(NT * p.Cp * 2, 256);
    s.bias[i] = off; off += align_up(NT * 4, 256);
  }
  for (int i = 0; i < ts.nsplit; ++i) {
    s.pimg[i] = off; off += align_up((size_t)ts.natoms * ts.NB * 128, 256);
    s.pbias[i] = off; off += align_up((size_t)ts.NB * 4, 256);
  }
  s.total = off;
  return s;
}

BwdImages bwd_images(const Plan& p, const Unit* units, int nu, const TokenSplit& tx) {
  BwdImages s{};
  size_t off = 0;
  for (int i = 0; i < nu; ++i) {
    s.img[i] = off; off += align_up((size_t)units[i].nheads * p.dp * p.Cp * 2, 256);
  }
  for (int i = 0; i < tx.nsplit; ++i) {
    s.ximg[i] = off; off += align_up((size_t)tx.natoms * tx.NB * 128, 256);
  }
  s.total = off;
  return s;
}

BwdScratch bwd_layout(const Plan& p) {
  BwdScratch s{};
  size_t off = 256;
  s.dO = off; off += align_up((size_t)p.T * p.nh * p.dp * 2, 256);
  s.dqkv = off; off += align_up((size_t)p.T * 3 * p.Ap * 2, 256);
  s.dummy = off; off += align_up((size_t)3 * p.C * p.C * 4, 256);
  s.total = off;
  return s;
}

}  // namespace

bool fast_path_ok(const Plan& p) {
  if (p.dtype != GSWA_BF16 || (p.flags & GSWA_FLAG_GENERIC)) return false;
  if (p.dqk != p.d || p.dv != p.d) return false;             // narrowed Q/K projections run on the shape-generic kernels
  if (p.M != 8 || p.d > 32 || (p.d & 1) || (p.C & 3) || p.C > 252 || p.G > 4) return false;
  if (p.nh * (p.d <= 16 ? 16 : 32) < 64) return false;       // padded rows must fill one TMA box of 64 columns
  if (p.nh * (p.d <= 16 ? 16 : 32) > 256) return false;      // the padded attention width is the N extent of one MMA (dW_proj)
  if (p.T >= (1LL << 30) / 4) return false;
  Plan q = p;
  q.dp = p.d <= 16 ? 16 : 32;
  q.Cp = (int)align_up((size_t)p.C, 64);
  q.Ap = p.nh * q.dp;
  Unit units[kMaxUnits];
  if (make_units(q, units, 2) <= 0 || make_units(q, units, 3) <= 0) return false;
  TokenSplit a, b;
  return token_split(p.C, q.Ap, &a) && token_split(p.C, 3 * q.Ap, &b);
}

void fast_plan_sizes(Plan* p) {
  p->fast = 1;
  p->dp = p->d <= 16 ? 16 : 32;
  p->Cp = (int)align_up((size_t)p->C, 64);
  p->Ap = p->nh * p->dp;
  Unit units[kMaxUnits], bunits[kMaxUnits];
  const int nu = make_units(*p, units, 2), bnu = make_units(*p, bunits, 3);
  TokenSplit tp, tx;
  token_split(p->C, p->Ap, &tp);
  token_split(p->C, 3 * p->Ap, &tx);
  const size_t T = (size_t)p->T;
  p->off_qkv = 0;
  p->off_A = align_up(T * 3 * p->nh * p->dp * 2, 256);
  p->off_L = p->off_A + align_up(T * p->Ap * 2, 256);
  p->off_bimg = p->off_L + align_up(T * p->nh * 4, 256);
  p->saved_bytes = p->off_bimg + bwd_images(*p, bunits, bnu, tx).total;
  p->fwd_scratch = fwd_layout(*p, units, nu, tp).total;
  p->infer_scratch = p->fwd_scratch + p->saved_bytes;
  p->bwd_scratch = bwd_layout(*p).total;
}

int fast_index_maps(const Plan& p, int group, int32_t* win_id, int32_t* slot, int32_t* region, int32_t* rel, cudaStream_t st) {
  return launch_fast_index_maps(make_geom(p), p.gs[group], win_id, slot, region, rel, st);
}

// A second stream per device for the two weight-gradient GEMMs of the backward pass.  Nothing downstream reads
// dW_proj or dW_qkv, so these kernels need not sit on the critical path: forked off the caller's stream with
// events, their ramp-down (every CTA adding its accumulator into the gradients through the L2 atomic units, SMs
// mostly idle) overlaps the start of the next kernel, whose CTAs take over the SMs as they come free.
struct SideStream {
  cudaStream_t s;
  cudaEvent_t fork1, fork2, join;
  std::mutex use;               // one backward call at a time enqueues on it (its events are re-recorded per call)
};
static SideStream* side_stream() {
  static std::mutex mu;
  static SideStream table[64];
  static int state[64];                     // 0 not tried, 1 ready, -1 unavailable
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return nullptr; }
  std::lock_guard<std::mutex> lk(mu);
  if (state[dev] == 0) {
    SideStream& t = table[dev];
    const bool ok = cudaStreamCreateWithFlags(&t.s, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&t.fork1, cudaEventDisableTiming) == cudaSuccess &&
                    cudaEventCreateWithFlags(&t.fork2, cudaEventDisableTiming) == cudaSuccess &&
                    cudaEventCreateWithFlags(&t.join, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) (void)cudaGetLastError();
    state[dev] = ok ? 1 : -1;
  }
  return state[dev] == 1 ? &table[dev] : nullptr;
}

// Work units of the attention kernels: one head per CTA when the unit table has room for every head (more,
// smaller CTAs per SM hide each other's latency), otherwise the head ranges of the GEMM units.
static void attn_units(const Plan& p, const FastGeom& geo, const Unit* units, int nu, AttnLaunch* L) {
  L->geo = geo;
  Unit heads[kMaxUnits];
  if (p.nh <= kMaxUnits) {
    nu = 0;
    for (int g = 0; g < p.G; ++g)
      for (int h = 0; h < p.gh[g]; ++h) heads[nu++] = Unit{g, p.gh0[g] + h, 1};
    units = heads;
  }
  L->nunits = nu;
  for (int i = 0; i < nu; ++i) {
    const Unit& u = units[i];
    const int hl0 = u.h0 - p.gh0[u.g], gh = p.gh[u.g];
    AttnUnit& a = L->u[i];
    a.g = u.g; a.h0 = u.h0; a.nheads = u.nheads; a.s = p.gs[u.g];
    a.qkv_off = geo.qkv_off[u.g] + (long long)hl0 * 3 * 64 * p.dp;
    a.do_off = geo.do_off[u.g] + (long long)hl0 * 64 * p.dp;
    a.l_off = geo.l_off[u.g] + (long long)hl0 * 64;
    a.qkv_wstride = (long long)gh * 3 * 64 * p.dp;
    a.do_wstride = (long long)gh * 64 * p.dp;
    a.l_wstride = (long long)gh * 64;
  }
}

int fast_forward(const Plan& p, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                 const void* b_proj, const void* table, void* y, void* saved, void* scratch, bool want_L,
                 cudaStream_t st, const void* resid) {
  using bf = __nv_bfloat16;
  // Units of the attention kernels when the layer has more heads than one-head units fit (cap 2), and of the QKV
  // GEMM: whole groups with the A operand in tensor memory where the rows can be fetched by bulk copies, else
  // units of at most two heads fed by the copy loaders.
  Unit units2[kMaxUnits], units[kMaxUnits];
  const int nu2 = make_units(p, units2, 2);
  const bool tm = !(p.flags & (GSWA_FLAG_FUSED_FWD | GSWA_FLAG_COPY_LOADERS)) && gwt_usable(x, p.C, p.H, p.W, p.gs, p.G);
  int nu = tm ? make_units_tm(p, units, 3, kMaxHeads) : -1;
  const bool use_tm = nu > 0;
  if (!use_tm) {
    nu = nu2;
    for (int i = 0; i < nu2; ++i) units[i] = units2[i];
  }
  TokenSplit tp;
  if (nu <= 0 || nu2 <= 0 || !token_split(p.C, p.Ap, &tp)) return GSWA_ERR_UNSUPPORTED;
  const FwdScratch fs = fwd_layout(p, units, nu, tp);
  const FastGeom geo = make_geom(p);
  char* sc = static_cast<char*>(scratch);
  char* sv = static_cast<char*>(saved);
  int* err = reinterpret_cast<int*>(sc);
  bf* qkv = reinterpret_cast<bf*>(sv + p.off_qkv);
  bf* A = reinterpret_cast<bf*>(sv + p.off_A);
  float* Lt = reinterpret_cast<float*>(sv + p.off_L);

  // With a spare K column (C < Cp) the QKV bias rides in the weight image and meets a column of ones in the A operand.
  const bool fold_bias = p.C < p.Cp && b_qkv != nullptr && !(p.flags & GSWA_FLAG_FUSED_FWD);
  // Likewise the output projection's bias meets the ones that column d of head 0 of the attention output holds.
  const bool fold_pbias = p.d < p.dp && b_proj != nullptr;
  PrepJob jobs[16];
  int nj = 0;
  for (int i = 0; i < nu; ++i)
    jobs[nj++] = PrepJob{PREP_QKV, (const bf*)w_qkv, (const bf*)b_qkv, (unsigned char*)sc + fs.img[i],
                         (float*)(sc + fs.bias[i]), p.C, p.d, p.dp, units[i].h0, units[i].nheads, 0,
                         units[i].nheads * 3 * p.dp, p.Cp, p.Ap, fold_bias ? 1 : 0};
  for (int i = 0; i < tp.nsplit; ++i)
    jobs[nj++] = PrepJob{PREP_PROJ, (const bf*)w_proj, (const bf*)b_proj, (unsigned char*)sc + fs.pimg[i],
                         (float*)(sc + fs.pbias[i]), p.C, p.d, p.dp, 0, 0, i * tp.NB, tp.NB, tp.natoms * 64, p.Ap,
                         fold_pbias ? 1 : 0};
  int rc = GSWA_OK;
  if (want_L) {
    // images of the backward GEMMs (see BwdImages), in the same launch when the job table has room
    Unit bunits[kMaxUnits];
    const int bnu = make_units(p, bunits, 3);
    TokenSplit tx;
    if (bnu <= 0 || !token_split(p.C, 3 * p.Ap, &tx)) return GSWA_ERR_UNSUPPORTED;
    const BwdImages bi = bwd_images(p, bunits, bnu, tx);
    unsigned char* base = reinterpret_cast<unsigned char*>(sv + p.off_bimg);
    if (nj + bnu + tx.nsplit > 16) {
      if ((rc = launch_prep(jobs, nj, st, err))) return rc;
      nj = 0;
    }
    for (int i = 0; i < bnu; ++i)
      jobs[nj++] = PrepJob{PREP_PROJ_T, (const bf*)w_proj, nullptr, base + bi.img[i], nullptr, p.C, p.d,
                           p.dp, bunits[i].h0, bunits[i].nheads, 0, bunits[i].nheads * p.dp, p.Cp, p.Ap};
    for (int i = 0; i < tx.nsplit; ++i)
      jobs[nj++] = PrepJob{PREP_QKV_T, (const bf*)w_qkv, nullptr, base + bi.ximg[i], nullptr, p.C, p.d,
                           p.dp, 0, 0, i * tx.NB, tx.NB, tx.natoms * 64, p.Ap};
  }
  if ((rc = launch_prep(jobs, nj, st, err))) return rc;     // also zeroes the error word

  const float qscale = 1.4426950408889634f / sqrtf((float)p.d);   // d^-1/2 and log2(e): attention works in the log2 domain
  int maxh = 0;
  for (int i = 0; i < nu; ++i) maxh = units[i].nheads > maxh ? units[i].nheads : maxh;
  if ((p.flags & GSWA_FLAG_FUSED_FWD) && fw_smem_bytes(p.Cp, p.dp, maxh, nullptr) != 0) {
    // fused (opt-in): projection and attention of a window pair in one CTA; q,k,v reach HBM only when
    // the backward pass will need them.  Measured slower than the two kernels below at C = 180 (the
    // twelve attention warps that fit beside the GEMM's shared memory cannot hide their own latency).
    FWLaunch fw{};
    fw.geo = geo; fw.table = (const bf*)table; fw.A = A; fw.err = err;
    for (int i = 0; i < nu; ++i) {
      const Unit& u = units[i];
      FWUnit& w = fw.u[i];
      const int hl0 = u.h0 - p.gh0[u.g];
      w.X = (const bf*)x; w.lda = p.C; w.kvalid = p.C;
      w.H = p.H; w.W = p.W; w.s = p.gs[u.g]; w.nW = p.nW; w.nWw = p.nWw; w.n_windows = geo.n_windows;
      w.Bimg = (const unsigned char*)sc + fs.img[i];
      w.bias = (const float*)(sc + fs.bias[i]);
      w.qscale = qscale;
      w.h0 = u.h0; w.nheads = u.nheads;
      w.qkv_out = want_L ? qkv + geo.qkv_off[u.g] + (long long)hl0 * 3 * 64 * p.dp : nullptr;
      w.qkv_wstride = (long long)p.gh[u.g] * 3 * 64 * p.dp;
      w.lt = want_L ? Lt + geo.l_off[u.g] + (long long)hl0 * 64 : nullptr;
      w.l_wstride = (long long)p.gh[u.g] * 64;
    }
    if ((rc = launch_fw(fw, nu, p.Cp, p.dp, st))) return rc;
  } else {
    GWLaunch gw{};
    gw.err = err;
    for (int i = 0; i < nu; ++i) {
      const Unit& u = units[i];
      GWUnit& w = gw.u[i];
      w.A = (const bf*)x; w.lda = p.C; w.kvalid = p.C;
      w.H = p.H; w.W = p.W; w.s = p.gs[u.g]; w.nW = p.nW; w.nWw = p.nWw; w.n_windows = geo.n_windows;
      w.Bimg = (const unsigned char*)sc + fs.img[i];
      w.bias = fold_bias || b_qkv == nullptr ? nullptr : (const float*)(sc + fs.bias[i]);
      w.ones_col = fold_bias ? 1 : 0;
      w.out = qkv + geo.qkv_off[u.g] + (long long)(u.h0 - p.gh0[u.g]) * 3 * 64 * p.dp;
      w.win_stride = (long long)p.gh[u.g] * 3 * 64 * p.dp;
      // copy loaders: one accumulator chunk per unit when its columns fit one MMA (N <= 256), else one per head;
      // A operand in tensor memory: one chunk per head (the chunks of a tile are drained while the next ones fill)
      if (!use_tm && u.nheads * 3 * p.dp <= 256) { w.nchunks = 1; w.cw = u.nheads * 3 * p.dp; }
      else { w.nchunks = u.nheads; w.cw = 3 * p.dp; }
      w.q_every3 = 1;
      w.qscale = qscale;
    }
    if ((rc = use_tm ? launch_gwt(gw, nu, p.Cp, p.dp, st, "qkv_gemm") : launch_gw(gw, nu, p.Cp, p.dp, st, "qkv_gemm"))) return rc;

    AttnLaunch al{};
    attn_units(p, geo, units2, nu2, &al);
    al.qkv = qkv; al.table = (const bf*)table; al.A = A; al.Lt = want_L ? Lt : nullptr; al.err = err;
    al.scale = 1.0f / sqrtf((float)p.d);
    if ((rc = launch_attn_fwd(al, st))) return rc;
  }

  GTLaunch gt{};
  if ((rc = make_tmap(&gt.tmA, A, p.T, p.Ap, 128))) return rc;
  gt.natoms = tp.natoms; gt.rows = p.T;
  gt.out = (bf*)y; gt.ldo = p.C; gt.resid = (const bf*)resid; gt.NB = tp.NB; gt.nstages = tp.nstages; gt.stream_b = tp.stream_b; gt.err = err;
  for (int i = 0; i < tp.nsplit; ++i) {
    const int col0 = i * tp.NB;
    gt.s[i] = GTSplit{(const unsigned char*)sc + fs.pimg[i], fold_pbias || b_proj == nullptr ? nullptr : (const float*)(sc + fs.pbias[i]), col0,
                      (p.C - col0 < tp.NB ? p.C - col0 : tp.NB)};
  }
  return launch_gt(gt, tp.nsplit, st, "proj_gemm");
}

int fast_backward(const Plan& p, const void* x, const void* w_qkv, const void* w_proj, const void* table,
                  const void* saved, const void* dy, void* dx, float* dw_qkv, float* db_qkv, float* dw_proj,
                  float* db_proj, float* dtable, void* scratch, cudaStream_t st) {
  using bf = __nv_bfloat16;
  Unit units[kMaxUnits];
  const int nu = make_units(p, units, 3);
  TokenSplit tx;
  if (nu <= 0 || !token_split(p.C, 3 * p.Ap, &tx)) return GSWA_ERR_UNSUPPORTED;
  const BwdScratch bs = bwd_layout(p);
  const FastGeom geo = make_geom(p);
  char* sc = static_cast<char*>(scratch);
  const char* sv = static_cast<const char*>(saved);
  int* err = reinterpret_cast<int*>(sc);
  const bf* qkv = reinterpret_cast<const bf*>(sv + p.off_qkv);
  const bf* A = reinterpret_cast<const bf*>(sv + p.off_A);
  const float* Lt = reinterpret_cast<const float*>(sv + p.off_L);
  bf* dO = reinterpret_cast<bf*>(sc + bs.dO);
  bf* dqkv = reinterpret_cast<bf*>(sc + bs.dqkv);
  float* dummy = reinterpret_cast<float*>(sc + bs.dummy);      // (the error word was zeroed together with the gradients)

  int rc = GSWA_OK;
  const BwdImages bi = bwd_images(p, units, nu, tx);          // built by the forward call
  const unsigned char* bimg = reinterpret_cast<const unsigned char*>(sv + p.off_bimg);

  // ---- everything that can fail on the host (tensor maps) comes first: once the side stream has been forked off,
  // the only remaining failures are launch errors, and those still pass through the join below
  GRLaunch grp{}, grx{};
  GTLaunch gt{};
  AttnLaunch al{};
  const bool want_dwproj = dw_proj || db_proj, want_dwqkv = dw_qkv || db_qkv;
  if (want_dwproj && (rc = make_tmap(&grp.tm, A, p.T, p.Ap, 64))) return rc;
  if (dx && (rc = make_tmap(&gt.tmA, dqkv, p.T, 3 * p.Ap, 128))) return rc;
  if (want_dwqkv && (rc = make_tmap(&grx.tm, dqkv, p.T, 3 * p.Ap, 64))) return rc;
  attn_units(p, geo, units, nu, &al);
  bool one_head_units = true;
  for (int i = 0; i < al.nunits; ++i) one_head_units = one_head_units && al.u[i].nheads == 1;
  const bool tc_attn = one_head_units && (p.flags & GSWA_FLAG_TCGEN05_ATTN);
  if (tc_attn) {
    if ((rc = make_tmap_window(&al.tm_out, dqkv, (long long)p.B * p.H, p.W, 3 * p.Ap, p.dp, 8, 8, true))) return rc;
    // A window of a shifted group that wraps around the image edge is stored as four boxes.  Their shared-
    // memory sources must start on 128-byte boundaries, which an even shift guarantees; units with another
    // shift store such windows row by row.
    al.wrap_s = 0;
    for (int i = 0; i < al.nunits && al.wrap_s == 0; ++i)
      if (al.u[i].s > 0 && al.u[i].s % 2 == 0) al.wrap_s = al.u[i].s;
    if (al.wrap_s > 0) {
      const int e = 8 - al.wrap_s, s = al.wrap_s;
      for (int k = 0; k < 4; ++k)
        if ((rc = make_tmap_window(&al.tm_wrap[k], dqkv, (long long)p.B * p.H, p.W, 3 * p.Ap, p.dp, (k & 1) ? s : e, (k & 2) ? s : e, false)))
          return rc;
    }
  }

  // the weight-gradient GEMMs go to the side stream (not while kernels are being timed one by one)
  SideStream* ss = profiling_enabled() ? nullptr : side_stream();
  std::unique_lock<std::mutex> ss_lock;
  if (ss) ss_lock = std::unique_lock<std::mutex>(ss->use);
  if (ss && (cudaEventRecord(ss->fork1, st) != cudaSuccess || cudaStreamWaitEvent(ss->s, ss->fork1, 0) != cudaSuccess)) {
    (void)cudaGetLastError();
    ss = nullptr;                                             // nothing was forked: stay on the caller's stream
  }
  cudaStream_t s2 = ss ? ss->s : st;
  // From here on every exit joins the side stream back into the caller's stream: whatever was enqueued there is
  // ordered before anything the caller enqueues next (and a stream capture is not left with an open fork).
  auto finish = [&](int code) {
    if (ss && (cudaEventRecord(ss->join, s2) != cudaSuccess || cudaStreamWaitEvent(st, ss->join, 0) != cudaSuccess)) {
      const int jrc = check_launch();
      return code ? code : jrc;
    }
    return code;
  };

  if (want_dwproj) {
    // dW^P = dy^T A (A fetched by TMA); db^P rides on the ones column of A when the head dim is padded
    grp.tma_is_L = 0;
    grp.P = (const bf*)dy; grp.ldp = p.C; grp.pvalid = p.C;
    const GrShape gs = gr_shape(p, 0);
    grp.Ap = p.Ap; grp.dp = p.dp; grp.d = p.d; grp.C = p.C; grp.M = gs.M; grp.rows = p.T;
    grp.NP = gs.NP; grp.mbpc = gs.mbpc; grp.nsplit = gs.nsplit;
    grp.out = dw_proj ? dw_proj : dummy; grp.colsum = p.d < p.dp ? db_proj : nullptr; grp.err = err;
    if ((rc = launch_gr(grp, s2, "dwproj_gemm"))) return finish(rc);
    if (db_proj && p.d == p.dp && (rc = launch_colsum_bf16((const bf*)dy, p.T, p.C, p.C, db_proj, s2))) return finish(rc);
  }

  // (dW^P runs first so that the dO tiles written next are still in L2 when the attention kernel reads them)
  // dO tiles = dy W^P restricted to each unit's heads, rows gathered in that group's window order
  GWLaunch gw{};
  gw.err = err;
  for (int i = 0; i < nu; ++i) {
    const Unit& u = units[i];
    GWUnit& w = gw.u[i];
    w.A = (const bf*)dy; w.lda = p.C; w.kvalid = p.C;
    w.H = p.H; w.W = p.W; w.s = p.gs[u.g]; w.nW = p.nW; w.nWw = p.nWw; w.n_windows = geo.n_windows;
    w.Bimg = bimg + bi.img[i];
    w.bias = nullptr;
    w.out = dO + geo.do_off[u.g] + (long long)(u.h0 - p.gh0[u.g]) * 64 * p.dp;
    w.win_stride = (long long)p.gh[u.g] * 64 * p.dp;
    w.nchunks = 1; w.cw = u.nheads * p.dp; w.q_every3 = 0; w.qscale = 1.f;
  }
  // (dO = dy W^P has few columns per tile: with the A operand in tensor memory its tile period is set by the load
  // latency of the two tiles it keeps in flight, 87 us against 62 us for the copy-fed kernel at C = 180, so the
  // backward pass keeps the copy loaders)
  if ((rc = launch_gw(gw, nu, p.Cp, p.dp, st, "dattn_gemm"))) return finish(rc);

  al.qkv = qkv; al.table = (const bf*)table; al.Lt = const_cast<float*>(Lt); al.dO = dO; al.dqkv = dqkv;
  al.dtable = dtable; al.scale = 1.0f / sqrtf((float)p.d); al.err = err;
  if ((rc = tc_attn ? launch_attn_bwd_tc(al, st) : launch_attn_bwd(al, st))) return finish(rc);
  // dqkv is complete on the caller's stream: dW_qkv may start on the side stream, next to dx
  if (ss && (cudaEventRecord(ss->fork2, st) != cudaSuccess || cudaStreamWaitEvent(s2, ss->fork2, 0) != cudaSuccess))
    return finish(check_launch());

  if (dx) {
    gt.natoms = tx.natoms; gt.rows = p.T;
    gt.out = (bf*)dx; gt.ldo = p.C; gt.NB = tx.NB; gt.nstages = tx.nstages; gt.stream_b = tx.stream_b; gt.err = err;
    for (int i = 0; i < tx.nsplit; ++i) {
      const int col0 = i * tx.NB;
      gt.s[i] = GTSplit{bimg + bi.ximg[i], nullptr, col0, (p.C - col0 < tx.NB ? p.C - col0 : tx.NB)};
    }
    if ((rc = launch_gt(gt, tx.nsplit, st, "dx_gemm"))) return finish(rc);
  }
  if (want_dwqkv) {
    // dW_qkv = dqkv^T x (dqkv fetched by TMA); db_qkv from a column of ones appended to x
    grx.tma_is_L = 1;
    grx.P = (const bf*)x; grx.ldp = p.C; grx.pvalid = p.C;
    const GrShape gs = gr_shape(p, 1);
    grx.Ap = p.Ap; grx.dp = p.dp; grx.d = p.d; grx.C = p.C; grx.M = gs.M; grx.rows = p.T;
    grx.NP = gs.NP; grx.mbpc = gs.mbpc; grx.nsplit = gs.nsplit;
    grx.out = dw_qkv ? dw_qkv : dummy; grx.colsum = db_qkv; grx.err = err;
    if ((rc = launch_gr(grx, s2, "dwqkv_gemm"))) return finish(rc);
  }
  // the caller's stream continues only after the side stream's work
  return finish(GSWA_OK);
}

}  // namespace gswa
