// Host side of libgswa: descriptor validation, buffer planning and the extern "C" entry points.
#include <atomic>
#include <mutex>
#include <vector>
#include <cstdio>
#include <cstring>

#include "fast.cuh"
#include "gswa_internal.h"

namespace gswa {

static std::atomic<uint64_t> g_launches{0};
static thread_local char g_cuda_msg[256] = "no CUDA error recorded";

// ---- optional per-launch timing (gswa_profile_enable / gswa_profile_read)
struct ProfRecord {
  const char* name;
  cudaEvent_t e0, e1;
};
static std::mutex g_prof_mu;
static bool g_prof_on = false;
static std::vector<ProfRecord> g_prof;

KernelScope::KernelScope(const char* name, cudaStream_t s) : st(s), slot(-1) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (!g_prof_on) return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  ProfRecord r{name, nullptr, nullptr};
  if (cudaEventCreate(&r.e0) != cudaSuccess || cudaEventCreate(&r.e1) != cudaSuccess) return;
  cudaEventRecord(r.e0, st);
  g_prof.push_back(r);
  slot = (int)g_prof.size() - 1;
}

KernelScope::~KernelScope() {
  if (slot < 0) return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  if (slot < (int)g_prof.size()) cudaEventRecord(g_prof[slot].e1, st);
}

bool profiling_enabled() { return g_prof_on; }

int device_sm_count() {
  constexpr int kMaxDev = 64;
  static std::atomic<int> cache[kMaxDev];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) { (void)cudaGetLastError(); return 148; }
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { (void)cudaGetLastError(); n = 148; }
    cache[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

int check_launch() {
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return GSWA_OK;
  snprintf(g_cuda_msg, sizeof(g_cuda_msg), "CUDA error: %s", cudaGetErrorString(e));
  return GSWA_ERR_CUDA;
}

static int cuda_rc(cudaError_t e) {
  if (e == cudaSuccess) return GSWA_OK;
  snprintf(g_cuda_msg, sizeof(g_cuda_msg), "CUDA error: %s", cudaGetErrorString(e));
  (void)cudaGetLastError();
  return GSWA_ERR_CUDA;
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr size_t kMaxBlockSmem = 227 * 1024;   // opt-in dynamic shared memory of one block on sm_100

int make_plan(const gswa_desc* desc, Plan* p) {
  if (desc == nullptr || p == nullptr) return GSWA_ERR_NULL;
  if (desc->group_heads == nullptr || desc->group_shift == nullptr) return GSWA_ERR_NULL;
  memset(p, 0, sizeof(*p));
  p->B = desc->B; p->H = desc->H; p->W = desc->W; p->C = desc->C;
  p->nh = desc->num_heads; p->M = desc->window; p->G = desc->num_groups;
  p->dtype = desc->dtype; p->flags = desc->flags;
  if (p->B < 0 || p->H <= 0 || p->W <= 0 || p->C <= 0 || p->nh <= 0 || p->M <= 0 || p->G <= 0) return GSWA_ERR_SHAPE;
  if (p->G > kMaxGroups || p->nh > kMaxHeads) return GSWA_ERR_UNSUPPORTED;
  if (p->C % p->nh != 0 || p->H % p->M != 0 || p->W % p->M != 0) return GSWA_ERR_SHAPE;
  if (p->dtype != GSWA_F32 && p->dtype != GSWA_BF16) return GSWA_ERR_UNSUPPORTED;
  p->d = p->C / p->nh;
  p->N = p->M * p->M;
  int sum = 0;
  for (int g = 0; g < p->G; ++g) {
    p->gh[g] = desc->group_heads[g];
    p->gs[g] = desc->group_shift[g];
    p->gh0[g] = sum;
    if (p->gh[g] <= 0 || p->gs[g] < 0 || p->gs[g] >= p->M) return GSWA_ERR_SHAPE;
    sum += p->gh[g];
  }
  if (sum != p->nh) return GSWA_ERR_SHAPE;
  if (desc->qk_dim < 0 || desc->v_dim < 0) return GSWA_ERR_SHAPE;
  p->dqk = desc->qk_dim ? desc->qk_dim : p->d;
  p->dv = desc->v_dim ? desc->v_dim : p->d;
  p->Cq = p->nh * p->dqk; p->Cv = p->nh * p->dv; p->Cqkv = 2 * p->Cq + p->Cv;
  if (p->N > 144 || p->dqk > 64 || p->dv > 64) return GSWA_ERR_UNSUPPORTED;
  const long long T = (long long)p->B * p->H * p->W;
  if (T * 3 * p->C >= (1LL << 40) || T >= (1LL << 31) / 2) return GSWA_ERR_UNSUPPORTED;
  p->T = T;
  p->nWh = p->H / p->M; p->nWw = p->W / p->M; p->nW = p->nWh * p->nWw;
  p->esize = p->dtype == GSWA_F32 ? 4 : 2;
  p->fast = 0;
  // generic path: saved = qkv[T,3C] | A[T,C] | L[T,nh] (float)
  const size_t es = (size_t)p->esize;
  p->off_qkv = 0;
  p->off_A = align_up((size_t)T * p->Cqkv * es, 256);
  p->off_L = p->off_A + align_up((size_t)T * p->Cv * es, 256);
  p->saved_bytes = p->off_L + align_up((size_t)T * p->nh * sizeof(float), 256);
  p->fwd_scratch = 0;
  p->infer_scratch = p->saved_bytes;
  p->bwd_scratch = align_up((size_t)T * (p->Cv + p->Cqkv) * es, 256);  // dA[T,Cv] | dqkv[T,Cqkv]
  if (fast_path_ok(*p)) {
    fast_plan_sizes(p);
  } else if (generic_attn_fwd_smem(*p) > kMaxBlockSmem || generic_attn_bwd_smem(*p) > kMaxBlockSmem) {
    return GSWA_ERR_UNSUPPORTED;   // one (window, head) problem must fit the shared memory of one block
  }
  return GSWA_OK;
}

static bool misaligned(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) != 0; }

// Argument checks and dispatch of one GSWA forward / backward for an already validated plan (shared by the plain
// entry points and by the layer entry points of astl.cu, which add a skip connection through `resid`).
int forward_impl(const Plan& p, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj, const void* b_proj,
                 const void* bias_table, void* y, void* saved, void* scratch, size_t scratch_bytes, cudaStream_t st,
                 const void* resid) {
  if (!x || !w_qkv || !w_proj || !bias_table || !y) return GSWA_ERR_NULL;
  if (p.T == 0) return GSWA_OK;
  const size_t need = saved ? p.fwd_scratch : p.infer_scratch;
  if (need > 0 && scratch == nullptr) return GSWA_ERR_NULL;
  if (misaligned(x) || misaligned(w_qkv) || misaligned(b_qkv) || misaligned(w_proj) || misaligned(b_proj) ||
      misaligned(bias_table) || misaligned(y) || misaligned(saved) || misaligned(scratch) || misaligned(resid))
    return GSWA_ERR_ALIGN;
  if (scratch_bytes < need) return GSWA_ERR_WORKSPACE;
  if (p.fast) {
    void* carry = saved ? saved : static_cast<char*>(scratch) + p.fwd_scratch;
    return fast_forward(p, x, w_qkv, b_qkv, w_proj, b_proj, bias_table, y, carry, scratch, saved != nullptr, st, resid);
  }
  void* carry = saved ? saved : scratch;
  return generic_forward(p, x, w_qkv, b_qkv, w_proj, b_proj, bias_table, y, carry, st, resid);
}

int backward_impl(const Plan& p, const void* x, const void* w_qkv, const void* w_proj, const void* bias_table,
                  const void* saved, const void* dy, void* dx, float* dw_qkv, float* db_qkv, float* dw_proj, float* db_proj,
                  float* dbias_table, void* scratch, size_t scratch_bytes, cudaStream_t st) {
  if (!x || !w_qkv || !w_proj || !bias_table || !saved || !dy) return GSWA_ERR_NULL;
  if (p.bwd_scratch > 0 && scratch == nullptr) return GSWA_ERR_NULL;
  if (misaligned(x) || misaligned(w_qkv) || misaligned(w_proj) || misaligned(bias_table) || misaligned(saved) ||
      misaligned(dy) || misaligned(dx) || misaligned(dw_qkv) || misaligned(db_qkv) || misaligned(dw_proj) ||
      misaligned(db_proj) || misaligned(dbias_table) || misaligned(scratch))
    return GSWA_ERR_ALIGN;
  if (scratch_bytes < p.bwd_scratch) return GSWA_ERR_WORKSPACE;
  int rc;
  {
    // one launch zeroes the parameter gradients (unless they accumulate) and, on the tensor-core path, the error
    // word at the head of the scratch buffer
    const size_t C = (size_t)p.C, Q = (size_t)p.Cqkv, Cv = (size_t)p.Cv, nrel = (size_t)(2 * p.M - 1) * (2 * p.M - 1);
    const bool z = !(p.flags & GSWA_FLAG_ACCUMULATE);
    float* const ptrs[6] = {z ? dw_qkv : nullptr, z ? db_qkv : nullptr, z ? dw_proj : nullptr, z ? db_proj : nullptr,
                            z ? dbias_table : nullptr, p.fast && p.T > 0 ? static_cast<float*>(scratch) : nullptr};
    const long long counts[6] = {(long long)(Q * C), (long long)Q, (long long)(C * Cv), (long long)C,
                                 (long long)(nrel * p.nh), 64};
    if ((rc = launch_zero(ptrs, counts, 6, st))) return rc;
  }
  if (p.T == 0) return GSWA_OK;
  if (p.fast)
    return fast_backward(p, x, w_qkv, w_proj, bias_table, saved, dy, dx, dw_qkv, db_qkv, dw_proj, db_proj, dbias_table,
                         scratch, st);
  return generic_backward(p, x, w_qkv, w_proj, bias_table, saved, dy, dx, dw_qkv, db_qkv, dw_proj, db_proj,
                          dbias_table, scratch, st);
}

// Scratch of gswa_forward_static: part of the device image, so no allocation call is ever made for
// it.  In host code this name is only a handle; the device address is looked up per device below.
static __device__ __align__(256) unsigned char g_static_scratch[GSWA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mu;
static void* g_static_ptr[kMaxDevices] = {};
static bool g_static_has_word[kMaxDevices] = {};   // the last gswa_forward_static on the device left an error word at the head of the array

// Device address of g_static_scratch on the current device (looked up once per device).
static int static_scratch(void** out) {
  int dev = -1;
  int rc = cuda_rc(cudaGetDevice(&dev));
  if (rc) return rc;
  if (dev < 0 || dev >= kMaxDevices) return GSWA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    rc = cuda_rc(cudaGetSymbolAddress(&ptr, g_static_scratch));
    if (rc) return rc;
    if (ptr == nullptr) return GSWA_ERR_CUDA;
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return GSWA_OK;
}

}  // namespace gswa

using namespace gswa;

extern "C" {

int gswa_workspace_query(const gswa_desc* desc, size_t* saved_bytes, size_t* fwd_scratch_bytes,
                         size_t* infer_scratch_bytes, size_t* bwd_scratch_bytes) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (saved_bytes) *saved_bytes = p.saved_bytes;
  if (fwd_scratch_bytes) *fwd_scratch_bytes = p.fwd_scratch;
  if (infer_scratch_bytes) *infer_scratch_bytes = p.infer_scratch;
  if (bwd_scratch_bytes) *bwd_scratch_bytes = p.bwd_scratch;
  return GSWA_OK;
}

int gswa_forward(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                 const void* b_proj, const void* bias_table, void* y, void* saved, void* scratch,
                 size_t scratch_bytes, void* cuda_stream) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  return forward_impl(p, x, w_qkv, b_qkv, w_proj, b_proj, bias_table, y, saved, scratch, scratch_bytes,
                      reinterpret_cast<cudaStream_t>(cuda_stream), nullptr);
}

int gswa_forward_static(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv,
                        const void* w_proj, const void* b_proj, const void* bias_table, void* y, void* cuda_stream) {
  Plan p;
  int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (p.infer_scratch > (size_t)GSWA_STATIC_SCRATCH_BYTES) return GSWA_ERR_WORKSPACE;   // layer too large for the built-in array
  void* scratch = nullptr;
  if ((rc = static_scratch(&scratch))) return rc;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) {
      std::lock_guard<std::mutex> lk(g_static_mu);
      g_static_has_word[dev] = p.fast && p.T > 0;          // the generic kernels have no bounded waits and keep no word
    }
  }
  // same path as gswa_forward with saved == NULL; the device error word at the head of the scratch
  // is cleared by that path on every call
  return gswa_forward(desc, x, w_qkv, b_qkv, w_proj, b_proj, bias_table, y, nullptr, scratch,
                      (size_t)GSWA_STATIC_SCRATCH_BYTES, cuda_stream);
}

int gswa_backward(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                  const void* bias_table, const void* saved, const void* dy, void* dx, float* dw_qkv,
                  float* db_qkv, float* dw_proj, float* db_proj, float* dbias_table, void* scratch,
                  size_t scratch_bytes, void* cuda_stream) {
  (void)b_qkv;
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  return backward_impl(p, x, w_qkv, w_proj, bias_table, saved, dy, dx, dw_qkv, db_qkv, dw_proj, db_proj, dbias_table,
                       scratch, scratch_bytes, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int gswa_index_maps(const gswa_desc* desc, int32_t group, int32_t* win, int32_t* slot, int32_t* region,
                    int32_t* token_of, int32_t* rel_index, void* cuda_stream) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (group < 0 || group >= p.G) return GSWA_ERR_SHAPE;
  return launch_index_maps(p, group, win, slot, region, token_of, rel_index, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int gswa_debug_index_maps(const gswa_desc* desc, int32_t group, int32_t* win_id, int32_t* slot, int32_t* region,
                          int32_t* rel_index, void* cuda_stream) {
  Plan p;
  int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (group < 0 || group >= p.G) return GSWA_ERR_SHAPE;
  if (p.T == 0) return GSWA_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (p.fast) return fast_index_maps(p, group, win_id, slot, region, rel_index, st);
  if ((slot || region || rel_index) && (rc = launch_index_maps(p, group, nullptr, slot, region, nullptr, rel_index, st))) return rc;
  return win_id ? launch_batch_window_ids(p, group, win_id, st) : GSWA_OK;
}

int gswa_debug_expire_wait(const gswa_desc* desc, void* scratch, void* cuda_stream) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (!p.fast) return GSWA_ERR_UNSUPPORTED;        // only the tensor-core path keeps an error word in its scratch
  if (scratch == nullptr) return GSWA_ERR_NULL;
  if (misaligned(scratch)) return GSWA_ERR_ALIGN;
  return launch_wait_timeout(static_cast<int*>(scratch), reinterpret_cast<cudaStream_t>(cuda_stream));
}

int gswa_static_status(void* cuda_stream) {
  void* scratch = nullptr;
  int rc = static_scratch(&scratch);
  if (rc) return rc;
  {
    int dev = 0;
    if ((rc = cuda_rc(cudaGetDevice(&dev)))) return rc;
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (dev < 0 || dev >= kMaxDevices || !g_static_has_word[dev]) return GSWA_OK;
  }
  int word = 0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  rc = cuda_rc(cudaMemcpyAsync(&word, scratch, sizeof(int), cudaMemcpyDeviceToHost, st));
  if (rc == GSWA_OK) rc = cuda_rc(cudaStreamSynchronize(st));
  if (rc) return rc;
  return word == 0 ? GSWA_OK : GSWA_ERR_DEVICE;
}

int gswa_step_host(const gswa_desc* desc, const void* x, const void* w_qkv, const void* b_qkv, const void* w_proj,
                   const void* b_proj, const void* bias_table, const void* dy, void* y, void* dx, float* dw_qkv,
                   float* db_qkv, float* dw_proj, float* db_proj, float* dbias_table, void* arena,
                   size_t arena_bytes, size_t* arena_bytes_needed, void* cuda_stream) {
  Plan p;
  int rc = make_plan(desc, &p);
  if (rc) return rc;
  const size_t es = (size_t)p.esize, C = (size_t)p.C, Q = (size_t)p.Cqkv, Cv = (size_t)p.Cv;
  const size_t nrel = (size_t)(2 * p.M - 1) * (2 * p.M - 1);
  const size_t act = align_up((size_t)p.T * C * es, 256);
  // arena layout
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
  const size_t o_x = take(act), o_dy = take(act), o_y = take(act), o_dx = take(act);
  const size_t o_wqkv = take(Q * C * es), o_bqkv = take(Q * es), o_wproj = take(C * Cv * es);
  const size_t o_bproj = take(C * es), o_tab = take(nrel * p.nh * es);
  const size_t o_dwqkv = take(Q * C * 4), o_dbqkv = take(Q * 4), o_dwproj = take(C * Cv * 4);
  const size_t o_dbproj = take(C * 4), o_dtab = take(nrel * p.nh * 4);
  const size_t o_saved = take(p.saved_bytes);
  const size_t scr = p.fwd_scratch > p.bwd_scratch ? p.fwd_scratch : p.bwd_scratch;
  const size_t o_scr = take(scr);
  if (arena_bytes_needed) *arena_bytes_needed = off;
  if (arena == nullptr || arena_bytes < off) return GSWA_ERR_WORKSPACE;
  if (!x || !w_qkv || !w_proj || !bias_table || !dy || !y || !dx || !dw_qkv || !db_qkv || !dw_proj || !db_proj ||
      !dbias_table)
    return GSWA_ERR_NULL;
  if (misaligned(arena)) return GSWA_ERR_ALIGN;
  char* a = static_cast<char*>(arena);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const size_t act_b = (size_t)p.T * C * es;
  auto h2d = [&](size_t o, const void* src, size_t bytes) {
    return cuda_rc(cudaMemcpyAsync(a + o, src, bytes, cudaMemcpyHostToDevice, st));
  };
  auto d2h = [&](void* dst, size_t o, size_t bytes) {
    return cuda_rc(cudaMemcpyAsync(dst, a + o, bytes, cudaMemcpyDeviceToHost, st));
  };
  if ((rc = h2d(o_x, x, act_b)) || (rc = h2d(o_dy, dy, act_b)) || (rc = h2d(o_wqkv, w_qkv, Q * C * es)) ||
      (rc = h2d(o_wproj, w_proj, C * Cv * es)) || (rc = h2d(o_tab, bias_table, nrel * p.nh * es)))
    return rc;
  if (b_qkv && (rc = h2d(o_bqkv, b_qkv, Q * es))) return rc;
  if (b_proj && (rc = h2d(o_bproj, b_proj, C * es))) return rc;
  rc = gswa_forward(desc, a + o_x, a + o_wqkv, b_qkv ? a + o_bqkv : nullptr, a + o_wproj, b_proj ? a + o_bproj : nullptr,
                    a + o_tab, a + o_y, a + o_saved, a + o_scr, scr, cuda_stream);
  if (rc) return rc;
  gswa_desc d2 = *desc;
  d2.flags &= ~GSWA_FLAG_ACCUMULATE;
  rc = gswa_backward(&d2, a + o_x, a + o_wqkv, b_qkv ? a + o_bqkv : nullptr, a + o_wproj, a + o_tab, a + o_saved,
                     a + o_dy, a + o_dx, (float*)(a + o_dwqkv), (float*)(a + o_dbqkv), (float*)(a + o_dwproj),
                     (float*)(a + o_dbproj), (float*)(a + o_dtab), a + o_scr, scr, cuda_stream);
  if (rc) return rc;
  if ((rc = d2h(y, o_y, act_b)) || (rc = d2h(dx, o_dx, act_b)) || (rc = d2h(dw_qkv, o_dwqkv, Q * C * 4)) ||
      (rc = d2h(db_qkv, o_dbqkv, Q * 4)) || (rc = d2h(dw_proj, o_dwproj, C * Cv * 4)) ||
      (rc = d2h(db_proj, o_dbproj, C * 4)) || (rc = d2h(dbias_table, o_dtab, nrel * p.nh * 4)))
    return rc;
  return cuda_rc(cudaStreamSynchronize(st));
}

int gswa_scratch_status(const gswa_desc* desc, const void* scratch, void* cuda_stream) {
  Plan p;
  const int rc = make_plan(desc, &p);
  if (rc) return rc;
  if (!p.fast || p.T == 0) return GSWA_OK;
  if (scratch == nullptr) return GSWA_ERR_NULL;
  int word = 0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int rc2 = cuda_rc(cudaMemcpyAsync(&word, scratch, sizeof(int), cudaMemcpyDeviceToHost, st));
  if (rc2 == GSWA_OK) rc2 = cuda_rc(cudaStreamSynchronize(st));
  if (rc2) return rc2;
  return word == 0 ? GSWA_OK : GSWA_ERR_DEVICE;
}

int gswa_profile_enable(int on) {
  std::lock_guard<std::mutex> lk(g_prof_mu);
  g_prof_on = on != 0;
  return GSWA_OK;
}

int gswa_profile_read(int32_t max_records, char* names, float* ms, int32_t* count) {
  std::lock_guard<std::mutex> lk(g_prof_mu);
  int n = 0, rc = GSWA_OK;
  for (auto& r : g_prof) {
    float t = 0.f;
    if (cudaEventSynchronize(r.e1) != cudaSuccess || cudaEventElapsedTime(&t, r.e0, r.e1) != cudaSuccess) {
      rc = cuda_rc(cudaGetLastError());
      if (rc == GSWA_OK) rc = GSWA_ERR_CUDA;
    }
    if (n < max_records && names && ms) {
      snprintf(names + (size_t)n * 32, 32, "%s", r.name);
      ms[n] = t;
      ++n;
    }
    cudaEventDestroy(r.e0);
    cudaEventDestroy(r.e1);
  }
  g_prof.clear();
  if (count) *count = n;
  return rc;
}

uint64_t gswa_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* gswa_status_string(int status) {
  switch (status) {
    case GSWA_OK: return "ok";
    case GSWA_ERR_NULL: return "a required pointer is NULL";
    case GSWA_ERR_SHAPE: return "inconsistent layer description";
    case GSWA_ERR_ALIGN: return "device pointer not 16-byte aligned";
    case GSWA_ERR_UNSUPPORTED: return "layer description not supported";
    case GSWA_ERR_WORKSPACE: return "scratch, arena or built-in scratch array too small for this layer";
    case GSWA_ERR_CUDA: return g_cuda_msg;
    case GSWA_ERR_DEVICE: return "a kernel gave up waiting on an internal barrier; results are invalid";
    default: return "unknown status";
  }
}

}  // extern "C"
