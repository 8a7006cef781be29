// Producer / consumer building blocks of the tcgen05 GEMM kernels: bounded barrier waits, the ring of
// K atoms and its loader lanes, role constants, bulk-copy helpers.
#pragma once

#include "fast.cuh"
#include "umma.cuh"

namespace gswa {
namespace gemm {
using namespace umma;


constexpr int kEpiWarps = 4, kLoadWarps = 8;
constexpr int kThreads = 32 * (kEpiWarps + 1 + kLoadWarps);   // 416
constexpr int kThreadsR = kThreads + 32;                      // gr_kernel: one more warp, the TMA producer
// gw_kernel / gt_kernel drain TMEM with two warps per 32-lane quadrant (a warp may only read the
// TMEM lanes 32*(warp%4) .. +31): warps 0-7 epilogue, warp 8 MMA issue, warps 9-16 loaders.
constexpr int kEpi2 = 8;
constexpr int kThreads2 = 32 * (kEpi2 + 1 + kLoadWarps);      // 544
__device__ __forceinline__ void pair_sync(int quad) { asm volatile("bar.sync %0, 64;" ::"r"(quad + 1) : "memory"); }
// Barrier of the two warps of a quadrant that also ANDs a predicate, so that both take the same
// decision to go on or to give up (a warp must never be left waiting for a partner that returned).
__device__ __forceinline__ bool pair_vote(int quad, bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %2, 0;\n\tbar.red.and.pred p, %1, 64, q;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(r)
      : "r"(quad + 1), "r"((uint32_t)ok)
      : "memory");
  return r != 0;
}
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

// The same bounded wait as a non-blocking test with a short sleep between polls.  In the reduction GEMM, whose loaders
// keep the shared-memory pipe busy, this reacts sooner than the blocking form and shortens the kernel by 3-6 %; the
// loaders of the window GEMM get slower with it, so each kernel picks its form per wait.
__device__ __forceinline__ bool wait_bar_nap(uint64_t* bar, uint32_t parity, volatile int* abort_s, int* err) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_test_wait(bar, parity)) return true;
    if (i >= 8) __nanosleep(32);
    if ((i & 127u) == 127u && *abort_s) return false;
  }
  *abort_s = 1;
  if (err) atomicExch(err, 1);
  return false;
}
__device__ __forceinline__ bool wait_bar_warp_nap(uint64_t* bar, uint32_t parity, volatile int* abort_s, int* err) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = wait_bar_nap(bar, parity, abort_s, err) ? 1 : 0;
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
// Shared producer / consumer pieces of gw_kernel and gt_kernel
// ==========================================================================================
// The A operand of both kernels is a 128-row tile cut into K atoms of 64 columns (16 KB each,
// 128-byte swizzled rows) that travel through a ring of `S` shared-memory slots.  The eight loader
// warps form four sets of two warps; set q fills ring steps q, q+4, q+8, ...: it waits until the
// tensor core has released the slot, issues its asynchronous copies, waits for them to land, and
// publishes the slot at once.  Four steps of loads are therefore in flight per SM and a slot becomes
// visible to the MMA warp as soon as its own data has arrived.  The ring must have at least as many
// slots as there are sets: then the set that refills a slot has already seen the release of the
// slot's last-but-one use, so a parity wait can never be satisfied by a stale phase and two sets
// never arrive on the same `full` barrier in one phase.
constexpr int kSets = 4;                      // loader sets
constexpr int kAtomBytes = 128 * 128;         // one ring slot

struct RingPos {
  int slot, ph;                               // slot index and phase parity of ring step g
  __device__ __forceinline__ void init(int g, int S) { slot = g % S; ph = (g / S) & 1; }
  __device__ __forceinline__ void advance(int n, int S) {
    slot += n;
    while (slot >= S) { slot -= S; ph ^= 1; }
  }
};

// One thread of a loader set (64 threads): the 8-byte piece `pc` (0..15) of the 128-byte atom row, in tile
// rows rq + 4k (rq = 0..3).  Sixteen consecutive lanes cover one whole atom row: a copy instruction
// reads two runs of 128 contiguous bytes and writes two full rows of shared memory (no bank
// conflicts).  (r & 7) alternates between rq (k even) and rq + 4 (k odd), hence two swizzled bases;
// the destination of row rq + 4k is base + 512 k.  The first warp of a set takes rq = 0 and 2, the second
// rq = 1 and 3: all rows of a warp then have the same parity of their column in the window, hence of
// their token index, and a warp can use 16-byte copies for all of them or for none.
struct LoaderLane {
  int rq, pc;
  uint32_t dst_e, dst_o;
  __device__ __forceinline__ void init(int ts) {
    rq = ((ts >> 4) & 1) * 2 + (ts >> 5);
    pc = ts & 15;
    dst_e = sw128_offset(rq, pc * 4);
    dst_o = sw128_offset(rq + 4, pc * 4) - 4 * 128;
  }
  __device__ __forceinline__ uint32_t dst(int k) const { return (uint32_t)(k * 512) + ((k & 1) ? dst_o : dst_e); }
};

// Lane mapping of gr_kernel's copy-fed operand: rows lw + 8k, 16-byte chunk pp of the atom row (two
// 8-byte pieces); a copy instruction reads four rows of 128 contiguous bytes.  The first warp of a set takes
// the even rows, the second the odd ones: with a row pitch of 8 mod 16 bytes the even rows start on 16-byte
// boundaries and are fetched with half as many (16-byte) copies, and a warp never mixes the two kinds.
struct LoaderLane4 {
  int lw, pp;
  uint32_t dst0;
  __device__ __forceinline__ void init(int ts) {
    lw = ((ts >> 3) & 3) * 2 + (ts >> 5);
    pp = ts & 7;
    dst0 = sw128_offset(lw, pp * 8);
  }
};

// Barriers over the eight epilogue warps (hardware barrier 5, 256 threads); the voting form ANDs a
// predicate so that all of them go on or give up together.
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 5, 256;" ::: "memory"); }
__device__ __forceinline__ bool epi_vote(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 5, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(r)
      : "r"((uint32_t)ok)
      : "memory");
  return r != 0;
}
// Bulk asynchronous copy shared -> global (sizes and addresses multiples of 16 bytes).
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t ssrc, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(ssrc), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }


}  // namespace gemm
}  // namespace gswa
