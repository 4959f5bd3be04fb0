// Shared host/device helpers of the DGQ library: status word, checked CUDA calls,
// mbarrier / TMA / tcgen05 PTX wrappers with bounded waits.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda.h>

#include <atomic>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <utility>
#include <vector>

#include "../../include/dgq.h"

namespace dgq {

// First error recorded by any kernel on this device since the last dgq_device_status().
__device__ int g_status_word = 0;

static std::atomic<uint64_t> g_launches{0};

__device__ __forceinline__ void record_error(int code) { atomicCAS(&g_status_word, 0, code); }

#define DGQ_CUDA_OK(expr)                        \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) return DGQ_ERR_CUDA; \
  } while (0)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ------------------------------------------------------------------ ordered-int encoding of floats
// Monotone map float -> int so that integer atomicMin / atomicMax order like the floats.
__host__ __device__ __forceinline__ int float_to_ordered(float f) {
#ifdef __CUDA_ARCH__
  int b = __float_as_int(f);
#else
  int b;
  std::memcpy(&b, &f, 4);
#endif
  return b >= 0 ? b : (b ^ 0x7FFFFFFF);
}
__host__ __device__ __forceinline__ float ordered_to_float(int k) {
  int b = k >= 0 ? k : (k ^ 0x7FFFFFFF);
#ifdef __CUDA_ARCH__
  return __int_as_float(b);
#else
  float f;
  std::memcpy(&f, &b, 4);
  return f;
#endif
}

// ------------------------------------------------------------------ Eq. 6 in the fixed fp32 order
// s = (hi - lo) * 2^-b floored at 1e-8, inv_s = 1 / s (IEEE division),
// Z = rint(clamp(-lo * inv_s, -2^30, 2^30)).
__host__ __device__ __forceinline__ void group_params(float lo, float hi, int bits, float& s, float& inv_s,
                                                       int& Z) {
#ifdef __CUDA_ARCH__
  float w = __fmul_rn(__fsub_rn(hi, lo), __int_as_float((127 - bits) << 23));
  s = w > 1e-8f ? w : 1e-8f;
  inv_s = __fdiv_rn(1.0f, s);
  Z = __float2int_rn(fminf(fmaxf(__fmul_rn(-lo, inv_s), -1073741824.0f), 1073741824.0f));
#else
  volatile float d = hi - lo;
  volatile float w = d * (1.0f / (float)(1u << bits));
  s = w > 1e-8f ? (float)w : 1e-8f;
  volatile float inv = 1.0f / s;
  inv_s = inv;
  volatile float t = -lo * inv_s;
  float tc = t < -1073741824.0f ? -1073741824.0f : (t > 1073741824.0f ? 1073741824.0f : (float)t);
  Z = (int)__builtin_rintf(tc);
#endif
}

// Launch with the programmatic-serialization attribute (see pdl_wait); DGQ_PDL=0 in the environment
// turns the attribute off.
inline bool pdl_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = std::getenv("DGQ_PDL");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v != 0;
}
#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif
#ifdef __CUDACC__
// Eq. 1: q = min(max(rint(x * inv_s) + Z, 0), L); NaN -> 0 (fmaxf returns the non-NaN operand).
__device__ __forceinline__ int quantize_code(float x, float inv_s, float Zf, float Lf) {
  float u = __fadd_rn(rintf(__fmul_rn(x, inv_s)), Zf);
  return __float2int_rn(fminf(fmaxf(u, 0.0f), Lf));
}

// ------------------------------------------------------------------ programmatic dependent launch
// Kernels of the hot path are launched so that the next kernel in the stream may be scheduled while
// the current one drains (its blocks become resident as this one's exit, without the launch gap):
// every such kernel calls pdl_launch_dependents() at its top and pdl_wait() before its first access
// to global memory that an earlier kernel may have written.  pdl_wait() returns once every
// preceding kernel has completed and its writes are visible; without the launch attribute both
// are no-ops.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------ shared-memory addresses
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Same test, but the hardware may park the thread for up to `ns` nanoseconds while the phase is
// still pending, so a waiting warp does not compete for issue slots with the working ones.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}

// Bounded wait: gives up after about a second (2^31 SM clocks) or as soon as another
// thread of the CTA has raised `*abort_flag`.  Returns false when it gave up; the caller
// must then leave through the kernel's common exit path.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait_parked(bar, parity, 4000u)) return true;
    if ((++spins & 63u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > (1ll << 31)) {
        *abort_flag = 1;
        record_error(DGQ_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

// Bounded wait without a return value, for hot loops: after `max_polls` (2^21) parked polls (of at most a
// microsecond each) it records a time-out and raises `*abort_flag`; once the flag is up every wait
// returns at its first failed poll.  The caller tests the flag at a coarser grain (once per tile)
// and leaves through the kernel's common exit path; what it does in between only touches memory
// the CTA owns.
__device__ __forceinline__ void mbar_wait_lean(uint32_t bar_addr, uint32_t parity, volatile int* abort_flag,
                                               uint32_t max_polls = 1u << 21) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity)
      : "memory");
  if (ok) return;
  if (*abort_flag) return;
  for (uint32_t spins = 0; spins < max_polls; ++spins) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar_addr), "r"(parity), "r"(1000u)
        : "memory");
    if (ok) return;
    if ((spins & 31u) == 31u && *abort_flag) return;
  }
  *abort_flag = 1;
  record_error(DGQ_ERR_TIMEOUT);
}
// Bounded wait for roles that may wait long while other warps of the CTA work: polls that answer at
// once (test_wait) with a growing sleep in between (32 ns doubling to 256 ns), so that the waiting
// warp takes almost no issue slots or shared-memory bandwidth from the working ones.  After 2^22
// polls (about a second) it records a time-out and raises `*abort_flag`; once the flag is up every
// wait returns at its first failed poll.
__device__ __forceinline__ void mbar_wait_backoff(uint32_t bar_addr, uint32_t parity, volatile int* abort_flag,
                                                  uint32_t max_polls = 1u << 22) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity)
      : "memory");
  if (ok) return;
  if (*abort_flag) return;
  uint32_t ns = 32;
  for (uint32_t spins = 0; spins < max_polls; ++spins) {
    asm volatile("nanosleep.u32 %0;" ::"r"(ns));
    if (ns < 256) ns <<= 1;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar_addr), "r"(parity)
        : "memory");
    if (ok) return;
    if ((spins & 63u) == 63u && *abort_flag) return;
  }
  *abort_flag = 1;
  record_error(DGQ_ERR_TIMEOUT);
}
// One non-blocking poll; the result can be consumed many instructions later.
__device__ __forceinline__ uint32_t mbar_try_addr(uint32_t bar_addr, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity)
      : "memory");
  return ok;
}
// The same without any waiting: try_wait may park the thread for a while when the phase is still
// pending, test_wait answers at once.
__device__ __forceinline__ uint32_t mbar_test_addr(uint32_t bar_addr, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity)
      : "memory");
  return ok;
}
// Read-only global loads that stay where they are written (a plain load may be moved next to its
// first use, which would expose its latency there).
__device__ __forceinline__ float ldg_f32_here(const float* p) {
  float v;
  asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ int ldg_s32_here(const int32_t* p) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
// Register re-balancing between the warpgroups of a CTA (every warp of an aligned group of four
// executes the same instruction).
template <int REGS>
__device__ __forceinline__ void reg_alloc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS));
}
template <int REGS>
__device__ __forceinline__ void reg_dealloc() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS));
}
// True in exactly one lane of a converged warp.  A loop that the whole warp runs with uniform control
// flow and whose tcgen05 instructions sit behind this test keeps its addresses and counters in the
// uniform datapath, which makes the issuing path markedly shorter than a loop run by one lane of a
// diverged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void mbar_arrive_addr(uint32_t bar_addr) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_addr) : "memory");
}

// Two fp32 lanes in one 64-bit register (the operand form of the packed fp32 instructions).
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// y += s * float(i) on two lanes: two conversions and one packed fused multiply-add.
__device__ __forceinline__ void cvt_fma_f32x2(unsigned long long& y, unsigned long long s2, uint32_t i0, uint32_t i1) {
  asm volatile("{\n\t.reg .f32 f0, f1;\n\t.reg .b64 t;\n\t"
      "cvt.rn.f32.s32 f0, %1;\n\t"
      "cvt.rn.f32.s32 f1, %2;\n\t"
      "mov.b64 t, {f0, f1};\n\t"
      "fma.rn.f32x2 %0, %3, t, %0;\n\t}"
      : "+l"(y)
      : "r"(i0), "r"(i1), "l"(s2));
}

// Two int32 -> fp32 conversions straight into one 64-bit register pair (the operand form of the packed
// fp32 instructions), so that no moves are needed to pair the results up.
__device__ __forceinline__ unsigned long long cvt_s32x2_f32x2(uint32_t i0, uint32_t i1) {
  unsigned long long r;
  asm("{\n\t.reg .f32 f0, f1;\n\t"
      "cvt.rn.f32.s32 f0, %1;\n\t"
      "cvt.rn.f32.s32 f1, %2;\n\t"
      "mov.b64 %0, {f0, f1};\n\t}"
      : "=l"(r)
      : "r"(i0), "r"(i1));
  return r;
}
// d = a * b + c on two lanes
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b,
                                                        unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}

__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ------------------------------------------------------------------ TMA tile loads (each CTA fetches its own tiles)
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], "
      "[%2];" ::"r"(smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

// TMA tile store shared -> global (bulk async-group completion).  Rows and columns outside the
// tensor are clipped by the hardware.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, const void* src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(smem_u32(src)), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all committed bulk stores of this thread have finished reading shared memory
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... and have completed
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ------------------------------------------------------------------ tcgen05 / tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// One 128 x N x 32 int8 MMA: D[tmem] (+)= A[smem] * B[smem]^T, issued by a single thread.
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with the two 64-bit shared-memory descriptors given as (low, high) words: the high words
// are constants of the layout and only the low word (the address field) changes from atom to atom,
// which keeps the single issuing thread's dependent instruction chain short.
__device__ __forceinline__ void mma_i8_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                            uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Low / high words of a K-major shared-memory descriptor (see smem_desc).
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ constexpr uint32_t smem_desc_hi(uint32_t sbo_bytes, uint32_t layout) {
  return (sbo_bytes >> 4) | (1u << 14) | (layout << 29);
}
// Arrives on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void mma_commit_addr(uint32_t bar_addr) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_addr)
               : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp receives row (lane base + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// 32 lanes x 8 consecutive 32-bit columns.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, K-major operand, rows of 128 B (SWIZZLE_128B) or 32 B (SWIZZLE_32B):
// start address >> 4 in bits [0,14), stride between 8-row groups >> 4 in bits [32,46), descriptor
// version 1 in bits [46,48), swizzle mode in bits [61,64) (2 = 128 B, 6 = 32 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t sbo_bytes, uint32_t layout) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)layout << 61);
}
#endif  // __CUDACC__

}  // namespace dgq
