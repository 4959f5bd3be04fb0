// Single translation unit of the DGQ library (one device status word, no relocatable device code).
#include <climits>
#include <cmath>
#include <mutex>

#include "common.cuh"
#include "groups.cuh"
#include "quantize.cuh"
#include "weights.cuh"
#include "linear.cuh"
#include "attention.cuh"
#include "self_attention.cuh"

// ---------------------------------------------------------------------------------------------
// Cross-attention for callers that cannot allocate a workspace: the scratch is this fixed array
// in the library image (one copy per GPU that loads the library).  In host code the name
// `g_noalloc_scratch` is only a handle for the runtime, never a device address; the address that
// kernels may use comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[DGQ_NOALLOC_SCRATCH_BYTES];

namespace {
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[64] = {nullptr};  // device address of the scratch array, per device ordinal
}  // namespace

extern "C" dgq_status dgq_cross_attn_logq_noalloc(const void* Q, const void* K, const void* V, int B, int H, int nq,
                                                  int nk, int d, int score_bits, int scale_gran,
                                                  const float* fixed_scale, void* O, float* scale_out,
                                                  uint8_t* codes_out, void* stream) {
  // the ordinary argument errors come first, then the limits of the built-in scratch
  dgq_status chk = dgq::attn_check_args(Q, K, V, B, H, nq, nk, d, score_bits, scale_gran, 0, O);
  if (chk != DGQ_OK) return chk;
  if ((int64_t)B * H > DGQ_NOALLOC_MAX_HEADS || (int64_t)B * H * nq > DGQ_NOALLOC_MAX_ROWS)
    return DGQ_ERR_WORKSPACE;  // larger than the built-in scratch: use dgq_cross_attn_logq
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return DGQ_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {  // first call on this device, which is the current one
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return DGQ_ERR_CUDA;
      g_noalloc_ptr[dev] = p;
    }
    scratch = g_noalloc_ptr[dev];
  }
  // The first kernel of the workspace path writes every partial maximum and every row statistic
  // that the second one reads, so stale contents from an earlier call are harmless.
  // (always the two-kernel form, which has no launch requirement beyond an ordinary kernel's)
  return dgq::attn_run(Q, K, V, B, H, nq, nk, d, score_bits, scale_gran, fixed_scale, 0, O, scale_out, codes_out,
                       scratch, (size_t)DGQ_NOALLOC_SCRATCH_BYTES, false, stream);
}

namespace dgq {
// One warp waits, with the caller's poll limit, on a barrier that nobody arrives at: the bounded wait
// gives up, records DGQ_ERR_TIMEOUT and the kernel ends normally.
__global__ void selftest_wait_kernel(uint32_t max_polls) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  mbar_wait_lean(smem_u32(&bar), 0u, &abort_flag, max_polls);
}
}  // namespace dgq

extern "C" dgq_status dgq_selftest_wait_timeout(uint32_t max_polls, void* stream) {
  if (max_polls == 0 || max_polls > (1u << 16)) return DGQ_ERR_INVALID_ARG;
  dgq::selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(max_polls);
  dgq::g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

extern "C" dgq_status dgq_device_status(int* status) {
  if (!status) return DGQ_ERR_INVALID_ARG;
  DGQ_CUDA_OK(cudaDeviceSynchronize());
  int v = 0;
  DGQ_CUDA_OK(cudaMemcpyFromSymbol(&v, dgq::g_status_word, sizeof(int)));
  *status = v;
  if (v != 0) {
    const int zero = 0;
    DGQ_CUDA_OK(cudaMemcpyToSymbol(dgq::g_status_word, &zero, sizeof(int)));
  }
  return DGQ_OK;
}

extern "C" const char* dgq_status_string(dgq_status s) {
  switch (s) {
    case DGQ_OK: return "ok";
    case DGQ_ERR_INVALID_ARG: return "invalid argument";
    case DGQ_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case DGQ_ERR_UNSUPPORTED: return "unsupported shape or mode";
    case DGQ_ERR_WORKSPACE: return "workspace missing or too small";
    case DGQ_ERR_CUDA: return "CUDA call failed";
    case DGQ_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case DGQ_ERR_NOT_CALIBRATED: return "table row of this timestep not calibrated";
    default: return "unknown status";
  }
}

extern "C" uint64_t dgq_launch_count(void) { return dgq::g_launches.load(); }
