// Single translation unit of the DGQ library (one device status word, no relocatable device code).
#include <climits>
#include <cmath>

#include "common.cuh"
#include "groups.cuh"
#include "quantize.cuh"
#include "weights.cuh"
#include "linear.cuh"
#include "attention.cuh"

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
