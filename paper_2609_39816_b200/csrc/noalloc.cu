// error_frobenius_noalloc: the Frobenius-error reduction for callers that cannot allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits — inside a CUDA-graph capture or another
// region where allocation would synchronise or fail, under a memory pool that is already fully committed, or
// in a host application whose policy forbids a library from growing its device footprint after start-up.
// The ordinary entry point asks such a caller for a workspace; this one brings its own, a fixed array that
// is part of the library image and therefore exists on every GPU that loads the library, from load to exit.
#include <cuda_runtime.h>

#include "kernels_stream.cuh"

namespace {

// One partial sum per block and per quantity.  The block count grows with the problem (one block per
// kElemsPerBlock elements), so the array bounds the problem size: kMaxBlocks * kElemsPerBlock elements.
constexpr int kElemsPerBlock = 32768;
constexpr int kMaxBlocks = 2048;
static __device__ __align__(256) double g_noalloc_partials[2 * kMaxBlocks];   // 32 KiB per GPU

constexpr int kMaxDevices = 64;
// Device address of the array, per device ordinal, kept for the life of the process: it does not survive a
// cudaDeviceReset of that device by the host application (the library must not be used across one).
double* g_scratch_ptr[kMaxDevices] = {};

// In host code the array's name is only a handle for the runtime, not an address the GPU understands:
// the device address has to be asked for, once per device, while that device is current.
fmm_status scratch_for_current_device(double** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FMM_ERR_CUDA;
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_partials) != cudaSuccess || p == nullptr) return FMM_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<double*>(p);
  }
  *out = g_scratch_ptr[dev];
  return FMM_OK;
}

}  // namespace

extern "C" {

int64_t error_frobenius_noalloc_max_elements(void) { return (int64_t)kMaxBlocks * kElemsPerBlock; }

fmm_status error_frobenius_noalloc(const fmm_gemm_desc* d, const void* dC, const double* dCstar, double* d_out,
                                   void* cuda_stream) {
  if (!d || !dC || !dCstar || !d_out) return FMM_ERR_ARG;
  if (d->M <= 0 || d->N <= 0 || d->ldc < d->N) return FMM_ERR_SHAPE;
  if (d->output != FMM_F32 && d->output != FMM_BF16) return FMM_ERR_DTYPE;
  // would not fit the fixed array (tested by division: M * N itself may not fit 64 bits)
  if (d->M > error_frobenius_noalloc_max_elements() / d->N) return FMM_ERR_LIMIT;
  const int64_t count = d->M * d->N;
  double* scratch = nullptr;
  fmm_status s = scratch_for_current_device(&scratch);
  if (s != FMM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int blocks = (int)((count + kElemsPerBlock - 1) / kElemsPerBlock);
  double* part_err = scratch;
  double* part_ref = scratch + kMaxBlocks;
  // every block overwrites its own slot of both arrays, so nothing left by an earlier call is read
  if (launch_frob_err_fixed_grid(d->output, dC, d->ldc, dCstar, d->M, d->N, part_err, part_ref, blocks, st) != cudaSuccess)
    return FMM_ERR_CUDA;
  if (launch_sum_partials(part_err, blocks, d_out, st) != cudaSuccess) return FMM_ERR_CUDA;
  if (launch_sum_partials(part_ref, blocks, d_out + 1, st) != cudaSuccess) return FMM_ERR_CUDA;
  return FMM_OK;
}

}  // extern "C"
