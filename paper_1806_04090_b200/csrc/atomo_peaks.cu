// Measured arithmetic peaks of the GPU the library runs on: a register-only chain of fused multiply-adds, fp32 or
// fp64, on every SM.  The benchmark reports kernels that are bound by plain ALU arithmetic (the register-resident
// Householder reduction, the Jacobi eigen-solver) against these figures instead of a number derived from lane counts.
#include <cstdio>

#include "atomo_kernels.cuh"

namespace atomo {

template <typename T>
__global__ void __launch_bounds__(512) fma_peak_kernel(T* __restrict__ out, int iters, T b, T c) {
  T a[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) a[j] = (T)(threadIdx.x + j) * (T)1e-3;
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int j = 0; j < 8; ++j) a[j] = fma(a[j], b, c);      // eight independent chains per thread
  }
  T s = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) s += a[j];
  out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace atomo

extern "C" int atomo_measure_fma_peak(int device, int fp64, double* tflops) {
  using namespace atomo;
  if (device < 0 || !tflops) return ATOMO_ERR_INVALID_ARG;
  if (cudaSetDevice(device) != cudaSuccess) return ATOMO_ERR_CUDA;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return ATOMO_ERR_CUDA;
  const int threads = 512, ctas = sms * 4, iters = fp64 ? 2048 : 4096;
  void* buf = nullptr;
  if (cudaMalloc(&buf, (size_t)ctas * threads * 8) != cudaSuccess) return ATOMO_ERR_CUDA;
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0); cudaEventCreate(&e1);
  float best = 1e30f;
  for (int rep = 0; rep < 4; ++rep) {                          // the first run warms up
    cudaEventRecord(e0);
    if (fp64) fma_peak_kernel<double><<<ctas, threads>>>(static_cast<double*>(buf), iters, 0.999999, 1e-6);
    else fma_peak_kernel<float><<<ctas, threads>>>(static_cast<float*>(buf), iters, 0.999999f, 1e-6f);
    cudaEventRecord(e1);
    if (cudaEventSynchronize(e1) != cudaSuccess) { cudaFree(buf); return ATOMO_ERR_CUDA; }
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && ms < best) best = ms;
  }
  cudaEventDestroy(e0); cudaEventDestroy(e1);
  cudaFree(buf);
  *tflops = 2.0 * 8.0 * (double)iters * (double)ctas * threads / (best * 1e-3) / 1e12;
  return ATOMO_OK;
}
