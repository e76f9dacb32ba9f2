// Measures the exp2 roof of the GPU: ex2.approx.ftz.f32 results per clock and SM from a kernel that does nothing else
// (16 independent chains per thread, each step one exponential and one fused multiply-add that keeps the value in
// range; registers only, no memory traffic). One block of 512 threads per SM. Prints one JSON line. The benchmark uses
// the figure as the denominator of the roofline of the wide-window scoring kernels, whose binding unit is the
// special-function pipe.
#include <algorithm>
#include <cstdio>
#include <vector>

#include <cuda_runtime.h>

__global__ void __launch_bounds__(512, 1) exp2_chain(float* out, long long* cycles, int iters, float a, float b) {
  float v[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = -0.01f * (threadIdx.x + i + 1);
  __syncthreads();
  const long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      float y;
      asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(v[i]));
      v[i] = fmaf(y, a, b);
    }
  }
  const long long t1 = clock64();
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) s += v[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

int main() {
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0) != cudaSuccess || sms <= 0) {
    printf("{\"error\": \"no CUDA device\"}\n");
    return 1;
  }
  const int threads = 512, iters = 20000;
  float* out = nullptr;
  long long* cyc = nullptr;
  cudaMalloc(&out, sizeof(float) * sms * threads);
  cudaMalloc(&cyc, sizeof(long long) * sms);
  exp2_chain<<<sms, threads>>>(out, cyc, 200, 0.25f, -0.3f);  // warm-up
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  cudaEventRecord(e0);
  exp2_chain<<<sms, threads>>>(out, cyc, iters, 0.25f, -0.3f);
  cudaEventRecord(e1);
  if (cudaEventSynchronize(e1) != cudaSuccess) {
    printf("{\"error\": \"%s\"}\n", cudaGetErrorString(cudaGetLastError()));
    return 1;
  }
  float ms = 0.f;
  cudaEventElapsedTime(&ms, e0, e1);
  std::vector<long long> h(sms);
  cudaMemcpy(h.data(), cyc, sizeof(long long) * sms, cudaMemcpyDeviceToHost);
  std::sort(h.begin(), h.end());
  const double c = (double)h[sms / 2];  // median over the SMs
  const double per_sm = 16.0 * iters * threads;
  printf("{\"exp2_per_clk_per_sm\": %.3f, \"sms\": %d, \"texp2_per_s\": %.3f, \"ms\": %.3f, \"implied_sm_mhz\": %.0f}\n",
         per_sm / c, sms, per_sm * sms / (ms * 1e-3) / 1e12, ms, c / (ms * 1e-3) / 1e6);
  cudaFree(out);
  cudaFree(cyc);
  return 0;
}
