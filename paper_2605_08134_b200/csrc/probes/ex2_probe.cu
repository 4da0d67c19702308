// Stand-alone probe (not part of libdare): issue rate of ex2.approx on the special-function unit, f32 against the
// packed bf16x2 / f16x2 forms; one CTA of 8 warps per SM, eight independent chains per thread.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o ex2_probe ex2_probe.cu && ./ex2_probe
#include <cstdio>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
template <int MODE>
__global__ void k(float* out, int iters) {
  float a[8];
  unsigned u[8];
  for (int i = 0; i < 8; ++i) { a[i] = -0.001f * (threadIdx.x + i); u[i] = 0xbc00bc00u + threadIdx.x + i; }
  long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (MODE == 0) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(a[i]));
      if (MODE == 1) asm volatile("ex2.approx.ftz.bf16x2 %0, %0;" : "+r"(u[i]));
      if (MODE == 2) asm volatile("ex2.approx.f16x2 %0, %0;" : "+r"(u[i]));
    }
  }
  long long t1 = clock64();
  float s = 0; for (int i = 0; i < 8; ++i) s += a[i] + __uint_as_float(u[i]);
  if (threadIdx.x == 0 && blockIdx.x == 0) { out[0] = (float)(t1 - t0); }
  if (s == 12345.f) out[1] = s;
}
int main() {
  float* d; cudaMalloc(&d, 16);
  const int iters = 4096;
  for (int mode = 0; mode < 3; ++mode) {
    for (int rep = 0; rep < 2; ++rep) {
      if (mode == 0) k<0><<<148, 256>>>(d, iters);
      if (mode == 1) k<1><<<148, 256>>>(d, iters);
      if (mode == 2) k<2><<<148, 256>>>(d, iters);
      cudaDeviceSynchronize();
    }
    float h[2]; cudaMemcpy(h, d, 8, cudaMemcpyDeviceToHost);
    // 8 warps per SM = 2 per SMSP; warp-instructions per SMSP = 2 * 8 * iters
    printf("mode %d: %.0f cycles, %.2f cycles per warp-instruction per SMSP (%d elements per lane-op)\n", mode, h[0],
           h[0] / (2.0 * 8 * iters), mode == 0 ? 1 : 2);
  }
  printf("%s\n", cudaGetErrorString(cudaGetLastError()));
  return 0;
}
