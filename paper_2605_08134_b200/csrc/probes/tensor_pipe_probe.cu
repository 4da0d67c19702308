// Stand-alone probe of the tensor pipe (not part of libdare): build and run with
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o tensor_pipe_probe tensor_pipe_probe.cu -lcuda
//   ./tensor_pipe_probe
// (1) cycles per tcgen05.mma (cta_group::1, M = 128, K = 16, bf16) for N = 256 / 128 / 64, with the A operand in
//     shared memory or in tensor memory and the B operand K-major or MN-major, issued back to back by one thread
//     with the operands resident in shared memory (no loads in flight): the rate of the pipe itself;
// (2) the layout of a tensor-memory A operand: lane = row, one 32-bit column = two consecutive k (low half first),
//     eight columns per K = 16 step; the product is compared with a CPU product.
// Every wait is bounded (the library's mbar_wait).
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../tc_ptx.cuh"

using namespace dare::ptx;

// mode 0: SS K-major B; 1: SS MN-major B (N=128 only layout as in PV); 2: TS K-major B; 3: TS MN-major B
template <int N, int MODE>
__global__ void __launch_bounds__(128, 1) probe(long long* out, int rounds) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t bar;
  __shared__ uint32_t slot;
  __shared__ int status;
  for (int i = threadIdx.x; i < (32 + 64) * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); fence_mbar_init(); status = 0; }
  if (threadIdx.x < 32) { tmem_alloc(&slot, 512); tmem_relinquish(); }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = slot;
  if (threadIdx.x == 0) {
    constexpr uint32_t idesc = idesc_bf16(128, N, (MODE & 1) != 0);
    const uint32_t a_addr = smem_u32(smem), b_addr = smem_u32(smem + 32 * 1024);
    long long t0 = clock64();
    for (int r = 0; r < rounds; ++r) {
      const uint32_t d = tm + (r & 1) * 256 * 0;   // same accumulator
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        uint64_t bd;
        if (MODE & 1) bd = smem_desc_mn_sw128(b_addr + kk * (16 * 128), 128 * 128);
        else bd = smem_desc_k_sw128(b_addr + (kk >> 2) * (N * 128) + (kk & 3) * 32);
        if (MODE & 2) umma_ts(d, tm + 256 + kk * 8, bd, idesc, kk != 0);
        else umma_ss(d, smem_desc_k_sw128(a_addr + (kk >> 2) * (128 * 128) + (kk & 3) * 32), bd, idesc, kk != 0);
      }
    }
    long long t1 = clock64();
    umma_commit(&bar);
    mbar_wait(&bar, 0, &status);
    long long t2 = clock64();
    out[blockIdx.x * 2] = t1 - t0;
    out[blockIdx.x * 2 + 1] = t2 - t0;
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) tmem_dealloc(tm, 512);
}

template <int N, int MODE>
void run(const char* name, int grid) {
  long long* d;
  cudaMalloc(&d, 2 * 148 * sizeof(long long));
  const int smem = 97 * 1024 + 1024;
  cudaFuncSetAttribute(probe<N, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  const int rounds = 64;
  for (int rep = 0; rep < 2; ++rep) probe<N, MODE><<<grid, 128, smem>>>(d, rounds);
  cudaError_t e = cudaDeviceSynchronize();
  long long h[2 * 148];
  cudaMemcpy(h, d, sizeof(h), cudaMemcpyDeviceToHost);
  double iss = 0, tot = 0;
  for (int i = 0; i < grid; ++i) { iss += h[2 * i]; tot += h[2 * i + 1]; }
  printf("%-28s grid %3d: issue %.1f clk/mma, complete %.1f clk/mma (%s)\n", name, grid, iss / grid / (rounds * 8),
         tot / grid / (rounds * 8), cudaGetErrorString(e));
  cudaFree(d);
}

// K = 32 (two MMAs) to check the column advance of A too.  b_mn: B stored MN-major (like V), else K-major (like K).
__global__ void __launch_bounds__(128, 1) ts_numerics(float* out, int b_mn) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t bar;
  __shared__ uint32_t slot;
  __shared__ int status;
  const int KT = 32;
  for (int i = threadIdx.x; i < 32 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0;
  __syncthreads();
  // B[n][k] = ((n + 2k) % 5) - 2
  __nv_bfloat16* bs = reinterpret_cast<__nv_bfloat16*>(smem);
  for (int e = threadIdx.x; e < 128 * KT; e += blockDim.x) {
    const int n = e / KT, k = e % KT;
    const float v = (float)((n + 2 * k) % 5) - 2.f;
    size_t off;
    if (!b_mn) {   // K-major: row n (128 B), unit u = k/8 swizzled by n&7
      off = (size_t)n * 128 + (((k >> 3) ^ (n & 7)) << 4) + (k & 7) * 2;
    } else {       // MN-major: row k (128 B = 64 n), unit (n%64)/8 swizzled by k&7; second 64 n at +LBO (KT*128... use 128 rows*128)
      off = (size_t)(n >> 6) * (128 * 128) + (size_t)k * 128 + ((((n & 63) >> 3) ^ (k & 7)) << 4) + (n & 7) * 2;
    }
    bs[off / 2] = __float2bfloat16(v);
  }
  if (threadIdx.x == 0) { mbar_init(&bar, 1); fence_mbar_init(); status = 0; }
  if (threadIdx.x < 32) { tmem_alloc(&slot, 512); tmem_relinquish(); }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = slot;
  const int r = threadIdx.x;
  const int quarter = threadIdx.x >> 5;
  // A[r][k] = (r % 7) + 0.5 k  -> packed pairs, column j = (A[r][2j], A[r][2j+1])
  {
    float v[32];
    for (int j = 0; j < 32; ++j) {
      if (j < KT / 2) {
        __nv_bfloat162 h = __floats2bfloat162_rn((float)(r % 7) + 0.5f * (2 * j), (float)(r % 7) + 0.5f * (2 * j + 1));
        v[j] = __uint_as_float(*reinterpret_cast<uint32_t*>(&h));
      } else v[j] = 0.f;
    }
    tmem_st_32x32(tm + 256 + ((uint32_t)(quarter * 32) << 16), v);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) {
    const uint32_t idesc = idesc_bf16(128, 128, b_mn != 0);
    const uint32_t b_addr = smem_u32(smem);
    for (int kk = 0; kk < KT / 16; ++kk) {
      uint64_t bd = b_mn ? smem_desc_mn_sw128(b_addr + kk * (16 * 128), 128 * 128) : smem_desc_k_sw128(b_addr + kk * 32);
      umma_ts(tm, tm + 256 + kk * 8, bd, idesc, kk != 0);
    }
    umma_commit(&bar);
    mbar_wait(&bar, 0, &status);
  }
  __syncthreads();
  tc_fence_after();
  for (int ch = 0; ch < 4; ++ch) {
    float v[32];
    tmem_ld_32x32(tm + ((uint32_t)(quarter * 32) << 16) + ch * 32, v);
    for (int i = 0; i < 32; ++i) out[r * 128 + ch * 32 + i] = v[i];
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) tmem_dealloc(tm, 512);
}

int main() {
  for (int b_mn = 0; b_mn < 2; ++b_mn) {
    float* d;
    cudaMalloc(&d, 128 * 128 * 4);
    cudaFuncSetAttribute(ts_numerics, cudaFuncAttributeMaxDynamicSharedMemorySize, 40 * 1024);
    ts_numerics<<<1, 128, 40 * 1024>>>(d, b_mn);
    cudaError_t e = cudaDeviceSynchronize();
    static float h[128 * 128];
    cudaMemcpy(h, d, sizeof(h), cudaMemcpyDeviceToHost);
    double maxerr = 0;
    for (int r = 0; r < 128; ++r)
      for (int n = 0; n < 128; ++n) {
        double ref = 0;
        for (int k = 0; k < 32; ++k) ref += ((r % 7) + 0.5 * k) * (double)(((n + 2 * k) % 5) - 2);
        maxerr = fmax(maxerr, fabs(ref - h[r * 128 + n]));
      }
    printf("A operand in tensor memory (B %s): max abs error vs CPU product %.4f (%s)\n",
           b_mn ? "MN-major" : "K-major", maxerr, cudaGetErrorString(e));
    cudaFree(d);
  }
  for (int grid : {1, 148}) {
    run<256, 0>("SS N256 K-major", grid);
    run<128, 0>("SS N128 K-major", grid);
    run<64, 0>("SS N64 K-major", grid);
    run<128, 1>("SS N128 MN-major B", grid);
    run<256, 2>("TS N256 K-major", grid);
    run<128, 2>("TS N128 K-major", grid);
    run<128, 3>("TS N128 MN-major B", grid);
    run<64, 2>("TS N64 K-major", grid);
  }
  return 0;
}
