// Stand-alone probe (not part of libdare): one tcgen05.mma.cta_group::2 tile over a cluster of two CTAs.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o pair_mma_probe pair_mma_probe.cu -lcuda && ./pair_mma_probe
// D[256 x 256] = A[256 x 64] * B[256 x 64]^T, bf16 in, fp32 out.  CTA r of the pair holds rows [128 r, 128 r + 128) of A
// and of B in its shared memory (K-major, 128-byte swizzle); the leader CTA (rank 0) issues four M256 N256 K16 MMAs;
// each CTA finds its 128 rows of D (all 256 columns) in its own tensor memory.  The result is compared with a CPU
// product, and the MMAs are timed.  Every wait is bounded; tensor memory is allocated and freed by both CTAs.
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../tc_ptx.cuh"

using namespace dare::ptx;

__device__ __forceinline__ void tmem_alloc2(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// arrive on the barrier at this offset in both CTAs of the pair once the MMAs issued so far have completed: one
// commit per CTA, each to that CTA's barrier by its cluster address
__device__ __forceinline__ void umma2_commit_both(uint64_t* bar) {
#pragma unroll
  for (uint32_t r = 0; r < 2; ++r)
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(map_to_cta(smem_u32(bar), r)) : "memory");
}
__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}

constexpr int KT = 64;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1)
pair_probe(float* out, long long* cycles, int* status_out, int rounds) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t bar;
  __shared__ uint32_t slot;
  __shared__ int status;
  const uint32_t rank = cluster_ctarank();
  for (int i = threadIdx.x; i < 32 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0;
  __syncthreads();
  // A rows and B rows of this CTA: global row = 128 rank + r;  A[m][k] = (m % 7) - 3 + 0.25 k,  B[n][k] = ((n + 3k) % 5) - 2
  __nv_bfloat16* as = reinterpret_cast<__nv_bfloat16*>(smem);
  __nv_bfloat16* bs = reinterpret_cast<__nv_bfloat16*>(smem + 16 * 1024);
  for (int e = threadIdx.x; e < 128 * KT; e += blockDim.x) {
    const int r = e / KT, k = e % KT, gr = 128 * (int)rank + r;
    const size_t off = (size_t)r * 128 + (((k >> 3) ^ (r & 7)) << 4) + (k & 7) * 2;
    as[off / 2] = __float2bfloat16((float)(gr % 7) - 3.f + 0.25f * (float)k);
    bs[off / 2] = __float2bfloat16((float)((gr + 3 * k) % 5) - 2.f);
  }
  if (threadIdx.x == 0) { mbar_init(&bar, 1); fence_mbar_init(); status = 0; }
  if (threadIdx.x < 32) { tmem_alloc2(&slot, 256); tmem_relinquish2(); }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                      // both CTAs: operands written, barriers initialised, tensor memory allocated
  tc_fence_after();
  // the accumulator address the leader's MMAs use: the leader's allocation (read from its shared memory)
  const uint32_t tm = ld_cluster_u32(map_to_cta(smem_u32(&slot), 0));
  long long t0 = 0, t1 = 0;
  if (rank == 0 && threadIdx.x == 0) {
    const uint32_t idesc = idesc_bf16(256, 256);
    const uint64_t a_desc = smem_desc_k_sw128(smem_u32(smem));
    const uint64_t b_desc = smem_desc_k_sw128(smem_u32(smem + 16 * 1024));
    t0 = clock64();
    for (int r = 0; r < rounds; ++r) {
#pragma unroll
      for (int k = 0; k < KT / 16; ++k) umma2_ss(tm, a_desc + 2 * k, b_desc + 2 * k, idesc, k != 0);
    }
    umma2_commit_both(&bar);
  }
  mbar_wait(&bar, 0, &status);
  if (rank == 0 && threadIdx.x == 0) { t1 = clock64(); cycles[0] = t1 - t0; }
  tc_fence_after();
  {
    const int q = threadIdx.x >> 5, lane = threadIdx.x & 31, r = q * 32 + lane;
    for (int ch = 0; ch < 8; ++ch) {
      float v[32];
      tmem_ld_32x32(tm + ((uint32_t)(q * 32) << 16) + ch * 32, v);
      for (int i = 0; i < 32; ++i) out[(size_t)(128 * rank + r) * 256 + ch * 32 + i] = v[i];
    }
  }
  if (threadIdx.x == 0 && status != 0) atomicExch(status_out, status);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                      // nobody frees tensor memory while the peer may still read through it
  if (threadIdx.x < 32) tmem_dealloc2(slot, 256);
}

int main() {
  float* d_out; long long* d_cyc; int* d_status;
  cudaMalloc(&d_out, 256 * 256 * 4); cudaMalloc(&d_cyc, 8); cudaMalloc(&d_status, 4);
  cudaMemset(d_out, 0, 256 * 256 * 4); cudaMemset(d_status, 0, 4);
  const int smem = 33 * 1024 + 1024;
  cudaFuncSetAttribute(pair_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  for (int rounds : {1, 64}) {
    pair_probe<<<2, 128, smem>>>(d_out, d_cyc, d_status, rounds);
    cudaError_t e = cudaDeviceSynchronize();
    static float h[256 * 256];
    long long cyc = 0; int st = 0;
    cudaMemcpy(h, d_out, sizeof(h), cudaMemcpyDeviceToHost);
    cudaMemcpy(&cyc, d_cyc, 8, cudaMemcpyDeviceToHost);
    cudaMemcpy(&st, d_status, 4, cudaMemcpyDeviceToHost);
    double maxerr = 0;
    for (int m = 0; m < 256; ++m)
      for (int n = 0; n < 256; ++n) {
        double ref = 0;
        for (int k = 0; k < KT; ++k) ref += ((m % 7) - 3 + 0.25 * k) * (double)(((n + 3 * k) % 5) - 2);
        maxerr = fmax(maxerr, fabs(ref - h[m * 256 + n]));
      }
    printf("rounds %2d: %s, wait status %d, max abs error vs CPU %.4f, %.1f cycles per M256 N256 K16 MMA\n", rounds,
           cudaGetErrorString(e), st, maxerr, (double)cyc / (rounds * (KT / 16)));
    if (e != cudaSuccess) break;
  }
  return 0;
}
