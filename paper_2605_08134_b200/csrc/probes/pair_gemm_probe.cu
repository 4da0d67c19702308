// Stand-alone probe (not part of libdare): a pipelined tile loop with tcgen05.mma.cta_group::2 over a cluster of two
// CTAs, operands by TMA, the loads of both CTAs completing on the leader's barrier.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o pair_gemm_probe pair_gemm_probe.cu -lcuda && ./pair_gemm_probe
// D[256 x 256] = A[256 x K] * W[256 x K]^T (bf16 in, fp32 out), K = 1024 in 16 blocks of 64, ring of 4 stages.
// CTA r of the pair loads rows [128 r, +128) of A and of W per k-block into its own shared memory (32 KB a stage
// instead of the 48 KB a single-CTA 128 x 256 tile needs); the leader's MMA thread waits for both CTAs' loads on its
// own full barrier, issues M256 N256 K16 MMAs and releases the stage in both CTAs with one commit per CTA.
// Every wait is bounded.
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>
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
// TMA load into this CTA's shared memory, completion (bytes) on a barrier given by its cluster address: the pair's
// leader's barrier
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* tmap, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}

constexpr int K = 1024, BK = 64, STAGES = 4, STAGE_BYTES = 32 * 1024;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1)
pair_gemm(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w, float* out,
          long long* cycles, int* status_out) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], accum_bar;
  __shared__ uint32_t slot;
  __shared__ int status;
  const uint32_t rank = cluster_ctarank();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&accum_bar, 1);
    fence_mbar_init();
    status = 0;
  }
  if (warp == 1) { tmem_alloc2(&slot, 256); tmem_relinquish2(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tm = ld_cluster_u32(map_to_cta(smem_u32(&slot), 0));
  const int nkb = K / BK;
  long long t0 = clock64();
  if (warp == 0 && lane == 0) {
    // producer of this CTA: its 128 rows of A and of W per stage; bytes are counted on the leader's full barrier
    for (int i = 0; i < nkb; ++i) {
      const int s = i % STAGES;
      mbar_wait(&empty_bar[s], ((i / STAGES) & 1) ^ 1, &status);
      if (rank == 0) mbar_arrive_expect_tx(&full_bar[s], 2 * STAGE_BYTES);     // both CTAs' bytes
      const uint32_t fb = map_to_cta(smem_u32(&full_bar[s]), 0);
      tma_load_2d_pair(smem + s * STAGE_BYTES, &tm_a, i * BK, 128 * (int)rank, fb);
      tma_load_2d_pair(smem + s * STAGE_BYTES + 16 * 1024, &tm_w, i * BK, 128 * (int)rank, fb);
    }
  } else if (warp == 1 && lane == 0 && rank == 0) {
    const uint32_t idesc = idesc_bf16(256, 256);
    for (int i = 0; i < nkb; ++i) {
      const int s = i % STAGES;
      mbar_wait(&full_bar[s], (i / STAGES) & 1, &status);
      tc_fence_after();
      const uint64_t a_desc = smem_desc_k_sw128(smem_u32(smem + s * STAGE_BYTES));
      const uint64_t b_desc = smem_desc_k_sw128(smem_u32(smem + s * STAGE_BYTES + 16 * 1024));
#pragma unroll
      for (int k = 0; k < BK / 16; ++k) umma2_ss(tm, a_desc + 2 * k, b_desc + 2 * k, idesc, (i | k) != 0);
      umma2_commit_both(&empty_bar[s]);
    }
    umma2_commit_both(&accum_bar);
  }
  __syncwarp();
  mbar_wait(&accum_bar, 0, &status);
  if (rank == 0 && threadIdx.x == 0) cycles[0] = clock64() - t0;
  tc_fence_after();
  {
    const int q = warp, r = q * 32 + lane;
    for (int ch = 0; ch < 8; ++ch) {
      float v[32];
      tmem_ld_32x32(tm + ((uint32_t)(q * 32) << 16) + ch * 32, v);
      for (int i = 0; i < 32; ++i) out[(size_t)(128 * rank + r) * 256 + ch * 32 + i] = v[i];
    }
  }
  if (threadIdx.x == 0 && status != 0) atomicExch(status_out, status);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) tmem_dealloc2(slot, 256);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int main() {
  void* fp = nullptr;
  cudaDriverEntryPointQueryResult q;
  cudaFree(0);
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &q) != cudaSuccess || !fp) return 1;
  EncodeTiledFn enc = (EncodeTiledFn)fp;
  std::vector<__nv_bfloat16> ha(256 * K), hw(256 * K);
  std::vector<float> fa(256 * K), fw(256 * K);
  srand(1);
  for (int i = 0; i < 256 * K; ++i) {
    fa[i] = (float)(rand() % 9 - 4) * 0.25f; fw[i] = (float)(rand() % 7 - 3) * 0.5f;
    ha[i] = __float2bfloat16(fa[i]); hw[i] = __float2bfloat16(fw[i]);
  }
  __nv_bfloat16 *da, *dw; float* d_out; long long* d_cyc; int* d_status;
  cudaMalloc(&da, 256 * K * 2); cudaMalloc(&dw, 256 * K * 2); cudaMalloc(&d_out, 256 * 256 * 4);
  cudaMalloc(&d_cyc, 8); cudaMalloc(&d_status, 4);
  cudaMemcpy(da, ha.data(), 256 * K * 2, cudaMemcpyHostToDevice);
  cudaMemcpy(dw, hw.data(), 256 * K * 2, cudaMemcpyHostToDevice);
  cudaMemset(d_status, 0, 4);
  CUtensorMap ma, mw;
  cuuint64_t dims[2] = {(cuuint64_t)K, 256}; cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {64, 128}; cuuint32_t estr[2] = {1, 1};
  if (enc(&ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, da, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return 2;
  if (enc(&mw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, dw, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return 2;
  const int smem = STAGES * STAGE_BYTES + 1024;
  cudaFuncSetAttribute(pair_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  for (int rep = 0; rep < 2; ++rep) pair_gemm<<<2, 128, smem>>>(ma, mw, d_out, d_cyc, d_status);
  cudaError_t e = cudaDeviceSynchronize();
  std::vector<float> h(256 * 256);
  long long cyc = 0; int st = 0;
  cudaMemcpy(h.data(), d_out, 256 * 256 * 4, cudaMemcpyDeviceToHost);
  cudaMemcpy(&cyc, d_cyc, 8, cudaMemcpyDeviceToHost);
  cudaMemcpy(&st, d_status, 4, cudaMemcpyDeviceToHost);
  double maxerr = 0;
  for (int m = 0; m < 256; ++m)
    for (int n = 0; n < 256; ++n) {
      double ref = 0;
      for (int k = 0; k < K; ++k) ref += (double)fa[m * K + k] * fw[n * K + k];
      maxerr = fmax(maxerr, fabs(ref - h[m * 256 + n]));
    }
  printf("%s, wait status %d, max abs error vs CPU %.4f, main loop %lld cycles for %d k-blocks (%.0f per k-block)\n",
         cudaGetErrorString(e), st, maxerr, cyc, K / BK, (double)cyc / (K / BK));
  return 0;
}
