// Scoring-head-first scheduling of a short DARE-KV step (Alg. 1 lines 2-6).  The refresh set needs only the
// scoring head's 128 columns of Q (Sec. 3.2): on a step of a few hundred tokens that sliver is computed first, with
// the reduction spread over many CTAs, the drift score (Sec. 3.1) is taken from it, and the gathered K/V projection
// can then run beside the full Q projection instead of behind it.
//   q_sliver_kernel    C[128 rows, 128] = x_norm[rows, k-slice] * W_Q[head rows, k-slice]^T on the tensor cores, one CTA
//                      per (row tile, slice of the reduction): every operand tile of the slice is requested at once (no
//                      ring), the fp32 accumulator goes from tensor memory to a buffer of partial sums
//   head_score_kernel  one warp per token: sums the partials in a fixed order (the result does not depend on which CTA
//                      finished first), scores against the stored query, stores the new one
#include "layer.h"
#include "tc.h"
#include "tc_ptx.cuh"

namespace dare {

using namespace ptx;

namespace {
constexpr int BM = 128, BN = 128, BK = 64;
constexpr int TILE_BYTES = BM * BK * 2;               // one operand tile of 64 k-elements: 16 KB
constexpr int STAGE_BYTES = 2 * TILE_BYTES;
constexpr int SMEM_BYTES = kSliverMaxKb * STAGE_BYTES + 256 + 1024;
}  // namespace

__global__ void __launch_bounds__(128, 1)
q_sliver_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w, const SliverParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kSliverMaxKb * STAGE_BYTES);
  uint64_t* accum_bar = full_bar + kSliverMaxKb;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_bar + 1);
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int mt = blockIdx.x, ks = blockIdx.y;
  const int kb0 = ks * p.kb_per_cta;
  const int nkb = min(p.kb_per_cta, p.K / BK - kb0);          // >= 1 by the launcher's choice of the grid
  if (threadIdx.x == 0) {
    for (int i = 0; i < nkb; ++i) mbar_init(&full_bar[i], 2);  // one arrival with the W tile's bytes, one with the A tile's
    mbar_init(accum_bar, 1);
    fence_mbar_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_w);
    // the weights do not depend on the kernel before this one
    for (int i = 0; i < nkb; ++i) {
      mbar_arrive_expect_tx(&full_bar[i], TILE_BYTES);
      tma_load_2d(smem + i * STAGE_BYTES + TILE_BYTES, &tm_w, (kb0 + i) * BK, p.w_row0, &full_bar[i]);
    }
  }
  if (warp == 1) { tmem_alloc(tmem_slot, BN); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();
  pdl_launch_dependents();
  // rows of this tile in the compact [tokens, K] matrix (a tile never crosses into rows it does not own in the
  // partial buffer: rows past the sequence's end are computed on whatever follows and never read)
  const int b = mt / p.tiles_per_seq, tis = mt - b * p.tiles_per_seq;
  const int a_row = b * p.seq_act + tis * BM;
  if (warp == 0) {
    if (elect_one()) {
      for (int i = 0; i < nkb; ++i) {
        mbar_arrive_expect_tx(&full_bar[i], TILE_BYTES);
        tma_load_2d(smem + i * STAGE_BYTES, &tm_a, (kb0 + i) * BK, a_row, &full_bar[i]);
      }
    }
    __syncwarp();
    constexpr uint32_t idesc = idesc_bf16(BM, BN);
    for (int i = 0; i < nkb; ++i) {
      mbar_wait(&full_bar[i], 0, p.status);
      tc_fence_after();
      if (elect_one()) {
        const uint32_t a_addr = smem_u32(smem + i * STAGE_BYTES);
        const uint64_t a_desc = smem_desc_k_sw128(a_addr), b_desc = smem_desc_k_sw128(a_addr + TILE_BYTES);
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) umma_ss(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, (i | k) != 0 ? 1u : 0u);
        if (i == nkb - 1) umma_commit(accum_bar);
      }
      __syncwarp();
    }
  }
  mbar_wait(accum_bar, 0, p.status);
  tc_fence_after();
  // tensor memory -> partial sums: thread <-> row (warp w holds TMEM lanes 32w .. 32w + 31), 32 columns at a time
  {
    const int r = warp * 32 + lane;
    float* dst = p.partial + ((size_t)ks * p.rows_pad + (size_t)mt * BM + r) * BN;
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
    for (int ch = 0; ch < BN / 32; ++ch) {
      float v[32];
      tmem_ld_32x32(t_lane + ch * 32, v);
#pragma unroll
      for (int g4 = 0; g4 < 8; ++g4)
        *reinterpret_cast<float4*>(dst + ch * 32 + 4 * g4) = make_float4(v[4 * g4], v[4 * g4 + 1], v[4 * g4 + 2], v[4 * g4 + 3]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, BN);
}

// Sec. 3.1 from the partial sums: s_t = 1 - cos(q_t, stored q_t), then the stored query becomes q_t.
__global__ void __launch_bounds__(256)
head_score_kernel(const float* __restrict__ partial, int ksplit, int rows_pad, int tiles_per_seq, StepGeom g,
                  float* __restrict__ q_prev, float* __restrict__ scores) {
  pdl_wait();
  pdl_launch_dependents();
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= g.tokens()) return;
  const int b = t / g.seq_act, i = t - b * g.seq_act;
  const size_t prow = (size_t)(b * tiles_per_seq + i / BM) * BM + (i % BM);
  float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int ks = 0; ks < ksplit; ++ks) {
    const float4 v = __ldcg(reinterpret_cast<const float4*>(partial + ((size_t)ks * rows_pad + prow) * BN) + lane);
    q.x += v.x; q.y += v.y; q.z += v.z; q.w += v.w;
  }
  float* qp = q_prev + (size_t)g.cache_row(t) * BN;
  const float4 a = *(reinterpret_cast<const float4*>(qp) + lane);
  float dot = q.x * a.x + q.y * a.y + q.z * a.z + q.w * a.w;
  float n1 = q.x * q.x + q.y * q.y + q.z * q.z + q.w * q.w;
  float n2 = a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    dot += __shfl_xor_sync(0xffffffffu, dot, o);
    n1 += __shfl_xor_sync(0xffffffffu, n1, o);
    n2 += __shfl_xor_sync(0xffffffffu, n2, o);
  }
  *(reinterpret_cast<float4*>(qp) + lane) = q;
  if (lane == 0) {
    const float den = sqrtf(n1) * sqrtf(n2);
    scores[t] = 1.f - (den > 0.f ? dot / den : 0.f);
  }
}

bool sliver_geometry(int K, int* ksplit, int* kb_per_cta) {
  const int KB = K / BK;
  int per = 4;                                        // 64 KB of operands per CTA: short main loop, many CTAs
  int split = (KB + per - 1) / per;
  if (split > kSliverMaxSplit) {
    split = kSliverMaxSplit;
    per = (KB + split - 1) / split;
  }
  if (per > kSliverMaxKb) return false;
  split = (KB + per - 1) / per;                       // no empty slice
  *ksplit = split;
  *kb_per_cta = per;
  return true;
}

cudaError_t launch_q_sliver(const CUtensorMap& a, const CUtensorMap& w, const SliverParams& p, int m_tiles, cudaStream_t st) {
  static std::atomic<unsigned long long> attr_done{0};
  if (cudaError_t e = ensure_dyn_smem(q_sliver_kernel, SMEM_BYTES, attr_done); e != cudaSuccess) return e;
  return launch_pdl(q_sliver_kernel, dim3(m_tiles, p.ksplit), dim3(128), SMEM_BYTES, st, 1, a, w, p);
}

cudaError_t launch_head_score(const SliverParams& p, const StepGeom& g, float* q_prev, float* scores, cudaStream_t st) {
  const int T_ = g.tokens();
  return launch_pdl(head_score_kernel, dim3((T_ + 7) / 8), dim3(256), 0, st, 1, (const float*)p.partial, p.ksplit, p.rows_pad,
                    p.tiles_per_seq, g, q_prev, scores);
}

}  // namespace dare
