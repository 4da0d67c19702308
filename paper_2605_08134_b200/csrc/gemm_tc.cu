// bf16 projection GEMMs on the 5th-generation tensor cores: C[m, n] = sum_k A[m, k] * W[n, k]  (W = [out, in],
// Alg. 1 lines 2, 7, 11).  One 128 x BN output tile per CTA:
//   warp 0    TMA producer: A and W tiles (64 k-elements = 128 bytes per row, 128-byte swizzle) into a ring of stages
//   warp 1    allocates tensor memory, one thread issues tcgen05.mma (M = 128, N = BN, K = 16) into fp32 accumulators
//             and commits each stage back to the producer
//   warps 2-5 epilogue: each thread owns one output row (one TMEM lane), reads it with tcgen05.ld and applies the
//             fused tail of that projection:
//               Q    drift score of the scoring head against the stored query (Sec. 3.1), store of the new query,
//                    rotary embedding, bf16 store
//               K/V  rotary embedding of K, scatter of both rows into the caches at the refresh-set rows (Eq. 3)
//               OUT  plain bf16 store of y
// Column mapping of a tile: BN/2 columns starting at `lo` and BN/2 columns starting at `lo + head_dim/2` of one head,
// so that both elements of every rotary pair sit in the same thread.
#include "layer.h"
#include "tc.h"
#include "tc_ptx.cuh"

namespace dare {

using namespace ptx;

template <int BN>
struct GemmSmem {
  static constexpr int BM = 128, BK = 64;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 128) ? 6 : 8;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;  // barriers + slack for 1024-byte alignment
};

template <int BN, int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
               const __grid_constant__ CUtensorMap tm_b1, const GemmParams p) {
  using S = GemmSmem<BN>;
  constexpr int STAGES = S::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + S::BAR_OFFSET);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* accum_bar = empty_bar + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_bar + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt = blockIdx.x, mt = blockIdx.y;

  // ---- which rows does this tile cover? (uniform over the CTA; a tile past the refresh set leaves at once)
  int a_row, t0, rows_valid;
  if (p.count != nullptr) {
    const int n = min(*p.count, p.m_total);
    t0 = mt * 128;
    if (t0 >= n) return;
    rows_valid = min(128, n - t0);
    a_row = t0;
  } else {
    const int b = mt / p.tiles_per_seq, tis = mt - b * p.tiles_per_seq;
    t0 = b * p.seq_act + tis * 128;
    rows_valid = min(128, p.seq_act - tis * 128);
    a_row = b * p.a_seq_stride + p.a_row0 + tis * 128;
  }
  // ---- which columns?
  const int tph = p.hd_map / BN;                 // tiles per head
  const int nt_local = nt < p.n_split ? nt : nt - p.n_split;
  const int head = nt_local / tph, jb = nt_local - head * tph;
  const int col_lo = head * p.hd_map + jb * (BN / 2);
  const int col_hi = col_lo + p.hd_map / 2;
  const CUtensorMap* tm_b = nt < p.n_split ? &tm_b0 : &tm_b1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(accum_bar, 1);
    fence_mbar_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(tm_b);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, BN < 32 ? 32 : BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int KB = p.K / 64;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        mbar_wait(&empty_bar[s], ((kb / STAGES) & 1) ^ 1, p.status);
        uint8_t* a_dst = smem + s * S::STAGE_BYTES;
        uint8_t* b_dst = a_dst + S::A_BYTES;
        mbar_arrive_expect_tx(&full_bar[s], S::STAGE_BYTES);
        tma_load_2d(a_dst, &tm_a, kb * 64, a_row, &full_bar[s]);
        tma_load_2d(b_dst, tm_b, kb * 64, col_lo, &full_bar[s]);
        tma_load_2d(b_dst + S::B_BYTES / 2, tm_b, kb * 64, col_hi, &full_bar[s]);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(128, BN);
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        mbar_wait(&full_bar[s], (kb / STAGES) & 1, p.status);
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + s * S::STAGE_BYTES);
        const uint64_t a_desc = smem_desc_k_sw128(a_addr);
        const uint64_t b_desc = smem_desc_k_sw128(a_addr + S::A_BYTES);
#pragma unroll
        for (int k = 0; k < 4; ++k)  // 16 k-elements = 32 bytes = 2 descriptor address units per MMA
          umma_ss(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
        umma_commit(&empty_bar[s]);
      }
      umma_commit(accum_bar);
    }
    __syncwarp();
  } else {
    // ---- epilogue: thread <-> output row
    mbar_wait(accum_bar, 0, p.status);
    tc_fence_after();
    const int quarter = warp & 3;               // TMEM lanes this warp may touch: 32*quarter .. +31
    const int r = quarter * 32 + lane;
    const bool valid = r < rows_valid;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    int t = 0;                                  // token (flat active index) of this row
    if (valid) t = p.idx ? p.idx[t0 + r] : t0 + r;
    const int pos = p.g.position(t);
    const size_t crow = (size_t)p.g.cache_row(t);
    constexpr int NCH = BN / 64;                // chunks of 32 column pairs
    constexpr int HALF_W = BN / 2;
    const bool is_b1 = nt >= p.n_split;

    float dot = 0.f, n1 = 0.f, n2 = 0.f;
#pragma unroll 1
    for (int c = 0; c < NCH; ++c) {
      float lo[32], hi[32];
      tmem_ld_32x32(t_lane + c * 32, lo);
      tmem_ld_32x32(t_lane + HALF_W + c * 32, hi);
      if (!valid) continue;
      const int j0 = jb * HALF_W + c * 32;       // index of lo[0] inside the head (rotary pair index)
      if (EPI == EPI_Q) {
        if (head == p.g.score_head) {
          float* qp = p.q_prev + crow * p.g.head_dim;
          if (p.has_prev) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const float4 a = *reinterpret_cast<const float4*>(qp + j0 + i);
              const float4 b = *reinterpret_cast<const float4*>(qp + p.g.head_dim / 2 + j0 + i);
              dot = fmaf(lo[i], a.x, dot); dot = fmaf(lo[i + 1], a.y, dot);
              dot = fmaf(lo[i + 2], a.z, dot); dot = fmaf(lo[i + 3], a.w, dot);
              dot = fmaf(hi[i], b.x, dot); dot = fmaf(hi[i + 1], b.y, dot);
              dot = fmaf(hi[i + 2], b.z, dot); dot = fmaf(hi[i + 3], b.w, dot);
              n2 = fmaf(a.x, a.x, n2); n2 = fmaf(a.y, a.y, n2); n2 = fmaf(a.z, a.z, n2); n2 = fmaf(a.w, a.w, n2);
              n2 = fmaf(b.x, b.x, n2); n2 = fmaf(b.y, b.y, n2); n2 = fmaf(b.z, b.z, n2); n2 = fmaf(b.w, b.w, n2);
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) { n1 = fmaf(lo[i], lo[i], n1); n1 = fmaf(hi[i], hi[i], n1); }
          }
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            *reinterpret_cast<float4*>(qp + j0 + i) = make_float4(lo[i], lo[i + 1], lo[i + 2], lo[i + 3]);
            *reinterpret_cast<float4*>(qp + p.g.head_dim / 2 + j0 + i) =
                make_float4(hi[i], hi[i + 1], hi[i + 2], hi[i + 3]);
          }
        }
      }
      const bool rotate = (EPI == EPI_Q) || (EPI == EPI_KV && !is_b1);
      if (rotate) {
        const float2* cs = p.rope + (size_t)pos * (p.g.head_dim / 2) + j0;
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float4 c2 = *reinterpret_cast<const float4*>(cs + i);   // (cos, sin) of two consecutive pairs
          const float a0 = lo[i], b0 = hi[i], a1 = lo[i + 1], b1 = hi[i + 1];
          lo[i] = a0 * c2.x - b0 * c2.y;  hi[i] = a0 * c2.y + b0 * c2.x;
          lo[i + 1] = a1 * c2.z - b1 * c2.w;  hi[i + 1] = a1 * c2.w + b1 * c2.z;
        }
      }
      __nv_bfloat16* out = is_b1 ? p.out1 : p.out0;
      const size_t orow = p.out_is_cache ? crow : (size_t)t;
      __nv_bfloat16* dst = out + orow * p.ld_out;
      uint4* d_lo = reinterpret_cast<uint4*>(dst + col_lo + c * 32);
      uint4* d_hi = reinterpret_cast<uint4*>(dst + col_hi + c * 32);
#pragma unroll
      for (int v = 0; v < 4; ++v) { d_lo[v] = pack8_bf16(lo + 8 * v); d_hi[v] = pack8_bf16(hi + 8 * v); }
    }
    if (EPI == EPI_Q) {
      if (valid && head == p.g.score_head) {
        float s;
        if (p.has_prev) {
          const float den = sqrtf(n1) * sqrtf(n2);
          s = 1.f - (den > 0.f ? dot / den : 0.f);
        } else {
          s = __int_as_float(0x7f800000);
        }
        p.scores[t] = s;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, BN < 32 ? 32 : BN);
}

template <int BN, int EPI>
static cudaError_t launch_one(const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1, const GemmParams& p,
                              int n_tiles, int m_tiles, cudaStream_t st) {
  static bool attr_set = false;
  auto kern = gemm_tc_kernel<BN, EPI>;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmSmem<BN>::TOTAL);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid(n_tiles, m_tiles);
  kern<<<grid, 192, GemmSmem<BN>::TOTAL, st>>>(a, b0, b1, p);
  return cudaGetLastError();
}

cudaError_t launch_gemm_tc(int bn, int epi, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                           const GemmParams& p, int n_tiles, int m_tiles, cudaStream_t st) {
  if (m_tiles <= 0 || n_tiles <= 0) return cudaSuccess;
  if (bn == 128) {
    if (epi == EPI_Q) return launch_one<128, EPI_Q>(a, b0, b1, p, n_tiles, m_tiles, st);
    if (epi == EPI_KV) return launch_one<128, EPI_KV>(a, b0, b1, p, n_tiles, m_tiles, st);
    return launch_one<128, EPI_OUT>(a, b0, b1, p, n_tiles, m_tiles, st);
  }
  if (bn == 64) {
    if (epi == EPI_KV) return launch_one<64, EPI_KV>(a, b0, b1, p, n_tiles, m_tiles, st);
    if (epi == EPI_OUT) return launch_one<64, EPI_OUT>(a, b0, b1, p, n_tiles, m_tiles, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace dare
