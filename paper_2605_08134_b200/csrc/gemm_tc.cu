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
  static constexpr int STAGES = (BN == 256) ? 4 : ((BN == 128) ? 6 : 8);
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
  const bool dbg = p.debug != nullptr && blockIdx.x == 0 && blockIdx.y == 0;
  if (dbg && threadIdx.x == 0) p.debug[0] = globaltimer_ns();
  const int lin = blockIdx.y * gridDim.x + blockIdx.x;
  if (EPI == EPI_Q && p.debug != nullptr && threadIdx.x == 0 && lin < 1024) {
    unsigned smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    p.debug[64 + 3 * lin] = smid;
    p.debug[64 + 3 * lin + 1] = globaltimer_ns();
  }

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
  // Each CTA walks the reduction dimension from its own starting block, so that the CTAs sharing an operand tile
  // do not all ask the L2 for the same lines at the same moment.
  const int k_rot = (int)((nt * p.rot_n + mt * p.rot_m) % KB);
  if (dbg && threadIdx.x == 0) p.debug[1] = globaltimer_ns();

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % STAGES;
        mbar_wait(&empty_bar[s], ((kb / STAGES) & 1) ^ 1, p.status);
        uint8_t* a_dst = smem + s * S::STAGE_BYTES;
        uint8_t* b_dst = a_dst + S::A_BYTES;
        mbar_arrive_expect_tx(&full_bar[s], S::STAGE_BYTES);
        int kx = kb + k_rot;
        if (kx >= KB) kx -= KB;
        tma_load_2d(a_dst, &tm_a, kx * 64, a_row, &full_bar[s]);
        if (p.b_single) {                       // both column halves are adjacent rows of W: one box
          tma_load_2d(b_dst, tm_b, kx * 64, col_lo, &full_bar[s]);
        } else {
          tma_load_2d(b_dst, tm_b, kx * 64, col_lo, &full_bar[s]);
          tma_load_2d(b_dst + S::B_BYTES / 2, tm_b, kx * 64, col_hi, &full_bar[s]);
        }
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
        if (dbg && kb == 0) p.debug[2] = globaltimer_ns();
        const uint32_t a_addr = smem_u32(smem + s * S::STAGE_BYTES);
        const uint64_t a_desc = smem_desc_k_sw128(a_addr);
        const uint64_t b_desc = smem_desc_k_sw128(a_addr + S::A_BYTES);
        for (int rep = 0; rep < p.mma_rep; ++rep)
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
    if (dbg && threadIdx.x == 64) p.debug[3] = globaltimer_ns();
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

    constexpr int ROW_BYTES = BN * 2;            // one staged output row (bf16)
    constexpr int UNITS = ROW_BYTES / 16;        // 16-byte units per staged row
    // The operand ring is idle once the accumulator is complete: its first 128 x ROW_BYTES bytes stage the tile so
    // that the global stores below are whole contiguous row segments.
    uint8_t* stg = smem;
    const size_t tm_rows = (size_t)p.q_prev_rows;  // row count of the transposed stored-query array
    const bool rotate = (EPI == EPI_Q) || (EPI == EPI_KV && !is_b1);
    const bool score_tile = (EPI == EPI_Q) && head == p.g.score_head;

    float dot = 0.f, n1 = 0.f, n2 = 0.f;
#pragma unroll 1
    for (int c = 0; c < NCH; ++c) {
      float lo[32], hi[32];
      tmem_ld_32x32(t_lane + c * 32, lo);
      tmem_ld_32x32(t_lane + HALF_W + c * 32, hi);
      const int j0 = jb * HALF_W + c * 32;       // index of lo[0] inside the head (rotary pair index)
      if (valid) {
        if (score_tile) {
          // stored query, transposed [head_dim][cache rows]: consecutive rows of a tile are consecutive addresses
          float* qa = p.q_prev + (size_t)j0 * tm_rows + crow;
          float* qb = p.q_prev + (size_t)(p.g.head_dim / 2 + j0) * tm_rows + crow;
          if (p.has_prev) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float a = qa[(size_t)i * tm_rows], b = qb[(size_t)i * tm_rows];
              dot = fmaf(lo[i], a, dot); dot = fmaf(hi[i], b, dot);
              n2 = fmaf(a, a, n2); n2 = fmaf(b, b, n2);
              n1 = fmaf(lo[i], lo[i], n1); n1 = fmaf(hi[i], hi[i], n1);
            }
          }
#pragma unroll
          for (int i = 0; i < 32; ++i) { qa[(size_t)i * tm_rows] = lo[i]; qb[(size_t)i * tm_rows] = hi[i]; }
        }
        if (rotate) {
          // rotary table, transposed [pair index][position]
          const float2* cs = p.rope + (size_t)j0 * p.g.max_seq + pos;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float2 cv = cs[(size_t)i * p.g.max_seq];
            const float a0 = lo[i], b0 = hi[i];
            lo[i] = a0 * cv.x - b0 * cv.y;
            hi[i] = a0 * cv.y + b0 * cv.x;
          }
        }
      }
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const int u_lo = c * 4 + v, u_hi = UNITS / 2 + c * 4 + v;
        *reinterpret_cast<uint4*>(stg + r * ROW_BYTES + ((u_lo ^ (r & (UNITS - 1))) << 4)) = pack8_bf16(lo + 8 * v);
        *reinterpret_cast<uint4*>(stg + r * ROW_BYTES + ((u_hi ^ (r & (UNITS - 1))) << 4)) = pack8_bf16(hi + 8 * v);
      }
    }
    if (score_tile && valid) {
      float sc;
      if (p.has_prev) {
        const float den = sqrtf(n1) * sqrtf(n2);
        sc = 1.f - (den > 0.f ? dot / den : 0.f);
      } else {
        sc = __int_as_float(0x7f800000);
      }
      p.scores[t] = sc;
    }
    __syncwarp();
    if (dbg && threadIdx.x == 64) p.debug[4] = globaltimer_ns();
    // ---- write-out: each warp stores its own 32 rows, UNITS lanes per row
    {
      __nv_bfloat16* out = is_b1 ? p.out1 : p.out0;
      const long long my_orow = valid ? (long long)(p.out_is_cache ? crow : (size_t)t) : -1;
      constexpr int ROWS_PER_IT = 32 / UNITS;
      const int unit = lane % UNITS;
      const int col = unit < UNITS / 2 ? col_lo + unit * 8 : col_hi + (unit - UNITS / 2) * 8;
#pragma unroll
      for (int rr = 0; rr < 32; rr += ROWS_PER_IT) {
        const int row_l = rr + lane / UNITS;
        const long long orow = __shfl_sync(0xffffffffu, my_orow, row_l);
        const int R = quarter * 32 + row_l;
        const uint4 v = *reinterpret_cast<const uint4*>(stg + R * ROW_BYTES + ((unit ^ (R & (UNITS - 1))) << 4));
        if (orow >= 0) *reinterpret_cast<uint4*>(out + (size_t)orow * p.ld_out + col) = v;
      }
    }
  }
  if (dbg && threadIdx.x == 64) p.debug[5] = globaltimer_ns();
  tc_fence_before();
  __syncthreads();
  if (p.debug != nullptr && threadIdx.x == 0) { atomicMax(&p.debug[6], globaltimer_ns()); atomicAdd(&p.debug[7], 1ull); }
  if (EPI == EPI_Q && p.debug != nullptr && threadIdx.x == 0 && lin < 1024) p.debug[64 + 3 * lin + 2] = globaltimer_ns();
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
  if (bn == 256 && epi == EPI_OUT) return launch_one<256, EPI_OUT>(a, b0, b1, p, n_tiles, m_tiles, st);
  if (bn == 64) {
    if (epi == EPI_KV) return launch_one<64, EPI_KV>(a, b0, b1, p, n_tiles, m_tiles, st);
    if (epi == EPI_OUT) return launch_one<64, EPI_OUT>(a, b0, b1, p, n_tiles, m_tiles, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace dare
