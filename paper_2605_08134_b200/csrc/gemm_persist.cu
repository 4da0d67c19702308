// Persistent form of the bf16 projection GEMM for launches of many row tiles (Alg. 1 lines 2, 7, 11 over thousands
// of tokens): C[m, n] = sum_k A[m, k] * W[n, k], one CTA per SM walking the 128 x 256 output tiles of the launch,
// the finishing pass of tile i running while the tensor core is already on tile i + 1.
//   warp 0     TMA producer: 128 rows of A and 256 rows of W per 64 k-elements into a ring of 4 stages that runs on
//              across tile boundaries
//   warp 1     one elected lane issues tcgen05.mma (M = 128, N = 256, K = 16) into one of TWO 128 x 256 fp32
//              accumulators in tensor memory (all 512 columns), alternating per tile
//   warps 2-5  finishing pass, one warp per TMEM lane quarter (32 rows), independent of one another: a quarter of
//              a head at a time (32 + 32 columns whose rotary partners they are) goes tensor memory -> registers
//              (thread <-> row) -> the warp's own 8 KB of shared memory -> registers (half-warp <-> row, lane <->
//              two column pairs), where the fused tail runs (score, stored query, rotary embedding, residual) and
//              the row segments are stored; the accumulator is handed back after the last read of tensor memory
// In the one-tile-per-CTA kernel of gemm_tc.cu a tile costs set-up + pipeline fill + finishing pass + the gap to the
// next CTA on top of its main loop (about 30 % at these sizes, measured); here the main loops follow one another.
// Listed launches (the rows of a refresh set, Alg. 1 line 6 / the gathered output projection, given by an index list
// with a device-side count): A is a compact copy of the listed rows, made by a copy kernel before the launch (row r of
// the list = row r of the copy), so that every operand comes through TMA; the number of row tiles is read from the
// count, so no CTA is spent on tiles past the refresh set; the finishing pass takes positions and cache rows from the
// tokens.  Such a launch is issued in both forms below (one-CTA and two-CTA tiles), and the one the count does not
// favour leaves at once.
// PAIR: the CTAs of a cluster of two take row tiles 2i and 2i + 1 of the same column tile as one
// M = 256 tcgen05.mma.cta_group::2 issued by the even CTA; each keeps its own 128 rows of A and 128 of the W tile's
// 256 rows (32 KB per stage, six stages), which takes a third off what an SM pulls from the L2 per flop: the
// one-CTA form runs its main loop at 667 cycles per 64 k-elements against 512 of tensor work, bound by that
// traffic (ncu: tensor pipe 87 % active).  Both CTAs' TMA loads complete on the even CTA's barriers, stages and
// accumulators are released to both by one commit each, and the finishing warps of both CTAs hand an accumulator
// back by arriving on the even CTA's barrier.
// No reduction split, epilogues Q, K/V, OUT, OUT_RES.
#include "layer.h"
#include "tc.h"
#include "tc_ptx.cuh"

namespace dare {

using namespace ptx;

namespace {
constexpr int BM = 128, BN = 256, BK = 64, HD = 128;
constexpr int A_BYTES = BM * BK * 2;
template <bool PAIR>
struct Ring {
  static constexpr int B_BYTES = (PAIR ? BN / 2 : BN) * BK * 2;    // this CTA's part of the W tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = PAIR ? 6 : 4;
};
constexpr int STG_OFFSET = Ring<false>::STAGES * Ring<false>::STAGE_BYTES;   // finishing warps' staging: 4 x (32 rows x 64 fp32)
static_assert(Ring<true>::STAGES * Ring<true>::STAGE_BYTES == STG_OFFSET, "both rings end where the staging begins");
constexpr int STG_ROW_BYTES = 64 * 4, STG_WARP_BYTES = 32 * STG_ROW_BYTES;
constexpr int ACC_OFFSET = STG_OFFSET + 4 * STG_WARP_BYTES;   // partial score sums: [128 rows][3] fp32
constexpr int BAR_OFFSET = ACC_OFFSET + BM * 12;
static_assert(BAR_OFFSET + 256 + 1024 <= 227 * 1024, "shared memory of one CTA");
constexpr int SMEM_TOTAL = BAR_OFFSET + 256 + 1024;  // barriers + slack for 1024-byte alignment
constexpr int kWarps = 6;

struct TileGeom {
  int nt, mt, n0, is_b1;
  int t0, rows_valid, a_row, pos0;
  size_t crow0;
};
// n_rows: rows of a gathered launch (the device-side count), unused otherwise
__device__ __forceinline__ TileGeom tile_geom(const GemmParams& p, int tile, int n_tiles, bool gather, int n_rows) {
  TileGeom t;
  t.nt = tile % n_tiles;
  t.mt = tile / n_tiles;
  t.is_b1 = t.nt >= p.n_split;
  t.n0 = (t.is_b1 ? t.nt - p.n_split : t.nt) * BN;
  if (gather) {                      // rows t0 .. of the index list; position and cache row come from the tokens
    t.t0 = t.mt * BM;
    t.rows_valid = min(BM, n_rows - t.t0);
    t.a_row = t.t0; t.pos0 = 0; t.crow0 = 0;     // (a_row: the row of a compact copy of the listed rows)
    return t;
  }
  const int b = t.mt / p.tiles_per_seq, tis = t.mt - b * p.tiles_per_seq;
  t.t0 = b * p.seq_act + tis * BM;
  t.rows_valid = min(BM, p.seq_act - tis * BM);
  t.a_row = b * p.a_seq_stride + p.a_row0 + tis * BM;
  t.pos0 = p.g.pos_begin + tis * BM;
  t.crow0 = (size_t)b * p.g.max_seq + t.pos0;
  return t;
}
}  // namespace

// GATHER: the rows of the launch are listed by an index list with a device-side count (row geometry and finishing
// pass by token); A maps a compact copy of them.
template <int EPI, bool GATHER, bool PAIR>
__global__ void __launch_bounds__(kWarps * 32, 1)
gemm_persist_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                    const __grid_constant__ CUtensorMap tm_b1, const GemmParams p, const int n_tiles,
                    const int total_tiles_dense) {
  constexpr int STAGES = Ring<PAIR>::STAGES, STAGE_BYTES = Ring<PAIR>::STAGE_BYTES, B_BYTES = Ring<PAIR>::B_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + BAR_OFFSET);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* acc_full = empty_bar + STAGES;     // [2] accumulator complete (MMA -> finishing warps)
  uint64_t* acc_empty = acc_full + 2;          // [2] accumulator read out (finishing warps -> MMA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const bool dbg = p.debug != nullptr && blockIdx.x == 0;
  if (dbg && threadIdx.x == 0) p.debug[0] = globaltimer_ns();
  // PAIR: place in the MMA pair (cluster of two along x); place 0 issues the MMAs and owns the barriers that count
  const int pr = PAIR ? (int)cluster_ctarank() : 0;
  // the walk over the launch's work: single tiles, or pairs of row tiles taken by the two CTAs of a cluster
  const int walker = PAIR ? (int)blockIdx.x / 2 : (int)blockIdx.x, n_walkers = PAIR ? (int)gridDim.x / 2 : (int)gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], PAIR ? 8 : 4); }
    fence_mbar_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b0);
    prefetch_tmap(&tm_b1);
  }
  if (warp == 1) {
    if (PAIR) { tmem_alloc2(tmem_slot, 512); tmem_relinquish2(); }
    else { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  }
  tc_fence_before();
  __syncthreads();
  uint32_t tmem_base;
  if (PAIR) {
    cluster_sync_all();              // both CTAs have their barriers and tensor memory before either touches the other's
    tc_fence_after();
    tmem_base = ld_cluster_u32(map_to_cta(smem_u32(tmem_slot), 0));
  } else {
    tc_fence_after();
    tmem_base = *tmem_slot;
  }
  // A (and everything the finishing pass reads) may be the previous kernel's output
  pdl_wait();
  pdl_launch_dependents();
  if (dbg && threadIdx.x == 0) p.debug[1] = globaltimer_ns();

  const int KB = p.K / BK;
  const int n_rows = GATHER ? checked_count(*p.count, p.m_total, p.status) : 0;
  // (PAIR: units = column tiles x pairs of row tiles; this CTA's row tile of unit u is 2 * (u / n_tiles) + pr, and
  // a row tile past the end of an odd count runs the main loop for its partner's sake and finishes no rows)
  const int m_tiles_live = GATHER ? (n_rows + BM - 1) / BM : p.m_tiles;
  int total_tiles = PAIR ? n_tiles * ((m_tiles_live + 1) / 2) : (GATHER ? m_tiles_live * n_tiles : total_tiles_dense);
  // A listed launch whose size only the device knows is issued in both forms; each looks at the count and one of them
  // leaves at once: pairs pay when there are enough units to keep every cluster busy for two rounds or more.
  if (GATHER && p.unit_gate > 0 && (n_tiles * ((m_tiles_live + 1) / 2) >= p.unit_gate) != PAIR) total_tiles = 0;
  // ... and in its listed and its dense form: the size of the refresh set decides which of the two runs
  if (p.gate_count != nullptr) {
    const int c = *p.gate_count;
    if (c < p.gate_lo || c >= p.gate_hi) total_tiles = 0;
  }
  auto tile_of = [&](int u) {
    if (!PAIR) return tile_geom(p, u, n_tiles, GATHER, n_rows);
    const int nt = u % n_tiles, mt = 2 * (u / n_tiles) + pr;
    if (GATHER) {                      // (the tile past an odd count has no rows: nothing stored)
      TileGeom t = tile_geom(p, mt * n_tiles + nt, n_tiles, true, n_rows);
      t.rows_valid = max(t.rows_valid, 0);
      return t;
    }
    TileGeom t = tile_geom(p, (mt < p.m_tiles ? mt : mt - 1) * n_tiles + nt, n_tiles, false, 0);
    if (mt >= p.m_tiles) t.rows_valid = 0;
    return t;
  };
  if (warp == 0) {
    // ---- producer
    uint32_t it = 0;
    for (int tile = walker; tile < total_tiles; tile += n_walkers) {
      const TileGeom t = tile_of(tile);
      const CUtensorMap* tm_b = t.is_b1 ? &tm_b1 : &tm_b0;
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % STAGES;
        mbar_wait(&empty_bar[s], ((it / STAGES) & 1) ^ 1, p.status);
        if (elect_one()) {
          uint8_t* dst = smem + s * STAGE_BYTES;
          if (PAIR) {
            // the bytes of both CTAs are counted on the even CTA's barrier; each brings its rows of A and its half
            // of the W tile's rows
            const uint32_t fb = map_to_cta(smem_u32(&full_bar[s]), 0);
            if (pr == 0) mbar_arrive_expect_tx(&full_bar[s], 2u * STAGE_BYTES);
            tma_load_2d_pair(dst, &tm_a, kb * BK, t.a_row, fb);
            tma_load_2d_pair(dst + A_BYTES, tm_b, kb * BK, t.n0 + pr * (BN / 2), fb);
          } else {
            mbar_arrive_expect_tx(&full_bar[s], (uint32_t)STAGE_BYTES);
            tma_load_2d(dst, &tm_a, kb * BK, t.a_row, &full_bar[s]);
            tma_load_2d(dst + A_BYTES, tm_b, kb * BK, t.n0, &full_bar[s]);
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1 && pr == 0) {
    // ---- MMA issuer (of a pair: the even CTA's)
    constexpr uint32_t idesc = idesc_bf16(PAIR ? 2 * BM : BM, BN);
    uint32_t it = 0, tcount = 0;
    for (int tile = walker; tile < total_tiles; tile += n_walkers, ++tcount) {
      const uint32_t buf = tcount & 1;
      mbar_wait(&acc_empty[buf], ((tcount >> 1) & 1) ^ 1, p.status);     // (passes at once the first two times)
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + buf * BN;
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % STAGES;
        mbar_wait(&full_bar[s], (it / STAGES) & 1, p.status);
        tc_fence_after();
        if (elect_one()) {
          const uint32_t a_addr = smem_u32(smem + s * STAGE_BYTES);
          const uint64_t a_desc = smem_desc_k_sw128(a_addr), b_desc = smem_desc_k_sw128(a_addr + A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if (PAIR) umma2_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            else umma_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          if (PAIR) {                      // the stage is free again, and the accumulator complete, in both CTAs
            umma2_commit(map_to_cta(smem_u32(&empty_bar[s]), 0));
            umma2_commit(map_to_cta(smem_u32(&empty_bar[s]), 1));
            if (kb == KB - 1) {
              umma2_commit(map_to_cta(smem_u32(&acc_full[buf]), 0));
              umma2_commit(map_to_cta(smem_u32(&acc_full[buf]), 1));
            }
          } else {
            umma_commit(&empty_bar[s]);
            if (kb == KB - 1) umma_commit(&acc_full[buf]);
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // (the odd CTA of a pair issues nothing)
  } else {
    // ---- finishing warps: quarter q of the TMEM lanes = rows 32q .. 32q + 31 of every tile
    const int q = warp & 3;
    uint8_t* stg = smem + STG_OFFSET + q * STG_WARP_BYTES;
    float* sc_acc = reinterpret_cast<float*>(smem + ACC_OFFSET) + q * 32 * 3;
    const uint32_t stg_w = smem_u32(stg) + (uint32_t)lane * STG_ROW_BYTES;    // this thread's row when it writes
    const int half_id = lane >> 4, l16 = lane & 15;
    uint32_t tcount = 0;
    for (int tile = walker; tile < total_tiles; tile += n_walkers, ++tcount) {
      const TileGeom t = tile_of(tile);
      const uint32_t buf = tcount & 1;
      mbar_wait(&acc_full[buf], (tcount >> 1) & 1, p.status);
      tc_fence_after();
      const uint32_t t_lane = tmem_base + buf * BN + ((uint32_t)(q * 32) << 16);
      // gathered rows: lane L holds the token of the warp's row L (-1 past the refresh set), lane-to-lane below
      int tok_own = -1, tok_first = 0;
      if (GATHER) {
        if (q * 32 + lane < t.rows_valid) {
          tok_own = p.idx[t.t0 + q * 32 + lane];
          if (!token_ok(tok_own, p.g.tokens(), p.status)) tok_own = -1;     // no row to write
        }
        tok_first = t.rows_valid > 0 ? p.idx[t.t0] : 0;  // a row that exists, for the table reads of rows that do not
        if ((unsigned)tok_first >= (unsigned)p.g.tokens()) tok_first = 0;
      }
      const bool rotate = (EPI == EPI_Q) || (EPI == EPI_KV && !t.is_b1);
      const int head0 = t.n0 / HD;
      const bool score_tile = (EPI == EPI_Q) && p.g.score_head >= head0 && p.g.score_head < head0 + BN / HD;
      __nv_bfloat16* out = t.is_b1 ? p.out1 : p.out0;
#pragma unroll 1
      for (int chunk = 0; chunk < 4; ++chunk) {
        const int hh = chunk >> 1, half = chunk & 1;
        const int c_lo = hh * HD + half * 32;            // tile columns [c_lo, c_lo + 32) and their partners + 64
        {
          float v[32];
          tmem_ld_32x32(t_lane + c_lo, v);
#pragma unroll
          for (int u = 0; u < 8; ++u)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg_w + (uint32_t)((u ^ (lane & 7)) << 4)),
                         "f"(v[4 * u]), "f"(v[4 * u + 1]), "f"(v[4 * u + 2]), "f"(v[4 * u + 3]) : "memory");
          tmem_ld_32x32(t_lane + c_lo + HD / 2, v);
#pragma unroll
          for (int u = 0; u < 8; ++u)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg_w + 128u + (uint32_t)((u ^ (lane & 7)) << 4)),
                         "f"(v[4 * u]), "f"(v[4 * u + 1]), "f"(v[4 * u + 2]), "f"(v[4 * u + 3]) : "memory");
        }
        if (chunk == 3) {                                // the accumulator is free for the tile after next
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[buf]), 0));   // (the issuing CTA's barrier)
            else mbar_arrive(&acc_empty[buf]);
          }
        }
        __syncwarp();
        const bool score_chunk = score_tile && head0 + hh == p.g.score_head;
        // 16 passes of two rows (one per half-warp), four passes at a time so that their table reads overlap
#pragma unroll 1
        for (int i0 = 0; i0 < 16; i0 += 4) {
          float2 lo[4], hi[4];
          float4 cs[4];
          float2 qa[4], qb[4];
          __nv_bfloat162 ra[4], rb[4];
          bool ok[4];
          int tok_k[4];
          size_t crow_k[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int rr = 2 * (i0 + k) + half_id, r = q * 32 + rr;
            ok[k] = r < t.rows_valid;
            const int rc = ok[k] ? r : 0;                // rows past the end read row 0's tables and are dropped
            int pos = t.pos0 + rc, tokr = t.t0 + rc;
            size_t crowr = t.crow0 + rc;
            if (GATHER) {
              const int tk = __shfl_sync(0xffffffffu, tok_own, rr);
              if (tk < 0) ok[k] = false;                 // (a token that failed its range check: the row is dropped)
              tokr = ok[k] ? tk : tok_first;
              pos = p.g.position(tokr);
              crowr = (size_t)p.g.cache_row(tokr);
            }
            tok_k[k] = tokr; crow_k[k] = crowr;
            if (!GATHER && EPI == EPI_KV && p.store_mask != nullptr && ok[k] && p.store_mask[crowr] != 0) ok[k] = false;
            const uint8_t* row = stg + rr * STG_ROW_BYTES;
            const uint32_t off = (uint32_t)((((l16 >> 1) ^ (rr & 7)) << 4) | ((l16 & 1) << 3));
            lo[k] = *reinterpret_cast<const float2*>(row + off);
            hi[k] = *reinterpret_cast<const float2*>(row + 128 + off);
            if (rotate)
              cs[k] = *reinterpret_cast<const float4*>(p.rope + (size_t)pos * (HD / 2) + half * 32 + 2 * l16);
            if (EPI == EPI_Q && score_chunk && p.has_prev) {
              const float* qp = p.q_prev + crowr * HD + half * 32 + 2 * l16;
              qa[k] = *reinterpret_cast<const float2*>(qp);
              qb[k] = *reinterpret_cast<const float2*>(qp + HD / 2);
            }
            if (EPI == EPI_OUT_RES) {
              const __nv_bfloat16* rs = p.resid + (size_t)tokr * p.ld_resid + t.n0 + c_lo + 2 * l16;
              ra[k] = *reinterpret_cast<const __nv_bfloat162*>(rs);
              rb[k] = *reinterpret_cast<const __nv_bfloat162*>(rs + HD / 2);
            }
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int rr = 2 * (i0 + k) + half_id, r = q * 32 + rr;
            const int tok = tok_k[k];
            const size_t crow = crow_k[k];
            float2 vlo = lo[k], vhi = hi[k];
            if (EPI == EPI_Q && score_chunk) {
              // Sec. 3.1 on the un-rotated query of the scoring head: 1 - cos(current, stored); this quarter of the
              // head adds its part of the three sums, the second half of the head finishes the row
              float dot = 0.f, n2 = 0.f;
              if (p.has_prev) {
                dot = vlo.x * qa[k].x + vlo.y * qa[k].y + vhi.x * qb[k].x + vhi.y * qb[k].y;
                n2 = qa[k].x * qa[k].x + qa[k].y * qa[k].y + qb[k].x * qb[k].x + qb[k].y * qb[k].y;
              }
              float n1 = vlo.x * vlo.x + vlo.y * vlo.y + vhi.x * vhi.x + vhi.y * vhi.y;
#pragma unroll
              for (int o = 8; o > 0; o >>= 1) {          // over the 16 lanes of the row
                dot += __shfl_xor_sync(0xffffffffu, dot, o);
                n1 += __shfl_xor_sync(0xffffffffu, n1, o);
                n2 += __shfl_xor_sync(0xffffffffu, n2, o);
              }
              if (ok[k]) {
                float* qp = p.q_prev + crow * HD + half * 32 + 2 * l16;
                *reinterpret_cast<float2*>(qp) = vlo;
                *reinterpret_cast<float2*>(qp + HD / 2) = vhi;
              }
              if (l16 == 0) {
                if (half == 0) {
                  sc_acc[3 * rr] = dot; sc_acc[3 * rr + 1] = n1; sc_acc[3 * rr + 2] = n2;
                } else if (ok[k]) {
                  dot += sc_acc[3 * rr]; n1 += sc_acc[3 * rr + 1]; n2 += sc_acc[3 * rr + 2];
                  float sc = __int_as_float(0x7f800000);   // +inf: nothing to compare with
                  if (p.has_prev) {
                    const float den = sqrtf(n1) * sqrtf(n2);
                    sc = 1.f - (den > 0.f ? dot / den : 0.f);
                  }
                  p.scores[tok] = sc;
                }
              }
            }
            if (!ok[k]) continue;
            if (rotate) {
              const float a0 = vlo.x, b0 = vhi.x, a1 = vlo.y, b1 = vhi.y;
              vlo.x = a0 * cs[k].x - b0 * cs[k].y; vhi.x = a0 * cs[k].y + b0 * cs[k].x;
              vlo.y = a1 * cs[k].z - b1 * cs[k].w; vhi.y = a1 * cs[k].w + b1 * cs[k].z;
            }
            if (EPI == EPI_OUT_RES) {
              const float2 fa = __bfloat1622float2(ra[k]), fb = __bfloat1622float2(rb[k]);
              vlo.x += fa.x; vlo.y += fa.y; vhi.x += fb.x; vhi.y += fb.y;
            }
            const size_t orow = p.out_is_cache == 1 ? crow : (p.out_is_cache == 2 ? (size_t)(t.t0 + r) : (size_t)tok);
            const __nv_bfloat162 o_lo = __floats2bfloat162_rn(vlo.x, vlo.y), o_hi = __floats2bfloat162_rn(vhi.x, vhi.y);
            __nv_bfloat16* dst = out + orow * p.ld_out + t.n0 + c_lo + 2 * l16;
            *reinterpret_cast<__nv_bfloat162*>(dst) = o_lo;
            *reinterpret_cast<__nv_bfloat162*>(dst + HD / 2) = o_hi;
            if ((EPI == EPI_OUT || EPI == EPI_OUT_RES) && p.out1 != nullptr) {   // the projected-output cache
              __nv_bfloat16* dst2 = p.out1 + crow * p.ld_out + t.n0 + c_lo + 2 * l16;
              *reinterpret_cast<__nv_bfloat162*>(dst2) = o_lo;
              *reinterpret_cast<__nv_bfloat162*>(dst2 + HD / 2) = o_hi;
            }
          }
        }
        __syncwarp();                                    // the staging rows are rewritten by the next quarter
      }
    }
  }
  tc_fence_before();
  // (a pair: nobody frees tensor memory or leaves while its partner's MMAs or barrier arrivals may still refer to it)
  if (PAIR) cluster_sync_relaxed(); else __syncthreads();
  if (p.debug != nullptr && threadIdx.x == 0) { atomicMax(&p.debug[6], globaltimer_ns()); atomicAdd(&p.debug[7], 1ull); }
  if (warp == 1) {
    if (PAIR) tmem_dealloc2(*tmem_slot, 512);
    else tmem_dealloc(tmem_base, 512);
  }
}

template <int EPI, bool GATHER, bool PAIR = false>
static cudaError_t launch_persist(const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1, const GemmParams& p,
                                  int n_tiles, int m_tiles, cudaStream_t st) {
  static std::atomic<unsigned long long> attr_done{0};
  auto kern = gemm_persist_kernel<EPI, GATHER, PAIR>;
  if (cudaError_t e = ensure_dyn_smem(kern, SMEM_TOTAL, attr_done); e != cudaSuccess) return e;
  int dev = 0, sms = 0;
  if (cudaError_t e = cudaGetDevice(&dev); e != cudaSuccess) return e;
  if (cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev); e != cudaSuccess) return e;
  const int total = n_tiles * m_tiles;
  GemmParams q = p;
  q.m_tiles = m_tiles;
  if (PAIR) {
    const int units = n_tiles * ((m_tiles + 1) / 2), clusters = units < sms / 2 ? units : sms / 2;
    return launch_pdl_xz(kern, dim3(2 * clusters), dim3(kWarps * 32), SMEM_TOTAL, st, 2, 1, a, b0, b1, q, n_tiles, total);
  }
  return launch_pdl(kern, dim3(total < sms ? total : sms), dim3(kWarps * 32), SMEM_TOTAL, st,
                    1, a, b0, b1, q, n_tiles, total);
}

// 256-wide tiles, no reduction split; b0 / b1 are maps with 256-row boxes (128-row boxes with pair != 0).  Listed
// launches (idx and count set, gather_src not; m_tiles = capacity of the row list in tiles): `a` maps a compact copy of
// the listed rows (row r of the list = row r of the copy).
cudaError_t launch_gemm_persist(int epi, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                                const GemmParams& p, int n_tiles, int m_tiles, cudaStream_t st, int pair) {
  if (m_tiles <= 0 || n_tiles <= 0) return cudaSuccess;
  if (p.b_pair || p.K % BK != 0) return cudaErrorInvalidValue;
  const bool listed = p.idx != nullptr, gather = p.gather_src != nullptr;
  if (listed != (p.count != nullptr) || (gather && !listed)) return cudaErrorInvalidValue;
  if (epi == EPI_OUT && p.resid != nullptr) epi = EPI_OUT_RES;
  if (gather) return cudaErrorInvalidValue;       // (rows fetched by index inside the kernel: gemm_tc.cu)
  if (listed) {          // A = compact copy of the listed rows
    if (pair) {
      if (epi == EPI_KV) return launch_persist<EPI_KV, true, true>(a, b0, b1, p, n_tiles, m_tiles, st);
      if (epi == EPI_OUT) return launch_persist<EPI_OUT, true, true>(a, b0, b1, p, n_tiles, m_tiles, st);
    } else {
      if (epi == EPI_KV) return launch_persist<EPI_KV, true, false>(a, b0, b1, p, n_tiles, m_tiles, st);
      if (epi == EPI_OUT) return launch_persist<EPI_OUT, true, false>(a, b0, b1, p, n_tiles, m_tiles, st);
    }
    return cudaErrorInvalidValue;
  }
  if (pair) {            // two-CTA MMAs: b0 / b1 are maps with 128-row boxes
    if (epi == EPI_Q) return launch_persist<EPI_Q, false, true>(a, b0, b1, p, n_tiles, m_tiles, st);
    if (epi == EPI_KV) return launch_persist<EPI_KV, false, true>(a, b0, b1, p, n_tiles, m_tiles, st);
    if (epi == EPI_OUT) return launch_persist<EPI_OUT, false, true>(a, b0, b1, p, n_tiles, m_tiles, st);
    if (epi == EPI_OUT_RES) return launch_persist<EPI_OUT_RES, false, true>(a, b0, b1, p, n_tiles, m_tiles, st);
    return cudaErrorInvalidValue;
  }
  if (epi == EPI_Q) return launch_persist<EPI_Q, false>(a, b0, b1, p, n_tiles, m_tiles, st);
  if (epi == EPI_KV) return launch_persist<EPI_KV, false>(a, b0, b1, p, n_tiles, m_tiles, st);
  if (epi == EPI_OUT) return launch_persist<EPI_OUT, false>(a, b0, b1, p, n_tiles, m_tiles, st);
  if (epi == EPI_OUT_RES) return launch_persist<EPI_OUT_RES, false>(a, b0, b1, p, n_tiles, m_tiles, st);
  return cudaErrorInvalidValue;
}

}  // namespace dare
