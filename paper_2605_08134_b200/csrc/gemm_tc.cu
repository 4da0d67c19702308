// bf16 projection GEMMs on the 5th-generation tensor cores: C[m, n] = sum_k A[m, k] * W[n, k]  (W = [out, in],
// Alg. 1 lines 2, 7, 11).  One CTA = one 128 x 256 output tile over one slice of the reduction dimension:
//   warp 0    TMA producer: a 128-row A tile and a 256-row W tile per 64 k-elements (128 bytes per row, 128-byte
//             swizzle) into a ring of 4 stages
//   warp 1    allocates tensor memory; one elected lane issues tcgen05.mma (M = 128, N = 256, K = 16) into a
//             128 x 256 fp32 accumulator and commits each stage back to the producer.  The tensor pipe runs at full
//             rate down to N = 128, but what an SM can pull from the L2 bounds the main loop of these projections,
//             and the widest tile re-reads the least per flop.
//   warps 2-7 wait for the accumulator (warps 2-5 are also the A-operand producers of a gathered launch); afterwards
//             all warps finish rows, and move the accumulator out of tensor memory first (thread <-> row; with eight
//             warps the two warps of a TMEM lane quarter take half of the columns each)
// Split-K: when a launch has too few tiles to fill the GPU, the two CTAs of a thread-block cluster share a tile, each
// over half of the reduction.  Every CTA first moves its fp32 accumulator from tensor memory into its own shared
// memory (the operand ring is idle by then).  The halves are then combined by a reduce-scatter over distributed
// shared memory: CTA k owns 64 rows of the tile and receives the partner's partial of those rows by one bulk copy
// per warp (32 KB, completion counted on an mbarrier of the receiver).  Each CTA finishes the rows it owns with all
// of its warps: one warp per row, lane <-> column pairs, so that table reads and output stores are contiguous.
// The fused epilogue work is thereby spread over both CTAs as well.
// Fused epilogues:
//   Q    drift score of the scoring head against the stored query (Sec. 3.1), store of the new query, rotary
//        embedding, bf16 store
//   K/V  rotary embedding of K, scatter of both rows into the caches at the refresh-set rows (Eq. 3)
//   OUT  bf16 store of y (OUT_RES: plus a residual row, read together with the row's tables)
//   SWIGLU  silu(gate) * up of a tile that holds both projections of the same 128 outputs (MLP of a stack)
//   F32  fp32 store (logits of a stack's LM head)
#include "layer.h"
#include "tc.h"
#include "tc_ptx.cuh"

namespace dare {

using namespace ptx;

namespace {
constexpr int BM = 128, BK = 64;
constexpr int A_BYTES = BM * BK * 2;
constexpr int HD = 128;                              // head width the rotary/score epilogues assume
// PAIR: two CTAs (row tiles 2i, 2i + 1 of the same column tile and reduction slice) share one M = 256 MMA; each
// keeps its own 128 rows of A and only half of the W tile's rows in shared memory: 32 KB instead of 48 KB per stage
// and CTA come through the L2, which is what bounds the main loop of the projections.
template <int BN, bool PAIR = false>
struct Cfg {
  static constexpr int B_BYTES = (PAIR ? BN / 2 : BN) * BK * 2;     // this CTA's part of the W tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (PAIR || BN != 256) ? 6 : 4;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int SMEM_TOTAL = BAR_OFFSET + 256 + 1024;  // barriers + slack for 1024-byte alignment
  static constexpr int PROW_BYTES = BN * 4;
  static constexpr int RECV_OFFSET = BM * PROW_BYTES;
};
// After the main loop the ring is reused: [0, 128 KB) this CTA's fp32 partial tile, [row][256 columns], 1 KB per row,
// the 16-byte units of a row XOR-swizzled with the row index (bank-conflict-free for row-per-thread writes and for
// row-per-warp reads); [128 KB, 192 KB) the partner's partial of the 64 rows this CTA owns (split-K only).
}  // namespace

// Finishing pass, per warp: RB rows at a time (rows rl0, rl0 + #warps, ...); their table reads are issued together.
// Warps of a CTA: producer, MMA issuer, the rest wait for the accumulator; all of them finish rows.
template <int BN>
struct Warps {
  static constexpr int N = 8;
  static constexpr int RB = 4;                       // rows a warp finishes at a time
};
template <int RB>
struct RowBatch {
  int tok[RB];
  int row[RB];            // place of the row in the launch's (possibly gathered) row list
  size_t crow[RB];
  bool ok[RB];
  float4 cs[RB];          // (cos, sin) of the two rotary pairs this lane owns
  float2 qa[RB], qb[RB];  // stored query of the scoring head: elements 2*lane.. and 64 + 2*lane..
  __nv_bfloat162 res[RB][2][2];   // residual row (output projection of a transformer block): this lane's pairs per head
};

template <int EPI, int RB, int kWarps, int BN>
__device__ __forceinline__ void load_row_batch(RowBatch<RB>& rb, const GemmParams& p, int rl0, int z, int rows_per_cta,
                                               int rows_valid, int t0, int pos0, size_t crow0, bool rotate,
                                               bool score_tile, int lane, int n0) {
#pragma unroll
  for (int k = 0; k < RB; ++k) {
    const int rl = rl0 + kWarps * k;
    const int r = z * rows_per_cta + rl;
    rb.ok[k] = rl < rows_per_cta && r < rows_valid;
    const int rc = rb.ok[k] ? r : 0;              // rows that do not exist read row 0's tables and are dropped later
    rb.row[k] = t0 + rc;
    int pos;
    if (p.idx) {
      rb.tok[k] = p.idx[t0 + rc];
      if (!token_ok(rb.tok[k], p.g.tokens(), p.status)) { rb.tok[k] = 0; rb.ok[k] = false; }   // no row to write
      pos = p.g.position(rb.tok[k]);
      rb.crow[k] = (size_t)p.g.cache_row(rb.tok[k]);
    } else {
      rb.tok[k] = t0 + rc;
      pos = pos0 + rc;
      rb.crow[k] = crow0 + rc;
    }
    // no instruction consumes these loads before the finishing pass, so they stay in flight across the exchange
    if (rotate) rb.cs[k] = *reinterpret_cast<const float4*>(p.rope + (size_t)pos * (HD / 2) + 2 * lane);
    if (EPI == EPI_Q && score_tile && p.has_prev) {
      rb.qa[k] = *reinterpret_cast<const float2*>(p.q_prev + rb.crow[k] * HD + 2 * lane);
      rb.qb[k] = *reinterpret_cast<const float2*>(p.q_prev + rb.crow[k] * HD + HD / 2 + 2 * lane);
    }
    if (EPI == EPI_OUT_RES) {
      const __nv_bfloat16* rs = p.resid + (size_t)rb.tok[k] * p.ld_resid + n0;
#pragma unroll
      for (int hh = 0; hh < BN / HD; ++hh) {
        rb.res[k][hh][0] = *reinterpret_cast<const __nv_bfloat162*>(rs + hh * HD + 2 * lane);
        rb.res[k][hh][1] = *reinterpret_cast<const __nv_bfloat162*>(rs + hh * HD + HD / 2 + 2 * lane);
      }
    }
  }
}

template <int EPI, int BN, bool PAIR>
__global__ void __launch_bounds__(Warps<BN>::N * 32, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
               const __grid_constant__ CUtensorMap tm_b1, const GemmParams p) {
  using C = Cfg<BN, PAIR>;
  constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES;
  constexpr int kWarps = Warps<BN>::N, RB = Warps<BN>::RB;
  constexpr int PROW_BYTES = C::PROW_BYTES, RECV_OFFSET = C::RECV_OFFSET;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + C::BAR_OFFSET);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* accum_bar = empty_bar + STAGES;
  uint64_t* recv_bar = accum_bar + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(recv_bar + 1);

  // the warp index through a shuffle: the compiler then knows the role decisions and the descriptors derived from
  // it to be uniform over the warp
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  // (a pair launch has the row tiles along x: the two CTAs of an MMA pair are neighbours in x)
  const int nt = (PAIR ? blockIdx.y : blockIdx.x) + p.nt0, mt_first = PAIR ? blockIdx.x : blockIdx.y;
  const int cl_splits = gridDim.z;              // = cluster size along z: slices of the reduction
  // cluster = (PAIR ? 2 : 1, 1, splits): rank = place in the MMA pair + 2 * reduction slice
  const int crank = (int)cluster_ctarank();
  const int pr = PAIR ? (crank & 1) : 0;        // place in the MMA pair; place 0 issues the MMAs
  const int cl_z = PAIR ? (crank >> 1) : crank; // this CTA's slice
  const uint32_t lead = (uint32_t)(crank & ~1); // cluster rank of the pair's issuing CTA
  auto rank_of_slice = [&](int zz) { return (uint32_t)(PAIR ? 2 * zz + pr : zz); };
  const bool dbg = p.debug != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && cl_z == 0;
  if (dbg && threadIdx.x == 0) p.debug[0] = globaltimer_ns();
  const int lin = (cl_z * (int)(PAIR ? gridDim.x : gridDim.y) + mt_first) * (int)(PAIR ? gridDim.y : gridDim.x) + nt;
  const bool rec = EPI == EPI_Q && p.debug != nullptr && lin < 1024;
  if (rec && threadIdx.x == 0) p.debug[64 + 3 * lin] = globaltimer_ns();

  // ---- which columns?  Tiles [0, n_split) belong to W0/out0, the rest to W1/out1.
  const bool is_b1 = !p.b_pair && nt >= p.n_split;
  const int n0 = p.b_pair ? nt * (BN / 2) : (is_b1 ? nt - p.n_split : nt) * BN;   // first output column / W row
  const CUtensorMap* tm_b = is_b1 ? &tm_b1 : &tm_b0;
  // ---- which slice of the reduction?
  // (a CTA walks the k-blocks from the start of its slice on, modulo KB: its slice when the tile's reduction is
  // split, all of them when it is not)
  const int KB = p.K / BK;
  const int kb0 = (int)(((long long)KB * cl_z) / cl_splits);
  auto kb_of = [&](int i) { const int k = kb0 + i; return k >= KB ? k - KB : k; };
  int tiles_done = 0;                           // (p.loop_rows) row tiles of the refresh set behind this cluster

  // A gathered launch of few row tiles (p.loop_rows) has one row of the grid: its CTAs take the row tiles of the
  // refresh set one after the other, setting their barriers up again for each (the refresh set is small, one tile
  // as a rule; a grid with a row of CTAs per possible tile would send hundreds of CTAs through the SMs this launch
  // leaves free only to look at the count and leave, and the next kernel cannot start before the last of them has).
  for (int iter = 0;; ++iter) {
  int mt = mt_first + iter;
  int splits = cl_splits, z = cl_z, tile_step = 1;   // (settled below, once the size of the refresh set is known)
  // Row tiles past the first one of a gathered launch are usually empty (the refresh set is small): they look at
  // the count before spending anything on set-up.  The others set up first and wait for the previous kernel later.
  const bool likely = p.count == nullptr || mt == 0 || iter > 0;
  if (!likely) {
    pdl_wait();
    if (mt * BM >= checked_count(*p.count, p.m_total, p.status)) return;     // uniform over the cluster
  }
  // Gathered A operand: the four epilogue warps fetch the rows of the refresh set themselves, 16 bytes at a time,
  // into the swizzled tile layout (the TMA producer then only brings the W tiles); each of them arrives on a stage
  // once its rows of that stage have landed.
  const bool gather = p.gather_src != nullptr;
  const uint32_t tx_bytes = gather ? (uint32_t)C::B_BYTES : (uint32_t)STAGE_BYTES;
  if (threadIdx.x == 0) {
    if (iter > 0) {                              // (every CTA of the cluster is past the previous tile: nothing is in flight)
      for (int s = 0; s < STAGES; ++s) { mbar_inval(&full_bar[s]); mbar_inval(&empty_bar[s]); }
      mbar_inval(accum_bar);
      mbar_inval(recv_bar);
    }
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], gather ? 5 : 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(accum_bar, 1);
    mbar_init(recv_bar, 1);
    fence_mbar_init();
    if (cl_splits > 1) mbar_arrive_expect_tx(recv_bar, (uint32_t)(BM / 2) * PROW_BYTES);   // the partner's 64 rows (if split)
    prefetch_tmap(&tm_a);
    prefetch_tmap(tm_b);
  }
  if (warp == 1 && iter == 0) {
    if (PAIR) { tmem_alloc2(tmem_slot, BN); tmem_relinquish2(); }
    else { tmem_alloc(tmem_slot, BN); tmem_relinquish(); }
  }
  tc_fence_before();
  __syncthreads();
  uint32_t tmem_base;
  if (PAIR) {
    // both CTAs of the pair have their barriers and their tensor memory before either touches the other's
    cluster_sync_all();
    tc_fence_after();
    tmem_base = ld_cluster_u32(map_to_cta(smem_u32(tmem_slot), lead));
  } else {
    tc_fence_after();
    tmem_base = *tmem_slot;
  }
  // The weights do not depend on the previous kernel in the stream: the producer starts their first tiles now, so
  // that they stream in while that kernel drains.  Everything it produced is needed only after pdl_wait().
  const int n_early = likely && iter == 0 ? (KB / cl_splits < STAGES ? KB / cl_splits : STAGES) : 0;
  if (warp == 0 && lane == 0) {
    for (int i = 0; i < n_early; ++i) {
      uint8_t* b_dst = smem + i * STAGE_BYTES + A_BYTES;
      if (PAIR) {
        // the bytes of both CTAs are counted on the issuing CTA's barrier; each CTA brings its half of the W rows
        // (a tile of two matrices: the even CTA brings the rows of the first, the odd one those of the second)
        if (pr == 0) mbar_arrive_expect_tx(&full_bar[i], 2 * STAGE_BYTES);
        tma_load_2d_pair(b_dst, p.b_pair ? (pr == 0 ? &tm_b0 : &tm_b1) : tm_b, kb_of(i) * BK,
                         p.b_pair ? n0 : n0 + pr * (BN / 2), map_to_cta(smem_u32(&full_bar[i]), lead));
        continue;
      }
      mbar_arrive_expect_tx(&full_bar[i], tx_bytes);
      if (p.b_pair) {
        tma_load_2d(b_dst, &tm_b0, kb_of(i) * BK, n0, &full_bar[i]);
        tma_load_2d(b_dst + C::B_BYTES / 2, &tm_b1, kb_of(i) * BK, n0, &full_bar[i]);
      } else {
        tma_load_2d(b_dst, tm_b, kb_of(i) * BK, n0, &full_bar[i]);
      }
    }
  }
  if (!p.wait_at_end) pdl_wait();
  pdl_launch_dependents();
  if (dbg && threadIdx.x == 0) p.debug[1] = globaltimer_ns();

  // ---- which rows does this tile cover? (uniform over the cluster; a tile past the refresh set has nothing to do)
  int a_row = 0, t0 = 0, rows_valid = 0;
  int pos0 = 0;          // dense tiles: position and cache row of the tile's first row
  size_t crow0 = 0;
  bool active = true;
  if (p.count != nullptr) {
    const int n = checked_count(*p.count, p.m_total, p.status);
    if (p.loop_rows) {
      // The cluster's two CTAs share one row tile (half of the reduction each, partial tiles exchanged) while there is
      // only one left; with two or more left each takes a row tile of its own over the whole reduction: one pass
      // over the weights for two tiles instead of two, and nothing to exchange.
      const int tiles_left = (n + BM - 1) / BM - tiles_done;
      if (!PAIR && cl_splits == 2 && tiles_left >= 2) { mt = tiles_done + cl_z; splits = 1; z = 0; tile_step = 2; }
      else mt = tiles_done;
    }
    t0 = mt * BM;
    active = t0 < n;
    rows_valid = min(BM, n - t0);
    a_row = t0;
  } else {
    // (a pair launch pads the row tiles to an even number: the tile past the end runs the main loop for its
    // partner's sake, on the first tile's rows, and finishes no rows)
    const bool exists = mt < p.m_tiles;
    const int mte = exists ? mt : 0;
    const int b = mte / p.tiles_per_seq, tis = mte - b * p.tiles_per_seq;
    t0 = b * p.seq_act + tis * BM;
    rows_valid = exists ? min(BM, p.seq_act - tis * BM) : 0;
    a_row = b * p.a_seq_stride + p.a_row0 + tis * BM;
    pos0 = p.g.pos_begin + tis * BM;
    crow0 = (size_t)b * p.g.max_seq + pos0;
  }

  // epilogue geometry
  const int rows_per_cta = BM / splits;           // rows of the tile this CTA finishes
  const int nkb = KB / splits;                    // k-blocks this CTA walks for the tile
  const int quarter = warp & 3;                   // TMEM lanes a warp may touch: 32*quarter .. +31
  const bool rotate = (EPI == EPI_Q) || (EPI == EPI_KV && !is_b1);
  const int head0 = n0 / HD;
  const bool score_tile = (EPI == EPI_Q) && p.g.score_head >= head0 && p.g.score_head < head0 + BN / HD;
  RowBatch<RB> rb;

  if (active) {
  // The producer and the MMA warp run their loops converged (every lane polls the barriers) and one elected lane
  // issues: the operands of the copies and MMAs are then warp-uniform values, which is what those instructions take.
  if (warp == 0) {
    if (!gather && elect_one()) {
      for (int i = 0; i < n_early; ++i) {        // the W halves of these stages are already on their way
        if (PAIR)
          tma_load_2d_pair(smem + i * STAGE_BYTES, &tm_a, kb_of(i) * BK, a_row, map_to_cta(smem_u32(&full_bar[i]), lead));
        else
          tma_load_2d(smem + i * STAGE_BYTES, &tm_a, kb_of(i) * BK, a_row, &full_bar[i]);
      }
    }
    __syncwarp();
    for (int i = n_early; i < nkb; ++i) {
      const int s = i % STAGES;
      mbar_wait(&empty_bar[s], ((i / STAGES) & 1) ^ 1, p.status);
      if (elect_one()) {
        uint8_t* a_dst = smem + s * STAGE_BYTES;
        if (PAIR) {
          const uint32_t fb = map_to_cta(smem_u32(&full_bar[s]), lead);
          if (pr == 0) mbar_arrive_expect_tx(&full_bar[s], 2 * STAGE_BYTES);
          tma_load_2d_pair(a_dst, &tm_a, kb_of(i) * BK, a_row, fb);
          tma_load_2d_pair(a_dst + A_BYTES, p.b_pair ? (pr == 0 ? &tm_b0 : &tm_b1) : tm_b, kb_of(i) * BK,
                           p.b_pair ? n0 : n0 + pr * (BN / 2), fb);
        } else {
          mbar_arrive_expect_tx(&full_bar[s], tx_bytes);
          if (!gather) tma_load_2d(a_dst, &tm_a, kb_of(i) * BK, a_row, &full_bar[s]);
          if (p.b_pair) {
            tma_load_2d(a_dst + A_BYTES, &tm_b0, kb_of(i) * BK, n0, &full_bar[s]);
            tma_load_2d(a_dst + A_BYTES + C::B_BYTES / 2, &tm_b1, kb_of(i) * BK, n0, &full_bar[s]);
          } else {
            tma_load_2d(a_dst + A_BYTES, tm_b, kb_of(i) * BK, n0, &full_bar[s]);
          }
        }
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    if (!PAIR || pr == 0) {
      // (in a pair only the even-ranked CTA issues: one M = 256 MMA covers both CTAs' rows)
      constexpr uint32_t idesc = idesc_bf16(PAIR ? 2 * BM : BM, BN);
      for (int i = 0; i < nkb; ++i) {
        const int s = i % STAGES;
        mbar_wait(&full_bar[s], (i / STAGES) & 1, p.status);
        tc_fence_after();
        if (dbg && i == 0 && lane == 0) p.debug[2] = globaltimer_ns();
        if (elect_one()) {
          const uint32_t a_addr = smem_u32(smem + s * STAGE_BYTES);
          const uint64_t a_desc = smem_desc_k_sw128(a_addr);
          const uint64_t b_desc = smem_desc_k_sw128(a_addr + A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {  // 16 k-elements = 32 bytes = 2 descriptor address units per MMA
            if (PAIR) umma2_ss(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, (i | k) != 0 ? 1u : 0u);
            else umma_ss(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, (i | k) != 0 ? 1u : 0u);
          }
          // the stage is free again, in both CTAs of a pair; after the last one the accumulators are complete
          if (PAIR) {
            umma2_commit(map_to_cta(smem_u32(&empty_bar[s]), lead));
            umma2_commit(map_to_cta(smem_u32(&empty_bar[s]), lead + 1));
            if (i == nkb - 1) {
              umma2_commit(map_to_cta(smem_u32(accum_bar), lead));
              umma2_commit(map_to_cta(smem_u32(accum_bar), lead + 1));
            }
          } else {
            umma_commit(&empty_bar[s]);
            if (i == nkb - 1) umma_commit(accum_bar);      // by the thread that issued the MMAs it covers
          }
        }
        __syncwarp();
      }
    }
  } else {
    // While the main loop runs, pull the table rows the finishing pass of this CTA will read into the L2
    // (dense tiles; 512 bytes = 4 lines per row and table).
    if (p.idx == nullptr) {
      for (int i = threadIdx.x - 64; i < rows_per_cta * 4; i += (kWarps - 2) * 32) {
        const int r = z * rows_per_cta + (i >> 2);
        if (r >= rows_valid) break;
        if (rotate) prefetch_l2(p.rope + (size_t)(pos0 + r) * (HD / 2) + (i & 3) * 16);
        if (score_tile && p.has_prev) prefetch_l2(p.q_prev + (crow0 + r) * HD + (i & 3) * 32);
      }
    }
    // the table reads of this warp's first rows of the finishing pass: in flight for the whole main loop
    // (a gathering warp asks for its rows' tokens before the table reads below stall on theirs: one round trip, not two)
    const int r_own = quarter * 32 + lane;                     // the row whose token this lane looks up
    int tok_own = -1;
    if (gather && warp < 6 && r_own < rows_valid) {
      tok_own = p.idx[t0 + r_own];
      if (!token_ok(tok_own, p.g.tokens(), p.status)) tok_own = -1;      // read as a row of zeros
    }
    load_row_batch<EPI, RB, kWarps, BN>(rb, p, warp, z, rows_per_cta, rows_valid, t0, pos0, crow0, rotate, score_tile, lane, n0);
    if (gather && warp < 6) {
      // One stage of the A tile = 128 rows x 128 bytes (64 k-elements).  A warp takes 32 rows; one of its copy
      // instructions covers four rows, eight consecutive lanes fetching the eight 16-byte units of a row, so every
      // request is a whole 128-byte line.
      const uint8_t* src_k[8];
      uint32_t dst_k[8], bytes_k[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int rw = k * 4 + (lane >> 3), r = quarter * 32 + rw, u = lane & 7;
        const int tok = __shfl_sync(0xffffffffu, tok_own, rw);
        const int srow = tok < 0 ? 0 : (p.gather_cache_rows ? p.g.cache_row(tok) : tok);
        src_k[k] = reinterpret_cast<const uint8_t*>(p.gather_src) + (size_t)srow * p.K * 2 +
                   u * 16;
        bytes_k[k] = tok >= 0 ? 16u : 0u;                       // rows past the refresh set are zero-filled
        dst_k[k] = smem_u32(smem) + (uint32_t)r * 128u + (uint32_t)((u ^ (r & 7)) << 4);
      }
      constexpr int LAG = STAGES - 2;                           // copy groups in flight per thread
      uint32_t koff = (uint32_t)kb0 * (BK * 2);                 // byte offset of k-block kb_of(i) in a row
      const uint32_t kwrap = (uint32_t)KB * (BK * 2);
      for (int i = 0; i < nkb + LAG; ++i) {
        if (i < nkb) {
          const int s = i % STAGES;
          mbar_wait(&empty_bar[s], ((i / STAGES) & 1) ^ 1, p.status);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            cp_async_16(dst_k[k] + (uint32_t)s * STAGE_BYTES, src_k[k] + koff, bytes_k[k]);
          koff += BK * 2;
          if (koff == kwrap) koff = 0;
        }
        cp_async_commit();                                      // (empty groups at the tail keep the lag uniform)
        if (i >= LAG) {
          cp_async_wait<LAG>();                                 // this thread's copies of stage i - LAG have landed
          fence_proxy_async_smem();                             // ... and are visible to the tensor core's reads
          __syncwarp();
          if (lane == 0) mbar_arrive(&full_bar[(i - LAG) % STAGES]);
        }
      }
    }
    mbar_wait(accum_bar, 0, p.status);
    tc_fence_after();
    if (dbg && threadIdx.x == 64) p.debug[3] = globaltimer_ns();
    if (rec && threadIdx.x == 64) p.debug[64 + 3 * lin + 1] = globaltimer_ns();
  }

  // The table reads of the first rows the producer and MMA warps will finish start now (those of the other warps
  // started before the main loop) and land during the exchange below.
  if (warp < 2) load_row_batch<EPI, RB, kWarps, BN>(rb, p, warp, z, rows_per_cta, rows_valid, t0, pos0, crow0, rotate, score_tile, lane, n0);

  // ---- every CTA of the cluster has finished its main loop: the rings are free to receive partial rows
  tc_fence_before();
  if (splits > 1) cluster_sync_relaxed(); else __syncthreads();
  tc_fence_after();
  if (dbg && EPI == EPI_Q && threadIdx.x == 64) p.debug[32] = globaltimer_ns();
  {
    // The partial accumulator: tensor memory -> own shared memory, thread <-> row.  With eight warps the two warps
    // of a lane quarter (w and w + 4) take half of the columns each.
    const int r = quarter * 32 + lane;
    // Layout of the partial tile in shared memory: [32-column chunk][row][128 bytes], the eight 16-byte units of a
    // row's chunk XOR-swizzled by the row (thread <-> row stores of one unit would otherwise hit the same banks).
    // The 32 rows a warp holds of one chunk are 4 KB in one piece: rows owned by the partner leave chunk by chunk,
    // as soon as the warp has written them, so that the copies overlap the rest of the read-out.
    const uint32_t dst = smem_u32(smem) + (uint32_t)r * 128u;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    static_assert(kWarps == 8, "two warps per lane quarter share the columns");
    constexpr int ch_n = BN / 64;
    const int ch0 = (warp >> 2) * ch_n;
    const int owner = r / rows_per_cta;                              // (uniform over the warp: 32 | rows_per_cta)
    const bool send = splits > 1 && owner != z;
    const int rl0 = quarter * 32 - owner * rows_per_cta;
    const uint32_t rbar = send ? map_to_cta(smem_u32(recv_bar), rank_of_slice(owner)) : 0u;
    const uint32_t rbase = send ? map_to_cta(smem_u32(smem + RECV_OFFSET), rank_of_slice(owner)) : 0u;
    // (the next chunk's tensor-memory load is in flight while this chunk is written and sent)
    float va[32], vb[32];
    tmem_ld_32x32_nowait(t_lane + ch0 * 32, va);
#pragma unroll
    for (int c2 = 0; c2 < ch_n; ++c2) {
      const int ch = ch0 + c2;
      float* v = (c2 & 1) ? vb : va;
      tmem_ld_wait();
      if (c2 + 1 < ch_n) tmem_ld_32x32_nowait(t_lane + (ch + 1) * 32, (c2 & 1) ? va : vb);
      const uint32_t cdst = dst + (uint32_t)ch * (uint32_t)(BM * 128);
#pragma unroll
      for (int g4 = 0; g4 < 8; ++g4)
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cdst + (uint32_t)((g4 ^ (r & 7)) << 4)),
                     "f"(v[4 * g4]), "f"(v[4 * g4 + 1]), "f"(v[4 * g4 + 2]), "f"(v[4 * g4 + 3]) : "memory");
      if (send) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0)
          bulk_copy_to_cta(rbase + (uint32_t)ch * (uint32_t)((BM / 2) * 128) + (uint32_t)rl0 * 128u,
                           smem_u32(smem) + (uint32_t)ch * (uint32_t)(BM * 128) + (uint32_t)(quarter * 32) * 128u, 32 * 128, rbar);
      }
    }
  }
  if (dbg && EPI == EPI_Q && threadIdx.x == 64) p.debug[33] = globaltimer_ns();
  __syncthreads();
  if (splits > 1) mbar_wait(recv_bar, 0, p.status);     // the partner's rows have landed
  if (dbg && threadIdx.x == 64) p.debug[4] = globaltimer_ns();

  // ---- finish the owned rows: one warp per row, lane <-> pairs (2*lane, 2*lane+1) of each head of the tile.
  // Rows are taken four at a time so that their table reads are in flight together.
  {
    __nv_bfloat16* out = is_b1 ? p.out1 : p.out0;
#pragma unroll 1
    for (int rl0 = warp; rl0 < rows_per_cta; rl0 += kWarps * RB) {
      if (rl0 != warp) load_row_batch<EPI, RB, kWarps, BN>(rb, p, rl0, z, rows_per_cta, rows_valid, t0, pos0, crow0, rotate, score_tile, lane, n0);
      if (dbg && EPI == EPI_Q && threadIdx.x == 64) p.debug[34 + (rl0 - warp) / (kWarps * RB) * 2] = globaltimer_ns();
      // (1) combine the partial rows: lane <-> pairs (2*lane, 2*lane+1) of each head
      float2 vlo[RB][BN / HD], vhi[RB][BN / HD];
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int rl = rb.ok[k] ? rl0 + kWarps * k : warp;     // rows that do not exist re-read an existing one
#pragma unroll
        for (int hh = 0; hh < BN / HD; ++hh) {
          const int c_lo = hh * HD + 2 * lane, c_hi = c_lo + HD / 2;
          // (unit of the column inside its 32-column chunk, swizzled by the row; rows_per_cta is a multiple of 8)
          const uint32_t in_lo = (uint32_t)(((((c_lo >> 2) & 7) ^ (rl & 7)) << 4) | ((c_lo & 3) << 2));
          const uint32_t in_hi = (uint32_t)(((((c_hi >> 2) & 7) ^ (rl & 7)) << 4) | ((c_hi & 3) << 2));
          const uint8_t* mine = smem + (size_t)(z * rows_per_cta + rl) * 128;             // this CTA's partial
          float2 lo = *reinterpret_cast<const float2*>(mine + (size_t)(c_lo >> 5) * (BM * 128) + in_lo);
          float2 hi = *reinterpret_cast<const float2*>(mine + (size_t)(c_hi >> 5) * (BM * 128) + in_hi);
          if (splits > 1) {
            const uint8_t* theirs = smem + RECV_OFFSET + (size_t)rl * 128;                // the partner's partial
            const float2 a = *reinterpret_cast<const float2*>(theirs + (size_t)(c_lo >> 5) * ((BM / 2) * 128) + in_lo);
            const float2 b = *reinterpret_cast<const float2*>(theirs + (size_t)(c_hi >> 5) * ((BM / 2) * 128) + in_hi);
            lo.x += a.x; lo.y += a.y; hi.x += b.x; hi.y += b.y;
          }
          vlo[k][hh] = lo; vhi[k][hh] = hi;
        }
      }
      // (2) Sec. 3.1 on the un-rotated query of the scoring head: 1 - cos(current, stored), all rows of the batch
      //     reduced across the lanes together; lane k finishes row k.  Then the current query is stored.
      if (EPI == EPI_Q && score_tile) {
        float dot[RB], n1[RB], n2[RB];
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          float2 lo = vlo[k][0], hi = vhi[k][0];
#pragma unroll
          for (int hh = 1; hh < BN / HD; ++hh)
            if (head0 + hh == p.g.score_head) { lo = vlo[k][hh]; hi = vhi[k][hh]; }
          const float2 a = rb.qa[k], b = rb.qb[k];
          dot[k] = lo.x * a.x + lo.y * a.y + hi.x * b.x + hi.y * b.y;
          n1[k] = lo.x * lo.x + lo.y * lo.y + hi.x * hi.x + hi.y * hi.y;
          n2[k] = a.x * a.x + a.y * a.y + b.x * b.x + b.y * b.y;
          if (rb.ok[k]) {
            float* qp = p.q_prev + rb.crow[k] * HD;
            *reinterpret_cast<float2*>(qp + 2 * lane) = lo;
            *reinterpret_cast<float2*>(qp + HD / 2 + 2 * lane) = hi;
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
          for (int k = 0; k < RB; ++k) {
            dot[k] += __shfl_xor_sync(0xffffffffu, dot[k], o);
            n1[k] += __shfl_xor_sync(0xffffffffu, n1[k], o);
            n2[k] += __shfl_xor_sync(0xffffffffu, n2[k], o);
          }
        }
        float my_dot = 0.f, my_n1 = 0.f, my_n2 = 0.f;
        int my_tok = -1;
#pragma unroll
        for (int k = 0; k < RB; ++k)
          if (lane == k) { my_dot = dot[k]; my_n1 = n1[k]; my_n2 = n2[k]; my_tok = rb.ok[k] ? rb.tok[k] : -1; }
        if (my_tok >= 0) {
          float sc = __int_as_float(0x7f800000);   // +inf: nothing to compare with
          if (p.has_prev) {
            const float den = sqrtf(my_n1) * sqrtf(my_n2);
            sc = 1.f - (den > 0.f ? my_dot / den : 0.f);
          }
          p.scores[my_tok] = sc;
        }
      }
      // (3) the projection's own tail and the store
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        if (!rb.ok[k]) continue;
        const size_t orow = p.out_is_cache == 1 ? rb.crow[k] : (p.out_is_cache == 2 ? (size_t)rb.row[k] : (size_t)rb.tok[k]);
        if (EPI == EPI_SWIGLU) {
          // columns [0, 128) of a 256-wide tile are the gate, [128, 256) the up projection of the same 128 outputs
          const float2 g_lo = vlo[k][0], g_hi = vhi[k][0], u_lo = vlo[k][BN / HD - 1], u_hi = vhi[k][BN / HD - 1];
          __nv_bfloat16* dst = out + orow * p.ld_out + n0;
          auto act = [](float g, float u) { return g / (1.f + __expf(-g)) * u; };
          *reinterpret_cast<__nv_bfloat162*>(dst + 2 * lane) = __floats2bfloat162_rn(act(g_lo.x, u_lo.x), act(g_lo.y, u_lo.y));
          *reinterpret_cast<__nv_bfloat162*>(dst + HD / 2 + 2 * lane) =
              __floats2bfloat162_rn(act(g_hi.x, u_hi.x), act(g_hi.y, u_hi.y));
          continue;
        }
        __nv_bfloat16* dst = out + orow * p.ld_out + n0;
#pragma unroll
        for (int hh = 0; hh < BN / HD; ++hh) {
          float2 lo = vlo[k][hh], hi = vhi[k][hh];
          const int c_lo = hh * HD + 2 * lane, c_hi = c_lo + HD / 2;
          if (rotate) {
            const float a0 = lo.x, b0 = hi.x, a1 = lo.y, b1 = hi.y;
            lo.x = a0 * rb.cs[k].x - b0 * rb.cs[k].y; hi.x = a0 * rb.cs[k].y + b0 * rb.cs[k].x;
            lo.y = a1 * rb.cs[k].z - b1 * rb.cs[k].w; hi.y = a1 * rb.cs[k].w + b1 * rb.cs[k].z;
          }
          if (EPI == EPI_F32) {
            float* d32 = p.out_f32 + orow * p.ld_out + n0;
            *reinterpret_cast<float2*>(d32 + c_lo) = lo;
            *reinterpret_cast<float2*>(d32 + c_hi) = hi;
            continue;
          }
          if (EPI == EPI_OUT_RES) {                                  // (read with the row's tables, long before)
            const float2 ra = __bfloat1622float2(rb.res[k][hh][0]), rb2 = __bfloat1622float2(rb.res[k][hh][1]);
            lo.x += ra.x; lo.y += ra.y; hi.x += rb2.x; hi.y += rb2.y;
          }
          const __nv_bfloat162 o_lo = __floats2bfloat162_rn(lo.x, lo.y), o_hi = __floats2bfloat162_rn(hi.x, hi.y);
          *reinterpret_cast<__nv_bfloat162*>(dst + c_lo) = o_lo;
          *reinterpret_cast<__nv_bfloat162*>(dst + c_hi) = o_hi;
          if ((EPI == EPI_OUT || EPI == EPI_OUT_RES) && p.out1 != nullptr) {       // second copy, by cache row: the projected-output cache
            __nv_bfloat16* dst2 = p.out1 + rb.crow[k] * p.ld_out + n0;
            *reinterpret_cast<__nv_bfloat162*>(dst2 + c_lo) = o_lo;
            *reinterpret_cast<__nv_bfloat162*>(dst2 + c_hi) = o_hi;
          }
        }
      }
      if (dbg && EPI == EPI_Q && threadIdx.x == 64) p.debug[35 + (rl0 - warp) / (kWarps * RB) * 2] = globaltimer_ns();
    }
  }
  if (dbg && threadIdx.x == 64) p.debug[5] = globaltimer_ns();
  } else if (warp == 0 && lane == 0) {
    // a tile past the refresh set: complete the stages whose W halves were started early, then let them land
    if (!gather) {
      for (int i = 0; i < n_early; ++i) tma_load_2d(smem + i * STAGE_BYTES, &tm_a, kb_of(i) * BK, 0, &full_bar[i]);
      for (int i = 0; i < n_early; ++i) mbar_wait(&full_bar[i], 0, p.status);
    } else {
      // the barrier also counts the four gathering warps, which do not run here: stand in for them
      for (int i = 0; i < n_early; ++i) {
        for (int k = 0; k < 4; ++k) mbar_arrive(&full_bar[i]);
        mbar_wait(&full_bar[i], 0, p.status);
      }
    }
  }
  tc_fence_before();
  // a launch that ran beside its predecessor leaves only once that one is complete: the next kernel's wait on this
  // grid then covers both
  if (p.wait_at_end) pdl_wait();
  // nobody leaves while a copy out of its shared memory may still be in flight (the partner has seen it land)
  // (nor frees tensor memory its MMA partner may still read through)
  if (splits > 1 || PAIR) cluster_sync_relaxed(); else __syncthreads();
  if (p.debug != nullptr && threadIdx.x == 0) { atomicMax(&p.debug[6], globaltimer_ns()); atomicAdd(&p.debug[7], 1ull); }
  if (rec && threadIdx.x == 0) p.debug[64 + 3 * lin + 2] = globaltimer_ns();
  if (!p.loop_rows || p.count == nullptr) break;
  tiles_done += tile_step;
  if (tiles_done * BM >= checked_count(*p.count, p.m_total, p.status)) break;    // uniform over the cluster
  }  // row tiles
  if (warp == 1) {
    if (PAIR) tmem_dealloc2(*tmem_slot, BN);
    else tmem_dealloc(*tmem_slot, BN);
  }
}

template <int EPI, int BN, bool PAIR>
static cudaError_t launch_one(const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1, const GemmParams& p,
                              int n_tiles, int m_tiles, int splits, cudaStream_t st) {
  static std::atomic<unsigned long long> attr_done{0};
  auto kern = gemm_tc_kernel<EPI, BN, PAIR>;
  constexpr int SMEM_TOTAL = Cfg<BN, PAIR>::SMEM_TOTAL;
  if (cudaError_t e = ensure_dyn_smem(kern, SMEM_TOTAL, attr_done); e != cudaSuccess) return e;
  GemmParams q = p;
  q.m_tiles = m_tiles;
  if (PAIR)
    return launch_pdl_xz(kern, dim3((m_tiles + 1) / 2 * 2, n_tiles, splits), dim3(Warps<BN>::N * 32), SMEM_TOTAL, st, 2,
                         splits, a, b0, b1, q);
  return launch_pdl_xz(kern, dim3(n_tiles, m_tiles, splits), dim3(Warps<BN>::N * 32), SMEM_TOTAL, st, 1, splits, a, b0, b1,
                       q);
}

// pair != 0: the launch uses two-CTA MMAs (256-wide tiles, A through the tensor map); b0 / b1 must then be maps with
// 128-row boxes.
cudaError_t launch_gemm_tc(int epi, int bn, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                           const GemmParams& p, int n_tiles, int m_tiles, int splits, cudaStream_t st, int pair) {
  if (m_tiles <= 0 || n_tiles <= 0) return cudaSuccess;
  if (epi == EPI_OUT && p.resid != nullptr) epi = EPI_OUT_RES;
  if ((splits != 1 && splits != 2) || splits > p.K / BK) return cudaErrorInvalidValue;
  if (pair && bn == 128) {
    // narrow pair tiles (256 rows x 128 columns per pair; b0 / b1 with 64-row boxes): twice the CTAs of the wide ones
    // for launches of two row tiles, whose main loops are bound by what one SM can pull from the L2
    if (p.gather_src != nullptr || p.count != nullptr || p.b_pair) return cudaErrorInvalidValue;
    if (epi == EPI_Q) return launch_one<EPI_Q, 128, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_OUT) return launch_one<EPI_OUT, 128, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_OUT_RES) return launch_one<EPI_OUT_RES, 128, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    return cudaErrorInvalidValue;
  }
  if (pair) {
    if (bn != 256 || p.gather_src != nullptr || p.count != nullptr || (p.b_pair != 0) != (epi == EPI_SWIGLU))
      return cudaErrorInvalidValue;
    if (epi == EPI_SWIGLU) return launch_one<EPI_SWIGLU, 256, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_Q) return launch_one<EPI_Q, 256, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_KV) return launch_one<EPI_KV, 256, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_OUT) return launch_one<EPI_OUT, 256, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_OUT_RES) return launch_one<EPI_OUT_RES, 256, true>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    return cudaErrorInvalidValue;
  }
  if (bn == 256) {
    if (epi == EPI_Q) return launch_one<EPI_Q, 256, false>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_KV) return launch_one<EPI_KV, 256, false>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_SWIGLU) return launch_one<EPI_SWIGLU, 256, false>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_F32) return launch_one<EPI_F32, 256, false>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    if (epi == EPI_OUT_RES) return launch_one<EPI_OUT_RES, 256, false>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
    return launch_one<EPI_OUT, 256, false>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
  }
  if (bn == 128 && epi == EPI_KV) return launch_one<EPI_KV, 128, false>(a, b0, b1, p, n_tiles, m_tiles, splits, st);
  return cudaErrorInvalidValue;
}

}  // namespace dare
