// Bidirectional (no mask) softmax attention on tcgen05 tensor cores, head_dim = 128, bf16 operands, fp32 softmax.
//   dense      : every query row of the step window                       (Alg. 1 line 10)
//   row-sparse : only the query rows of the refresh set, gathered by index (Alg. 2 lines 6, 8; Eq. 4)
// The result rows are written straight into the attention-output cache at their cache rows; rows that are not
// computed keep their cached value (Alg. 2 lines 9-10).
//
// One CTA = one head x one tile of up to 128 query rows of one sequence, walking the keys in blocks of 128.  The key
// blocks alternate between two independent streams (even blocks: stream 0, odd blocks: stream 1); each stream has
// its own running maximum, row sum and accumulator, and the two are merged at the end like the partials of a key
// split.  While one stream's softmax warps are busy on the special-function unit the other stream's are moving
// data, so both the tensor pipe and the exponentials stay busy.  Per stream:
//   warp s       TMA producer: K block and V block of the cache (two 64-column boxes each, 128-byte swizzle)
//   warp 2+s     one lane issues S = Q K^T (M128 N128 K16 x 8, both operands in shared memory) and O += P V
//                (M128 N128 K16 x 8, P read from tensor memory, V from shared memory as an MN-major operand)
//   warps 4+4s.. four softmax warps, thread <-> query row: reads its row of S from tensor memory, exponentiates, and
//                writes P as bf16 over the first 64 columns of S (two keys per 32-bit column, the layout of a
//                tensor-memory A operand), so P never passes through shared memory.  O accumulates in tensor
//                memory; it is rescaled in place only when the running maximum has grown by more than 2^8 (the
//                exponentials are taken against the older maximum until then, which changes nothing in exact
//                arithmetic: numerator and row sum share the factor).
// A single-CTA MMA with both operands in shared memory reads 8 KB per 64 cycles there, all the bandwidth shared
// memory has; the TMA writes of K and V and any P traffic come on top.  Shared-memory traffic, not the tensor pipe,
// bounds this kernel, which is why P stays in tensor memory.
// Key split: when a launch has few (tile, head) pairs - the row-sparse case with one row tile per sequence - the
// gridDim.z CTAs of a cluster share a pair, CTA z taking key blocks z, z + gridDim.z, ...  Each CTA leaves its
// un-normalised accumulator, running maximum and row sum in shared memory; CTA k owns 128/gridDim.z of the rows and
// receives the other CTAs' partials of those rows by bulk copies over distributed shared memory, then merges them
// (the usual rescaling by exp(m_z - max_z m_z)) and writes the rows out.
#include "layer.h"
#include "tc.h"
#include "tc_ptx.cuh"

namespace dare {

using namespace ptx;

namespace {

constexpr int BQ = 128;    // query rows per CTA
constexpr int BKV = 128;   // keys per block
constexpr int HD = 128;

struct AttnSmem {
  static constexpr int Q_BYTES = BQ * HD * 2;          // two 64-column chunks of [128 x 128 B]
  static constexpr int K_BYTES = BKV * HD * 2;         // two chunks of [64 x 128 B]
  static constexpr int V_BYTES = BKV * HD * 2;
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_OFF + Q_BYTES;        // one buffer per stream
  static constexpr int V_OFF = K_OFF + 2 * K_BYTES;    // two buffers per stream: V(j) is wanted last in a block and
                                                       // its buffer is released last, so one buffer leaves no slack
  static constexpr int BAR_OFF = V_OFF + 4 * V_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
  // merge of the two streams: a stream's running maxima [128] and row sums [128] go to its first V buffer, idle
  // after its last product
  // after the key loop the operand buffers are idle; the merge of a key split reuses them:
  static constexpr int DUMP_OFF = 0;                   // this CTA's accumulator [128 rows][128 cols] fp32, 64 KB
  static constexpr int STAT_OFF = DUMP_OFF + BQ * HD * 4;   // running maximum [128], row sum [128]
  static constexpr int RECV_OFF = STAT_OFF + 2 * BQ * 4;    // up to 3 senders x (rows x 512 B + rows x 8 B)
};
static_assert(AttnSmem::TOTAL <= 232448, "shared memory");
// (the key-split buffers may overlap the streams' statistics: they are filled after the statistics were read)

// 2^x for x <= 0 on the special-function unit; results below the normal range flush to zero (they are softmax
// weights 2^-126 times smaller than the row's largest).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// max(a, b, c) in one instruction
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

constexpr int kThreads = 384;
constexpr int kSoftmaxThreads = 256;
// S of stream 0 / 1: columns [0, 128) / [128, 256), P over the first 64 of them; O: [256, 384) / [384, 512)
constexpr uint32_t kTmemCols = 512;
constexpr int kPairMinDense = 128;      // dense launches with longer windows take the two-tile kernel
constexpr int kPairMinSparse = 1024;    // row-sparse launches from this window length on
constexpr float kRescaleStep = 8.f;     // log2 of the growth of the running maximum that triggers a rescale of O

}  // namespace

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const AttnParams p) {
  using S = AttnSmem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::BAR_OFF);
  // one of each per stream
  uint64_t* k_full = bars;          // [2]
  uint64_t* k_empty = bars + 2;     // [2]
  uint64_t* s_full = bars + 4;      // [2]
  uint64_t* p_full = bars + 6;      // [2]
  uint64_t* o_full = bars + 8;      // [2]
  uint64_t* v_full = bars + 10;     // [2 streams][2 buffers]
  uint64_t* v_empty = bars + 14;    // [2 streams][2 buffers]
  uint64_t* recv_bar = bars + 18;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 19);

  // the warp index through a shuffle, so that the compiler knows it (and every role decision and shared-memory
  // descriptor derived from it) to be uniform over the warp
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int ksplit = gridDim.z;                      // = cluster size along z
  const int z = ksplit > 1 ? (int)cluster_ctarank() : 0;
  const int rows_own = BQ / ksplit;                   // rows of the tile this CTA writes out
  const bool dbg = p.debug != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
  if (dbg && threadIdx.x == 0) p.debug[0] = globaltimer_ns();
  const StepGeom& g = p.g;
  // CTA -> (head, sequence, row tile), in launch order:
  //   row-sparse: heads fastest, then sequences, then row tiles: the first row tile of every sequence comes first,
  //               so that the CTAs that have work are scheduled before the (many) tiles past the refresh set
  //   dense     : row tiles fastest, then heads, then sequences: the CTAs resident at any time share the K and V of
  //               a few (sequence, head) pairs, which then stay in the L2 instead of being streamed from HBM by
  //               every row tile again
  int h, b, tile;
  {
    const int lin = blockIdx.y * gridDim.x + blockIdx.x;
    if (p.idx != nullptr) {
      h = lin % g.n_heads;
      const int rest = lin / g.n_heads;
      tile = rest / g.batch;
      b = rest - tile * g.batch;
    } else {
      const int tps = (g.seq_act + BQ - 1) / BQ;
      tile = lin % tps;
      const int rest = lin / tps;
      h = rest % g.n_heads;
      b = rest / g.n_heads;
    }
  }

  // Row tiles past the first one of a sequence are usually empty in the row-sparse case: they look at the refresh
  // set before spending anything on set-up.
  // A launch issued in two forms (row-sparse over the refresh set, dense with its stores masked) runs in the one
  // the size of the refresh set favours; the other leaves here, before it has set anything up.
  if (p.gate_count != nullptr) {
    pdl_wait();
    const int c = __ldcg(p.gate_count);
    if (c < p.gate_lo || c >= p.gate_hi) return;          // uniform over the launch
  }
  if (p.idx != nullptr && tile > 0) {
    pdl_wait();
    if (__ldcg(p.batch_off + b) + tile * BQ >= __ldcg(p.batch_off + b + 1)) return;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[2 * i], 1); mbar_init(&v_full[2 * i + 1], 1);
      mbar_init(&v_empty[2 * i], 1); mbar_init(&v_empty[2 * i + 1], 1);
      mbar_init(&s_full[i], 1); mbar_init(&o_full[i], 1);
      mbar_init(&p_full[i], kSoftmaxThreads / 64);     // one arrival per softmax warp of the stream
    }
    mbar_init(recv_bar, 1);
    fence_mbar_init();
    if (ksplit > 1) mbar_arrive_expect_tx(recv_bar, (uint32_t)((ksplit - 1) * rows_own * (HD * 4 + 8)));
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
  }
  if (warp == 2) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  // The previous kernel in the stream (the K/V projection) writes the K and V caches only.  The queries and the
  // refresh set come from kernels further back, which are complete by the time any CTA of this grid runs (every
  // kernel lets its successor start only after its own wait): they are read without waiting, so that the gather
  // of the Q tile overlaps the projection's tail.  Those reads go to the L2 (ld.global.cg): ahead of the wait this
  // SM's L1 may still hold the lines an earlier step's CTA read from the same addresses.  Warp 0 waits right away and starts the first K and V blocks.
  // (unless the step's launch order puts their producer right before this kernel: then everybody waits first)
  if (p.wait_first) pdl_wait();
  // ---- rows of this tile (uniform over the CTA)
  int row0 = 0, rows_valid = 0;
  bool active = true;
  if (p.idx != nullptr) {
    const int lo = __ldcg(p.batch_off + b), hi = __ldcg(p.batch_off + b + 1);
    row0 = lo + tile * BQ;
    active = slice_ok(lo, hi, g.tokens(), p.status) && row0 < hi;
    rows_valid = active ? min(BQ, hi - row0) : 0;
  } else {
    row0 = b * g.seq_act + tile * BQ;
    rows_valid = min(BQ, g.seq_act - tile * BQ);
    if (p.store_mask != nullptr) {
      // dense form of a row-sparse step: a tile none of whose rows was refreshed has nothing to store
      // (the gate above has waited for the selection)
      const int r = (int)threadIdx.x;
      const int mine = r < rows_valid && __ldcg(p.store_mask + g.cache_row(row0 + r)) == 0;
      active = __syncthreads_or(mine) != 0;
    }
  }
  const int n_blocks_all = (g.kv_len + BKV - 1) / BKV;
  const int n_blocks = n_blocks_all > z ? (n_blocks_all - z + ksplit - 1) / ksplit : 0;   // blocks z, z + ksplit, ...
  const int kv_row0 = b * g.max_seq;
  // The first K and V block of each stream start as soon as the projection is complete, by the thread that
  // initialised the barriers, so that they are in flight while the Q tile is gathered.
  if (warp == 0) {
    pdl_wait();
    pdl_launch_dependents();
  }
  if (threadIdx.x == 0 && active) {
    for (int s2 = 0; s2 < 2 && s2 < n_blocks; ++s2) {
      const int row = kv_row0 + (z + s2 * ksplit) * BKV;
      uint8_t* kd = smem + S::K_OFF + s2 * S::K_BYTES;
      uint8_t* vd = smem + S::V_OFF + 2 * s2 * S::V_BYTES;
      mbar_arrive_expect_tx(&k_full[s2], S::K_BYTES);
      tma_load_2d(kd, &tm_k, h * HD, row, &k_full[s2]);
      tma_load_2d(kd + S::K_BYTES / 2, &tm_k, h * HD + 64, row, &k_full[s2]);
      mbar_arrive_expect_tx(&v_full[2 * s2], S::V_BYTES);
      tma_load_2d(vd, &tm_v, h * HD, row, &v_full[2 * s2]);
      tma_load_2d(vd + S::V_BYTES / 2, &tm_v, h * HD + 64, row, &v_full[2 * s2]);
    }
  }
  // ---- Q tile: gathered rows -> shared memory in the K-major 128-byte-swizzled layout (16-byte units), by the
  // warps other than warp 0
  if (active && warp != 0) {
    uint8_t* qs = smem + S::Q_OFF;
    constexpr int kGather = kThreads - 32;
    constexpr int QU = (BQ * 16 + kGather - 1) / kGather;     // 16-byte units per thread
    const int u0 = (int)threadIdx.x - 32;
    int tok[QU];
    uint4 qv[QU];
    // all index loads first, then all row loads, then the stores: one memory round trip each instead of one per unit
#pragma unroll
    for (int k = 0; k < QU; ++k) {
      const int u = u0 + k * kGather, r = u >> 4;              // 16 units of 8 bf16 per row
      tok[k] = -1;
      if (u < BQ * 16 && r < rows_valid) tok[k] = p.idx ? __ldcg(p.idx + row0 + r) : row0 + r;
      if (p.idx && tok[k] >= 0 && !token_ok(tok[k], g.tokens(), p.status)) tok[k] = -1;      // read as a row of zeros
    }
#pragma unroll
    for (int k = 0; k < QU; ++k) {
      const int unit = (u0 + k * kGather) & 15;
      qv[k] = make_uint4(0u, 0u, 0u, 0u);
      if (tok[k] >= 0) qv[k] = __ldcg(reinterpret_cast<const uint4*>(p.q + (size_t)tok[k] * g.d + h * HD + unit * 8));
    }
#pragma unroll
    for (int k = 0; k < QU; ++k) {
      const int u = u0 + k * kGather, r = u >> 4, unit = u & 15;
      const int chunk = unit >> 3, uc = unit & 7;
      if (u < BQ * 16) *reinterpret_cast<uint4*>(qs + chunk * (BQ * 128) + r * 128 + ((uc ^ (r & 7)) << 4)) = qv[k];
    }
    fence_proxy_async_smem();
  }
  if (warp != 0) {
    pdl_wait();                       // every thread waits before it can touch what the projection wrote, or leave
    pdl_launch_dependents();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (dbg && threadIdx.x == 0) p.debug[1] = globaltimer_ns();

  if (active) {
  // stream of this warp (producers 0/1, issuers 2/3, softmax warps 4-7 / 8-11) and its share of the key blocks:
  // local blocks st, st + 2, ... of this CTA's blocks, local block i being key block z + i * ksplit
  const int st = warp < 4 ? (warp & 1) : ((warp - 4) >> 2);
  const int n_st = (n_blocks - st + 1) / 2;
  const int n_other = n_blocks - n_st;
  const uint32_t tmem_s = tmem_base + st * BKV, tmem_o = tmem_base + 2 * BKV + st * HD;
  // The producer and issuer warps run their loops converged (every lane polls the barriers); one elected lane
  // issues the copies and the MMAs.  Their operands are then warp-uniform values, which is what those instructions take.
  if (warp < 2) {
    uint8_t* kd = smem + S::K_OFF + st * S::K_BYTES;
    for (int j = 1; j < n_st; ++j) {                        // block 0 of the stream was started before the Q gather
      const int vb = 2 * st + (j & 1);
      uint8_t* vd = smem + S::V_OFF + vb * S::V_BYTES;
      const int row = kv_row0 + (z + (2 * j + st) * ksplit) * BKV;
      mbar_wait(&k_empty[st], (j & 1) ^ 1, p.status);       // S(j-1) = Q K(j-1)^T has been computed
      if (elect_one()) {
        mbar_arrive_expect_tx(&k_full[st], S::K_BYTES);
        tma_load_2d(kd, &tm_k, h * HD, row, &k_full[st]);
        tma_load_2d(kd + S::K_BYTES / 2, &tm_k, h * HD + 64, row, &k_full[st]);
      }
      __syncwarp();
      mbar_wait(&v_empty[vb], ((j >> 1) & 1) ^ 1, p.status);       // O += P(j-2) V(j-2) has been computed
      if (elect_one()) {
        mbar_arrive_expect_tx(&v_full[vb], S::V_BYTES);
        tma_load_2d(vd, &tm_v, h * HD, row, &v_full[vb]);
        tma_load_2d(vd + S::V_BYTES / 2, &tm_v, h * HD + 64, row, &v_full[vb]);
      }
      __syncwarp();
    }
  } else if (warp < 4) {
    constexpr uint32_t idesc_qk = idesc_bf16(BQ, BKV, false);
    constexpr uint32_t idesc_pv = idesc_bf16(BQ, HD, true);
    const uint64_t q_desc = smem_desc_k_sw128(smem_u32(smem + S::Q_OFF));
    const uint64_t k_desc = smem_desc_k_sw128(smem_u32(smem + S::K_OFF + st * S::K_BYTES));
    const uint64_t v_desc0 = smem_desc_mn_sw128(smem_u32(smem + S::V_OFF + 2 * st * S::V_BYTES), BKV * 128);
    auto issue_qk = [&](int j) {
      mbar_wait(&k_full[st], j & 1, p.status);
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk)
          umma_ss(tmem_s, q_desc + (((kk >> 2) * (BQ * 128) + (kk & 3) * 32) >> 4),
                  k_desc + (((kk >> 2) * (BKV * 128) + (kk & 3) * 32) >> 4), idesc_qk, kk != 0 ? 1u : 0u);
        umma_commit(&s_full[st]);
        umma_commit(&k_empty[st]);
      }
      __syncwarp();
    };
    if (n_st > 0) issue_qk(0);
    for (int j = 0; j < n_st; ++j) {
      mbar_wait(&p_full[st], j & 1, p.status);      // P(j) has replaced S(j) in tensor memory
      const int vb = 2 * st + (j & 1);
      mbar_wait(&v_full[vb], (j >> 1) & 1, p.status);
      tc_fence_after();
      if (elect_one()) {
        const uint64_t v_desc = v_desc0 + (uint64_t)((j & 1) * (S::V_BYTES >> 4));
#pragma unroll
        for (int ks = 0; ks < BKV / 16; ++ks)       // 16 keys of P = 8 columns
          umma_ts(tmem_o, tmem_s + ks * 8, v_desc + ((ks * (16 * 128)) >> 4), idesc_pv, (j | ks) != 0 ? 1u : 0u);
        umma_commit(&o_full[st]);
        umma_commit(&v_empty[vb]);
      }
      __syncwarp();
      // the tensor pipe runs MMAs in issue order: the next scores overwrite P(j) only after the product above read it
      if (j + 1 < n_st) issue_qk(j + 1);
    }
  } else {
    // ---- softmax of this stream's blocks: thread <-> query row
    const int quarter = warp & 3;               // TMEM lane quarter of this warp
    const int r = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float c = rsqrtf((float)HD) * 1.4426950408889634f;   // softmax scale folded into the exp2 argument
    float m = -INFINITY, l = 0.f;               // maximum the exponentials are taken against; row sum against it
    // the token whose cache row this thread writes at the end: asked for now, so that the read is not the first thing
    // the epilogue waits for
    const int t_row = r < rows_valid ? (p.idx ? __ldcg(p.idx + row0 + r) : row0 + r) : -1;

    // a warp none of whose 32 rows exists (a partly filled row-sparse tile) only passes the blocks on: its rows of P
    // and O are whatever the score buffer held, belong to no token and are never stored
    const bool warp_has_rows = quarter * 32 < rows_valid;
    for (int j = 0; j < n_st; ++j) {
      mbar_wait(&s_full[st], j & 1, p.status);
      tc_fence_after();
      if (dbg && j == 0 && threadIdx.x == 128) p.debug[2] = globaltimer_ns();
      if (!warp_has_rows && ksplit == 1) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[st]);
        continue;
      }
      const int key0 = (z + (2 * j + st) * ksplit) * BKV;
      const int n_keys = min(BKV, g.kv_len - key0);   // the last block may be ragged: keys past kv_len do not exist
      // O and the row sum move to a new maximum only when it grew by more than kRescaleStep (in log2 units); the
      // product that last wrote O has to be complete before O is rescaled in place
      auto settle_max = [&](float m_new) {
        if (j == 0) {
          m = m_new;
        } else {
          const bool grow = (m_new - m) * c > kRescaleStep;
          if (__any_sync(0xffffffffu, grow)) {
            const float alpha = grow ? fast_exp2((m - m_new) * c) : 1.f;
            if (grow) { m = m_new; l *= alpha; }
            mbar_wait(&o_full[st], (j - 1) & 1, p.status);
            tc_fence_after();
#pragma unroll 1
            for (int ch = 0; ch < 4; ++ch) {
              float o[32];
              tmem_ld_32x32(tmem_o + lane_addr + ch * 32, o);
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] *= alpha;
              tmem_st_32x32(tmem_o + lane_addr + ch * 32, o);
            }
          }
        }
      };
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      // the row of S: four loads in flight together
      float v[128];
      tmem_ld_32x32_nowait(tmem_s + lane_addr, v);
      tmem_ld_32x32_nowait(tmem_s + lane_addr + 32, v + 32);
      tmem_ld_32x32_nowait(tmem_s + lane_addr + 64, v + 64);
      tmem_ld_32x32_nowait(tmem_s + lane_addr + 96, v + 96);
      tmem_ld_wait();
      if (n_keys < BKV) {
#pragma unroll
        for (int i = 0; i < 128; ++i)
          if (i >= n_keys) v[i] = -INFINITY;
      }
      // row maximum: four independent chains of three-input maxima
      float mx4[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) mx4[k] = fmaxf(v[k], v[4 + k]);
#pragma unroll
      for (int i = 8; i < 128; i += 8) {
#pragma unroll
        for (int k = 0; k < 4; ++k) mx4[k] = fmax3(mx4[k], v[i + k], v[i + 4 + k]);
      }
      settle_max(fmax3(m, fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])));
      // exponentials against m (masked keys: 2^-inf = 0) and the row sum, the scaling and the sum two keys per
      // instruction (packed fp32)
      const float2 c2 = make_float2(c, c), nmc2 = make_float2(-m * c, -m * c);
      float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      // P as bf16 over the first 64 columns of this row of S: column i = keys (2i, 2i+1); packed as it is produced,
      // so that the scores leave the register file pair by pair
      float pk[64];
#pragma unroll
      for (int i = 0; i < 128; i += 2) {
        float2 e = __ffma2_rn(make_float2(v[i], v[i + 1]), c2, nmc2);
        e.x = fast_exp2(e.x);
        e.y = fast_exp2(e.y);
        sum2[(i >> 1) & 1] = __fadd2_rn(sum2[(i >> 1) & 1], e);
        __nv_bfloat162 h2 = __floats2bfloat162_rn(e.x, e.y);
        pk[i >> 1] = __uint_as_float(*reinterpret_cast<uint32_t*>(&h2));
      }
      sum4[0] = sum2[0].x; sum4[1] = sum2[0].y; sum4[2] = sum2[1].x; sum4[3] = sum2[1].y;
      tmem_st_32x32_nowait(tmem_s + lane_addr, pk);
      tmem_st_32x32_nowait(tmem_s + lane_addr + 32, pk + 32);
      tmem_st_wait();
      l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[st]);
    }
    if (n_st > 0) {
      mbar_wait(&o_full[st], (n_st - 1) & 1, p.status);
      tc_fence_after();
    }
    if (dbg && threadIdx.x == 128) p.debug[3] = globaltimer_ns();
    // ---- merge the two streams: thread (stream st, row r) finishes columns [64 st, 64 st + 64) of the row
    float* stat_mine = reinterpret_cast<float*>(smem + S::V_OFF + 2 * st * S::V_BYTES);
    const float* stat_other = reinterpret_cast<const float*>(smem + S::V_OFF + 2 * (st ^ 1) * S::V_BYTES);
    stat_mine[r] = m;
    stat_mine[BQ + r] = l;
    tc_fence_before();
    asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");
    tc_fence_after();
    const float m_o = n_other > 0 ? stat_other[r] : -INFINITY, l_o = n_other > 0 ? stat_other[BQ + r] : 0.f;
    const float m_all = fmaxf(m, m_o);
    const float w_mine = n_st > 0 ? fast_exp2((m - m_all) * c) : 0.f;
    const float w_other = n_other > 0 ? fast_exp2((m_o - m_all) * c) : 0.f;
    const float l_row = w_mine * l + w_other * l_o;
    const uint32_t t_mine = tmem_o + lane_addr + st * 64;
    const uint32_t t_other = tmem_base + 2 * BKV + (st ^ 1) * HD + lane_addr + st * 64;
    float acc[64];
#pragma unroll
    for (int cgrp = 0; cgrp < 2; ++cgrp) {
      float a[32];
      if (n_st > 0) {
        tmem_ld_32x32(t_mine + cgrp * 32, a);
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[cgrp * 32 + i] = a[i] * w_mine;
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[cgrp * 32 + i] = 0.f;
      }
      if (n_other > 0) {
        tmem_ld_32x32(t_other + cgrp * 32, a);
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[cgrp * 32 + i] = fmaf(a[i], w_other, acc[cgrp * 32 + i]);
      }
    }
    if (ksplit == 1) {
      // normalise, store
      const float inv = 1.f / l_row;
      const int t = t_row;
      if (t >= 0 && (p.idx == nullptr ? (p.store_mask == nullptr || __ldcg(p.store_mask + g.cache_row(t)) == 0)
                                      : token_ok(t, g.tokens(), p.status))) {      // (else: no cache row to write)
        __nv_bfloat16* dst = p.oc + (size_t)g.cache_row(t) * g.d + h * HD + st * 64;
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] *= inv;
#pragma unroll
        for (int v = 0; v < 8; ++v) reinterpret_cast<uint4*>(dst)[v] = pack8_bf16(acc + 8 * v);
      }
    } else {
      // key split: leave the un-normalised row, its maximum and its sum in shared memory for the merge.  The
      // operand buffers those go to are idle: both streams' last products were complete before the barrier above.
      float* dump = reinterpret_cast<float*>(smem + S::DUMP_OFF) + (size_t)r * HD;
#pragma unroll
      for (int v = 0; v < 16; ++v) {
        const int unit = st * 16 + v;                    // 32 sixteen-byte units per 512-byte row, XOR-swizzled
        *reinterpret_cast<float4*>(dump + ((unit ^ (r & 7)) << 2)) =
            make_float4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
      }
      if (st == 0) {
        float* stat = reinterpret_cast<float*>(smem + S::STAT_OFF);
        stat[r] = m_all;
        stat[BQ + r] = l_row;
      }
      fence_proxy_async_smem();
    }
  }
  if (ksplit > 1) {
    // ---- merge of the key split (all warps)
    __syncthreads();
    tc_fence_before();
    cluster_sync_relaxed();                              // every CTA of the cluster is past its key loop
    tc_fence_after();
    if (warp == 4 && lane < ksplit && lane != z) {
      // hand the rows owned by CTA `lane` to it: the rows, their maxima, their sums
      const int k = lane;
      const int slot = z < k ? z : z - 1;
      const uint32_t slot_bytes = (uint32_t)rows_own * (HD * 4 + 8);
      const uint32_t dst = map_to_cta(smem_u32(smem + S::RECV_OFF) + slot * slot_bytes, (uint32_t)k);
      const uint32_t bar = map_to_cta(smem_u32(recv_bar), (uint32_t)k);
      bulk_copy_to_cta(dst, smem_u32(smem + S::DUMP_OFF + (size_t)k * rows_own * HD * 4), rows_own * HD * 4, bar);
      bulk_copy_to_cta(dst + rows_own * HD * 4, smem_u32(smem + S::STAT_OFF + k * rows_own * 4), rows_own * 4, bar);
      bulk_copy_to_cta(dst + rows_own * HD * 4 + rows_own * 4, smem_u32(smem + S::STAT_OFF + (BQ + k * rows_own) * 4),
                       rows_own * 4, bar);
    }
    mbar_wait(recv_bar, 0, p.status);
    const float c = rsqrtf((float)HD) * 1.4426950408889634f;
    const float* dump = reinterpret_cast<const float*>(smem + S::DUMP_OFF);
    const float* stat = reinterpret_cast<const float*>(smem + S::STAT_OFF);
    const uint32_t slot_floats = (uint32_t)rows_own * (HD + 2);
    const float* recv = reinterpret_cast<const float*>(smem + S::RECV_OFF);
    for (int rl = warp; rl < rows_own; rl += kThreads / 32) {
      const int r = z * rows_own + rl;
      if (r >= rows_valid) break;
      float mz[4], lz[4];
      mz[0] = stat[r]; lz[0] = stat[BQ + r];
      float mx = mz[0];
      for (int s2 = 0; s2 < ksplit - 1; ++s2) {
        const float* sl = recv + s2 * slot_floats;
        mz[s2 + 1] = sl[rows_own * HD + rl];
        lz[s2 + 1] = sl[rows_own * HD + rows_own + rl];
        mx = fmaxf(mx, mz[s2 + 1]);
      }
      const int off = ((lane ^ (r & 7)) << 2);           // this lane's 4 columns inside the swizzled row
      float w = exp2f((mz[0] - mx) * c);
      float4 o = *reinterpret_cast<const float4*>(dump + (size_t)r * HD + off);
      o.x *= w; o.y *= w; o.z *= w; o.w *= w;
      float lsum = w * lz[0];
      for (int s2 = 0; s2 < ksplit - 1; ++s2) {
        w = exp2f((mz[s2 + 1] - mx) * c);
        const float4 a = *reinterpret_cast<const float4*>(recv + s2 * slot_floats + (size_t)rl * HD + off);
        o.x = fmaf(a.x, w, o.x); o.y = fmaf(a.y, w, o.y); o.z = fmaf(a.z, w, o.z); o.w = fmaf(a.w, w, o.w);
        lsum = fmaf(w, lz[s2 + 1], lsum);
      }
      const float inv = 1.f / lsum;
      const int t = p.idx ? __ldcg(p.idx + row0 + r) : row0 + r;
      if (p.idx != nullptr && !token_ok(t, g.tokens(), p.status)) continue;        // no cache row to write
      if (p.idx == nullptr && p.store_mask != nullptr && __ldcg(p.store_mask + g.cache_row(t)) != 0) continue;   // a reused row
      __nv_bfloat16* dst = p.oc + (size_t)g.cache_row(t) * g.d + h * HD + 4 * lane;
      __nv_bfloat162 lo2 = __floats2bfloat162_rn(o.x * inv, o.y * inv), hi2 = __floats2bfloat162_rn(o.z * inv, o.w * inv);
      uint2 packed;
      packed.x = *reinterpret_cast<uint32_t*>(&lo2);
      packed.y = *reinterpret_cast<uint32_t*>(&hi2);
      *reinterpret_cast<uint2*>(dst) = packed;
    }
  }
  }  // active
  tc_fence_before();
  // nobody leaves while a copy out of its shared memory may still be in flight (its receiver has seen it land)
  if (ksplit > 1) cluster_sync_relaxed(); else __syncthreads();
  if (dbg && threadIdx.x == 0) p.debug[4] = globaltimer_ns();
  if (p.debug != nullptr && threadIdx.x == 0) {      // latest end over the CTAs that had work, and their number
    atomicMax(&p.debug[6], globaltimer_ns());
    atomicAdd(&p.debug[7], 1ull);
  }
  if (warp == 2) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------------------------ two query tiles
// The variant for launches with many query rows per (sequence, head): one CTA = one head x up to 256 query rows, i.e.
// two 128-row tiles, each with its own softmax warps, issuer warp, S/P and O regions of tensor memory - the two
// streams of the kernel above - but now the streams walk the same key blocks and share them: every K and V block is
// brought into shared memory once for both tiles, which halves what a CTA pulls from the L2 per flop (that traffic,
// 64 KB per key block and tile, is what the kernel above runs into when every SM does it at once).  No merge at the
// end: a stream owns its rows.
// Tensor memory per stream: two score buffers of 64 columns and the 128-column O accumulator.  The unit of the
// pipeline is a half block of 64 keys: S(h) goes to buffer h & 1, and the issuer keeps S(h + 1) in flight while the
// softmax warps are on S(h) (tcgen05.ld, maximum, exp2, P(h) as bf16 back into the first 32 columns of the buffer),
// then issues P(h) V and, behind it in issue order, S(h + 2) into the buffer P(h) was read from.  With one score
// buffer per stream the softmax warps idled through their own stream's two products of every block (measured: the
// special-function unit is only 13 % of the kernel's time; the chain S -> softmax -> P V -> S was the rest).
// The softmax warps can therefore be up to two P V products ahead of the tensor core; they wait for a product only
// to rescale O or to read it out, on one of two barriers per stream (product h signals barrier h & 1) so that a
// parity wait never has to tell more than two consecutive phases apart.
namespace {
struct PairSmem {
  static constexpr int Q_BYTES = BQ * HD * 2;
  static constexpr int KV_BYTES = BKV * HD * 2;
  static constexpr int Q_OFF = 0;                        // two tiles
  static constexpr int K_OFF = Q_OFF + 2 * Q_BYTES;      // ring of 2
  static constexpr int V_OFF = K_OFF + 2 * KV_BYTES;     // ring of 2
  static constexpr int BAR_OFF = V_OFF + 2 * KV_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
};
static_assert(PairSmem::TOTAL <= 232448, "shared memory");
constexpr int kPairRows = 2 * BQ;
constexpr int kHalf = BKV / 2;     // keys per score buffer
}  // namespace

__global__ void __launch_bounds__(kThreads, 1)
attn_pair_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const AttnParams p) {
  using S = PairSmem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::BAR_OFF);
  uint64_t* k_full = bars;          // [2 ring slots]
  uint64_t* k_empty = bars + 2;     // [2]: one arrival per stream
  uint64_t* v_full = bars + 4;      // [2]
  uint64_t* v_empty = bars + 6;     // [2]: one arrival per stream
  uint64_t* s_full = bars + 8;      // [2 streams][2 score buffers]
  uint64_t* p_full = bars + 12;     // [2 streams][2 score buffers]
  uint64_t* o_full = bars + 16;     // [2 streams][2]: product h signals o_full[stream][h & 1]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const StepGeom& g = p.g;
  // Which form runs?  A launch that carries both (dense_from > 0) decides here, from the size of the refresh set:
  // below dense_from the rows of the refresh set, from there on every row with only the refreshed ones stored.
  const int* idx = p.idx;
  const int* batch_off = p.batch_off;
  const int* store_mask = p.store_mask;
  if (p.gate_count != nullptr) {
    pdl_wait();
    const int c = __ldcg(p.gate_count);
    if (p.dense_from > 0) {
      if (c >= p.dense_from) { idx = nullptr; batch_off = nullptr; store_mask = p.dense_mask; }
    } else if (c < p.gate_lo || c >= p.gate_hi) {
      return;                                             // uniform over the launch
    }
  }
  // CTA -> (head, sequence, 256-row tile): same launch orders as the kernel above
  const int tps = (g.seq_act + kPairRows - 1) / kPairRows;
  int h, b, tile;
  {
    const int lin = blockIdx.y * gridDim.x + blockIdx.x;
    if (idx != nullptr) {
      h = lin % g.n_heads;
      const int rest = lin / g.n_heads;
      tile = rest / g.batch;
      b = rest - tile * g.batch;
    } else {
      tile = lin % tps;
      const int rest = lin / tps;
      h = rest % g.n_heads;
      b = rest / g.n_heads;
    }
  }
  if (idx != nullptr && tile > 0) {
    pdl_wait();
    if (__ldcg(batch_off + b) + tile * kPairRows >= __ldcg(batch_off + b + 1)) return;
  }
  // diagnostics: [0] first CTA's start, [1] its set-up done, [3] its key loop done, [4] its end; over the CTAs with
  // work: [5] latest start, [6] latest end, [7] their number
  const bool dbg = p.debug != nullptr && blockIdx.x == 0 && blockIdx.y == 0;
  unsigned long long t_start = 0;
  if (p.debug != nullptr && threadIdx.x == 0) {
    t_start = globaltimer_ns();
    if (dbg) p.debug[0] = t_start;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&v_full[i], 1); mbar_init(&k_empty[i], 2); mbar_init(&v_empty[i], 2);
      for (int b = 0; b < 2; ++b) {
        mbar_init(&s_full[2 * i + b], 1); mbar_init(&p_full[2 * i + b], kSoftmaxThreads / 64); mbar_init(&o_full[2 * i + b], 1);
      }
    }
    fence_mbar_init();
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
  }
  if (warp == 2) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  // (as in the kernel above: queries and refresh set are read without waiting for the K/V projection; warp 0 waits
  // right away and starts the first key blocks, the other warps gather the Q tiles first)
  if (p.wait_first) pdl_wait();
  // ---- rows of the two tiles (uniform over the CTA)
  int row0 = 0, rows_all = 0;
  bool active = true;
  if (idx != nullptr) {
    const int lo = __ldcg(batch_off + b), hi = __ldcg(batch_off + b + 1);
    row0 = lo + tile * kPairRows;
    active = slice_ok(lo, hi, g.tokens(), p.status) && row0 < hi;
    rows_all = active ? min(kPairRows, hi - row0) : 0;
  } else {
    row0 = b * g.seq_act + tile * kPairRows;
    rows_all = min(kPairRows, g.seq_act - tile * kPairRows);
    if (store_mask != nullptr) {
      const int r = (int)threadIdx.x;
      const int mine = r < rows_all && __ldcg(store_mask + g.cache_row(row0 + r)) == 0;
      active = __syncthreads_or(mine) != 0;
    }
  }
  const int n_blocks = (g.kv_len + BKV - 1) / BKV;
  const int n_half = (g.kv_len + kHalf - 1) / kHalf;   // half blocks: the unit of the score / softmax / P V pipeline
  const int kv_row0 = b * g.max_seq;
  auto load_kv = [&](int i) {        // one thread: key block i into ring slot i & 1
    const int slot = i & 1, row = kv_row0 + i * BKV;
    uint8_t* kd = smem + S::K_OFF + slot * S::KV_BYTES;
    uint8_t* vd = smem + S::V_OFF + slot * S::KV_BYTES;
    mbar_arrive_expect_tx(&k_full[slot], S::KV_BYTES);
    tma_load_2d(kd, &tm_k, h * HD, row, &k_full[slot]);
    tma_load_2d(kd + S::KV_BYTES / 2, &tm_k, h * HD + 64, row, &k_full[slot]);
    mbar_arrive_expect_tx(&v_full[slot], S::KV_BYTES);
    tma_load_2d(vd, &tm_v, h * HD, row, &v_full[slot]);
    tma_load_2d(vd + S::KV_BYTES / 2, &tm_v, h * HD + 64, row, &v_full[slot]);
  };
  // the first two key blocks start as soon as the projection is complete, by the thread that initialised the
  // barriers: in flight during the Q gather
  if (warp == 0) {
    pdl_wait();
    pdl_launch_dependents();
  }
  if (threadIdx.x == 0 && active) {
    for (int i = 0; i < 2 && i < n_blocks; ++i) load_kv(i);
  }
  // ---- both Q tiles: gathered rows -> shared memory in the K-major 128-byte-swizzled layout (16-byte units)
  if (active && warp != 0) {
    constexpr int kGather = kThreads - 32;
    constexpr int QU = (kPairRows * 16 + kGather - 1) / kGather;
    const int u0 = (int)threadIdx.x - 32;
    int tok[QU];
    uint4 qv[QU];
#pragma unroll
    for (int k = 0; k < QU; ++k) {
      const int u = u0 + k * kGather, r = u >> 4;
      tok[k] = -1;
      if (u < kPairRows * 16 && r < rows_all) tok[k] = idx ? __ldcg(idx + row0 + r) : row0 + r;
      if (idx && tok[k] >= 0 && !token_ok(tok[k], g.tokens(), p.status)) tok[k] = -1;      // read as a row of zeros
    }
#pragma unroll
    for (int k = 0; k < QU; ++k) {
      const int unit = (u0 + k * kGather) & 15;
      qv[k] = make_uint4(0u, 0u, 0u, 0u);
      if (tok[k] >= 0) qv[k] = __ldcg(reinterpret_cast<const uint4*>(p.q + (size_t)tok[k] * g.d + h * HD + unit * 8));
    }
#pragma unroll
    for (int k = 0; k < QU; ++k) {
      const int u = u0 + k * kGather, r = u >> 4, unit = u & 15;
      const int chunk = unit >> 3, uc = unit & 7, rt = r & (BQ - 1);
      uint8_t* qs = smem + S::Q_OFF + (r >> 7) * S::Q_BYTES;
      if (u < kPairRows * 16) *reinterpret_cast<uint4*>(qs + chunk * (BQ * 128) + rt * 128 + ((uc ^ (rt & 7)) << 4)) = qv[k];
    }
    fence_proxy_async_smem();
  }
  if (warp != 0) {
    pdl_wait();
    pdl_launch_dependents();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (dbg && threadIdx.x == 0) p.debug[1] = globaltimer_ns();

  if (active) {
  // stream = query tile: warps 2/3 issue for tile 0/1, softmax warps 4-7 / 8-11; warp 0 brings the key blocks
  const int st = warp < 4 ? (warp & 1) : ((warp - 4) >> 2);
  const int rows_valid = max(0, min(BQ, rows_all - st * BQ));       // rows of this stream's tile
  const bool st_active = rows_valid > 0;                             // the second tile of a short tail is empty
  const uint32_t tmem_s = tmem_base + st * BKV, tmem_o = tmem_base + 2 * BKV + st * HD;
  if (warp == 0) {
    for (int i = 2; i < n_blocks; ++i) {
      const int slot = i & 1;
      // both streams have finished with block i - 2: their score products ...
      mbar_wait(&k_empty[slot], ((i >> 1) & 1) ^ 1, p.status);
      // ... and their P V products
      mbar_wait(&v_empty[slot], ((i >> 1) & 1) ^ 1, p.status);
      if (elect_one()) load_kv(i);
      __syncwarp();
    }
  } else if (warp == 2 || warp == 3) {
    constexpr uint32_t idesc_qk = idesc_bf16(BQ, kHalf, false);
    constexpr uint32_t idesc_pv = idesc_bf16(BQ, HD, true);
    const uint64_t q_desc = smem_desc_k_sw128(smem_u32(smem + S::Q_OFF + st * S::Q_BYTES));
    const uint64_t k_desc0 = smem_desc_k_sw128(smem_u32(smem + S::K_OFF));
    const uint64_t v_desc0 = smem_desc_mn_sw128(smem_u32(smem + S::V_OFF), BKV * 128);
    if (!st_active) {
      // an empty tile still releases the ring slots it shares: one arrival per block and barrier, never ahead of
      // the block's data
      for (int i = 0; i < n_blocks; ++i) {
        const int slot = i & 1;
        mbar_wait(&k_full[slot], (i >> 1) & 1, p.status);
        if (elect_one()) mbar_arrive(&k_empty[slot]);
        __syncwarp();
        mbar_wait(&v_full[slot], (i >> 1) & 1, p.status);
        if (elect_one()) mbar_arrive(&v_empty[slot]);
        __syncwarp();
      }
    } else {
      // Half blocks of 64 keys, h = 0 .. n_half - 1, scores of half h into buffer h & 1: S(h + 1) is computed while
      // the softmax warps are on S(h), so they go from one half to the next without waiting for the tensor core.
      auto issue_qk = [&](int hf) {
        const int i = hf >> 1, slot = i & 1, hb = hf & 1;
        if (hb == 0) mbar_wait(&k_full[slot], (i >> 1) & 1, p.status);   // (the second half: same block, already here)
        tc_fence_after();
        if (elect_one()) {
          const uint64_t k_desc = k_desc0 + (uint64_t)(slot * (S::KV_BYTES >> 4)) + (uint64_t)((hb * kHalf * 128) >> 4);
#pragma unroll
          for (int kk = 0; kk < HD / 16; ++kk)
            umma_ss(tmem_s + hb * kHalf, q_desc + (((kk >> 2) * (BQ * 128) + (kk & 3) * 32) >> 4),
                    k_desc + (((kk >> 2) * (BKV * 128) + (kk & 3) * 32) >> 4), idesc_qk, kk != 0 ? 1u : 0u);
          umma_commit(&s_full[2 * st + hb]);
          if (hb == 1 || hf == n_half - 1) umma_commit(&k_empty[slot]);   // the block's keys are done with
        }
        __syncwarp();
      };
      if (n_half > 0) issue_qk(0);
      if (n_half > 1) issue_qk(1);
      for (int hf = 0; hf < n_half; ++hf) {
        const int i = hf >> 1, slot = i & 1, hb = hf & 1;
        mbar_wait(&p_full[2 * st + hb], (hf >> 1) & 1, p.status);   // P(hf) has replaced S(hf) in tensor memory
        if (hb == 0) mbar_wait(&v_full[slot], (i >> 1) & 1, p.status);
        tc_fence_after();
        if (elect_one()) {
          const uint64_t v_desc = v_desc0 + (uint64_t)(slot * (S::KV_BYTES >> 4));
#pragma unroll
          for (int k4 = 0; k4 < kHalf / 16; ++k4)
            umma_ts(tmem_o, tmem_s + hb * kHalf + k4 * 8, v_desc + (((hb * (kHalf / 16) + k4) * (16 * 128)) >> 4), idesc_pv,
                    (hf | k4) != 0 ? 1u : 0u);
          umma_commit(&o_full[2 * st + hb]);
          if (hb == 1 || hf == n_half - 1) umma_commit(&v_empty[slot]);
        }
        __syncwarp();
        if (hf + 2 < n_half) issue_qk(hf + 2);          // in issue order behind the product that reads P(hf)
      }
    }
  } else if (warp >= 4 && st_active) {
    // ---- softmax of this tile: thread <-> query row (as in the kernel above, over every key block)
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float c = rsqrtf((float)HD) * 1.4426950408889634f;
    float m = -INFINITY, l = 0.f;
    // (the token whose cache row this thread writes at the end: asked for now, not in the epilogue)
    const int t_row = idx ? __ldcg(idx + row0 + st * BQ + (r < rows_valid ? r : 0)) : row0 + st * BQ + (r < rows_valid ? r : 0);
    const bool warp_has_rows = quarter * 32 < rows_valid;   // (else: pass the half blocks on; rows of no token, never stored)
    for (int hf = 0; hf < n_half; ++hf) {
      const uint32_t sbuf = tmem_s + (hf & 1) * kHalf + lane_addr;      // scores of half block hf, then its P
      mbar_wait(&s_full[2 * st + (hf & 1)], (hf >> 1) & 1, p.status);
      tc_fence_after();
      if (!warp_has_rows) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[2 * st + (hf & 1)]);
        continue;
      }

      if (dbg && hf == 0 && threadIdx.x == 128) p.debug[2] = globaltimer_ns();
      const int n_keys = min(kHalf, g.kv_len - hf * kHalf);
      float v[kHalf];
      tmem_ld_32x32_nowait(sbuf, v);
      tmem_ld_32x32_nowait(sbuf + 32, v + 32);
      tmem_ld_wait();
      if (n_keys < kHalf) {
#pragma unroll
        for (int i = 0; i < kHalf; ++i)
          if (i >= n_keys) v[i] = -INFINITY;
      }
      float mx4[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) mx4[k] = fmaxf(v[k], v[4 + k]);
#pragma unroll
      for (int i = 8; i < kHalf; i += 8) {
#pragma unroll
        for (int k = 0; k < 4; ++k) mx4[k] = fmax3(mx4[k], v[i + k], v[i + 4 + k]);
      }
      const float m_new = fmax3(m, fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      if (hf == 0) {
        m = m_new;
      } else {
        const bool grow = (m_new - m) * c > kRescaleStep;
        if (__any_sync(0xffffffffu, grow)) {
          const float alpha = grow ? fast_exp2((m - m_new) * c) : 1.f;
          if (grow) { m = m_new; l *= alpha; }
          // P(hf - 1) V has been added.  (The softmax warps may be two products ahead of the tensor core, and a
          // parity wait tells apart only two consecutive phases: hence one barrier per parity of hf, each of which
          // these warps are at most one phase behind.)
          mbar_wait(&o_full[2 * st + ((hf - 1) & 1)], ((hf - 1) >> 1) & 1, p.status);
          tc_fence_after();
#pragma unroll 1
          for (int ch = 0; ch < 4; ++ch) {
            float o[32];
            tmem_ld_32x32(tmem_o + lane_addr + ch * 32, o);
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] *= alpha;
            tmem_st_32x32(tmem_o + lane_addr + ch * 32, o);
          }
        }
      }
      const float2 c2 = make_float2(c, c), nmc2 = make_float2(-m * c, -m * c);
      float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      float pk[kHalf / 2];
#pragma unroll
      for (int i = 0; i < kHalf; i += 2) {
        float2 e = __ffma2_rn(make_float2(v[i], v[i + 1]), c2, nmc2);
        e.x = fast_exp2(e.x);
        e.y = fast_exp2(e.y);
        sum2[(i >> 1) & 1] = __fadd2_rn(sum2[(i >> 1) & 1], e);
        __nv_bfloat162 h2 = __floats2bfloat162_rn(e.x, e.y);
        pk[i >> 1] = __uint_as_float(*reinterpret_cast<uint32_t*>(&h2));
      }
      tmem_st_32x32_nowait(sbuf, pk);
      tmem_st_wait();
      l += (sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[2 * st + (hf & 1)]);
    }
    for (int hh = max(0, n_half - 2); hh < n_half; ++hh)       // the last two products
      mbar_wait(&o_full[2 * st + (hh & 1)], (hh >> 1) & 1, p.status);
    tc_fence_after();
    if (dbg && threadIdx.x == 128) p.debug[3] = globaltimer_ns();
    // ---- normalise and store this row (the tensor-memory loads are warp-wide; rows past the tile's end only skip
    // the store)
    {
      bool ok = r < rows_valid;
      const float inv = 1.f / l;
      int t = t_row;
      if (idx != nullptr && ok && !token_ok(t, g.tokens(), p.status)) { ok = false; t = 0; }   // no cache row to write
      if (idx == nullptr && store_mask != nullptr && ok && __ldcg(store_mask + g.cache_row(t)) != 0) ok = false;   // a reused row
      __nv_bfloat16* dst = p.oc + (size_t)g.cache_row(t) * g.d + h * HD;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        float o[32];
        tmem_ld_32x32(tmem_o + lane_addr + ch * 32, o);
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] *= inv;
        if (ok) {
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) reinterpret_cast<uint4*>(dst + ch * 32)[v4] = pack8_bf16(o + 8 * v4);
        }
      }
    }
  }
  }  // active
  tc_fence_before();
  __syncthreads();
  if (p.debug != nullptr && threadIdx.x == 0 && active) {
    const unsigned long long t_end = globaltimer_ns();
    if (dbg) p.debug[4] = t_end;
    atomicMax(&p.debug[5], t_start);
    atomicMax(&p.debug[6], t_end);
    atomicAdd(&p.debug[7], 1ull);
  }
  if (warp == 2) tmem_dealloc(tmem_base, kTmemCols);
}

namespace {
// -> two query tiles per CTA?  else *ksplit = key split of the one-tile kernel
bool pick_form(const StepGeom& g, bool row_sparse, int* ksplit_out) {
  const int tps = (g.seq_act + BQ - 1) / BQ;
  // CTAs expected to have work: every row tile (dense) or one row tile per sequence (row-sparse, small refresh set)
  const int expected = g.n_heads * g.batch * (row_sparse ? 1 : tps);
  const int n_blocks = (g.kv_len + BKV - 1) / BKV;
  // The merge of a key split costs about as much as four key blocks (three cluster-wide barriers and the copies), so
  // the keys are split only when every CTA still keeps at least four blocks.
  int ksplit = 1;
  while (ksplit < 4 && expected * ksplit * 2 <= 160 && ksplit * 2 * 4 <= n_blocks) ksplit *= 2;
  *ksplit_out = ksplit;
  // Many query rows per sequence (and enough work to fill the GPU without a key split): two tiles per CTA share
  // the key blocks.  A row-sparse launch cannot know the size of the refresh set; the window length decides: long
  // windows are where refresh sets of several tiles are.
  const int tps2 = (g.seq_act + kPairRows - 1) / kPairRows;
  return ksplit == 1 && (row_sparse ? g.seq_act >= kPairMinSparse && g.n_heads * g.batch >= 64
                                    : g.seq_act > kPairMinDense && g.n_heads * g.batch * tps2 >= 148);
}
}  // namespace

bool attention_tc_two_tiles(const StepGeom& g, bool row_sparse) {
  int ksplit;
  return pick_form(g, row_sparse, &ksplit);
}

cudaError_t launch_attention_tc(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnParams& p,
                                cudaStream_t st) {
  static std::atomic<unsigned long long> attr_one{0}, attr_pair{0};
  if (cudaError_t e = ensure_dyn_smem(attn_tc_kernel, AttnSmem::TOTAL, attr_one); e != cudaSuccess) return e;
  if (cudaError_t e = ensure_dyn_smem(attn_pair_kernel, PairSmem::TOTAL, attr_pair); e != cudaSuccess) return e;
  const int tps = (p.g.seq_act + BQ - 1) / BQ;
  const int tps2 = (p.g.seq_act + kPairRows - 1) / kPairRows;
  int ksplit = 1;
  const bool pair = pick_form(p.g, p.idx != nullptr, &ksplit);
  if (pair) {
    dim3 grid(p.g.n_heads, p.g.batch * tps2, 1);
    if (grid.y == 0) return cudaSuccess;
    return launch_pdl(attn_pair_kernel, grid, dim3(kThreads), PairSmem::TOTAL, st, 1, tm_k, tm_v, p);
  }
  dim3 grid(p.g.n_heads, p.g.batch * tps, ksplit);
  if (grid.y == 0) return cudaSuccess;
  return launch_pdl(attn_tc_kernel, grid, dim3(kThreads), AttnSmem::TOTAL, st, ksplit, tm_k, tm_v, p);
}

}  // namespace dare
