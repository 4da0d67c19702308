// Bidirectional (no mask) softmax attention on tcgen05 tensor cores, head_dim = 128, bf16 operands, fp32 softmax.
//   dense      : every query row of the step window                       (Alg. 1 line 10)
//   row-sparse : only the query rows of the refresh set, gathered by index (Alg. 2 lines 6, 8; Eq. 4)
// The result rows are written straight into the attention-output cache at their cache rows; rows that are not
// computed keep their cached value (Alg. 2 lines 9-10).
//
// One CTA = one head x one tile of up to 128 query rows of one sequence, walking the keys in blocks of 128:
//   warp 0       TMA producer: K block and V block of the cache (two 64-column boxes each, 128-byte swizzle),
//                double buffered
//   warp 1       one thread issues S(i) = Q K(i)^T (M128 N128 K16 x 8) into tensor memory; S is double buffered there
//                and S(i+1) is issued as soon as S(i-1) has been read, so the tensor pipe works on O_blk(i-1) and
//                S(i+1) while the softmax warps are on S(i)
//   warp 2       one thread issues O_blk(i) = P(i) V(i) (M128 N128 K16 x 8, V as an MN-major operand); a warp of its
//                own because issuing eight MMAs next to busy softmax warps takes longer than executing them
//   warps 3-10   softmax: thread <-> (query row, half): each reads its 64 of the row's 128 scores from tensor memory,
//                the two halves agree on the running maximum through shared memory; each exponentiates its keys,
//                writes them as bf16 into the swizzled P tile in shared memory, and rescales/accumulates its 64 of
//                the 128 output columns in registers (the product of block i-1 is folded in after the exponentials
//                of block i).
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
  static constexpr int P_BYTES = BQ * BKV * 2;         // two 64-key chunks of [128 x 128 B]
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_OFF + Q_BYTES;        // 2 buffers
  static constexpr int V_OFF = K_OFF + 2 * K_BYTES;    // 2 buffers
  static constexpr int P_OFF = V_OFF + 2 * V_BYTES;
  static constexpr int L_OFF = P_OFF + P_BYTES;        // float[2][128] partial row sums
  static constexpr int MX_OFF = L_OFF + 2 * BQ * 4;     // float[2][2][128] half-row maxima, by key-block parity
  static constexpr int BAR_OFF = MX_OFF + 4 * BQ * 4;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;
  // after the key loop the operand buffers are idle; the merge of a key split reuses them:
  static constexpr int DUMP_OFF = 0;                   // this CTA's accumulator [128 rows][128 cols] fp32, 64 KB
  static constexpr int STAT_OFF = DUMP_OFF + BQ * HD * 4;   // running maximum [128], row sum [128]
  static constexpr int RECV_OFF = STAT_OFF + 2 * BQ * 4;    // up to 3 senders x (rows x 512 B + rows x 8 B)
};

// 2^x for x <= 0 on the special-function unit; results below the normal range flush to zero (they are softmax
// weights 2^-126 times smaller than the row's largest).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

constexpr int kThreads = 352;
constexpr int kSoftmaxThreads = 256;
constexpr uint32_t kTmemCols = 512;     // S of even / odd key blocks: columns [0, 128) / [128, 256); O_blk: [256, 384)

}  // namespace

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const AttnParams p) {
  using S = AttnSmem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::BAR_OFF);
  uint64_t* k_full = bars;          // [2]
  uint64_t* v_full = bars + 2;      // [2]
  uint64_t* k_empty = bars + 4;     // [2]
  uint64_t* v_empty = bars + 6;     // [2]
  uint64_t* s_full = bars + 8;      // [2]
  uint64_t* s_free = bars + 10;     // [2]
  uint64_t* p_full = bars + 12;
  uint64_t* o_full = bars + 13;
  uint64_t* recv_bar = bars + 14;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 15);
  float* l_part = reinterpret_cast<float*>(smem + S::L_OFF);
  float* mx_part = reinterpret_cast<float*>(smem + S::MX_OFF);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.x;
  const int ksplit = gridDim.z;                      // = cluster size along z
  const int z = ksplit > 1 ? (int)cluster_ctarank() : 0;
  const int rows_own = BQ / ksplit;                   // rows of the tile this CTA writes out
  const bool dbg = p.debug != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
  if (dbg && threadIdx.x == 0) p.debug[0] = globaltimer_ns();
  const StepGeom& g = p.g;
  // blockIdx.y = tile * batch + b: the first row tile of every sequence comes first in launch order, so that in the
  // row-sparse case the CTAs that have work are scheduled before the (many) tiles past the refresh set
  const int tile = blockIdx.y / g.batch, b = blockIdx.y - tile * g.batch;

  // Row tiles past the first one of a sequence are usually empty in the row-sparse case: they look at the refresh
  // set before spending anything on set-up.
  if (p.idx != nullptr && tile > 0) {
    pdl_wait();
    if (p.batch_off[b] + tile * BQ >= p.batch_off[b + 1]) return;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&v_full[i], 1); mbar_init(&k_empty[i], 1); mbar_init(&v_empty[i], 1);
      mbar_init(&s_full[i], 1); mbar_init(&s_free[i], kSoftmaxThreads / 32);
    }
    mbar_init(p_full, kSoftmaxThreads / 32);
    mbar_init(o_full, 1);
    mbar_init(recv_bar, 1);
    fence_mbar_init();
    if (ksplit > 1) mbar_arrive_expect_tx(recv_bar, (uint32_t)((ksplit - 1) * rows_own * (HD * 4 + 8)));
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  // The set-up above overlapped the tail of the previous kernel in the stream; its results are needed from here on.
  pdl_wait();
  pdl_launch_dependents();
  // ---- rows of this tile (uniform over the CTA)
  int row0 = 0, rows_valid = 0;
  bool active = true;
  if (p.idx != nullptr) {
    const int lo = p.batch_off[b], hi = p.batch_off[b + 1];
    row0 = lo + tile * BQ;
    active = row0 < hi;
    rows_valid = min(BQ, hi - row0);
  } else {
    row0 = b * g.seq_act + tile * BQ;
    rows_valid = min(BQ, g.seq_act - tile * BQ);
  }
  const int n_blocks_all = (g.kv_len + BKV - 1) / BKV;
  const int n_blocks = n_blocks_all > z ? (n_blocks_all - z + ksplit - 1) / ksplit : 0;   // blocks z, z + ksplit, ...
  const int kv_row0 = b * g.max_seq;
  // ---- Q tile: gathered rows -> shared memory in the K-major 128-byte-swizzled layout (16-byte units)
  {
    uint8_t* qs = smem + S::Q_OFF;
    for (int u = threadIdx.x; active && u < BQ * 16; u += kThreads) {
      const int r = u >> 4, unit = u & 15;           // 16 units of 8 bf16 per row
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < rows_valid) {
        const int t = p.idx ? p.idx[row0 + r] : row0 + r;
        v = *reinterpret_cast<const uint4*>(p.q + (size_t)t * g.d + h * HD + unit * 8);
      }
      const int chunk = unit >> 3, uc = unit & 7;
      *reinterpret_cast<uint4*>(qs + chunk * (BQ * 128) + r * 128 + ((uc ^ (r & 7)) << 4)) = v;
    }
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 2 * BKV;
  if (dbg && threadIdx.x == 0) p.debug[1] = globaltimer_ns();

  if (active) {
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < n_blocks; ++i) {
        const int buf = i & 1;
        uint8_t* kd = smem + S::K_OFF + buf * S::K_BYTES;
        uint8_t* vd = smem + S::V_OFF + buf * S::V_BYTES;
        const int row = kv_row0 + (z + i * ksplit) * BKV;
        mbar_wait(&k_empty[buf], ((i >> 1) & 1) ^ 1, p.status);     // S(i-2) = Q K(i-2)^T has been computed
        mbar_arrive_expect_tx(&k_full[buf], S::K_BYTES);
        tma_load_2d(kd, &tm_k, h * HD, row, &k_full[buf]);
        tma_load_2d(kd + S::K_BYTES / 2, &tm_k, h * HD + 64, row, &k_full[buf]);
        mbar_wait(&v_empty[buf], ((i >> 1) & 1) ^ 1, p.status);     // O_blk(i-2) = P(i-2) V(i-2) has been computed
        mbar_arrive_expect_tx(&v_full[buf], S::V_BYTES);
        tma_load_2d(vd, &tm_v, h * HD, row, &v_full[buf]);
        tma_load_2d(vd + S::V_BYTES / 2, &tm_v, h * HD + 64, row, &v_full[buf]);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- S(i) = Q K(i)^T, issued as soon as the softmax warps have read S(i-2) out of its buffer: while they work
    // on S(i) the tensor pipe computes O_blk(i-1) and S(i+1)
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_bf16(BQ, BKV, false);
      const uint64_t q_desc = smem_desc_k_sw128(smem_u32(smem + S::Q_OFF));
      for (int i = 0; i < n_blocks; ++i) {
        const int buf = i & 1;
        if (i >= 2) mbar_wait(&s_free[buf], ((i >> 1) - 1) & 1, p.status);
        mbar_wait(&k_full[buf], (i >> 1) & 1, p.status);
        tc_fence_after();
        const uint64_t k_desc = smem_desc_k_sw128(smem_u32(smem + S::K_OFF + buf * S::K_BYTES));
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk)
          umma_ss(tmem_s + buf * BKV, q_desc + (((kk >> 2) * (BQ * 128) + (kk & 3) * 32) >> 4),
                  k_desc + (((kk >> 2) * (BKV * 128) + (kk & 3) * 32) >> 4), idesc_qk, kk != 0 ? 1u : 0u);
        umma_commit(&s_full[buf]);
        umma_commit(&k_empty[buf]);
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ---- O_blk(i) = P(i) V(i), from its own warp so that its issue does not queue behind the score products'
    if (lane == 0) {
      constexpr uint32_t idesc_pv = idesc_bf16(BQ, HD, true);
      const uint64_t p_desc = smem_desc_k_sw128(smem_u32(smem + S::P_OFF));
      for (int i = 0; i < n_blocks; ++i) {
        const int buf = i & 1;
        // P(i) is in shared memory and O_blk(i-1) has been read out of tensor memory
        mbar_wait(p_full, i & 1, p.status);
        mbar_wait(&v_full[buf], (i >> 1) & 1, p.status);
        tc_fence_after();
        const uint64_t v_desc = smem_desc_mn_sw128(smem_u32(smem + S::V_OFF + buf * S::V_BYTES), BKV * 128);
#pragma unroll
        for (int ks = 0; ks < BKV / 16; ++ks)
          umma_ss(tmem_o, p_desc + (((ks >> 2) * (BQ * 128) + (ks & 3) * 32) >> 4), v_desc + ((ks * (16 * 128)) >> 4),
                  idesc_pv, ks != 0 ? 1u : 0u);
        umma_commit(o_full);
        umma_commit(&v_empty[buf]);
      }
    }
    __syncwarp();
  } else {
    // ---- softmax and output accumulation
    const int sw = warp - 3;                    // 0..7
    const int half = sw >> 2;                   // which 32 keys of a block / which 64 output columns
    const int quarter = warp & 3;               // TMEM lane quarter of this warp
    const int r = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float c = rsqrtf((float)HD) * 1.4426950408889634f;   // softmax scale folded into the exp2 argument
    float m = -INFINITY, l = 0.f, alpha_prev = 1.f;
    float acc[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) acc[i] = 0.f;
    uint8_t* ps = smem + S::P_OFF;

    for (int i = 0; i < n_blocks; ++i) {
      const uint32_t tmem_si = tmem_s + (i & 1) * BKV;
      mbar_wait(&s_full[i & 1], (i >> 1) & 1, p.status);
      tc_fence_after();
      if (dbg && i == 0 && threadIdx.x == 96) p.debug[2] = globaltimer_ns();
      const int key0 = (z + i * ksplit) * BKV;
      const bool ragged = key0 + BKV > g.kv_len;      // last block: keys past kv_len do not exist
      float s_mine[64];
      {
        float t0_[32], t1_[32];
        tmem_ld_32x32(tmem_si + lane_addr + half * 64, t0_);
        tmem_ld_32x32(tmem_si + lane_addr + half * 64 + 32, t1_);
#pragma unroll
        for (int j = 0; j < 32; ++j) { s_mine[j] = t0_[j]; s_mine[32 + j] = t1_[j]; }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_free[i & 1]);            // this warp's part of S(i) is in registers
      if (ragged) {
#pragma unroll
        for (int j = 0; j < 64; ++j)
          if (key0 + half * 64 + j >= g.kv_len) s_mine[j] = -INFINITY;
      }
      // row maximum: four independent chains over this half, then the other half's through shared memory (the two
      // threads of a row sit in the two warps of one tensor-memory lane quarter and meet on that quarter's barrier)
      float mx4[4] = {s_mine[0], s_mine[1], s_mine[2], s_mine[3]};
#pragma unroll
      for (int j = 4; j < 64; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], s_mine[j]);
      const float mx_half = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      float* mxp = mx_part + (i & 1) * 2 * BQ;
      mxp[half * BQ + r] = mx_half;
      asm volatile("bar.sync %0, 64;" ::"r"(2 + quarter) : "memory");
      const float mx = fmaxf(m, fmaxf(mx_half, mxp[(half ^ 1) * BQ + r]));
      const float alpha = fast_exp2((m - mx) * c);
      m = mx;
      const float mc = mx * c;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < 64; ++j) {
        s_mine[j] = fast_exp2(fmaf(s_mine[j], c, -mc));
        sum4[j & 3] += s_mine[j];
      }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l = l * alpha + sum;
      uint4 pk[8];
#pragma unroll
      for (int v = 0; v < 8; ++v) pk[v] = pack8_bf16(s_mine + 8 * v);
      // The previous block's product has had the whole softmax above to finish: fold it into the accumulator (its
      // completion also frees the P tile).
      if (i > 0) {
        mbar_wait(o_full, (i - 1) & 1, p.status);
        tc_fence_after();
#pragma unroll
        for (int cgrp = 0; cgrp < 2; ++cgrp) {
          float o[32];
          tmem_ld_32x32(tmem_o + lane_addr + half * 64 + cgrp * 32, o);
#pragma unroll
          for (int j = 0; j < 32; ++j) acc[cgrp * 32 + j] = fmaf(acc[cgrp * 32 + j], alpha_prev, o[j]);
        }
      }
      alpha_prev = alpha;
      // P row segment: this half's 64 keys are one 128-byte row of 64-key chunk `half`, 8 swizzled 16-byte units
#pragma unroll
      for (int v = 0; v < 8; ++v)
        *reinterpret_cast<uint4*>(ps + half * (BQ * 128) + r * 128 + ((v ^ (r & 7)) << 4)) = pk[v];
      fence_proxy_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full);
    }
    if (n_blocks > 0) {
      mbar_wait(o_full, (n_blocks - 1) & 1, p.status);
      tc_fence_after();
#pragma unroll
      for (int cgrp = 0; cgrp < 2; ++cgrp) {
        float o[32];
        tmem_ld_32x32(tmem_o + lane_addr + half * 64 + cgrp * 32, o);
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[cgrp * 32 + j] = fmaf(acc[cgrp * 32 + j], alpha_prev, o[j]);
      }
    }
    if (dbg && threadIdx.x == 96) p.debug[3] = globaltimer_ns();
    // ---- combine the two halves' row sums
    l_part[half * BQ + r] = l;
    asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");
    const float l_row = l_part[r] + l_part[BQ + r];
    if (ksplit == 1) {
      // normalise, store
      const float inv = 1.f / l_row;
      if (r < rows_valid) {
        const int t = p.idx ? p.idx[row0 + r] : row0 + r;
        __nv_bfloat16* dst = p.oc + (size_t)g.cache_row(t) * g.d + h * HD + half * 64;
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] *= inv;
#pragma unroll
        for (int v = 0; v < 8; ++v) reinterpret_cast<uint4*>(dst)[v] = pack8_bf16(acc + 8 * v);
      }
    } else {
      // key split: leave the un-normalised row, its maximum and its sum in shared memory for the merge
      asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");      // every l_part read is done
      float* dump = reinterpret_cast<float*>(smem + S::DUMP_OFF) + (size_t)r * HD;
#pragma unroll
      for (int v = 0; v < 16; ++v) {
        const int unit = half * 16 + v;                  // 32 sixteen-byte units per 512-byte row, XOR-swizzled
        *reinterpret_cast<float4*>(dump + ((unit ^ (r & 7)) << 2)) =
            make_float4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
      }
      if (half == 0) {
        float* stat = reinterpret_cast<float*>(smem + S::STAT_OFF);
        stat[r] = m;
        stat[BQ + r] = l_row;
      }
      fence_proxy_async_smem();
    }
  }
  if (ksplit > 1) {
    // ---- merge of the key split (all warps)
    __syncthreads();
    tc_fence_before();
    cluster_sync_all();                                  // every CTA of the cluster is past its key loop
    tc_fence_after();
    if (warp == 3 && lane < ksplit && lane != z) {
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
      const int t = p.idx ? p.idx[row0 + r] : row0 + r;
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
  if (ksplit > 1) cluster_sync_all(); else __syncthreads();
  if (dbg && threadIdx.x == 0) p.debug[4] = globaltimer_ns();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

cudaError_t launch_attention_tc(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnParams& p,
                                cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem::TOTAL);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int tps = (p.g.seq_act + BQ - 1) / BQ;
  // CTAs expected to have work: every row tile (dense) or one row tile per sequence (row-sparse, small refresh set)
  const int expected = p.g.n_heads * p.g.batch * (p.idx ? 1 : tps);
  const int n_blocks = (p.g.kv_len + BKV - 1) / BKV;
  // The merge of a key split costs about as much as four key blocks (three cluster-wide barriers and the copies), so
  // the keys are split only when every CTA still keeps at least four blocks.
  int ksplit = 1;
  while (ksplit < 4 && expected * ksplit * 2 <= 160 && ksplit * 2 * 4 <= n_blocks) ksplit *= 2;
  dim3 grid(p.g.n_heads, p.g.batch * tps, ksplit);
  if (grid.y == 0) return cudaSuccess;
  return launch_pdl(attn_tc_kernel, grid, dim3(kThreads), AttnSmem::TOTAL, st, ksplit, tm_k, tm_v, p);
}

}  // namespace dare
