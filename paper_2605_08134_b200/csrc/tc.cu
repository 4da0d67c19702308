// Host side of the tensor-core path: TMA tensor maps and the per-step kernel sequence.
#include <new>

#include "layer.h"
#include "tc.h"

namespace dare {

struct TcState {
  CUtensorMap a_xn, a_oc;                  // A operands, box 64 x 128 rows
  CUtensorMap a_xg;                        // compact copy of a refresh set's rows (the input staging buffer, idle after RMSNorm)
  CUtensorMap w_q, w_k, w_v, w_o;          // weights, box 64 x 256 rows
  CUtensorMap w_k128, w_v128, w_q128, w_o128;   // weights, box 64 x 128 rows
  CUtensorMap w_q64, w_o64;                // weights, box 64 x 64 rows (narrow pair tiles)
  CUtensorMap kc64, vc64;                  // K/V caches as attention operands, box 64 x 128 rows (keys)
};

namespace {

bool use_pairs(int n_tiles, int m_tiles, int splits) { return pairs_pay(n_tiles, m_tiles, splits); }
// units (column tile x pair of row tiles) from which the two-CTA form of a listed launch runs: two rounds of the 74 clusters
constexpr int kPairUnitGate = 148;
bool use_persist(int n_tiles, int m_tiles, int splits) { return persist_pays(n_tiles, m_tiles, splits); }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Reduction splits for a launch with `tiles` output tiles: enough CTAs to cover the SMs, never more than the
// k-blocks or the scratch allow.
int pick_splits(int tiles, int kblocks) {
  int s = 1;
  while (s < 2 && tiles * s * 2 <= 160 && s * 2 <= kblocks) s *= 2;
  return s;
}

}  // namespace

// Row-major bf16 matrix [rows, cols]; box = 64 columns (128 bytes, the swizzle span) x box_rows rows.
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool tc_supported(const dare_layer_config_t& c) {
  return c.dtype == DARE_BF16 && c.head_dim == 128 && c.d_model % 256 == 0;
}
size_t tc_maps_bytes() { return sizeof(TcState); }

dare_status_t tc_create(dare_layer* L) {
  TcState* s = new (std::nothrow) TcState();
  if (!s) return DARE_ERR_INVALID_ARG;
  const uint64_t Tm = (uint64_t)L->cfg.max_batch * L->cfg.max_seq, d = L->cfg.d_model;
  bool ok = make_map(&s->a_xn, L->buf.xn, Tm, d, 128) && make_map(&s->a_xg, L->buf.x_stage, Tm, d, 128) &&
            make_map(&s->a_oc, L->buf.oc, Tm, d, 128) && make_map(&s->w_q, L->w.w_q, d, d, 256) &&
            make_map(&s->w_k, L->w.w_k, d, d, 256) && make_map(&s->w_v, L->w.w_v, d, d, 256) &&
            make_map(&s->w_o, L->w.w_o, d, d, 256) && make_map(&s->w_k128, L->w.w_k, d, d, 128) &&
            make_map(&s->w_v128, L->w.w_v, d, d, 128) && make_map(&s->w_q128, L->w.w_q, d, d, 128) &&
            make_map(&s->w_o128, L->w.w_o, d, d, 128) && make_map(&s->w_q64, L->w.w_q, d, d, 64) &&
            make_map(&s->w_o64, L->w.w_o, d, d, 64) && make_map(&s->kc64, L->buf.kc, Tm, d, 128) &&
            make_map(&s->vc64, L->buf.vc, Tm, d, 128);
  if (!ok) { delete s; return DARE_ERR_CUDA; }
  L->tc = s;
  return DARE_OK;
}

void tc_destroy(dare_layer* L) {
  delete L->tc;
  L->tc = nullptr;
}

dare_status_t step_tc(dare_layer* L, const void* x, const StepGeom& g, int mode, float tau, void* y, cudaStream_t st,
                      bool add_input) {
  typedef __nv_bfloat16 bf16;
  const Buffers& B = L->buf;
  const TcState& S = *L->tc;
  const int T_ = g.tokens(), d = g.d;
  const bool has_prev = L->has_prev;
  const bool kv_sparse = has_prev && (mode & DARE_MODE_KV);
  const bool o_sparse = has_prev && (mode & DARE_MODE_O);
  // the input staging buffer doubles as the compact copy of a refresh set's rows once x has been normalised; not
  // when x is still needed later (the residual of a transformer block reads it in the output projection)
  const bool compact_ok = !add_input || x != B.x_stage;
  const int tiles_per_seq = (g.seq_act + 127) / 128;
  const int m_tiles_dense = g.batch * tiles_per_seq;
  const int kblocks = d / 64;
  int launches = 0;
  cudaError_t e;

  GemmParams base;
  base.K = d; base.m_total = T_; base.seq_act = g.seq_act; base.tiles_per_seq = tiles_per_seq;
  base.a_seq_stride = g.seq_act; base.a_row0 = 0; base.idx = nullptr; base.count = nullptr; base.g = g;
  base.gather_src = nullptr; base.gather_cache_rows = 0; base.unit_gate = 0;
  base.n_split = 1 << 30; base.out0 = nullptr; base.out1 = nullptr; base.ld_out = d;
  base.out_is_cache = 0; base.resid = nullptr; base.ld_resid = 0; base.out_f32 = nullptr; base.b_pair = 0;
  base.rope = reinterpret_cast<const float2*>(B.rope_cs); base.q_prev = B.q_prev;
  base.scores = B.scores; base.has_prev = has_prev ? 1 : 0; base.status = B.status;
  base.debug = nullptr; base.wait_at_end = 0; base.loop_rows = 0; base.nt0 = 0;
  base.gate_count = nullptr; base.gate_lo = 0; base.gate_hi = 1 << 30; base.store_mask = nullptr;
  // Steps of many row tiles: from these refresh-set sizes on the dense forms of the K/V projection, of attention and of
  // the output projection (results kept for the refreshed rows only) are faster than the listed forms.  Measured on
  // the long-context sweep (batch 4 x 4096): the listed K/V projection with its compact copy passes the dense form's
  // time at about 78 % of the tokens, row-sparse attention + gathered output projection with its copy of the reused
  // rows at about 80 %, all of them together at about 85 %.
  const int gate_kv = (int)(0.75 * T_), gate_o = (int)(0.80 * T_);
  unsigned long long* dbg = L->debug_on ? B.debug : nullptr;
  // (no clearing between steps: a copy or memset in the stream would break the kernels' launch overlap; the stamps
  // are plain stores or maxima of a clock that only grows)

  prof_begin(L);
  // Alg. 1/2 line 1
  prof_mark(L, SLOT_NORM, st);
  launch_rmsnorm<bf16>((const bf16*)x, L->w.rms_gain, (bf16*)B.xn, T_, d, L->cfg.rms_eps, st, dbg ? dbg + 40 : nullptr);
  ++launches;
  // line 2 + line 3 + stored-query update + rotary embedding, one kernel
  {
    GemmParams p = base;
    p.out0 = (bf16*)B.q;
    p.debug = dbg;
    const int n_tiles = d / 256;
    prof_mark(L, SLOT_Q_GEMM, st);
    const int sp = pick_splits(n_tiles * m_tiles_dense, kblocks);
    if (narrow_pairs_pay(d, m_tiles_dense, kblocks))
      e = launch_gemm_tc(EPI_Q, 128, S.a_xn, S.w_q64, S.w_q64, p, d / 128, m_tiles_dense, 2, st, 1);
    else if (use_persist(n_tiles, m_tiles_dense, sp))
      e = launch_gemm_persist(EPI_Q, S.a_xn, S.w_q128, S.w_q128, p, n_tiles, m_tiles_dense, st, 1);
    else if (use_pairs(n_tiles, m_tiles_dense, sp))
      e = launch_gemm_tc(EPI_Q, 256, S.a_xn, S.w_q128, S.w_q128, p, n_tiles, m_tiles_dense, sp, st, 1);
    else
      e = launch_gemm_tc(EPI_Q, 256, S.a_xn, S.w_q, S.w_q, p, n_tiles, m_tiles_dense, sp, st);
    ++launches;
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  }
  // A dense K/V projection (Alg. 2 line 7, or the full forward of Appendix E.2) needs nothing from the Q projection
  // or the selection.  On a short step (launches of about one wave, where fixed costs and the hand-off between
  // kernels decide) it is issued right behind the Q projection and runs beside it: the two launches are one fused
  // Q/K/V projection of the step's rows, spread over two grids because the Q tiles take a split reduction and the
  // K/V tiles do not.  The selection then follows both.
  const bool kv_beside_q = !kv_sparse && m_tiles_dense <= 8;
  // lines 4-5 + Sec. 4
  const bool select_all = !has_prev || mode == DARE_MODE_DENSE;
  auto select_now = [&]() {
    prof_mark(L, SLOT_SELECT, st);
    // (a selection that refreshes everything reads no scores: behind the two projections it runs beside them)
    const float* tau_dev = step_threshold_on_device(L, g, mode, st, &launches);
    launch_select(B.scores, tau, select_all, g, B.idx, B.count, B.batch_off, B.delta, st, kv_beside_q && select_all, tau_dev);
    ++launches;
    if (L->inject) inject_selection_error(L, g, st);
  };
  if (!kv_beside_q) select_now();
  // K/V projection with rotary embedding and cache scatter
  {
    GemmParams p = base;
    p.n_split = d / 256;
    p.out0 = (bf16*)B.kc; p.out1 = (bf16*)B.vc; p.out_is_cache = 1;
    p.debug = dbg ? dbg + 8 : nullptr;
    const int n_tiles = 2 * d / 256;
    if (kv_sparse) {
      // Alg. 1 line 6: the projection fetches the refresh set's rows of x_norm by index as its A operand
      p.idx = B.idx; p.count = B.count; p.gather_src = (const bf16*)B.xn;
      const int m_tiles = (T_ + 127) / 128;
      prof_mark(L, SLOT_KV_GEMM, st);
      if (m_tiles <= 8) {
        // Few tokens: the refresh set fits one or two row tiles and the projection is a stream of the weights.
        // Narrower tiles put twice as many CTAs on it; the reduction split is sized for one row tile.
        p.n_split = d / 128;
        const int n_tiles128 = 2 * d / 128;
        p.loop_rows = 1;                         // one row of CTAs: no CTA that only looks at the count and leaves
        e = launch_gemm_tc(EPI_KV, 128, S.a_xn, S.w_k128, S.w_v128, p, n_tiles128, 1,
                           pick_splits(n_tiles128, kblocks), st); ++launches;
      } else {
        // Many tokens: even a small refreshed fraction fills the GPU with 256-wide tiles, which re-read the least.
        if (use_persist(n_tiles, m_tiles, 1) && compact_ok) {
          // a compact copy of the refresh set's rows first (a stream of n x d elements), then the projection with
          // every operand through TMA and two-CTA MMAs; beyond gate_kv refreshed tokens the dense form instead: every
          // row of the step projected, the rows of the refresh set stored (the others keep their cached K and V)
          const bool dense_form = use_persist(n_tiles, m_tiles_dense, 1);
          const int hi = dense_form ? gate_kv : 1 << 30;
          launch_gather_step_rows((const bf16*)B.xn, B.idx, B.count, (bf16*)B.x_stage, g, false, st, B.status, hi); ++launches;
          p.gather_src = nullptr;
          p.unit_gate = kPairUnitGate;
          p.gate_count = B.count; p.gate_hi = hi;
          e = launch_gemm_persist(EPI_KV, S.a_xg, S.w_k128, S.w_v128, p, n_tiles, m_tiles, st, 1); ++launches;
          if (e == cudaSuccess) e = launch_gemm_persist(EPI_KV, S.a_xg, S.w_k, S.w_v, p, n_tiles, m_tiles, st, 0);
          if (dense_form && e == cudaSuccess) {
            GemmParams pd = p;
            pd.idx = nullptr; pd.count = nullptr; pd.unit_gate = 0;
            pd.gate_lo = gate_kv; pd.gate_hi = 1 << 30; pd.store_mask = B.delta;
            ++launches;
            e = launch_gemm_persist(EPI_KV, S.a_xn, S.w_k128, S.w_v128, pd, n_tiles, m_tiles_dense, st, 1);
          }
        } else
          e = launch_gemm_tc(EPI_KV, 256, S.a_xn, S.w_k, S.w_v, p, n_tiles, m_tiles, 1, st);
        ++launches;
      }
    } else {
      prof_mark(L, SLOT_KV_GEMM, st);
      p.wait_at_end = kv_beside_q ? 1 : 0;
      const int sp = pick_splits(n_tiles * m_tiles_dense, kblocks);
      if (use_persist(n_tiles, m_tiles_dense, sp))
        e = launch_gemm_persist(EPI_KV, S.a_xn, S.w_k128, S.w_v128, p, n_tiles, m_tiles_dense, st, 1);
      else if (use_pairs(n_tiles, m_tiles_dense, sp))
        e = launch_gemm_tc(EPI_KV, 256, S.a_xn, S.w_k128, S.w_v128, p, n_tiles, m_tiles_dense, sp, st, 1);
      else
        e = launch_gemm_tc(EPI_KV, 256, S.a_xn, S.w_k, S.w_v, p, n_tiles, m_tiles_dense, sp, st);
      ++launches;
    }
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  }
  if (kv_beside_q) select_now();
  // attention (row-sparse over the refresh set when O reuse is on)
  prof_mark(L, SLOT_ATTN, st);
  {
    AttnParams p;
    p.q = (const bf16*)B.q; p.oc = (bf16*)B.oc; p.idx = o_sparse ? B.idx : nullptr;
    p.batch_off = o_sparse ? B.batch_off : nullptr; p.g = g; p.status = B.status;
    p.debug = dbg ? dbg + 16 : nullptr;
    // the refresh set then comes from the kernel right before; or the two kernels before ran beside the Q projection
    // without waiting for it, so the queries are not known to be complete before this kernel's own wait
    p.wait_first = kv_beside_q ? 1 : 0;
    p.gate_count = nullptr; p.gate_lo = 0; p.gate_hi = 1 << 30; p.store_mask = nullptr;
    // a long row-sparse step is issued in both forms: over the refresh set's rows, and dense with only the refreshed
    // rows stored (tiles without one skipped); the size of the set decides on the device which of them runs
    const bool both_forms = o_sparse && m_tiles_dense > 8 && use_persist(d / 256, m_tiles_dense, 1);
    // (one launch carries both when both take the kernel with two query tiles per CTA: its CTAs pick the form; a
    // launch that only looks at the count and leaves still costs a wave of CTAs per 148 of them)
    const bool one_launch = both_forms && attention_tc_two_tiles(g, true) && attention_tc_two_tiles(g, false);
    p.dense_from = 0; p.dense_mask = nullptr;
    if (both_forms) {
      p.gate_count = B.count;
      if (one_launch) { p.dense_from = gate_o; p.dense_mask = B.delta; }
      else p.gate_hi = gate_o;
    }
    e = launch_attention_tc(S.kc64, S.vc64, p, st); ++launches;
    if (both_forms && !one_launch && e == cudaSuccess) {
      AttnParams pd = p;
      pd.idx = nullptr; pd.batch_off = nullptr; pd.debug = nullptr;
      pd.gate_lo = gate_o; pd.gate_hi = 1 << 30; pd.store_mask = B.delta;
      e = launch_attention_tc(S.kc64, S.vc64, pd, st); ++launches;
    }
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  }
  // Output projection, read from the O cache.  Alg. 2 line 11 projects every row of the window.  A row whose
  // attention output was reused projects to what it projected to before (W_O acts row by row), so with many tokens
  // the library keeps those projections by cache row and, on a step that reuses attention outputs, projects the
  // refresh set's rows only (fetched from the O cache by index, like the rows of the gathered K/V projection) and
  // copies the others.  With few tokens the projection is a stream of W_O whatever the row count, and stays dense.
  {
    const bool many = m_tiles_dense > 8 && !add_input;
    const bool y_sparse = o_sparse && many && L->yc_valid;
    GemmParams p = base;
    p.a_seq_stride = g.max_seq; p.a_row0 = g.pos_begin;
    p.out0 = (bf16*)y;
    if (many) p.out1 = (bf16*)B.yc;                                   // kept by cache row for later steps
    if (add_input) { p.resid = (const bf16*)x; p.ld_resid = d; }      // y = x + W_O O (residual block)
    p.debug = dbg ? dbg + 24 : nullptr;
    const int n_tiles = d / 256;
    prof_mark(L, SLOT_OUT_GEMM, st);
    if (y_sparse) {
      p.idx = B.idx; p.count = B.count; p.gather_src = (const bf16*)B.oc; p.gather_cache_rows = 1;
      bool dense_form = false;
      if (use_persist(n_tiles, (T_ + 127) / 128, 1) && compact_ok) {
        // (beyond gate_o refreshed tokens the dense projection of every row instead: Alg. 2 line 11 as written)
        dense_form = use_persist(n_tiles, m_tiles_dense, 1);
        const int hi = dense_form ? gate_o : 1 << 30;
        launch_gather_step_rows((const bf16*)B.oc, B.idx, B.count, (bf16*)B.x_stage, g, true, st, B.status, hi); ++launches;
        p.gather_src = nullptr;
        p.unit_gate = kPairUnitGate;
        p.gate_count = B.count; p.gate_hi = hi;
        e = launch_gemm_persist(EPI_OUT, S.a_xg, S.w_o128, S.w_o128, p, n_tiles, (T_ + 127) / 128, st, 1); ++launches;
        if (e == cudaSuccess) e = launch_gemm_persist(EPI_OUT, S.a_xg, S.w_o, S.w_o, p, n_tiles, (T_ + 127) / 128, st, 0);
        if (dense_form && e == cudaSuccess) {
          GemmParams pd = p;
          pd.idx = nullptr; pd.count = nullptr; pd.unit_gate = 0; pd.gather_cache_rows = 0;
          pd.gate_lo = gate_o; pd.gate_hi = 1 << 30;
          ++launches;
          e = launch_gemm_persist(EPI_OUT, S.a_oc, S.w_o128, S.w_o128, pd, n_tiles, m_tiles_dense, st, 1);
        }
      } else
        e = launch_gemm_tc(EPI_OUT, 256, S.a_oc, S.w_o, S.w_o, p, n_tiles, (T_ + 127) / 128, 1, st);
      ++launches;
      if (e != cudaSuccess) return DARE_ERR_CUDA;
      launch_copy_reused_rows((const bf16*)B.yc, (bf16*)y, B.delta, g, st, dense_form ? B.count : nullptr, gate_o); ++launches;
    } else {
      const int sp = pick_splits(n_tiles * m_tiles_dense, kblocks);
      if (narrow_pairs_pay(d, m_tiles_dense, kblocks))
        e = launch_gemm_tc(EPI_OUT, 128, S.a_oc, S.w_o64, S.w_o64, p, d / 128, m_tiles_dense, 2, st, 1);
      else if (use_persist(n_tiles, m_tiles_dense, sp))
        e = launch_gemm_persist(EPI_OUT, S.a_oc, S.w_o128, S.w_o128, p, n_tiles, m_tiles_dense, st, 1);
      else if (use_pairs(n_tiles, m_tiles_dense, sp))
        e = launch_gemm_tc(EPI_OUT, 256, S.a_oc, S.w_o128, S.w_o128, p, n_tiles, m_tiles_dense, sp, st, 1);
      else
        e = launch_gemm_tc(EPI_OUT, 256, S.a_oc, S.w_o, S.w_o, p, n_tiles, m_tiles_dense, sp, st);
      ++launches;
      if (e != cudaSuccess) return DARE_ERR_CUDA;
      // the cache is complete once a dense projection has covered every cached row, and stays so while every
      // later step maintains it
      if (many) {
        if (g.pos_begin == 0 && g.seq_act == g.kv_len) L->yc_valid = true;
      } else {
        L->yc_valid = false;
      }
    }
  }
  prof_end(L, st);
  L->last_launches = launches;
  if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
  return DARE_OK;
}

}  // namespace dare
