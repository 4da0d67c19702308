// Host side of the tensor-core path: TMA tensor maps and the per-step kernel sequence.
#include <new>
#include <stdlib.h>

#include "layer.h"
#include "tc.h"

namespace dare {

struct TcState {
  CUtensorMap a_xn, a_xg, a_oc;            // A operands, box 64 x 128
  CUtensorMap w_q, w_k, w_v, w_o;          // weights, box 64 x 64 (two boxes per 128-column tile)
  CUtensorMap w_k32, w_v32;                // weights, box 64 x 32 (two boxes per 64-column tile)
  CUtensorMap w_o128;                      // experiment: box 64 x 128
  CUtensorMap kc64, vc64;                  // K/V caches as attention operands, box 64 x 64
};

namespace {

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

}  // namespace

bool tc_supported(const dare_layer_config_t& c) {
  return c.dtype == DARE_BF16 && c.head_dim == 128 && c.d_model % 128 == 0;
}
size_t tc_maps_bytes() { return sizeof(TcState); }

dare_status_t tc_create(dare_layer* L) {
  TcState* s = new (std::nothrow) TcState();
  if (!s) return DARE_ERR_INVALID_ARG;
  const uint64_t Tm = (uint64_t)L->cfg.max_batch * L->cfg.max_seq, d = L->cfg.d_model;
  bool ok = make_map(&s->a_xn, L->buf.xn, Tm, d, 128) && make_map(&s->a_xg, L->buf.xg, Tm + 128, d, 128) &&
            make_map(&s->a_oc, L->buf.oc, Tm, d, 128) && make_map(&s->w_q, L->w.w_q, d, d, 64) &&
            make_map(&s->w_k, L->w.w_k, d, d, 64) && make_map(&s->w_v, L->w.w_v, d, d, 64) &&
            make_map(&s->w_o, L->w.w_o, d, d, 64) && make_map(&s->w_k32, L->w.w_k, d, d, 32) &&
            make_map(&s->w_v32, L->w.w_v, d, d, 32) && make_map(&s->kc64, L->buf.kc, Tm, d, 64) &&
            make_map(&s->vc64, L->buf.vc, Tm, d, 64) && make_map(&s->w_o128, L->w.w_o, d, d, 128);
  if (!ok) { delete s; return DARE_ERR_CUDA; }
  L->tc = s;
  return DARE_OK;
}

void tc_destroy(dare_layer* L) {
  delete L->tc;
  L->tc = nullptr;
}

dare_status_t step_tc(dare_layer* L, const void* x, const StepGeom& g, int mode, float tau, void* y, cudaStream_t st) {
  typedef __nv_bfloat16 bf16;
  const Buffers& B = L->buf;
  const TcState& S = *L->tc;
  const int T_ = g.tokens(), d = g.d;
  const bool has_prev = L->has_prev;
  const bool kv_sparse = has_prev && (mode & DARE_MODE_KV);
  const bool o_sparse = has_prev && (mode & DARE_MODE_O);
  const int tiles_per_seq = (g.seq_act + 127) / 128;
  const int m_tiles_dense = g.batch * tiles_per_seq;
  int launches = 0;
  cudaError_t e;

  GemmParams base;
  static const int rot_n = getenv("DARE_ROT_N") ? atoi(getenv("DARE_ROT_N")) : 0;
  static const int rot_m = getenv("DARE_ROT_M") ? atoi(getenv("DARE_ROT_M")) : 0;
  base.rot_n = rot_n; base.rot_m = rot_m; base.b_single = 0;
  static const int mma_rep = getenv("DARE_MMA_REP") ? atoi(getenv("DARE_MMA_REP")) : 1;
  base.mma_rep = mma_rep;
  static const int single = getenv("DARE_B_SINGLE") ? atoi(getenv("DARE_B_SINGLE")) : 0;
  base.K = d; base.m_total = T_; base.seq_act = g.seq_act; base.tiles_per_seq = tiles_per_seq;
  base.a_seq_stride = g.seq_act; base.a_row0 = 0; base.idx = nullptr; base.count = nullptr; base.g = g;
  base.hd_map = g.head_dim; base.n_split = 1 << 30; base.out0 = nullptr; base.out1 = nullptr; base.ld_out = d;
  base.out_is_cache = 0; base.rope = reinterpret_cast<const float2*>(B.rope_cs); base.q_prev = B.q_prev;
  base.q_prev_rows = L->cfg.max_batch * L->cfg.max_seq;
  base.scores = B.scores; base.has_prev = has_prev ? 1 : 0; base.status = B.status;
  base.debug = nullptr;
  unsigned long long* dbg = L->debug_on ? B.debug : nullptr;
  if (dbg) cudaMemsetAsync(dbg, 0, (64 + 3 * 1024) * sizeof(unsigned long long), st);

  prof_begin(L);
  // Alg. 1/2 line 1
  prof_mark(L, SLOT_NORM, st);
  launch_rmsnorm<bf16>((const bf16*)x, L->w.rms_gain, (bf16*)B.xn, T_, d, L->cfg.rms_eps, st); ++launches;
  // line 2 + line 3 + stored-query update + rotary embedding, one kernel
  {
    GemmParams p = base;
    p.out0 = (bf16*)B.q;
    p.debug = dbg;
    prof_mark(L, SLOT_Q_GEMM, st);
    e = launch_gemm_tc(128, EPI_Q, S.a_xn, S.w_q, S.w_q, p, d / 128, m_tiles_dense, st); ++launches;
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  }
  // lines 4-5 + Sec. 4
  prof_mark(L, SLOT_SELECT, st);
  launch_select(B.scores, tau, !has_prev || mode == DARE_MODE_DENSE, g, B.idx, B.count, B.batch_off, B.delta, B.status,
                st); ++launches;
  // K/V projection with rotary embedding and cache scatter
  if (kv_sparse) {
    prof_mark(L, SLOT_GATHER, st);
    launch_gather_rows<bf16>((const bf16*)B.xn, B.idx, B.count, (bf16*)B.xg, T_, d, st); ++launches;
    GemmParams p = base;
    p.idx = B.idx; p.count = B.count; p.n_split = d / 64;
    p.out0 = (bf16*)B.kc; p.out1 = (bf16*)B.vc; p.out_is_cache = 1;
    p.debug = dbg ? dbg + 8 : nullptr;
    prof_mark(L, SLOT_KV_GEMM, st);
    e = launch_gemm_tc(64, EPI_KV, S.a_xg, S.w_k32, S.w_v32, p, 2 * d / 64, (T_ + 127) / 128, st); ++launches;
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  } else {
    GemmParams p = base;
    p.n_split = d / 128;
    p.out0 = (bf16*)B.kc; p.out1 = (bf16*)B.vc; p.out_is_cache = 1;
    p.debug = dbg ? dbg + 8 : nullptr;
    prof_mark(L, SLOT_KV_GEMM, st);
    e = launch_gemm_tc(128, EPI_KV, S.a_xn, S.w_k, S.w_v, p, 2 * d / 128, m_tiles_dense, st); ++launches;
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  }
  // attention (row-sparse over the refresh set when O reuse is on)
  prof_mark(L, SLOT_ATTN, st);
  {
    AttnParams p;
    p.q = (const bf16*)B.q; p.oc = (bf16*)B.oc; p.idx = o_sparse ? B.idx : nullptr;
    p.batch_off = o_sparse ? B.batch_off : nullptr; p.g = g; p.status = B.status;
    p.debug = dbg ? dbg + 16 : nullptr;
    e = launch_attention_tc(S.kc64, S.vc64, p, st); ++launches;
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  }
  // output projection of every row of the window, read from the O cache
  {
    GemmParams p = base;
    static const int out_bn = getenv("DARE_OUT_BN") ? atoi(getenv("DARE_OUT_BN")) : 128;
    p.a_seq_stride = g.max_seq; p.a_row0 = g.pos_begin; p.hd_map = out_bn;
    p.out0 = (bf16*)y;
    p.debug = dbg ? dbg + 24 : nullptr;
    prof_mark(L, SLOT_OUT_GEMM, st);
    p.b_single = (single && out_bn == 128) ? 1 : 0;
    e = launch_gemm_tc(out_bn, EPI_OUT, S.a_oc, (out_bn == 256 || p.b_single) ? S.w_o128 : S.w_o, S.w_o, p, d / out_bn, m_tiles_dense, st); ++launches;
    if (e != cudaSuccess) return DARE_ERR_CUDA;
  }
  prof_end(L, st);
  L->last_launches = launches;
  if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
  return DARE_OK;
}

}  // namespace dare
