// A stack of DARE attention layers inside pre-norm SwiGLU blocks, and block-wise greedy decoding (dare_stack.h).
// Everything heavy reuses the layer step and the tensor-core GEMM; this file adds the glue kernels (embedding
// gather, candidate list, per-row softmax statistics, choice) and the per-step kernel sequence.
#include <math.h>
#include <new>
#include <string.h>
#include <vector>

#include "dare_stack.h"
#include "layer.h"
#include "tc.h"

using namespace dare;

namespace dare {
dare_status_t layer_enqueue(dare_layer* L, const void* x, int batch, int seq_act, int pos_begin, int mode, float tau,
                            void* y, cudaStream_t st, bool add_input);
}

namespace {

typedef __nv_bfloat16 bf16;
constexpr uint32_t kStackMagic = 0x57AC4DA2u;
constexpr size_t kAlign = 256;
constexpr int kMaxCand = 128;       // candidates per decoding step: batch * block <= 128

size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct BlockMaps { CUtensorMap w_gate, w_up, w_down, w_down128, w_down64; };   // w_down: 256-row boxes, w_down64: 64, the others 128

// x[t, :] = emb[tokens[b, pos_begin + i], :]   (t = b*seq_act + i)
__global__ void __launch_bounds__(256) embed_kernel(const int* __restrict__ tokens, int seq_total, int seq_act,
                                                    int pos_begin, const uint4* __restrict__ emb, uint4* __restrict__ x,
                                                    int row_vecs, int vocab) {
  const int t = blockIdx.x;
  const int b = t / seq_act, i = t - b * seq_act;
  int id = tokens[(size_t)b * seq_total + pos_begin + i];
  id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
  const uint4* src = emb + (size_t)id * row_vecs;
  uint4* dst = x + (size_t)t * row_vecs;
  for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) dst[v] = src[v];
}

// Masked positions of the active block, ascending per sequence: cand_row = row of the window's hidden states,
// cand_pos = position, cand_off[b] = start of sequence b's slice.  One warp per sequence (block <= 32).
__global__ void cand_kernel(const int* __restrict__ tokens, int batch, int seq_total, int lo, int hi, int mask_id,
                            int pos_begin, int seq_act, int* __restrict__ cand_row, int* __restrict__ cand_pos,
                            int* __restrict__ cand_off, int* __restrict__ cand_count) {
  __shared__ int cnt[32];
  const int b = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pos = lo + lane;
  const bool is = b < batch && pos < hi && tokens[(size_t)b * seq_total + pos] == mask_id;
  const unsigned bal = __ballot_sync(0xffffffffu, is);
  if (lane == 0 && b < 32) cnt[b] = __popc(bal);
  __syncthreads();
  int off = 0;
  for (int k = 0; k < b; ++k) off += cnt[k];
  if (is) {
    const int o = off + __popc(bal & ((1u << lane) - 1u));
    cand_row[o] = b * seq_act + pos - pos_begin;
    cand_pos[o] = pos;
  }
  if (lane == 0 && b < batch) cand_off[b] = off;
  if (threadIdx.x == 0) {
    int tot = 0;
    for (int k = 0; k < batch; ++k) tot += cnt[k];
    cand_off[batch] = tot;
    *cand_count = tot;
  }
}

// Per candidate row of the logits: argmax (lowest index on ties, the mask id excluded) and its softmax probability.
// One pass over the row: every thread keeps a running maximum (with its index) and the sum of exp(v - maximum),
// rescaled when the maximum moves; the triples are then merged over the warp and the CTA.
struct RowStat {
  float m, s;
  int arg;
};
__device__ __forceinline__ void stat_add(RowStat& a, float v, int j) {
  if (v > a.m) {
    a.s = a.s * __expf(a.m - v) + 1.f;      // (exp(-inf) = 0 covers the first element)
    a.m = v; a.arg = j;
  } else {
    a.s += __expf(v - a.m);
  }
}
__device__ __forceinline__ void stat_merge(RowStat& a, float om, float os, int oa) {
  const bool take = om > a.m || (om == a.m && oa < a.arg);
  const float M = fmaxf(a.m, om);
  const float sa = a.m == -INFINITY ? 0.f : a.s * __expf(a.m - M), sb = om == -INFINITY ? 0.f : os * __expf(om - M);
  a.s = sa + sb; a.m = M;
  if (take) a.arg = oa;
}
__global__ void __launch_bounds__(1024) rowstats_kernel(const float* __restrict__ logits, const int* __restrict__ count,
                                                        int vocab, int mask_id, int* __restrict__ tok,
                                                        float* __restrict__ prob) {
  __shared__ float s_max[32], s_sum[32];
  __shared__ int s_arg[32];
  const int r = blockIdx.x;
  if (r >= *count) return;
  const float* row = logits + (size_t)r * vocab;
  RowStat a{-INFINITY, 0.f, 0x7fffffff};
  if ((vocab & 3) == 0) {                                   // rows then start on 16-byte boundaries
    const float4* row4 = reinterpret_cast<const float4*>(row);
    for (int j4 = threadIdx.x; j4 < vocab / 4; j4 += blockDim.x) {
      const float4 v = row4[j4];
      const int j = 4 * j4;
      if (j != mask_id) stat_add(a, v.x, j);
      if (j + 1 != mask_id) stat_add(a, v.y, j + 1);
      if (j + 2 != mask_id) stat_add(a, v.z, j + 2);
      if (j + 3 != mask_id) stat_add(a, v.w, j + 3);
    }
  } else {
    for (int j = threadIdx.x; j < vocab; j += blockDim.x)
      if (j != mask_id) stat_add(a, row[j], j);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, a.m, o), os = __shfl_xor_sync(0xffffffffu, a.s, o);
    const int oa = __shfl_xor_sync(0xffffffffu, a.arg, o);
    stat_merge(a, om, os, oa);
  }
  if (lane == 0) { s_max[warp] = a.m; s_sum[warp] = a.s; s_arg[warp] = a.arg; }
  __syncthreads();
  if (warp == 0) {
    a.m = s_max[lane]; a.s = s_sum[lane]; a.arg = s_arg[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, a.m, o), os = __shfl_xor_sync(0xffffffffu, a.s, o);
      const int oa = __shfl_xor_sync(0xffffffffu, a.arg, o);
      stat_merge(a, om, os, oa);
    }
    if (lane == 0) {
      tok[r] = a.arg;
      prob[r] = 1.f / a.s;                                  // exp(max - max) / sum
    }
  }
}

// Per sequence: the candidate with the largest probability (first one on ties); its token goes into the buffer
// unless a forced (position, token) is given.
__global__ void pick_kernel(const int* __restrict__ cand_off, const int* __restrict__ cand_pos,
                            const int* __restrict__ tok, const float* __restrict__ prob, int batch, int seq_total,
                            int* __restrict__ tokens, const int* __restrict__ forced_pos,
                            const int* __restrict__ forced_tok, int* __restrict__ pos_out, int* __restrict__ tok_out,
                            float* __restrict__ prob_out) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  int best = -1;
  float bp = -1.f;
  for (int i = cand_off[b]; i < cand_off[b + 1]; ++i)
    if (prob[i] > bp) { bp = prob[i]; best = i; }
  int p_ = -1, t_ = -1;
  if (best >= 0) { p_ = cand_pos[best]; t_ = tok[best]; }
  if (pos_out) pos_out[b] = p_;
  if (tok_out) tok_out[b] = t_;
  if (prob_out) prob_out[b] = best >= 0 ? bp : 0.f;
  int wp = p_, wt = t_;
  if (forced_pos != nullptr) { wp = forced_pos[b]; wt = forced_tok[b]; }
  if (wp >= 0 && wp < seq_total) tokens[(size_t)b * seq_total + wp] = wt;
}

struct StackBuffers {
  bf16 *xa, *hb, *n2, *act, *hidden, *lm_a;
  float* logits;
  int *cand_row, *cand_pos, *cand_off, *cand_count, *cand_tok, *forced;
  float* cand_prob;
};

size_t carve_stack(const dare_stack_config_t* c, char* base, StackBuffers* b, std::vector<void*>* layer_ws,
                   size_t layer_bytes) {
  const size_t Tm = (size_t)c->layer.max_batch * c->layer.max_seq, d = c->layer.d_model;
  size_t off = 0;
  auto take = [&](size_t bytes) -> void* {
    void* p = base ? base + off : nullptr;
    off += align_up(bytes);
    return p;
  };
  StackBuffers tmp;
  StackBuffers& B = b ? *b : tmp;
  B.xa = (bf16*)take(Tm * d * 2);
  B.hb = (bf16*)take(Tm * d * 2);
  B.n2 = (bf16*)take((Tm + 128) * d * 2);
  B.act = (bf16*)take((Tm + 128) * (size_t)c->d_ff * 2);
  B.hidden = (bf16*)take(Tm * d * 2);
  B.lm_a = (bf16*)take((size_t)(kMaxCand + 128) * d * 2);
  B.logits = (float*)take((size_t)kMaxCand * c->vocab * sizeof(float));
  B.cand_row = (int*)take(kMaxCand * sizeof(int));
  B.cand_pos = (int*)take(kMaxCand * sizeof(int));
  B.cand_off = (int*)take(64 * sizeof(int));
  B.cand_count = (int*)take(sizeof(int));
  B.cand_tok = (int*)take(kMaxCand * sizeof(int));
  B.cand_prob = (float*)take(kMaxCand * sizeof(float));
  B.forced = (int*)take(2 * 64 * sizeof(int));
  for (int l = 0; l < c->n_layers; ++l) {
    void* p = take(layer_bytes);
    if (layer_ws) layer_ws->push_back(p);
  }
  return off;
}

bool valid_stack_config(const dare_stack_config_t* c) {
  if (!c || c->struct_size != sizeof(dare_stack_config_t)) return false;
  if (c->n_layers <= 0 || c->n_layers > 1024 || c->d_ff <= 0 || c->d_ff % 128 != 0) return false;
  if (c->vocab <= 0 || c->vocab % 256 != 0 || c->mask_id < 0 || c->mask_id >= c->vocab) return false;
  if (c->block <= 0 || c->block > 32) return false;
  if (c->layer.dtype != DARE_BF16 || c->layer.head_dim != 128 || c->layer.d_model % 256 != 0) return false;
  if (c->layer.max_batch * c->block > kMaxCand || c->layer.max_batch > 32) return false;
  return true;
}

}  // namespace

struct dare_stack {
  uint32_t magic;
  dare_stack_config_t cfg;
  std::vector<dare_layer*> layers;
  std::vector<dare_block_weights_t> blocks;
  std::vector<BlockMaps> maps;
  CUtensorMap a_n2, a_act, a_lm, w_head;
  const void* emb;
  const float* final_gain;
  StackBuffers buf;
  int sm_count;               // SMs of the device the stack was created on
  int capture_layer;          // test hook: copy this layer's input and output of every pass (-1 = off)
  void* capture_x;
  void* capture_h;
};

namespace {

dare_status_t check_stack(const dare_stack* S) {
  if (!S) return DARE_ERR_INVALID_ARG;
  if (S->magic != kStackMagic) return DARE_ERR_STATE;
  return DARE_OK;
}

GemmParams base_params(const dare_stack* S, int batch, int seq_act, int pos_begin) {
  GemmParams p;
  memset(&p, 0, sizeof(p));
  const dare_layer_config_t& lc = S->cfg.layer;
  p.g.batch = batch; p.g.seq_act = seq_act; p.g.pos_begin = pos_begin; p.g.max_seq = lc.max_seq; p.g.kv_len = lc.max_seq;
  p.g.d = lc.d_model; p.g.n_heads = lc.n_heads; p.g.head_dim = lc.head_dim; p.g.score_head = 0;
  p.K = lc.d_model; p.m_total = batch * seq_act; p.seq_act = seq_act; p.tiles_per_seq = (seq_act + 127) / 128;
  p.a_seq_stride = seq_act; p.a_row0 = 0; p.n_split = 1 << 30; p.ld_out = lc.d_model;
  p.status = S->layers[0]->buf.status;
  return p;
}

int pick_splits(int tiles, int kblocks) { return (tiles * 2 <= 160 && kblocks >= 2) ? 2 : 1; }

dare_status_t forward(dare_stack* S, const int* tokens, int batch, int seq_total, int seq_act, int pos_begin, int mode,
                      const float* taus, void* hidden_out, cudaStream_t st) {
  const dare_layer_config_t& lc = S->cfg.layer;
  const int T_ = batch * seq_act, d = lc.d_model, f = S->cfg.d_ff;
  const StackBuffers& B = S->buf;
  embed_kernel<<<T_, 256, 0, st>>>(tokens, seq_total, seq_act, pos_begin, (const uint4*)S->emb, (uint4*)B.xa, d / 8,
                                   S->cfg.vocab);
  const int m_tiles = batch * ((seq_act + 127) / 128);
  for (int l = 0; l < S->cfg.n_layers; ++l) {
    // h = x + DARE attention
    if (l == S->capture_layer && S->capture_x)
      cudaMemcpyAsync(S->capture_x, B.xa, (size_t)T_ * d * 2, cudaMemcpyDeviceToDevice, st);
    dare_status_t s = layer_enqueue(S->layers[l], B.xa, batch, seq_act, pos_begin, mode, taus[l], B.hb, st, true);
    if (s != DARE_OK) return s;
    if (l == S->capture_layer && S->capture_h)
      cudaMemcpyAsync(S->capture_h, B.hb, (size_t)T_ * d * 2, cudaMemcpyDeviceToDevice, st);
    // n = RMSNorm_2(h)
    launch_rmsnorm<bf16>(B.hb, S->blocks[l].gain2, B.n2, T_, d, lc.rms_eps, st);
    // act = silu(W_G n) * (W_U n)
    {
      GemmParams p = base_params(S, batch, seq_act, pos_begin);
      p.b_pair = 1; p.out0 = B.act; p.ld_out = f;
      const int n_tiles = f / 128;
      const int sp = pick_splits(n_tiles * m_tiles, d / 64);
      const bool pairs = pairs_pay(n_tiles, m_tiles, sp);
      // Pair tiles over the whole reduction fill the SM pairs in waves; a last wave that is less than half full (96
      // tiles on 74 pairs) is issued as a launch of its own with the reduction split in two, which puts twice as many
      // SM pairs on it for half as long.  It needs nothing from the launch before it and runs behind it as SMs come
      // free (it waits for its predecessors only before it leaves).
      const int wave = S->sm_count / 2;
      const int rest = pairs && sp == 1 && m_tiles == 2 && wave > 0 ? n_tiles % wave : 0;
      if (rest > 0 && n_tiles > wave && 2 * rest <= wave) {
        const int full = n_tiles - rest;
        if (launch_gemm_tc(EPI_SWIGLU, 256, S->a_n2, S->maps[l].w_gate, S->maps[l].w_up, p, full, m_tiles, 1, st, 1) != cudaSuccess)
          return DARE_ERR_CUDA;
        GemmParams q = p;
        q.nt0 = full; q.wait_at_end = 1;
        if (launch_gemm_tc(EPI_SWIGLU, 256, S->a_n2, S->maps[l].w_gate, S->maps[l].w_up, q, rest, m_tiles, 2, st, 1) != cudaSuccess)
          return DARE_ERR_CUDA;
      } else if (launch_gemm_tc(EPI_SWIGLU, 256, S->a_n2, S->maps[l].w_gate, S->maps[l].w_up, p, n_tiles, m_tiles, sp, st,
                                pairs ? 1 : 0) != cudaSuccess) {
        return DARE_ERR_CUDA;
      }
    }
    // x_next = h + W_D act
    {
      GemmParams p = base_params(S, batch, seq_act, pos_begin);
      p.K = f; p.out0 = B.xa; p.resid = B.hb; p.ld_resid = d;
      const int n_tiles = d / 256;
      const int sp = pick_splits(n_tiles * m_tiles, f / 64);
      const bool pair = pairs_pay(n_tiles, m_tiles, sp);
      if (narrow_pairs_pay(d, m_tiles, f / 64)) {
        if (launch_gemm_tc(EPI_OUT, 128, S->a_act, S->maps[l].w_down64, S->maps[l].w_down64, p, d / 128, m_tiles, 2, st,
                           1) != cudaSuccess) return DARE_ERR_CUDA;
      } else {
        const CUtensorMap& wd = pair ? S->maps[l].w_down128 : S->maps[l].w_down;
        if (launch_gemm_tc(EPI_OUT, 256, S->a_act, wd, wd, p, n_tiles, m_tiles, sp, st, pair ? 1 : 0) != cudaSuccess)
          return DARE_ERR_CUDA;
      }
    }
  }
  launch_rmsnorm<bf16>(B.xa, S->final_gain, B.hidden, T_, d, lc.rms_eps, st);
  if (hidden_out)
    if (cudaMemcpyAsync(hidden_out, B.hidden, (size_t)T_ * d * 2, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return DARE_ERR_CUDA;
  if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
  return DARE_OK;
}

}  // namespace

extern "C" {

size_t dare_stack_workspace_bytes(const dare_stack_config_t* cfg) {
  if (!valid_stack_config(cfg)) return 0;
  dare_layer_config_t lc = cfg->layer;
  lc.kernel_path = DARE_PATH_TENSOR;
  const size_t lb = dare_layer_workspace_bytes(&lc);
  if (lb == 0) return 0;
  return carve_stack(cfg, nullptr, nullptr, nullptr, align_up(lb));
}

dare_status_t dare_stack_create(const dare_stack_config_t* cfg, const dare_stack_weights_t* w, void* workspace,
                                size_t workspace_bytes, dare_stack_t** out) {
  if (!out) return DARE_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || !w || !workspace || !w->blocks_host || !w->emb || !w->head || !w->final_gain) return DARE_ERR_INVALID_ARG;
  if (!valid_stack_config(cfg)) return DARE_ERR_UNSUPPORTED;
  const size_t need = dare_stack_workspace_bytes(cfg);
  if (need == 0) return DARE_ERR_UNSUPPORTED;
  if (workspace_bytes < need) return DARE_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign != 0) return DARE_ERR_ALIGN;
  dare_stack* S = new (std::nothrow) dare_stack();
  if (!S) return DARE_ERR_INVALID_ARG;
  S->magic = kStackMagic;
  S->cfg = *cfg;
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess)
      S->sm_count = sms;
    else
      S->sm_count = 0;
  }
  S->cfg.layer.kernel_path = DARE_PATH_TENSOR;
  S->emb = w->emb;
  S->final_gain = w->final_gain;
  S->capture_layer = -1;
  S->capture_x = S->capture_h = nullptr;
  const size_t lb = align_up(dare_layer_workspace_bytes(&S->cfg.layer));
  std::vector<void*> layer_ws;
  carve_stack(&S->cfg, (char*)workspace, &S->buf, &layer_ws, lb);
  const uint64_t Tm = (uint64_t)cfg->layer.max_batch * cfg->layer.max_seq, d = cfg->layer.d_model, f = cfg->d_ff;
  dare_status_t st = DARE_OK;
  for (int l = 0; l < cfg->n_layers && st == DARE_OK; ++l) {
    const dare_block_weights_t& bw = w->blocks_host[l];
    if (!bw.gain2 || !bw.w_gate || !bw.w_up || !bw.w_down) { st = DARE_ERR_INVALID_ARG; break; }
    dare_layer* L = nullptr;
    st = dare_layer_create(&S->cfg.layer, &bw.attn, layer_ws[l], lb, &L);
    if (st != DARE_OK) break;
    S->layers.push_back(L);
    S->blocks.push_back(bw);
    BlockMaps m;
    if (!make_map(&m.w_gate, bw.w_gate, f, d, 128) || !make_map(&m.w_up, bw.w_up, f, d, 128) ||
        !make_map(&m.w_down, bw.w_down, d, f, 256) || !make_map(&m.w_down128, bw.w_down, d, f, 128) ||
        !make_map(&m.w_down64, bw.w_down, d, f, 64))
      st = DARE_ERR_CUDA;
    S->maps.push_back(m);
  }
  if (st == DARE_OK) {
    if (!make_map(&S->a_n2, S->buf.n2, Tm + 128, d, 128) || !make_map(&S->a_act, S->buf.act, Tm + 128, f, 128) ||
        !make_map(&S->a_lm, S->buf.lm_a, kMaxCand + 128, d, 128) || !make_map(&S->w_head, w->head, cfg->vocab, d, 256))
      st = DARE_ERR_CUDA;
  }
  if (st == DARE_OK && cudaMemset(S->buf.lm_a, 0, (size_t)(kMaxCand + 128) * d * 2) != cudaSuccess) st = DARE_ERR_CUDA;
  if (st != DARE_OK) {
    for (dare_layer* L : S->layers) dare_layer_destroy(L);
    delete S;
    return st;
  }
  *out = S;
  return DARE_OK;
}

dare_status_t dare_stack_reset(dare_stack_t* S) {
  dare_status_t s = check_stack(S);
  if (s != DARE_OK) return s;
  for (dare_layer* L : S->layers) dare_layer_reset(L);
  return DARE_OK;
}

dare_status_t dare_stack_destroy(dare_stack_t* S) {
  dare_status_t s = check_stack(S);
  if (s != DARE_OK) return s;
  for (dare_layer* L : S->layers) dare_layer_destroy(L);
  S->magic = 0;
  delete S;
  return DARE_OK;
}

dare_layer_t* dare_stack_layer(dare_stack_t* S, int index) {
  if (check_stack(S) != DARE_OK || index < 0 || index >= (int)S->layers.size()) return nullptr;
  return S->layers[index];
}

dare_status_t dare_stack_forward(dare_stack_t* S, const int32_t* tokens, int batch, int seq_total, int seq_act,
                                 int pos_begin, int mode, const float* taus_host, void* hidden_out, void* cuda_stream) {
  dare_status_t s = check_stack(S);
  if (s != DARE_OK) return s;
  if (!tokens || !taus_host) return DARE_ERR_INVALID_ARG;
  if (batch <= 0 || batch > S->cfg.layer.max_batch || seq_act <= 0 || pos_begin < 0 ||
      pos_begin + seq_act > seq_total || seq_total > S->cfg.layer.max_seq) return DARE_ERR_SHAPE;
  for (int l = 0; l < S->cfg.n_layers; ++l)
    if (isnan(taus_host[l])) return DARE_ERR_INVALID_ARG;
  return forward(S, tokens, batch, seq_total, seq_act, pos_begin, mode, taus_host, hidden_out, (cudaStream_t)cuda_stream);
}

dare_status_t dare_stack_set_capture(dare_stack_t* S, int layer_index, void* x_out, void* h_out) {
  dare_status_t s = check_stack(S);
  if (s != DARE_OK) return s;
  if (layer_index >= (int)S->layers.size()) return DARE_ERR_SHAPE;
  S->capture_layer = layer_index;
  S->capture_x = x_out;
  S->capture_h = h_out;
  return DARE_OK;
}

dare_status_t dare_stack_last_hidden(dare_stack_t* S, void* dst_host, size_t bytes, void* cuda_stream) {
  dare_status_t s = check_stack(S);
  if (s != DARE_OK) return s;
  if (!dst_host) return DARE_ERR_INVALID_ARG;
  const size_t cap = (size_t)S->cfg.layer.max_batch * S->cfg.layer.max_seq * S->cfg.layer.d_model * 2;
  if (bytes > cap) return DARE_ERR_SHAPE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemcpyAsync(dst_host, S->buf.hidden, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return DARE_ERR_CUDA; }
  return DARE_OK;
}

dare_status_t dare_stack_decode_step(dare_stack_t* S, int32_t* tokens, int batch, int seq_total, int prompt_len,
                                     int block_index, int first, int mode, const float* taus_host,
                                     const int32_t* forced_pos_host, const int32_t* forced_tok_host, int32_t* pos_out,
                                     int32_t* tok_out, float* prob_out, void* cuda_stream) {
  dare_status_t s = check_stack(S);
  if (s != DARE_OK) return s;
  if (!tokens || !taus_host) return DARE_ERR_INVALID_ARG;
  if ((forced_pos_host == nullptr) != (forced_tok_host == nullptr)) return DARE_ERR_INVALID_ARG;
  const int blk = S->cfg.block;
  const int lo = prompt_len + block_index * blk, hi = lo + blk;
  if (batch <= 0 || batch > S->cfg.layer.max_batch || prompt_len < 0 || block_index < 0 || hi > seq_total ||
      seq_total > S->cfg.layer.max_seq) return DARE_ERR_SHAPE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int pos_begin = first ? 0 : prompt_len;
  const int seq_act = seq_total - pos_begin;
  s = dare_stack_forward(S, tokens, batch, seq_total, seq_act, pos_begin, mode, taus_host, nullptr, cuda_stream);
  if (s != DARE_OK) return s;
  const StackBuffers& B = S->buf;
  const int d = S->cfg.layer.d_model, V = S->cfg.vocab;
  cand_kernel<<<1, 32 * 32, 0, st>>>(tokens, batch, seq_total, lo, hi, S->cfg.mask_id, pos_begin, seq_act, B.cand_row,
                                     B.cand_pos, B.cand_off, B.cand_count);
  launch_gather_rows<bf16>(B.hidden, B.cand_row, B.cand_count, B.lm_a, kMaxCand, d, st);
  {
    GemmParams p = base_params(S, batch, seq_act, pos_begin);
    p.idx = B.cand_row; p.count = B.cand_count; p.m_total = kMaxCand;
    p.out_f32 = B.logits; p.ld_out = V; p.out_is_cache = 2;
    if (launch_gemm_tc(EPI_F32, 256, S->a_lm, S->w_head, S->w_head, p, V / 256, 1, 1, st) != cudaSuccess)
      return DARE_ERR_CUDA;
  }
  rowstats_kernel<<<kMaxCand, 1024, 0, st>>>(B.logits, B.cand_count, V, S->cfg.mask_id, B.cand_tok, B.cand_prob);
  const int* fpos = nullptr;
  const int* ftok = nullptr;
  if (forced_pos_host) {
    if (cudaMemcpyAsync(B.forced, forced_pos_host, batch * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(B.forced + 64, forced_tok_host, batch * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess)
      return DARE_ERR_CUDA;
    fpos = B.forced; ftok = B.forced + 64;
  }
  pick_kernel<<<1, 32, 0, st>>>(B.cand_off, B.cand_pos, B.cand_tok, B.cand_prob, batch, seq_total, tokens, fpos, ftok,
                                pos_out, tok_out, prob_out);
  if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
  return DARE_OK;
}

}  // extern "C"
