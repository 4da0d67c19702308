// C ABI of libdare: handle life cycle, argument validation, workspace layout and the per-step kernel sequence.
#include <math.h>
#include <new>
#include <string.h>

#include "layer.h"
#include "tc.h"

using namespace dare;

namespace {

constexpr uint32_t kMagic = 0xDA2E1A7Eu;
constexpr size_t kAlign = 256;

size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

bool valid_config(const dare_layer_config_t* c) {
  if (!c || c->struct_size != sizeof(dare_layer_config_t)) return false;
  if (c->d_model <= 0 || c->n_heads <= 0 || c->head_dim <= 0 || c->max_batch <= 0 || c->max_seq <= 0) return false;
  if ((long)c->n_heads * c->head_dim != c->d_model) return false;
  if (c->d_model % 16 != 0) return false;
  if (c->dtype != DARE_F32 && c->dtype != DARE_BF16) return false;
  if (c->score_head < 0 || c->score_head >= c->n_heads) return false;
  if (c->kernel_path < DARE_PATH_AUTO || c->kernel_path > DARE_PATH_TENSOR) return false;
  if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return false;
  if ((long)c->max_batch * c->max_seq > (1L << 24)) return false;
  return true;
}

bool simt_geometry_ok(const dare_layer_config_t* c) {
  return c->head_dim == 32 || c->head_dim == 64 || c->head_dim == 128 || c->head_dim == 256;
}

// Decides the kernel path; returns false when the configuration has no kernels.
bool pick_path(const dare_layer_config_t* c, bool* use_tc) {
  const bool tc = tc_supported(*c);
  if (c->kernel_path == DARE_PATH_TENSOR) { *use_tc = true; return tc; }
  if (c->kernel_path == DARE_PATH_SIMT) { *use_tc = false; return simt_geometry_ok(c); }
  *use_tc = tc;
  return tc || simt_geometry_ok(c);
}

// Carves the workspace.  With base == nullptr only the total size is computed.
size_t carve(const dare_layer_config_t* c, bool use_tc, char* base, Buffers* b) {
  const size_t Tm = (size_t)c->max_batch * c->max_seq;
  const size_t e = c->dtype == DARE_BF16 ? 2 : 4;
  const size_t d = c->d_model, hd = c->head_dim;
  size_t off = 0;
  auto take = [&](size_t bytes) -> void* {
    void* p = base ? base + off : nullptr;
    off += align_up(bytes);
    return p;
  };
  Buffers tmp;
  Buffers& B = b ? *b : tmp;
  B.rope_cs = (float*)take((size_t)c->max_seq * (hd / 2) * 2 * sizeof(float));
  B.xn = take(Tm * d * e);
  B.q = take(Tm * d * e);
  B.kc = take(Tm * d * e);
  B.vc = take(Tm * d * e);
  B.oc = take(Tm * d * e);
  B.q_prev = (float*)take(Tm * hd * sizeof(float));
  B.scores = (float*)take(Tm * sizeof(float));
  B.idx = (int*)take(Tm * sizeof(int));
  B.delta = (int*)take(Tm * sizeof(int));
  B.batch_off = (int*)take(((size_t)c->max_batch + 1) * sizeof(int));
  B.count = (int*)take(sizeof(int));
  B.status = (int*)take(sizeof(int));
  B.debug = (unsigned long long*)take((64 + 3 * 1024) * sizeof(unsigned long long));
  B.x_stage = take(Tm * d * e);
  B.y_stage = take(Tm * d * e);
  B.tmp = use_tc ? nullptr : (float*)take(Tm * 2 * d * sizeof(float));
  B.yc = use_tc ? take(Tm * d * e) : nullptr;
  B.tau_dev = (float*)take(sizeof(float));
  return off;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

dare_status_t check_handle(const dare_layer_t* L) {
  if (!L) return DARE_ERR_INVALID_ARG;
  if (L->magic != kMagic) return DARE_ERR_STATE;
  return DARE_OK;
}

#define CUDA_TRY(expr)                                  \
  do {                                                  \
    cudaError_t e_ = (expr);                            \
    if (e_ != cudaSuccess) { cudaGetLastError(); return DARE_ERR_CUDA; } \
  } while (0)

}  // namespace
namespace dare {
// A step that was asked to reuse its k least-drifted tokens works its threshold out from the scores the Q projection
// just left (one more kernel ahead of the selection); returns where the selection finds it, or nullptr when the
// caller's threshold applies (also on a first step and in dense mode, which refresh everything anyway).
const float* step_threshold_on_device(dare_layer* L, const StepGeom& g, int mode, cudaStream_t st, int* launches) {
  L->last_tau_on_device = false;
  if (L->reuse_count < 0 || !L->has_prev || mode == DARE_MODE_DENSE) return nullptr;
  launch_kth_score(L->buf.scores, g.tokens(), L->reuse_count, L->buf.tau_dev, st);
  ++*launches;
  L->last_tau_on_device = true;
  return L->buf.tau_dev;
}
// Diagnostics (dare_layer_debug_inject): overwrites one value of the selection just made, once.
void inject_selection_error(dare_layer* L, const StepGeom& g, cudaStream_t st) {
  if (L->inject == 1) launch_poke_int(L->buf.idx, g.tokens(), st);            // first list entry: one past the step's tokens
  else if (L->inject == 2) launch_poke_int(L->buf.count, g.tokens() + 3, st); // list longer than the step
  L->inject = 0;
}
}  // namespace dare
namespace {

template <typename T>
dare_status_t step_simt(dare_layer_t* L, const T* x, const StepGeom& g, int mode, float tau, T* y, cudaStream_t st) {
  const Buffers& B = L->buf;
  const int T_ = g.tokens(), d = g.d;
  const bool has_prev = L->has_prev;
  const bool kv_sparse = has_prev && (mode & DARE_MODE_KV);
  const bool o_sparse = has_prev && (mode & DARE_MODE_O);
  int launches = 0;
  prof_begin(L);
  // Alg. 1/2 line 1
  prof_mark(L, SLOT_NORM, st);
  launch_rmsnorm<T>(x, L->w.rms_gain, (T*)B.xn, T_, d, L->cfg.rms_eps, st); ++launches;
  // line 2: dense Q projection
  prof_mark(L, SLOT_Q_GEMM, st);
  launch_gemm_simt<T>((const T*)B.xn, nullptr, nullptr, (const T*)L->w.w_q, B.tmp, T_, d, d, d, st); ++launches;
  // line 3 + stored-query update + rotary embedding
  prof_mark(L, SLOT_Q_POST, st);
  launch_q_post_simt<T>(B.tmp, d, B.rope_cs, B.q_prev, B.scores, has_prev, (T*)B.q, g, st); ++launches;
  // lines 4-5: refresh set as a compacted index list; Sec. 4 staleness
  prof_mark(L, SLOT_SELECT, st);
  const float* tau_dev = step_threshold_on_device(L, g, mode, st, &launches);
  launch_select(B.scores, tau, !has_prev || mode == DARE_MODE_DENSE, g, B.idx, B.count, B.batch_off, B.delta, st, false,
                tau_dev); ++launches;
  inject_selection_error(L, g, st);
  // K/V: Alg. 1 lines 6-9 (refresh set only) or Alg. 2 line 7 (all rows)
  const int* kv_idx = kv_sparse ? B.idx : nullptr;
  const int* kv_cnt = kv_sparse ? B.count : nullptr;
  prof_mark(L, SLOT_KV_GEMM, st);
  launch_gemm_simt<T>((const T*)B.xn, kv_idx, kv_cnt, (const T*)L->w.w_k, B.tmp, T_, d, d, 2 * d, st, T_, B.status); ++launches;
  launch_gemm_simt<T>((const T*)B.xn, kv_idx, kv_cnt, (const T*)L->w.w_v, B.tmp + d, T_, d, d, 2 * d, st, T_, B.status); ++launches;
  prof_mark(L, SLOT_KV_POST, st);
  launch_kv_post_simt<T>(B.tmp, 2 * d, kv_idx, kv_cnt, B.rope_cs, (T*)B.kc, (T*)B.vc, g, st, B.status); ++launches;
  // attention: Alg. 1 line 10 (all rows) or Alg. 2 lines 6, 8-10 (refresh set rows, others keep the cache)
  prof_mark(L, SLOT_ATTN, st);
  launch_attention_simt<T>((const T*)B.q, (const T*)B.kc, (const T*)B.vc, o_sparse ? B.idx : nullptr,
                           o_sparse ? B.count : nullptr, (T*)B.oc, g, st, B.status); ++launches;
  // last line: output projection of every row
  prof_mark(L, SLOT_OUT_GEMM, st);
  launch_out_proj_simt<T>((const T*)B.oc, (const T*)L->w.w_o, B.tmp, y, g, st); ++launches;
  prof_end(L, st);
  L->last_launches = launches;
  CUDA_TRY(cudaGetLastError());
  return DARE_OK;
}

dare_status_t validate_step(dare_layer_t* L, const void* x, int batch, int seq_act, int pos_begin, int mode,
                            float tau, void* y) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (!x || !y) return DARE_ERR_INVALID_ARG;
  if (mode < DARE_MODE_DENSE || mode > DARE_MODE_BOTH) return DARE_ERR_INVALID_ARG;
  if (isnan(tau)) return DARE_ERR_INVALID_ARG;
  if (batch <= 0 || seq_act <= 0 || pos_begin < 0) return DARE_ERR_SHAPE;
  if (batch > L->cfg.max_batch || (long)pos_begin + seq_act > L->cfg.max_seq) return DARE_ERR_SHAPE;
  if (L->has_prev) {
    if (batch != L->batch) return DARE_ERR_STATE;
    if (pos_begin + seq_act > L->kv_len) return DARE_ERR_STATE;
  } else if (pos_begin != 0) {
    return DARE_ERR_STATE;
  }
  return DARE_OK;
}

dare_status_t enqueue_step(dare_layer_t* L, const void* x, int batch, int seq_act, int pos_begin, int mode, float tau,
                           void* y, cudaStream_t st, bool add_input = false) {
  StepGeom g;
  g.batch = batch; g.seq_act = seq_act; g.pos_begin = pos_begin; g.max_seq = L->cfg.max_seq;
  g.kv_len = L->has_prev ? L->kv_len : seq_act;
  g.d = L->cfg.d_model; g.n_heads = L->cfg.n_heads; g.head_dim = L->cfg.head_dim; g.score_head = L->cfg.score_head;
  dare_status_t s;
  if (L->use_tc) {
    s = step_tc(L, x, g, mode, tau, y, st, add_input);
  } else if (L->cfg.dtype == DARE_BF16) {
    s = step_simt<__nv_bfloat16>(L, (const __nv_bfloat16*)x, g, mode, tau, (__nv_bfloat16*)y, st);
  } else {
    s = step_simt<float>(L, (const float*)x, g, mode, tau, (float*)y, st);
  }
  if (s != DARE_OK) return s;
  // (a step may use the input staging buffer as scratch; once the asynchronous host-buffer entry point is in use, its
  // next copy in waits for this step, whichever entry point issued it)
  if (L->host_async_ready && cudaEventRecord(L->ev_consumed, st) != cudaSuccess) return DARE_ERR_CUDA;
  if (!L->has_prev) { L->kv_len = seq_act; L->batch = batch; }
  L->has_prev = true;
  L->last_geom = g;
  L->last_tau = tau;
  return DARE_OK;
}

}  // namespace

namespace dare {
// The layer step for callers inside the library (the stack): same validation as dare_layer_step; add_input makes the
// output x + W_O O (tensor-core path only).
dare_status_t layer_enqueue(dare_layer* L, const void* x, int batch, int seq_act, int pos_begin, int mode, float tau,
                            void* y, cudaStream_t st, bool add_input) {
  dare_status_t s = validate_step(L, x, batch, seq_act, pos_begin, mode, tau, y);
  if (s != DARE_OK) return s;
  if (add_input && !L->use_tc) return DARE_ERR_UNSUPPORTED;
  return enqueue_step(L, x, batch, seq_act, pos_begin, mode, tau, y, st, add_input);
}
}  // namespace dare

extern "C" {

int dare_abi_version(void) { return 1; }

const char* dare_status_string(dare_status_t s) {
  switch (s) {
    case DARE_OK: return "ok";
    case DARE_ERR_INVALID_ARG: return "invalid argument";
    case DARE_ERR_SHAPE: return "shape outside the configured limits";
    case DARE_ERR_STATE: return "call not legal in this state";
    case DARE_ERR_ALIGN: return "pointer not aligned";
    case DARE_ERR_WORKSPACE: return "workspace too small";
    case DARE_ERR_CUDA: return "CUDA call failed";
    case DARE_ERR_TIMEOUT: return "device-side wait timed out";
    case DARE_ERR_UNSUPPORTED: return "configuration not supported";
    case DARE_ERR_DEVICE_CHECK: return "device-side range check failed";
  }
  return "unknown status";
}

size_t dare_layer_workspace_bytes(const dare_layer_config_t* cfg) {
  bool use_tc = false;
  if (!valid_config(cfg) || !pick_path(cfg, &use_tc)) return 0;
  return carve(cfg, use_tc, nullptr, nullptr);
}

dare_status_t dare_layer_create(const dare_layer_config_t* cfg, const dare_layer_weights_t* w, void* workspace,
                                size_t workspace_bytes, dare_layer_t** out) {
  if (!out) return DARE_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || !w || !workspace) return DARE_ERR_INVALID_ARG;
  if (!valid_config(cfg)) return DARE_ERR_INVALID_ARG;
  bool use_tc = false;
  if (!pick_path(cfg, &use_tc)) return DARE_ERR_UNSUPPORTED;
  if (!w->w_q || !w->w_k || !w->w_v || !w->w_o || !w->rms_gain) return DARE_ERR_INVALID_ARG;
  if (!aligned16(w->w_q) || !aligned16(w->w_k) || !aligned16(w->w_v) || !aligned16(w->w_o) || !aligned16(w->rms_gain))
    return DARE_ERR_ALIGN;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign != 0) return DARE_ERR_ALIGN;
  const size_t need = carve(cfg, use_tc, nullptr, nullptr);
  if (workspace_bytes < need) return DARE_ERR_WORKSPACE;
  dare_layer_t* L = new (std::nothrow) dare_layer_t();
  if (!L) return DARE_ERR_INVALID_ARG;
  L->magic = kMagic;
  L->cfg = *cfg;
  L->w = *w;
  L->use_tc = use_tc;
  L->has_prev = false;
  L->yc_valid = false;
  L->batch = 0;
  L->kv_len = 0;
  L->last_launches = 0;
  L->tc = nullptr;
  L->prof_on = false;
  L->prof_n = 0;
  L->prof_ev_ready = false;
  L->debug_on = false;
  L->inject = 0;
  L->reuse_count = -1;
  L->last_tau = 0.f;
  L->last_tau_on_device = false;
  L->host_async_ready = false;
  memset(&L->last_geom, 0, sizeof(L->last_geom));
  carve(cfg, use_tc, (char*)workspace, &L->buf);
  L->workspace = workspace;
  L->workspace_bytes = need;
  cudaError_t e = cudaMemset(L->buf.status, 0, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(L->buf.count, 0, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(L->buf.delta, 0, (size_t)cfg->max_batch * cfg->max_seq * sizeof(int));
  {
    // caches start finite: tiles that reach past the valid extent are masked, but must not carry NaN bit patterns
    const size_t cache_bytes = (size_t)cfg->max_batch * cfg->max_seq * cfg->d_model * (cfg->dtype == DARE_BF16 ? 2 : 4);
    if (e == cudaSuccess) e = cudaMemset(L->buf.kc, 0, cache_bytes);
    if (e == cudaSuccess) e = cudaMemset(L->buf.vc, 0, cache_bytes);
    if (e == cudaSuccess) e = cudaMemset(L->buf.oc, 0, cache_bytes);
  }
  if (e == cudaSuccess) {
    launch_rope_table(L->buf.rope_cs, cfg->max_seq, cfg->head_dim, (double)cfg->rope_theta, 0);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { cudaGetLastError(); delete L; return DARE_ERR_CUDA; }
  if (use_tc) {
    dare_status_t s = tc_create(L);
    if (s != DARE_OK) { delete L; return s; }
  }
  *out = L;
  return DARE_OK;
}

dare_status_t dare_layer_step(dare_layer_t* L, const void* x, int batch, int seq_act, int pos_begin, int mode,
                              float threshold, void* y, void* cuda_stream) {
  dare_status_t s = validate_step(L, x, batch, seq_act, pos_begin, mode, threshold, y);
  if (s != DARE_OK) return s;
  if (!aligned16(x) || !aligned16(y)) return DARE_ERR_ALIGN;
  return enqueue_step(L, x, batch, seq_act, pos_begin, mode, threshold, y, (cudaStream_t)cuda_stream);
}

dare_status_t dare_layer_step_quantile(dare_layer_t* L, const void* x, int batch, int seq_act, int pos_begin, int mode,
                                       int reuse_count, void* y, void* cuda_stream) {
  dare_status_t s = validate_step(L, x, batch, seq_act, pos_begin, mode, 0.f, y);
  if (s != DARE_OK) return s;
  if (!aligned16(x) || !aligned16(y)) return DARE_ERR_ALIGN;
  if (reuse_count < 0) return DARE_ERR_INVALID_ARG;
  L->reuse_count = reuse_count;
  s = enqueue_step(L, x, batch, seq_act, pos_begin, mode, 0.f, y, (cudaStream_t)cuda_stream);
  L->reuse_count = -1;
  return s;
}

dare_status_t dare_layer_last_threshold(dare_layer_t* L, float* tau_host, void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (!tau_host) return DARE_ERR_INVALID_ARG;
  if (!L->has_prev) return DARE_ERR_STATE;
  if (!L->last_tau_on_device) { *tau_host = L->last_tau; return DARE_OK; }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CUDA_TRY(cudaMemcpyAsync(tau_host, L->buf.tau_dev, sizeof(float), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  return DARE_OK;
}

dare_status_t dare_score_kth(const float* scores, int64_t n_tokens, int64_t k, float* tau_out, void* cuda_stream) {
  if (!scores || !tau_out) return DARE_ERR_INVALID_ARG;
  if (n_tokens <= 0 || n_tokens > (int64_t)1 << 24) return DARE_ERR_SHAPE;
  const int kk = k < 0 ? 0 : (k > n_tokens ? (int)n_tokens : (int)k);
  launch_kth_score(scores, (int)n_tokens, kk, tau_out, (cudaStream_t)cuda_stream);
  CUDA_TRY(cudaGetLastError());
  return DARE_OK;
}

dare_status_t dare_layer_step_host(dare_layer_t* L, const void* x_host, int batch, int seq_act, int pos_begin, int mode,
                                   float threshold, void* y_host, void* cuda_stream) {
  dare_status_t s = validate_step(L, x_host, batch, seq_act, pos_begin, mode, threshold, y_host);
  if (s != DARE_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t e = L->cfg.dtype == DARE_BF16 ? 2 : 4;
  const size_t bytes = (size_t)batch * seq_act * L->cfg.d_model * e;
  if (L->host_async_ready) CUDA_TRY(cudaStreamWaitEvent(st, L->ev_out, 0));   // (an earlier asynchronous copy out)
  CUDA_TRY(cudaMemcpyAsync(L->buf.x_stage, x_host, bytes, cudaMemcpyHostToDevice, st));
  s = enqueue_step(L, L->buf.x_stage, batch, seq_act, pos_begin, mode, threshold, L->buf.y_stage, st);
  if (s != DARE_OK) return s;
  CUDA_TRY(cudaMemcpyAsync(y_host, L->buf.y_stage, bytes, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  return DARE_OK;
}

dare_status_t dare_layer_step_host_async(dare_layer_t* L, const void* x_host, int batch, int seq_act, int pos_begin,
                                         int mode, float threshold, void* y_host, void* cuda_stream) {
  dare_status_t s = validate_step(L, x_host, batch, seq_act, pos_begin, mode, threshold, y_host);
  if (s != DARE_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (!L->host_async_ready) {
    CUDA_TRY(cudaStreamCreateWithFlags(&L->copy_in, cudaStreamNonBlocking));
    CUDA_TRY(cudaStreamCreateWithFlags(&L->copy_out, cudaStreamNonBlocking));
    CUDA_TRY(cudaEventCreateWithFlags(&L->ev_in, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&L->ev_consumed, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&L->ev_out, cudaEventDisableTiming));
    // (never-recorded events: waiting on them returns at once, which is right for the first step)
    L->host_async_ready = true;
    // steps issued before through the other entry points may still be using the staging buffers
    CUDA_TRY(cudaEventRecord(L->ev_consumed, st));
    CUDA_TRY(cudaEventRecord(L->ev_out, st));
  }
  const size_t e = L->cfg.dtype == DARE_BF16 ? 2 : 4;
  const size_t bytes = (size_t)batch * seq_act * L->cfg.d_model * e;
  // copy in: once the layer's previous step has read the staging buffer
  CUDA_TRY(cudaStreamWaitEvent(L->copy_in, L->ev_consumed, 0));
  CUDA_TRY(cudaMemcpyAsync(L->buf.x_stage, x_host, bytes, cudaMemcpyHostToDevice, L->copy_in));
  CUDA_TRY(cudaEventRecord(L->ev_in, L->copy_in));
  // the step: behind the copy in, and behind the previous copy out of the output staging buffer
  CUDA_TRY(cudaStreamWaitEvent(st, L->ev_in, 0));
  CUDA_TRY(cudaStreamWaitEvent(st, L->ev_out, 0));
  s = enqueue_step(L, L->buf.x_stage, batch, seq_act, pos_begin, mode, threshold, L->buf.y_stage, st);   // records ev_consumed
  if (s != DARE_OK) return s;
  // copy out: behind the step, on its own stream
  CUDA_TRY(cudaStreamWaitEvent(L->copy_out, L->ev_consumed, 0));
  CUDA_TRY(cudaMemcpyAsync(y_host, L->buf.y_stage, bytes, cudaMemcpyDeviceToHost, L->copy_out));
  CUDA_TRY(cudaEventRecord(L->ev_out, L->copy_out));
  return DARE_OK;
}

dare_status_t dare_layer_wait_host(dare_layer_t* L) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (L->host_async_ready) CUDA_TRY(cudaEventSynchronize(L->ev_out));
  return DARE_OK;
}

dare_status_t dare_layer_reset(dare_layer_t* L) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  L->has_prev = false;
  L->yc_valid = false;
  L->batch = 0;
  L->kv_len = 0;
  return DARE_OK;
}

dare_status_t dare_layer_destroy(dare_layer_t* L) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (L->use_tc) tc_destroy(L);
  if (L->prof_ev_ready)
    for (int i = 0; i <= kMaxMarks; ++i) cudaEventDestroy(L->prof_ev[i]);
  if (L->host_async_ready) {
    cudaStreamSynchronize(L->copy_in);
    cudaStreamSynchronize(L->copy_out);
    cudaEventDestroy(L->ev_in); cudaEventDestroy(L->ev_consumed); cudaEventDestroy(L->ev_out);
    cudaStreamDestroy(L->copy_in); cudaStreamDestroy(L->copy_out);
  }
  L->magic = 0;
  delete L;
  return DARE_OK;
}

dare_status_t dare_layer_status(dare_layer_t* L, void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int dev = 0;
  CUDA_TRY(cudaMemcpyAsync(&dev, L->buf.status, sizeof(int), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  if (dev == kDevTimeout) return DARE_ERR_TIMEOUT;
  if (dev != kDevOk) return DARE_ERR_DEVICE_CHECK;
  return DARE_OK;
}

dare_status_t dare_layer_last_selection(dare_layer_t* L, int32_t* idx_host, int32_t* count_host,
                                        int32_t* batch_off_host, float* scores_host, int32_t* delta_host,
                                        void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (!L->has_prev) return DARE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const StepGeom& g = L->last_geom;
  const int T_ = g.tokens();
  int count = 0;
  CUDA_TRY(cudaMemcpyAsync(&count, L->buf.count, sizeof(int), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  if (count < 0 || count > T_) return DARE_ERR_DEVICE_CHECK;
  if (count_host) *count_host = count;
  if (idx_host && count > 0)
    CUDA_TRY(cudaMemcpyAsync(idx_host, L->buf.idx, (size_t)count * sizeof(int), cudaMemcpyDeviceToHost, st));
  if (batch_off_host)
    CUDA_TRY(cudaMemcpyAsync(batch_off_host, L->buf.batch_off, ((size_t)g.batch + 1) * sizeof(int),
                             cudaMemcpyDeviceToHost, st));
  if (scores_host)
    CUDA_TRY(cudaMemcpyAsync(scores_host, L->buf.scores, (size_t)T_ * sizeof(float), cudaMemcpyDeviceToHost, st));
  if (delta_host)
    CUDA_TRY(cudaMemcpy2DAsync(delta_host, (size_t)g.seq_act * sizeof(int), L->buf.delta + g.pos_begin,
                               (size_t)g.max_seq * sizeof(int), (size_t)g.seq_act * sizeof(int), g.batch,
                               cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  return DARE_OK;
}

dare_status_t dare_layer_read_caches(dare_layer_t* L, void* k_host, void* v_host, void* o_host, float* q_prev_host,
                                     void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (!L->has_prev) return DARE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t e = L->cfg.dtype == DARE_BF16 ? 2 : 4;
  const size_t d = L->cfg.d_model, hd = L->cfg.head_dim;
  const size_t row = d * e;
  const void* src[3] = {L->buf.kc, L->buf.vc, L->buf.oc};
  void* dst[3] = {k_host, v_host, o_host};
  for (int i = 0; i < 3; ++i)
    if (dst[i])
      CUDA_TRY(cudaMemcpy2DAsync(dst[i], (size_t)L->kv_len * row, src[i], (size_t)L->cfg.max_seq * row,
                                 (size_t)L->kv_len * row, L->batch, cudaMemcpyDeviceToHost, st));
  if (q_prev_host)
    CUDA_TRY(cudaMemcpy2DAsync(q_prev_host, (size_t)L->kv_len * hd * 4, L->buf.q_prev, (size_t)L->cfg.max_seq * hd * 4,
                               (size_t)L->kv_len * hd * 4, L->batch, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  return DARE_OK;
}

struct StateHeader {
  uint32_t magic;
  int32_t has_prev, batch, kv_len;
  int32_t d_model, head_dim, max_batch, max_seq, dtype;
  int32_t reserved[7];
};

size_t dare_layer_state_bytes(const dare_layer_t* L) {
  if (check_handle(L) != DARE_OK) return 0;
  const size_t Tm = (size_t)L->cfg.max_batch * L->cfg.max_seq;
  const size_t e = L->cfg.dtype == DARE_BF16 ? 2 : 4;
  return sizeof(StateHeader) + Tm * L->cfg.head_dim * 4 + 3 * Tm * L->cfg.d_model * e + Tm * 4;
}

dare_status_t dare_layer_export_state(dare_layer_t* L, void* dst_host, size_t bytes, void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (!dst_host) return DARE_ERR_INVALID_ARG;
  if (bytes < dare_layer_state_bytes(L)) return DARE_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t Tm = (size_t)L->cfg.max_batch * L->cfg.max_seq;
  const size_t e = L->cfg.dtype == DARE_BF16 ? 2 : 4;
  StateHeader h;
  memset(&h, 0, sizeof(h));
  h.magic = kMagic; h.has_prev = L->has_prev; h.batch = L->batch; h.kv_len = L->kv_len;
  h.d_model = L->cfg.d_model; h.head_dim = L->cfg.head_dim; h.max_batch = L->cfg.max_batch; h.max_seq = L->cfg.max_seq;
  h.dtype = L->cfg.dtype;
  char* p = (char*)dst_host;
  memcpy(p, &h, sizeof(h)); p += sizeof(h);
  const void* src[5] = {L->buf.q_prev, L->buf.kc, L->buf.vc, L->buf.oc, L->buf.delta};
  const size_t sz[5] = {Tm * L->cfg.head_dim * 4, Tm * L->cfg.d_model * e, Tm * L->cfg.d_model * e,
                        Tm * L->cfg.d_model * e, Tm * 4};
  for (int i = 0; i < 5; ++i) {
    CUDA_TRY(cudaMemcpyAsync(p, src[i], sz[i], cudaMemcpyDeviceToHost, st));
    p += sz[i];
  }
  CUDA_TRY(cudaStreamSynchronize(st));
  return DARE_OK;
}

dare_status_t dare_layer_import_state(dare_layer_t* L, const void* src_host, size_t bytes, void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (!src_host) return DARE_ERR_INVALID_ARG;
  if (bytes < dare_layer_state_bytes(L)) return DARE_ERR_WORKSPACE;
  StateHeader h;
  memcpy(&h, src_host, sizeof(h));
  if (h.magic != kMagic || h.d_model != L->cfg.d_model || h.head_dim != L->cfg.head_dim ||
      h.max_batch != L->cfg.max_batch || h.max_seq != L->cfg.max_seq || h.dtype != L->cfg.dtype)
    return DARE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t Tm = (size_t)L->cfg.max_batch * L->cfg.max_seq;
  const size_t e = L->cfg.dtype == DARE_BF16 ? 2 : 4;
  const char* p = (const char*)src_host + sizeof(h);
  void* dst[5] = {L->buf.q_prev, L->buf.kc, L->buf.vc, L->buf.oc, L->buf.delta};
  const size_t sz[5] = {Tm * L->cfg.head_dim * 4, Tm * L->cfg.d_model * e, Tm * L->cfg.d_model * e,
                        Tm * L->cfg.d_model * e, Tm * 4};
  for (int i = 0; i < 5; ++i) {
    CUDA_TRY(cudaMemcpyAsync(dst[i], p, sz[i], cudaMemcpyHostToDevice, st));
    p += sz[i];
  }
  CUDA_TRY(cudaStreamSynchronize(st));
  L->has_prev = h.has_prev != 0;
  L->yc_valid = false;                 // the projected-output cache is not part of the state: rebuilt by the next
                                       // step that projects every cached row
  L->batch = h.batch;
  L->kv_len = h.kv_len;
  return DARE_OK;
}

dare_status_t dare_layer_set_profiling(dare_layer_t* L, int enable) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (enable && !L->prof_ev_ready) {
    for (int i = 0; i <= kMaxMarks; ++i) CUDA_TRY(cudaEventCreate(&L->prof_ev[i]));
    L->prof_ev_ready = true;
  }
  L->prof_on = enable != 0;
  L->prof_n = 0;
  return DARE_OK;
}

dare_status_t dare_layer_last_kernel_times(dare_layer_t* L, int32_t* slot_host, float* ms_host, int capacity,
                                           int* n_out) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (!n_out) return DARE_ERR_INVALID_ARG;
  *n_out = 0;
  if (!L->prof_on || L->prof_n == 0) return DARE_ERR_STATE;
  CUDA_TRY(cudaEventSynchronize(L->prof_ev[L->prof_n]));
  const int n = L->prof_n < capacity ? L->prof_n : capacity;
  for (int i = 0; i < n; ++i) {
    float ms = 0.f;
    CUDA_TRY(cudaEventElapsedTime(&ms, L->prof_ev[i], L->prof_ev[i + 1]));
    if (slot_host) slot_host[i] = L->prof_slot[i];
    if (ms_host) ms_host[i] = ms;
  }
  *n_out = n;
  return DARE_OK;
}

dare_status_t dare_layer_debug_timestamps(dare_layer_t* L, int enable, uint64_t* out_host, void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (out_host) {
    CUDA_TRY(cudaMemcpyAsync(out_host, L->buf.debug, (64 + 3 * 1024) * sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
  }
  if (enable && !L->debug_on) {
    // cleared once, when the stamps are switched on (not per step: a memset in the stream would break the kernels'
    // launch overlap); the stamps are plain stores or maxima of a clock that only grows
    CUDA_TRY(cudaMemsetAsync(L->buf.debug, 0, (64 + 3 * 1024) * sizeof(uint64_t), st));
  }
  L->debug_on = enable != 0;
  return DARE_OK;
}

dare_status_t dare_layer_clear_status(dare_layer_t* L, void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  CUDA_TRY(cudaMemsetAsync(L->buf.status, 0, sizeof(int), (cudaStream_t)cuda_stream));
  return DARE_OK;
}

dare_status_t dare_layer_debug_wait_probe(dare_layer_t* L, uint64_t limit_ns, uint64_t* waited_ns_host, void* cuda_stream) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (limit_ns == 0 || limit_ns > 1000000000ull) return DARE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  unsigned long long* slot = L->buf.debug + 63;          // (a slot no kernel of a step writes)
  launch_wait_probe(L->buf.status, limit_ns, slot, st);
  CUDA_TRY(cudaGetLastError());
  unsigned long long waited = 0;
  CUDA_TRY(cudaMemcpyAsync(&waited, slot, sizeof(waited), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  if (waited_ns_host) *waited_ns_host = waited;
  return DARE_OK;
}

dare_status_t dare_layer_debug_inject(dare_layer_t* L, int what) {
  dare_status_t s = check_handle(L);
  if (s != DARE_OK) return s;
  if (what < 0 || what > 2) return DARE_ERR_INVALID_ARG;
  L->inject = what;
  return DARE_OK;
}

const char* dare_kernel_slot_name(int slot) {
  switch (slot) {
    case SLOT_NORM: return "rmsnorm";
    case SLOT_Q_GEMM: return "q_gemm";
    case SLOT_Q_POST: return "q_post";
    case SLOT_SELECT: return "select_compact";
    case SLOT_GATHER: return "gather_rows";
    case SLOT_KV_GEMM: return "kv_gemm";
    case SLOT_KV_POST: return "kv_post";
    case SLOT_ATTN: return "attention";
    case SLOT_OUT_GEMM: return "out_gemm";
  }
  return "?";
}

dare_status_t dare_drift_scores(const float* q_now, const float* q_prev, int64_t rows, int head_dim, float* scores,
                                void* cuda_stream) {
  if (!q_now || !q_prev || !scores) return DARE_ERR_INVALID_ARG;
  if (rows < 0 || head_dim <= 0 || head_dim % 4 != 0) return DARE_ERR_SHAPE;
  if (!aligned16(q_now) || !aligned16(q_prev)) return DARE_ERR_ALIGN;
  CUDA_TRY(launch_drift_scores(q_now, q_prev, rows, head_dim, scores, (cudaStream_t)cuda_stream));
  return DARE_OK;
}

dare_status_t dare_rmsnorm(const void* x, const float* gain, void* y, int64_t rows, int d_model, float eps, int dtype,
                           void* cuda_stream) {
  if (!x || !gain || !y) return DARE_ERR_INVALID_ARG;
  if (dtype != DARE_F32 && dtype != DARE_BF16) return DARE_ERR_INVALID_ARG;
  if (rows < 0 || rows > (int64_t)1 << 24 || d_model <= 0 || d_model % 16 != 0 || !(eps >= 0.f)) return DARE_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(y) || !aligned16(gain)) return DARE_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (dtype == DARE_BF16)
    launch_rmsnorm<__nv_bfloat16>((const __nv_bfloat16*)x, gain, (__nv_bfloat16*)y, (int)rows, d_model, eps, st);
  else
    launch_rmsnorm<float>((const float*)x, gain, (float*)y, (int)rows, d_model, eps, st);
  CUDA_TRY(cudaGetLastError());
  return DARE_OK;
}

size_t dare_select_compact_scratch_bytes(int64_t n_tokens) {
  if (n_tokens < 0 || n_tokens > (int64_t)1 << 30) return 0;
  return align_up((size_t)select_large_tiles(n_tokens) * sizeof(int)) * 2 + align_up(select_large_flag_bytes(n_tokens)) +
         kAlign;
}

dare_status_t dare_select_compact(const float* scores, int64_t n_tokens, float threshold, int32_t* idx, int32_t* count,
                                  void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!scores || !idx || !count || !scratch) return DARE_ERR_INVALID_ARG;
  if (isnan(threshold)) return DARE_ERR_INVALID_ARG;
  if (n_tokens < 0 || n_tokens > (int64_t)1 << 30) return DARE_ERR_SHAPE;
  if (!aligned16(scores) || !aligned16(scratch)) return DARE_ERR_ALIGN;
  if (scratch_bytes < dare_select_compact_scratch_bytes(n_tokens)) return DARE_ERR_WORKSPACE;
  const size_t half = align_up((size_t)select_large_tiles(n_tokens) * sizeof(int));
  int* counts = (int*)scratch;
  int* offsets = (int*)((char*)scratch + half);
  unsigned* flags = (unsigned*)((char*)scratch + 2 * half);
  CUDA_TRY(launch_select_large(scores, n_tokens, threshold, idx, count, counts, offsets, flags,
                               (cudaStream_t)cuda_stream));
  return DARE_OK;
}

int dare_layer_last_launch_count(const dare_layer_t* L) {
  if (check_handle(L) != DARE_OK) return 0;
  return L->last_launches;
}

}  // extern "C"
