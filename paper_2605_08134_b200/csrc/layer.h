// The layer handle (host side) and the hooks of the tensor-core path.
#pragma once

#include "dare_internal.h"

namespace dare {

// Device buffers carved from the caller's workspace.
struct Buffers {
  float* rope_cs;   // [max_seq, head_dim/2] (cos, sin)
  void* xn;         // [T, d]  normalised hidden states (layer dtype)
  void* q;          // [T, d]  rotated queries (layer dtype)
  void* kc;         // [max_batch*max_seq, d] K cache (rotated)
  void* vc;         // [max_batch*max_seq, d] V cache
  void* oc;         // [max_batch*max_seq, d] attention-output cache (before W_O)
  float* q_prev;    // [max_batch*max_seq, head_dim] un-rotated scoring-head query of the previous step, fp32
  float* scores;    // [T]
  int* idx;         // [T] refresh set, ascending
  int* delta;       // [max_batch*max_seq] staleness counters
  int* batch_off;   // [max_batch+1]
  int* count;       // [1]
  int* status;      // [1] device status word
  unsigned long long* debug;  // [64] kernel phase timestamps (diagnostics, written by block (0,0) when enabled)
  void* x_stage;    // [T, d] staging for the host-buffer entry point
  void* y_stage;
  void* yc;         // tensor-core path: cache of projected outputs y = W_O O by cache row (gathered output projection)
  float* tmp;       // SIMT path: fp32 projection results [T, 2d]
  float* tau_dev;   // [1] threshold of a step that takes it from its own scores (dare_layer_step_quantile)
};

struct TcState;

// Kernel slots for the optional per-kernel timing.
enum { SLOT_NORM = 0, SLOT_Q_GEMM, SLOT_Q_POST, SLOT_SELECT, SLOT_GATHER, SLOT_KV_GEMM, SLOT_KV_POST, SLOT_ATTN,
       SLOT_OUT_GEMM, SLOT_COUNT };
constexpr int kMaxMarks = 16;

}  // namespace dare

struct dare_layer {
  uint32_t magic;
  dare_layer_config_t cfg;
  dare_layer_weights_t w;
  dare::Buffers buf;
  void* workspace;
  size_t workspace_bytes;
  bool use_tc;
  bool has_prev;
  bool yc_valid;    // the projected-output cache holds the current W_O O of every cached row
  int batch;
  int kv_len;
  int last_launches;
  dare::StepGeom last_geom;
  dare::TcState* tc;
  // optional per-kernel timing (events recorded between the kernels of a step)
  bool prof_on;
  int prof_n;                                  // marks recorded by the last step
  int prof_slot[dare::kMaxMarks];
  cudaEvent_t prof_ev[dare::kMaxMarks + 1];
  bool prof_ev_ready;
  bool debug_on;
  int reuse_count;  // >= 0 while a step is being enqueued that derives its threshold from its scores; -1 otherwise
  float last_tau;   // threshold of the last step when it was given by the caller
  bool last_tau_on_device;
  int inject;       // diagnostics: what the next step's selection is overwritten with (0 = nothing); see dare.h
  // asynchronous host-buffer steps: copy streams and the events that order staging-buffer reuse (created on first use)
  bool host_async_ready;
  cudaStream_t copy_in, copy_out;
  cudaEvent_t ev_in, ev_consumed, ev_out;
};

namespace dare {
// Records an event before the kernel that occupies `slot` (no-op unless profiling is on).
inline void prof_mark(dare_layer* L, int slot, cudaStream_t st) {
  if (!L->prof_on || L->prof_n >= kMaxMarks) return;
  L->prof_slot[L->prof_n] = slot;
  cudaEventRecord(L->prof_ev[L->prof_n], st);
  ++L->prof_n;
}
inline void prof_begin(dare_layer* L) { L->prof_n = 0; }
inline void prof_end(dare_layer* L, cudaStream_t st) {
  if (L->prof_on) cudaEventRecord(L->prof_ev[L->prof_n], st);
}
void inject_selection_error(dare_layer* L, const StepGeom& g, cudaStream_t st);
const float* step_threshold_on_device(dare_layer* L, const StepGeom& g, int mode, cudaStream_t st, int* launches);
dare_status_t tc_create(dare_layer* L);
void tc_destroy(dare_layer* L);
// add_input: y = x + W_O O instead of y = W_O O (the residual connection of a transformer block)
dare_status_t step_tc(dare_layer* L, const void* x, const StepGeom& g, int mode, float tau, void* y, cudaStream_t st,
                      bool add_input = false);
}  // namespace dare
