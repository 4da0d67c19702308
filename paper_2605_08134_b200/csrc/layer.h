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
  void* x_stage;    // [T, d] staging for the host-buffer entry point
  void* y_stage;
  void* xg;         // tensor-core path: gathered x_norm rows
  float* tmp;       // SIMT path: fp32 projection results [T, 2d]
};

struct TcState;

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
  int batch;
  int kv_len;
  int last_launches;
  dare::StepGeom last_geom;
  dare::TcState* tc;
};

namespace dare {
dare_status_t tc_create(dare_layer* L);
void tc_destroy(dare_layer* L);
dare_status_t step_tc(dare_layer* L, const void* x, const StepGeom& g, int mode, float tau, void* y, cudaStream_t st);
}  // namespace dare
