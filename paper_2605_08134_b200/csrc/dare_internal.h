// Internal declarations shared by the translation units of libdare (not part of the C ABI).
#pragma once

#include <atomic>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dare.h"

namespace dare {

// Device status word values (mirrors dare_status_t for the two device-reported codes).
constexpr int kDevOk = 0;
constexpr int kDevTimeout = DARE_ERR_TIMEOUT;
constexpr int kDevCheck = DARE_ERR_DEVICE_CHECK;

#ifdef __CUDACC__
// Range checks on what a kernel reads from the device-side selection before it uses it as an address: a token of the
// refresh list must be a token of the step, the list's length and a sequence's slice of it must lie inside the step.
// A value that fails is recorded in the layer's status word (DARE_ERR_DEVICE_CHECK; the first error of a handle stays)
// and the access that would have used it is skipped.  They cost a compare per index and stand in for a memory checker.
__device__ __forceinline__ void flag_device_check(int* status) {
  if (status) atomicCAS(status, kDevOk, kDevCheck);
}
__device__ __forceinline__ bool token_ok(int tok, int n_tokens, int* status) {
  if ((unsigned)tok < (unsigned)n_tokens) return true;
  flag_device_check(status);
  return false;
}
// the list's length, clamped into [0, cap]
__device__ __forceinline__ int checked_count(int count, int cap, int* status) {
  if ((unsigned)count <= (unsigned)cap) return count;
  flag_device_check(status);
  return count < 0 ? 0 : cap;
}
// a sequence's slice [lo, hi) of a list of at most cap entries; an impossible slice is flagged and read as empty
__device__ __forceinline__ bool slice_ok(int lo, int hi, int cap, int* status) {
  if (lo >= 0 && lo <= hi && hi <= cap) return true;
  flag_device_check(status);
  return false;
}
#endif

// Geometry of one step, passed by value to kernels.
struct StepGeom {
  int batch;      // B
  int seq_act;    // rows of each sequence covered by this step
  int pos_begin;  // first covered position
  int max_seq;    // row stride between sequences inside the caches
  int kv_len;     // keys [0, kv_len) of each sequence are valid
  int d;          // d_model
  int n_heads;
  int head_dim;
  int score_head;
  __host__ __device__ int tokens() const { return batch * seq_act; }
  // flat active index -> row inside the [max_batch*max_seq] caches
  __host__ __device__ int cache_row(int t) const { return (t / seq_act) * max_seq + pos_begin + (t % seq_act); }
  __host__ __device__ int position(int t) const { return pos_begin + (t % seq_act); }
};

// Raises a kernel's dynamic shared-memory limit once per device: the attribute belongs to the device's context, and a
// process may hold layers on several devices.  `done` is the caller's bit mask of devices already served.
template <typename K>
inline cudaError_t ensure_dyn_smem(K kernel, int bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) done.fetch_or(bit, std::memory_order_release);
  return e;
}

// Launch with programmatic stream serialization (the kernel calls griddepcontrol.wait before touching global data)
// and, optionally, a thread-block cluster along x and z.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_xz(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_x,
                          int cluster_z, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1 || cluster_z > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = cluster_z;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_z,
                       Args&&... args) {
  return launch_pdl_xz(kernel, grid, block, smem, st, 1, cluster_z, static_cast<Args&&>(args)...);
}

// ---- kernels common to both paths (common.cu) -------------------------------------------------------------
void launch_rope_table(float* cs, int max_seq, int head_dim, double theta, cudaStream_t st);
template <typename T>
void launch_rmsnorm(const T* x, const float* gain, T* xn, int rows, int d, float eps, cudaStream_t st,
                    unsigned long long* dbg = nullptr);
// Threshold + ballot/prefix-sum compaction + staleness update.  `scores == nullptr` or `select_all` selects all.
// y[t] = yc[cache_row(t)] for the tokens of the step that were not refreshed (staleness counter != 0 after the
// selection of the step): the rows a gathered output projection leaves out.
template <typename T>
void launch_copy_reused_rows(const T* yc, T* y, const int* delta, const StepGeom& g, cudaStream_t st,
                             const int* gate_count = nullptr, int gate_hi = 0);   // leaves at once when *gate_count >= gate_hi
void launch_select(const float* scores, float tau, bool select_all, const StepGeom& g, int* idx, int* count,
                   int* batch_off, int* delta, cudaStream_t st, bool beside_predecessor = false,
                   const float* tau_dev = nullptr);   // tau_dev: read the threshold from device memory instead
// *tau_out = the k-th smallest of n scores (see common.cu); one CTA
void launch_kth_score(const float* scores, int n, int k, float* tau_out, cudaStream_t st);
template <typename T>
void launch_gather_rows(const T* src, const int* idx, const int* count, T* dst, int max_rows, int d, cudaStream_t st);
// dst[r, :] = src[idx[r] (or its cache row), :] for the rows of a step's refresh set
template <typename T>
void launch_gather_step_rows(const T* src, const int* idx, const int* count, T* dst, const StepGeom& g, bool by_cache_row,
                             cudaStream_t st, int* status = nullptr, int gate_hi = 1 << 30);  // leaves at once when *count >= gate_hi

// diagnostics: a bounded wait that nothing ends (one CTA, one barrier); a single int written in stream order
void launch_wait_probe(int* status, unsigned long long limit_ns, unsigned long long* waited_ns, cudaStream_t st);
void launch_poke_int(int* dst, int value, cudaStream_t st);

// ---- stand-alone score / compaction for large token counts (select_large.cu)
int select_large_tiles(long long n);
cudaError_t launch_drift_scores(const float* a, const float* b, long long rows, int hd, float* scores, cudaStream_t st);
cudaError_t launch_select_large(const float* scores, long long n, float tau, int* idx, int* count, int* tile_counts,
                                int* tile_offsets, unsigned* flags, cudaStream_t st);
size_t select_large_flag_bytes(long long n);   // bytes of the decision words for n scores

// ---- SIMT path (simt.cu) ----------------------------------------------------------------------------------
// C[m, n] (fp32, ld = ldc) = sum_k A[arow(m), k] * W[n, k];  arow(m) = a_idx ? a_idx[m] : m;
// rows m >= *count (when count != nullptr) are skipped.
template <typename T>
void launch_gemm_simt(const T* a, const int* a_idx, const int* count, const T* w, float* c, int m_max, int n, int k,
                      int ldc, cudaStream_t st, int a_rows = 0, int* status = nullptr);   // a_rows: rows of a that a_idx may name
// Q post-pass: score of the scoring head against q_prev (fp32, cache rows), q_prev update, rotary embedding,
// store Q in the layer dtype.
template <typename T>
void launch_q_post_simt(const float* qf, int ldq, const float* rope_cs, float* q_prev, float* scores, bool has_prev,
                        T* q, const StepGeom& g, cudaStream_t st);
// K/V post-pass: rows r < *count (or all when idx == nullptr): rotary embedding on K, store K and V to cache rows.
template <typename T>
void launch_kv_post_simt(const float* kvf, int ld, const int* idx, const int* count, const float* rope_cs, T* kc,
                         T* vc, const StepGeom& g, cudaStream_t st, int* status = nullptr);
// Attention: query rows = idx[0..count) (or all rows when idx == nullptr), one warp per (row, head);
// output rows go to the O cache.
template <typename T>
void launch_attention_simt(const T* q, const T* kc, const T* vc, const int* idx, const int* count, T* oc,
                           const StepGeom& g, cudaStream_t st, int* status = nullptr);
// y[t, :] = W_O oc[cache_row(t), :]
template <typename T>
void launch_out_proj_simt(const T* oc, const T* w_o, float* tmp, T* y, const StepGeom& g, cudaStream_t st);

// ---- tensor-core path (gemm_tc.cu, attn_tc.cu) -----------------------------------------------------------
struct TcLayerMaps;  // tensor maps and launch state, owned by the handle
bool tc_supported(const dare_layer_config_t& cfg);
size_t tc_maps_bytes();

}  // namespace dare
