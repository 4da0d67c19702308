// CUDA-core (SIMT) kernel path: fp32 accumulate everywhere, any supported geometry.  This is the path of the
// fp32 configuration (tensor-core tf32 would not hold a 1e-4 bound) and the cross-check for the tensor-core path.
#include "dare_internal.h"

namespace dare {

template <typename T>
__device__ __forceinline__ float to_f(T v);
template <>
__device__ __forceinline__ float to_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_f(float v);
template <>
__device__ __forceinline__ float from_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ------------------------------------------------------------------------------------------------ GEMM
// C[m, n] = sum_k A[arow(m), k] * W[n, k]  (W stored [out, in]: Alg. 1 line 2).  64x64 tile, 4x4 per thread.
// Row map of A: identity, an index list (Alg. 1 line 6), or the cache-row map of the step window.
struct ARowMap {
  const int* idx;   // gathered rows, or nullptr
  int use_cache_row;
  StepGeom g;
  int a_rows;       // rows of A an index may name (range check)
  int* status;
};

template <typename T, typename TC>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ a, ARowMap map,
                                                        const int* __restrict__ count, const T* __restrict__ w,
                                                        TC* __restrict__ c, int m_max, int n, int k, int ldc) {
  constexpr int BM = 64, BN = 64, BK = 16;
  const int m_eff = count ? checked_count(*count, m_max, map.status) : m_max;
  const int m0 = blockIdx.y * BM;
  if (m0 >= m_eff) return;
  const int n0 = blockIdx.x * BN;
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const int tid = threadIdx.x;
  const int lrow = tid >> 2, lk = (tid & 3) * 4;
  const int gm = m0 + lrow;
  bool a_ok = gm < m_eff;
  size_t a_row = 0;
  if (a_ok && map.idx) {
    const int t = map.idx[gm];
    a_ok = token_ok(t, map.a_rows, map.status);          // a row that is not a row of A is read as zeros
    a_row = a_ok ? (size_t)t : 0;
  } else if (a_ok) {
    a_row = map.use_cache_row ? (size_t)map.g.cache_row(gm) : (size_t)gm;
  }
  const bool w_ok = (n0 + lrow) < n;
  const T* ap = a + a_row * k + lk;
  const T* wp = w + (size_t)(n0 + lrow) * k + lk;
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < k; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      As[lk + i][lrow] = a_ok ? to_f<T>(ap[k0 + i]) : 0.f;
      Ws[lk + i][lrow] = w_ok ? to_f<T>(wp[k0 + i]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      float4 wv = *reinterpret_cast<const float4*>(&Ws[kk][tx * 4]);
      float ar[4] = {av.x, av.y, av.z, av.w}, wr[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], wr[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= m_eff) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int nn = n0 + tx * 4 + j;
      if (nn < n) c[(size_t)m * ldc + nn] = from_f<TC>(acc[i][j]);
    }
  }
}

template <typename T>
void launch_gemm_simt(const T* a, const int* a_idx, const int* count, const T* w, float* c, int m_max, int n, int k,
                      int ldc, cudaStream_t st, int a_rows, int* status) {
  if (m_max <= 0) return;
  ARowMap map{a_idx, 0, StepGeom{}, a_rows > 0 ? a_rows : m_max, status};
  dim3 grid((n + 63) / 64, (m_max + 63) / 64);
  gemm_simt_kernel<T, float><<<grid, 256, 0, st>>>(a, map, count, w, c, m_max, n, k, ldc);
}
template void launch_gemm_simt<float>(const float*, const int*, const int*, const float*, float*, int, int, int, int,
                                      cudaStream_t, int, int*);
template void launch_gemm_simt<__nv_bfloat16>(const __nv_bfloat16*, const int*, const int*, const __nv_bfloat16*,
                                              float*, int, int, int, int, cudaStream_t, int, int*);

template <typename T>
void launch_out_proj_simt(const T* oc, const T* w_o, float* tmp, T* y, const StepGeom& g, cudaStream_t st) {
  (void)tmp;
  const int T_ = g.tokens();
  if (T_ <= 0) return;
  ARowMap map{nullptr, 1, g, 0, nullptr};
  dim3 grid((g.d + 63) / 64, (T_ + 63) / 64);
  gemm_simt_kernel<T, T><<<grid, 256, 0, st>>>(oc, map, nullptr, w_o, y, T_, g.d, g.d, g.d);
}
template void launch_out_proj_simt<float>(const float*, const float*, float*, float*, const StepGeom&, cudaStream_t);
template void launch_out_proj_simt<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, float*, __nv_bfloat16*,
                                                  const StepGeom&, cudaStream_t);

// ------------------------------------------------------------------------------------------------ Q post-pass
// Per token: drift score of the scoring head (Sec. 3.1) against the stored query of the previous step, then the
// store of this step's query for the next one (Sec. 3.2), then the rotary embedding of all heads.
template <typename T>
__global__ void __launch_bounds__(128) q_post_kernel(const float* __restrict__ qf, int ldq,
                                                     const float2* __restrict__ rope_cs, float* __restrict__ q_prev,
                                                     float* __restrict__ scores, int has_prev, T* __restrict__ q,
                                                     StepGeom g) {
  __shared__ float red[3][4];
  const int t = blockIdx.x;
  const int hd = g.head_dim, half = hd >> 1;
  const float* row = qf + (size_t)t * ldq;
  const int cr = g.cache_row(t);
  float* qp = q_prev + (size_t)cr * hd;
  const float* q0 = row + g.score_head * hd;
  float dot = 0.f, n1 = 0.f, n2 = 0.f;
  for (int j = threadIdx.x; j < hd; j += blockDim.x) {
    const float a = q0[j];
    if (has_prev) {
      const float b = qp[j];
      dot = fmaf(a, b, dot); n1 = fmaf(a, a, n1); n2 = fmaf(b, b, n2);
    }
    qp[j] = a;
  }
  if (has_prev) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      dot += __shfl_xor_sync(0xffffffffu, dot, o);
      n1 += __shfl_xor_sync(0xffffffffu, n1, o);
      n2 += __shfl_xor_sync(0xffffffffu, n2, o);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { red[0][warp] = dot; red[1][warp] = n1; red[2][warp] = n2; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float D = 0.f, A = 0.f, B = 0.f;
      for (int w_ = 0; w_ < (int)(blockDim.x >> 5); ++w_) { D += red[0][w_]; A += red[1][w_]; B += red[2][w_]; }
      const float den = sqrtf(A) * sqrtf(B);
      const float c = den > 0.f ? D / den : 0.f;
      scores[t] = 1.f - c;
    }
  } else if (threadIdx.x == 0) {
    scores[t] = __int_as_float(0x7f800000);  // +inf: nothing to compare with
  }
  const int pos = g.position(t);
  const float2* cs = rope_cs + (size_t)pos * half;
  T* out = q + (size_t)t * g.d;
  for (int p = threadIdx.x; p < g.d / 2; p += blockDim.x) {
    const int h = p / half, j = p - h * half;
    const float a = row[h * hd + j], b = row[h * hd + j + half];
    const float2 c = cs[j];
    out[h * hd + j] = from_f<T>(a * c.x - b * c.y);
    out[h * hd + j + half] = from_f<T>(a * c.y + b * c.x);
  }
}

template <typename T>
void launch_q_post_simt(const float* qf, int ldq, const float* rope_cs, float* q_prev, float* scores, bool has_prev,
                        T* q, const StepGeom& g, cudaStream_t st) {
  if (g.tokens() <= 0) return;
  q_post_kernel<T><<<g.tokens(), 128, 0, st>>>(qf, ldq, reinterpret_cast<const float2*>(rope_cs), q_prev, scores,
                                               has_prev ? 1 : 0, q, g);
}
template void launch_q_post_simt<float>(const float*, int, const float*, float*, float*, bool, float*, const StepGeom&,
                                        cudaStream_t);
template void launch_q_post_simt<__nv_bfloat16>(const float*, int, const float*, float*, float*, bool, __nv_bfloat16*,
                                                const StepGeom&, cudaStream_t);

// ------------------------------------------------------------------------------------------------ K/V post-pass
// Eq. 3 / Alg. 1 lines 8-9: the refreshed rows replace their cache rows; every other cache row is left untouched.
template <typename T>
__global__ void __launch_bounds__(128) kv_post_kernel(const float* __restrict__ kvf, int ld,
                                                      const int* __restrict__ idx, const int* __restrict__ count,
                                                      const float2* __restrict__ rope_cs, T* __restrict__ kc,
                                                      T* __restrict__ vc, StepGeom g, int* status) {
  const int r = blockIdx.x;
  if (count && r >= checked_count(*count, g.tokens(), status)) return;
  const int t = idx ? idx[r] : r;
  if (idx && !token_ok(t, g.tokens(), status)) return;   // no cache row to write
  const int hd = g.head_dim, half = hd >> 1, d = g.d;
  const size_t cr = (size_t)g.cache_row(t);
  const float* krow = kvf + (size_t)r * ld;
  const float* vrow = krow + d;
  const float2* cs = rope_cs + (size_t)g.position(t) * half;
  T* ko = kc + cr * d;
  T* vo = vc + cr * d;
  for (int p = threadIdx.x; p < d / 2; p += blockDim.x) {
    const int h = p / half, j = p - h * half;
    const float a = krow[h * hd + j], b = krow[h * hd + j + half];
    const float2 c = cs[j];
    ko[h * hd + j] = from_f<T>(a * c.x - b * c.y);
    ko[h * hd + j + half] = from_f<T>(a * c.y + b * c.x);
  }
  for (int j = threadIdx.x; j < d; j += blockDim.x) vo[j] = from_f<T>(vrow[j]);
}

template <typename T>
void launch_kv_post_simt(const float* kvf, int ld, const int* idx, const int* count, const float* rope_cs, T* kc,
                         T* vc, const StepGeom& g, cudaStream_t st, int* status) {
  if (g.tokens() <= 0) return;
  kv_post_kernel<T><<<g.tokens(), 128, 0, st>>>(kvf, ld, idx, count, reinterpret_cast<const float2*>(rope_cs), kc, vc,
                                                g, status);
}
template void launch_kv_post_simt<float>(const float*, int, const int*, const int*, const float*, float*, float*,
                                         const StepGeom&, cudaStream_t, int*);
template void launch_kv_post_simt<__nv_bfloat16>(const float*, int, const int*, const int*, const float*,
                                                 __nv_bfloat16*, __nv_bfloat16*, const StepGeom&, cudaStream_t, int*);

// ------------------------------------------------------------------------------------------------ attention
// Eq. 4 / Alg. 2 line 8 (row-sparse) and Alg. 1 line 10 (all rows): bidirectional softmax attention, no mask,
// one warp per (query row, head), online softmax in fp32.  The result row is written into the O cache; rows
// that are not computed keep what they hold (Alg. 2 lines 9-10).
template <typename T, int EPL>
__global__ void __launch_bounds__(128) attention_simt_kernel(const T* __restrict__ q, const T* __restrict__ kc,
                                                             const T* __restrict__ vc, const int* __restrict__ idx,
                                                             const int* __restrict__ count, T* __restrict__ oc,
                                                             StepGeom g, int rows_max, int* status) {
  const int task = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int r = task / g.n_heads, h = task - r * g.n_heads;
  const int n_rows = count ? checked_count(*count, rows_max, status) : rows_max;
  if (r >= n_rows) return;
  const int t = idx ? idx[r] : r;
  if (idx && !token_ok(t, rows_max, status)) return;     // neither a query row to read nor a cache row to write
  const int b = t / g.seq_act;
  const int hd = g.head_dim, d = g.d;
  const float scale = rsqrtf((float)hd);
  float qv[EPL], acc[EPL];
  const T* qrow = q + (size_t)t * d + h * hd + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; ++e) { qv[e] = to_f<T>(qrow[e]) * scale; acc[e] = 0.f; }
  float m = -INFINITY, l = 0.f;
  const T* kbase = kc + (size_t)b * g.max_seq * d + h * hd + lane * EPL;
  const T* vbase = vc + (size_t)b * g.max_seq * d + h * hd + lane * EPL;
  for (int j = 0; j < g.kv_len; ++j) {
    const T* kr = kbase + (size_t)j * d;
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) s = fmaf(qv[e], to_f<T>(kr[e]), s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float m_new = fmaxf(m, s);
    const float corr = __expf(m - m_new);
    const float p = __expf(s - m_new);
    l = l * corr + p;
    const T* vr = vbase + (size_t)j * d;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(acc[e], corr, p * to_f<T>(vr[e]));
    m = m_new;
  }
  const float inv = 1.f / l;
  T* orow = oc + (size_t)g.cache_row(t) * d + h * hd + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; ++e) orow[e] = from_f<T>(acc[e] * inv);
}

template <typename T>
void launch_attention_simt(const T* q, const T* kc, const T* vc, const int* idx, const int* count, T* oc,
                           const StepGeom& g, cudaStream_t st, int* status) {
  const int rows_max = g.tokens();
  if (rows_max <= 0) return;
  const long tasks = (long)rows_max * g.n_heads;
  const int grid = (int)((tasks + 3) / 4);
  switch (g.head_dim / 32) {
    case 1: attention_simt_kernel<T, 1><<<grid, 128, 0, st>>>(q, kc, vc, idx, count, oc, g, rows_max, status); break;
    case 2: attention_simt_kernel<T, 2><<<grid, 128, 0, st>>>(q, kc, vc, idx, count, oc, g, rows_max, status); break;
    case 4: attention_simt_kernel<T, 4><<<grid, 128, 0, st>>>(q, kc, vc, idx, count, oc, g, rows_max, status); break;
    case 8: attention_simt_kernel<T, 8><<<grid, 128, 0, st>>>(q, kc, vc, idx, count, oc, g, rows_max, status); break;
    default: break;  // rejected at creation
  }
}
template void launch_attention_simt<float>(const float*, const float*, const float*, const int*, const int*, float*,
                                           const StepGeom&, cudaStream_t, int*);
template void launch_attention_simt<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
                                                   const int*, const int*, __nv_bfloat16*, const StepGeom&,
                                                   cudaStream_t, int*);

}  // namespace dare
