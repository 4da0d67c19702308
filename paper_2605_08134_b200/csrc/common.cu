// Memory-bound kernels shared by both kernel paths: rotary table, RMSNorm, threshold + compaction, row gather.
#include <type_traits>
#include "dare_internal.h"
#include "tc_ptx.cuh"

namespace dare {

// ------------------------------------------------------------------------------------------------ rotary table
// cs[pos][j] = (cos, sin)(pos * theta^(-2j/head_dim)), evaluated in fp64 and stored as fp32.
__global__ void rope_table_kernel(float2* cs, int max_seq, int half, double theta, int head_dim) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_seq * half) return;
  int pos = i / half, j = i % half;
  double inv_freq = pow(theta, -2.0 * (double)j / (double)head_dim);
  double s, c;
  sincos((double)pos * inv_freq, &s, &c);
  cs[i] = make_float2((float)c, (float)s);
}

void launch_rope_table(float* cs, int max_seq, int head_dim, double theta, cudaStream_t st) {
  int half = head_dim / 2;
  int n = max_seq * half;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(reinterpret_cast<float2*>(cs), max_seq, half, theta, head_dim);
}

// ------------------------------------------------------------------------------------------------ RMSNorm
// Alg. 1/2 line 1.  One CTA per token row, 16-byte accesses, the row held in registers between the two passes.
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* p, float (&v)[4]) {
    float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&v)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
    uint4 t = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&t);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint4 t;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&t);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = t;
  }
};

__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (lane < nw) ? red[lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  __syncthreads();
  return t;
}

// kEarlyGain: the gain (a weight, independent of the previous kernel in the stream) is read before the dependency
// wait, which takes one memory round trip off a short step's critical path; it costs registers (half the resident
// CTAs), so steps with many rows, which are bandwidth-bound, read it afterwards.
template <typename T, int MAXV, bool kEarlyGain>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const T* __restrict__ x, const float* __restrict__ gain,
                                                      T* __restrict__ xn, int d, float eps,
                                                      unsigned long long* dbg) {
  constexpr int N = Vec16<T>::N;
  __shared__ float red[32];
  if (dbg && threadIdx.x == 0) {
    const unsigned long long t = ptx::globaltimer_ns();
    if (blockIdx.x == 0) dbg[0] = t;
    atomicMax(&dbg[4], t);                     // latest CTA start
  }
  const int nvec0 = d / N;
  float gn[kEarlyGain ? MAXV : 1][N];
#pragma unroll
  for (int i = 0; i < (kEarlyGain ? MAXV : 0); ++i) {
    const int vi = threadIdx.x + i * blockDim.x;
    if (vi < nvec0) {
#pragma unroll
      for (int e = 0; e < N; e += 4) {
        const float4 t = *reinterpret_cast<const float4*>(gain + vi * N + e);
        gn[i][e] = t.x; gn[i][e + 1] = t.y; gn[i][e + 2] = t.z; gn[i][e + 3] = t.w;
      }
    }
  }
  // x may be the output of the previous kernel in the stream (the previous layer of a model), so it is read only
  // after that kernel has completed.  Its lines are asked into the L2 before that, though (the L2 is where a later
  // write of the producer lands too, so nothing stale can come of it): an input that lies in HBM is then on its way
  // while this CTA waits.
  if (kEarlyGain) {
    const char* xb = reinterpret_cast<const char*>(x + (size_t)blockIdx.x * d);
    const int row_bytes = d * (int)sizeof(T);
    for (int off = (int)threadIdx.x * 128; off < row_bytes; off += (int)blockDim.x * 128) ptx::prefetch_l2(xb + off);
  }
  ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  if (dbg && threadIdx.x == 0) {
    const unsigned long long t = ptx::globaltimer_ns();
    if (blockIdx.x == 0) dbg[2] = t;
    atomicMax(&dbg[3], t);                     // latest return from the wait
  }
  const size_t row = blockIdx.x;
  const T* xr = x + row * d;
  T* yr = xn + row * d;
  const int nvec = d / N;
  float v[MAXV][N];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    int vi = threadIdx.x + i * blockDim.x;
    if (vi < nvec) {
      Vec16<T>::load(xr + vi * N, v[i]);
#pragma unroll
      for (int e = 0; e < N; ++e) ss += v[i][e] * v[i][e];
    }
  }
  for (int vi = threadIdx.x + MAXV * blockDim.x; vi < nvec; vi += blockDim.x) {  // rows wider than the register file
    float t[N];
    Vec16<T>::load(xr + vi * N, t);
#pragma unroll
    for (int e = 0; e < N; ++e) ss += t[e] * t[e];
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)d + eps);
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    int vi = threadIdx.x + i * blockDim.x;
    if (vi < nvec) {
      if (!kEarlyGain) {
#pragma unroll
        for (int e = 0; e < N; e += 4) {
          const float4 t = *reinterpret_cast<const float4*>(gain + vi * N + e);
          gn[0][e] = t.x; gn[0][e + 1] = t.y; gn[0][e + 2] = t.z; gn[0][e + 3] = t.w;
        }
      }
#pragma unroll
      for (int e = 0; e < N; ++e) v[i][e] = v[i][e] * r * gn[kEarlyGain ? i : 0][e];
      Vec16<T>::store(yr + vi * N, v[i]);
    }
  }
  for (int vi = threadIdx.x + MAXV * blockDim.x; vi < nvec; vi += blockDim.x) {
    float t[N];
    Vec16<T>::load(xr + vi * N, t);
#pragma unroll
    for (int e = 0; e < N; ++e) t[e] = t[e] * r * gain[vi * N + e];
    Vec16<T>::store(yr + vi * N, t);
  }
  if (dbg && threadIdx.x == 0) atomicMax(&dbg[5], ptx::globaltimer_ns());   // latest CTA end
}

// Many rows (the step is then a stream through HBM): a CTA takes ROWS consecutive rows at once, all of their loads in
// flight before the one block reduction they share, the data kept as packed bf16 between the two passes.
// d <= 4096 (two 16-byte vectors per thread).
template <int ROWS>
__global__ void __launch_bounds__(256) rmsnorm_stream_kernel(const __nv_bfloat16* __restrict__ x,
                                                             const float* __restrict__ gain,
                                                             __nv_bfloat16* __restrict__ xn, int rows, int d, float eps) {
  __shared__ float red[8][ROWS];
  ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  const int nvec = d / 8, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const size_t row0 = (size_t)blockIdx.x * ROWS;
  uint4 raw[ROWS][2];
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int vi = threadIdx.x + i * 256;
      raw[r][i] = make_uint4(0u, 0u, 0u, 0u);
      if (vi < nvec && row0 + r < (size_t)rows) raw[r][i] = *reinterpret_cast<const uint4*>(x + (row0 + r) * d + vi * 8);
    }
  }
  float ss[ROWS];
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    ss[r] = 0.f;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw[r][i]);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(h[e]);
        ss[r] += f.x * f.x + f.y * f.y;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss[r] += __shfl_xor_sync(0xffffffffu, ss[r], o);
    if (lane == 0) red[warp][r] = ss[r];
  }
  __syncthreads();
  float gn[2][8];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int vi = threadIdx.x + i * 256;
    if (vi < nvec) {
#pragma unroll
      for (int e = 0; e < 8; e += 4) {
        const float4 t = *reinterpret_cast<const float4*>(gain + vi * 8 + e);
        gn[i][e] = t.x; gn[i][e + 1] = t.y; gn[i][e + 2] = t.z; gn[i][e + 3] = t.w;
      }
    }
  }
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w][r];
    const float sc = rsqrtf(tot / (float)d + eps);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int vi = threadIdx.x + i * 256;
      if (vi < nvec && row0 + r < (size_t)rows) {
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw[r][i]);
        uint4 o;
        __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(h[e]);
          oh[e] = __floats2bfloat162_rn(f.x * sc * gn[i][2 * e], f.y * sc * gn[i][2 * e + 1]);
        }
        *reinterpret_cast<uint4*>(xn + (row0 + r) * d + vi * 8) = o;
      }
    }
  }
}

template <typename T>
void launch_rmsnorm(const T* x, const float* gain, T* xn, int rows, int d, float eps, cudaStream_t st,
                    unsigned long long* dbg) {
  if (rows <= 0) return;
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    constexpr int ROWS = 2;        // measured at 16384 rows of 4096: 56 us (1 row per CTA: 65, 4: 65, 8: 93)
    if (rows > 2048 && d % 8 == 0 && d / 8 <= 512 && dbg == nullptr) {
      launch_pdl(rmsnorm_stream_kernel<ROWS>, dim3((rows + ROWS - 1) / ROWS), dim3(256), 0, st, 1, x, gain, xn, rows, d,
                 eps);
      return;
    }
  }
  int nvec = d / Vec16<T>::N;
  int threads = nvec >= 512 ? 256 : (nvec >= 128 ? 128 : ((nvec + 31) / 32) * 32);
  if (threads > 256) threads = 256;
  if (rows <= 2048)
    launch_pdl(rmsnorm_kernel<T, 2, true>, dim3(rows), dim3(threads), 0, st, 1, x, gain, xn, d, eps, dbg);
  else
    launch_pdl(rmsnorm_kernel<T, 2, false>, dim3(rows), dim3(threads), 0, st, 1, x, gain, xn, d, eps, dbg);
}
template void launch_rmsnorm<float>(const float*, const float*, float*, int, int, float, cudaStream_t,
                                    unsigned long long*);
template void launch_rmsnorm<__nv_bfloat16>(const __nv_bfloat16*, const float*, __nv_bfloat16*, int, int, float,
                                            cudaStream_t, unsigned long long*);

// ------------------------------------------------------------------------------------------------ selection
// Eq. 2 and its complement: token t is refreshed iff !(s_t <= tau) (a NaN score refreshes).  The refresh set is
// written as an ascending index list: every thread takes four consecutive tokens of a chunk of 4096, a warp scan
// and a scan over the warp totals give each thread its place; the staleness counters of Sec. 4 and the start of
// every sequence's slice of the list come out of the same pass.  One CTA walks the chunks, which keeps the list
// ordered without any inter-CTA hand-off (T <= a few 10^4 per layer step).
// With more than one chunk the launch has one CTA per chunk, and none waits for another: a CTA first counts the
// refreshed tokens of the chunks before its own from their scores (a few 16-byte loads per thread, from the L2), which
// is where its part of the list starts.
// ---- the step's own threshold (Sec. 3.1 speaks of dynamic thresholding; the reuse-rate allocation turns a rate into
// the matching quantile of the drift scores): tau_t = the k-th smallest score of this step, so that the k tokens that
// drifted least are reused (and every token tied with the k-th).  Exact selection by four passes over the scores'
// order-preserving 32-bit keys, eight bits at a time (histogram in shared memory, then the bin that holds rank k);
// one CTA: a step has at most a few 10^4 tokens.  NaN scores sort last and are never reused.
// k <= 0: tau = -inf (nothing reused); k >= n or more than the scores that are numbers: +inf.
__device__ __forceinline__ unsigned score_key(float s) {
  if (s != s) return 0xffffffffu;
  const unsigned u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__global__ void __launch_bounds__(1024) kth_score_kernel(const float* __restrict__ scores, int n, int k,
                                                         float* __restrict__ tau_out) {
  __shared__ int hist[256];
  __shared__ unsigned s_prefix;
  __shared__ int s_rank;
  ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  if (k <= 0 || k >= n) {
    if (threadIdx.x == 0) *tau_out = __int_as_float(k <= 0 ? 0xff800000 : 0x7f800000);
    return;
  }
  unsigned prefix = 0u, mask = 0u;
  int rank = k;                                       // rank (1-based) of the wanted key among the keys that match the prefix
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      const unsigned key = score_key(scores[i]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int cum = 0, b = 0;
      for (; b < 255; ++b) {
        if (cum + hist[b] >= rank) break;
        cum += hist[b];
      }
      s_prefix = prefix | ((unsigned)b << shift);
      s_rank = rank - cum;
    }
    __syncthreads();
    prefix = s_prefix;
    rank = s_rank;
    mask |= 255u << shift;
  }
  if (threadIdx.x == 0) {
    const unsigned u = (prefix & 0x80000000u) ? (prefix & 0x7fffffffu) : ~prefix;
    float tau = __uint_as_float(u);
    if (tau != tau) tau = __int_as_float(0x7f800000);         // rank k falls among the NaN scores: every number is reused
    *tau_out = tau;
  }
}
void launch_kth_score(const float* scores, int n, int k, float* tau_out, cudaStream_t st) {
  launch_pdl(kth_score_kernel, dim3(1), dim3(1024), 0, st, 1, scores, n, k, tau_out);
}

constexpr int kSelPerThread = 4;
__global__ void __launch_bounds__(1024) select_kernel(const float* __restrict__ scores, float tau, int select_all,
                                                      StepGeom g, int* __restrict__ idx, int* __restrict__ count,
                                                      int* __restrict__ batch_off, int* __restrict__ delta,
                                                      int wait_at_end, const float* __restrict__ tau_dev) {
  __shared__ int warp_tot[32];
  __shared__ int before_chunk;
  if (threadIdx.x == 0) before_chunk = 0;
  if (!wait_at_end) ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  if (tau_dev != nullptr) tau = *tau_dev;                // the threshold the step worked out itself
  const int T = g.tokens();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kChunk = 1024 * kSelPerThread;
  const int chunk0 = (int)blockIdx.x * kChunk;            // this CTA's chunk: tokens [chunk0, chunk0 + kChunk)
  int base = 0;
  if (blockIdx.x > 0) {
    if (select_all) {
      base = chunk0;
    } else {
      __syncthreads();
      int c = 0;
      for (int i = (int)threadIdx.x * 4; i < chunk0; i += kChunk) {     // whole chunks: no tail, 16-byte aligned
        const float4 v = *reinterpret_cast<const float4*>(scores + i);
        c += (!(v.x <= tau) ? 1 : 0) + (!(v.y <= tau) ? 1 : 0) + (!(v.z <= tau) ? 1 : 0) + (!(v.w <= tau) ? 1 : 0);
      }
      c = __reduce_add_sync(0xffffffffu, c);
      if (lane == 0 && c != 0) atomicAdd(&before_chunk, c);
      __syncthreads();
      base = before_chunk;
    }
  }
  for (int start = chunk0; start < chunk0 + kChunk && start < T; start += kChunk) {
    const int t0 = start + threadIdx.x * kSelPerThread;
    // all loads of the chunk first (scores and staleness counters): one memory round trip
    float sc[kSelPerThread];
    int cr[kSelPerThread], stale[kSelPerThread];
#pragma unroll
    for (int k = 0; k < kSelPerThread; ++k) {
      const int t = t0 + k;
      sc[k] = 0.f; cr[k] = 0; stale[k] = 0;
      if (t < T) {
        cr[k] = g.cache_row(t);
        if (!select_all) sc[k] = scores[t];
        stale[k] = delta[cr[k]];
      }
    }
    bool sel[kSelPerThread];
    int mine = 0;
#pragma unroll
    for (int k = 0; k < kSelPerThread; ++k) {
      sel[k] = t0 + k < T && (select_all ? true : !(sc[k] <= tau));
      mine += sel[k] ? 1 : 0;
    }
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += n;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    // (32 warp totals: every thread sums the ones before its warp; lane w of a warp holds total w)
    const int wt = warp_tot[lane];
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 32; ++w) {
      const int v = __shfl_sync(0xffffffffu, wt, w);
      before += w < warp ? v : 0;
      total += v;
    }
    int out = base + before + inc - mine;
#pragma unroll
    for (int k = 0; k < kSelPerThread; ++k) {
      const int t = t0 + k;
      if (t < T) {
        // a sequence starts at this token: its slice of the ascending list starts at the current place
        if (t % g.seq_act == 0) batch_off[t / g.seq_act] = out;
        if (sel[k]) idx[out++] = t;
        delta[cr[k]] = sel[k] ? 0 : stale[k] + 1;
      }
    }
    base += total;
    __syncthreads();
  }
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
    *count = base;
    batch_off[g.batch] = base;
  }
  if (wait_at_end) ptx::pdl_wait();
}

// The same for short steps: one token per thread and chunk of 1024, warp ballot + popcount (less index arithmetic
// per token, which is what a step of a few hundred tokens pays for).
__global__ void __launch_bounds__(1024) select_small_kernel(const float* __restrict__ scores, float tau, int select_all,
                                                      StepGeom g, int* __restrict__ idx, int* __restrict__ count,
                                                      int* __restrict__ batch_off, int* __restrict__ delta,
                                                      int wait_at_end, const float* __restrict__ tau_dev) {
  __shared__ int warp_excl[32];
  __shared__ int chunk_total;
  const int T = g.tokens();
  // (the staleness counters are this kernel's own: their lines are asked into the L2 while it waits for the scores)
  for (int t = threadIdx.x * 32; t < T; t += 1024 * 32) ptx::prefetch_l2(delta + g.cache_row(t));
  if (!wait_at_end) ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  if (tau_dev != nullptr) tau = *tau_dev;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int base = 0;
  for (int start = 0; start < T; start += 1024) {
    const int t = start + threadIdx.x;
    const bool valid = t < T;
    // both loads of the token first (score and staleness counter): one memory round trip instead of two
    const int cr = valid ? g.cache_row(t) : 0;
    const int stale = valid ? delta[cr] : 0;
    bool sel = false;
    if (valid) sel = select_all ? true : !(scores[t] <= tau);
    const unsigned bal = __ballot_sync(0xffffffffu, sel);
    const int lane_prefix = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_excl[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {
      int v = warp_excl[lane], inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      warp_excl[lane] = inc - v;
      if (lane == 31) chunk_total = inc;
    }
    __syncthreads();
    if (valid) {
      const int out = base + warp_excl[warp] + lane_prefix;     // place of this token in the list, were it selected
      if (sel) idx[out] = t;
      // a sequence starts at this token: its slice of the ascending list starts here
      if (t % g.seq_act == 0) batch_off[t / g.seq_act] = out;
      delta[cr] = sel ? 0 : stale + 1;
    }
    base += chunk_total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    *count = base;
    batch_off[g.batch] = base;
  }
  if (wait_at_end) ptx::pdl_wait();
}

// beside_predecessor: the selection refreshes every token (it reads no scores) and nothing the kernel before it in the
// stream touches, so it runs beside that kernel and waits for it only before it leaves.
void launch_select(const float* scores, float tau, bool select_all, const StepGeom& g, int* idx, int* count,
                   int* batch_off, int* delta, cudaStream_t st, bool beside_predecessor, const float* tau_dev) {
  const int all = (select_all || scores == nullptr) ? 1 : 0;
  const int late = (beside_predecessor && all) ? 1 : 0;
  if (g.tokens() <= 2048)
    launch_pdl(select_small_kernel, dim3(1), dim3(1024), 0, st, 1, scores, tau, all, g, idx, count, batch_off, delta, late,
               tau_dev);
  else
    launch_pdl(select_kernel, dim3((g.tokens() + 1024 * kSelPerThread - 1) / (1024 * kSelPerThread)), dim3(1024), 0, st, 1,
               scores, tau, all, g, idx, count, batch_off, delta, late, tau_dev);
}

// ------------------------------------------------------------------------------------------------ diagnostics
// A wait nobody ends, with a short limit: the bounded wait of the tensor-core kernels on a barrier no thread and no
// copy ever arrives on.  It must give up after `limit_ns`, record the time-out in the status word and return normally.
__global__ void wait_probe_kernel(int* status, unsigned long long limit_ns, unsigned long long* waited_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const unsigned long long t0 = ptx::globaltimer_ns();
  const bool ok = ptx::mbar_wait(&bar, 0, status, limit_ns);
  if (threadIdx.x == 0 && waited_ns) *waited_ns = ok ? 0ull : ptx::globaltimer_ns() - t0;
}
void launch_wait_probe(int* status, unsigned long long limit_ns, unsigned long long* waited_ns, cudaStream_t st) {
  wait_probe_kernel<<<1, 32, 0, st>>>(status, limit_ns, waited_ns);
}
__global__ void poke_int_kernel(int* dst, int value) { *dst = value; }
void launch_poke_int(int* dst, int value, cudaStream_t st) { poke_int_kernel<<<1, 1, 0, st>>>(dst, value); }

// ------------------------------------------------------------------------------------------------ reused rows
// One warp per token row; rows refreshed in this step (staleness 0) are written by the projection itself.
template <typename T>
__global__ void __launch_bounds__(256) copy_reused_rows_kernel(const T* __restrict__ yc, T* __restrict__ y,
                                                               const int* __restrict__ delta, StepGeom g,
                                                               const int* __restrict__ gate_count, int gate_hi) {
  ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  if (gate_count != nullptr && *gate_count >= gate_hi) return;     // the dense form of the projection writes every row
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= g.tokens()) return;
  const int cr = g.cache_row(t);
  if (delta[cr] == 0) return;
  const uint4* s = reinterpret_cast<const uint4*>(yc + (size_t)cr * g.d);
  uint4* o = reinterpret_cast<uint4*>(y + (size_t)t * g.d);
  const int nvec = g.d * (int)sizeof(T) / 16;
  for (int v = threadIdx.x & 31; v < nvec; v += 32) o[v] = s[v];
}

template <typename T>
void launch_copy_reused_rows(const T* yc, T* y, const int* delta, const StepGeom& g, cudaStream_t st,
                             const int* gate_count, int gate_hi) {
  const int T_ = g.tokens();
  if (T_ <= 0) return;
  launch_pdl(copy_reused_rows_kernel<T>, dim3((T_ + 7) / 8), dim3(256), 0, st, 1, yc, y, delta, g, gate_count, gate_hi);
}
template void launch_copy_reused_rows<__nv_bfloat16>(const __nv_bfloat16*, __nv_bfloat16*, const int*, const StepGeom&,
                                                     cudaStream_t, const int*, int);

// ------------------------------------------------------------------------------------------------ row gather
// dst[r, :] = src[idx[r], :] for r < *count (Alg. 1 line 6: x_norm restricted to the refresh set).
template <typename T>
__global__ void __launch_bounds__(256) gather_rows_kernel(const T* __restrict__ src, const int* __restrict__ idx,
                                                          const int* __restrict__ count, T* __restrict__ dst,
                                                          int max_rows, int d) {
  const int n = min(*count, max_rows);
  constexpr int N = 16 / sizeof(T);
  const int nvec = d / N;
  for (int r = blockIdx.x; r < n; r += gridDim.x) {
    const uint4* s = reinterpret_cast<const uint4*>(src + (size_t)idx[r] * d);
    uint4* o = reinterpret_cast<uint4*>(dst + (size_t)r * d);
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) o[v] = s[v];
  }
}

template <typename T>
void launch_gather_rows(const T* src, const int* idx, const int* count, T* dst, int max_rows, int d, cudaStream_t st) {
  if (max_rows <= 0) return;
  int grid = max_rows < 148 * 8 ? max_rows : 148 * 8;
  gather_rows_kernel<T><<<grid, 256, 0, st>>>(src, idx, count, dst, max_rows, d);
}
// The same for the rows of a step's refresh set, by flat token index or (by_cache_row) by cache row: a stream of
// n * d elements, chained with programmatic dependent launch.
template <typename T>
__global__ void __launch_bounds__(256) gather_step_rows_kernel(const T* __restrict__ src, const int* __restrict__ idx,
                                                               const int* __restrict__ count, T* __restrict__ dst,
                                                               StepGeom g, int by_cache_row, int* status, int gate_hi) {
  ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  const int n = checked_count(*count, g.tokens(), status);
  if (n >= gate_hi) return;                              // the launch that would read the copy leaves as well
  constexpr int N = 16 / sizeof(T);
  const int nvec = g.d / N;
  for (int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < n; r += gridDim.x * (blockDim.x >> 5)) {
    const int tok = idx[r];
    if (!token_ok(tok, g.tokens(), status)) continue;      // the row of the compact copy keeps what it held
    const size_t srow = by_cache_row ? (size_t)g.cache_row(tok) : (size_t)tok;
    const uint4* s = reinterpret_cast<const uint4*>(src + srow * g.d);
    uint4* o = reinterpret_cast<uint4*>(dst + (size_t)r * g.d);
    for (int v = threadIdx.x & 31; v < nvec; v += 32) o[v] = s[v];
  }
}
template <typename T>
void launch_gather_step_rows(const T* src, const int* idx, const int* count, T* dst, const StepGeom& g, bool by_cache_row,
                             cudaStream_t st, int* status, int gate_hi) {
  const int T_ = g.tokens();
  if (T_ <= 0) return;
  const int grid = (T_ + 7) / 8 < 148 * 8 ? (T_ + 7) / 8 : 148 * 8;
  launch_pdl(gather_step_rows_kernel<T>, dim3(grid), dim3(256), 0, st, 1, src, idx, count, dst, g, by_cache_row ? 1 : 0,
             status, gate_hi);
}
template void launch_gather_step_rows<__nv_bfloat16>(const __nv_bfloat16*, const int*, const int*, __nv_bfloat16*,
                                                     const StepGeom&, bool, cudaStream_t, int*, int);
template void launch_gather_rows<float>(const float*, const int*, const int*, float*, int, int, cudaStream_t);
template void launch_gather_rows<__nv_bfloat16>(const __nv_bfloat16*, const int*, const int*, __nv_bfloat16*, int, int,
                                                cudaStream_t);

}  // namespace dare
