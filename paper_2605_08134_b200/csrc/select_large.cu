// Stand-alone drift score and threshold/compaction for token counts far beyond one layer step (millions of rows):
// the same arithmetic as inside the layer step, organised for HBM bandwidth.
//   drift score (Sec. 3.1): one warp per row, 16-byte loads of both query rows, shuffle reduction
//   compaction (Eq. 2, complement): three passes over tiles of 16384 scores; the scores are read once
//     (1) per-tile count of refreshed tokens and the decisions themselves, a plain bit array -> scratch
//     (2) exclusive scan of the tile counts (one CTA) -> scratch, total -> *count
//     (3) per-tile compaction from the decision bits, written at the tile's offset: ascending index list
// No CTA waits for another; the order of the list does not depend on scheduling.  Passes 2 and 3 are launched
// programmatically dependent: their launch latency hides behind the pass before.
// A single pass (tiles handed out by ticket, every CTA publishing its tile's count and adding up the counts published
// before it back to the nearest known running total, entries staged in shared memory and written as whole lines) was
// built as well, list and count identical, and measured on the same 2^24 scores against 22.6 us for the three passes:
// 27.7-32.3 us with one tile per CTA (16384 down to 4096 scores per tile, walk by one warp), 33-40 us with the walk by
// the whole CTA, 40-65 us with resident CTAs that have the next two tiles copied into shared memory (bulk copies on
// an mbarrier) while they work.  All CTAs of a wave reach the walk at the same time, so the nearest known total is a
// whole wave back, and a CTA's loads do not overlap its walk: the chain per tile (scores -> scan -> publish -> walk
// -> write) is several microseconds long, and what a CTA has in flight during it does not cover it.
#include <math.h>
#include <mutex>

#include "dare_internal.h"
#include "tc_ptx.cuh"

namespace dare {

namespace {
constexpr int kThreads = 1024, kVecs = 4;
constexpr int kTile = kThreads * kVecs * 4;     // 16384 scores per CTA: four 16-byte vectors per thread
constexpr int kTileWords = kTile / 32;          // 512 words of decision bits per tile

__global__ void __launch_bounds__(256) drift_score_kernel(const float* __restrict__ a, const float* __restrict__ b,
                                                          long long rows, int hd, float* __restrict__ scores) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long r = warp0; r < rows; r += nwarps) {
    const float4* pa = reinterpret_cast<const float4*>(a + r * hd);
    const float4* pb = reinterpret_cast<const float4*>(b + r * hd);
    float dot = 0.f, n1 = 0.f, n2 = 0.f;
    for (int v = lane; v < hd / 4; v += 32) {
      const float4 x = pa[v], y = pb[v];
      dot += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
      n1 += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
      n2 += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      dot += __shfl_xor_sync(0xffffffffu, dot, o);
      n1 += __shfl_xor_sync(0xffffffffu, n1, o);
      n2 += __shfl_xor_sync(0xffffffffu, n2, o);
    }
    if (lane == 0) {
      const float den = sqrtf(n1) * sqrtf(n2);
      scores[r] = 1.f - (den > 0.f ? dot / den : 0.f);
    }
  }
}

// refreshed <=> !(s <= tau): a NaN score refreshes.
// Thread t of a tile owns the four 16-byte vectors k = 0..3 at scores[base + (k * 1024 + t) * 4 ...]: every load
// instruction of a warp covers 512 contiguous bytes, and all four are in flight before the first is used.  Returns
// its 16 decisions, bit 4k + j <-> element j of vector k.
__device__ __forceinline__ unsigned tile_flags(const float* __restrict__ scores, long long n, long long base, float tau) {
  float4 v[kVecs];
  bool full[kVecs];
#pragma unroll
  for (int k = 0; k < kVecs; ++k) {
    const long long i0 = base + ((long long)k * kThreads + threadIdx.x) * 4;
    full[k] = i0 + 3 < n;
    v[k] = make_float4(0.f, 0.f, 0.f, 0.f);                 // 0 <= tau or not, a missing element is masked out below
    if (full[k]) {
      v[k] = __ldcs(reinterpret_cast<const float4*>(scores + i0));
    } else {
      if (i0 < n) v[k].x = scores[i0];
      if (i0 + 1 < n) v[k].y = scores[i0 + 1];
      if (i0 + 2 < n) v[k].z = scores[i0 + 2];
    }
  }
  unsigned bits = 0;
#pragma unroll
  for (int k = 0; k < kVecs; ++k) {
    const long long i0 = base + ((long long)k * kThreads + threadIdx.x) * 4;
    unsigned b = (!(v[k].x <= tau) ? 1u : 0u) | (!(v[k].y <= tau) ? 2u : 0u) | (!(v[k].z <= tau) ? 4u : 0u) |
                 (!(v[k].w <= tau) ? 8u : 0u);
    if (!full[k]) {
      const long long left = n - i0;                        // elements of this vector that exist: <= 3, maybe <= 0
      b &= left <= 0 ? 0u : ((1u << (int)left) - 1u);
    }
    bits |= b << (4 * k);
  }
  return bits;
}

// exclusive prefix of `v` over the threads of the CTA (whole warps, at most 32 of them); *total = sum
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T v, T* warp_sums, T* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  T inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const T n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const T w = lane < (int)(blockDim.x >> 5) ? warp_sums[lane] : T(0);
    T winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const T n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_sums[lane] = winc - w;
    if (lane == 31) *total = winc;
  }
  __syncthreads();
  return warp_sums[warp] + inc - v;
}

// pass 1: the only pass that reads the scores.  Leaves the decisions as a plain bit array (bit i of the array <->
// score i) and the tile's count.  For one vector index k the 32 lanes of a warp hold the decisions on 128 consecutive
// scores, four bits each: eight lanes' nibbles make one 32-bit word of the array, put together with three shuffles.
__global__ void __launch_bounds__(kThreads) tile_flag_kernel(const float* __restrict__ scores, long long n, float tau,
                                                             int* __restrict__ tile_counts,
                                                             unsigned* __restrict__ flags) {
  __shared__ int total;
  ptx::pdl_launch_dependents();            // the scan's CTA may take its place now; it waits for this grid to complete
  if (threadIdx.x == 0) total = 0;
  __syncthreads();
  const unsigned bits = tile_flags(scores, n, (long long)blockIdx.x * kTile, tau);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned* tile_words = flags + (size_t)blockIdx.x * kTileWords;
#pragma unroll
  for (int k = 0; k < kVecs; ++k) {
    unsigned v = ((bits >> (4 * k)) & 0xfu) << (4 * (lane & 7));
    v |= __shfl_xor_sync(0xffffffffu, v, 1);
    v |= __shfl_xor_sync(0xffffffffu, v, 2);
    v |= __shfl_xor_sync(0xffffffffu, v, 4);
    // scores [(k * 1024 + 32 * warp + 8 * w) * 4, + 32) of the tile, w = lane / 8
    if ((lane & 7) == 0) tile_words[k * (kThreads / 8) + warp * 4 + (lane >> 3)] = v;
  }
  const int c = __reduce_add_sync(0xffffffffu, __popc(bits));
  if (lane == 0) atomicAdd(&total, c);
  __syncthreads();
  if (threadIdx.x == 0) tile_counts[blockIdx.x] = total;
}

// pass 2: exclusive scan of the tile counts, one CTA
__global__ void __launch_bounds__(kThreads) tile_scan_kernel(const int* __restrict__ tile_counts, int n_tiles,
                                                             int* __restrict__ tile_offsets, int* __restrict__ count) {
  __shared__ int warp_sums[32];
  __shared__ int total;
  ptx::pdl_wait();
  ptx::pdl_launch_dependents();
  int base = 0;
  for (int start = 0; start < n_tiles; start += kThreads) {
    const int i = start + threadIdx.x;
    const int v = i < n_tiles ? tile_counts[i] : 0;
    const int ex = block_exclusive_scan<int>(v, warp_sums, &total);
    if (i < n_tiles) tile_offsets[i] = base + ex;
    base += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) *count = base;
}

// pass 3: from the decision bits alone (4 bytes per thread instead of 128 bytes of scores).  One thread per word of
// 32 consecutive scores, 512 threads per tile: one scan of the words' popcounts places every thread, which then
// writes the indices of its set bits, ascending, at consecutive places.  Every lane of such a store lands in another
// sector (ncu: 10.7 sectors per request), yet the pass is bound by the chain load -> scan -> stores of its CTAs
// rather than by the stores: two other forms measured slower on the same 2^24 scores (22.7 us per call for this one):
// lane-consecutive stores, each list entry found by a binary search over the words' first places in shared memory
// (27.5 us), and 256-thread CTAs with two words per thread so that every tile is resident at once (25.5 us).
// No store goes past entry n - 1 of the list, whatever the offsets say: if another call raced on a shared scratch
// array, the list is wrong but the caller's buffer is the only memory written.
__global__ void __launch_bounds__(kTileWords) tile_scatter_kernel(const unsigned* __restrict__ flags,
                                                                  const int* __restrict__ tile_offsets,
                                                                  int* __restrict__ idx, long long n) {
  __shared__ int warp_sums[32];
  __shared__ int total;
  ptx::pdl_wait();                         // before any read: decisions (two kernels back) and offsets (one back)
  unsigned word = flags[(size_t)blockIdx.x * kTileWords + threadIdx.x];
  long long out = tile_offsets[blockIdx.x];
  out += block_exclusive_scan<int>(__popc(word), warp_sums, &total);
  const int i0 = (int)((long long)blockIdx.x * kTile) + (int)threadIdx.x * 32;
  while (word != 0u) {
    if (out >= 0 && out < n) idx[out] = i0 + __ffs((int)word) - 1;
    ++out;
    word &= word - 1u;
  }
}

}  // namespace

int select_large_tiles(long long n) { return (int)((n + kTile - 1) / kTile); }
size_t select_large_flag_bytes(long long n) { return (size_t)select_large_tiles(n) * kTileWords * sizeof(unsigned); }

cudaError_t launch_drift_scores(const float* a, const float* b, long long rows, int hd, float* scores,
                                cudaStream_t st) {
  if (rows <= 0) return cudaSuccess;
  long long blocks = (rows + 7) / 8;
  if (blocks > 148 * 16) blocks = 148 * 16;
  drift_score_kernel<<<(int)blocks, 256, 0, st>>>(a, b, rows, hd, scores);
  return cudaGetLastError();
}

// tile_counts and tile_offsets: device arrays of select_large_tiles(n) ints each; flags: 512 32-bit words per tile
cudaError_t launch_select_large(const float* scores, long long n, float tau, int* idx, int* count, int* tile_counts,
                                int* tile_offsets, unsigned* flags, cudaStream_t st) {
  const int tiles = select_large_tiles(n);
  if (tiles == 0) return cudaMemsetAsync(count, 0, sizeof(int), st);
  tile_flag_kernel<<<tiles, kThreads, 0, st>>>(scores, n, tau, tile_counts, flags);
  cudaError_t e = launch_pdl(tile_scan_kernel, dim3(1), dim3(kThreads), 0, st, 1, (const int*)tile_counts, tiles,
                             tile_offsets, count);
  if (e != cudaSuccess) return e;
  e = launch_pdl(tile_scatter_kernel, dim3(tiles), dim3(kTileWords), 0, st, 1, (const unsigned*)flags,
                 (const int*)tile_offsets, idx, n);
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

}  // namespace dare

// ------------------------------------------------------------------------------------------------------------------
// Compaction without any caller-provided or allocated scratch.
//
// Some hosts of this library hand all of the device's memory to one arena at start-up and forbid every later
// cudaMalloc (an inference server with a fixed memory plan), or sit in a latency-critical loop where the device-wide
// synchronisation an allocation implies is not acceptable.  For them the per-tile counts and offsets and the decision
// bits of the three-pass compaction live in arrays that are part of the library image: 2 x 1024 ints + 1024 x 512
// 32-bit words = 2 MB + 8 KB of device memory on every GPU that loads the library, held until the process exits.
// That bounds the call at 1024 tiles = 16,777,216 scores.
//
// In host code the name `g_select_scratch` is only a stand-in for the symbol; the address a kernel may use comes from
// cudaGetSymbolAddress, asked once per device with that device current (the first call on a device does this; make
// that first call outside any stream capture).  All calls on a device share the array: it still holds the previous
// call's tile counts when the next one starts (every entry a call reads is written by that call first, so nothing
// needs clearing), and two calls that overlap on the GPU (different streams) race on it.
namespace dare {
namespace {
constexpr int kStaticTiles = 1024;
// [0, 2 * tiles) ints: counts, offsets; behind them the decision words
static __device__ __align__(256) int g_select_scratch[2 * kStaticTiles + kStaticTiles * kTileWords];
constexpr int kMaxDevices = 64;
int* g_select_scratch_addr[kMaxDevices] = {};
std::mutex g_select_scratch_mutex;

cudaError_t static_scratch_for_current_device(int** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_select_scratch_mutex);
  if (g_select_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_select_scratch);
    if (e != cudaSuccess) return e;
    g_select_scratch_addr[dev] = static_cast<int*>(p);
  }
  *out = g_select_scratch_addr[dev];
  return cudaSuccess;
}
}  // namespace
}  // namespace dare

extern "C" int64_t dare_select_compact_static_max_tokens(void) { return (int64_t)dare::kStaticTiles * dare::kTile; }

extern "C" dare_status_t dare_select_compact_static(const float* scores, int64_t n_tokens, float threshold, int32_t* idx,
                                                    int32_t* count, void* cuda_stream) {
  if (!scores || !idx || !count) return DARE_ERR_INVALID_ARG;
  if (isnan(threshold)) return DARE_ERR_INVALID_ARG;
  if (n_tokens < 0 || n_tokens > dare_select_compact_static_max_tokens()) return DARE_ERR_SHAPE;   // beyond the array
  if ((reinterpret_cast<uintptr_t>(scores) & 15u) != 0) return DARE_ERR_ALIGN;
  int* scratch = nullptr;
  if (dare::static_scratch_for_current_device(&scratch) != cudaSuccess) { cudaGetLastError(); return DARE_ERR_CUDA; }
  cudaError_t e = dare::launch_select_large(scores, n_tokens, threshold, idx, count, scratch,
                                            scratch + dare::kStaticTiles,
                                            reinterpret_cast<unsigned*>(scratch + 2 * dare::kStaticTiles),
                                            (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) { cudaGetLastError(); return DARE_ERR_CUDA; }
  return DARE_OK;
}
