// Stand-alone drift score and threshold/compaction for token counts far beyond one layer step (millions of rows):
// the same arithmetic as inside the layer step, organised for HBM bandwidth.
//   drift score (Sec. 3.1): one warp per row, 16-byte loads of both query rows, shuffle reduction
//   compaction (Eq. 2, complement): three passes over tiles of 4096 scores
//     (1) per-tile count of refreshed tokens  -> scratch
//     (2) exclusive scan of the tile counts (one CTA) -> scratch, total -> *count
//     (3) per-tile ballot/popcount compaction written at the tile's offset: ascending index list
// No CTA waits for another; the order of the list does not depend on scheduling.
#include <math.h>
#include <mutex>

#include "dare_internal.h"

namespace dare {

namespace {
constexpr int kTile = 4096;          // scores per CTA (1024 threads x 4)

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

// refreshed <=> !(s <= tau): a NaN score refreshes
__device__ __forceinline__ int tile_flags(const float* __restrict__ scores, long long n, long long base, float tau,
                                          bool (&sel)[4]) {
  int c = 0;
  const long long i0 = base + (long long)threadIdx.x * 4;
  if (i0 + 3 < n) {
    const float4 v = *reinterpret_cast<const float4*>(scores + i0);
    sel[0] = !(v.x <= tau); sel[1] = !(v.y <= tau); sel[2] = !(v.z <= tau); sel[3] = !(v.w <= tau);
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) sel[k] = (i0 + k < n) ? !(scores[i0 + k] <= tau) : false;
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) c += sel[k] ? 1 : 0;
  return c;
}

// exclusive prefix of `v` over the 1024 threads of the CTA; *total = sum
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const int w = warp_sums[lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_sums[lane] = winc - w;
    if (lane == 31) *total = winc;
  }
  __syncthreads();
  return warp_sums[warp] + inc - v;
}

__global__ void __launch_bounds__(1024) tile_count_kernel(const float* __restrict__ scores, long long n, float tau,
                                                          int* __restrict__ tile_counts) {
  __shared__ int warp_sums[32];
  __shared__ int total;
  bool sel[4];
  const int c = tile_flags(scores, n, (long long)blockIdx.x * kTile, tau, sel);
  block_exclusive_scan(c, warp_sums, &total);
  if (threadIdx.x == 0) tile_counts[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) tile_scan_kernel(const int* __restrict__ tile_counts, int n_tiles,
                                                         int* __restrict__ tile_offsets, int* __restrict__ count) {
  __shared__ int warp_sums[32];
  __shared__ int total;
  int base = 0;
  for (int start = 0; start < n_tiles; start += 1024) {
    const int i = start + threadIdx.x;
    const int v = i < n_tiles ? tile_counts[i] : 0;
    const int ex = block_exclusive_scan(v, warp_sums, &total);
    if (i < n_tiles) tile_offsets[i] = base + ex;
    base += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) *count = base;
}

__global__ void __launch_bounds__(1024) tile_scatter_kernel(const float* __restrict__ scores, long long n, float tau,
                                                            const int* __restrict__ tile_offsets,
                                                            int* __restrict__ idx) {
  __shared__ int warp_sums[32];
  __shared__ int total;
  bool sel[4];
  const long long base = (long long)blockIdx.x * kTile;
  const int c = tile_flags(scores, n, base, tau, sel);
  int out = tile_offsets[blockIdx.x] + block_exclusive_scan(c, warp_sums, &total);
#pragma unroll
  for (int k = 0; k < 4; ++k)
    if (sel[k]) idx[out++] = (int)(base + (long long)threadIdx.x * 4 + k);
}

}  // namespace

int select_large_tiles(long long n) { return (int)((n + kTile - 1) / kTile); }

cudaError_t launch_drift_scores(const float* a, const float* b, long long rows, int hd, float* scores,
                                cudaStream_t st) {
  if (rows <= 0) return cudaSuccess;
  long long blocks = (rows + 7) / 8;
  if (blocks > 148 * 16) blocks = 148 * 16;
  drift_score_kernel<<<(int)blocks, 256, 0, st>>>(a, b, rows, hd, scores);
  return cudaGetLastError();
}

// tile_counts and tile_offsets: device arrays of select_large_tiles(n) ints each
cudaError_t launch_select_large(const float* scores, long long n, float tau, int* idx, int* count, int* tile_counts,
                                int* tile_offsets, cudaStream_t st) {
  const int tiles = select_large_tiles(n);
  if (tiles == 0) return cudaMemsetAsync(count, 0, sizeof(int), st);
  tile_count_kernel<<<tiles, 1024, 0, st>>>(scores, n, tau, tile_counts);
  tile_scan_kernel<<<1, 1024, 0, st>>>(tile_counts, tiles, tile_offsets, count);
  tile_scatter_kernel<<<tiles, 1024, 0, st>>>(scores, n, tau, tile_offsets, idx);
  return cudaGetLastError();
}

}  // namespace dare

// ------------------------------------------------------------------------------------------------------------------
// Compaction without any caller-provided or allocated scratch.
//
// Some hosts of this library hand all of the device's memory to one arena at start-up and forbid every later
// cudaMalloc (an inference server with a fixed memory plan), or sit in a latency-critical loop where the device-wide
// synchronisation an allocation implies is not acceptable.  For them the per-tile counts and offsets of the three-pass
// compaction live in a small array that is part of the library image: 2 x 4096 ints = 32 KB of device memory on every
// GPU that loads the library, held until the process exits.  That bounds the call at 4096 tiles = 16,777,216 scores.
//
// In host code the name `g_select_scratch` is only a stand-in for the symbol; the address a kernel may use comes from
// cudaGetSymbolAddress, asked once per device with that device current (the first call on a device does this; make
// that first call outside any stream capture).  All calls on a device share the array: it still holds the previous
// call's tile counts when the next one starts (every entry a call reads is written by that call first, so nothing
// needs clearing), and two calls that overlap on the GPU (different streams) race on it.
namespace dare {
namespace {
constexpr int kStaticTiles = 4096;
static __device__ __align__(256) int g_select_scratch[2 * kStaticTiles];
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
                                            scratch + dare::kStaticTiles, (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) { cudaGetLastError(); return DARE_ERR_CUDA; }
  return DARE_OK;
}
