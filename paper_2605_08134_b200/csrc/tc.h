// Declarations of the tensor-core path (tcgen05 GEMM and attention kernels) shared between its translation units.
#pragma once

#include <cuda.h>

#include "dare_internal.h"

namespace dare {

enum { EPI_Q = 0, EPI_KV = 1, EPI_OUT = 2, EPI_SWIGLU = 3, EPI_F32 = 4,
       EPI_OUT_RES = 5 };   // EPI_OUT plus a residual row (chosen by the launcher when GemmParams::resid is set)

struct GemmParams {
  int K;                 // reduction length (multiple of 64)
  int m_tiles;           // row tiles of the launch (set by the launcher; a pair launch pads its grid to an even count)
  int m_total;           // dense: tokens of the step; gathered: capacity of the row list
  int seq_act;           // dense row mapping: rows per sequence ...
  int tiles_per_seq;     // ... and 128-row tiles per sequence
  int a_seq_stride;      // rows between sequences in A's row space
  int a_row0;            // first row of the window in A's row space
  const int* idx;        // gathered: token of each A row (ascending refresh set), else nullptr
  const int* count;      // gathered: device count of rows, else nullptr
  const __nv_bfloat16* gather_src;  // gathered: the matrix [*, K] whose rows idx[] the kernel fetches itself as its A
                                    // operand (Alg. 1 line 6); nullptr: A comes through the tensor map
  int gather_cache_rows; // gather_src is addressed by cache row (the O cache) instead of by flat token index
  int unit_gate;         // persistent listed launches issued as a pair of kernels: the two-CTA form runs when the count
                         // gives it at least this many (column tile, row-tile pair) units, the one-CTA form otherwise;
                         // 0: no gate
  StepGeom g;
  int n_split;           // n-tiles [0, n_split) use W0/out0, the rest W1/out1
  __nv_bfloat16* out0;
  __nv_bfloat16* out1;
  int ld_out;
  int out_is_cache;      // output rows addressed by cache row (1), by flat token index (0), or by the row's place
                         // in the gathered list (2)
  const __nv_bfloat16* resid;  // EPI_OUT: rows added to the result (indexed like a token-addressed output), or nullptr
  int ld_resid;
  float* out_f32;        // EPI_F32: fp32 output instead of out0
  int b_pair;            // the W tile is BN/2 rows of W0 followed by BN/2 rows of W1, both at row nt*BN/2 (EPI_SWIGLU:
                         // gate and up projections of the same BN/2 outputs)
  const float2* rope;    // rotary table [max_seq][head_dim/2]
  float* q_prev;         // stored scoring-head query [cache rows][head_dim], fp32
  float* scores;
  int has_prev;
  int* status;
  unsigned long long* debug;   // 8 timestamp slots of this kernel or nullptr
  // A step whose refresh set is large runs its projections and attention in their dense forms (every operand through
  // TMA straight from the step's buffers, no compact copy, two-CTA MMAs) and only keeps the results of the rows that
  // were refreshed; only the device knows the set's size, so both forms of a launch are issued and each looks at the
  // count: a launch runs when gate_lo <= *gate_count < gate_hi and leaves at once otherwise (gate_count == nullptr:
  // always runs).  store_mask (the staleness counters, by cache row): a dense-form K/V projection stores a row only
  // where the counter is 0, i.e. where this step's selection refreshed the token (Eq. 3: every other row keeps its
  // cached K and V).
  const int* gate_count;
  int gate_lo, gate_hi;
  const int* store_mask;
  int nt0;               // first column tile of this launch (a projection issued as two launches over its column tiles)
  int loop_rows;         // gathered launch with ONE row of CTAs in the grid: each takes the refresh set's row tiles in turn
  int wait_at_end;       // 1: the launch reads nothing its predecessor in the stream writes and writes nothing that one
                         // reads, so it runs beside it: its CTAs start as soon as the predecessor's have passed their own
                         // dependency wait (everything further back is then complete), and wait for the predecessor
                         // only before they leave, which keeps completion transitive along the stream
};

struct AttnParams {
  const __nv_bfloat16* q;   // [T, d] rotated queries of the step (flat token rows)
  __nv_bfloat16* oc;        // attention-output cache
  const int* idx;           // refresh set (row-sparse) or nullptr (all rows)
  const int* batch_off;     // [batch+1] slice of idx per sequence (row-sparse only)
  StepGeom g;
  int* status;
  unsigned long long* debug;
  const int* gate_count;    // as in GemmParams: the launch runs when gate_lo <= *gate_count < gate_hi
  int gate_lo, gate_hi;
  const int* store_mask;    // dense form of a row-sparse step: a row's output is stored only where the staleness counter
                            // (by cache row) is 0 (Eq. 4: every other row keeps its cached output); tiles without such
                            // a row are skipped
  int wait_first;           // 1: the queries or the refresh set come from the kernel just before this one in the stream,
                            // so nothing of the step is read ahead of the dependency wait
  int dense_from;           // > 0 (two-tile kernel, row-sparse parameters above, gate_count set): one launch carries both
  const int* dense_mask;    // forms; with *gate_count >= dense_from its CTAs run the dense form with this store mask
};

// does a launch of this geometry take the kernel with two query tiles per CTA?
bool attention_tc_two_tiles(const StepGeom& g, bool row_sparse);

cudaError_t launch_attention_tc(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnParams& p,
                                cudaStream_t st);

// grid = (n_tiles of bn columns, m_tiles of 128 rows, splits of the reduction dimension = cluster size: 1 or 2);
// bn = 256 (least re-reading per flop) or 128 (more CTAs for the weight-streaming K/V projection of a small refresh
// set).
// The W tensor maps must have a box of bn rows.
// Row-major bf16 matrix [rows, cols] as a TMA tensor map with a box of 64 columns x box_rows rows, 128-byte swizzle.
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);

// Two-CTA MMAs (pairs of row tiles share their W tile: a third less operand traffic from the L2 per CTA) pay where
// the main loop is bound by that traffic: launches of at most four row tiles, or of about one wave.  Launches of
// many waves measured slower with them (they are bound by the tensor pipe under the power cap, and the pair adds two
// cluster barriers and ties two SMs' pipelines together).
inline bool pairs_pay(int n_tiles, int m_tiles, int splits) {
  const int ctas = n_tiles * ((m_tiles + 1) / 2 * 2) * splits;
  return m_tiles >= 2 && (ctas <= 160 || m_tiles <= 4);
}

// ... and with exactly two row tiles (a window of up to 256 rows) the narrow pair tiles (256 x 128 per pair, reduction
// split in two) put twice as many CTAs on the launch: d/128 column tiles x 2 x 2 CTAs, if that still is one wave.
inline bool narrow_pairs_pay(int d_out, int m_tiles, int kblocks) {
  return m_tiles == 2 && kblocks >= 4 && (d_out / 128) * 2 * 2 <= 160;
}

cudaError_t launch_gemm_tc(int epi, int bn, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                           const GemmParams& p, int n_tiles, int m_tiles, int splits, cudaStream_t st, int pair = 0);


// Persistent form for launches of many row tiles (dense rows, 256-wide tiles, no reduction split, epilogues Q, K/V,
// OUT): one CTA per SM walks the tiles, finishing pass overlapped with the next tile's main loop.
// pair != 0 (dense launches only): two-CTA MMAs over pairs of row tiles, b0 / b1 with 128-row boxes.
cudaError_t launch_gemm_persist(int epi, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                                const GemmParams& p, int n_tiles, int m_tiles, cudaStream_t st, int pair = 0);
// ... pays from about two waves of tiles on.
inline bool persist_pays(int n_tiles, int m_tiles, int splits) { return splits == 1 && n_tiles * m_tiles >= 296; }

}  // namespace dare
