// Internal definitions shared by the kernels: per-layer views of the caller-owned cache memory,
// the byte layout constants, and the small numeric helpers whose results must be bit-exact.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mixkvq.h"

namespace mixkvq {

constexpr int kD = 128;                 // head dimension
constexpr int kStateBytes = 1152;       // acc fp64[128] | cnt u32 | extras_used16 u32 | zeros
constexpr int kPartialFloats = 8 * 130; // per (CTA, stream) split partial: 8 heads x {m, l, o[128]}
constexpr int kMaxCtas = 148 * 8;       // upper bound on the attention grid (sizes the workspace)

enum Tier : uint8_t { kU2 = 0, kU4 = 1, kBF16 = 2 };

// Geometry + pointers of one layer, passed by value to every kernel.
constexpr int kMaxRaggedBatch = 128;   // sequences of a batch whose fills may differ

struct LayerView {
  // geometry
  int B, Hq, Hkv, g;          // batch, query heads, KV heads, GQA group size
  int R, G, U, NG, VG;        // residual length, group size, units/block, key groups/block, value groups/token
  int max_blocks;
  int n_blocks, r;            // current fill (same for all streams)
  int tile;                   // 1: tile layout (R == 128 only), 0: fragment layout
  int dense_hi;               // 1: 4-bit base (tau_u4 < 0): dense UINT4 high plane in the fragment layout
  uint32_t base_bytes, unit_bytes;
  uint64_t extras_budget;     // bytes per stream
  // method parameters
  int score_bits, importance_mode;
  float tau_bf16, tau_u4;
  int v_bits;                 // 2, or 4: a second plane of 2-bit value codes follows the value scales in every unit
  int budget_bf16, budget_u4; // fixed-budget tiering when their sum is positive (the thresholds are then unused)
  // per-stream arrays (base pointer + stride in bytes)
  char* state;  uint64_t state_stride;
  char* table;  uint64_t table_stride;
  char* resk;   uint64_t resk_stride;
  char* resv;   uint64_t resv_stride;
  char* base;   uint64_t base_stride;
  char* extras; uint64_t extras_stride;
  char* sink;   uint64_t sink_stride;   // per stream: keys [sink_len][128] bf16, then values
  int sink_len, n_sink;       // capacity and current fill of the sink (same for all streams)
  uint32_t* status;           // sticky device status word
  // fused decode step: the new token's key and value rows [S][128] (bf16 bits); null for plain attention.
  // The attention kernel then stores them at residual slot r - 1 and adds |q| to the importance accumulator itself.
  const uint16_t* new_k;
  const uint16_t* new_v;
  // decode attention may stage its first packed units before it waits for the kernel launched before it: set by the
  // host when that kernel did not write this layer's packed blocks
  int stage_early;
  // waits on staged copies and on hand-overs between warps give up after this many polls (0: the kernel's default)
  uint32_t wait_polls;
  // test hook for the give-up path: the barrier of every warp pair's first staged copy is armed for this many bytes
  // more than are copied, so that it never completes (0 in normal use)
  uint32_t debug_extra_tx;
  // Ragged batch (sequences of different fill): per sequence (n_blocks, r, n_sink, split positions of one of its
  // streams) and the prefix sums over the sequences of Hkv * positions ([B + 1], the last one = seq_total), both in
  // device memory; null when every sequence has the fill n_blocks, r, n_sink above.
  const int4* seq;
  const int* seq_prefix;
  long long seq_total;
};

__host__ __device__ inline uint32_t extras_header_bytes(int n16, int n4) {
  int n16p = (n16 + 1) >> 1, n4p = ((n4 + 1) >> 1) << 1;
  return 16u * ((2 * n16p + n4p + 15) >> 4);
}
// With a 4-bit base precision (tau_u4 < 0: every channel that is not promoted is UINT4) the high plane of a block is
// stored densely: 1024 bytes per unit in the bit order of the low plane (zero where the channel is BF16) instead of
// 16 bytes per channel pair, so that the attention kernel runs it through the low plane's code path without gathering
// scales and query entries.  `dense` is a property of the cache's configuration, the same for all its blocks.
__host__ __device__ inline uint32_t extras_unit_bytes(int n16, int n4, bool dense) {
  int n16p = (n16 + 1) >> 1, n4p = ((n4 + 1) >> 1) << 1;
  return 128u * n16p + (dense ? 1024u : 8u * n4p);
}

// fragment layout: the key-meta group of G tokens sits directly before the first 32-token unit of those tokens, so a
// unit and its group's scales are one contiguous piece
__host__ __device__ inline uint32_t frag_meta_off(int kg, int G, uint32_t unit_bytes) {
  return (uint32_t)(kg * (G / 32)) * unit_bytes + 512u * (uint32_t)kg;
}
__host__ __device__ inline uint32_t frag_unit_off(int u, int G, uint32_t unit_bytes) {
  return (uint32_t)u * unit_bytes + 512u * (uint32_t)((u * 32) / G + 1);
}

// tile layout (R == 128): header [chan16: 2*n16p][chan4: 16*n4w][pad to 16], body (n16p + n4w) x 128 words
__host__ __device__ inline uint32_t tile_extras_header_bytes(int n16, int n4) {
  int n16p = (n16 + 1) >> 1, n4w = (n4 + 15) >> 4;
  return 16u * ((2 * n16p + 16 * n4w + 15) >> 4);
}
__host__ __device__ inline uint32_t tile_extras_body_bytes(int n16, int n4) {
  int n16p = (n16 + 1) >> 1, n4w = (n4 + 15) >> 4;
  return 512u * (n16p + n4w);
}

// ---- bf16 bit helpers (no rounding involved)
__device__ inline float bf16_bits_to_float(uint32_t u16) { return __uint_as_float(u16 << 16); }
__device__ inline uint32_t float_to_bf16_bits_exact(float f) { return __float_as_uint(f) >> 16; }

// Scale of Eq. 2 as stored: fp32 (max - min) / levels, rounded up to bf16 (returned as float).
__device__ inline float stored_scale(float mx, float mn, float levels) {
  float q = __fdiv_rn(__fsub_rn(mx, mn), levels);
  uint32_t b = __float_as_uint(q);
  if (b & 0xFFFFu) b = (b + 0x10000u) & 0xFFFF0000u;
  return __uint_as_float(b);
}

// Code of Eq. 2: round-half-even of the IEEE fp32 quotient (x - z) / s, clamped; 0 when s == 0.
__device__ inline int quant_code(float x, float z, float s, int max_code) {
  if (s == 0.0f) return 0;
  float y = __fdiv_rn(__fsub_rn(x, z), s);
  int c = __float2int_rn(y);
  return min(max(c, 0), max_code);
}

// The same code by a shortcut, bit-identical to quant_code for every input: with r = RN(1 / s) the product (x - z) * r is
// within 2e-6 of the IEEE quotient (codes are at most 15), so it rounds to the same integer unless it lies within 1e-4
// of a half-integer; only then is the IEEE division carried out.  r is computed once per group.
__device__ inline int quant_code_fast(float x, float z, float s, float r, int max_code) {
  if (s == 0.0f) return 0;
  const float y = __fmul_rn(__fsub_rn(x, z), r);
  const float frac = y - floorf(y);
  if (fabsf(frac - 0.5f) < 1e-4f) return quant_code(x, z, s, max_code);
  int c = __float2int_rn(y);
  return min(max(c, 0), max_code);
}

// Section 4.2: A_d = (acc / cnt) * (range / (2^B - 1)) in fp64; tier by the two thresholds.
// error_only (the ablation without the query term): I_d = 1, so A_d = S_d.
__device__ inline uint8_t salience_tier(double acc, uint32_t cnt, float mx, float mn, int score_bits,
                                        float tau_bf16, float tau_u4, double* a_out, bool error_only = false) {
  double range = (double)mx - (double)mn;
  double S = __ddiv_rn(range, (double)((1 << score_bits) - 1));
  double I = error_only ? 1.0 : __ddiv_rn(acc, (double)cnt);
  double A = __dmul_rn(I, S);
  if (a_out) *a_out = A;
  if (A > (double)tau_bf16) return kBF16;
  if (A > (double)tau_u4) return kU4;
  return kU2;
}

// Fixed-budget form of the tier rule: channel d's rank among the 128 saliences (descending, equal values by channel
// index) against the two quotas.
__device__ inline uint8_t budget_tier(const double* A, int d, int budget_bf16, int budget_u4) {
  const double a = A[d];
  int rank = 0;
  for (int e = 0; e < kD; ++e) {
    const double b = A[e];
    rank += (b > a || (b == a && e < d)) ? 1 : 0;
  }
  return rank < budget_bf16 ? kBF16 : (rank < budget_bf16 + budget_u4 ? kU4 : kU2);
}

// ---- fragment layout: positions inside a 32-token unit.  The codes are ordered so that one 16-byte load per lane
// yields the four A-operand registers of an m16n8k16 tile for all eight 16-channel k-tiles.
// K low-plane code of (token jj in unit, channel d): 32-bit word index inside the unit's K codes, bit offset.
__host__ __device__ inline void k_code_pos(int jj, int d, int* word, int* bit) {
  int mt = jj >> 4, row = jj & 15, r = row & 7, rh = row >> 3;
  int kt = d >> 4, col = d & 15, ch = col >> 3, t = (col & 7) >> 1, e = col & 1;
  *word = mt * 128 + (4 * r + t) * 4 + (2 * ch + rh);
  *bit = 16 * e + 2 * kt;
}
// V code of (token jj in unit, channel c).
__host__ __device__ inline void v_code_pos(int jj, int c, int* word, int* bit) {
  int ct = c >> 4, row = c & 15, r = row & 7, rh = row >> 3;
  int ks = jj >> 4, col = jj & 15, ch = col >> 3, t = (col & 7) >> 1, e = col & 1;
  *word = (ct >> 2) * 128 + (4 * r + t) * 4 + (ct & 3);
  *bit = 16 * e + 2 * (4 * rh + 2 * ks + ch);
}
// UINT4 high-plane code of (token jj, half e) inside a channel pair's four words.
__host__ __device__ inline void hi_plane_pos(int jj, int e, int* word, int* bit) {
  int mt = jj >> 4, row = jj & 15, r = row & 7, rh = row >> 3;
  *word = r & 3;
  *bit = 16 * e + 8 * (r >> 2) + 2 * (2 * mt + rh);
}

// Even split of `total` work units over `parts`: [begin(i), begin(i+1)).
__host__ __device__ inline long long split_begin(long long total, int parts, int i) {
  return (total * (long long)i) / parts;
}

}  // namespace mixkvq

// launchers implemented in the .cu files (host side, all asynchronous on `stream`)
namespace mixkvq {
cudaError_t launch_append(const LayerView& lv, const void* k, const void* v, const void* q, int n_tokens, int t0,
                          int m, cudaStream_t stream);
cudaError_t launch_sink_append(const LayerView& lv, const void* k, const void* v, int n_tokens, int t0, int m,
                               cudaStream_t stream);
// causal full-precision attention over a prompt (tcgen05)
cudaError_t launch_prefill_attention(const void* q, const void* k, const void* v, float* out, void* scratch, int B, int Hq,
                                     int Hkv, int L, float scale, uint32_t* status, uint32_t max_polls, uint32_t debug_extra_tx,
                                     cudaStream_t stream);
size_t prefill_scratch_bytes(int B, int Hkv, int L);
cudaError_t prefill_attention_setup();
int attention_ws_positions_of(int n_blocks, int r, int n_sink, int U);
// writes a ragged batch's table: fill[3 b + {0, 1, 2}] = (n_blocks, r, n_sink) of sequence b, positions w[b] per stream
struct SeqTableArgs { int n, Hkv; int fill[3 * kMaxRaggedBatch]; int w[kMaxRaggedBatch]; };
cudaError_t launch_seq_table(const SeqTableArgs& a, int4* seq, int* seq_prefix, cudaStream_t stream);
cudaError_t launch_empty_partial(float* out, float* lse, int rows, cudaStream_t stream);
cudaError_t launch_merge_partials(const float* o_parts, const float* lse_parts, int n_parts, int rows, float* out,
                                  cudaStream_t stream);
cudaError_t launch_rope(void* k, void* q, const float* cos_t, const float* sin_t, int B, int Hkv, int Hq, int n_tokens,
                        int pos0, cudaStream_t stream);
cudaError_t launch_flush(const LayerView& lv, cudaStream_t stream);
cudaError_t launch_flush_bulk(const LayerView& lv, const void* k, const void* v, const void* q, int n_tokens, int t0,
                              int nb, cudaStream_t stream);
cudaError_t launch_select_window(const LayerView& lv, uint8_t* tiers, double* salience, cudaStream_t stream);
cudaError_t launch_select_raw(const void* q, const void* k, int B, int Hq, int Hkv, int lq, int lk, int score_bits,
                              float tau_bf16, float tau_u4, uint8_t* tiers, double* salience, cudaStream_t stream);
// decode attention: writes split partials to `ws`, then the combine kernel writes `out`; returns launches made
cudaError_t launch_attention_simt(const LayerView& lv, const void* q, float* out, float scale, float* ws,
                                  int n_sms, cudaStream_t stream, int* launches);
cudaError_t launch_attention_ws(const LayerView& lv, const void* q, float* out, float scale, float* ws,
                                int n_sms, cudaStream_t stream, int* launches, float* lse_out = nullptr);
cudaError_t attention_ws_setup();
// tile layout (R == 128): tcgen05 kernel
cudaError_t launch_attention_tc(const LayerView& lv, const void* q, float* out, float scale, float* ws,
                                int n_sms, cudaStream_t stream, int* launches);
cudaError_t attention_tc_setup();
}  // namespace mixkvq
