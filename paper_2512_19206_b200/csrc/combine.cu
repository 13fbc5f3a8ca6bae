// Log-sum-exp merge of the split partials of decode attention.
#include "common.cuh"

namespace mixkvq {

// Partials live at ws[slot * kPartialFloats + h * 130 + {0: m (log2 domain), 1: l, 2..129: o}].
// mode 0: stream s owns slots [s*n, s*n + n).  mode 1: the attention grid of `n` CTAs split the
// S*units_per_stream work units evenly; CTA c wrote its part of stream s to slot c + s.
__global__ void __launch_bounds__(128)
combine_kernel(const float* __restrict__ ws, float* __restrict__ out, int g, int Hkv, int Hq, int mode, int n,
               long long units_per_stream, int S, const int4* __restrict__ seq, const int* __restrict__ seq_prefix,
               float* __restrict__ lse_out) {
  const int s = blockIdx.x / g, h = blockIdx.x % g, c = threadIdx.x;
  int first, count;
  // started early (programmatic dependent launch): wait here for the kernel that wrote the partials
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (mode == 0) {
    first = s * n;
    count = n;
  } else if (seq != nullptr) {
    // ragged batch: sequence b's streams own positions [prefix[b] + hk * w, + w), w = seq[b].w (none when w == 0)
    const int bq = s / Hkv, w = seq[bq].w;
    const long long total = seq_prefix[S / Hkv];
    const long long x0 = (long long)seq_prefix[bq] + (long long)(s % Hkv) * w, x1 = x0 + w - 1;
    const int c0 = w ? (int)(((x0 + 1) * n - 1) / total) : 0, c1 = w ? (int)(((x1 + 1) * n - 1) / total) : -1;
    first = c0 + s;
    count = c1 - c0 + 1;
  } else {
    const long long total = units_per_stream * S;
    const long long x0 = units_per_stream * s, x1 = units_per_stream * (s + 1) - 1;
    const int c0 = (int)(((x0 + 1) * n - 1) / total), c1 = (int)(((x1 + 1) * n - 1) / total);
    first = c0 + s;
    count = c1 - c0 + 1;
  }
  const int b = s / Hkv, hk = s % Hkv;
  const float* base = ws + (size_t)first * kPartialFloats + h * 130;
  // one pass with a running maximum; the loads of a chunk of partials are independent of one another, so a stream with
  // up to kChunk partials costs one round trip to memory
  constexpr int kChunk = 12;
  float M = -INFINITY, l = 0.f, o = 0.f;
  for (int i0 = 0; i0 < count; i0 += kChunk) {
    float m[kChunk], ll[kChunk], oo[kChunk];
#pragma unroll
    for (int j = 0; j < kChunk; ++j) {
      const bool in = i0 + j < count;
      const float* p = base + (size_t)(in ? i0 + j : i0) * kPartialFloats;
      m[j] = in ? p[0] : -INFINITY;
      ll[j] = p[1];
      oo[j] = p[2 + c];
    }
    float Mn = M;
#pragma unroll
    for (int j = 0; j < kChunk; ++j) Mn = fmaxf(Mn, m[j]);
    const float f0 = (M == -INFINITY) ? 0.f : exp2f(M - Mn);
    l *= f0;
    o *= f0;
#pragma unroll
    for (int j = 0; j < kChunk; ++j) {
      const float f = (m[j] == -INFINITY) ? 0.f : exp2f(m[j] - Mn);
      l += f * ll[j];
      o += f * oo[j];
    }
    M = Mn;
  }
  // l == 0 only when every split gave up (its partial is then m = -inf, l = 0, o = 0 and the status word says so) or
  // when the sequence of a ragged batch holds no token
  out[((size_t)b * Hq + hk * g + h) * kD + c] = l > 0.f ? o / l : 0.f;
  // natural logarithm of the softmax denominator (the maximum M is kept in the base-2 domain)
  if (lse_out != nullptr && c == 0) lse_out[(size_t)b * Hq + hk * g + h] = l > 0.f ? (M + log2f(l)) * 0.6931471805599453f : -INFINITY;
}

cudaError_t launch_combine(const float* ws, float* out, int g, int Hkv, int Hq, int mode, int n,
                           long long units_per_stream, int S, cudaStream_t stream, const int4* seq, const int* seq_prefix,
                           float* lse_out) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(S * g));
  cfg.blockDim = dim3(128);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, combine_kernel, ws, out, g, Hkv, Hq, mode, n, units_per_stream, S, seq, seq_prefix, lse_out);
}

// The table of a ragged batch, from the host's per-sequence fill (kernel arguments: no copy, ordered in the stream).
__global__ void seq_table_kernel(SeqTableArgs a, int4* __restrict__ seq, int* __restrict__ seq_prefix) {
  // a link of the chain of dependent launches: started early, waits for everything before it (a kernel that still
  // reads the table's previous contents included), and only then lets the attention kernel behind it start
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int b = threadIdx.x;
  if (b < a.n) seq[b] = make_int4(a.fill[3 * b], a.fill[3 * b + 1], a.fill[3 * b + 2], a.w[b]);
  if (b == 0) {
    int acc = 0;
    for (int i = 0; i < a.n; ++i) {
      seq_prefix[i] = acc;
      acc += a.Hkv * a.w[i];
    }
    seq_prefix[a.n] = acc;
  }
}

cudaError_t launch_seq_table(const SeqTableArgs& a, int4* seq, int* seq_prefix, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1);
  cfg.blockDim = dim3(kMaxRaggedBatch);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, seq_table_kernel, a, seq, seq_prefix);
}

// Softmax attention over the union of disjoint token sets from the per-set results: o = sum_r w_r o_r / sum_r w_r with
// w_r = exp(lse_r - max_r lse_r).  o_parts [n_parts][rows][128], lse_parts [n_parts][rows]; a part with lse = -inf
// (no tokens) has weight 0; all parts empty: zeros.
__global__ void __launch_bounds__(128)
merge_partials_kernel(const float* __restrict__ o_parts, const float* __restrict__ lse_parts, int n_parts, int rows,
                      float* __restrict__ out) {
  const int row = blockIdx.x, c = threadIdx.x;
  float top = -INFINITY;
  for (int r = 0; r < n_parts; ++r) top = fmaxf(top, lse_parts[(size_t)r * rows + row]);
  float den = 0.f, num = 0.f;
  if (top != -INFINITY) {
    for (int r = 0; r < n_parts; ++r) {
      const float w = expf(lse_parts[(size_t)r * rows + row] - top);
      den += w;
      num += w * o_parts[((size_t)r * rows + row) * kD + c];
    }
  }
  out[(size_t)row * kD + c] = den > 0.f ? num / den : 0.f;
}

// The partial of a cache that holds no token: zeros and lse = -inf.
__global__ void __launch_bounds__(128) empty_partial_kernel(float* __restrict__ out, float* __restrict__ lse) {
  out[(size_t)blockIdx.x * kD + threadIdx.x] = 0.f;
  if (threadIdx.x == 0) lse[blockIdx.x] = -INFINITY;
}

cudaError_t launch_empty_partial(float* out, float* lse, int rows, cudaStream_t stream) {
  empty_partial_kernel<<<rows, 128, 0, stream>>>(out, lse);
  return cudaGetLastError();
}

cudaError_t launch_merge_partials(const float* o_parts, const float* lse_parts, int n_parts, int rows, float* out,
                                  cudaStream_t stream) {
  merge_partials_kernel<<<rows, 128, 0, stream>>>(o_parts, lse_parts, n_parts, rows, out);
  return cudaGetLastError();
}

// Two sets of partials per stream (packed blocks, residual window), each written by a grid that split its
// S * units work items evenly over n CTAs or groups: member c of set k wrote its part of stream s to slot
// base_k + c + s.
__device__ inline void slot_range(int s, int S, int n, long long units, int* first, int* count) {
  const long long total = units * S;
  const long long x0 = units * s, x1 = units * (s + 1) - 1;
  const int c0 = (int)(((x0 + 1) * n - 1) / total), c1 = (int)(((x1 + 1) * n - 1) / total);
  *first = c0 + s;
  *count = c1 - c0 + 1;
}

__global__ void __launch_bounds__(128)
combine2_kernel(const float* __restrict__ ws, float* __restrict__ out, int g, int Hkv, int Hq, int S, int n1,
                long long units1, int slot2, int n2, long long units2) {
  const int s = blockIdx.x / g, h = blockIdx.x % g, c = threadIdx.x;
  int f1, c1, f2, c2;
  slot_range(s, S, n1, units1, &f1, &c1);
  slot_range(s, S, n2, units2, &f2, &c2);
  f2 += slot2;
  const int b = s / Hkv, hk = s % Hkv;
  float M = -INFINITY;
  for (int i = 0; i < c1 + c2; ++i) {
    const int slot = i < c1 ? f1 + i : f2 + (i - c1);
    M = fmaxf(M, ws[(size_t)slot * kPartialFloats + h * 130]);
  }
  float l = 0.f, o = 0.f;
#pragma unroll 4
  for (int i = 0; i < c1 + c2; ++i) {
    const int slot = i < c1 ? f1 + i : f2 + (i - c1);
    const float* p = ws + (size_t)slot * kPartialFloats + h * 130;
    const float m = p[0];
    const float f = (m == -INFINITY) ? 0.f : exp2f(m - M);
    l += f * p[1];
    o += f * p[2 + c];
  }
  out[((size_t)b * Hq + hk * g + h) * kD + c] = l > 0.f ? o / l : 0.f;
}

cudaError_t launch_combine2(const float* ws, float* out, int g, int Hkv, int Hq, int S, int n1, long long units1,
                            int slot2, int n2, long long units2, cudaStream_t stream) {
  combine2_kernel<<<S * g, 128, 0, stream>>>(ws, out, g, Hkv, Hq, S, n1, units1, slot2, n2, units2);
  return cudaGetLastError();
}

}  // namespace mixkvq
