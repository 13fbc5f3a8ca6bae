// Residual append and query-magnitude accumulation (Appendix D.1 first step, Appendix D.2).
#include "common.cuh"

namespace mixkvq {

// One CTA per stream.  Stores m tokens (input tokens t0..t0+m-1) into residual slots r0..r0+m-1 with 16-byte copies
// and adds |q| of the g heads of the group to the fp64 accumulator in token-major, head-ascending order (the defined
// order of the sum): the queries of kChunk tokens at a time are staged in shared memory by all threads, then thread d
// adds channel d's magnitudes one after the other.
constexpr int kChunk = 16;     // tokens staged per round: kChunk * 8 heads * 256 bytes = 32 KB

__global__ void __launch_bounds__(256)
append_tokens_kernel(LayerView lv, const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                     const __nv_bfloat16* __restrict__ q, int n_tokens, int t0, int m, int r0) {
  __shared__ __align__(16) uint16_t qS[kChunk * 8 * kD];      // [token][head][128] bf16 bits
  const int s = blockIdx.x, tid = threadIdx.x;
  const int b = s / lv.Hkv, hk = s % lv.Hkv, g = lv.g;
  // ---- key and value rows: contiguous in the tensors (per stream) and in the residual store
  {
    const uint4* ksrc = reinterpret_cast<const uint4*>(k + ((size_t)s * n_tokens + t0) * kD);
    const uint4* vsrc = reinterpret_cast<const uint4*>(v + ((size_t)s * n_tokens + t0) * kD);
    uint4* kdst = reinterpret_cast<uint4*>(lv.resk + (size_t)s * lv.resk_stride) + (size_t)r0 * 16;
    uint4* vdst = reinterpret_cast<uint4*>(lv.resv + (size_t)s * lv.resv_stride) + (size_t)r0 * 16;
    for (int i = tid; i < m * 16; i += 256) {
      kdst[i] = ksrc[i];
      vdst[i] = vsrc[i];
    }
  }
  // ---- importance accumulator
  double* acc = reinterpret_cast<double*>(lv.state + (size_t)s * lv.state_stride);
  double a = tid < kD ? acc[tid] : 0.0;
  const uint16_t* qw = reinterpret_cast<const uint16_t*>(q) + (((size_t)b * lv.Hq + hk * g) * n_tokens + t0) * kD;
  const size_t head_stride = (size_t)n_tokens * kD;
  for (int i0 = 0; i0 < m; i0 += kChunk) {
    const int tc = min(kChunk, m - i0);
    for (int i = tid; i < tc * g * 16; i += 256) {
      const int row = i >> 4, c16 = i & 15, jj = row / g, h = row - jj * g;
      reinterpret_cast<uint4*>(qS)[i] =
          *reinterpret_cast<const uint4*>(qw + (size_t)(i0 + jj) * kD + h * head_stride + 8 * c16);
    }
    __syncthreads();
    if (tid < kD)
      for (int row = 0; row < tc * g; ++row)
        a = __dadd_rn(a, (double)fabsf(bf16_bits_to_float(qS[row * kD + tid])));
    __syncthreads();
  }
  if (tid < kD) acc[tid] = a;
  if (tid == 0) {
    uint32_t* cnt = reinterpret_cast<uint32_t*>(lv.state + (size_t)s * lv.state_stride + 1024);
    *cnt += (uint32_t)(m * g);
  }
}

// Sink tokens: m rows of keys and of values go to sink slots n_sink .. n_sink + m - 1 of every stream, nothing else happens.
__global__ void __launch_bounds__(256)
sink_append_kernel(LayerView lv, const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, int n_tokens,
                   int t0, int m) {
  const int s = blockIdx.x, tid = threadIdx.x;
  const uint4* ksrc = reinterpret_cast<const uint4*>(k + ((size_t)s * n_tokens + t0) * kD);
  const uint4* vsrc = reinterpret_cast<const uint4*>(v + ((size_t)s * n_tokens + t0) * kD);
  uint4* kdst = reinterpret_cast<uint4*>(lv.sink + (size_t)s * lv.sink_stride) + (size_t)lv.n_sink * 16;
  uint4* vdst = kdst + (size_t)lv.sink_len * 16;
  for (int i = tid; i < m * 16; i += 256) {
    kdst[i] = ksrc[i];
    vdst[i] = vsrc[i];
  }
}

cudaError_t launch_sink_append(const LayerView& lv, const void* k, const void* v, int n_tokens, int t0, int m,
                               cudaStream_t stream) {
  sink_append_kernel<<<lv.B * lv.Hkv, 256, 0, stream>>>(lv, static_cast<const __nv_bfloat16*>(k),
                                                        static_cast<const __nv_bfloat16*>(v), n_tokens, t0, m);
  return cudaGetLastError();
}

cudaError_t launch_append(const LayerView& lv, const void* k, const void* v, const void* q, int n_tokens, int t0,
                          int m, cudaStream_t stream) {
  append_tokens_kernel<<<lv.B * lv.Hkv, 256, 0, stream>>>(
      lv, static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v),
      static_cast<const __nv_bfloat16*>(q), n_tokens, t0, m, lv.r);
  return cudaGetLastError();
}

}  // namespace mixkvq
