// Residual append and query-magnitude accumulation (Appendix D.1 first step, Appendix D.2).
#include "common.cuh"

namespace mixkvq {

// One CTA per stream, one thread per channel.  Stores m tokens (input tokens t0..t0+m-1) into residual
// slots r0..r0+m-1 and adds |q| of the g heads of the group to the fp64 accumulator in token-major,
// head-ascending order (the defined order of the sum).
__global__ void __launch_bounds__(128)
append_tokens_kernel(LayerView lv, const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                     const __nv_bfloat16* __restrict__ q, int n_tokens, int t0, int m, int r0) {
  const int s = blockIdx.x, d = threadIdx.x;
  const int b = s / lv.Hkv, hk = s % lv.Hkv;
  const size_t kv_base = ((size_t)s * n_tokens + t0) * kD + d;
  __nv_bfloat16* resk = reinterpret_cast<__nv_bfloat16*>(lv.resk + (size_t)s * lv.resk_stride);
  __nv_bfloat16* resv = reinterpret_cast<__nv_bfloat16*>(lv.resv + (size_t)s * lv.resv_stride);
  double* acc = reinterpret_cast<double*>(lv.state + (size_t)s * lv.state_stride);
  double a = acc[d];
  const __nv_bfloat16* qw = q + (((size_t)b * lv.Hq + hk * lv.g) * n_tokens + t0) * kD + d;
  const size_t head_stride = (size_t)n_tokens * kD;
  for (int i0 = 0; i0 < m; i0 += 4) {
    // the loads of up to four tokens go out together; the fp64 additions keep the defined order
    float mag[4][8];
    __nv_bfloat16 kk[4], vv[4];
#pragma unroll
    for (int ii = 0; ii < 4; ++ii) {
      const bool on = i0 + ii < m;
      kk[ii] = on ? k[kv_base + (size_t)(i0 + ii) * kD] : __float2bfloat16(0.f);
      vv[ii] = on ? v[kv_base + (size_t)(i0 + ii) * kD] : __float2bfloat16(0.f);
#pragma unroll
      for (int h = 0; h < 8; ++h)
        mag[ii][h] = (on && h < lv.g) ? fabsf(__bfloat162float(qw[(size_t)(i0 + ii) * kD + h * head_stride])) : 0.f;
    }
#pragma unroll
    for (int ii = 0; ii < 4; ++ii) {
      if (i0 + ii < m) {
        resk[(size_t)(r0 + i0 + ii) * kD + d] = kk[ii];
        resv[(size_t)(r0 + i0 + ii) * kD + d] = vv[ii];
#pragma unroll
        for (int h = 0; h < 8; ++h)
          if (h < lv.g) a = __dadd_rn(a, (double)mag[ii][h]);
      }
    }
  }
  acc[d] = a;
  if (d == 0) {
    uint32_t* cnt = reinterpret_cast<uint32_t*>(lv.state + (size_t)s * lv.state_stride + 1024);
    *cnt += (uint32_t)(m * lv.g);
  }
}

cudaError_t launch_append(const LayerView& lv, const void* k, const void* v, const void* q, int n_tokens, int t0,
                          int m, cudaStream_t stream) {
  append_tokens_kernel<<<lv.B * lv.Hkv, 128, 0, stream>>>(
      lv, static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v),
      static_cast<const __nv_bfloat16*>(q), n_tokens, t0, m, lv.r);
  return cudaGetLastError();
}

}  // namespace mixkvq
