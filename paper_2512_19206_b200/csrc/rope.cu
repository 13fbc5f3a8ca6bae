// Rotary position embedding of the keys and queries of an append, in place (Appendix D: importance scores and keys
// are taken after the rotation, so every caller rotates right before it appends).
//
// Channel pairing (i, i + 64) ("rotate-half").  With c = cos[p][i], s = sin[p][i] from the caller's tables:
//   y[i] = x[i] c - x[i + 64] s,   y[i + 64] = x[i + 64] c + x[i] s
// Every product and the sum are single fp32 operations rounded to nearest (no fused multiply-add), and the result is
// rounded to bf16 (nearest, ties to even): the rotated bits are a defined function of the inputs and the tables.
#include "common.cuh"

namespace mixkvq {

namespace {

// rows: the B * Hkv * n key rows, then the B * Hq * n query rows; token index of a row = row % n.
// One thread rotates eight pairs of one row: channels 8c .. 8c+7 and 64 + 8c .. 64 + 8c+7.
__global__ void __launch_bounds__(256)
rope_kernel(__nv_bfloat16* __restrict__ k, __nv_bfloat16* __restrict__ q, const float* __restrict__ cos_t,
            const float* __restrict__ sin_t, long long k_rows, long long rows, int n_tokens, int pos0) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long row = idx >> 3;
  const int c = (int)(idx & 7);
  if (row >= rows) return;
  __nv_bfloat16* x = (row < k_rows ? k + row * kD : q + (row - k_rows) * kD) + 8 * c;
  const int pos = pos0 + (int)(row % n_tokens);
  const float4* cp = reinterpret_cast<const float4*>(cos_t + (size_t)pos * 64 + 8 * c);
  const float4* sp = reinterpret_cast<const float4*>(sin_t + (size_t)pos * 64 + 8 * c);
  const float4 c0 = cp[0], c1 = cp[1], s0 = sp[0], s1 = sp[1];
  const float cs[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
  const float sn[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
  const uint4 lo = *reinterpret_cast<const uint4*>(x), hi = *reinterpret_cast<const uint4*>(x + 64);
  const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w}, hw[4] = {hi.x, hi.y, hi.z, hi.w};
  uint32_t ol[4], oh[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float y1[2], y2[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const float x1 = bf16_bits_to_float(e ? lw[j] >> 16 : lw[j] & 0xFFFFu);
      const float x2 = bf16_bits_to_float(e ? hw[j] >> 16 : hw[j] & 0xFFFFu);
      const float cc = cs[2 * j + e], ss = sn[2 * j + e];
      y1[e] = __fsub_rn(__fmul_rn(x1, cc), __fmul_rn(x2, ss));
      y2[e] = __fadd_rn(__fmul_rn(x2, cc), __fmul_rn(x1, ss));
    }
    const __nv_bfloat162 a = __floats2bfloat162_rn(y1[0], y1[1]), b = __floats2bfloat162_rn(y2[0], y2[1]);
    ol[j] = *reinterpret_cast<const uint32_t*>(&a);
    oh[j] = *reinterpret_cast<const uint32_t*>(&b);
  }
  *reinterpret_cast<uint4*>(x) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
  *reinterpret_cast<uint4*>(x + 64) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
}

}  // namespace

cudaError_t launch_rope(void* k, void* q, const float* cos_t, const float* sin_t, int B, int Hkv, int Hq, int n_tokens,
                        int pos0, cudaStream_t stream) {
  const long long k_rows = (long long)B * Hkv * n_tokens, rows = k_rows + (long long)B * Hq * n_tokens;
  const long long threads = rows * 8;
  rope_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(static_cast<__nv_bfloat16*>(k),
                                                                   static_cast<__nv_bfloat16*>(q), cos_t, sin_t, k_rows,
                                                                   rows, n_tokens, pos0);
  return cudaGetLastError();
}

}  // namespace mixkvq
