// Query-aware key-channel scoring and tier assignment (Section 4.2), on the current residual window
// of a layer and on explicit (Q, K) windows.
#include "common.cuh"

namespace mixkvq {

__global__ void __launch_bounds__(128)
select_window_kernel(LayerView lv, uint8_t* __restrict__ tiers, double* __restrict__ salience) {
  const int s = blockIdx.x, d = threadIdx.x;
  const __nv_bfloat16* resk = reinterpret_cast<const __nv_bfloat16*>(lv.resk + (size_t)s * lv.resk_stride);
  float mx = -INFINITY, mn = INFINITY;
  for (int j = 0; j < lv.r; ++j) {
    float x = __bfloat162float(resk[(size_t)j * kD + d]);
    mx = fmaxf(mx, x);
    mn = fminf(mn, x);
  }
  const char* st = lv.state + (size_t)s * lv.state_stride;
  double acc = reinterpret_cast<const double*>(st)[d];
  uint32_t cnt = *reinterpret_cast<const uint32_t*>(st + 1024);
  double A;
  uint8_t t = salience_tier(acc, cnt, mx, mn, lv.score_bits, lv.tau_bf16, lv.tau_u4, &A, lv.importance_mode == 2);
  if (lv.budget_bf16 + lv.budget_u4 > 0) {       // fixed budget: rank among the 128 saliences
    __shared__ double aS[kD];
    aS[d] = A;
    __syncthreads();
    t = budget_tier(aS, d, lv.budget_bf16, lv.budget_u4);
  }
  tiers[(size_t)s * kD + d] = t;
  if (salience) salience[(size_t)s * kD + d] = A;
}

__global__ void __launch_bounds__(128)
select_raw_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, int Hq, int Hkv, int lq,
                  int lk, int score_bits, float tau_bf16, float tau_u4, uint8_t* __restrict__ tiers,
                  double* __restrict__ salience) {
  const int s = blockIdx.x, d = threadIdx.x;
  const int b = s / Hkv, hk = s % Hkv, g = Hq / Hkv;
  double acc = 0.0;
  for (int i = 0; i < lq; ++i)
    for (int h = 0; h < g; ++h) {
      size_t qi = (((size_t)b * Hq + hk * g + h) * lq + i) * kD + d;
      acc = __dadd_rn(acc, (double)fabsf(__bfloat162float(q[qi])));
    }
  float mx = -INFINITY, mn = INFINITY;
  for (int j = 0; j < lk; ++j) {
    float x = __bfloat162float(k[((size_t)s * lk + j) * kD + d]);
    mx = fmaxf(mx, x);
    mn = fminf(mn, x);
  }
  double A;
  uint8_t t = salience_tier(acc, (uint32_t)(lq * g), mx, mn, score_bits, tau_bf16, tau_u4, &A);
  tiers[(size_t)s * kD + d] = t;
  if (salience) salience[(size_t)s * kD + d] = A;
}

cudaError_t launch_select_window(const LayerView& lv, uint8_t* tiers, double* salience, cudaStream_t stream) {
  select_window_kernel<<<lv.B * lv.Hkv, 128, 0, stream>>>(lv, tiers, salience);
  return cudaGetLastError();
}

cudaError_t launch_select_raw(const void* q, const void* k, int B, int Hq, int Hkv, int lq, int lk, int score_bits,
                              float tau_bf16, float tau_u4, uint8_t* tiers, double* salience, cudaStream_t stream) {
  select_raw_kernel<<<B * Hkv, 128, 0, stream>>>(static_cast<const __nv_bfloat16*>(q),
                                                 static_cast<const __nv_bfloat16*>(k), Hq, Hkv, lq, lk, score_bits,
                                                 tau_bf16, tau_u4, tiers, salience);
  return cudaGetLastError();
}

}  // namespace mixkvq
