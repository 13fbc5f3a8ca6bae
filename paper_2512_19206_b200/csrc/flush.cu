// The lazy update of Appendix D.1 for one full residual window: channel statistics, salience and tiers
// (Section 4.2), per-channel mixed-precision key quantization and per-token 2-bit value quantization
// (Eq. 2), and bit-packing into the block layout.  One CTA per stream.
#include "common.cuh"

namespace mixkvq {

__global__ void __launch_bounds__(256)
flush_kernel(LayerView lv) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int R = lv.R, G = lv.G, U = lv.U, NG = lv.NG, VG = lv.VG;
  uint16_t* kS = reinterpret_cast<uint16_t*>(smem);      // [R][128] residual keys (bf16 bits)
  uint8_t* cS = smem + (size_t)R * 256;                   // [R][128] codes (keys, later values)
  uint8_t* tierS = cS + (size_t)R * 128;                  // [128]
  uint8_t* chan16S = tierS + 128;                         // [128]
  uint8_t* chan4S = chan16S + 128;                        // [128]
  int* misc = reinterpret_cast<int*>(chan4S + 128);       // n16, n4, extras offset (16-byte units)

  const int s = blockIdx.x, tid = threadIdx.x;
  char* state = lv.state + (size_t)s * lv.state_stride;
  char* blk = lv.base + (size_t)s * lv.base_stride + (size_t)lv.n_blocks * lv.base_bytes;
  const uint4* resk4 = reinterpret_cast<const uint4*>(lv.resk + (size_t)s * lv.resk_stride);
  const uint16_t* resv = reinterpret_cast<const uint16_t*>(lv.resv + (size_t)s * lv.resv_stride);

  for (int i = tid; i < R * 16; i += 256) reinterpret_cast<uint4*>(kS)[i] = resk4[i];
  __syncthreads();

  // ---- statistics, salience, tier and key codes: one thread per channel
  if (tid < kD) {
    const int d = tid;
    float wmx = -INFINITY, wmn = INFINITY;
    for (int j = 0; j < R; ++j) {
      float x = bf16_bits_to_float(kS[j * kD + d]);
      wmx = fmaxf(wmx, x);
      wmn = fminf(wmn, x);
    }
    double acc = reinterpret_cast<const double*>(state)[d];
    uint32_t cnt = *reinterpret_cast<const uint32_t*>(state + 1024);
    uint8_t tier = salience_tier(acc, cnt, wmx, wmn, lv.score_bits, lv.tau_bf16, lv.tau_u4, nullptr);
    tierS[d] = tier;
    const int max_code = (tier == kU4) ? 15 : 3;
    for (int kg = 0; kg < NG; ++kg) {
      uint32_t meta = 0;
      if (tier == kBF16) {
        for (int j = kg * G; j < (kg + 1) * G; ++j) cS[j * kD + d] = 0;
      } else {
        float gmx = -INFINITY, gmn = INFINITY;
        for (int j = kg * G; j < (kg + 1) * G; ++j) {
          float x = bf16_bits_to_float(kS[j * kD + d]);
          gmx = fmaxf(gmx, x);
          gmn = fminf(gmn, x);
        }
        float sc = stored_scale(gmx, gmn, (float)max_code);
        for (int j = kg * G; j < (kg + 1) * G; ++j)
          cS[j * kD + d] = (uint8_t)quant_code(bf16_bits_to_float(kS[j * kD + d]), gmn, sc, max_code);
        meta = float_to_bf16_bits_exact(sc) | (float_to_bf16_bits_exact(gmn) << 16);
      }
      reinterpret_cast<uint32_t*>(blk + kg * 512)[d] = meta;
    }
  }
  __syncthreads();

  // ---- channel lists, extras allocation, table entry
  if (tid == 0) {
    int n16 = 0, n4 = 0;
    for (int d = 0; d < kD; ++d) {
      if (tierS[d] == kBF16) chan16S[n16++] = (uint8_t)d;
      else if (tierS[d] == kU4) chan4S[n4++] = (uint8_t)d;
    }
    uint32_t* used = reinterpret_cast<uint32_t*>(state + 1028);
    uint32_t off16 = *used;
    uint32_t need = lv.tile ? tile_extras_header_bytes(n16, n4) + tile_extras_body_bytes(n16, n4)
                            : extras_header_bytes(n16, n4) + (uint32_t)U * extras_unit_bytes(n16, n4);
    if ((uint64_t)off16 * 16 + need > lv.extras_budget) {
      atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_EXTRAS_FULL);
      n16 = 0;
      n4 = 0;      // nothing is written to the arena; the block is invalid and the status says so
    } else {
      *used = off16 + need / 16;
    }
    uint32_t* entry = reinterpret_cast<uint32_t*>(lv.table + (size_t)s * lv.table_stride + (size_t)lv.n_blocks * 8);
    entry[0] = off16;
    entry[1] = (uint32_t)n16 | ((uint32_t)n4 << 8);
    misc[0] = n16;
    misc[1] = n4;
    misc[2] = (int)off16;
  }
  __syncthreads();
  const int n16 = misc[0], n4 = misc[1];
  const int n16p = (n16 + 1) >> 1, n4p = ((n4 + 1) >> 1) << 1;
  char* ex = lv.extras + (size_t)s * lv.extras_stride + (size_t)misc[2] * 16;
  const uint32_t hdr = extras_header_bytes(n16, n4), exunit = extras_unit_bytes(n16, n4);

  if (lv.tile) {
    // ---- tile layout (R = 128): a token's key codes are 32 contiguous bytes (two 16-byte halves)
    char* kplane = blk + NG * 512;
    for (int i = tid; i < 128 * 8; i += 256) {
      const int j = i >> 3, W = i & 7;
      uint32_t w = 0;
#pragma unroll
      for (int f = 0; f < 8; ++f)
#pragma unroll
        for (int e = 0; e < 2; ++e) w |= (uint32_t)(cS[j * kD + 16 * W + 2 * f + e] & 3) << (16 * e + 2 * f);
      *reinterpret_cast<uint32_t*>(kplane + (W >> 2) * 2048 + j * 16 + (W & 3) * 4) = w;
    }
    const int n4w = (n4 + 15) >> 4;
    const uint32_t thdr = tile_extras_header_bytes(n16, n4);
    for (int i = tid; i < (int)thdr; i += 256) {
      uint8_t b = 0;
      if (i < 2 * n16p) b = (i < n16) ? chan16S[i] : 0xFF;
      else if (i < 2 * n16p + 16 * n4w) b = (i - 2 * n16p < n4) ? chan4S[i - 2 * n16p] : 0xFF;
      ex[i] = (char)b;
    }
    uint32_t* xw = reinterpret_cast<uint32_t*>(ex + thdr);
    for (int i = tid; i < n16p * 128; i += 256) {
      const int p = i >> 7, j = i & 127;
      uint32_t w = kS[j * kD + chan16S[2 * p]];
      if (2 * p + 1 < n16) w |= (uint32_t)kS[j * kD + chan16S[2 * p + 1]] << 16;
      xw[i] = w;
    }
    for (int i = tid; i < n4w * 128; i += 256) {
      const int wq = i >> 7, j = i & 127;
      uint32_t w = 0;
      for (int k = 0; k < 16 && 16 * wq + k < n4; ++k)
        w |= (uint32_t)(cS[j * kD + chan4S[16 * wq + k]] >> 2) << (16 * (k & 1) + 2 * (k >> 1));
      xw[n16p * 128 + i] = w;
    }
  } else {
    // ---- key low plane, fragment order
    for (int i = tid; i < U * 256; i += 256) {
      const int u = i >> 8, wi = i & 255;
      const int mt = wi >> 7, lane = (wi >> 2) & 31, a = wi & 3;
      const int r = lane >> 2, t = lane & 3, ch = a >> 1, rh = a & 1;
      const int j = 32 * u + mt * 16 + rh * 8 + r;
      uint32_t w = 0;
#pragma unroll
      for (int kt = 0; kt < 8; ++kt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int d = kt * 16 + ch * 8 + 2 * t + e;
          w |= (uint32_t)(cS[j * kD + d] & 3) << (16 * e + 2 * kt);
        }
      reinterpret_cast<uint32_t*>(blk + NG * 512 + (size_t)u * lv.unit_bytes)[wi] = w;
    }
    // ---- extras: header, BF16 pairs, UINT4 high plane
    for (int i = tid; i < (int)hdr; i += 256) {
      uint8_t b = 0;
      if (i < 2 * n16p) b = (i < n16) ? chan16S[i] : 0xFF;
      else if (i < 2 * n16p + n4p) b = (i - 2 * n16p < n4) ? chan4S[i - 2 * n16p] : 0xFF;
      ex[i] = (char)b;
    }
    for (int i = tid; i < U * n16p * 32; i += 256) {
      const int u = i / (n16p * 32), rem = i % (n16p * 32), p = rem >> 5, jj = rem & 31;
      const int j = 32 * u + jj;
      uint32_t w = kS[j * kD + chan16S[2 * p]];
      if (2 * p + 1 < n16) w |= (uint32_t)kS[j * kD + chan16S[2 * p + 1]] << 16;
      reinterpret_cast<uint32_t*>(ex + hdr + (size_t)u * exunit)[rem] = w;
    }
    for (int i = tid; i < U * (n4p / 2) * 4; i += 256) {
      const int u = i / (n4p * 2), rem = i % (n4p * 2), p = rem >> 2, wj = rem & 3;
      uint32_t w = 0;
      for (int e = 0; e < 2; ++e) {
        if (2 * p + e >= n4) continue;
        const int d = chan4S[2 * p + e];
        for (int rhi = 0; rhi < 2; ++rhi)
          for (int mt = 0; mt < 2; ++mt)
            for (int rh = 0; rh < 2; ++rh) {
              const int j = 32 * u + mt * 16 + rh * 8 + wj + 4 * rhi;
              w |= (uint32_t)(cS[j * kD + d] >> 2) << (16 * e + 8 * rhi + 2 * (2 * mt + rh));
            }
      }
      reinterpret_cast<uint32_t*>(ex + hdr + (size_t)u * exunit + 128 * n16p)[rem] = w;
    }
  }
  __syncthreads();

  // ---- values: per token, per group of G channels, 2 bits
  for (int i = tid; i < R * VG; i += 256) {
    const int j = i % R, vg = i / R;
    float gmx = -INFINITY, gmn = INFINITY;
    for (int c = vg * G; c < (vg + 1) * G; ++c) {
      float x = bf16_bits_to_float(resv[(size_t)c * R + j]);
      gmx = fmaxf(gmx, x);
      gmn = fminf(gmn, x);
    }
    float sc = stored_scale(gmx, gmn, 3.0f);
    for (int c = vg * G; c < (vg + 1) * G; ++c)
      cS[j * kD + c] = (uint8_t)quant_code(bf16_bits_to_float(resv[(size_t)c * R + j]), gmn, sc, 3);
    const int u = j >> 5, jj = j & 31;
    uint32_t* vmeta = lv.tile ? reinterpret_cast<uint32_t*>(blk + NG * 512 + 8192) + j * VG
                              : reinterpret_cast<uint32_t*>(blk + NG * 512 + (size_t)u * lv.unit_bytes + 2048) + jj * VG;
    vmeta[vg] = float_to_bf16_bits_exact(sc) | (float_to_bf16_bits_exact(gmn) << 16);
  }
  __syncthreads();
  if (lv.tile) {
    // a channel's value codes over the 128 tokens are 32 contiguous bytes (two 16-byte halves)
    char* vplane = blk + NG * 512 + 4096;
    for (int i = tid; i < 128 * 8; i += 256) {
      const int c = i & 127, W = i >> 7;
      uint32_t w = 0;
#pragma unroll
      for (int f = 0; f < 8; ++f)
#pragma unroll
        for (int e = 0; e < 2; ++e) w |= (uint32_t)cS[(16 * W + 2 * f + e) * kD + c] << (16 * e + 2 * f);
      *reinterpret_cast<uint32_t*>(vplane + (W >> 2) * 2048 + c * 16 + (W & 3) * 4) = w;
    }
  } else {
    for (int i = tid; i < U * 256; i += 256) {
      const int u = i >> 8, wi = i & 255;
      const int ct = (wi >> 7) * 4 + (wi & 3), lane = (wi >> 2) & 31;
      const int r = lane >> 2, t = lane & 3;
      uint32_t w = 0;
#pragma unroll
      for (int rh = 0; rh < 2; ++rh)
#pragma unroll
        for (int ks = 0; ks < 2; ++ks)
#pragma unroll
          for (int ch = 0; ch < 2; ++ch)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int c = ct * 16 + rh * 8 + r;
              const int j = 32 * u + ks * 16 + ch * 8 + 2 * t + e;
              w |= (uint32_t)cS[j * kD + c] << (16 * e + 2 * (4 * rh + 2 * ks + ch));
            }
      reinterpret_cast<uint32_t*>(blk + NG * 512 + (size_t)u * lv.unit_bytes + 1024)[wi] = w;
    }
  }

  // ---- window importance: the accumulator restarts with the next window (Section 4.2)
  if (lv.importance_mode == 0) {
    if (tid < kD) reinterpret_cast<double*>(state)[tid] = 0.0;
    if (tid == 0) *reinterpret_cast<uint32_t*>(state + 1024) = 0u;
  }
}

static size_t flush_smem_bytes(int R) { return (size_t)R * 384 + 3 * 128 + 16; }

cudaError_t launch_flush(const LayerView& lv, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(flush_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)flush_smem_bytes(256));
  if (e != cudaSuccess) return e;
  flush_kernel<<<lv.B * lv.Hkv, 256, flush_smem_bytes(lv.R), stream>>>(lv);
  return cudaGetLastError();
}

}  // namespace mixkvq
