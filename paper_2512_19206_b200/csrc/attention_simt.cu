// Decode attention over the mixed-precision cache on the plain fp32 ALUs: one lane per token, codes
// decoded element by element from the packed layout.  Kept as the comparison point for the
// tensor-core kernel: it is arithmetic-bound far below the memory roofline.
#include "common.cuh"

namespace mixkvq {

cudaError_t launch_combine(const float* ws, float* out, int g, int Hkv, int Hq, int mode, int n,
                           long long units_per_stream, int S, cudaStream_t stream, const int4* seq = nullptr,
                           const int* seq_prefix = nullptr, float* lse_out = nullptr);

__global__ void __launch_bounds__(128)
attention_simt_kernel(LayerView lv, const __nv_bfloat16* __restrict__ q, float scale_log2e, float* __restrict__ ws,
                      int nsplit) {
  __shared__ float qS[8][kD];
  __shared__ float oS[4][8][kD];
  __shared__ float mS[4][8], lS[4][8];
  __shared__ uint8_t slot16[4][kD], slot4[4][kD];

  const int s = blockIdx.x, split = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = s / lv.Hkv, hk = s % lv.Hkv, g = lv.g;
  for (int i = threadIdx.x; i < 8 * kD; i += 128) {
    const int h = i >> 7, d = i & 127;
    qS[h][d] = (h < g) ? __bfloat162float(q[((size_t)b * lv.Hq + hk * g + h) * kD + d]) : 0.f;
  }
  __syncthreads();

  const int packed_units = lv.n_blocks * lv.U;
  const int res_units = (lv.r + 31) / 32;                            // then the units of the sink
  const int units = packed_units + res_units + (lv.n_sink + 31) / 32;
  const int ub = (int)split_begin(units, nsplit, split), ue = (int)split_begin(units, nsplit, split + 1);
  const int wb = ub + (int)split_begin(ue - ub, 4, warp), we = ub + (int)split_begin(ue - ub, 4, warp + 1);

  const char* base = lv.base + (size_t)s * lv.base_stride;
  const char* extras = lv.extras + (size_t)s * lv.extras_stride;
  const uint32_t* table = reinterpret_cast<const uint32_t*>(lv.table + (size_t)s * lv.table_stride);
  const uint16_t* resk = reinterpret_cast<const uint16_t*>(lv.resk + (size_t)s * lv.resk_stride);
  const uint16_t* resv = reinterpret_cast<const uint16_t*>(lv.resv + (size_t)s * lv.resv_stride);
  const uint16_t* sinkk = reinterpret_cast<const uint16_t*>(lv.sink + (size_t)s * lv.sink_stride);
  const uint16_t* sinkv = sinkk + (size_t)lv.sink_len * kD;

  float m[8], l[8], o[8][4];
  for (int h = 0; h < 8; ++h) {
    m[h] = -INFINITY;
    l[h] = 0.f;
    for (int i = 0; i < 4; ++i) o[h][i] = 0.f;
  }

  int cur_block = -1, n16 = 0, n4 = 0;
  const char* ex = nullptr;
  for (int unit = wb; unit < we; ++unit) {
    float dot[8];
    for (int h = 0; h < 8; ++h) dot[h] = 0.f;
    bool valid = true;
    const char* ub_ptr = nullptr;
    if (unit < packed_units) {
      const int bi = unit / lv.U, u = unit % lv.U;
      if (bi != cur_block) {
        cur_block = bi;
        const uint32_t off16 = table[2 * bi], nn = table[2 * bi + 1];
        n16 = nn & 0xFF;
        n4 = (nn >> 8) & 0xFF;
        ex = extras + (size_t)off16 * 16;
        __syncwarp();
        for (int i = lane; i < kD; i += 32) slot16[warp][i] = slot4[warp][i] = 0xFF;
        __syncwarp();
        for (int i = lane; i < n16; i += 32) slot16[warp][(uint8_t)ex[i]] = (uint8_t)i;
        for (int i = lane; i < n4; i += 32) slot4[warp][(uint8_t)ex[2 * ((n16 + 1) >> 1) + i]] = (uint8_t)i;
        __syncwarp();
      }
      const char* blk = base + (size_t)bi * lv.base_bytes;
      ub_ptr = blk + frag_unit_off(u, lv.G, lv.unit_bytes);
      const uint32_t* kmeta = reinterpret_cast<const uint32_t*>(
          blk + (lv.tile ? (uint32_t)((u * 32) / lv.G) * 512u : frag_meta_off((u * 32) / lv.G, lv.G, lv.unit_bytes)));
      const uint32_t* kcodes = reinterpret_cast<const uint32_t*>(ub_ptr);
      const char* exu = ex + extras_header_bytes(n16, n4) + (size_t)u * extras_unit_bytes(n16, n4, lv.dense_hi != 0);
      const int n16p = (n16 + 1) >> 1;
      // tile layout (R == 128): planes of the whole block, token j of the block
      const int jt = 32 * u + lane;
      const char* kplane = blk + lv.NG * 512;
      const uint32_t* txw = reinterpret_cast<const uint32_t*>(ex + tile_extras_header_bytes(n16, n4));
      for (int d = 0; d < kD; ++d) {
        float kval;
        const uint8_t s16 = slot16[warp][d];
        if (s16 != 0xFF) {
          const uint32_t w = lv.tile ? txw[(s16 >> 1) * 128 + jt]
                                     : reinterpret_cast<const uint32_t*>(exu)[(s16 >> 1) * 32 + lane];
          kval = bf16_bits_to_float((s16 & 1) ? (w >> 16) : (w & 0xFFFF));
        } else {
          int code;
          const uint8_t s4 = slot4[warp][d];
          if (lv.tile) {
            const uint32_t kw = *reinterpret_cast<const uint32_t*>(kplane + (d >> 6) * 2048 + jt * 16 + ((d & 63) >> 4) * 4);
            code = (kw >> (16 * (d & 1) + 2 * ((d & 15) >> 1))) & 3;
            if (s4 != 0xFF) {
              const uint32_t w = txw[(n16p + (s4 >> 4)) * 128 + jt];
              code += 4 * ((w >> (16 * (s4 & 1) + 2 * ((s4 & 15) >> 1))) & 3);
            }
          } else {
            int word, bit;
            k_code_pos(lane, d, &word, &bit);
            code = (kcodes[word] >> bit) & 3;
            if (s4 != 0xFF && lv.dense_hi) {
              code += 4 * ((reinterpret_cast<const uint32_t*>(exu + 128 * n16p)[word] >> bit) & 3);
            } else if (s4 != 0xFF) {
              int hw, hb;
              hi_plane_pos(lane, s4 & 1, &hw, &hb);
              const uint32_t w = reinterpret_cast<const uint32_t*>(exu + 128 * n16p)[(s4 >> 1) * 4 + hw];
              code += 4 * ((w >> hb) & 3);
            }
          }
          const uint32_t mz = kmeta[d];
          kval = fmaf((float)code, bf16_bits_to_float(mz & 0xFFFF), bf16_bits_to_float(mz >> 16));
        }
        for (int h = 0; h < 8; ++h) dot[h] = fmaf(qS[h][d], kval, dot[h]);
      }
    } else {
      const int bu = unit - packed_units;
      const bool in_sink = bu >= res_units;
      const int j = (in_sink ? bu - res_units : bu) * 32 + lane;
      const uint16_t* rows = in_sink ? sinkk : resk;
      valid = j < (in_sink ? lv.n_sink : lv.r);
      if (valid)
        for (int d = 0; d < kD; ++d) {
          const float kval = bf16_bits_to_float(rows[(size_t)j * kD + d]);
          for (int h = 0; h < 8; ++h) dot[h] = fmaf(qS[h][d], kval, dot[h]);
        }
    }
    // online softmax (log2 domain)
    float p[8];
    for (int h = 0; h < 8; ++h) {
      const float x = valid ? dot[h] * scale_log2e : -INFINITY;
      float mx = x;
      for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float mn = fmaxf(m[h], mx);
      const float alpha = (m[h] == -INFINITY) ? 0.f : exp2f(m[h] - mn);
      p[h] = valid ? exp2f(x - mn) : 0.f;
      float ps = p[h];
      for (int off = 16; off; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
      l[h] = l[h] * alpha + ps;
      m[h] = mn;
      for (int i = 0; i < 4; ++i) o[h][i] *= alpha;
    }
    // P.V: lane owns channels 4*lane .. 4*lane+3
    for (int jj = 0; jj < 32; ++jj) {
      float vv[4];
      if (unit < packed_units) {
        const uint32_t* vcodes = reinterpret_cast<const uint32_t*>(ub_ptr + 1024);
        const uint32_t* vmeta = reinterpret_cast<const uint32_t*>(ub_ptr + 2048);
        const int u = unit % lv.U, t = 32 * u + jj;                  // tile layout: token t of the block
        const char* tblk = base + (size_t)(unit / lv.U) * lv.base_bytes + lv.NG * 512;
        for (int i = 0; i < 4; ++i) {
          const int c = 4 * lane + i;
          int code;
          uint32_t mz;
          if (lv.tile) {
            const uint32_t vw = *reinterpret_cast<const uint32_t*>(tblk + 4096 + (t >> 6) * 2048 + c * 16 + ((t & 63) >> 4) * 4);
            code = (vw >> (16 * (t & 1) + 2 * ((t & 15) >> 1))) & 3;
            mz = reinterpret_cast<const uint32_t*>(tblk + 8192)[t * lv.VG + c / lv.G];
          } else {
            int word, bit;
            v_code_pos(jj, c, &word, &bit);
            code = (vcodes[word] >> bit) & 3;
            if (lv.v_bits == 4)      // the high plane follows the value scales
              code |= ((reinterpret_cast<const uint32_t*>(ub_ptr + 2048 + 128 * lv.VG)[word] >> bit) & 3) << 2;
            mz = vmeta[jj * lv.VG + c / lv.G];
          }
          vv[i] = fmaf((float)code, bf16_bits_to_float(mz & 0xFFFF), bf16_bits_to_float(mz >> 16));
        }
      } else {
        const int bu = unit - packed_units;
        const bool in_sink = bu >= res_units;
        const int j = (in_sink ? bu - res_units : bu) * 32 + jj;
        const uint16_t* rows = in_sink ? sinkv : resv;
        for (int i = 0; i < 4; ++i)
          vv[i] = (j < (in_sink ? lv.n_sink : lv.r)) ? bf16_bits_to_float(rows[(size_t)j * kD + 4 * lane + i]) : 0.f;
      }
      for (int h = 0; h < 8; ++h) {
        const float ph = __shfl_sync(0xffffffffu, p[h], jj);
        for (int i = 0; i < 4; ++i) o[h][i] = fmaf(ph, vv[i], o[h][i]);
      }
    }
  }

  // merge the four warps, write the split partial
  for (int h = 0; h < 8; ++h) {
    if (lane == 0) {
      mS[warp][h] = m[h];
      lS[warp][h] = l[h];
    }
    for (int i = 0; i < 4; ++i) oS[warp][h][4 * lane + i] = o[h][i];
  }
  __syncthreads();
  float* part = ws + ((size_t)s * nsplit + split) * kPartialFloats;
  for (int h = 0; h < 8; ++h) {
    const int c = threadIdx.x;
    float M = -INFINITY;
    for (int w = 0; w < 4; ++w) M = fmaxf(M, mS[w][h]);
    float ll = 0.f, oo = 0.f;
    for (int w = 0; w < 4; ++w) {
      const float f = (mS[w][h] == -INFINITY) ? 0.f : exp2f(mS[w][h] - M);
      ll += f * lS[w][h];
      oo += f * oS[w][h][c];
    }
    part[h * 130 + 2 + c] = oo;
    if (c == 0) {
      part[h * 130] = M;
      part[h * 130 + 1] = ll;
    }
  }
}

cudaError_t launch_attention_simt(const LayerView& lv, const void* q, float* out, float scale, float* ws, int n_sms,
                                  cudaStream_t stream, int* launches) {
  const int S = lv.B * lv.Hkv;
  const int units = lv.n_blocks * lv.U + (lv.r + 31) / 32 + (lv.n_sink + 31) / 32;
  int nsplit = (4 * n_sms + S - 1) / S;
  nsplit = max(1, min(nsplit, min(units, kMaxCtas / S > 0 ? kMaxCtas / S : 1)));
  attention_simt_kernel<<<dim3(S, nsplit), 128, 0, stream>>>(lv, static_cast<const __nv_bfloat16*>(q),
                                                             scale * 1.4426950408889634f, ws, nsplit);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  e = launch_combine(ws, out, lv.g, lv.Hkv, lv.Hq, 0, nsplit, 0, S, stream);
  *launches = 2;
  return e;
}

}  // namespace mixkvq
