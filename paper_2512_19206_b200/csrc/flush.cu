// The lazy update of Appendix D.1 for one full residual window: channel statistics, salience and tiers
// (Section 4.2), per-channel mixed-precision key quantization and per-token 2-bit value quantization
// (Eq. 2), and bit-packing into the block layout.  One CTA per stream and block.
//
// Two sources: the residual window of the cache (decode: one block per call), or R-token windows taken straight
// from the tensors of a bulk append (prefill: grid.y blocks per call, the block's importance computed from its own
// queries).  The bulk form runs in two passes around a per-stream prefix sum, because a block's place in the
// promoted-channel arena depends on the tier counts of the blocks before it.
#include "common.cuh"

namespace mixkvq {

struct BulkSrc {
  const uint16_t* k;      // [S][n_tokens][128] bf16 bits
  const uint16_t* v;      // [S][n_tokens][128]
  const uint16_t* q;      // [B][Hq][n_tokens][128]
  int n_tokens, t0;       // tokens per stream in the tensors, first token of block 0 of this call
  int phase;              // 0: residual window; 1: bulk, tier counts only; 2: bulk, quantize and pack
};

__host__ __device__ inline uint32_t flush_extras_bytes(const LayerView& lv, int n16, int n4) {
  return lv.tile ? tile_extras_header_bytes(n16, n4) + tile_extras_body_bytes(n16, n4)
                 : extras_header_bytes(n16, n4) + (uint32_t)lv.U * extras_unit_bytes(n16, n4, lv.dense_hi != 0);
}

// Bulk append, between the two passes: one thread per stream walks the new blocks in order, gives each its offset in
// the promoted-channel arena and advances the arena pointer.  A block that no longer fits gets nothing in the arena and
// a table entry without promoted channels (its base part is still written; its BF16-tier channels then read as 0 and
// its UINT4 channels lose their high plane), and the status word says so: the same rule as for a single flush.
__global__ void bulk_prefix_kernel(LayerView lv, int nb) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= lv.B * lv.Hkv) return;
  char* state = lv.state + (size_t)s * lv.state_stride;
  uint32_t* used = reinterpret_cast<uint32_t*>(state + 1028);
  uint32_t off16 = *used;
  uint2* table = reinterpret_cast<uint2*>(lv.table + (size_t)s * lv.table_stride) + lv.n_blocks;
  for (int i = 0; i < nb; ++i) {
    uint2 e = table[i];
    const int n16 = e.y & 0xFF, n4 = (e.y >> 8) & 0xFF;
    const uint32_t need = flush_extras_bytes(lv, n16, n4);
    e.x = off16;
    if ((uint64_t)off16 * 16 + need > lv.extras_budget) {
      atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_EXTRAS_FULL);
      e.y = 0u;
    } else {
      off16 += need / 16;
    }
    table[i] = e;
  }
  *used = off16;
}

// Cumulative importance (Appendix D.2) in a bulk append: the running |q| sums continue across the windows, and the order of
// the sum is part of its definition, so one CTA per stream walks the nb windows in token order (queries staged 16 tokens at
// a time, thread d adds channel d).  It leaves the sums and the count as they stand at the end of each window in bytes
// 128.. of that window's (still unwritten) block, where the first bulk pass reads them, and the final values in the state.
constexpr int kSnapshotOff = 128, kSnapshotCntOff = 128 + 1024;

__global__ void __launch_bounds__(256)
bulk_importance_kernel(LayerView lv, BulkSrc src, int nb) {
  __shared__ __align__(16) uint16_t qS[16 * 8 * kD];      // [token][head][128] bf16 bits
  const int s = blockIdx.x, tid = threadIdx.x, g = lv.g, R = lv.R;
  const int b = s / lv.Hkv, hk = s % lv.Hkv;
  char* state = lv.state + (size_t)s * lv.state_stride;
  double a = tid < kD ? reinterpret_cast<const double*>(state)[tid] : 0.0;
  uint32_t cnt = *reinterpret_cast<const uint32_t*>(state + 1024);
  const uint16_t* qw = src.q + (((size_t)b * lv.Hq + hk * g) * src.n_tokens + src.t0) * kD;
  const size_t head_stride = (size_t)src.n_tokens * kD;
  // the queries of the next 16 tokens are requested (into registers) before the sums of the current 16 are taken
  const int n_rounds = nb * (R / 16), per_round = 16 * g * 16;       // 16-byte pieces per round (<= 2048)
  uint4 pre[8];
  auto request = [&](int round) {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int i = tid + 256 * k;
      if (i < per_round) {
        const int row = i >> 4, c16 = i & 15, jj = row / g, h = row - jj * g;
        pre[k] = *reinterpret_cast<const uint4*>(qw + (size_t)(round * 16 + jj) * kD + h * head_stride + 8 * c16);
      }
    }
  };
  request(0);
  for (int w = 0; w < nb; ++w) {
    for (int j0 = 0; j0 < R; j0 += 16) {
      const int round = w * (R / 16) + j0 / 16;
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (tid + 256 * k < per_round) reinterpret_cast<uint4*>(qS)[tid + 256 * k] = pre[k];
      __syncthreads();
      if (round + 1 < n_rounds) request(round + 1);
      if (tid < kD)
        for (int row = 0; row < 16 * g; ++row)
          a = __dadd_rn(a, (double)fabsf(bf16_bits_to_float(qS[row * kD + tid])));
      __syncthreads();
    }
    cnt += (uint32_t)(R * g);
    char* blk = lv.base + (size_t)s * lv.base_stride + (size_t)(lv.n_blocks + w) * lv.base_bytes;
    if (tid < kD) reinterpret_cast<double*>(blk + kSnapshotOff)[tid] = a;
    if (tid == 0) *reinterpret_cast<uint32_t*>(blk + kSnapshotCntOff) = cnt;
  }
  if (tid < kD) reinterpret_cast<double*>(state)[tid] = a;
  if (tid == 0) *reinterpret_cast<uint32_t*>(state + 1024) = cnt;
}

__global__ void __launch_bounds__(256)
flush_kernel(LayerView lv, BulkSrc src) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int R = lv.R, G = lv.G, U = lv.U, NG = lv.NG, VG = lv.VG;
  uint16_t* kS = reinterpret_cast<uint16_t*>(smem);      // [R][128] residual keys (bf16 bits)
  uint8_t* cS = smem + (size_t)R * 256;                   // [R][128] codes (keys, later values)
  uint8_t* tierS = cS + (size_t)R * 128;                  // [128]
  uint8_t* chan16S = tierS + 128;                         // [128]
  uint8_t* chan4S = chan16S + 128;                        // [128]
  int* misc = reinterpret_cast<int*>(chan4S + 128);       // n16, n4, extras offset (16-byte units)
  float* wS = reinterpret_cast<float*>(chan4S + 128 + 16); // [2 halves][128]{max, min} of the window, later the tier counts
  double* aS = reinterpret_cast<double*>(chan4S + 128 + 16 + 2048);   // [128] saliences of the window

  const int s = blockIdx.x, tid = threadIdx.x;
  const bool bulk = src.phase != 0;
  int first_block = lv.n_blocks;
  if (lv.seq != nullptr) {
    // ragged batch (single flush only): the sequences whose window is full take part, each with its own block count
    const int4 f = lv.seq[s / lv.Hkv];
    if (f.y != R) return;
    first_block = f.x;
  }
  const int block_index = first_block + (bulk ? (int)blockIdx.y : 0);
  const size_t tok0 = (size_t)s * src.n_tokens + src.t0 + (size_t)blockIdx.y * R;     // bulk: first token of the window
  char* state = lv.state + (size_t)s * lv.state_stride;
  char* blk = lv.base + (size_t)s * lv.base_stride + (size_t)block_index * lv.base_bytes;
  const uint4* resk4 = bulk ? reinterpret_cast<const uint4*>(src.k + tok0 * kD)
                            : reinterpret_cast<const uint4*>(lv.resk + (size_t)s * lv.resk_stride);
  const uint16_t* resv = reinterpret_cast<const uint16_t*>(lv.resv + (size_t)s * lv.resv_stride);
  uint2* table_entry = reinterpret_cast<uint2*>(lv.table + (size_t)s * lv.table_stride + (size_t)block_index * 8);

  // a window of R rows of 256 bytes: the loads of a thread go out together, then the stores
  auto load_window = [&](const uint4* from) {
    for (int i0 = 0; i0 < R * 16; i0 += 8 * 256) {
      uint4 tmp[8];
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (i0 + tid + 256 * k < R * 16) tmp[k] = from[i0 + tid + 256 * k];
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (i0 + tid + 256 * k < R * 16) reinterpret_cast<uint4*>(kS)[i0 + tid + 256 * k] = tmp[k];
    }
  };

  // ---- bulk, first pass: importance of this window from its own queries, before the key window takes the shared
  // memory.  All threads stage as many tokens of the g heads as the key and code areas hold (16-byte loads); thread d
  // then adds |q| of channel d token-major and head-ascending, the order of the running accumulator of the decode path.
  double bulk_acc = 0.0;
  uint32_t bulk_cnt = (uint32_t)(R * lv.g);
  if (src.phase == 1 && lv.importance_mode == 1) {
    // cumulative importance: the sums at the end of this window were left in the block by bulk_importance_kernel
    if (tid < kD) bulk_acc = reinterpret_cast<const double*>(blk + kSnapshotOff)[tid];
    bulk_cnt = *reinterpret_cast<const uint32_t*>(blk + kSnapshotCntOff);
  } else if (src.phase == 1) {
    const int b = s / lv.Hkv, hk = s % lv.Hkv;
    const uint16_t* qw = src.q + (((size_t)b * lv.Hq + hk * lv.g) * src.n_tokens + src.t0 + (size_t)blockIdx.y * R) * kD;
    const size_t head_stride = (size_t)src.n_tokens * kD;
    uint16_t* qS = reinterpret_cast<uint16_t*>(smem);                // [tc tokens][g heads][128]
    const int tc = min(R, (R * 384) / (lv.g * 256));                 // tokens per round: R * 384 bytes of key + code area
    for (int j0 = 0; j0 < R; j0 += tc) {
      const int tn = min(tc, R - j0), pieces = tn * lv.g * 16;
      for (int i0 = 0; i0 < pieces; i0 += 4 * 256) {       // four loads per thread in flight, then the stores
        uint4 tmp[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int i = i0 + tid + 256 * k;
          if (i < pieces) {
            const int row = i >> 4, c16 = i & 15, jj = row / lv.g, h = row - jj * lv.g;
            tmp[k] = *reinterpret_cast<const uint4*>(qw + (size_t)(j0 + jj) * kD + h * head_stride + 8 * c16);
          }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (i0 + tid + 256 * k < pieces) reinterpret_cast<uint4*>(qS)[i0 + tid + 256 * k] = tmp[k];
      }
      __syncthreads();
      if (tid < kD)
        for (int row = 0; row < tn * lv.g; ++row)
          bulk_acc = __dadd_rn(bulk_acc, (double)fabsf(bf16_bits_to_float(qS[row * kD + tid])));
      __syncthreads();
    }
  }

  load_window(resk4);
  if (src.phase == 2) {
    // the first pass left the 128 tiers in the first bytes of the block; fetch them before anything is written there
    if (tid < kD) tierS[tid] = reinterpret_cast<const uint8_t*>(blk)[tid];
  }
  __syncthreads();

  // ---- statistics, salience, tier and key codes: two threads per channel (halves of the window for its extrema,
  // alternate key groups for the codes)
  {
    const int d = tid & (kD - 1), half = tid >> 7;
    if (src.phase != 2) {
      float wmx = -INFINITY, wmn = INFINITY;
      for (int j = half * (R / 2); j < (half + 1) * (R / 2); ++j) {
        float x = bf16_bits_to_float(kS[j * kD + d]);
        wmx = fmaxf(wmx, x);
        wmn = fminf(wmn, x);
      }
      wS[(half * kD + d) * 2] = wmx;
      wS[(half * kD + d) * 2 + 1] = wmn;
      __syncthreads();
      if (half == 0) {
        wmx = fmaxf(wS[d * 2], wS[(kD + d) * 2]);
        wmn = fminf(wS[d * 2 + 1], wS[(kD + d) * 2 + 1]);
        double acc;
        uint32_t cnt;
        if (bulk) {
          acc = bulk_acc;
          cnt = bulk_cnt;
        } else {
          acc = reinterpret_cast<const double*>(state)[d];
          cnt = *reinterpret_cast<const uint32_t*>(state + 1024);
        }
        double A;
        const uint8_t tier =
            salience_tier(acc, cnt, wmx, wmn, lv.score_bits, lv.tau_bf16, lv.tau_u4, &A, lv.importance_mode == 2);
        aS[d] = A;
        tierS[d] = tier;
      }
      if (lv.budget_bf16 + lv.budget_u4 > 0) {     // fixed budget: the rank among the window's saliences decides
        __syncthreads();
        if (half == 0) tierS[d] = budget_tier(aS, d, lv.budget_bf16, lv.budget_u4);
      }
      if (half == 0 && src.phase == 1) reinterpret_cast<uint8_t*>(blk)[d] = tierS[d];
      __syncthreads();
    }
    if (src.phase != 1) {
      const uint8_t tier = tierS[d];
      const int max_code = (tier == kU4) ? 15 : 3;
      for (int kg = half; kg < NG; kg += 2) {
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
          const float rs = __frcp_rn(sc);
#pragma unroll 4
          for (int j = kg * G; j < (kg + 1) * G; ++j)
            cS[j * kD + d] = (uint8_t)quant_code_fast(bf16_bits_to_float(kS[j * kD + d]), gmn, sc, rs, max_code);
          meta = float_to_bf16_bits_exact(sc) | (float_to_bf16_bits_exact(gmn) << 16);
        }
        reinterpret_cast<uint32_t*>(blk + (lv.tile ? (uint32_t)kg * 512u : frag_meta_off(kg, G, lv.unit_bytes)))[d] = meta;
      }
    }
  }
  __syncthreads();

  // ---- channel lists (ascending channel order inside each tier: warp ballots and a prefix over the four warps)
  {
    int* cntS = reinterpret_cast<int*>(wS);          // [2][4] per-warp counts (the extrema are no longer needed)
    unsigned m16 = 0, m4 = 0;
    const int warp = tid >> 5, lane = tid & 31;
    if (tid < kD) {
      const uint8_t tier = tierS[tid];
      m16 = __ballot_sync(0xffffffffu, tier == kBF16);
      m4 = __ballot_sync(0xffffffffu, tier == kU4);
      if (lane == 0) {
        cntS[warp] = __popc(m16);
        cntS[4 + warp] = __popc(m4);
      }
    }
    __syncthreads();
    if (tid < kD) {
      int b16 = 0, b4 = 0;
      for (int w2 = 0; w2 < warp; ++w2) {
        b16 += cntS[w2];
        b4 += cntS[4 + w2];
      }
      const unsigned below = (1u << lane) - 1u;
      if (m16 & (1u << lane)) chan16S[b16 + __popc(m16 & below)] = (uint8_t)tid;
      if (m4 & (1u << lane)) chan4S[b4 + __popc(m4 & below)] = (uint8_t)tid;
    }
  }
  // ---- extras allocation, table entry
  if (tid == 0) {
    const int* cntS = reinterpret_cast<const int*>(wS);
    int n16 = cntS[0] + cntS[1] + cntS[2] + cntS[3], n4 = cntS[4] + cntS[5] + cntS[6] + cntS[7];
    uint32_t off16 = 0;
    if (src.phase == 1) {
      // bulk, first pass: only the tier counts; the offsets come from the per-stream prefix sum
      *table_entry = make_uint2(0u, (uint32_t)n16 | ((uint32_t)n4 << 8));
    } else if (src.phase == 2) {
      // bulk, second pass: the prefix sum placed the block (and cleared the counts if the arena was full)
      const uint2 e = *table_entry;
      off16 = e.x;
      if ((e.y & 0xFFFFu) == 0u) {
        n16 = 0;
        n4 = 0;
      }
    } else {
      uint32_t* used = reinterpret_cast<uint32_t*>(state + 1028);
      off16 = *used;
      const uint32_t need = flush_extras_bytes(lv, n16, n4);
      if ((uint64_t)off16 * 16 + need > lv.extras_budget) {
        atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_EXTRAS_FULL);
        n16 = 0;
        n4 = 0;      // nothing goes to the arena and the entry records no promoted channel; the status word says so
      } else {
        *used = off16 + need / 16;
      }
      *table_entry = make_uint2(off16, (uint32_t)n16 | ((uint32_t)n4 << 8));
    }
    misc[0] = n16;
    misc[1] = n4;
    misc[2] = (int)off16;
  }
  __syncthreads();
  if (src.phase == 1) return;
  const int n16 = misc[0], n4 = misc[1];
  const int n16p = (n16 + 1) >> 1, n4p = ((n4 + 1) >> 1) << 1;
  char* ex = lv.extras + (size_t)s * lv.extras_stride + (size_t)misc[2] * 16;
  const uint32_t hdr = extras_header_bytes(n16, n4), exunit = extras_unit_bytes(n16, n4, lv.dense_hi != 0);

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
      reinterpret_cast<uint32_t*>(blk + frag_unit_off(u, G, lv.unit_bytes))[wi] = w;
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
    if (lv.dense_hi) {
      // dense high plane: the low plane's fragment order, code >> 2 of UINT4 channels, 0 elsewhere
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
            if (tierS[d] == kU4) w |= (uint32_t)(cS[j * kD + d] >> 2) << (16 * e + 2 * kt);
          }
        reinterpret_cast<uint32_t*>(ex + hdr + (size_t)u * exunit + 128 * n16p)[wi] = w;
      }
    }
    for (int i = tid; i < (lv.dense_hi ? 0 : U * (n4p / 2) * 4); i += 256) {
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

  // ---- values: per token, per group of G channels, 2 bits.  The key window is no longer needed: the value window
  // takes its place in shared memory (token-major in the residual store and in a tensor alike).
  {
    const uint4* vsrc = bulk ? reinterpret_cast<const uint4*>(src.v + tok0 * kD) : reinterpret_cast<const uint4*>(resv);
    load_window(vsrc);
  }
  __syncthreads();
  auto vmeta_of = [&](int j) -> uint32_t* {
    const int u = j >> 5, jj = j & 31;
    return lv.tile ? reinterpret_cast<uint32_t*>(blk + NG * 512 + 8192) + j * VG
                   : reinterpret_cast<uint32_t*>(blk + frag_unit_off(u, G, lv.unit_bytes) + 2048) + jj * VG;
  };
  {
    // token-major window: a warp takes a token, lane l the channels 4l .. 4l+3 (one 8-byte load); a group of G channels
    // is G / 4 neighbouring lanes, its extrema a butterfly over those lanes
    const int warp = tid >> 5, lane = tid & 31;
#pragma unroll 2
    for (int j = warp; j < R; j += 8) {
      const uint2 raw = *reinterpret_cast<const uint2*>(&kS[j * kD + 4 * lane]);
      const float x[4] = {bf16_bits_to_float(raw.x & 0xFFFFu), bf16_bits_to_float(raw.x >> 16),
                          bf16_bits_to_float(raw.y & 0xFFFFu), bf16_bits_to_float(raw.y >> 16)};
      float gmx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), gmn = fminf(fminf(x[0], x[1]), fminf(x[2], x[3]));
      for (int off = 1; off < G / 4; off <<= 1) {
        gmx = fmaxf(gmx, __shfl_xor_sync(0xffffffffu, gmx, off));
        gmn = fminf(gmn, __shfl_xor_sync(0xffffffffu, gmn, off));
      }
      const int vmax = lv.v_bits == 4 ? 15 : 3;
      const float sc = stored_scale(gmx, gmn, (float)vmax);
      const float rs = __frcp_rn(sc);
      uint32_t codes = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) codes |= (uint32_t)quant_code_fast(x[k], gmn, sc, rs, vmax) << (8 * k);
      *reinterpret_cast<uint32_t*>(&cS[j * kD + 4 * lane]) = codes;
      if ((4 * lane) % G == 0)
        vmeta_of(j)[(4 * lane) / G] = float_to_bf16_bits_exact(sc) | (float_to_bf16_bits_exact(gmn) << 16);
    }
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
              w |= (uint32_t)(cS[j * kD + c] & 3) << (16 * e + 2 * (4 * rh + 2 * ks + ch));
            }
      reinterpret_cast<uint32_t*>(blk + frag_unit_off(u, G, lv.unit_bytes) + 1024)[wi] = w;
    }
    // 4-bit values: the high plane (code >> 2) in the same bit order, after the unit's value scales
    for (int i = tid; i < (lv.v_bits == 4 ? U * 256 : 0); i += 256) {
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
              w |= (uint32_t)(cS[j * kD + c] >> 2) << (16 * e + 2 * (4 * rh + 2 * ks + ch));
            }
      reinterpret_cast<uint32_t*>(blk + frag_unit_off(u, G, lv.unit_bytes) + 2048 + 128 * VG)[wi] = w;
    }
  }

  // ---- window importance: the accumulator restarts with the next window (Section 4.2)
  if (lv.importance_mode != 1 && !bulk) {
    if (tid < kD) reinterpret_cast<double*>(state)[tid] = 0.0;
    if (tid == 0) *reinterpret_cast<uint32_t*>(state + 1024) = 0u;
  }
}

static size_t flush_smem_bytes(int R) { return (size_t)R * 384 + 3 * 128 + 16 + 2048 + 1024; }

cudaError_t launch_flush(const LayerView& lv, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(flush_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)flush_smem_bytes(256));
  if (e != cudaSuccess) return e;
  flush_kernel<<<lv.B * lv.Hkv, 256, flush_smem_bytes(lv.R), stream>>>(lv, BulkSrc{nullptr, nullptr, nullptr, 0, 0, 0});
  return cudaGetLastError();
}

// nb complete R-token windows starting at token t0 of the append's tensors go straight to packed blocks
// (three launches, four with cumulative importance).  Precondition (checked by the caller): empty residual window.
cudaError_t launch_flush_bulk(const LayerView& lv, const void* k, const void* v, const void* q, int n_tokens, int t0,
                              int nb, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(flush_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)flush_smem_bytes(256));
  if (e != cudaSuccess) return e;
  const int S = lv.B * lv.Hkv;
  BulkSrc src{static_cast<const uint16_t*>(k), static_cast<const uint16_t*>(v), static_cast<const uint16_t*>(q), n_tokens, t0, 1};
  const dim3 grid(S, nb);
  if (lv.importance_mode == 1) bulk_importance_kernel<<<S, 256, 0, stream>>>(lv, src, nb);
  flush_kernel<<<grid, 256, flush_smem_bytes(lv.R), stream>>>(lv, src);
  bulk_prefix_kernel<<<(S + 127) / 128, 128, 0, stream>>>(lv, nb);
  src.phase = 2;
  flush_kernel<<<grid, 256, flush_smem_bytes(lv.R), stream>>>(lv, src);
  return cudaGetLastError();
}

}  // namespace mixkvq
