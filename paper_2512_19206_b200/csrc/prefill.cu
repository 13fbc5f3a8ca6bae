// Causal full-precision attention over a prompt (the prefill phase of Section 4.2: the prompt is attended in full
// precision, then quantized into the cache) on the tcgen05 tensor cores with tensor-memory accumulators.
//
// One CTA of 128 threads per (batch element, query head, tile of 128 query positions).  It walks the key/value tiles
// 0 .. its own (causal).  Per tile:
//   S = Q K^T      one tcgen05.mma chain (M = 128 queries, N = 128 keys, K = 128 channels; bf16 operands from shared
//                  memory in the canonical K-major layout, fp32 accumulator in tensor memory);
//   softmax        thread j owns query row j: it reads its row of S from tensor memory (tcgen05.ld), applies the scale
//                  and the causal mask, keeps the running maximum and sum, and writes its row of P (fp16) as the A
//                  operand of the second product;
//   O_tile = P V   a second chain (M = 128 queries, N = 128 channels, K = 128 keys; V converted to fp16 on its way to
//                  shared memory, MN-major), into a second accumulator that the thread adds to its fp32 output row.
// P and V are fp16 (11 significant bits): bf16 probabilities alone would cost up to 2^-9 of the value range.
// Every wait on a barrier is bounded; a wait that runs out sets the status word and the CTA finishes.
#include "common.cuh"

namespace mixkvq {

namespace {

constexpr int kTile = 128;                       // query rows and key rows per tile
constexpr int kTileBytes = kTile * kD * 2;       // one 128 x 128 tile of 16-bit elements
constexpr int kSmem = 4 * kTileBytes + 64;       // Q, K, V, P tiles; barrier and tensor-memory slot
constexpr uint32_t kPolls = 1u << 21;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// canonical layout without swizzle: 8 x 16-byte core matrices; row r, 16-bit element k of a 128 x 128 tile
__device__ __forceinline__ uint32_t tile_off(int r, int k) {
  return (uint32_t)((r >> 3) * 2048 + (k >> 3) * 128 + (r & 7) * 16 + (k & 7) * 2);
}
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46);
}
// instruction descriptor of kind::f16: fp32 accumulator; operand formats 0 = fp16, 1 = bf16; B K-major (0) or MN-major (1)
__device__ __forceinline__ constexpr uint32_t make_idesc(int M, int N, int fmt, int b_mn_major) {
  return (1u << 4) | ((uint32_t)fmt << 7) | ((uint32_t)fmt << 10) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool mbar_wait_polls(uint32_t bar, uint32_t parity, uint32_t max_polls) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .u32 n;\n\tmov.u32 n, 0;\n"
      "PREFILL_WAIT:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 1000;\n\t"
      "@p bra PREFILL_DONE;\n\t"
      "add.u32 n, n, 1;\n\t"
      "setp.lt.u32 q, n, %3;\n\t"
      "@q bra PREFILL_WAIT;\n"
      "PREFILL_DONE:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(max_polls)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D (tensor memory) = A (shared memory) * B (shared memory) [+ D]
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&r)[32]) {
  uint32_t u[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
        "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]),
        "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]),
        "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) r[i] = __uint_as_float(u[i]);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
  return pack_half2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

// q [B, Hq, L, 128], k, v [B, Hkv, L, 128] bf16; out [B, Hq, L, 128] fp32.  blockIdx.x counts the query tiles from the
// last one down (the last tile has the most key tiles: the long CTAs start first), blockIdx.y = b * Hq + h.
__global__ void __launch_bounds__(128, 1)
prefill_attention_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                         const __nv_bfloat16* __restrict__ v, float* __restrict__ out, int Hq, int Hkv, int L,
                         float scale_log2e, uint32_t* status, uint32_t max_polls) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* Qs = smem;
  unsigned char* Ks = smem + kTileBytes;
  unsigned char* Vs = smem + 2 * kTileBytes;
  unsigned char* Ps = smem + 3 * kTileBytes;
  const uint32_t bar = smem_u32(smem + 4 * kTileBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 4 * kTileBytes + 16);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;
  const int bh = blockIdx.y, b = bh / Hq, h = bh % Hq, hk = h / (Hq / Hkv);
  const __nv_bfloat16* qg = q + ((size_t)(b * Hq + h) * L) * kD;
  const __nv_bfloat16* kg = k + ((size_t)(b * Hkv + hk) * L) * kD;
  const __nv_bfloat16* vg = v + ((size_t)(b * Hkv + hk) * L) * kD;

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = *tmem_slot;
  const uint32_t trow = tbase + ((uint32_t)(warp * 32) << 16);       // this warp's 32 lanes of tensor memory

  // a 128 x 128 bf16 tile of rows [row0, row0 + 128) of a [L][128] matrix -> shared memory; rows past L are zero.
  // Piece i (16 bytes): row 8 (i / 128) + i % 8, chunk (i / 8) % 16: eight rows of one chunk are 128 contiguous bytes.
  auto load_tile = [&](unsigned char* dst, const __nv_bfloat16* src, int row0, bool to_f16_mn_major) {
#pragma unroll 4
    for (int i = tid; i < kTile * 16; i += 128) {
      const int r = 8 * (i >> 7) + (i & 7), c = (i >> 3) & 15;
      uint4 x = make_uint4(0u, 0u, 0u, 0u);
      if (row0 + r < L) x = *reinterpret_cast<const uint4*>(src + (size_t)(row0 + r) * kD + 8 * c);
      if (to_f16_mn_major) {
        // B operand of P V: element (key r, channel d) at (d / 8) * 2048 + (r / 8) * 128 + (r % 8) * 16 + (d % 8) * 2
        x = make_uint4(bf16x2_to_f16x2(x.x), bf16x2_to_f16x2(x.y), bf16x2_to_f16x2(x.z), bf16x2_to_f16x2(x.w));
        *reinterpret_cast<uint4*>(dst + c * 2048 + (r >> 3) * 128 + (r & 7) * 16) = x;
      } else {
        *reinterpret_cast<uint4*>(dst + tile_off(r, 8 * c)) = x;
      }
    }
  };
  load_tile(Qs, qg, qt * kTile, false);

  const uint32_t idesc_qk = make_idesc(128, 128, 1, 0), idesc_pv = make_idesc(128, 128, 0, 1);
  const uint64_t q_desc = make_desc(smem_u32(Qs), 128, 2048), k_desc = make_desc(smem_u32(Ks), 128, 2048);
  const uint64_t p_desc = make_desc(smem_u32(Ps), 128, 2048), v_desc = make_desc(smem_u32(Vs), 128, 2048);
  uint32_t phase = 0;
  bool dead = false;
  auto wait_mma = [&]() {
    if (!dead && !mbar_wait_polls(bar, phase, max_polls)) {
      dead = true;
      atomicOr(status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
    }
    phase ^= 1u;
    tc_fence_after();
  };

  const int pos = qt * kTile + tid;                 // this thread's query position
  float o[kD];
#pragma unroll
  for (int d = 0; d < kD; ++d) o[d] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;

  for (int t = 0; t <= qt; ++t) {
    load_tile(Ks, kg, t * kTile, false);
    load_tile(Vs, vg, t * kTile, true);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the tiles written above are read by the tensor core
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) tc_mma_ss(tbase, q_desc + (uint64_t)(ks * 16), k_desc + (uint64_t)(ks * 16), idesc_qk, ks > 0);
      tc_commit(bar);
    }
    wait_mma();
    // ---- this thread's row of S: maximum first, then the probabilities
    const int tok0 = t * kTile;
    const int n_valid = min(min(pos - tok0 + 1, L - tok0), kTile);      // columns 0 .. n_valid - 1 take part (>= 1)
    float mx = -INFINITY;
#pragma unroll 1
    for (int cc = 0; cc < 4; ++cc) {
      float s[32];
      tmem_ld32(trow + 32 * cc, s);
#pragma unroll
      for (int i = 0; i < 32; ++i) mx = fmaxf(mx, 32 * cc + i < n_valid ? s[i] : -INFINITY);
    }
    const float m_new = fmaxf(m_run, mx * scale_log2e);
    const float alpha = ex2(m_run - m_new);            // 0 on the first tile
    float sum = 0.f;
#pragma unroll 1
    for (int cc = 0; cc < 4; ++cc) {
      float s[32];
      tmem_ld32(trow + 32 * cc, s);
#pragma unroll
      for (int i8 = 0; i8 < 4; ++i8) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int c0 = 32 * cc + 8 * i8 + 2 * j;
          // the probabilities are rounded to fp16 for the second product; the denominator sums the rounded ones
          const __half2 hp = __floats2half2_rn(c0 < n_valid ? ex2(fmaf(s[8 * i8 + 2 * j], scale_log2e, -m_new)) : 0.f,
                                               c0 + 1 < n_valid ? ex2(fmaf(s[8 * i8 + 2 * j + 1], scale_log2e, -m_new)) : 0.f);
          const float2 pf = __half22float2(hp);
          sum += pf.x + pf.y;
          w[j] = *reinterpret_cast<const uint32_t*>(&hp);
        }
        *reinterpret_cast<uint4*>(Ps + tile_off(tid, 32 * cc + 8 * i8)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
    l_run = l_run * alpha + sum;
    m_run = m_new;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        tc_mma_ss(tbase + 128, p_desc + (uint64_t)(ks * 16), v_desc + (uint64_t)(ks * 16), idesc_pv, ks > 0);
      tc_commit(bar);
    }
    wait_mma();
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      float x[32];
      tmem_ld32(trow + 128 + 32 * cc, x);
#pragma unroll
      for (int i = 0; i < 32; ++i) o[32 * cc + i] = fmaf(o[32 * cc + i], alpha, x[i]);
    }
    tc_fence_before();
    __syncthreads();           // everyone is done with the tiles and both accumulators
  }
  if (pos < L) {
    const float inv = 1.f / l_run;
    float4* dst = reinterpret_cast<float4*>(out + ((size_t)(b * Hq + h) * L + pos) * kD);
#pragma unroll
    for (int d = 0; d < kD; d += 4) dst[d >> 2] = make_float4(o[d] * inv, o[d + 1] * inv, o[d + 2] * inv, o[d + 3] * inv);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(256) : "memory");
}

}  // namespace

cudaError_t prefill_attention_setup() {
  return cudaFuncSetAttribute(prefill_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
}

cudaError_t launch_prefill_attention(const void* q, const void* k, const void* v, float* out, int B, int Hq, int Hkv, int L,
                                     float scale, uint32_t* status, uint32_t max_polls, cudaStream_t stream) {
  const int n_tiles = (L + kTile - 1) / kTile;
  dim3 grid((unsigned)n_tiles, (unsigned)(B * Hq));
  prefill_attention_kernel<<<grid, 128, kSmem, stream>>>(static_cast<const __nv_bfloat16*>(q),
                                                        static_cast<const __nv_bfloat16*>(k),
                                                        static_cast<const __nv_bfloat16*>(v), out, Hq, Hkv, L,
                                                        scale * 1.4426950408889634f, status, max_polls ? max_polls : kPolls);
  return cudaGetLastError();
}

}  // namespace mixkvq
