// Causal full-precision attention over a prompt (the prefill phase of Section 4.2: the prompt is attended in full
// precision, then quantized into the cache) on the tcgen05 tensor cores with tensor-memory accumulators.
//
// Two kernels.  prefill_pack_kernel rewrites K (bf16) and V (converted to fp16) of the prompt into images of 128-token
// tiles in the tensor core's canonical shared-memory layout, so that a tile reaches shared memory as ONE 32 KB bulk
// copy.  prefill_attention_kernel runs one CTA of 384 threads per (batch element, query head, 256 query positions):
//   warps 0-3, 4-7   two softmax groups, one per 128 query rows (thread = row = lane of tensor memory);
//   warp 8           one thread issues every tcgen05.mma;
//   warp 9           one thread issues the bulk copies of the K and V tiles into two-stage rings.
// Per key tile j and row group g:
//   S_g = Q_g K_j^T   bf16 operands from shared memory, fp32 accumulator in tensor memory;
//   softmax           the thread reads its row of S (tcgen05.ld), applies scale and causal mask, keeps the running
//                     maximum and sum, and writes its row of P as fp16 over the columns S occupied (tcgen05.st);
//   T_g = P_g V_j     A operand from tensor memory, V from shared memory (MN-major), into a second accumulator that
//                     the thread folds into its fp32 output row in registers: o = o * alpha + T.
// The issue order S_A(j+1) behind P_A V(j), S_B(j+1) behind P_B V(j) keeps the tensor core busy on one row group while
// the other one is in its softmax.  P and V are fp16 (11 significant bits): bf16 probabilities alone would cost up to
// 2^-9 of the value range.  Every wait on a barrier is bounded; a wait that runs out sets the status word and the
// role that saw it stops, after which the others run out too and the CTA finishes.
#include "common.cuh"

namespace mixkvq {

namespace {

constexpr int kTile = 128;                       // query rows and key rows per tile
constexpr int kTileBytes = kTile * kD * 2;       // one 128 x 128 tile of 16-bit elements
constexpr int kQRows = 2 * kTile;                // query rows per CTA
constexpr int kThreads = 384;
constexpr int kBars = 17;
constexpr int kSmem = 6 * kTileBytes + 256;      // two Q tiles, two K and two V stages; barriers and tensor-memory slot
enum Bar { kKFull = 0, kVFull = 2, kKEmpty = 4, kVEmpty = 6, kSFull = 8, kPReady = 10, kTFull = 12, kTFree = 14, kDone = 16 };
constexpr uint32_t kPolls = 1u << 21;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Canonical layout without swizzle: 8-row x 16-byte core matrices; row r, 16-bit element k of a 128 x 128 K-major tile
// sits at byte (r / 8) * 2048 + (k / 8) * 128 + (r % 8) * 16 + (k % 8) * 2.
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
// A load of 32 columns of the thread's tensor-memory lane.  The registers are valid only after tmem_wait_ld32 / tmem_wait_ld16 on them (the wait
// names the registers as operands, so that no use of them is scheduled before it).  tcgen05.wait::ld covers every load
// the thread has issued, so a load issued before a block of arithmetic and waited for after it runs under that arithmetic.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&u)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
        "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]),
        "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]),
        "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld32(uint32_t (&u)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(u[0]), "+r"(u[1]), "+r"(u[2]), "+r"(u[3]), "+r"(u[4]), "+r"(u[5]), "+r"(u[6]), "+r"(u[7]), "+r"(u[8]),
                 "+r"(u[9]), "+r"(u[10]), "+r"(u[11]), "+r"(u[12]), "+r"(u[13]), "+r"(u[14]), "+r"(u[15]), "+r"(u[16]),
                 "+r"(u[17]), "+r"(u[18]), "+r"(u[19]), "+r"(u[20]), "+r"(u[21]), "+r"(u[22]), "+r"(u[23]), "+r"(u[24]),
                 "+r"(u[25]), "+r"(u[26]), "+r"(u[27]), "+r"(u[28]), "+r"(u[29]), "+r"(u[30]), "+r"(u[31])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&u)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
        "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld16(uint32_t (&u)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(u[0]), "+r"(u[1]), "+r"(u[2]), "+r"(u[3]), "+r"(u[4]), "+r"(u[5]), "+r"(u[6]), "+r"(u[7]), "+r"(u[8]),
                 "+r"(u[9]), "+r"(u[10]), "+r"(u[11]), "+r"(u[12]), "+r"(u[13]), "+r"(u[14]), "+r"(u[15])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&w)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(w[0]), "r"(w[1]),
               "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
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


__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// D (tensor memory) = A (tensor memory, 16-bit pairs per column) * B (shared memory) [+ D]
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// K, V [B * Hkv][L][128] bf16 -> tile images [B * Hkv][n_tiles][32 KB]: K as the K-major B operand of Q K^T (bf16),
// V as the MN-major B operand of P V (fp16); rows past L are zero.  Consecutive threads write consecutive 16 bytes.
__global__ void __launch_bounds__(256)
prefill_pack_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, unsigned char* __restrict__ kt,
                    unsigned char* __restrict__ vt, int L, int n_tiles) {
  const int t = blockIdx.x, s = blockIdx.y;
  const __nv_bfloat16* kg = k + ((size_t)s * L + (size_t)t * kTile) * kD;
  const __nv_bfloat16* vg = v + ((size_t)s * L + (size_t)t * kTile) * kD;
  uint4* kd = reinterpret_cast<uint4*>(kt + ((size_t)s * n_tiles + t) * kTileBytes);
  uint4* vd = reinterpret_cast<uint4*>(vt + ((size_t)s * n_tiles + t) * kTileBytes);
  const int rows = min(kTile, L - t * kTile);
#pragma unroll 2
  for (int i = threadIdx.x; i < kTile * 16; i += 256) {
    {  // K: byte offset (r / 8) * 2048 + c * 128 + (r % 8) * 16 of row r, 16-byte chunk c
      const int r = 8 * (i >> 7) + (i & 7), c = (i >> 3) & 15;
      uint4 x = make_uint4(0u, 0u, 0u, 0u);
      if (r < rows) x = *reinterpret_cast<const uint4*>(kg + (size_t)r * kD + 8 * c);
      kd[i] = x;
    }
    {  // V: byte offset c * 2048 + (r / 8) * 128 + (r % 8) * 16
      const int r = (i & 127), c = i >> 7;
      uint4 x = make_uint4(0u, 0u, 0u, 0u);
      if (r < rows) x = *reinterpret_cast<const uint4*>(vg + (size_t)r * kD + 8 * c);
      vd[i] = make_uint4(bf16x2_to_f16x2(x.x), bf16x2_to_f16x2(x.y), bf16x2_to_f16x2(x.z), bf16x2_to_f16x2(x.w));
    }
  }
}

// One 128-key tile of one row group's softmax.  The thread owns one row of S (128 fp32 columns of its tensor-memory
// lane at s_addr); columns >= n_valid are masked.  Writes P (fp16 pairs) over columns [0, 64) of the same range.
template <bool kMask>
__device__ __forceinline__ void softmax_tile(uint32_t s_addr, int n_valid, float scale_log2e, float& m_run, float& l_run,
                                             float& alpha) {
  // ---- pass 1: the row maximum; chunk c + 1 is in flight while chunk c is reduced
  float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};      // four independent chains
  {
    uint32_t a[32], b[32];
    auto reduce = [&](const uint32_t (&u)[32], int cc) {
#pragma unroll
      for (int i = 0; i < 32; ++i)
        mx4[i & 3] = fmaxf(mx4[i & 3], (!kMask || 32 * cc + i < n_valid) ? __uint_as_float(u[i]) : -INFINITY);
    };
    tmem_ld32_issue(s_addr, a);
    tmem_wait_ld32(a);
    tmem_ld32_issue(s_addr + 32, b);
    reduce(a, 0);
    tmem_wait_ld32(b);
    tmem_ld32_issue(s_addr + 64, a);
    reduce(b, 1);
    tmem_wait_ld32(a);
    tmem_ld32_issue(s_addr + 96, b);
    reduce(a, 2);
    tmem_wait_ld32(b);
    reduce(b, 3);
  }
  const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
  const float m_new = fmaxf(m_run, mx * scale_log2e);
  alpha = ex2(m_run - m_new);                       // 0 on the first tile
  // ---- pass 2: probabilities in chunks of 16 columns, the next chunk in flight; P chunk c (8 columns of fp16 pairs)
  // lies inside the S columns of chunks <= c, which are already in registers
  float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
  {
    uint32_t a[16], b[16];
    auto probs = [&](const uint32_t (&u)[16], int cc) {
      uint32_t w[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c0 = 16 * cc + 2 * i;
        const float p0 = (!kMask || c0 < n_valid) ? ex2(fmaf(__uint_as_float(u[2 * i]), scale_log2e, -m_new)) : 0.f;
        const float p1 = (!kMask || c0 + 1 < n_valid) ? ex2(fmaf(__uint_as_float(u[2 * i + 1]), scale_log2e, -m_new)) : 0.f;
        if (i & 1) {
          sum2 += p0;
          sum3 += p1;
        } else {
          sum0 += p0;
          sum1 += p1;
        }
        w[i] = pack_half2(p0, p1);
      }
      tmem_st8(s_addr + 8 * cc, w);
    };
    tmem_ld16_issue(s_addr, a);
    tmem_wait_ld16(a);
#pragma unroll
    for (int cc = 0; cc < 8; cc += 2) {
      tmem_ld16_issue(s_addr + 16 * (cc + 1), b);
      probs(a, cc);                                // writes columns [8 cc, 8 cc + 8): all inside chunks <= cc
      tmem_wait_ld16(b);
      if (cc + 2 < 8) tmem_ld16_issue(s_addr + 16 * (cc + 2), a);
      probs(b, cc + 1);
      if (cc + 2 < 8) tmem_wait_ld16(a);
    }
  }
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  l_run = l_run * alpha + ((sum0 + sum1) + (sum2 + sum3));
  m_run = m_new;
}

// q [B, Hq, L, 128] bf16; kt, vt the tile images of prefill_pack_kernel; out [B, Hq, L, 128] fp32.  blockIdx.x / BH
// counts the 256-row query tiles from the last one down (it has the most key tiles: the long CTAs start first),
// blockIdx.x % BH = b * Hq + h.
__global__ void __launch_bounds__(kThreads, 1)
prefill_attention_kernel(const __nv_bfloat16* __restrict__ q, const unsigned char* __restrict__ kt,
                         const unsigned char* __restrict__ vt, float* __restrict__ out, int BH, int Hq, int Hkv, int L,
                         int n_tiles, int n_qtiles, float scale_log2e, uint32_t* status, uint32_t max_polls, uint32_t debug_extra_tx) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* Qs = smem;                              // two tiles
  unsigned char* Ks = smem + 2 * kTileBytes;             // two stages
  unsigned char* Vs = smem + 4 * kTileBytes;             // two stages
  const uint32_t bars = smem_u32(smem + 6 * kTileBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 6 * kTileBytes + 8 * kBars);
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int qt = n_qtiles - 1 - (int)blockIdx.x / BH;
  const int bh = (int)blockIdx.x % BH, b = bh / Hq, h = bh % Hq, hk = h / (Hq / Hkv);
  const __nv_bfloat16* qg = q + ((size_t)(b * Hq + h) * L) * kD;
  const unsigned char* ktg = kt + (size_t)(b * Hkv + hk) * n_tiles * kTileBytes;
  const unsigned char* vtg = vt + (size_t)(b * Hkv + hk) * n_tiles * kTileBytes;
  // key tiles of the two row groups: rows [256 qt, +128) see tiles 0 .. 2 qt, rows [256 qt + 128, +128) one more
  const int n_a = 2 * qt + 1, n_b = min(2 * qt + 2, n_tiles);

  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 9 * 32) {
    for (int i = 0; i < kBars; ++i) mbar_init(bar(i), (i >= kPReady && i < kTFull) || (i >= kTFree && i < kDone) ? kTile : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // both Q tiles: piece i of a tile is 16 bytes at byte 16 i of its image (rows past L are zero)
  for (int i = tid; i < 2 * kTile * 16; i += kThreads) {
    const int ii = i & 2047, r = (i >> 11) * kTile + 8 * (ii >> 7) + (ii & 7), c = (ii >> 3) & 15;
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    if (qt * kQRows + r < L) x = *reinterpret_cast<const uint4*>(qg + (size_t)(qt * kQRows + r) * kD + 8 * c);
    reinterpret_cast<uint4*>(Qs)[i] = x;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");        // Q is read by the tensor core
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = *tmem_slot;
  // tensor-memory columns: S_A / P_A at 0, S_B / P_B at 128, T_A at 256, T_B at 384
  bool dead = false;
  auto wait = [&](int i, uint32_t parity) {
    if (!dead && !mbar_wait_polls(bar(i), parity, max_polls)) {
      dead = true;
      atomicOr(status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
    }
    return !dead;
  };

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;" ::: "memory");
    if (warp == 8 && lane == 0) {
      // ---------------------------------------------------------------- tensor-core issue
      const uint32_t idesc_qk = make_idesc(128, 128, 1, 0), idesc_pv = make_idesc(128, 128, 0, 1);
      auto issue_s = [&](int g, int j) {                 // S_g = Q_g K_j^T
        const uint64_t qd = make_desc(smem_u32(Qs + g * kTileBytes), 128, 2048);
        const uint64_t kd = make_desc(smem_u32(Ks + (j & 1) * kTileBytes), 128, 2048);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) tc_mma_ss(tbase + 128 * g, qd + (uint64_t)(ks * 16), kd + (uint64_t)(ks * 16), idesc_qk, ks > 0);
        tc_commit(bar(kSFull + g));
      };
      auto issue_t = [&](int g, int j) {                 // T_g = P_g V_j
        const uint64_t vd = make_desc(smem_u32(Vs + (j & 1) * kTileBytes), 128, 2048);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) tc_mma_ts(tbase + 256 + 128 * g, tbase + 128 * g + 8 * ks, vd + (uint64_t)(ks * 16), idesc_pv, ks > 0);
        tc_commit(bar(kTFull + g));
      };
      if (wait(kKFull, 0)) {
        tc_fence_after();
        issue_s(0, 0);
        issue_s(1, 0);
        tc_commit(bar(kKEmpty));
      }
      for (int j = 0; j < n_b && !dead; ++j) {
        const int st = j & 1, nx = (j + 1) & 1;
        const uint32_t ph = (uint32_t)(j >> 1) & 1u, ph_nx = (uint32_t)((j + 1) >> 1) & 1u;
        if (!wait(kVFull + st, ph)) break;
        if (j < n_a) {
          if (!wait(kPReady, (uint32_t)j & 1u)) break;
          if (j > 0 && !wait(kTFree, (uint32_t)(j - 1) & 1u)) break;
          tc_fence_after();
          issue_t(0, j);
          if (j + 1 < n_a) {
            if (!wait(kKFull + nx, ph_nx)) break;
            tc_fence_after();
            issue_s(0, j + 1);
          }
        }
        if (!wait(kPReady + 1, (uint32_t)j & 1u)) break;
        if (j > 0 && !wait(kTFree + 1, (uint32_t)(j - 1) & 1u)) break;
        tc_fence_after();
        issue_t(1, j);
        tc_commit(bar(kVEmpty + st));
        if (j + 1 < n_b) {
          if (!wait(kKFull + nx, ph_nx)) break;
          tc_fence_after();
          issue_s(1, j + 1);
          tc_commit(bar(kKEmpty + nx));
        }
      }
      tc_commit(bar(kDone));                             // every product issued above has finished when this one fires
      dead = false;
      wait(kDone, 0);
    } else if (warp == 9 && lane == 0) {
      // ---------------------------------------------------------------- bulk copies of the K and V tiles
      int issued = 0;
      for (int j = 0; j < n_b; ++j) {
        const int st = j & 1;
        const uint32_t ph_prev = (uint32_t)((j >> 1) - 1) & 1u;
        if (j >= 2 && !wait(kKEmpty + st, ph_prev)) break;
        // (test hook: the first copy's barrier can be armed for more bytes than arrive, so that it never completes)
        mbar_expect_tx(bar(kKFull + st), kTileBytes + (j == 0 ? debug_extra_tx : 0u));
        bulk_copy(smem_u32(Ks + st * kTileBytes), ktg + (size_t)j * kTileBytes, kTileBytes, bar(kKFull + st));
        if (j >= 2 && !wait(kVEmpty + st, ph_prev)) {   // the K copy above is awaited below like the others
          issued = j + 1;
          mbar_expect_tx(bar(kVFull + st), 0);
          break;
        }
        mbar_expect_tx(bar(kVFull + st), kTileBytes);
        bulk_copy(smem_u32(Vs + st * kTileBytes), vtg + (size_t)j * kTileBytes, kTileBytes, bar(kVFull + st));
        issued = j + 1;
      }
      // no copy may be in flight when the CTA ends: the last copy into each stage has landed once its barrier's phase is over
      for (int j = max(0, issued - 2); j < issued; ++j) {
        dead = false;                                    // every one of these waits is made, whatever the others did
        wait(kKFull + (j & 1), (uint32_t)(j >> 1) & 1u);
        dead = false;
        wait(kVFull + (j & 1), (uint32_t)(j >> 1) & 1u);
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;" ::: "memory");
    // ------------------------------------------------------------------ softmax and output rows
    const int g = warp >> 2, row = tid & 127;
    const uint32_t lane_base = tbase + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t s_addr = lane_base + 128 * g, t_addr = lane_base + 256 + 128 * g;
    const int n = g == 0 ? n_a : n_b;
    const int pos = qt * kQRows + g * kTile + row;     // this thread's query position
    float o[kD];
#pragma unroll
    for (int d = 0; d < kD; ++d) o[d] = 0.f;
    float m_run = -INFINITY, l_run = 0.f, alpha = 0.f;
#pragma unroll 1
    for (int j = 0; j < n; ++j) {
      if (!wait(kSFull + g, (uint32_t)j & 1u)) break;
      tc_fence_after();
      if ((j + 1) * kTile - 1 > qt * kQRows + g * kTile)      // the tile reaches past the group's first row
        softmax_tile<true>(s_addr, pos - j * kTile + 1, scale_log2e, m_run, l_run, alpha);
      else
        softmax_tile<false>(s_addr, kTile, scale_log2e, m_run, l_run, alpha);
      tc_fence_before();
      mbar_arrive(bar(kPReady + g));
      if (!wait(kTFull + g, (uint32_t)j & 1u)) break;
      tc_fence_after();
      {
        uint32_t xa[32], xb[32];
        tmem_ld32_issue(t_addr, xa);
        tmem_wait_ld32(xa);
        tmem_ld32_issue(t_addr + 32, xb);
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = fmaf(o[i], alpha, __uint_as_float(xa[i]));
        tmem_wait_ld32(xb);
        tmem_ld32_issue(t_addr + 64, xa);
#pragma unroll
        for (int i = 0; i < 32; ++i) o[32 + i] = fmaf(o[32 + i], alpha, __uint_as_float(xb[i]));
        tmem_wait_ld32(xa);
        tmem_ld32_issue(t_addr + 96, xb);
#pragma unroll
        for (int i = 0; i < 32; ++i) o[64 + i] = fmaf(o[64 + i], alpha, __uint_as_float(xa[i]));
        tmem_wait_ld32(xb);
        // T is in registers: the tensor core may overwrite it while the last chunk is folded in
        tc_fence_before();
        mbar_arrive(bar(kTFree + g));
#pragma unroll
        for (int i = 0; i < 32; ++i) o[96 + i] = fmaf(o[96 + i], alpha, __uint_as_float(xb[i]));
      }
    }
    if (pos < L && !dead) {
      const float inv = 1.f / l_run;
      float4* dst = reinterpret_cast<float4*>(out + ((size_t)(b * Hq + h) * L + pos) * kD);
#pragma unroll
      for (int d = 0; d < kD; d += 4) dst[d >> 2] = make_float4(o[d] * inv, o[d + 1] * inv, o[d + 2] * inv, o[d + 3] * inv);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(512) : "memory");
}

}  // namespace

cudaError_t prefill_attention_setup() {
  return cudaFuncSetAttribute(prefill_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
}

size_t prefill_scratch_bytes(int B, int Hkv, int L) {
  return (size_t)2 * B * Hkv * ((L + kTile - 1) / kTile) * kTileBytes;
}

cudaError_t launch_prefill_attention(const void* q, const void* k, const void* v, float* out, void* scratch, int B, int Hq,
                                     int Hkv, int L, float scale, uint32_t* status, uint32_t max_polls, uint32_t debug_extra_tx,
                                     cudaStream_t stream) {
  const int n_tiles = (L + kTile - 1) / kTile, n_qtiles = (L + kQRows - 1) / kQRows;
  unsigned char* kt = static_cast<unsigned char*>(scratch);
  unsigned char* vt = kt + (size_t)B * Hkv * n_tiles * kTileBytes;
  prefill_pack_kernel<<<dim3((unsigned)n_tiles, (unsigned)(B * Hkv)), 256, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v), kt, vt, L, n_tiles);
  prefill_attention_kernel<<<(unsigned)(n_qtiles * B * Hq), kThreads, kSmem, stream>>>(
      static_cast<const __nv_bfloat16*>(q), kt, vt, out, B * Hq, Hq, Hkv, L, n_tiles, n_qtiles,
      scale * 1.4426950408889634f, status, max_polls ? max_polls : kPolls, debug_extra_tx);
  return cudaGetLastError();
}

}  // namespace mixkvq
