// Fused split-K GQA decode attention over the tile layout (blocks of R = 128 tokens) on the tcgen05 tensor cores
// (Eq. 1 with the dequantization of Eq. 3 applied on the fly).
//
// One CTA per SM, three independent worker groups of 128 threads, each walking its own contiguous run of
// 128-token blocks (a split).  For a block, thread j of the group
//   1. expands the 2-bit key codes of token j (32 contiguous bytes) into fp16 *subnormals* c * 2^(p-24) with one
//      logic op per two codes and stores them to tensor memory as row j of the A operand (tcgen05.st);
//   2. reads row j of S = K~ q'^T from tensor memory (tcgen05.ld), does the online softmax in the log2 domain
//      (block maximum by redux.sync.max.f32 + one group barrier), writes p * s_v as row j of the P operand in
//      shared memory and keeps sum p and sum p * z_v in registers;
//   3. expands the 2-bit value codes of channel j the same way as row j of V~^T.
// A control warp per group stages blocks with 1-D bulk (TMA) copies, folds the per-channel key scales into the
// query (B operand q * s * 2^(4-p) in shared memory, so the A operand needs no multiply), computes the key
// zero-point term q . z per key group with one small mma.sync chain, and issues the tcgen05.mma instructions
// (M = 128 tokens or channels, N = 8 heads x groups, A from tensor memory, B from shared memory, fp32
// accumulators in tensor memory).  Promoted (BF16) channels and the UINT4 high plane are extra K columns.
// The residual window is handled by the mma.sync kernel; a combine kernel merges all partials.
#include "common.cuh"

namespace mixkvq {

cudaError_t launch_combine2(const float* ws, float* out, int g, int Hkv, int Hq, int S, int n1, long long units1,
                            int slot2, int n2, long long units2, cudaStream_t stream);
int attention_ws_grid(const LayerView& lv, int n_sms);
long long attention_ws_positions(const LayerView& lv);

namespace {

constexpr int kWG = 3;                       // worker groups per CTA
constexpr int kStages = 3;                   // staged blocks per group
constexpr int kThreads = 512;                // 12 worker warps, 3 control warps, 1 idle warp
constexpr int kStageExtras = 64 + 4 * 512;   // extras that travel with the block: header + up to 4 word rows
constexpr int kPass0Extra = 1;               // extra k-steps beside the 8 base k-steps (A columns 64..71)
constexpr int kPassSteps = 9;                // k-steps of a later pass (A columns 0..71)
constexpr int kBqSBO = 18 * 128;             // B operand of q.K^T: 144 rows = 18 chunks of 8, 128 B each
constexpr int kColsPerWG = 168;              // tensor-memory columns: A 0..71, S 72..135 (high | low part), O 136..167
constexpr int kColS = 72, kColO = 136;
constexpr uint32_t kSpinLimit = 1u << 22;

template <int G>
struct Geo {
  static constexpr int NG = 128 / G, VG = 128 / G;
  static constexpr int NQ = NG * 16;    // columns (part, key group, head): the fp16 high and low parts of q * s
  static constexpr int NV = VG * 8 < 16 ? 16 : VG * 8;
  static constexpr int kBase = NG * 512 + 8192 + 512 * VG;
  static constexpr int kStage = (kBase + kStageExtras + 127) / 128 * 128;
  // per-group shared memory map
  static constexpr int oStages = 0;
  static constexpr int oBq = oStages + kStages * kStage;
  static constexpr int oPb = oBq + (NQ / 8) * kBqSBO;
  static constexpr int oQh = oPb + (NV / 8) * 2048;     // [8][128] half: query of the current stream
  static constexpr int oQt = oQh + 2048;                // [16 chunks][8 heads][8] half: the same query, chunk-major
  static constexpr int oSh = oQt + 2048;                // [NG][128] half: key scales * 2^(4-p)
  static constexpr int oZh = oSh + NG * 256;            // [NG][128] half: key zero-points
  static constexpr int oZq = oZh + NG * 256;            // [NG][8] float: q . z * scale * log2(e)
  static constexpr int oMred = oZq + 128;               // [4][8] float
  static constexpr int oRed = oMred + 128;              // [4][40] float
  static constexpr int oEnt = oRed + 640;               // [kStages] uint2 table entries, dead flag at +32
  static constexpr int oBars = oEnt + 64;               // 12 mbarriers
  static constexpr int kGroup = (oBars + 128 + 127) / 128 * 128;
  static constexpr int kSmem = kWG * kGroup + 128;
};

// bit position p of the 2-bit field number f (0..7) of a 16-bit half after the expansion below
__host__ __device__ constexpr int field_pos(int f) { return f < 5 ? 2 * f : 2 * (f - 5); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t hfma2_u(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t hmul2_u(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// ---- mbarrier / bulk copy
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  After one wait of the group gave up, every later wait of the group returns at once, so the
// kernel always terminates; the results are then invalid and the status word says so.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* dead, uint32_t* status) {
  if (*dead) return;
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return;
  *dead = 1u;
  atomicOr(status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
}
__device__ __forceinline__ void bar_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- tcgen05
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};" ::
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};" ::"r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
// shared-memory matrix descriptor: no swizzle, sm_100 version field
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46);
}
// instruction descriptor: fp32 accumulate, fp16 A and B, A K-major (tensor memory), B K-major (0) or MN-major (1)
__device__ __forceinline__ constexpr uint32_t make_idesc(int M, int N, int b_mn_major) {
  return (1u << 4) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float redux_max(float x) {
  float m;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(m) : "f"(x));
  return m;
}

// One 32-bit word = 16 two-bit codes (number 2f+e at bit 16e + 2f)  ->  8 registers of two fp16 subnormals:
// register f holds codes (2f, 2f+1) as c * 2^(field_pos(f) - 24).
__device__ __forceinline__ void expand_word(uint32_t x, uint32_t* a) {
  const uint32_t y = x >> 10;
  a[0] = x & 0x00030003u;
  a[1] = x & 0x000C000Cu;
  a[2] = x & 0x00300030u;
  a[3] = x & 0x00C000C0u;
  a[4] = x & 0x03000300u;
  a[5] = y & 0x00030003u;
  a[6] = y & 0x000C000Cu;
  a[7] = y & 0x00300030u;
}
__device__ __forceinline__ void expand4(const uint4 w, uint32_t (&a)[32]) {
  expand_word(w.x, a);
  expand_word(w.y, a + 8);
  expand_word(w.z, a + 16);
  expand_word(w.w, a + 24);
}

struct Bars {   // byte offsets inside the group's barrier area
  static constexpr int full = 0, empty = 8 * kStages, a_ready = 16 * kStages, s_done = a_ready + 8, ctl_ready = a_ready + 16,
                       p_ready = a_ready + 24, o_done = a_ready + 32, max_ready = a_ready + 40;
};
__device__ __forceinline__ bool elect_one() {
  uint32_t p;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(p));
  return p != 0;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int G>
__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(LayerView lv, const __nv_bfloat16* __restrict__ q, float scale_log2e, float* __restrict__ ws) {
  using L = Geo<G>;
  constexpr int NG = L::NG, VG = L::VG;
  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // warp-uniform
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kWG * L::kGroup);

  // ---- set-up: tensor memory, barriers
  if (warp == 12) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (threadIdx.x < kWG) {
    unsigned char* gs = smem + threadIdx.x * L::kGroup;
    const uint32_t bars = smem_u32(gs + L::oBars);
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bars + Bars::full + 8 * i, 1);
      mbar_init(bars + Bars::empty + 8 * i, 4);
    }
    mbar_init(bars + Bars::a_ready, 4);
    mbar_init(bars + Bars::s_done, 1);
    mbar_init(bars + Bars::ctl_ready, 1);
    mbar_init(bars + Bars::p_ready, 4);
    mbar_init(bars + Bars::o_done, 1);
    mbar_init(bars + Bars::max_ready, 4);
    *reinterpret_cast<volatile uint32_t*>(gs + L::oEnt + 32) = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // zero the P operand once: with one value group only columns 0..7 of its 16 are ever written
  for (int i = threadIdx.x; i < kWG * (L::NV / 8) * 2048 / 16; i += kThreads) {
    const int gidx = i / ((L::NV / 8) * 128), rem = i % ((L::NV / 8) * 128);
    reinterpret_cast<uint4*>(smem + gidx * L::kGroup + L::oPb)[rem] = make_uint4(0, 0, 0, 0);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = *tmem_slot;

  const int S = lv.B * lv.Hkv, nblk = lv.n_blocks;
  const long long total = (long long)S * nblk;
  const int nwg = (int)min((long long)gridDim.x * kWG, total);     // groups that get work (each at least one block)

  if (warp < 12) {
    // =============================================================== worker groups
    const int wg = warp >> 2, quad = warp & 3, j = threadIdx.x & 127;
    unsigned char* gs = smem + wg * L::kGroup;
    const uint32_t bars = smem_u32(gs + L::oBars);
    volatile uint32_t* dead = reinterpret_cast<volatile uint32_t*>(gs + L::oEnt + 32);
    const int wgg = blockIdx.x * kWG + wg;
    const long long xb = wgg < nwg ? split_begin(total, nwg, wgg) : 0, xe = wgg < nwg ? split_begin(total, nwg, wgg + 1) : 0;
    const uint32_t tA = tbase + (uint32_t)(kColsPerWG * wg) + ((uint32_t)(quad * 32) << 16);
    const int grp = (quad * 32) / G;            // key group of this thread's token
    const int vgc = (quad * 32) / G;            // value group of this thread's channel
    const float sc20 = scale_log2e * 1048576.0f;      // the tensor-core logits carry the factor 2^-20 of the subnormal codes
    const float pscale = (float)(1 << 4) / (float)(1 << field_pos((j & 15) >> 1));   // 2^(4 - p) of token j
    float* zqS = reinterpret_cast<float*>(gs + L::oZq);
    float* mredS = reinterpret_cast<float*>(gs + L::oMred);
    float* redS = reinterpret_cast<float*>(gs + L::oRed);
    const uint2* entS = reinterpret_cast<const uint2*>(gs + L::oEnt);
    const __half* qhS = reinterpret_cast<const __half*>(gs + L::oQh);

    float mref[8], accL[8], accZ[VG][8];
    int cur_s = -1, i = 0;
    uint32_t npass = 0;
    bool first = true;

    auto finalize = [&](int s, int i_last) {
      mbar_wait(bars + Bars::o_done, (uint32_t)i_last & 1u, dead, lv.status);
      tc_fence_after();
      // sums over the 128 threads of the group
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        float v = accL[h];
#pragma unroll
        for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0) redS[quad * 40 + h] = v;
#pragma unroll
        for (int vg = 0; vg < VG; ++vg) {
          float z = accZ[vg][h];
#pragma unroll
          for (int off = 16; off; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
          if (lane == 0) redS[quad * 40 + 8 + vg * 8 + h] = z;
        }
      }
      bar_sync(1 + wg, 128);
      uint32_t ov[8];
      tmem_ld8(tA + kColO + 8 * vgc, ov);
      tc_wait_ld();
      float* part = ws + (size_t)(wgg + s) * kPartialFloats;
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        const float zsum = redS[8 + vgc * 8 + h] + redS[40 + 8 + vgc * 8 + h] + redS[80 + 8 + vgc * 8 + h] +
                           redS[120 + 8 + vgc * 8 + h];
        part[h * 130 + 2 + j] = __uint_as_float(ov[h]) * 1048576.0f + zsum;
        if (j == 0) {
          part[h * 130] = mref[h];
          part[h * 130 + 1] = redS[h] + redS[40 + h] + redS[80 + h] + redS[120 + h];
        }
      }
      tc_fence_before();
      bar_sync(1 + wg, 128);
    };

    for (long long x = xb; x < xe; ++x, ++i) {
      const int s = (int)(x / nblk);
      if (s != cur_s) {
        if (cur_s >= 0) finalize(cur_s, i - 1);
        cur_s = s;
        first = true;
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          mref[h] = -INFINITY;
          accL[h] = 0.f;
#pragma unroll
          for (int vg = 0; vg < VG; ++vg) accZ[vg][h] = 0.f;
        }
      }
      const int stage = i % kStages;
      mbar_wait(bars + Bars::full + 8 * stage, (uint32_t)(i / kStages) & 1u, dead, lv.status);
      const unsigned char* st = gs + L::oStages + stage * L::kStage;
      const uint2 ent = entS[stage];
      const int n16 = ent.y & 0xFF, n4 = (ent.y >> 8) & 0xFF;
      const int n16p = (n16 + 1) >> 1, n4w = (n4 + 15) >> 4, KP = (n16p + 7) >> 3, E = KP + n4w;
      const bool fits = (n16p + n4w) <= 4;
      const unsigned char* exh = fits ? st + L::kBase
                                      : reinterpret_cast<const unsigned char*>(lv.extras) + (size_t)s * lv.extras_stride +
                                            (size_t)ent.x * 16;
      const uint32_t* exb = reinterpret_cast<const uint32_t*>(exh + tile_extras_header_bytes(n16, n4));
      const uint32_t* kmetaS = reinterpret_cast<const uint32_t*>(st);       // [NG][128] {s, z}

      // one extra k-step (8 columns): promoted pairs as fp16 * 2^-10, or one word of the UINT4 high plane
      auto extra_step = [&](int e, uint32_t taddr) {
        uint32_t a8[8];
        if (e < KP) {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const int p = 8 * e + c;
            const uint32_t w = (p < n16p) ? exb[p * 128 + j] : 0u;
            a8[c] = pack_half2(bf_lo(w) * 0.0009765625f, bf_hi(w) * 0.0009765625f);
          }
        } else {
          expand_word(exb[(n16p + (e - KP)) * 128 + j], a8);
        }
        tmem_st8(taddr, a8);
      };

      // rows of the B operand (q * s, fp16 high and low parts) for extra k-steps [e0, e1), placed from row `row0`:
      // thread = (chunk of 8 rows, head), all key groups
      auto build_extra_rows = [&](int e0, int e1, int row0) {
        const int hq = j & 7;
        for (int c8 = j >> 3; c8 < 2 * (e1 - e0); c8 += 16) {
          const int e = e0 + (c8 >> 1), half = c8 & 1;
          float qv[8], wgt[8];
          int chn[8];
#pragma unroll
          for (int r8 = 0; r8 < 8; ++r8) {
            const int r16 = 8 * half + r8;                          // row inside the k-step
            int ch;
            if (e < KP) {
              ch = exh[16 * e + r16];                               // promoted: list position 16e + r16
              wgt[r8] = 0.0009765625f;
            } else {
              ch = exh[2 * n16p + 16 * (e - KP) + r16];             // UINT4 high plane: list position 16(e-KP) + r16
              wgt[r8] = 4.0f * (float)(1 << 4) / (float)(1 << field_pos(r16 >> 1));
            }
            const bool ok = (e < KP) ? (16 * e + r16 < 2 * n16p && ch < 128) : (ch < 128);
            chn[r8] = ok ? ch : -1;
            qv[r8] = ok ? __half2float(qhS[hq * kD + ch]) : 0.f;
          }
#pragma unroll
          for (int kg = 0; kg < NG; ++kg) {
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int r2 = 0; r2 < 4; ++r2) {
              float v[2];
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                const int r8 = 2 * r2 + u;
                float sc = 1.0f;
                if (e >= KP && chn[r8] >= 0) sc = bf_lo(kmetaS[kg * 128 + chn[r8]]);
                v[u] = qv[r8] * wgt[r8] * sc;
              }
              hi[r2] = pack_half2(v[0], v[1]);
              const float2 back = __half22float2(*reinterpret_cast<const __half2*>(&hi[r2]));
              lo[r2] = pack_half2(v[0] - back.x, v[1] - back.y);
            }
            *reinterpret_cast<uint4*>(gs + L::oBq + kg * kBqSBO + (row0 / 8 + c8) * 128 + hq * 16) =
                make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(gs + L::oBq + (NG + kg) * kBqSBO + (row0 / 8 + c8) * 128 + hq * 16) =
                make_uint4(lo[0], lo[1], lo[2], lo[3]);
          }
        }
      };

      if (i > 0) mbar_wait(bars + Bars::o_done, (uint32_t)(i - 1) & 1u, dead, lv.status);   // A columns free again
      tc_fence_after();
      // ---- keys: row j of the A operand
      const int P = 1 + (E > kPass0Extra ? (E - kPass0Extra + kPassSteps - 1) / kPassSteps : 0);
      for (int p = 0; p < P; ++p) {
        if (p == 0) {
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t a[32];
            expand4(*reinterpret_cast<const uint4*>(st + NG * 512 + hh * 2048 + j * 16), a);
            tmem_st32(tA + 32 * hh, a);
          }
          const int e1 = min(E, kPass0Extra);
          for (int e = 0; e < e1; ++e) extra_step(e, tA + 64 + 8 * e);
          // B operand, base rows: q[h][d] * s[kg][d] * 2^(4 - p(d)) as an exact fp16 pair (product, remainder);
          // thread = (chunk of 8 channels, head), all key groups.  The scale table comes from the control warp.
          mbar_wait(bars + Bars::ctl_ready, (uint32_t)i & 1u, dead, lv.status);
          {
            const int hq = j & 7, kc = j >> 3;
            const uint4 q8 = *reinterpret_cast<const uint4*>(gs + L::oQt + j * 16);
#pragma unroll
            for (int kg = 0; kg < NG; ++kg) {
              const uint4 s8 = *reinterpret_cast<const uint4*>(gs + L::oSh + (kg * kD + 8 * kc) * 2);
              const uint4 hi = make_uint4(hmul2_u(q8.x, s8.x), hmul2_u(q8.y, s8.y), hmul2_u(q8.z, s8.z), hmul2_u(q8.w, s8.w));
              const uint4 lo = make_uint4(hfma2_u(q8.x, s8.x, hi.x ^ 0x80008000u), hfma2_u(q8.y, s8.y, hi.y ^ 0x80008000u),
                                          hfma2_u(q8.z, s8.z, hi.z ^ 0x80008000u), hfma2_u(q8.w, s8.w, hi.w ^ 0x80008000u));
              *reinterpret_cast<uint4*>(gs + L::oBq + kg * kBqSBO + kc * 128 + hq * 16) = hi;
              *reinterpret_cast<uint4*>(gs + L::oBq + (NG + kg) * kBqSBO + kc * 128 + hq * 16) = lo;
            }
          }
          build_extra_rows(0, e1, 128);
        } else {
          mbar_wait(bars + Bars::s_done, (npass - 1) & 1u, dead, lv.status);      // A columns and B rows free again
          tc_fence_after();
          const int e0 = kPass0Extra + kPassSteps * (p - 1), e1 = min(E, e0 + kPassSteps);
          for (int e = e0; e < e1; ++e) extra_step(e, tA + 8 * (e - e0));
          build_extra_rows(e0, e1, 0);
        }
        tc_wait_st();
        tc_fence_before();
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + Bars::a_ready);
        ++npass;
      }

      // ---- softmax of row j
      mbar_wait(bars + Bars::s_done, (npass - 1) & 1u, dead, lv.status);
      tc_fence_after();
      float xv[8];
      {
        uint32_t sv[8], sl[8];
        tmem_ld8(tA + kColS + 8 * grp, sv);
        tmem_ld8(tA + kColS + 8 * (NG + grp), sl);
        tc_wait_ld();
        const float4 z0 = *reinterpret_cast<const float4*>(zqS + grp * 8), z1 = *reinterpret_cast<const float4*>(zqS + grp * 8 + 4);
        const float zq[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
#pragma unroll
        for (int h = 0; h < 8; ++h) xv[h] = fmaf(__uint_as_float(sv[h]) + __uint_as_float(sl[h]), sc20, zq[h]);
      }
      {
        float bm[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) bm[h] = redux_max(xv[h]);
        if (lane == 0) {
          *reinterpret_cast<float4*>(mredS + quad * 8) = make_float4(bm[0], bm[1], bm[2], bm[3]);
          *reinterpret_cast<float4*>(mredS + quad * 8 + 4) = make_float4(bm[4], bm[5], bm[6], bm[7]);
          mbar_arrive(bars + Bars::max_ready);
        }
        // values while the other warps' maxima arrive: row j (= channel j) of V~^T (the key rows are consumed)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t a[32];
          expand4(*reinterpret_cast<const uint4*>(st + NG * 512 + 4096 + hh * 2048 + j * 16), a);
          tmem_st32(tA + 32 * hh, a);
        }
        mbar_wait(bars + Bars::max_ready, (uint32_t)i & 1u, dead, lv.status);
        bool grow = false;
        float mn[8];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const float4 m0 = *reinterpret_cast<const float4*>(mredS + 4 * hf), m1 = *reinterpret_cast<const float4*>(mredS + 8 + 4 * hf);
          const float4 m2 = *reinterpret_cast<const float4*>(mredS + 16 + 4 * hf), m3 = *reinterpret_cast<const float4*>(mredS + 24 + 4 * hf);
          mn[4 * hf + 0] = fmaxf(fmaxf(m0.x, m1.x), fmaxf(m2.x, m3.x));
          mn[4 * hf + 1] = fmaxf(fmaxf(m0.y, m1.y), fmaxf(m2.y, m3.y));
          mn[4 * hf + 2] = fmaxf(fmaxf(m0.z, m1.z), fmaxf(m2.z, m3.z));
          mn[4 * hf + 3] = fmaxf(fmaxf(m0.w, m1.w), fmaxf(m2.w, m3.w));
        }
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          mn[h] = fmaxf(mref[h], mn[h]);
          grow |= mn[h] > mref[h];
        }
        if (grow) {
          if (!first) {
            float al[8];
#pragma unroll
            for (int h = 0; h < 8; ++h) {
              al[h] = ex2(mref[h] - mn[h]);
              accL[h] *= al[h];
#pragma unroll
              for (int vg = 0; vg < VG; ++vg) accZ[vg][h] *= al[h];
            }
            uint32_t ov[8];
            tmem_ld8(tA + kColO + 8 * vgc, ov);
            tc_wait_ld();
#pragma unroll
            for (int h = 0; h < 8; ++h) ov[h] = __float_as_uint(__uint_as_float(ov[h]) * al[h]);
            tmem_st8(tA + kColO + 8 * vgc, ov);
          }
#pragma unroll
          for (int h = 0; h < 8; ++h) mref[h] = mn[h];
        }
      }
      {
        float pv[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          pv[h] = ex2(xv[h] - mref[h]);
          accL[h] += pv[h];
        }
        const uint32_t* vmeta = reinterpret_cast<const uint32_t*>(st + NG * 512 + 8192) + j * VG;
#pragma unroll
        for (int vg = 0; vg < VG; ++vg) {
          const uint32_t mz = vmeta[vg];
          const float sv = bf_lo(mz), zv = bf_hi(mz);
#pragma unroll
          for (int h = 0; h < 8; ++h) accZ[vg][h] = fmaf(pv[h], zv, accZ[vg][h]);
          const float sp = sv * pscale;                                    // products in fp32, rounded to fp16 once
          *reinterpret_cast<uint4*>(gs + L::oPb + vg * 2048 + j * 16) =
              make_uint4(pack_half2(pv[0] * sp, pv[1] * sp), pack_half2(pv[2] * sp, pv[3] * sp),
                         pack_half2(pv[4] * sp, pv[5] * sp), pack_half2(pv[6] * sp, pv[7] * sp));
        }
      }
      tc_wait_st();
      tc_fence_before();
      fence_async_smem();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bars + Bars::p_ready);
        mbar_arrive(bars + Bars::empty + 8 * stage);
      }
      first = false;
    }
    if (cur_s >= 0) finalize(cur_s, i - 1);
  } else if (warp < 12 + kWG) {
    // =============================================================== control warps
    const int wg = warp - 12;
    unsigned char* gs = smem + wg * L::kGroup;
    const uint32_t bars = smem_u32(gs + L::oBars);
    volatile uint32_t* dead = reinterpret_cast<volatile uint32_t*>(gs + L::oEnt + 32);
    const int wgg = blockIdx.x * kWG + wg;
    const long long xb = wgg < nwg ? split_begin(total, nwg, wgg) : 0, xe = wgg < nwg ? split_begin(total, nwg, wgg + 1) : 0;
    const int nb = (int)(xe - xb);
    const uint32_t tW = tbase + (uint32_t)(kColsPerWG * wg);
    __half* qh = reinterpret_cast<__half*>(gs + L::oQh);
    __half* sh = reinterpret_cast<__half*>(gs + L::oSh);
    __half* zh = reinterpret_cast<__half*>(gs + L::oZh);
    float* zqS = reinterpret_cast<float*>(gs + L::oZq);
    uint2* entS = reinterpret_cast<uint2*>(gs + L::oEnt);
    const uint32_t idesc1 = make_idesc(128, L::NQ, 0), idesc2 = make_idesc(128, L::NV, 1);
    const uint32_t bq_addr = smem_u32(gs + L::oBq), pb_addr = smem_u32(gs + L::oPb);

    // lane 0: stage block x as the group's block number i
    auto entry_of = [&](long long x) -> uint2 {
      const int s = (int)(x / nblk), bi = (int)(x - (long long)s * nblk);
      return *reinterpret_cast<const uint2*>(lv.table + (size_t)s * lv.table_stride + (size_t)bi * 8);
    };
    auto issue = [&](long long x, int i, const uint2 ent) {
      const int s = (int)(x / nblk), bi = (int)(x - (long long)s * nblk);
      const int n16 = ent.y & 0xFF, n4 = (ent.y >> 8) & 0xFF;
      const int n16p = (n16 + 1) >> 1, n4w = (n4 + 15) >> 4;
      const bool fits = (n16p + n4w) <= 4;
      const uint32_t exbytes = fits ? tile_extras_header_bytes(n16, n4) + tile_extras_body_bytes(n16, n4) : 0u;
      const int stage = i % kStages;
      const uint32_t bar = bars + Bars::full + 8 * stage;
      const uint32_t dst = smem_u32(gs + L::oStages + stage * L::kStage);
      entS[stage] = ent;
      mbar_expect_tx(bar, (uint32_t)L::kBase + exbytes);
      bulk_g2s(dst, lv.base + (size_t)s * lv.base_stride + (size_t)bi * lv.base_bytes, (uint32_t)L::kBase, bar);
      if (exbytes) bulk_g2s(dst + L::kBase, lv.extras + (size_t)s * lv.extras_stride + (size_t)ent.x * 16, exbytes, bar);
    };
    if (lane == 0)
      for (int k = 0; k < min(kStages, nb); ++k) issue(xb + k, k, entry_of(xb + k));

    int cur_s = -1;
    uint32_t npass = 0;
    bool first = true;
    // table entries are fetched two blocks before the copy that needs them, so their latency is never waited for
    uint2 ent_refill = make_uint2(0u, 0u);
    if (lane == 0 && kStages < nb) ent_refill = entry_of(xb + kStages);
    for (int i = 0; i < nb; ++i) {
      const long long x = xb + i;
      const int s = (int)(x / nblk);
      const int stage = i % kStages;
      uint2 ent_ahead = make_uint2(0u, 0u);         // table entry of the block that refills the next stage
      if (lane == 0 && i + 1 + kStages < nb) ent_ahead = entry_of(x + 1 + kStages);
      if (s != cur_s) {
        // query of the new stream as fp16, heads >= g zero.  The previous block's tensor-core reads of the B
        // operand are complete (its softmax ran), and only this warp reads qh.
        cur_s = s;
        first = true;
        const int b = s / lv.Hkv, hk = s % lv.Hkv;
        __half* qt = reinterpret_cast<__half*>(gs + L::oQt);
        for (int t = lane; t < 8 * kD; t += 32) {
          const int h = t >> 7, d = t & 127;
          const __half v = (h < lv.g) ? __float2half_rn(__bfloat162float(q[((size_t)b * lv.Hq + hk * lv.g + h) * kD + d]))
                                      : __float2half_rn(0.f);
          qh[t] = v;
          qt[((d >> 3) * 8 + h) * 8 + (d & 7)] = v;
        }
        __syncwarp();
      }
      mbar_wait(bars + Bars::full + 8 * stage, (uint32_t)(i / kStages) & 1u, dead, lv.status);
      const unsigned char* st = gs + L::oStages + stage * L::kStage;
      const uint2 ent = entS[stage];
      const int n16 = ent.y & 0xFF, n4 = (ent.y >> 8) & 0xFF;
      const int n16p = (n16 + 1) >> 1, n4w = (n4 + 15) >> 4, KP = (n16p + 7) >> 3, E = KP + n4w;
      const uint32_t* kmeta = reinterpret_cast<const uint32_t*>(st);       // [NG][128] {s, z}

      // key scales (times the field weight of the channel's code) and zero-points as fp16 tables
      for (int t = lane; t < NG * 64; t += 32) {
        const int d = (2 * t) & 127;
        const uint2 m2 = *reinterpret_cast<const uint2*>(kmeta + 2 * t);
        const float mult = (float)(1 << 4) / (float)(1 << field_pos((d & 15) >> 1));
        reinterpret_cast<uint32_t*>(sh)[t] = pack_half2(bf_lo(m2.x) * mult, bf_lo(m2.y) * mult);
        reinterpret_cast<uint32_t*>(zh)[t] = pack_half2(bf_hi(m2.x), bf_hi(m2.y));
      }
      __syncwarp();

      // zero-point term of the logits: zq[kg][h] = sum_d q[h][d] z[kg][d], times scale * log2(e)
      {
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        const int r = lane >> 2, t = lane & 3;
#pragma unroll
        for (int kt = 0; kt < 8; ++kt) {
          uint32_t a0 = 0u, a2 = 0u;
          if (r < NG) {
            a0 = *reinterpret_cast<const uint32_t*>(zh + r * kD + 16 * kt + 2 * t);
            a2 = *reinterpret_cast<const uint32_t*>(zh + r * kD + 16 * kt + 8 + 2 * t);
          }
          const uint32_t b0 = *reinterpret_cast<const uint32_t*>(qh + r * kD + 16 * kt + 2 * t);
          const uint32_t b1 = *reinterpret_cast<const uint32_t*>(qh + r * kD + 16 * kt + 8 + 2 * t);
          mma_f16(c, a0, 0u, a2, 0u, b0, b1);
        }
        if (r < NG) {
          zqS[r * 8 + 2 * t] = c[0] * scale_log2e;
          zqS[r * 8 + 2 * t + 1] = c[1] * scale_log2e;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + Bars::ctl_ready);     // tables and zq of this block are in place

      // ---- q . K~^T: one group of tcgen05.mma per pass, issued by one elected lane from warp-uniform operands
      const int P = 1 + (E > kPass0Extra ? (E - kPass0Extra + kPassSteps - 1) / kPassSteps : 0);
      const uint64_t bq_desc = make_desc(bq_addr, 128, kBqSBO);
      for (int p = 0; p < P; ++p) {
        const int n_steps = (p == 0) ? 8 + min(E, kPass0Extra)
                                     : min(E, kPass0Extra + kPassSteps * p) - (kPass0Extra + kPassSteps * (p - 1));
        mbar_wait(bars + Bars::a_ready, npass & 1u, dead, lv.status);
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < kPassSteps; ++ks)
            if (ks < n_steps) tc_mma(tW + kColS, tW + 8 * ks, bq_desc + (uint64_t)(ks * 16), idesc1, (p > 0 || ks > 0) ? 1u : 0u);
          tc_commit(bars + Bars::s_done);
        }
        __syncwarp();
        ++npass;
      }

      // ---- P . V~ once the group's P rows and value rows are in place
      mbar_wait(bars + Bars::p_ready, (uint32_t)i & 1u, dead, lv.status);
      tc_fence_after();
      if (elect_one()) {
        const uint64_t pb_desc = make_desc(pb_addr, 128, 2048);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          tc_mma(tW + kColO, tW + 8 * ks, pb_desc + (uint64_t)(ks * 16), idesc2, (first && ks == 0) ? 0u : 1u);
        tc_commit(bars + Bars::o_done);
      }
      __syncwarp();
      first = false;
      if (i + kStages < nb) {
        mbar_wait(bars + Bars::empty + 8 * stage, (uint32_t)(i / kStages) & 1u, dead, lv.status);
        if (lane == 0) issue(x + kStages, i + kStages, ent_refill);
        __syncwarp();
      }
      ent_refill = ent_ahead;
    }
    // the group's last commit must have landed before tensor memory is released
    if (nb > 0) mbar_wait(bars + Bars::o_done, (uint32_t)(nb - 1) & 1u, dead, lv.status);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 12) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(512) : "memory");
}

template <int G>
cudaError_t launch_g(const LayerView& lv, const void* q, float scale, float* ws, int grid, cudaStream_t stream) {
  attention_tc_kernel<G><<<grid, kThreads, Geo<G>::kSmem, stream>>>(lv, static_cast<const __nv_bfloat16*>(q),
                                                                     scale * 1.4426950408889634f, ws);
  return cudaGetLastError();
}

}  // namespace

cudaError_t attention_tc_setup() {
  cudaError_t e;
  e = cudaFuncSetAttribute(attention_tc_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<32>::kSmem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attention_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<64>::kSmem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attention_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<128>::kSmem);
}

// Packed blocks on the tcgen05 kernel, residual window on the mma.sync kernel (its partials follow the first
// kernel's in the workspace), then one combine over both sets of partials.
cudaError_t launch_attention_tc(const LayerView& lv, const void* q, float* out, float scale, float* ws, int n_sms,
                                cudaStream_t stream, int* launches) {
  *launches = 0;
  if (lv.n_blocks == 0) return launch_attention_ws(lv, q, out, scale, ws, n_sms, stream, launches);
  const int S = lv.B * lv.Hkv;
  const long long total = (long long)S * lv.n_blocks;
  int grid = (int)min((long long)min(n_sms, kMaxCtas / (2 * kWG)), (total + kWG - 1) / kWG);
  if (grid < 1) grid = 1;
  cudaError_t e;
  if (lv.G == 32) e = launch_g<32>(lv, q, scale, ws, grid, stream);
  else if (lv.G == 64) e = launch_g<64>(lv, q, scale, ws, grid, stream);
  else e = launch_g<128>(lv, q, scale, ws, grid, stream);
  *launches = 1;
  if (e != cudaSuccess || out == nullptr) return e;       // out == nullptr: the packed-block kernel alone (timing)
  LayerView res = lv;
  res.n_blocks = 0;
  const int n1 = (int)min((long long)grid * kWG, total);      // worker groups that own packed blocks
  const int slot2 = n1 + S;
  int l2 = 0;
  e = launch_attention_ws(res, q, nullptr, scale, ws + (size_t)slot2 * kPartialFloats, n_sms, stream, &l2);
  *launches += l2;
  if (e != cudaSuccess) return e;
  e = launch_combine2(ws, out, lv.g, lv.Hkv, lv.Hq, S, n1, lv.n_blocks, slot2, attention_ws_grid(res, n_sms),
                      attention_ws_positions(res), stream);
  *launches += 1;
  return e;
}

}  // namespace mixkvq
