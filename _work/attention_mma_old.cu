// Fused split-K GQA decode attention over the mixed-precision cache (Eq. 1 with Eq. 3 applied on the fly).
//
// Work unit = 32 tokens of one stream.  All units of all streams are split evenly over the CTAs; inside a
// CTA every warp owns a contiguous run of units and is an independent split: it stages its units into its
// own shared-memory ring with 1-D bulk (TMA) copies signalled on mbarriers, expands the 2-bit codes into
// tensor-core A fragments with one logic op (plus one fp16 FMA for keys) per pair of codes, and runs
// q.K^T, online softmax and P.V on mma.sync m16n8k16 tiles with the g query heads of the KV head as the
// N dimension.  The packed layout stores the codes in A-fragment order, so a lane's 16-byte shared-memory
// load is exactly its registers; nothing dequantized is ever written back to shared memory.
//
//   keys    A = c*s (exact in fp16: 2-bit code x 8-bit scale), B = q (exact), zero-points enter through
//           one extra tile per key group (A = z broadcast over rows) that initializes the accumulators.
//   values  A = raw codes read as fp16 subnormals (c * 4^i * 2^-24), B = P * s_v * 4^-i * 2^4, zero-points
//           and the softmax denominator through one extra tile (rows = value groups and a row of ones).
//   promoted (BF16) key channels and the UINT4 high plane come from the block's extras with a gathered q.
//   residual (unquantized) tokens use bf16 tiles straight from global memory.
#include <type_traits>

#include "common.cuh"

namespace mixkvq {

cudaError_t launch_combine(const float* ws, float* out, int g, int Hkv, int Hq, int mode, int n,
                           long long units_per_stream, int S, cudaStream_t stream);

namespace {

constexpr int kWarps = 6;
constexpr int kStages = 3;
// one ring stage: a key-meta group (512 B) followed by the unit (<= 2560 B; <= 3584 B with 4-bit values), as in the block
__host__ __device__ constexpr int stage_bytes(bool v4) { return v4 ? 4096 : 3072; }
constexpr int kKeyMetaOff = 0;
constexpr int kUnitOff = 512;
constexpr int kPrepBytes = 2560;             // kprep 576 | zprep 576 | svp 320 | zvp 1088
constexpr int kBarBytes = 256;                 // mbarriers: a ring per warp and one more per warp for the residual window
constexpr int kSharedTail = kBarBytes + 2048 + 2048 + 2 * kWarps * 32;
__host__ __device__ constexpr int smem_bytes(bool v4) { return kWarps * (kStages * stage_bytes(v4) + kPrepBytes) + kSharedTail; }
constexpr int kCtasPerSm = 2;
constexpr int kCtasPerSmDense = 2;           // with a 4-bit base two key planes are in flight: more registers per thread, fewer CTAs
static_assert((kWarps * kStages + kWarps) * 8 <= kBarBytes, "the mbarrier area at the start of the shared tail is too small");
constexpr int kResidualWeight = 3;           // a 32-token unit of the residual window counts as this many packed units in the split
constexpr uint32_t kSpinLimit = 1u << 22;    // bounded wait on a staged copy
constexpr int kMergeStride = 132;            // floats per head row of a warp's output in the merge (bank-conflict-free stores)
constexpr float kMaxSlack = 3.0f;            // a packed unit's probabilities are at most 2^kMaxSlack (log2 domain)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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
// Waits for a phase with an iteration limit; false if it gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// d = a * b + c with the accumulator input in other registers than the result
__device__ __forceinline__ void mma_f16_to(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                           uint32_t b1, float c0, float c1, float c2, float c3) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
               : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c0), "f"(c1), "f"(c2), "f"(c3));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
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
// 2^x by the special-function unit alone (no range fix-up): inputs here are <= 0 or -inf
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
// two bf16 in one word -> two fp16 in one word (exact inside the fp16 range)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) { return pack_half2(bf_lo(w), bf_hi(w)); }

// First 32-bit word of k-tile kt in the per-warp scale and zero-point tables (16 words per k-tile; the extra four words
// every second k-tile keep the stores of the preparation step free of bank conflicts).
__device__ __forceinline__ constexpr int prep_word(int kt) { return 16 * kt + 4 * (kt >> 1); }
// The same for the scale table, which has two words per (k-tile, t): 8 words per k-tile, two extra after the fourth.
__device__ __forceinline__ constexpr int scale_word(int kt) { return 8 * kt + 2 * (kt >> 2); }
// Bit position (inside each 16-bit half, after the shift below) of k-tile kt's 2-bit field.
__device__ __forceinline__ constexpr int key_pos(int kt) { return (0x86486464u >> (4 * kt)) & 0xF; }
// k-tiles 0,1 are read from (w << 4), 2..4 from w, 5..7 from (w >> 6)
__device__ __forceinline__ uint32_t key_shift(uint32_t w, int kt) { return kt < 2 ? (w << 4) : (kt < 5 ? w : (w >> 6)); }

// kU4: how the configuration can use the UINT4 tier: 0 = never (tau_u4 >= tau_bf16), 1 = some channels (high plane stored
// per channel pair, gathered), 2 = 4-bit base (dense high plane)
// kV4: 4-bit values (a second plane of 2-bit value codes per unit, scale 4 s_v)
template <int G, int kU4, bool kV4>
__global__ void __launch_bounds__(kWarps * 32, kU4 == 2 ? kCtasPerSmDense : kCtasPerSm)
attention_mma_kernel(LayerView lv, const __nv_bfloat16* __restrict__ q, float scale_log2e, float* __restrict__ ws,
                     uint32_t four2) {
  constexpr int VG = kD / G;              // value groups per token
  constexpr int TPG = 8 / VG;             // 16-channel tiles per value group
  constexpr int kStageBytes = stage_bytes(kV4);
  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, r = lane >> 2, t = lane & 3;

  unsigned char* ring = smem + warp * (kStages * kStageBytes);
  unsigned char* prep = smem + kWarps * kStages * kStageBytes + warp * kPrepBytes;
  uint32_t* kprep = reinterpret_cast<uint32_t*>(prep);          // [8 kt: scale_word][4 t]{s ch0, s ch1} half2 (first 288 of 576 bytes)
  // the zero-point tiles are stored as whole A fragments (four registers), so one 16-byte load feeds the MMA
  uint32_t* zprep = reinterpret_cast<uint32_t*>(prep + 576);    // [8 kt][4 t]{z ch0, z ch0, z ch1, z ch1} half2 z / mult
  // (20 words per t and 144 per ks instead of 16 and 128: the preparation's 16-bit stores then hit distinct banks)
  uint32_t* svp = reinterpret_cast<uint32_t*>(prep + 1152);     // [4 t: 20 words][4 vg][2 ks][2 ch] half2 s_v'
  uint32_t* zvp = reinterpret_cast<uint32_t*>(prep + 1472);     // [2 ks][8 rows][4 t]{ch0, 0, ch1, 0} half2: rows < VG z_v, row 4 ones
  unsigned char* tail = smem + kWarps * (kStages * kStageBytes + kPrepBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tail);           // [kWarps][kStages]
  uint16_t* qb16 = reinterpret_cast<uint16_t*>(tail + kBarBytes);           // [8][128] q, bf16 bits (0 for heads >= g)
  __half* qf16 = reinterpret_cast<__half*>(tail + kBarBytes + 2048);        // [8][128] q, fp16
  float* mS = reinterpret_cast<float*>(tail + kBarBytes + 4096);            // [kWarps][8]
  float* lS = mS + kWarps * 8;                                              // [kWarps][8]

  if (threadIdx.x == 0) {
    for (int i = 0; i < kWarps * kStages + kWarps; ++i) mbar_init(smem_u32(&bars[i]), 1);   // rings + one per warp for the residual window
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // constant rows of the zero-point / denominator tile: row 4 is all ones, the other rows >= VG stay zero
#pragma unroll
  for (int i = 0; i < 9; ++i) {
    const int idx = lane + 32 * i, rem = idx % 144, row = rem >> 4;      // [2 ks: 144 words][8 rows][4 t][4]
    if (idx < 272) zvp[idx] = (row == 4 && (idx & 1) == 0) ? 0x3C003C00u : 0u;
  }
  __syncthreads();

  // per-lane constants of the per-unit preparation steps
  // keys: the lane converts channels 4*lane .. 4*lane+3 (k-tile lane / 4)
  const float pk_zs = __uint_as_float((119u + (uint32_t)key_pos(lane >> 2)) << 23);        // 2^(pos - 8)
  const int pk_zp = prep_word(lane >> 2) + 8 * (lane & 1) + ((lane & 3) >> 1) * 2;         // zprep word of the first pair
  const int pk_kp = scale_word(lane >> 2) + 4 * (lane & 1) + ((lane & 3) >> 1);            // kprep word of the first pair
  // values: the lane converts the scales and zero-points of token `lane`
  const float pv_up = __uint_as_float((131u - 2u * (uint32_t)(lane >> 3)) << 23);          // 2^(4 - 2 * (2 ks + ch))
  const int pv_sv = ((((lane & 7) >> 1) * 20 + (lane >> 3)) * 2) + (lane & 1);             // svp half index of group 0
  const int pv_zv = (((lane >> 4) * 144 + ((lane & 7) >> 1) * 4 + 2 * ((lane >> 3) & 1)) * 2) + (lane & 1);   // zvp half index of group 0
  // codes of 32 tokens: keys 1024, values 1024, value scales (and the values' high plane 1024)
  constexpr uint32_t kUnitBytes = 2048u + 128u * (kD / G) + (kV4 ? 1024u : 0u);
  constexpr int UPG = G / 32;                                 // units per key group

  const int S = lv.B * lv.Hkv, U = lv.U, g = lv.g;
  const int packed_units = lv.n_blocks * U;
  // unquantized 32-token units: those of the residual window, then those of the sink
  const int res_units = (lv.r + 31) / 32, bf16_units = res_units + (lv.n_sink + 31) / 32;
  const int Us = packed_units + kResidualWeight * bf16_units;             // split positions; an unquantized unit spans several
  const long long total = (long long)Us * S;
  const long long cb = split_begin(total, gridDim.x, blockIdx.x), ce = split_begin(total, gridDim.x, blockIdx.x + 1);

  uint32_t res_phase = 0;         // phase of this warp's residual-staging barrier
  // Programmatic dependent launch: the grid may have been started while the kernel before it in the stream was still
  // running.  Nothing above touches global memory; everything below does, so wait here for that kernel's results,
  // and let the kernel after this one be started early in the same way.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  uint32_t ring_stage = 0;        // ring stage of the next packed unit this warp consumes
  uint32_t ring_parity = 0;       // phase parity of that stage's barrier
  bool gave_up = false;

  for (long long seg = cb; seg < ce;) {
    const int s = (int)(seg / Us);
    const int ub = (int)(seg - (long long)s * Us);
    const int ue = (int)min((long long)Us, ce - (long long)s * Us);
    seg += ue - ub;
    // ---- the query of this stream is requested before anything else: the burst of staged copies below would delay it
    uint4 q_regs = make_uint4(0u, 0u, 0u, 0u);      // thread (h, c) of the first 128: head h, channels 8c .. 8c+7
    {
      const int b = s / lv.Hkv, hk = s % lv.Hkv, h = threadIdx.x >> 4, c = threadIdx.x & 15;
      if (h < g) q_regs = *reinterpret_cast<const uint4*>(q + ((size_t)b * lv.Hq + hk * g + h) * kD + 8 * c);
    }
    // ---- this warp's share of the segment.  The residual units of the segment go to different warps (unit i to warp
    // kWarps - 1 - i % kWarps), so that their copies and their arithmetic run side by side; the packed units are split
    // in order so that every warp carries about the same weight.
    const int pk_b = min(ub, packed_units), pk_e = min(ue, packed_units);
    const int res_b = (max(ub, packed_units) - packed_units + kResidualWeight - 1) / kResidualWeight;
    const int res_e = ue > packed_units ? (ue - packed_units + kResidualWeight - 1) / kResidualWeight : res_b;
    const int n_res = res_e - res_b;
    int wb = pk_b, we = pk_b;
    {
      const int weight = (pk_e - pk_b) + kResidualWeight * n_res;
      int remaining = pk_e - pk_b;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const int share = weight * (w + 1) / kWarps - weight * w / kWarps;       // weight < 2^24: 32-bit arithmetic
        const int first_i = kWarps - 1 - w;                                   // residual units first_i, first_i + kWarps, ...
        const int res_w = n_res > first_i ? (n_res - first_i + kWarps - 1) / kWarps : 0;
        int p = min(remaining, max(0, share - kResidualWeight * res_w));
        if (w == kWarps - 1) p = remaining;
        if (w == warp) {
          wb = pk_e - remaining;
          we = wb + p;
        }
        remaining -= p;
      }
    }

    const char* base = lv.base + (size_t)s * lv.base_stride;
    const char* extras = lv.extras + (size_t)s * lv.extras_stride;
    const uint2* table = reinterpret_cast<const uint2*>(lv.table + (size_t)s * lv.table_stride);

    // ---- the first copies of this segment go out before anything else: they do not depend on the query.
    // The packed units of a stream are one uniform sequence (a group's scales, then its units), whatever the block size,
    // so the copy source only ever moves forward: `isrc` is the next unit to stage, `ig` its index inside its key group.
    const int n_pack = we - wb;
    int issued = 0;
    const char* isrc = base + (size_t)wb * kUnitBytes + 512u * (size_t)(wb / UPG + 1);
    int ig = wb & (UPG - 1);
    auto issue = [&](uint32_t dst, uint32_t bar, bool first) {
      // all lanes keep the position; lane 0 stages the unit at ring offset dst, signalled on bar
      if (UPG == 1 || ig == 0) {        // the group's scales lie directly before the unit: one copy
        if (lane == 0) {
          mbar_expect_tx(bar, kUnitBytes + 512u);
          bulk_g2s(dst + kKeyMetaOff, isrc - 512, 512u + kUnitBytes, bar);
        }
      } else if (lane == 0) {
        mbar_expect_tx(bar, kUnitBytes + (first ? 512u : 0u));
        bulk_g2s(dst + kUnitOff, isrc, kUnitBytes, bar);
        if (first) bulk_g2s(dst + kKeyMetaOff, isrc - (size_t)ig * kUnitBytes - 512, 512u, bar);
      }
      isrc += kUnitBytes;
      if (UPG == 1) {
        isrc += 512;
      } else {
        ig = (ig + 1) & (UPG - 1);
        if (ig == 0) isrc += 512;
      }
    };
    // the ring continues where the previous segment left it: stage ring_stage, barrier phase parity ring_parity
    const uint32_t ring_u32 = smem_u32(ring), bar_u32 = smem_u32(&bars[warp * kStages]);
    if (!gave_up) {
      uint32_t sg = ring_stage;
      for (; issued < min(n_pack, kStages); ++issued) {
        issue(ring_u32 + sg * kStageBytes, bar_u32 + sg * 8u, issued == 0);
        sg = (sg == kStages - 1) ? 0u : sg + 1u;
      }
    }

    // the first block's table entry is requested now as well, long before the first unit arrives
    int bi = 0, u = 0;                     // block and unit inside it of the next unit to consume
    uint2 pf_entry = make_uint2(0, 0);
    if (n_pack > 0) {
      bi = wb / U;
      u = wb - bi * U;
      pf_entry = table[bi];
    }
    bool new_block = true;
    int n16 = 0, n4 = 0, n16p = 0;
    uint32_t xb0 = 0u, xb1 = 0u;          // B fragments of the block's first 16 promoted channels
    // the block's first 32 UINT4 channels (two tiles of eight pairs): B fragments (gathered fp16 query pairs) and, per
    // pair, where the two channels' scales sit in the scale table (half index, 0xFFFF: no channel)
    uint32_t u4q[2][2] = {{0u, 0u}, {0u, 0u}}, u4s[2][2] = {{~0u, ~0u}, {~0u, ~0u}};
    const char* ex = nullptr;             // the block's extras
    const char* exu = nullptr;            // ... of the current unit
    uint32_t ex_unit = 0;

    // ---- query of this stream: bf16 and fp16 tables for the gathered paths
    {
      __syncthreads();
      {
        // heads >= g are zero rows
        const int h = threadIdx.x >> 4, c = threadIdx.x & 15;
        if (h < 8) {
          const uint4 v = q_regs;
          *reinterpret_cast<uint4*>(&qb16[h * kD + 8 * c]) = v;
          *reinterpret_cast<uint4*>(&qf16[h * kD + 8 * c]) =
              make_uint4(bf16x2_to_f16x2(v.x), bf16x2_to_f16x2(v.y), bf16x2_to_f16x2(v.z), bf16x2_to_f16x2(v.w));
        }
      }
      __syncthreads();
    }
    // B fragments of q for the base key tiles: head r, channels 16kt + {2t, 2t+1} and {2t+8, 2t+9}, times mult(kt)
    uint32_t bq[8][2];
#pragma unroll
    for (int kt = 0; kt < 8; ++kt) {
      const float mult = (float)(1 << (8 - key_pos(kt)));
#pragma unroll
      for (int hch = 0; hch < 2; ++hch) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(&qb16[r * kD + 16 * kt + 8 * hch + 2 * t]);
        bq[kt][hch] = pack_half2(bf_lo(w) * mult, bf_hi(w) * mult);
      }
    }

    float O[8][4];       // O^T tiles: [channel tile] x (channels r, r+8) x (heads 2t, 2t+1); packed part scaled 2^-20
    float Zc[4] = {0.f, 0.f, 0.f, 0.f};   // rows 0..VG-1: sum p * z_v per value group; row 4: sum p
    float zl0 = 0.f, zl1 = 0.f;           // key zero-point term (q . z) * scale of the current key group, heads 2t, 2t+1
    float m0 = -INFINITY, m1 = -INFINITY; // running max (log2 domain) of heads 2t, 2t+1
#pragma unroll
    for (int ct = 0; ct < 8; ++ct)
#pragma unroll
      for (int i = 0; i < 4; ++i) O[ct][i] = 0.f;
    bool o_true_scale = false;

    // A fragments of the first 16 promoted channels of a unit: lane (r, t) holds channel pairs t and t + 4 for tokens
    // r, r + 8 of both m-tiles.  Pairs past the block's count read an existing pair instead (their query entries are 0).
    uint32_t xa[2][4];
    bool xa_loaded = false;
    auto load_xa = [&](const char* e) {
      const uint32_t* xw = reinterpret_cast<const uint32_t*>(e) + (min(t, n16p - 1) * 32 + r);
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        xa[mt][0] = xw[mt * 16];
        xa[mt][1] = xw[mt * 16 + 8];
      }
      if (n16p > 4) {       // more than 8 promoted channels (uniform over the warp)
        const uint32_t* xv = reinterpret_cast<const uint32_t*>(e) + (min(t + 4, n16p - 1) * 32 + r);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          xa[mt][2] = xv[mt * 16];
          xa[mt][3] = xv[mt * 16 + 8];
        }
      }
    };
    int consumed = 0;
    for (; consumed < n_pack && !gave_up; ++consumed) {
      if (new_block) {
        const uint2 entry = pf_entry;
        if (bi + 1 < lv.n_blocks) pf_entry = table[bi + 1];
        n16 = entry.y & 0xFF;
        n4 = (entry.y >> 8) & 0xFF;
        n16p = (n16 + 1) >> 1;
        ex = extras + (size_t)entry.x * 16;
        ex_unit = extras_unit_bytes(n16, n4, kU4 == 2);
        exu = ex + extras_header_bytes(n16, n4) + (size_t)u * ex_unit;
        // the block's promoted channels are the same for its units: gather their query entries once
        xb0 = xb1 = 0u;
        if (n16 > 0) {
          auto gather_q = [&](int p) -> uint32_t {
            if (p >= n16p) return 0u;
            const uint32_t ids = *reinterpret_cast<const uint16_t*>(ex + 2 * p);
            const uint32_t c0 = ids & 0xFF, c1 = (ids >> 8) & 0xFF;
            const uint32_t lo = (c0 < 128) ? qb16[r * kD + c0] : 0u, hi = (c1 < 128) ? qb16[r * kD + c1] : 0u;
            return lo | (hi << 16);
          };
          xb0 = gather_q(t);
          xb1 = gather_q(t + 4);
        }
        if (kU4 == 1 && n4 > 0) {
          const int n4pairs = (n4 + 1) >> 1;
          const unsigned char* ids4 = reinterpret_cast<const unsigned char*>(ex) + 2 * n16p;
#pragma unroll
          for (int kk = 0; kk < 2; ++kk)
#pragma unroll
            for (int hp = 0; hp < 2; ++hp) {
              const int p = 8 * kk + 4 * hp + t;
              uint32_t c0 = 255u, c1 = 255u;
              if (p < n4pairs) {
                c0 = ids4[2 * p];
                c1 = ids4[2 * p + 1];
              }
              auto scale_index = [&](uint32_t c) -> uint32_t {      // half index of channel c's scale in kprep
                const int kt = c >> 4, col = c & 15;
                return c < 128 ? (uint32_t)(((scale_word(kt) + ((col & 7) >> 1) * 2 + (col >> 3)) << 1) + (col & 1)) : 0xFFFFu;
              };
              const uint32_t q0 = c0 < 128 ? (uint32_t)__half_as_ushort(qf16[r * kD + c0]) : 0u;
              const uint32_t q1 = c1 < 128 ? (uint32_t)__half_as_ushort(qf16[r * kD + c1]) : 0u;
              u4q[kk][hp] = q0 | (q1 << 16);
              u4s[kk][hp] = scale_index(c0) | (scale_index(c1) << 16);
            }
        }
        new_block = false;
        xa_loaded = false;
      }
      if (!mbar_wait_bounded(bar_u32 + ring_stage * 8u, ring_parity)) {
        gave_up = true;
        break;
      }
      const unsigned char* stg = ring + ring_stage * kStageBytes;
      const unsigned char* st = stg + kUnitOff;        // the unit's codes and value scales
      const bool has_meta = (UPG == 1) || (consumed == 0) || ((u & (UPG - 1)) == 0);

      // ---- extras of this unit (BF16 pairs of the first 16 promoted channels), unless the previous unit already
      // requested them
      if (n16 > 0 && !xa_loaded) load_xa(exu);
      // the UINT4 high-plane words of the first two tiles of this unit are requested early as well
      uint32_t u4w[2][2] = {{0u, 0u}, {0u, 0u}};
      if (kU4 == 1 && n4 > 0) {
        const int n4pairs = (n4 + 1) >> 1;
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(exu + 128 * n16p);
#pragma unroll
        for (int kk = 0; kk < 2; ++kk)
#pragma unroll
          for (int hp = 0; hp < 2; ++hp) {
            const int p = 8 * kk + 4 * hp + t;
            if (p < n4pairs) u4w[kk][hp] = hw[p * 4 + (r & 3)];
          }
      }
      // the key codes: two 16-byte loads per lane are the A fragments of all sixteen key tiles (with a 4-bit base the
      // first plane to run is the high plane, which lies with the block's extras in global memory)
      const uint4* kplane = (kU4 == 2) ? reinterpret_cast<const uint4*>(exu + 128 * n16p) : reinterpret_cast<const uint4*>(st);
      const uint4 hw0 = kplane[lane], hw1 = kplane[32 + lane];

      // ---- value-group preparation (lane = token).  The tables of the previous unit were last read before the
      // warp barrier that closed it, so they can be overwritten right away.
      {
        const uint32_t* vmeta = reinterpret_cast<const uint32_t*>(st + 2048) + lane * VG;
        __half* svh = reinterpret_cast<__half*>(svp) + pv_sv;
        __half* zvh = reinterpret_cast<__half*>(zvp) + pv_zv;
#pragma unroll
        for (int vg = 0; vg < VG; ++vg) {
          const uint32_t mz = vmeta[vg];
          svh[8 * vg] = __float2half_rn(bf_lo(mz) * pv_up);
          zvh[32 * vg] = __float2half_rn(bf_hi(mz));
        }
      }

      // ---- key-group preparation: fp16 scale pairs in fragment order, zero-point tile
      if (has_meta) {
        const uint4 mz = reinterpret_cast<const uint4*>(stg + kKeyMetaOff)[lane];   // channels 4*lane .. 4*lane+3
        const uint32_t ma = pack_half2(bf_lo(mz.x), bf_lo(mz.y)), mb = pack_half2(bf_lo(mz.z), bf_lo(mz.w));
        kprep[pk_kp] = ma;
        kprep[pk_kp + 2] = mb;
        const uint32_t za = pack_half2(bf_hi(mz.x) * pk_zs, bf_hi(mz.y) * pk_zs);
        const uint32_t zb = pack_half2(bf_hi(mz.z) * pk_zs, bf_hi(mz.w) * pk_zs);
        *reinterpret_cast<uint2*>(&zprep[pk_zp]) = make_uint2(za, za);
        *reinterpret_cast<uint2*>(&zprep[pk_zp + 4]) = make_uint2(zb, zb);
      }
      __syncwarp();      // the tables written above are read by other lanes below
      if (has_meta) {
        // the zero-point term q . z of the group: its own accumulator chain, added to the logits after the key tiles
        // (the tile's rows are equal, so are the rows of the result)
        float zc[4];
#pragma unroll
        for (int kt2 = 0; kt2 < 8; ++kt2) {
          const uint4 zz = *reinterpret_cast<const uint4*>(&zprep[prep_word(kt2) + 4 * t]);
          if (kt2 == 0) mma_f16_to(zc, zz.x, zz.y, zz.z, zz.w, bq[0][0], bq[0][1], 0.f, 0.f, 0.f, 0.f);
          else mma_f16(zc, zz.x, zz.y, zz.z, zz.w, bq[kt2][0], bq[kt2][1]);
        }
        zl0 = zc[0] * scale_log2e;
        zl1 = zc[1] * scale_log2e;
      }

      // ---- q.K^T on the key tiles.  One pass over a plane of 2-bit codes: the base (low) plane with the scales s, and,
      // with a 4-bit base, first the dense high plane (codes c >> 2, laid out like the low plane) with the scales 4s.
      float Sx[2][4];
      auto key_pass = [&](const uint4& w0, const uint4& w1, auto first_tag, auto high_tag) {
        constexpr bool first = decltype(first_tag)::value, high = decltype(high_tag)::value;
        const uint32_t kw[2][4] = {{w0.x, w0.y, w0.z, w0.w}, {w1.x, w1.y, w1.z, w1.w}};
#pragma unroll
        for (int kt = 0; kt < 8; ++kt) {
          // scales of the lane's channel pairs (16kt + 2t, +1) and (16kt + 8 + 2t, +1); code bias 4 -> offset -4 s
          const uint2 sc = *reinterpret_cast<const uint2*>(&kprep[scale_word(kt) + 2 * t]);
          const uint32_t neg4 = 0xC400C400u;   // half2(-4, -4)
          uint4 kp = make_uint4(sc.x, hmul2_u(sc.x, neg4), sc.y, hmul2_u(sc.y, neg4));
          if (high) kp = make_uint4(hmul2_u(kp.x, four2), hmul2_u(kp.y, four2), hmul2_u(kp.z, four2), hmul2_u(kp.w, four2));
          const uint32_t mask = 0x00030003u << key_pos(kt);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            uint32_t a[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t code = (key_shift(kw[mt][j], kt) & mask) | four2;           // 4 + c * 2^(pos-8)
              a[j] = hfma2_u(code, j < 2 ? kp.x : kp.z, j < 2 ? kp.y : kp.w);            // c * s * 2^(pos-8)
            }
            if (first && kt == 0) mma_f16_to(Sx[mt], a[0], a[1], a[2], a[3], bq[0][0], bq[0][1], 0.f, 0.f, 0.f, 0.f);
            else mma_f16(Sx[mt], a[0], a[1], a[2], a[3], bq[kt][0], bq[kt][1]);
          }
        }
      };
      if constexpr (kU4 == 2) {
        key_pass(hw0, hw1, std::true_type{}, std::true_type{});
        const uint4 kw0 = reinterpret_cast<const uint4*>(st)[lane];
        const uint4 kw1 = reinterpret_cast<const uint4*>(st)[32 + lane];
        key_pass(kw0, kw1, std::false_type{}, std::false_type{});
      } else {
        key_pass(hw0, hw1, std::true_type{}, std::false_type{});
      }
      // ---- promoted channels (raw bf16 keys) with a gathered q
      if (n16 > 0) {
        if (n16p > 4) {
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) mma_bf16(Sx[mt], xa[mt][0], xa[mt][1], xa[mt][2], xa[mt][3], xb0, xb1);
        } else {
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) mma_bf16(Sx[mt], xa[mt][0], xa[mt][1], 0u, 0u, xb0, 0u);
        }
        // the registers are free again: request the next unit's pairs now, most of an iteration ahead of their use
        xa_loaded = (u + 1 < U) && (consumed + 1 < n_pack);
        if (xa_loaded) load_xa(exu + ex_unit);
        for (int kk = 1; kk * 8 < n16p; ++kk) {       // more than 16 promoted channels
          uint32_t a[2][4], id0 = 0xFFFFFFFFu, id1 = 0xFFFFFFFFu;
          const uint32_t* xw = reinterpret_cast<const uint32_t*>(exu);
          const int p0 = 8 * kk + t, p1 = p0 + 4;
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) a[mt][0] = a[mt][1] = a[mt][2] = a[mt][3] = 0;
          if (p0 < n16p) {
            id0 = *reinterpret_cast<const uint16_t*>(ex + 2 * p0);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              a[mt][0] = xw[p0 * 32 + mt * 16 + r];
              a[mt][1] = xw[p0 * 32 + mt * 16 + 8 + r];
            }
          }
          if (p1 < n16p) {
            id1 = *reinterpret_cast<const uint16_t*>(ex + 2 * p1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              a[mt][2] = xw[p1 * 32 + mt * 16 + r];
              a[mt][3] = xw[p1 * 32 + mt * 16 + 8 + r];
            }
          }
          auto gather_bf16 = [&](uint32_t ids) -> uint32_t {
            const uint32_t c0 = ids & 0xFF, c1 = (ids >> 8) & 0xFF;
            const uint32_t lo = (c0 < 128) ? qb16[r * kD + c0] : 0u, hi = (c1 < 128) ? qb16[r * kD + c1] : 0u;
            return lo | (hi << 16);
          };
          const uint32_t b0 = gather_bf16(id0), b1 = gather_bf16(id1);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) mma_bf16(Sx[mt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], b0, b1);
        }
      }
      // ---- UINT4 high plane: c_hi * 4s, gathered q in fp16.  The first two tiles (32 channels) use the block's gathered
      // query pairs and scale positions; further tiles look their channels up per unit.
      if (kU4 == 1 && n4 > 0) {
        const int n4pairs = (n4 + 1) >> 1;
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(exu + 128 * n16p);
        const unsigned char* ids4 = reinterpret_cast<const unsigned char*>(ex) + 2 * n16p;
        const unsigned short* kph = reinterpret_cast<const unsigned short*>(kprep);
        auto plane_tile = [&](const uint32_t (&words)[2], const uint32_t (&sidx)[2], const uint32_t (&qb)[2]) {
          uint32_t a[2][4];
#pragma unroll
          for (int hp = 0; hp < 2; ++hp) {
            const uint32_t w = words[hp] >> (8 * (r >> 2));
            const uint32_t i0 = sidx[hp] & 0xFFFFu, i1 = sidx[hp] >> 16;
            const uint32_t sc = (i0 != 0xFFFFu ? (uint32_t)kph[i0] : 0u) | ((i1 != 0xFFFFu ? (uint32_t)kph[i1] : 0u) << 16);
            const uint32_t m4 = hmul2_u(sc, four2);                // 4s
            const uint32_t o4 = hmul2_u(sc, 0xCC00CC00u);          // -16s
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
              for (int rh = 0; rh < 2; ++rh) {
                const int f = 2 * mt + rh;
                const uint32_t code = ((w << (8 - 2 * f)) & 0x03000300u) | four2;          // 4 + c_hi
                a[mt][2 * hp + rh] = hfma2_u(code, m4, o4);                                // c_hi * 4s
              }
          }
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) mma_f16(Sx[mt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], qb[0], qb[1]);
        };
        plane_tile(u4w[0], u4s[0], u4q[0]);
        if (n4pairs > 8) plane_tile(u4w[1], u4s[1], u4q[1]);
        for (int kk = 2; kk * 8 < n4pairs; ++kk) {
          uint32_t sidx[2], qb[2], words[2] = {0u, 0u};
#pragma unroll
          for (int hp = 0; hp < 2; ++hp) {
            const int p = 8 * kk + 4 * hp + t;
            uint32_t c0 = 255u, c1 = 255u;
            if (p < n4pairs) {
              c0 = ids4[2 * p];
              c1 = ids4[2 * p + 1];
              words[hp] = hw[p * 4 + (r & 3)];
            }
            auto scale_index = [&](uint32_t c) -> uint32_t {
              const int kt = c >> 4, col = c & 15;
              return c < 128 ? (uint32_t)(((scale_word(kt) + ((col & 7) >> 1) * 2 + (col >> 3)) << 1) + (col & 1)) : 0xFFFFu;
            };
            const uint32_t q0 = c0 < 128 ? (uint32_t)__half_as_ushort(qf16[r * kD + c0]) : 0u;
            const uint32_t q1 = c1 < 128 ? (uint32_t)__half_as_ushort(qf16[r * kD + c1]) : 0u;
            qb[hp] = q0 | (q1 << 16);
            sidx[hp] = scale_index(c0) | (scale_index(c1) << 16);
          }
          plane_tile(words, sidx, qb);
        }
      }

      // ---- online softmax (log2 domain); heads 2t, 2t+1; tokens r, r+8 of each m-tile.
      // logit = (Sx + zc) * scale: the zero-point term zc is the same for every token of the unit
      float u0 = fmaxf(fmaxf(Sx[0][0], Sx[0][2]), fmaxf(Sx[1][0], Sx[1][2]));
      float u1 = fmaxf(fmaxf(Sx[0][1], Sx[0][3]), fmaxf(Sx[1][1], Sx[1][3]));
      u0 = fmaf(u0, scale_log2e, zl0);
      u1 = fmaf(u1, scale_log2e, zl1);
      // The reference maximum only has to keep the probabilities inside the fp16 range: it is raised (to the true
      // maximum so far, with the accumulators rescaled) when a logit of this unit exceeds it by more than kMaxSlack.
      if (__any_sync(0xffffffffu, (u0 > m0 + kMaxSlack) || (u1 > m1 + kMaxSlack))) {
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
          u0 = fmaxf(u0, __shfl_xor_sync(0xffffffffu, u0, off));
          u1 = fmaxf(u1, __shfl_xor_sync(0xffffffffu, u1, off));
        }
        const float n0 = fmaxf(m0, u0), n1 = fmaxf(m1, u1);
        const float a0 = exp2f(m0 - n0), a1 = exp2f(m1 - n1);    // exp2(-inf) = 0 on the first unit
#pragma unroll
        for (int ct = 0; ct < 8; ++ct) {
          O[ct][0] *= a0; O[ct][1] *= a1; O[ct][2] *= a0; O[ct][3] *= a1;
        }
        Zc[0] *= a0; Zc[1] *= a1; Zc[2] *= a0; Zc[3] *= a1;
        m0 = n0;
        m1 = n1;
      }
      const float c0 = zl0 - m0, c1 = zl1 - m1;
      uint32_t Pt[2][2];    // P^T B fragments: [k-step][tokens 2t.. / 2t+8..], head r
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t plo = pack_half2(ex2_approx(fmaf(Sx[mt][0], scale_log2e, c0)), ex2_approx(fmaf(Sx[mt][1], scale_log2e, c1)));   // token r
        const uint32_t phi = pack_half2(ex2_approx(fmaf(Sx[mt][2], scale_log2e, c0)), ex2_approx(fmaf(Sx[mt][3], scale_log2e, c1)));   // token r + 8
        Pt[mt][0] = movmatrix_trans(plo);
        Pt[mt][1] = movmatrix_trans(phi);
      }

      // ---- zero-point and denominator tile: rows 0..VG-1 = z_v of the group, row 4 = ones, the rest zero
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const uint4 zz = *reinterpret_cast<const uint4*>(&zvp[ks * 144 + (r * 4 + t) * 4]);
        mma_f16(Zc, zz.x, zz.y, zz.z, zz.w, Pt[ks][0], Pt[ks][1]);
      }
      // ---- P.V: codes as fp16 subnormals, scales folded into P
      {
        const uint4 vw0 = reinterpret_cast<const uint4*>(st + 1024)[lane];
        const uint4 vw1 = reinterpret_cast<const uint4*>(st + 1024)[32 + lane];
        const uint32_t vw[8] = {vw0.x, vw0.y, vw0.z, vw0.w, vw1.x, vw1.y, vw1.z, vw1.w};
#pragma unroll
        for (int vg = 0; vg < VG; ++vg) {
          const uint4 sv = *reinterpret_cast<const uint4*>(&svp[t * 20 + vg * 4]);
          const uint32_t Bp[2][2] = {{hmul2_u(Pt[0][0], sv.x), hmul2_u(Pt[0][1], sv.y)},
                                     {hmul2_u(Pt[1][0], sv.z), hmul2_u(Pt[1][1], sv.w)}};
#pragma unroll
          for (int c = 0; c < TPG; ++c) {
            const int ct = vg * TPG + c;
            const uint32_t x0 = vw[ct], x1 = vw[ct] >> 8;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
              const uint32_t mk0 = 0x00030003u << (4 * ks), mk1 = 0x00030003u << (4 * ks + 2);
              mma_f16(O[ct], x0 & mk0, x1 & mk0, x0 & mk1, x1 & mk1, Bp[ks][0], Bp[ks][1]);
            }
          }
        }
      }
      // ---- 4-bit values: the high plane (codes >> 2, the low plane's bit order) with four times the scale
      if constexpr (kV4) {
        const uint4 vw0 = reinterpret_cast<const uint4*>(st + 2048 + 128 * VG)[lane];
        const uint4 vw1 = reinterpret_cast<const uint4*>(st + 2048 + 128 * VG)[32 + lane];
        const uint32_t vw[8] = {vw0.x, vw0.y, vw0.z, vw0.w, vw1.x, vw1.y, vw1.z, vw1.w};
#pragma unroll
        for (int vg = 0; vg < VG; ++vg) {
          const uint4 sv = *reinterpret_cast<const uint4*>(&svp[t * 20 + vg * 4]);
          const uint32_t Bp[2][2] = {{hmul2_u(hmul2_u(Pt[0][0], sv.x), four2), hmul2_u(hmul2_u(Pt[0][1], sv.y), four2)},
                                     {hmul2_u(hmul2_u(Pt[1][0], sv.z), four2), hmul2_u(hmul2_u(Pt[1][1], sv.w), four2)}};
#pragma unroll
          for (int c = 0; c < TPG; ++c) {
            const int ct = vg * TPG + c;
            const uint32_t x0 = vw[ct], x1 = vw[ct] >> 8;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
              const uint32_t mk0 = 0x00030003u << (4 * ks), mk1 = 0x00030003u << (4 * ks + 2);
              mma_f16(O[ct], x0 & mk0, x1 & mk0, x0 & mk1, x1 & mk1, Bp[ks][0], Bp[ks][1]);
            }
          }
        }
      }

      // ---- release the stage and refill it, then move on to the next unit
      __syncwarp();
      if (issued < n_pack) {
        issue(ring_u32 + ring_stage * kStageBytes, bar_u32 + ring_stage * 8u, false);
        ++issued;
      }
      if (++ring_stage == kStages) {
        ring_stage = 0;
        ring_parity ^= 1u;
      }
      exu += ex_unit;
      if (++u == U) {
        u = 0;
        ++bi;
        new_block = true;
      }
    }
    if (gave_up) {
      // drain what is still in flight (bounded); later segments stage nothing but still join the CTA barriers
      for (; consumed < issued; ++consumed) {
        mbar_wait_bounded(bar_u32 + ring_stage * 8u, ring_parity);
        if (++ring_stage == kStages) {
          ring_stage = 0;
          ring_parity ^= 1u;
        }
      }
      if (lane == 0) atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
    }

    // ---- residual (unquantized) tokens of this warp's range: 32 token rows of 256 B staged through the (now idle)
    // ring with ONE bulk copy, first the keys, then the values over them (small bulk copies are slow: a copy per row
    // cost tens of microseconds).  Value tiles are transposed on the way to registers with ldmatrix.trans.
    for (int ri = kWarps - 1 - warp; ri < n_res && !gave_up; ri += kWarps) {
      const int bu = res_b + ri;                        // unquantized unit: residual window first, then the sink
      const bool in_sink = bu >= res_units;
      const int wu = in_sink ? bu - res_units : bu;     // unit inside its window
      const int rt = in_sink ? lv.n_sink : lv.r;        // tokens in that window
      const uint32_t rbar = smem_u32(&bars[kWarps * kStages + warp]);
      const uint16_t* resk = reinterpret_cast<const uint16_t*>(in_sink ? lv.sink + (size_t)s * lv.sink_stride
                                                                       : lv.resk + (size_t)s * lv.resk_stride);
      const uint16_t* resv = reinterpret_cast<const uint16_t*>(in_sink ? lv.sink + (size_t)s * lv.sink_stride + (size_t)lv.sink_len * 256
                                                                       : lv.resv + (size_t)s * lv.resv_stride);
      // fused decode step: the newest token (slot r - 1) is not in the residual store yet; the warp whose unit holds it
      // takes its rows from the step's tensors (into the staged tile and into the store) and updates the accumulator
      const int jn = lv.r - 1;
      const bool holds_new = !in_sink && lv.new_k != nullptr && jn >= wu * 32 && jn < wu * 32 + 32;
      {
        const int j0s = wu * 32, nv = min(32, rt - j0s) - (holds_new ? 1 : 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (nv > 0) {
          if (lane == 0) {
            mbar_expect_tx(rbar, (uint32_t)nv * 256u);
            bulk_g2s(smem_u32(ring), resk + (size_t)j0s * kD, (uint32_t)nv * 256u, rbar);
          }
          if (!mbar_wait_bounded(rbar, res_phase)) {
            gave_up = true;
            if (lane == 0) atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
            break;
          }
          res_phase ^= 1u;
        }
        if (holds_new) {
          const uint2 kn = reinterpret_cast<const uint2*>(lv.new_k + (size_t)s * kD)[lane];
          reinterpret_cast<uint2*>(ring + (jn - j0s) * 256)[lane] = kn;
          reinterpret_cast<uint2*>(lv.resk + (size_t)s * lv.resk_stride + (size_t)jn * 256)[lane] = kn;
          // importance accumulator: channels 4*lane .. 4*lane+3, heads ascending (the order of the plain append)
          double* acc = reinterpret_cast<double*>(lv.state + (size_t)s * lv.state_stride);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int d = 4 * lane + c;
            double a = acc[d];
            for (int h = 0; h < g; ++h) a = __dadd_rn(a, (double)fabsf(__uint_as_float((uint32_t)qb16[h * kD + d] << 16)));
            acc[d] = a;
          }
          if (lane == 0) *reinterpret_cast<uint32_t*>(lv.state + (size_t)s * lv.state_stride + 1024) += (uint32_t)g;
          __syncwarp();
        }
      }
      if (!o_true_scale) {
#pragma unroll
        for (int ct = 0; ct < 8; ++ct)
#pragma unroll
          for (int j = 0; j < 4; ++j) O[ct][j] *= 1048576.0f;
        o_true_scale = true;
      }
      const int j0 = wu * 32;
      float Sx[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
      for (int kt = 0; kt < 8; ++kt) {
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(&qb16[r * kD + 16 * kt + 2 * t]);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(&qb16[r * kD + 16 * kt + 8 + 2 * t]);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          const int ta = j0 + mt * 16 + r, tb = ta + 8;
          const uint32_t* ka = reinterpret_cast<const uint32_t*>(ring + (mt * 16 + r) * 256 + (16 * kt + 2 * t) * 2);
          const uint32_t* kb = reinterpret_cast<const uint32_t*>(ring + (mt * 16 + 8 + r) * 256 + (16 * kt + 2 * t) * 2);
          const uint32_t a0 = ta < rt ? ka[0] : 0u, a1 = tb < rt ? kb[0] : 0u;
          const uint32_t a2 = ta < rt ? ka[4] : 0u, a3 = tb < rt ? kb[4] : 0u;
          mma_bf16(Sx[mt], a0, a1, a2, a3, b0, b1);
        }
      }
      float xl[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const bool va = (j0 + mt * 16 + r) < rt, vb = (j0 + mt * 16 + 8 + r) < rt;
        xl[mt][0] = va ? Sx[mt][0] * scale_log2e : -INFINITY;
        xl[mt][1] = va ? Sx[mt][1] * scale_log2e : -INFINITY;
        xl[mt][2] = vb ? Sx[mt][2] * scale_log2e : -INFINITY;
        xl[mt][3] = vb ? Sx[mt][3] * scale_log2e : -INFINITY;
      }
      float u0 = fmaxf(fmaxf(xl[0][0], xl[0][2]), fmaxf(xl[1][0], xl[1][2]));
      float u1 = fmaxf(fmaxf(xl[0][1], xl[0][3]), fmaxf(xl[1][1], xl[1][3]));
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        u0 = fmaxf(u0, __shfl_xor_sync(0xffffffffu, u0, off));
        u1 = fmaxf(u1, __shfl_xor_sync(0xffffffffu, u1, off));
      }
      const float n0 = fmaxf(m0, u0), n1 = fmaxf(m1, u1);
      if (__any_sync(0xffffffffu, (n0 > m0) || (n1 > m1))) {
        const float a0 = exp2f(m0 - n0), a1 = exp2f(m1 - n1);
#pragma unroll
        for (int ct = 0; ct < 8; ++ct) {
          O[ct][0] *= a0; O[ct][1] *= a1; O[ct][2] *= a0; O[ct][3] *= a1;
        }
        Zc[0] *= a0; Zc[1] *= a1; Zc[2] *= a0; Zc[3] *= a1;
        m0 = n0;
        m1 = n1;
      }
      uint32_t Pt[2][2];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        Pt[mt][0] = movmatrix_trans(pack_half2(exp2f(xl[mt][0] - m0), exp2f(xl[mt][1] - m1)));
        Pt[mt][1] = movmatrix_trans(pack_half2(exp2f(xl[mt][2] - m0), exp2f(xl[mt][3] - m1)));
      }
      const uint32_t ones = (r == 4) ? 0x3C003C00u : 0u;
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) mma_f16(Zc, ones, 0u, ones, 0u, Pt[ks][0], Pt[ks][1]);
      // the key rows are consumed: stage the value rows of these 32 tokens over them
      __syncwarp();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      const int nvv = min(32, rt - j0) - (holds_new ? 1 : 0);
      if (nvv > 0) {
        if (lane == 0) {
          mbar_expect_tx(rbar, (uint32_t)nvv * 256u);
          bulk_g2s(smem_u32(ring), resv + (size_t)j0 * kD, (uint32_t)nvv * 256u, rbar);
        }
        if (!mbar_wait_bounded(rbar, res_phase)) {
          gave_up = true;
          if (lane == 0) atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
          break;
        }
        res_phase ^= 1u;
      }
      if (holds_new) {
        const uint2 vn = reinterpret_cast<const uint2*>(lv.new_v + (size_t)s * kD)[lane];
        reinterpret_cast<uint2*>(ring + (jn - j0) * 256)[lane] = vn;
        reinterpret_cast<uint2*>(lv.resv + (size_t)s * lv.resv_stride + (size_t)jn * 256)[lane] = vn;
        __syncwarp();
      }
      // tile (ct, ks): A = V^T, 16 channels x 16 tokens, from four transposed 8x8 tiles of the token-major rows:
      // matrix i of the ldmatrix has tokens 16ks + 8(i >> 1) .., channels 16ct + 8(i & 1) ..; lane l gives row l % 8 of matrix l / 8
      const uint32_t lm_row = smem_u32(ring) + (uint32_t)((8 * (lane >> 4) + (lane & 7)) * 256 + 16 * ((lane >> 3) & 1));
#pragma unroll
      for (int ct = 0; ct < 8; ++ct) {
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
          uint32_t a0, a1, a2, a3;
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                       : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3)
                       : "r"(lm_row + (uint32_t)(ks * 16 * 256 + ct * 32)));
          // tokens of this lane's pairs: 16ks + 2t, +1 (a0, a1) and 16ks + 8 + 2t, +1 (a2, a3); rows past r are stale
          const int ja = j0 + 16 * ks + 2 * t, jb = ja + 8;
          const uint32_t ma = ja + 1 < rt ? 0xFFFFFFFFu : (ja < rt ? 0x0000FFFFu : 0u);
          const uint32_t mb = jb + 1 < rt ? 0xFFFFFFFFu : (jb < rt ? 0x0000FFFFu : 0u);
          mma_f16(O[ct], bf16x2_to_f16x2(a0 & ma), bf16x2_to_f16x2(a1 & ma), bf16x2_to_f16x2(a2 & mb), bf16x2_to_f16x2(a3 & mb),
                  Pt[ks][0], Pt[ks][1]);
        }
      }
    }

    // ---- finish this warp's split: true scale, zero-point terms, denominator
    if (!o_true_scale) {
#pragma unroll
      for (int ct = 0; ct < 8; ++ct)
#pragma unroll
        for (int j = 0; j < 4; ++j) O[ct][j] *= 1048576.0f;
    }
#pragma unroll
    for (int ct = 0; ct < 8; ++ct) {
      const int vg = ct / TPG;
      const float z0 = __shfl_sync(0xffffffffu, Zc[0], vg * 4 + t), z1 = __shfl_sync(0xffffffffu, Zc[1], vg * 4 + t);
      O[ct][0] += z0; O[ct][1] += z1; O[ct][2] += z0; O[ct][3] += z1;
    }
    const float l0 = __shfl_sync(0xffffffffu, Zc[0], 16 + t), l1 = __shfl_sync(0xffffffffu, Zc[1], 16 + t);

    // ---- merge the warps of the CTA, write the partial of (CTA, stream).  Every warp leaves its (m, l) and its
    // unnormalized output in shared memory, the output in its own, now idle, ring as [8 heads][132] floats; then
    // the 16 threads that own a head add the four warps' rows with the factors 2^(m_w - M).
    if (r == 0) {
      mS[warp * 8 + 2 * t] = m0;
      mS[warp * 8 + 2 * t + 1] = m1;
      lS[warp * 8 + 2 * t] = l0;
      lS[warp * 8 + 2 * t + 1] = l1;
    }
    {
      float* mine = reinterpret_cast<float*>(ring);
#pragma unroll
      for (int ct = 0; ct < 8; ++ct) {
        mine[(2 * t) * kMergeStride + 16 * ct + r] = O[ct][0];
        mine[(2 * t + 1) * kMergeStride + 16 * ct + r] = O[ct][1];
        mine[(2 * t) * kMergeStride + 16 * ct + 8 + r] = O[ct][2];
        mine[(2 * t + 1) * kMergeStride + 16 * ct + 8 + r] = O[ct][3];
      }
    }
    __syncthreads();
    if (threadIdx.x < 128) {
      const int h = threadIdx.x >> 4, c0 = threadIdx.x & 15;
      float M = -INFINITY, L = 0.f, f[kWarps];
#pragma unroll
      for (int w = 0; w < kWarps; ++w) M = fmaxf(M, mS[w * 8 + h]);
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float mw = mS[w * 8 + h];
        f[w] = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
        L += f[w] * lS[w * 8 + h];
      }
      float* part = ws + (size_t)(blockIdx.x + s) * kPartialFloats + h * 130;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int c = c0 + 16 * k;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
          acc += f[w] * reinterpret_cast<const float*>(smem + w * (kStages * kStageBytes))[h * kMergeStride + c];
        part[2 + c] = acc;
      }
      if (c0 == 0) {
        part[0] = M;
        part[1] = L;
      }
    }
    if (seg < ce) {
      // another segment follows: its copies are staged into the rings that were just read
      __syncthreads();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
  }
}

template <int G, int kU4, bool kV4>
cudaError_t launch_v(const LayerView& lv, const __nv_bfloat16* qb, float sl, float* ws, int grid, cudaStream_t stream) {
  // launched with programmatic stream serialization: the kernel itself waits for its predecessor (griddepcontrol.wait)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kWarps * 32);
  cfg.dynamicSmemBytes = smem_bytes(kV4);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attention_mma_kernel<G, kU4, kV4>, lv, qb, sl, ws, 0x44004400u);
}
template <int G, int kU4>
cudaError_t launch_one(const LayerView& lv, const __nv_bfloat16* qb, float sl, float* ws, int grid, cudaStream_t stream) {
  return lv.v_bits == 4 ? launch_v<G, kU4, true>(lv, qb, sl, ws, grid, stream)
                        : launch_v<G, kU4, false>(lv, qb, sl, ws, grid, stream);
}

template <int G>
cudaError_t launch_g(const LayerView& lv, const void* q, float scale, float* ws, int grid, cudaStream_t stream) {
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  const float sl = scale * 1.4426950408889634f;
  if (lv.dense_hi) return launch_one<G, 2>(lv, qb, sl, ws, grid, stream);
  const bool uses_u4 = (lv.budget_bf16 + lv.budget_u4 > 0) ? lv.budget_u4 > 0 : lv.tau_u4 < lv.tau_bf16;
  if (uses_u4) return launch_one<G, 1>(lv, qb, sl, ws, grid, stream);
  return launch_one<G, 0>(lv, qb, sl, ws, grid, stream);
}

}  // namespace

template <int G, int kU4, bool kV4>
static cudaError_t setup_v() {
  cudaError_t e = cudaFuncSetAttribute(attention_mma_kernel<G, kU4, kV4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       smem_bytes(kV4));
  if (e != cudaSuccess) return e;
  // the CTAs of an SM only fit with the largest shared-memory carve-out; ask for it explicitly
  return cudaFuncSetAttribute(attention_mma_kernel<G, kU4, kV4>, cudaFuncAttributePreferredSharedMemoryCarveout,
                              (int)cudaSharedmemCarveoutMaxShared);
}
template <int G, int kU4>
static cudaError_t setup_one() {
  cudaError_t e = setup_v<G, kU4, false>();
  return e != cudaSuccess ? e : setup_v<G, kU4, true>();
}
template <int G>
static cudaError_t setup_g() {
  cudaError_t e = setup_one<G, 0>();
  if (e != cudaSuccess) return e;
  e = setup_one<G, 1>();
  return e != cudaSuccess ? e : setup_one<G, 2>();
}

cudaError_t attention_mma_setup() {
  cudaError_t e = setup_g<32>();
  if (e != cudaSuccess) return e;
  e = setup_g<64>();
  if (e != cudaSuccess) return e;
  return setup_g<128>();
}

// Number of CTAs the split kernel runs for this layer state (also the number of partial-slot owners).
// Split positions per stream: packed units plus the weighted units of the residual window.
long long attention_mma_positions(const LayerView& lv) {
  return (long long)lv.n_blocks * lv.U + (long long)kResidualWeight * ((lv.r + 31) / 32 + (lv.n_sink + 31) / 32);
}

// Number of CTAs the split kernel runs for this layer state (also the number of partial-slot owners).  When there are
// fewer streams than CTA slots the grid is a multiple of the stream count, so that no CTA straddles two streams
// (a second segment costs a pipeline drain, a query load and a second partial).
int attention_mma_grid(const LayerView& lv, int n_sms) {
  const int S = lv.B * lv.Hkv;
  const long long total = attention_mma_positions(lv) * S;
  int grid = (int)min((long long)min(n_sms * (lv.dense_hi ? kCtasPerSmDense : kCtasPerSm), kMaxCtas / 2), total);
  if (grid > S) grid = grid / S * S;
  return grid < 1 ? 1 : grid;
}

cudaError_t launch_attention_mma(const LayerView& lv, const void* q, float* out, float scale, float* ws, int n_sms,
                                 cudaStream_t stream, int* launches) {
  const int S = lv.B * lv.Hkv;
  const long long Us = attention_mma_positions(lv);
  const int grid = attention_mma_grid(lv, n_sms);
  cudaError_t e;
  if (lv.G == 32) e = launch_g<32>(lv, q, scale, ws, grid, stream);
  else if (lv.G == 64) e = launch_g<64>(lv, q, scale, ws, grid, stream);
  else e = launch_g<128>(lv, q, scale, ws, grid, stream);
  *launches = 1;
  if (e != cudaSuccess || out == nullptr) return e;     // out == nullptr: split kernel only (timing)
  e = launch_combine(ws, out, lv.g, lv.Hkv, lv.Hq, 1, grid, Us, S, stream);
  *launches = 2;
  return e;
}

}  // namespace mixkvq
