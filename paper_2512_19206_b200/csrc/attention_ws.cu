// Fused split-K GQA decode attention over the mixed-precision cache (Eq. 1 with Eq. 3 applied on the fly),
// warp-specialised form.
//
// Work unit = 32 tokens of one stream.  All units of all streams are split evenly over the CTAs; inside a CTA they
// are split over PAIRS of warps.  A pair shares one ring of staged units (1-D bulk copies signalled on mbarriers):
//
//   the logits warp   expands the unit's 2-bit key codes into tensor-core A fragments (one logic op and one fp16 FMA
//                     per pair of codes: A = c*s, exact in fp16) and runs q.K^T on mma.sync m16n8k16 tiles with the g
//                     query heads of the KV head as the N dimension.  The zero-point term q.z of the key group (one
//                     extra tile chain per group) is the initial value of the accumulators; the promoted (BF16)
//                     channels and the UINT4 high plane are further tiles.  The unit's 32 x 8 logits go to the
//                     partner through shared memory.
//   the values warp   keeps the online softmax (lazily raised reference maximum), builds the unit's value-scale tables,
//                     folds the value scales into the probabilities and runs P.V with the raw value codes as fp16
//                     subnormals in the A operand (one logic op per pair of codes); value zero-points and the softmax
//                     denominator ride on one extra tile.  It owns the output accumulators and refills the ring.
//
// Neither warp holds the other's state, so both need far fewer registers than a warp that does everything, more warps
// fit an SM, and the logits of unit n+1 overlap the values of unit n.  The packed layout stores the codes in A-fragment
// order: a lane's 16-byte shared-memory load is exactly its registers; nothing dequantized is ever written back to
// shared memory.  Unquantized units (residual window, sink) are read straight from global memory in bf16 and are taken
// first, while the first staged copies are in flight.
#include "common.cuh"

namespace mixkvq {

cudaError_t launch_combine(const float* ws, float* out, int g, int Hkv, int Hq, int mode, int n,
                           long long units_per_stream, int S, cudaStream_t stream, const int4* seq = nullptr,
                           const int* seq_prefix = nullptr, float* lse_out = nullptr);

namespace {

#ifndef MIXKVQ_WS_PAIRS
#define MIXKVQ_WS_PAIRS 4
#define MIXKVQ_WS_CTAS 2
#endif
constexpr int kPairs = MIXKVQ_WS_PAIRS;      // warp pairs per CTA
constexpr int kThreads = kPairs * 64;
constexpr int kCtasPerSm = MIXKVQ_WS_CTAS;
constexpr int kStages = 4;                   // ring stages per pair (a power of two)
// one ring stage: a key-meta group (512 B) followed by the unit (<= 2560 B; <= 3584 B with 4-bit values), as in the block
__host__ __device__ constexpr int stage_bytes(bool v4) { return v4 ? 4096 : 3072; }
constexpr int kKeyMetaOff = 0;
constexpr int kUnitOff = 512;
// per-pair tables: key scales {s, -4s} (576) | key zero-point tiles (576) | value scales (320) | value zero-point tile (1088)
constexpr int kKprepOff = 0, kZprepOff = 576, kSvpOff = 1152, kZvpOff = 1472, kPrepBytes = 2560;
// hand-over of a unit's logits: 32 bytes per lane, then 8 bytes per lane with the zero-point term of the unit's key
// group; one buffer per ring stage and one for unquantized units
constexpr int kLBufBytes = 1280, kLBufZeroOff = 1024;
__host__ __device__ constexpr int pair_bytes(bool v4) {
  return kStages * stage_bytes(v4) + kPrepBytes + (kStages + 1) * kLBufBytes;
}
// mbarriers of a pair: staged copy landed [kStages], logits ready [kStages], then for unquantized units: ready, taken
constexpr int kBarsPerPair = 2 * kStages + 2;
constexpr int kQS = 136;                     // halves per row of the query tables (272 bytes: rows fall on different banks)
constexpr int kBarBytes = ((kPairs * kBarsPerPair * 8 + 127) / 128) * 128;
constexpr int kPrefixBytes = ((kMaxRaggedBatch + 1) * 4 + 15) / 16 * 16;     // a ragged batch's prefix sums
constexpr int kSharedTail = kBarBytes + 2 * 8 * kQS * 2 + 2 * kPairs * 32 + kPrefixBytes;
__host__ __device__ constexpr int smem_bytes(bool v4) { return kPairs * pair_bytes(v4) + kSharedTail; }
constexpr int kResidualWeight = 3;           // an unquantized 32-token unit counts as this many packed units in the split
constexpr int kMergeStride = 132;            // floats per head row of a pair's output in the merge
// With three tiers and with a 4-bit base the logits warp is by far the longer role (further tiles for the UINT4 high
// plane, or a second key pass): the promoted channels' tile is then the values warp's work.  With two tiers it stays with
// the logits warp: a stall of the values warp on global loads delays the ring's refill, which costs more there than the
// tile does.  (The gathered UINT4 tiles stay with the logits warp in every case: moved, they made the values warp the
// longer role and the kernel slower.)
__host__ __device__ constexpr bool promoted_in_values(int u4) { return u4 != 0; }
constexpr float kMaxSlack = 3.0f;            // a packed unit's probabilities are at most 2^kMaxSlack (log2 domain)
// A wait on a barrier polls at most this many times; a poll suspends the thread for up to about a microsecond, so
// the wait gives up after about two seconds at the latest (a few milliseconds if the polls return at once).
constexpr uint32_t kWaitPolls = 1u << 21;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
// Polls a phase of a barrier up to max_polls times; false if it never completed.
__device__ __forceinline__ bool mbar_wait_polls(uint32_t bar, uint32_t parity, uint32_t max_polls) {
  uint32_t ok;
  asm volatile(
      "{\n\t"
      ".reg .pred p, q;\n\t"
      ".reg .u32 n;\n\t"
      "mov.u32 n, 0;\n"
      "MIXKVQ_WAIT:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 1000;\n\t"
      "@p bra MIXKVQ_DONE;\n\t"
      "add.u32 n, n, 1;\n\t"
      "setp.lt.u32 q, n, %3;\n\t"
      "@q bra MIXKVQ_WAIT;\n"
      "MIXKVQ_DONE:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t"
      "}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(max_polls)
      : "memory");
  return ok != 0;
}
// one lane of the (converged) warp arrives on the barrier
__device__ __forceinline__ void mbar_arrive_one(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\t@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(bar)
      : "memory");
}
// one lane of the (converged) warp stages `bytes` from global memory at shared address dst and arms the barrier for
// bytes + extra (extra > 0 only in the test of the give-up path); nothing happens when `enabled` is 0
__device__ __forceinline__ void stage_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint32_t extra,
                                           uint32_t enabled) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .u32 tx;\n\t"
      "setp.ne.u32 e, %5, 0;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "and.pred p, p, e;\n\t"
      "add.u32 tx, %2, %4;\n\t"
      "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%3], tx;\n\t"
      "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n\t"
      "}" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "r"(extra), "r"(enabled)
      : "memory");
}
// the same for a unit whose key-group scales do not lie directly before it: two copies on one barrier
__device__ __forceinline__ void stage_copy2(uint32_t dst_a, const void* src_a, uint32_t bytes_a, uint32_t dst_b,
                                            const void* src_b, uint32_t bytes_b, uint32_t bar, uint32_t extra) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .u32 tx;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "add.u32 tx, %2, %5;\n\t"
      "add.u32 tx, tx, %7;\n\t"
      "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%6], tx;\n\t"
      "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%6];\n\t"
      "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%3], [%4], %5, [%6];\n\t"
      "}" ::"r"(dst_a),
      "l"(src_a), "r"(bytes_a), "r"(dst_b), "l"(src_b), "r"(bytes_b), "r"(bar), "r"(extra)
      : "memory");
}
// shared-memory accesses by 32-bit shared address (the offsets added at the call sites fold into the instruction)
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t a) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t a, uint32_t x, uint32_t y) {
  asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(a), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t x) {
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(x) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t a, uint32_t x) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"((uint16_t)x) : "memory");
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
// 2^x by the special-function unit alone (no range fix-up): inputs here are <= kMaxSlack or -inf
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_bf162(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
// two bf16 in one word -> two fp16 in one word (exact inside the fp16 range)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) { return pack_half2(bf_lo(w), bf_hi(w)); }

// Byte offset of (k-tile kt, lane column t) in the key-scale table: 16 bytes {s_a, -4 s_a, s_b, -4 s_b} (half2 each: the
// lane's channel pairs 16kt + 2t, +1 and 16kt + 8 + 2t, +1); 16 bytes of padding after every second k-tile keep the
// preparation's stores free of bank conflicts.
__device__ __forceinline__ constexpr int kprep_off(int kt, int t) { return 144 * (kt >> 1) + 64 * (kt & 1) + 16 * t; }
// First 32-bit word of k-tile kt in the zero-point tile table (16 words per k-tile, four extra every second k-tile).
__device__ __forceinline__ constexpr int zprep_word(int kt) { return 16 * kt + 4 * (kt >> 1); }
// Bit position (inside each 16-bit half, after the shift below) of k-tile kt's 2-bit field.
__device__ __forceinline__ constexpr int key_pos(int kt) { return (0x86486464u >> (4 * kt)) & 0xF; }
// k-tiles 0,1 are read from (w << 4), 2..4 from w, 5..7 from (w >> 6)
__device__ __forceinline__ uint32_t key_shift(uint32_t w, int kt) { return kt < 2 ? (w << 4) : (kt < 5 ? w : (w >> 6)); }

// warp w of the CTA: pair w / 2; the logits warps are spread evenly over the four schedulers of the SM (w mod 4)
__device__ __forceinline__ bool is_logits_warp(int warp) { return ((warp ^ (warp >> 2)) & 1) == 0; }

// kU4: how the configuration can use the UINT4 tier: 0 = never (tau_u4 >= tau_bf16), 1 = some channels (high plane stored
// per channel pair, gathered), 2 = 4-bit base (dense high plane)
// kV4: 4-bit values (a second plane of 2-bit value codes per unit, scale 4 s_v)
template <int G, int kU4, bool kV4>
#ifdef MIXKVQ_WS_MAXNREG
__global__ void __maxnreg__(MIXKVQ_WS_MAXNREG)
#else
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
#endif
attention_ws_kernel(LayerView lv, const __nv_bfloat16* __restrict__ q, float scale_log2e, float* __restrict__ ws,
                    uint32_t four2) {
  constexpr int VG = kD / G;              // value groups per token
  constexpr int TPG = 8 / VG;             // 16-channel tiles per value group
  constexpr int kStageBytes = stage_bytes(kV4);
  constexpr int kPairBytes = pair_bytes(kV4);
  constexpr int kPrepBase = kStages * kStageBytes;             // offsets inside a pair's shared memory
  constexpr int kLBufBase = kPrepBase + kPrepBytes;
  constexpr int kRBufBase = kLBufBase + kStages * kLBufBytes;
  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, r = lane >> 2, t = lane & 3;
  const int pair = warp >> 1;
  const bool logits_role = is_logits_warp(warp);

  const uint32_t smem_base = smem_u32(smem);
  const uint32_t ring_u32 = smem_base + pair * kPairBytes;                  // the pair's shared memory starts with its ring
  const uint32_t tail_u32 = smem_base + kPairs * kPairBytes;
  const uint32_t bar_u32 = tail_u32 + pair * (kBarsPerPair * 8);            // staged copy landed [kStages]
  const uint32_t lfull_u32 = bar_u32 + kStages * 8;                         // logits ready [kStages]
  const uint32_t rfull_u32 = bar_u32 + 2 * kStages * 8, rempty_u32 = rfull_u32 + 8;
  const uint32_t qb16_u32 = tail_u32 + kBarBytes;                           // [8][kQS] q, bf16 bits (0 for heads >= g)
  const uint32_t qf16_u32 = qb16_u32 + 8 * kQS * 2;                         // [8][kQS] q, fp16
  float* mS = reinterpret_cast<float*>(smem + kPairs * kPairBytes + kBarBytes + 2 * 8 * kQS * 2);    // [kPairs][8]
  float* lS = mS + kPairs * 8;                                                                       // [kPairs][8]
  int* prefS = reinterpret_cast<int*>(lS + kPairs * 8);                     // ragged batch: seq_prefix[0 .. B]

  if (threadIdx.x < kPairs * kBarsPerPair) {
    mbar_init(tail_u32 + 8 * threadIdx.x, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (!logits_role) {
    // constant rows of the zero-point / denominator tile: row 4 is all ones, the other rows >= VG stay zero
#pragma unroll
    for (int i = 0; i < 9; ++i) {
      const int idx = lane + 32 * i, rem = idx % 144, row = rem >> 4;      // [2 ks: 144 words][8 rows][4 t][4]
      if (idx < 272) sts32(ring_u32 + kPrepBase + kZvpOff + 4 * idx, (row == 4 && (idx & 1) == 0) ? 0x3C003C00u : 0u);
    }
  }
  __syncthreads();

  // codes of 32 tokens: keys 1024, values 1024, value scales (and the values' high plane 1024)
  constexpr uint32_t kUnitBytes = 2048u + 128u * (kD / G) + (kV4 ? 1024u : 0u);
  constexpr int UPG = G / 32;                                 // units per key group

  const int S = lv.B * lv.Hkv, U = lv.U, g = lv.g;
  // Fill of the stream at hand: the same for every stream, or (ragged batch) taken per sequence from the table in
  // device memory at the start of every segment.
  int f_nb = lv.n_blocks, f_r = lv.r, f_ns = lv.n_sink;
  int packed_units = f_nb * U;
  // unquantized 32-token units: those of the residual window, then those of the sink
  int res_units = (f_r + 31) / 32, bf16_units = res_units + (f_ns + 31) / 32;
  int Us = packed_units + kResidualWeight * bf16_units;             // split positions; an unquantized unit spans several

  // Programmatic dependent launch: the grid may have been started while the kernel before it in the stream was still
  // running.  Nothing above touches global memory.  dep_wait() waits for that kernel's results and lets the kernel after
  // this one be started early in the same way; every thread calls it before its first access to global memory, with one
  // exception: when the host knows that the kernel before this one did not write this layer's packed blocks
  // (stage_early), the first staged copies of the packed units go out before the wait.  That is safe because a kernel
  // of this library triggers its successor only after its own wait, so that everything two launches back is complete.
  bool dep_waited = false;
  auto dep_wait = [&]() {
    if (!dep_waited) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      dep_waited = true;
    }
  };
  if (!lv.stage_early || lv.seq != nullptr) dep_wait();     // the table of a ragged batch is read right below
  if (lv.seq != nullptr) {
    // the prefix sums go to shared memory in one round trip: the segments below search them
    for (int i = threadIdx.x; i <= lv.B; i += kThreads) prefS[i] = lv.seq_prefix[i];
    __syncthreads();
  }
  const long long total = lv.seq != nullptr ? (long long)prefS[lv.B] : (long long)Us * S;
  const long long cb = split_begin(total, gridDim.x, blockIdx.x), ce = split_begin(total, gridDim.x, blockIdx.x + 1);

  uint32_t ring_stage = 0;        // ring stage of the next packed unit this pair consumes
  uint32_t ring_parity = 0;       // phase parity of that stage's barriers
  uint32_t rit = 0;               // unquantized units handed over by this pair so far (both warps count them alike)
  bool gave_up = false;
  // A wait that runs out sets gave_up; the warp carries on with whatever the shared memory holds (every address it
  // forms stays inside the CTA's shared memory and the stream's arrays), its later waits are skipped, and the pair's
  // result is replaced by zeros at the end.  Straight-line code: no exit in the middle of a unit.
  auto wait_or_give_up = [&](uint32_t bar, uint32_t parity) {
    if (!gave_up && !mbar_wait_polls(bar, parity, lv.wait_polls ? lv.wait_polls : kWaitPolls)) gave_up = true;
  };
  auto advance_stage = [&]() {
    ring_stage = (ring_stage + 1u) & (kStages - 1);
    ring_parity ^= (ring_stage == 0u) ? 1u : 0u;
  };

  for (long long seg = cb; seg < ce;) {
    int s, ub, ue;
    if (lv.seq != nullptr) {
      // ragged batch: the sequence whose positions hold seg (sequences without positions are stepped over)
      int b = 0;
      while (b + 1 < lv.B && (long long)prefS[b + 1] <= seg) ++b;
      const int4 f = lv.seq[b];
      f_nb = f.x; f_r = f.y; f_ns = f.z; Us = f.w;
      packed_units = f_nb * U;
      res_units = (f_r + 31) / 32;
      bf16_units = res_units + (f_ns + 31) / 32;
      const long long rel = seg - (long long)prefS[b];
      const int hk = (int)(rel / Us);
      s = b * lv.Hkv + hk;
      ub = (int)(rel - (long long)hk * Us);
      ue = (int)min((long long)Us, ce - (long long)prefS[b] - (long long)hk * Us);
    } else {
      s = (int)(seg / Us);
      ub = (int)(seg - (long long)s * Us);
      ue = (int)min((long long)Us, ce - (long long)s * Us);
    }
    seg += ue - ub;
    // ---- this pair's share of the segment.  The unquantized units of the segment go to different pairs (unit i to
    // pair kPairs - 1 - i % kPairs); the packed units are split in order so that every pair carries about the same weight.
    const int pk_b = min(ub, packed_units), pk_e = min(ue, packed_units);
    const int res_b = (max(ub, packed_units) - packed_units + kResidualWeight - 1) / kResidualWeight;
    const int res_e = ue > packed_units ? (ue - packed_units + kResidualWeight - 1) / kResidualWeight : res_b;
    const int n_res = res_e - res_b;
    int wb = pk_b, we = pk_b;
    {
      const int weight = (pk_e - pk_b) + kResidualWeight * n_res;
      int remaining = pk_e - pk_b;
#pragma unroll
      for (int w = 0; w < kPairs; ++w) {
        const int share = weight * (w + 1) / kPairs - weight * w / kPairs;       // weight < 2^24: 32-bit arithmetic
        const int first_i = kPairs - 1 - w;                                   // unquantized units first_i, first_i + kPairs, ...
        const int res_w = n_res > first_i ? (n_res - first_i + kPairs - 1) / kPairs : 0;
        int p = min(remaining, max(0, share - kResidualWeight * res_w));
        if (w == kPairs - 1) p = remaining;
        if (w == pair) {
          wb = pk_e - remaining;
          we = wb + p;
        }
        remaining -= p;
      }
    }
    const int n_pack = we - wb;

    // ---- the first copies of this segment go out before anything else (values warp): they do not depend on the query.
    // The packed units of a stream are one uniform sequence (a group's scales, then its units), whatever the block size,
    // so the copy source only ever moves forward: `isrc` is the next unit to stage, `ig` its index inside its key group.
    int issued = 0;
    const char* isrc = lv.base + (size_t)s * lv.base_stride + (size_t)wb * kUnitBytes + 512u * (size_t)(wb / UPG + 1);
    int ig = wb & (UPG - 1);
    // stages the next unit (if there is one left) in ring stage sg; all lanes keep the position
    auto issue = [&](uint32_t sg, bool first) {
      const uint32_t dst = ring_u32 + sg * kStageBytes, bar = bar_u32 + sg * 8u;
      const uint32_t enabled = issued < n_pack ? 1u : 0u;
      if (UPG == 1) {
        // the group's scales lie directly before the unit: one copy
        stage_copy(dst + kKeyMetaOff, isrc - 512, 512u + kUnitBytes, bar, first ? lv.debug_extra_tx : 0u, enabled);
        isrc += kUnitBytes + 512;
      } else {
        if (enabled) {
          if (ig == 0) stage_copy(dst + kKeyMetaOff, isrc - 512, 512u + kUnitBytes, bar, first ? lv.debug_extra_tx : 0u, 1u);
          else if (first)
            stage_copy2(dst + kUnitOff, isrc, kUnitBytes, dst + kKeyMetaOff, isrc - (size_t)ig * kUnitBytes - 512, 512u, bar,
                        lv.debug_extra_tx);
          else stage_copy(dst + kUnitOff, isrc, kUnitBytes, bar, 0u, 1u);
        }
        isrc += kUnitBytes;
        ig = (ig + 1) & (UPG - 1);
        if (ig == 0) isrc += 512;
      }
      issued += (int)enabled;
    };
    const uint32_t stage0 = ring_stage, parity0 = ring_parity;
    // the logits warp's first block: its table entry and the head of its extras (the lists of promoted channels) are a
    // chain of two dependent loads; they go out here, with the first copies
    const char* extras = lv.extras + (size_t)s * lv.extras_stride;
    const uint2* table = reinterpret_cast<const uint2*>(lv.table + (size_t)s * lv.table_stride);
    uint2 pf_entry = make_uint2(0u, 0u), pf_entry_next = make_uint2(0u, 0u);
    uint4 pf_head = make_uint4(~0u, ~0u, ~0u, ~0u);
    uint32_t pf_ids[4] = {0xFFFFu, 0xFFFFu, 0xFFFFu, 0xFFFFu};   // three tiers: the lane's four pairs of UINT4 channel numbers
    // the channel lists of the block with table entry e: the head of its extras and (three tiers) the UINT4 channel
    // numbers of the lane's pairs t, t + 4, t + 8, t + 12
    auto request_lists = [&](const uint2& e) {
      if (e.y & 0xFFFFu) {
        const char* ex = extras + (size_t)e.x * 16;
        pf_head = *reinterpret_cast<const uint4*>(ex);
        if constexpr (kU4 == 1) {
          const int n16p = ((e.y & 0xFF) + 1) >> 1, n4pairs = (((e.y >> 8) & 0xFF) + 1) >> 1;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int p = 4 * i + (lane & 3);
            pf_ids[i] = p < n4pairs ? (uint32_t)*reinterpret_cast<const uint16_t*>(ex + 2 * n16p + 2 * p) : 0xFFFFu;
          }
        }
      }
    };
    if (!logits_role) {
#pragma unroll 1
      for (int i = 0; i < kStages; ++i) issue((ring_stage + i) & (kStages - 1), i == 0);
    }
    if (n_pack > 0 && lv.stage_early && (logits_role || promoted_in_values(kU4))) {
      pf_entry = table[wb / U];
      if (wb / U + 1 < f_nb) pf_entry_next = table[wb / U + 1];
      if (logits_role ? kU4 != 2 : promoted_in_values(kU4)) request_lists(pf_entry);     // whoever needs the lists
    }
    dep_wait();

    // ---- query of this stream: bf16 and fp16 tables (heads >= g are zero rows)
    {
      uint4 q_regs = make_uint4(0u, 0u, 0u, 0u);      // thread (h, c) of the first 128: head h, channels 8c .. 8c+7
      const int b = s / lv.Hkv, hk = s % lv.Hkv, h = threadIdx.x >> 4, c = threadIdx.x & 15;
      if (h < g) q_regs = *reinterpret_cast<const uint4*>(q + ((size_t)b * lv.Hq + hk * g + h) * kD + 8 * c);
      __syncthreads();          // the previous segment's readers of the tables are done
      if (h < 8) {
        sts128(qb16_u32 + (h * kQS + 8 * c) * 2, q_regs.x, q_regs.y, q_regs.z, q_regs.w);
        if (kU4 == 1)      // the fp16 table is for the gathered UINT4 channels
          sts128(qf16_u32 + (h * kQS + 8 * c) * 2, bf16x2_to_f16x2(q_regs.x), bf16x2_to_f16x2(q_regs.y),
                 bf16x2_to_f16x2(q_regs.z), bf16x2_to_f16x2(q_regs.w));
      }
      __syncthreads();
    }

    // unquantized units of this pair: first_res, first_res + kPairs, ... < n_res
    const int first_res = kPairs - 1 - pair;
    // fused decode step: the newest token (slot r - 1) is not in the residual store yet; the pair whose unit holds it
    // takes its rows from the step's tensors, stores them and updates the importance accumulator
    const int jn = f_r - 1;

    if (logits_role) {
      // =====================================================================================================
      // logits warp
      // =====================================================================================================
      const uint32_t qrow_u32 = qb16_u32 + r * (kQS * 2), qfrow_u32 = qf16_u32 + r * (kQS * 2);
      // ---- unquantized units: bf16 keys straight from global memory.  The channel a k-slot stands for is free as long as
      // both operands agree: lane column t of k-tile 2j (2j+1) takes channels 32j + 8t + 0..3 (4..7), so that a lane's
      // four k-tiles' worth of a token row is one 16-byte load.
      for (int ri = first_res; ri < n_res; ri += kPairs) {
        const int bu = res_b + ri;                        // unquantized unit: residual window first, then the sink
        const bool in_sink = bu >= res_units;
        const int wu = in_sink ? bu - res_units : bu;     // unit inside its window
        const int rt = in_sink ? f_ns : f_r;        // tokens in that window
        const int j0 = wu * 32;
        const char* resk = in_sink ? lv.sink + (size_t)s * lv.sink_stride : lv.resk + (size_t)s * lv.resk_stride;
        const bool holds_new = !in_sink && lv.new_k != nullptr && jn >= j0 && jn < j0 + 32;
        float Sx[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          const int ta = j0 + mt * 16 + r, tb = ta + 8;
          const uint4* rowa = reinterpret_cast<const uint4*>(resk + (size_t)ta * 256);
          const uint4* rowb = reinterpret_cast<const uint4*>(resk + (size_t)tb * 256);
          if (holds_new && ta == jn) rowa = reinterpret_cast<const uint4*>(lv.new_k + (size_t)s * kD);
          if (holds_new && tb == jn) rowb = reinterpret_cast<const uint4*>(lv.new_k + (size_t)s * kD);
          uint4 ka[4], kb[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            ka[j] = ta < rt ? rowa[4 * j + t] : make_uint4(0u, 0u, 0u, 0u);
            kb[j] = tb < rt ? rowb[4 * j + t] : make_uint4(0u, 0u, 0u, 0u);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint4 qq = lds128(qrow_u32 + (32 * j + 8 * t) * 2);
            mma_bf16(Sx[mt], ka[j].x, kb[j].x, ka[j].y, kb[j].y, qq.x, qq.y);
            mma_bf16(Sx[mt], ka[j].z, kb[j].z, ka[j].w, kb[j].w, qq.z, qq.w);
          }
        }
        if (holds_new) {
          // store the new key row and add |q| to the importance accumulator (channels 4*lane .. 4*lane+3, heads
          // ascending: the order of the plain append)
          const uint2 kn = reinterpret_cast<const uint2*>(lv.new_k + (size_t)s * kD)[lane];
          reinterpret_cast<uint2*>(lv.resk + (size_t)s * lv.resk_stride + (size_t)jn * 256)[lane] = kn;
          double* acc = reinterpret_cast<double*>(lv.state + (size_t)s * lv.state_stride);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int d = 4 * lane + c;
            double a = acc[d];
            for (int h = 0; h < g; ++h) a = __dadd_rn(a, (double)fabsf(__uint_as_float(lds16(qb16_u32 + (h * kQS + d) * 2) << 16)));
            acc[d] = a;
          }
          if (lane == 0) *reinterpret_cast<uint32_t*>(lv.state + (size_t)s * lv.state_stride + 1024) += (uint32_t)g;
        }
        // hand over (the buffer is free once the partner has taken the previous unquantized unit)
        wait_or_give_up(rempty_u32, (rit & 1u) ^ 1u);
        const uint32_t rb = ring_u32 + kRBufBase + lane * 32;
        sts128(rb, __float_as_uint(Sx[0][0]), __float_as_uint(Sx[0][1]), __float_as_uint(Sx[0][2]), __float_as_uint(Sx[0][3]));
        sts128(rb + 16, __float_as_uint(Sx[1][0]), __float_as_uint(Sx[1][1]), __float_as_uint(Sx[1][2]), __float_as_uint(Sx[1][3]));
        __syncwarp();
        mbar_arrive_one(rfull_u32);
        ++rit;
      }

      // ---- packed units
      int bi = 0, u = 0;                     // block and unit inside it of the next unit to consume
      if (n_pack > 0) {
        bi = wb / U;
        u = wb - bi * U;
        if (!lv.stage_early) {
          pf_entry = table[bi];
          if (bi + 1 < f_nb) pf_entry_next = table[bi + 1];
          if constexpr (kU4 != 2) request_lists(pf_entry);
        }
      }
      // B fragments of q for the base key tiles: head r, channels 16kt + {2t, 2t+1} and {2t+8, 2t+9}, times mult(kt)
      uint32_t bq[8][2];
#pragma unroll
      for (int kt = 0; kt < 8; ++kt) {
        const float mult = (float)(1 << (8 - key_pos(kt)));
#pragma unroll
        for (int hch = 0; hch < 2; ++hch) {
          const uint32_t w = lds32(qrow_u32 + (16 * kt + 8 * hch + 2 * t) * 2);
          bq[kt][hch] = pack_half2(bf_lo(w) * mult, bf_hi(w) * mult);
        }
      }
      // per-lane constants of the key-group preparation: the lane converts channels 4*lane .. 4*lane+3 (k-tile lane / 4)
      const float pk_zs = __uint_as_float((119u + (uint32_t)key_pos(lane >> 2)) << 23);        // 2^(pos - 8)
      // zero-point tiles: [8 kt][4 t]{z ch0, z ch0, z ch1, z ch1} half2 z / mult; the lane's first pair
      const uint32_t zp_wr = ring_u32 + kPrepBase + kZprepOff + 4 * (zprep_word(lane >> 2) + 8 * (lane & 1) + ((lane & 3) >> 1) * 2);
      const uint32_t kp_wr = ring_u32 + kPrepBase + kKprepOff + kprep_off(lane >> 2, 2 * (lane & 1)) + 8 * ((lane >> 1) & 1);
      const uint32_t kp_rd = ring_u32 + kPrepBase + kKprepOff + 16 * t;
      const uint32_t zp_rd = ring_u32 + kPrepBase + kZprepOff + 16 * t;
      const uint32_t lane16 = ring_u32 + lane * 16, lane32 = ring_u32 + kLBufBase + lane * 32;
      const uint32_t lane8 = ring_u32 + kLBufBase + kLBufZeroOff + lane * 8;
      // byte offset inside the scale table of channel c's scale (half)
      auto scale_byte = [&](uint32_t c) -> uint32_t {
        const int kt = c >> 4, col = c & 15;
        return c < 128 ? (uint32_t)(kprep_off(kt, (col & 7) >> 1) + 8 * (col >> 3) + 2 * (col & 1)) : 0xFFFFu;
      };
      float zc[4] = {0.f, 0.f, 0.f, 0.f};   // zero-point term q . z of the current key group (every row the same)

      int done = 0;
      while (done < n_pack) {
        // ---- a block: its table entry, its promoted channels' query entries
        const uint2 entry = pf_entry;
        const uint4 head = pf_head;              // the first 16 bytes of the block's extras: up to 8 pairs of promoted channels
        const uint32_t ids[4] = {pf_ids[0], pf_ids[1], pf_ids[2], pf_ids[3]};
        // Everything a block needs from global memory before its first unit was requested a whole block earlier: here
        // go out the lists of block bi + 1 (its table entry arrived during the block before) and the entry of bi + 2.
        pf_entry = pf_entry_next;
        if constexpr (kU4 != 2) {          // the UINT4 channel numbers (three tiers) or the promoted channels' (two tiers)
          if (bi + 1 < f_nb) request_lists(pf_entry);
        }
        if (bi + 2 < f_nb) pf_entry_next = table[bi + 2];
        const int n16 = entry.y & 0xFF, n4 = (entry.y >> 8) & 0xFF, n16p = (n16 + 1) >> 1;
        const char* ex = extras + (size_t)entry.x * 16;                       // the block's extras
        const uint32_t ex_unit = extras_unit_bytes(n16, n4, kU4 == 2);
        const char* exu = ex + extras_header_bytes(n16, n4) + (size_t)u * ex_unit;   // ... of the current unit
        const int nu = min(U - u, n_pack - done);                                 // units of this block for this warp
        // B fragments of the block's first 16 promoted channels (gathered query entries; 0 past the block's count)
        uint32_t xb0 = 0u, xb1 = 0u;
        // A fragments of the first 16 promoted channels of a unit: lane (r, t) holds channel pairs t and t + 4 for tokens
        // r, r + 8 of both m-tiles.  Pairs past the block's count read an existing pair instead (their query entries are 0).
        uint32_t xa[2][4] = {{0u, 0u, 0u, 0u}, {0u, 0u, 0u, 0u}};
        const int xa_lo = (min(t, n16p - 1) * 32 + r) * 4, xa_hi = (min(t + 4, n16p - 1) * 32 + r) * 4;
        auto load_xa = [&](const char* e) {
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            xa[mt][0] = *reinterpret_cast<const uint32_t*>(e + xa_lo + mt * 64);
            xa[mt][1] = *reinterpret_cast<const uint32_t*>(e + xa_lo + mt * 64 + 32);
            xa[mt][2] = *reinterpret_cast<const uint32_t*>(e + xa_hi + mt * 64);
            xa[mt][3] = *reinterpret_cast<const uint32_t*>(e + xa_hi + mt * 64 + 32);
          }
        };
        if (!promoted_in_values(kU4) && n16 > 0) {
          load_xa(exu);
          auto gather_q = [&](int p, uint32_t word) -> uint32_t {       // pair p < 8: its two channel numbers are in `word`
            if (p >= n16p) return 0u;
            const uint32_t ids = word >> (16 * (p & 1));
            const uint32_t c0 = ids & 0xFF, c1 = (ids >> 8) & 0xFF;
            const uint32_t lo = (c0 < 128) ? lds16(qrow_u32 + 2 * c0) : 0u, hi = (c1 < 128) ? lds16(qrow_u32 + 2 * c1) : 0u;
            return lo | (hi << 16);
          };
          xb0 = gather_q(t, (t & 2) ? head.y : head.x);
          xb1 = gather_q(t + 4, (t & 2) ? head.w : head.z);
        }
        // the block's first 32 UINT4 channels (two tiles of eight pairs): B fragments (gathered fp16 query pairs) and, per
        // pair, where the two channels' scales sit in the scale table (byte offset of the half, 0xFFFF: no channel)
        uint32_t u4q[2][2] = {{0u, 0u}, {0u, 0u}}, u4s[2][2] = {{~0u, ~0u}, {~0u, ~0u}};
        if (kU4 == 1 && n4 > 0) {
#pragma unroll
          for (int kk = 0; kk < 2; ++kk)
#pragma unroll
            for (int hp = 0; hp < 2; ++hp) {
              // pair 8 kk + 4 hp + t: its channel numbers were requested a block ahead (0xFF: no channel)
              const uint32_t c0 = ids[2 * kk + hp] & 0xFFu, c1 = ids[2 * kk + hp] >> 8;
              const uint32_t q0 = c0 < 128 ? lds16(qfrow_u32 + 2 * c0) : 0u;
              const uint32_t q1 = c1 < 128 ? lds16(qfrow_u32 + 2 * c1) : 0u;
              u4q[kk][hp] = q0 | (q1 << 16);
              u4s[kk][hp] = scale_byte(c0) | (scale_byte(c1) << 16);
            }
        }

        // The UINT4 high-plane words of a unit's first two tiles (three tiers) are requested one unit ahead inside a block.
        uint32_t u4n[2][2] = {{0u, 0u}, {0u, 0u}};
        auto request_plane = [&](const char* e) {
          if constexpr (kU4 == 1) {
            if (n4 > 0) {
              const int n4pairs = (n4 + 1) >> 1;
              const uint32_t* hw = reinterpret_cast<const uint32_t*>(e + 128 * n16p);
#pragma unroll
              for (int kk = 0; kk < 2; ++kk)
#pragma unroll
                for (int hp = 0; hp < 2; ++hp) {
                  const int pp = 8 * kk + 4 * hp + t;
                  u4n[kk][hp] = pp < n4pairs ? hw[pp * 4 + (r & 3)] : 0u;
                }
            }
          }
        };
        if constexpr (kU4 == 1) request_plane(exu);

#pragma unroll 1
        for (int iu = 0; iu < nu; ++iu) {
          wait_or_give_up(bar_u32 + ring_stage * 8u, ring_parity);
          const uint32_t stg = lane16 + ring_stage * kStageBytes;         // this lane's 16 bytes of the stage's first section
          const bool has_meta = (UPG == 1) || (done + iu == 0) || (((u + iu) & (UPG - 1)) == 0);
          // this unit's UINT4 high-plane words (requested a unit ago); the next unit's are requested right away
          const uint32_t u4w[2][2] = {{u4n[0][0], u4n[0][1]}, {u4n[1][0], u4n[1][1]}};
          if constexpr (kU4 == 1) {
            if (iu + 1 < nu) request_plane(exu + ex_unit);
          }
          // the key codes: two 16-byte loads per lane are the A fragments of all sixteen key tiles (with a 4-bit base the
          // first plane to run is the high plane, which lies with the block's extras in global memory)
          uint4 hw0, hw1;
          if constexpr (kU4 == 2) {
            const uint4* kplane = reinterpret_cast<const uint4*>(exu + 128 * n16p);
            hw0 = kplane[lane];
            hw1 = kplane[32 + lane];
          } else {
            hw0 = lds128(stg + kUnitOff);
            hw1 = lds128(stg + kUnitOff + 512);
          }

          // ---- key-group preparation: fp16 scale pairs {s, -4s} in fragment order, zero-point tile.  The tables of the
          // previous group were last read by this warp alone.
          if (has_meta) {
            __syncwarp();
            const uint4 mz = lds128(stg + kKeyMetaOff);   // channels 4*lane .. 4*lane+3
            const uint32_t neg4 = 0xC400C400u;   // half2(-4, -4)
            const uint32_t ma = pack_half2(bf_lo(mz.x), bf_lo(mz.y)), mb = pack_half2(bf_lo(mz.z), bf_lo(mz.w));
            sts64(kp_wr, ma, hmul2_u(ma, neg4));
            sts64(kp_wr + 16, mb, hmul2_u(mb, neg4));
            const uint32_t za = pack_half2(bf_hi(mz.x) * pk_zs, bf_hi(mz.y) * pk_zs);
            const uint32_t zb = pack_half2(bf_hi(mz.z) * pk_zs, bf_hi(mz.w) * pk_zs);
            sts64(zp_wr, za, za);
            sts64(zp_wr + 16, zb, zb);
            __syncwarp();      // the tables written above are read by other lanes below
            // the zero-point term q . z of the group: a tile chain of its own (the tile's rows are equal, so are the rows
            // of the result), independent of the key tiles below; the partner adds it to the logits
#pragma unroll
            for (int kt2 = 0; kt2 < 8; ++kt2) {
              const uint4 zz = lds128(zp_rd + 4 * zprep_word(kt2));
              if (kt2 == 0) mma_f16_to(zc, zz.x, zz.y, zz.z, zz.w, bq[0][0], bq[0][1], 0.f, 0.f, 0.f, 0.f);
              else mma_f16(zc, zz.x, zz.y, zz.z, zz.w, bq[kt2][0], bq[kt2][1]);
            }
          }

          // ---- q.K^T on the key tiles.  One pass over a plane of 2-bit codes: the base (low) plane with the scales s, and,
          // with a 4-bit base, first the dense high plane (codes c >> 2, laid out like the low plane) with the scales 4s.
          float Sx[2][4];
          auto key_pass = [&](const uint4& w0, const uint4& w1, bool first, bool high) {
            const uint32_t kw[2][4] = {{w0.x, w0.y, w0.z, w0.w}, {w1.x, w1.y, w1.z, w1.w}};
#pragma unroll
            for (int kt = 0; kt < 8; ++kt) {
              // scales of the lane's channel pairs (16kt + 2t, +1) and (16kt + 8 + 2t, +1); code bias 4 -> offset -4 s
              uint4 kp = lds128(kp_rd + kprep_off(kt, 0));
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
            key_pass(hw0, hw1, true, true);
            const uint4 kw0 = lds128(stg + kUnitOff);
            const uint4 kw1 = lds128(stg + kUnitOff + 512);
            key_pass(kw0, kw1, false, false);
          } else {
            key_pass(hw0, hw1, true, false);
          }
          // ---- promoted channels (raw bf16 keys) with a gathered q
          if (!promoted_in_values(kU4) && n16 > 0) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) mma_bf16(Sx[mt], xa[mt][0], xa[mt][1], xa[mt][2], xa[mt][3], xb0, xb1);
            // the registers are free again: request the next unit's pairs now, most of an iteration ahead of their use
            if (iu + 1 < nu) load_xa(exu + ex_unit);
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
                const uint32_t lo = (c0 < 128) ? lds16(qrow_u32 + 2 * c0) : 0u, hi = (c1 < 128) ? lds16(qrow_u32 + 2 * c1) : 0u;
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
            const uint32_t kpb = ring_u32 + kPrepBase + kKprepOff;
            auto plane_tile = [&](const uint32_t (&words)[2], const uint32_t (&sidx)[2], const uint32_t (&qb)[2]) {
              uint32_t a[2][4];
#pragma unroll
              for (int hp = 0; hp < 2; ++hp) {
                const uint32_t w = words[hp] >> (8 * (r >> 2));
                const uint32_t i0 = sidx[hp] & 0xFFFFu, i1 = sidx[hp] >> 16;
                const uint32_t s0 = i0 != 0xFFFFu ? lds16(kpb + i0) : 0u;
                const uint32_t s1 = i1 != 0xFFFFu ? lds16(kpb + i1) : 0u;
                const uint32_t sc = s0 | (s1 << 16);
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
                const uint32_t q0 = c0 < 128 ? lds16(qfrow_u32 + 2 * c0) : 0u;
                const uint32_t q1 = c1 < 128 ? lds16(qfrow_u32 + 2 * c1) : 0u;
                qb[hp] = q0 | (q1 << 16);
                sidx[hp] = scale_byte(c0) | (scale_byte(c1) << 16);
              }
              plane_tile(words, sidx, qb);
            }
          }

          // ---- hand the logits over: [m-tile][tokens r / r + 8] x heads 2t, 2t+1.  The buffer of this stage is free: the
          // partner took its last contents before it refilled the stage.
          {
            const uint32_t lb = lane32 + ring_stage * kLBufBytes;
            sts128(lb, __float_as_uint(Sx[0][0]), __float_as_uint(Sx[0][1]), __float_as_uint(Sx[0][2]), __float_as_uint(Sx[0][3]));
            sts128(lb + 16, __float_as_uint(Sx[1][0]), __float_as_uint(Sx[1][1]), __float_as_uint(Sx[1][2]), __float_as_uint(Sx[1][3]));
            sts64(lane8 + ring_stage * kLBufBytes, __float_as_uint(zc[0]), __float_as_uint(zc[1]));
            __syncwarp();
            mbar_arrive_one(lfull_u32 + ring_stage * 8u);
          }
          advance_stage();
          exu += ex_unit;
        }
        done += nu;
        u = 0;
        ++bi;
      }
      if (gave_up && lane == 0) atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
    } else {
      // =====================================================================================================
      // values warp
      // =====================================================================================================
      float O[8][4];       // O^T tiles: [channel tile] x (channels r, r+8) x (heads 2t, 2t+1), scaled 2^-20
      float Zc[4] = {0.f, 0.f, 0.f, 0.f};   // rows 0..VG-1: sum p * z_v per value group; row 4: sum p
      float m0 = -INFINITY, m1 = -INFINITY; // running reference maximum (log2 domain) of heads 2t, 2t+1
#pragma unroll
      for (int ct = 0; ct < 8; ++ct)
#pragma unroll
        for (int i = 0; i < 4; ++i) O[ct][i] = 0.f;
      // raises the reference maximum to max(reference, u) and rescales what has been accumulated
      auto raise_reference = [&](float u0, float u1) {
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
      };

      // ---- unquantized units: bf16 values straight from global memory, 8x8 tiles transposed in registers
      for (int ri = first_res; ri < n_res; ri += kPairs) {
        const int bu = res_b + ri;
        const bool in_sink = bu >= res_units;
        const int wu = in_sink ? bu - res_units : bu;
        const int rt = in_sink ? f_ns : f_r;
        const int j0 = wu * 32;
        const char* resv = in_sink ? lv.sink + (size_t)s * lv.sink_stride + (size_t)lv.sink_len * 256
                                   : lv.resv + (size_t)s * lv.resv_stride;
        const bool holds_new = !in_sink && lv.new_v != nullptr && jn >= j0 && jn < j0 + 32;
        // rows of this lane: tokens j0 + 8i + r, i = 0..3; word 2t.. of a 16-channel tile
        const uint32_t* rowp[4];
        bool rowv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int tok = j0 + 8 * i + r;
          rowv[i] = tok < rt;
          rowp[i] = reinterpret_cast<const uint32_t*>(resv + (size_t)tok * 256) + t;
          if (holds_new && tok == jn) rowp[i] = reinterpret_cast<const uint32_t*>(lv.new_v + (size_t)s * kD) + t;
        }
        if (holds_new) {
          const uint2 vn = reinterpret_cast<const uint2*>(lv.new_v + (size_t)s * kD)[lane];
          reinterpret_cast<uint2*>(lv.resv + (size_t)s * lv.resv_stride + (size_t)jn * 256)[lane] = vn;
        }
        // the first tile's loads go out before the wait for the logits
        uint32_t x[2][4];      // [ks][{tokens r, channels lo}, {tokens r, channels hi}, {tokens r + 8, lo}, {tokens r + 8, hi}]
        auto load_tile = [&](int ct) {
#pragma unroll
          for (int ks = 0; ks < 2; ++ks)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              x[ks][2 * hh] = rowv[2 * ks + hh] ? rowp[2 * ks + hh][8 * ct] : 0u;
              x[ks][2 * hh + 1] = rowv[2 * ks + hh] ? rowp[2 * ks + hh][8 * ct + 4] : 0u;
            }
        };
        load_tile(0);
        wait_or_give_up(rfull_u32, rit & 1u);
        const uint32_t rb = ring_u32 + kRBufBase + lane * 32;
        const uint4 s0 = lds128(rb), s1 = lds128(rb + 16);
        __syncwarp();
        mbar_arrive_one(rempty_u32);
        ++rit;
        // logits (log2 domain) of tokens j0 + 16 mt + r (+ 8), heads 2t, 2t+1; tokens past the window count for nothing
        float xl[2][4];
        {
          const float sx[2][4] = {{__uint_as_float(s0.x), __uint_as_float(s0.y), __uint_as_float(s0.z), __uint_as_float(s0.w)},
                                  {__uint_as_float(s1.x), __uint_as_float(s1.y), __uint_as_float(s1.z), __uint_as_float(s1.w)}};
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            const bool va = (j0 + mt * 16 + r) < rt, vb = (j0 + mt * 16 + 8 + r) < rt;
            xl[mt][0] = va ? sx[mt][0] * scale_log2e : -INFINITY;
            xl[mt][1] = va ? sx[mt][1] * scale_log2e : -INFINITY;
            xl[mt][2] = vb ? sx[mt][2] * scale_log2e : -INFINITY;
            xl[mt][3] = vb ? sx[mt][3] * scale_log2e : -INFINITY;
          }
        }
        raise_reference(fmaxf(fmaxf(xl[0][0], xl[0][2]), fmaxf(xl[1][0], xl[1][2])),
                        fmaxf(fmaxf(xl[0][1], xl[0][3]), fmaxf(xl[1][1], xl[1][3])));
        // probabilities scaled 2^-20 (the scale of the accumulators), as an exact bf16 pair (high part, remainder);
        // B fragments [k-step][tokens 2t.. / 2t+8..] of head r
        uint32_t Bh[2][2], Bl[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const float p0 = exp2f(xl[mt][2 * hh] - m0) * 9.5367431640625e-07f;
            const float p1 = exp2f(xl[mt][2 * hh + 1] - m1) * 9.5367431640625e-07f;
            const uint32_t hi = pack_bf162(p0, p1);
            Bh[mt][hh] = movmatrix_trans(hi);
            Bl[mt][hh] = movmatrix_trans(pack_bf162(p0 - bf_lo(hi), p1 - bf_hi(hi)));
          }
        // denominator: row 4 of the extra tile is 2^20, which undoes the scale of the probabilities
        const uint32_t ones = (r == 4) ? 0x49804980u : 0u;
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
          mma_bf16(Zc, ones, 0u, ones, 0u, Bh[ks][0], Bh[ks][1]);
          mma_bf16(Zc, ones, 0u, ones, 0u, Bl[ks][0], Bl[ks][1]);
        }
        // tile (ct, ks): A = V^T, 16 channels x 16 tokens: a0 = (channels r, tokens 2t..), a1 = (channels r + 8, tokens 2t..),
        // a2 = (channels r, tokens 8 + 2t..), a3 = (channels r + 8, tokens 8 + 2t..)
#pragma unroll
        for (int ct = 0; ct < 8; ++ct) {
          uint32_t a[2][4];
#pragma unroll
          for (int ks = 0; ks < 2; ++ks) {
            a[ks][0] = movmatrix_trans(x[ks][0]);
            a[ks][1] = movmatrix_trans(x[ks][1]);
            a[ks][2] = movmatrix_trans(x[ks][2]);
            a[ks][3] = movmatrix_trans(x[ks][3]);
          }
          if (ct + 1 < 8) load_tile(ct + 1);
#pragma unroll
          for (int ks = 0; ks < 2; ++ks) {
            mma_bf16(O[ct], a[ks][0], a[ks][1], a[ks][2], a[ks][3], Bh[ks][0], Bh[ks][1]);
            mma_bf16(O[ct], a[ks][0], a[ks][1], a[ks][2], a[ks][3], Bl[ks][0], Bl[ks][1]);
          }
        }
      }

      // ---- packed units
      // per-lane constants of the value-group preparation: the lane converts the scales and zero-points of token `lane`
      // value scales: [4 t: 20 words][4 vg][2 ks][2 ch] half2 s_v'; zero-point tile: [2 ks][8 rows][4 t]{ch0, 0, ch1, 0} half2
      // (rows < VG z_v, row 4 ones)
      const float pv_up = __uint_as_float((131u - 2u * (uint32_t)(lane >> 3)) << 23);          // 2^(4 - 2 * (2 ks + ch))
      const uint32_t sv_wr = ring_u32 + kPrepBase + kSvpOff + 2 * (((((lane & 7) >> 1) * 20 + (lane >> 3)) * 2) + (lane & 1));
      const uint32_t zv_wr = ring_u32 + kPrepBase + kZvpOff +
                             2 * ((((lane >> 4) * 144 + ((lane & 7) >> 1) * 4 + 2 * ((lane >> 3) & 1)) * 2) + (lane & 1));
      const uint32_t sv_rd = ring_u32 + kPrepBase + kSvpOff + t * 80;
      const uint32_t lane16 = ring_u32 + lane * 16, lane32 = ring_u32 + kLBufBase + lane * 32;
      const uint32_t lane8 = ring_u32 + kLBufBase + kLBufZeroOff + lane * 8;
      const uint32_t vm_rd = ring_u32 + kUnitOff + 2048 + lane * (4 * VG);
      // ---- three tiers, 4-bit base: the promoted channels' tile (raw bf16 keys from the blocks' extras, a gathered q) is added here
      // to the logits the partner hands over.  Requested ahead like everything from global memory: table entries two
      // blocks, channel lists one block, a unit's rows one unit.
      const uint32_t qrow_v = qb16_u32 + r * (kQS * 2);
      int vbi = 0, vcur = 0, vleft = 0;           // block, unit inside it, units of the block left for this warp
      int n16 = 0, n16p = 0;
      const char* ex = extras;                    // the block's extras, and those of the current unit
      const char* exu = extras;
      uint32_t ex_unit = 0;
      uint32_t xb0 = 0u, xb1 = 0u, xa[2][4] = {{0u, 0u, 0u, 0u}, {0u, 0u, 0u, 0u}};     // as in the logits warp
      auto load_xa = [&](const char* e) {
        const int xa_lo = (min(t, n16p - 1) * 32 + r) * 4, xa_hi = (min(t + 4, n16p - 1) * 32 + r) * 4;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          xa[mt][0] = *reinterpret_cast<const uint32_t*>(e + xa_lo + mt * 64);
          xa[mt][1] = *reinterpret_cast<const uint32_t*>(e + xa_lo + mt * 64 + 32);
          xa[mt][2] = *reinterpret_cast<const uint32_t*>(e + xa_hi + mt * 64);
          xa[mt][3] = *reinterpret_cast<const uint32_t*>(e + xa_hi + mt * 64 + 32);
        }
      };
      if constexpr (promoted_in_values(kU4)) {
        if (n_pack > 0) {
          vbi = wb / U;
          vcur = wb - vbi * U;
          if (!lv.stage_early) {
            pf_entry = table[vbi];
            if (vbi + 1 < f_nb) pf_entry_next = table[vbi + 1];
            request_lists(pf_entry);
          }
        }
      }
#pragma unroll 1
      for (int done = 0; done < n_pack; ++done) {
        if constexpr (promoted_in_values(kU4)) {
          if (vleft == 0) {
            // a block: its table entry and lists arrived a block ago; the next block's lists and the entry after that go out now
            const uint2 entry = pf_entry;
            const uint4 head = pf_head;          // the first 16 bytes of the block's extras: up to 8 pairs of promoted channels
            pf_entry = pf_entry_next;
            if (vbi + 1 < f_nb) request_lists(pf_entry);
            if (vbi + 2 < f_nb) pf_entry_next = table[vbi + 2];
            n16 = entry.y & 0xFF;
            n16p = (n16 + 1) >> 1;
            const int n4 = (entry.y >> 8) & 0xFF;
            ex = extras + (size_t)entry.x * 16;
            ex_unit = extras_unit_bytes(n16, n4, kU4 == 2);
            exu = ex + extras_header_bytes(n16, n4) + (size_t)vcur * ex_unit;
            vleft = min(U - vcur, n_pack - done);
            xb0 = xb1 = 0u;
            if (n16 > 0) {
              load_xa(exu);
              auto gather_q = [&](int p, uint32_t word) -> uint32_t {     // pair p < 8: its two channel numbers are in `word`
                if (p >= n16p) return 0u;
                const uint32_t cc = word >> (16 * (p & 1));
                const uint32_t c0 = cc & 0xFF, c1 = (cc >> 8) & 0xFF;
                const uint32_t lo = (c0 < 128) ? lds16(qrow_v + 2 * c0) : 0u, hi = (c1 < 128) ? lds16(qrow_v + 2 * c1) : 0u;
                return lo | (hi << 16);
              };
              xb0 = gather_q(t, (t & 2) ? head.y : head.x);
              xb1 = gather_q(t + 4, (t & 2) ? head.w : head.z);
            }
          }
        }
        wait_or_give_up(bar_u32 + ring_stage * 8u, ring_parity);
        const uint32_t st = lane16 + ring_stage * kStageBytes + kUnitOff;      // this lane's 16 bytes of the unit's first section
        // ---- value-group preparation (lane = token).  The tables of the previous unit were last read before the
        // warp barrier that closed it.
        {
          uint32_t mzv[4] = {0u, 0u, 0u, 0u};
          const uint32_t vm = vm_rd + ring_stage * kStageBytes;
          if constexpr (VG == 4) {
            const uint4 m = lds128(vm);
            mzv[0] = m.x; mzv[1] = m.y; mzv[2] = m.z; mzv[3] = m.w;
          } else if constexpr (VG == 2) {
            const uint2 m = lds64(vm);
            mzv[0] = m.x; mzv[1] = m.y;
          } else {
            mzv[0] = lds32(vm);
          }
#pragma unroll
          for (int vg = 0; vg < VG; ++vg) {
            sts16(sv_wr + 16 * vg, __half_as_ushort(__float2half_rn(bf_lo(mzv[vg]) * pv_up)));
            sts16(zv_wr + 64 * vg, __half_as_ushort(__float2half_rn(bf_hi(mzv[vg]))));
          }
        }
        const uint4 vw0 = lds128(st + 1024);
        const uint4 vw1 = lds128(st + 1536);
        __syncwarp();      // the tables written above are read by other lanes below
        wait_or_give_up(lfull_u32 + ring_stage * 8u, ring_parity);
        const uint32_t lb = lane32 + ring_stage * kLBufBytes;
        const uint4 s0 = lds128(lb), s1 = lds128(lb + 16);
        const uint2 zq = lds64(lane8 + ring_stage * kLBufBytes);
        float sx[2][4] = {{__uint_as_float(s0.x), __uint_as_float(s0.y), __uint_as_float(s0.z), __uint_as_float(s0.w)},
                          {__uint_as_float(s1.x), __uint_as_float(s1.y), __uint_as_float(s1.z), __uint_as_float(s1.w)}};
        if constexpr (promoted_in_values(kU4)) {
          // ---- promoted channels (raw bf16 keys) with a gathered q
          if (n16 > 0) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) mma_bf16(sx[mt], xa[mt][0], xa[mt][1], xa[mt][2], xa[mt][3], xb0, xb1);
            // the registers are free again: request the next unit's pairs now, a whole iteration ahead of their use
            if (vleft > 1) load_xa(exu + ex_unit);
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
              auto gather_bf16 = [&](uint32_t cc) -> uint32_t {
                const uint32_t c0 = cc & 0xFF, c1 = (cc >> 8) & 0xFF;
                const uint32_t lo = (c0 < 128) ? lds16(qrow_v + 2 * c0) : 0u, hi = (c1 < 128) ? lds16(qrow_v + 2 * c1) : 0u;
                return lo | (hi << 16);
              };
              const uint32_t b0 = gather_bf16(id0), b1 = gather_bf16(id1);
#pragma unroll
              for (int mt = 0; mt < 2; ++mt) mma_bf16(sx[mt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], b0, b1);
            }
          }
        }
        // logit = (sx + q . z) * scale: the zero-point term of the key group is the same for every token of the unit
        const float zl0 = __uint_as_float(zq.x) * scale_log2e, zl1 = __uint_as_float(zq.y) * scale_log2e;
        // ---- online softmax (log2 domain); heads 2t, 2t+1; tokens r, r+8 of each m-tile.
        // The reference maximum only has to keep the probabilities inside the fp16 range: it is raised (to the true
        // maximum so far, with the accumulators rescaled) when a logit of this unit exceeds it by more than kMaxSlack.
        {
          const float u0 = fmaf(fmaxf(fmaxf(sx[0][0], sx[0][2]), fmaxf(sx[1][0], sx[1][2])), scale_log2e, zl0);
          const float u1 = fmaf(fmaxf(fmaxf(sx[0][1], sx[0][3]), fmaxf(sx[1][1], sx[1][3])), scale_log2e, zl1);
          if (__any_sync(0xffffffffu, (u0 > m0 + kMaxSlack) || (u1 > m1 + kMaxSlack))) raise_reference(u0, u1);
        }
        const float c0 = zl0 - m0, c1 = zl1 - m1;
        // P^T B fragments: [k-step][tokens 2t.. / 2t+8..], head r
        uint32_t Pt[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          Pt[mt][0] = movmatrix_trans(pack_half2(ex2_approx(fmaf(sx[mt][0], scale_log2e, c0)), ex2_approx(fmaf(sx[mt][1], scale_log2e, c1))));
          Pt[mt][1] = movmatrix_trans(pack_half2(ex2_approx(fmaf(sx[mt][2], scale_log2e, c0)), ex2_approx(fmaf(sx[mt][3], scale_log2e, c1))));
        }
        // ---- zero-point and denominator tile: rows 0..VG-1 = z_v of the group, row 4 = ones, the rest zero
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
          const uint4 zz = lds128(lane16 + kPrepBase + kZvpOff + ks * 576);
          mma_f16(Zc, zz.x, zz.y, zz.z, zz.w, Pt[ks][0], Pt[ks][1]);
        }
        // ---- P.V: codes as fp16 subnormals, scales folded into P
        {
          const uint32_t vw[8] = {vw0.x, vw0.y, vw0.z, vw0.w, vw1.x, vw1.y, vw1.z, vw1.w};
#pragma unroll
          for (int vg = 0; vg < VG; ++vg) {
            const uint4 sv = lds128(sv_rd + vg * 16);
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
          const uint4 xw0 = lds128(st + 2048 + 128 * VG);
          const uint4 xw1 = lds128(st + 2048 + 128 * VG + 512);
          const uint32_t vw[8] = {xw0.x, xw0.y, xw0.z, xw0.w, xw1.x, xw1.y, xw1.z, xw1.w};
#pragma unroll
          for (int vg = 0; vg < VG; ++vg) {
            const uint4 sv = lds128(sv_rd + vg * 16);
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
        // ---- both warps are done with the unit: refill the stage
        __syncwarp();
        issue(ring_stage, false);
        advance_stage();
        if constexpr (promoted_in_values(kU4)) {
          exu += ex_unit;
          ++vcur;
          if (--vleft == 0) {
            ++vbi;
            vcur = 0;
          }
        }
      }
      if (gave_up) {
        if (lane == 0) atomicOr(lv.status, (uint32_t)MIXKVQ_DEV_COPY_TIMEOUT);
        // after the wait that ran out no wait was made, so the last copies may still be on their way, and they write to
        // the ring: wait for them (bounded) before the ring is reused below or the CTA ends
        for (int i = max(0, issued - kStages); i < issued; ++i) {
          const uint32_t pos = stage0 + (uint32_t)i;
          mbar_wait_polls(bar_u32 + (pos % kStages) * 8u, parity0 ^ ((pos / kStages) & 1u), lv.wait_polls ? lv.wait_polls : kWaitPolls);
        }
        // what this warp accumulated is not a result: the pair contributes nothing
#pragma unroll
        for (int ct = 0; ct < 8; ++ct)
#pragma unroll
          for (int i = 0; i < 4; ++i) O[ct][i] = 0.f;
        Zc[0] = Zc[1] = Zc[2] = Zc[3] = 0.f;
        m0 = m1 = -INFINITY;
      }

      // ---- finish this pair's split: true scale, zero-point terms, denominator
#pragma unroll
      for (int ct = 0; ct < 8; ++ct) {
        const int vg = ct / TPG;
        const float z0 = __shfl_sync(0xffffffffu, Zc[0], vg * 4 + t), z1 = __shfl_sync(0xffffffffu, Zc[1], vg * 4 + t);
        O[ct][0] = fmaf(O[ct][0], 1048576.0f, z0);
        O[ct][1] = fmaf(O[ct][1], 1048576.0f, z1);
        O[ct][2] = fmaf(O[ct][2], 1048576.0f, z0);
        O[ct][3] = fmaf(O[ct][3], 1048576.0f, z1);
      }
      const float l0 = __shfl_sync(0xffffffffu, Zc[0], 16 + t), l1 = __shfl_sync(0xffffffffu, Zc[1], 16 + t);
      if (r == 0) {
        mS[pair * 8 + 2 * t] = m0;
        mS[pair * 8 + 2 * t + 1] = m1;
        lS[pair * 8 + 2 * t] = l0;
        lS[pair * 8 + 2 * t + 1] = l1;
      }
      // the pair's unnormalized output goes to its own, now idle, ring as [8 heads][132] floats
      float* mine = reinterpret_cast<float*>(smem + pair * kPairBytes);
#pragma unroll
      for (int ct = 0; ct < 8; ++ct) {
        mine[(2 * t) * kMergeStride + 16 * ct + r] = O[ct][0];
        mine[(2 * t + 1) * kMergeStride + 16 * ct + r] = O[ct][1];
        mine[(2 * t) * kMergeStride + 16 * ct + 8 + r] = O[ct][2];
        mine[(2 * t + 1) * kMergeStride + 16 * ct + 8 + r] = O[ct][3];
      }
    }

    // ---- merge the pairs of the CTA, write the partial of (CTA, stream): the 16 threads that own a head add the pairs'
    // rows with the factors 2^(m_p - M).
    __syncthreads();
    for (int idx = threadIdx.x; idx < 256; idx += kThreads) {
      const int h = idx >> 5, c = 4 * (idx & 31);          // head, first of the thread's four channels
      float M = -INFINITY, L = 0.f, f[kPairs];
#pragma unroll
      for (int w = 0; w < kPairs; ++w) M = fmaxf(M, mS[w * 8 + h]);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < kPairs; ++w) {
        const float mw = mS[w * 8 + h];
        f[w] = (mw == -INFINITY) ? 0.f : ex2_approx(mw - M);
        L += f[w] * lS[w * 8 + h];
        const float4 o = *reinterpret_cast<const float4*>(smem + w * kPairBytes + (h * kMergeStride + c) * 4);
        acc.x += f[w] * o.x; acc.y += f[w] * o.y; acc.z += f[w] * o.z; acc.w += f[w] * o.w;
      }
      float* part = ws + (size_t)(blockIdx.x + s) * kPartialFloats + h * 130;
      *reinterpret_cast<float2*>(part + 2 + c) = make_float2(acc.x, acc.y);
      *reinterpret_cast<float2*>(part + 4 + c) = make_float2(acc.z, acc.w);
      if (c == 0) *reinterpret_cast<float2*>(part) = make_float2(M, L);
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
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes(kV4);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attention_ws_kernel<G, kU4, kV4>, lv, qb, sl, ws, 0x44004400u);
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
  cudaError_t e = cudaFuncSetAttribute(attention_ws_kernel<G, kU4, kV4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       smem_bytes(kV4));
  if (e != cudaSuccess) return e;
  // the CTAs of an SM only fit with the largest shared-memory carve-out; ask for it explicitly
  return cudaFuncSetAttribute(attention_ws_kernel<G, kU4, kV4>, cudaFuncAttributePreferredSharedMemoryCarveout,
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

cudaError_t attention_ws_setup() {
  cudaError_t e = setup_g<32>();
  if (e != cudaSuccess) return e;
  e = setup_g<64>();
  if (e != cudaSuccess) return e;
  return setup_g<128>();
}

// Split positions per stream: packed units plus the weighted units of the residual window and the sink.
long long attention_ws_positions(const LayerView& lv) {
  return (long long)lv.n_blocks * lv.U + (long long)kResidualWeight * ((lv.r + 31) / 32 + (lv.n_sink + 31) / 32);
}

// Split positions of one stream with the given fill (the entry w of a ragged batch's table)
int attention_ws_positions_of(int n_blocks, int r, int n_sink, int U) {
  return n_blocks * U + kResidualWeight * ((r + 31) / 32 + (n_sink + 31) / 32);
}

// Number of CTAs the split kernel runs for this layer state (also the number of partial-slot owners).  When there are
// fewer streams than CTA slots the grid is a multiple of the stream count, so that no CTA straddles two streams
// (a second segment costs a pipeline drain, a query load and a second partial).  Ragged batch: the positions of all
// streams are split evenly, wherever the boundaries fall.
int attention_ws_grid(const LayerView& lv, int n_sms) {
  const int S = lv.B * lv.Hkv;
  const long long total = lv.seq != nullptr ? lv.seq_total : attention_ws_positions(lv) * S;
  int grid = (int)min((long long)min(n_sms * kCtasPerSm, kMaxCtas / 2), total);
  if (grid > S && lv.seq == nullptr) grid = grid / S * S;
  return grid < 1 ? 1 : grid;
}

cudaError_t launch_attention_ws(const LayerView& lv, const void* q, float* out, float scale, float* ws, int n_sms,
                                cudaStream_t stream, int* launches, float* lse_out) {
  const int S = lv.B * lv.Hkv;
  const long long Us = attention_ws_positions(lv);
  const int grid = attention_ws_grid(lv, n_sms);
  cudaError_t e;
  if (lv.G == 32) e = launch_g<32>(lv, q, scale, ws, grid, stream);
  else if (lv.G == 64) e = launch_g<64>(lv, q, scale, ws, grid, stream);
  else e = launch_g<128>(lv, q, scale, ws, grid, stream);
  *launches = 1;
  if (e != cudaSuccess || out == nullptr) return e;     // out == nullptr: split kernel only (timing)
  e = launch_combine(ws, out, lv.g, lv.Hkv, lv.Hq, 1, grid, Us, S, stream, lv.seq, lv.seq_prefix, lse_out);
  *launches = 2;
  return e;
}

}  // namespace mixkvq
