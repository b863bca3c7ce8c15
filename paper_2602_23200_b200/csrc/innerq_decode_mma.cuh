// Fused decode attention over a packed cache with pair-ordered codes (Store::perm = 0), one launch.  Built today for
// the outer-grouped comparison cache only (OUTER = true: innerq_decode_mma_outer.cu); inner-grouped caches keep their
// codes in byte order and are decoded by the integer-operand kernel (innerq_decode_i8.cuh), which shares this file's
// launch shape, pipeline helpers, tail tiles and merge.  The description below is of the inner-grouped form, from
// which the outer-grouped one differs in where scales and zero-points are applied (see OUTER in the kernel).
//   q.K^T on packed key rows  ->  online softmax  ->  p.V on packed value chunks, split over token
//   ranges, fp16 windows and the K/V skew zone as 16-token tiles dealt to the same warps, cross-CTA merge by
//   the last CTA to finish.
//
// Work decomposition.  A CTA owns one (batch, KV head) unit and a range of value groups; each of its
// 8 warps owns a contiguous sub-range and streams it chunk by chunk (32 tokens) through a private ring
// of shared-memory stages filled by 1-D bulk async copies (cp.async.bulk + mbarrier): packed key rows,
// key scale/zero words, the packed value chunk and, at the end of each value group, its scale/zero
// words.  The warp never synchronises with other warps until the final merge.
//
// Arithmetic.  Codes are never dequantised element by element.  Inner-dimension grouping lets scale and
// zero-point leave the inner sum (Section "InnerQ": one scale per group, reused):
//     q'.x^_t = sum_g ( S_tg * sum_{c in g} q'_c u_tc  +  z_tg * sum_{c in g} q'_c )
//     sum_t p_t v^_tc = sum_j ( S_jc * sum_{t in j} p_t u_tc  +  z_jc * sum_{t in j} p_t )
// The raw-code sums run on the tensor pipe (mma.sync m16n8k16, fp32 accumulate) so that the ALU pipe only
// unpacks: `word & (field << pos)` is already an fp16 pair (two codes as subnormals scaled by 2^pos,
// the scale folded into the other operand).  The other operand (q' or p) is split into fp16 hi + lo
// columns, so the products carry fp32-level accuracy; up to 4 query heads of the KV head share one pass
// over the codes (the 8 mma columns are 4 heads x {hi, lo}).  Scale and zero-point are then applied once
// per (token, group) for keys and once per (group, channel) for values, in fp32.
#pragma once
#include "innerq_device.cuh"
#include "innerq_kernels.h"
#include "innerq_decode_mma.h"

namespace iq {


namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kHeads = 4;              // query heads per pass (hi/lo columns: 8 mma columns)
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait: gives up after kWaitLimit polls and reports it (the caller records an error and
// skips the data instead of spinning forever).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit = kWaitLimit) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// same with a zero accumulator input (lets the assembler use the zero register instead of clearing four)
__device__ __forceinline__ void mma16816_z(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                           uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
// Programmatic dependent launch: wait for the kernels this one depends on (no-op without the launch attribute);
// allow the next kernel in the stream to be launched before this one has finished.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Decoder parameters from a metadata word (fp16 scale with the mask in its sign bit | fp16 zero << 16):
// s = |scale|, z = Z if the mask is set (scale <= -0), else -s * 2^(b-1) (Z is stored as 0 then).
__device__ __forceinline__ void decode_fast(uint32_t meta, float neg_half, float& s, float& z) {
  const __half2 h = *reinterpret_cast<const __half2*>(&meta);
  const float sg = __low2float(h), Z = __high2float(h);
  s = fabsf(sg);
  // neg_half * max(sg, 0) as (neg_half / 2) * (sg + |sg|): the same value exactly, on the fp32 pipe only
  z = fmaf(0.5f * neg_half, sg + fabsf(sg), Z);
}
__device__ __forceinline__ float h2f_bits(uint32_t bits) { return __half2float(__ushort_as_half((unsigned short)bits)); }
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// fp16 hi / lo split of x, packed (hi in the low half-word, lo in the high half-word)
__device__ __forceinline__ uint32_t split_hi_lo(float x) {
  const __half hi = __float2half_rn(x);
  const __half lo = __float2half_rn(x - __half2float(hi));
  return (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
}
// fp16(lo) in the low half-word, fp16(hi) in the high one, with one packing conversion (not the conversion unit's
// single-value cvt, which costs a sub-partition 8 cycles per warp instruction)
__device__ __forceinline__ uint32_t pack_half2_rn(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ float pow2i(int e) { return __int_as_float((e + 127) << 23); }   // 2^e, -126 <= e <= 127

// Per bit-width constants of the packed formats (see innerq_layout.h).
template <int BITS> struct Fmt;
template <> struct Fmt<2> {
  static constexpr uint32_t kField = 0x00030003u;
  static constexpr int kKstepsPerWindow = 2;   // an 8-bit window of each half-word feeds 2 key k-steps
  static constexpr int kRowWordsPerLane = 2;
  static constexpr int kChunkWordsPerLane = 8;
};
template <> struct Fmt<4> {
  static constexpr uint32_t kField = 0x000F000Fu;
  static constexpr int kKstepsPerWindow = 1;
  static constexpr int kRowWordsPerLane = 4;
  static constexpr int kChunkWordsPerLane = 16;
};

// Shared-memory stage = the byte range of CPI consecutive chunk records as it lies in HBM (value metadata
// follows the last chunk of each value group), fetched with one bulk copy.
template <int KB, int VB, int G, int KM, int VM, int CPI> struct StageLayout {
  static constexpr int kNG = kD / G;
  static constexpr int kCH = G / kChunk;                          // chunks per value group
  static constexpr int kKCodes = kChunk * 16 * KB;
  static constexpr int kKMeta = kChunk * kNG * KM;
  static constexpr int kVCodes = 512 * VB;
  static constexpr int kVMeta = kD * VM;
  static constexpr int kOffKMeta = kKCodes;
  static constexpr int kOffVCodes = kOffKMeta + kKMeta;
  static constexpr int kRec = kOffVCodes + kVCodes;               // bytes of one chunk record
  static constexpr int kGroupRec = kCH * kRec + kVMeta;           // bytes of one group record
  // offset of chunk cc of an iteration inside the stage (iterations start on a group boundary or, when a
  // group spans several iterations, inside one group)
  __host__ __device__ static constexpr int off(int cc) { return cc * kRec + (cc / kCH) * kVMeta; }
  static constexpr int kBytes = CPI * kRec + (CPI / kCH > 0 ? CPI / kCH : 1) * kVMeta;
  // (three stages of the 4 KB records of 3-bit keys with 3-bit values fit as well and were measured: no gain)
  static constexpr int kStages = kBytes <= 3072 ? 4 : 2;
  static constexpr int kWarpBytes = kBytes * kStages;
  static constexpr int kSideBytes = 4 * kD * 4;                   // per warp: value metadata of the last 4 groups
  static constexpr int kTableBytes = 8448;                        // q tables and B fragments of the prologue
  static constexpr int kOffSide = kWarpBytes * kWarps;
  static constexpr int kSideArea = kSideBytes * kWarps > kTableBytes ? kSideBytes * kWarps : kTableBytes;
  static constexpr int kOffBars = kOffSide + kSideArea;
  static constexpr int kCtaBytes = kOffBars + 256;
};


// True when the unit's append counter (see Layout::appended_off) holds N, looked at up to kAppendPolls times about
// 0.2 us apart (whole warp, same answer in every lane).  The append that writes it precedes this kernel in the
// stream and lets its dependents start only once all of its CTAs are running, so it makes progress whatever this
// kernel does, and it publishes the counter long before it ends (its last CTA stays until the previous decode has
// ended).  A caller that gets false waits for its predecessor's completion instead, which is always right; looking
// only once sent most warps down that road and tied this decode's tail tiles to the END of the previous decode, which
// costs nothing with one wave of CTAs per launch and most of the overlap when launches are small enough to share
// the GPU (config 2 at four splits per unit: 28.1 us per step, 17.5 us with the bounded look).
constexpr int kAppendPolls = 48;
__device__ __forceinline__ bool append_count_is(const uint32_t* flag, uint32_t N) {
  bool there = false;
  for (int tries = 0; tries < kAppendPolls && !there; ++tries) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    there = __all_sync(0xffffffffu, v == N);
    if (!there) __nanosleep(200);
  }
  return there;
}

// Cross-CTA merge, run by the last CTA of a unit to finish: log-sum-exp combination of the n_parts partial results
// (rows prow0 .. of kPartialStride floats: acc[128], max, sum) of nh query rows, fp16 results to rows orow of out.
// Kept out of line so that its registers do not add to the streaming loop's.
__device__ __noinline__ void merge_parts(const float* __restrict__ partials, float* wm, __half* __restrict__ out, int nh,
                                         int n_parts, int prow0, int4 orow, int max_splits) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // Warp w merges parts w, w + 8, ... (four parts per round of loads, lane l the channels 4l .. 4l+3, running
  // max / rescale as in the streaming loop), then the eight warp results are combined through shared memory.
  // The loops over heads and rounds stay rolled: this code runs once per unit on a cold instruction cache,
  // where its size costs more than its latency.
#pragma unroll 1
  for (int h = 0; h < nh; ++h) {
    float M = -INFINITY, den = 0.f, n0 = 0.f, n1 = 0.f, n2 = 0.f, n3 = 0.f;
    const float* Ph = partials + (size_t)(prow0 + h) * max_splits * kPartialStride;
#pragma unroll 1
    for (int s0 = warp; s0 < n_parts; s0 += 4 * kWarps) {
      float4 v[4];
      float2 ml[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int s = s0 + e * kWarps;
        const float* P = Ph + (size_t)(s < n_parts ? s : s0) * kPartialStride;
        v[e] = __ldg(reinterpret_cast<const float4*>(P) + lane);
        ml[e] = __ldg(reinterpret_cast<const float2*>(P + kD));
        if (s >= n_parts) ml[e] = make_float2(-INFINITY, 0.f);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float m_new = fmaxf(M, ml[e].x);
        const float a_old = M == -INFINITY ? 0.f : ex2_approx(M - m_new);
        const float a_new = ml[e].x == -INFINITY ? 0.f : ex2_approx(ml[e].x - m_new);
        M = m_new;
        den = fmaf(den, a_old, ml[e].y * a_new);
        n0 = fmaf(n0, a_old, v[e].x * a_new);
        n1 = fmaf(n1, a_old, v[e].y * a_new);
        n2 = fmaf(n2, a_old, v[e].z * a_new);
        n3 = fmaf(n3, a_old, v[e].w * a_new);
      }
    }
    float* mine = wm + ((size_t)warp * kHeads + h) * (kD + 2);
    *reinterpret_cast<float2*>(mine + 4 * lane) = make_float2(n0, n1);
    *reinterpret_cast<float2*>(mine + 4 * lane + 2) = make_float2(n2, n3);
    if (lane == 0) { mine[kD] = M; mine[kD + 1] = den; }
  }
  __syncthreads();
  for (int i = tid; i < nh * kD; i += kThreads) {
    const int h = i >> 7, c = i & (kD - 1);
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, wm[((size_t)w * kHeads + h) * (kD + 2) + kD]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float* r_ = wm + ((size_t)w * kHeads + h) * (kD + 2);
      const float wgt = r_[kD] == -INFINITY ? 0.f : ex2_approx(r_[kD] - M);
      num = fmaf(r_[c], wgt, num);
      den = fmaf(r_[kD + 1], wgt, den);
    }
    const int row = h == 0 ? orow.x : h == 1 ? orow.y : h == 2 ? orow.z : orow.w;
    out[(size_t)row * kD + c] = __float2half_rn(num / den);
  }
}

// ---- the kernel -------------------------------------------------------------------------------------
// CPI = chunks (of 32 tokens) a warp processes per loop iteration: one barrier wait, one soft-max update and
// one refill per iteration, and CPI*2 independent key accumulator chains in flight.
// KB / VB: bits of the key / value codes (3 = a 2-bit plane plus a 1-bit plane, two MMAs per k-step);
// KM / VM: bytes of a metadata entry (4: scale|zero, 2: scale only, symmetric mode).
// SPLIT (one query head per KV head, G = 32): the 8 mma columns are not 4 heads x {hi, lo} but
// 4 groups x {hi, lo}: for keys, column pair g holds q'' restricted to channel group g, so one accumulator
// chain over all 8 k-steps yields the four per-group code sums at once and lane j of each quad applies the
// scale / zero-point of group j only (then the quad adds up); for values, column pair w holds p
// restricted to the w-th value group of a window of four, and lane j applies group j's metadata once per
// window.  This removes the 4x redundancy a quad otherwise has in decoding per-group metadata.
// OUTER: the outer-grouped comparison cache (keys grouped per channel along tokens, values per token along
// channels, asymmetric).  Same records, same pipeline, other arithmetic: the scale can no longer leave the inner
// sum, so it goes INTO the second operand: for keys q'' * S_j (rebuilt for every group of G tokens from the group's
// metadata, which leads the group record), for values p_t * S_{t,g} (one operand set per channel group the
// m-tile's rows fall into); zero-points contribute sum_c q''_c Z_jc per group and sum_t p_t Z_{t,g} per channel
// group.  One chunk per iteration, four heads per pass.
// ABL (timing experiments only, results wrong on purpose): bit 0 leaves out the key side's unpack + MMA work of the
// streaming loop (scores taken as 0), bit 1 the value side's; all bytes are still streamed.
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false, bool PAGED = false, int ABL = 0>
__device__ __forceinline__ void decode_mma_body(const Layout& L, const Counts& cn, const DecodeArgs& a, const int u,
                                                const PageIds* ptab = nullptr) {
  constexpr int KP = KB == 3 ? 2 : KB, VP = VB == 3 ? 2 : VB;     // bits of the primary code plane
  using F = Fmt<KP>;
  using FV = Fmt<VP>;
  using SL = StageLayout<KB, VB, G, KM, VM, CPI>;
  constexpr int NG = SL::kNG;                   // key groups per token
  constexpr int KS_PER_G = G / 16;              // key k-steps per group
  constexpr int CH = SL::kCH;                   // chunks per value group
  constexpr int NST = SL::kStages;
  constexpr int RW = 4 * KB;                    // 32-bit words per packed key row
  constexpr int RWL = F::kRowWordsPerLane;
  constexpr int KPW = F::kKstepsPerWindow;
  constexpr int RU = CH;                        // chunks per range unit: one value group
  constexpr int WIN = 4;                        // SPLIT: value groups per window (one per lane of a quad)
  // q'' fragments are scaled below 2^QE; the 1-bit plane of 3-bit keys reuses them times up to 2^2 * 2^0
  constexpr int QE = KB == 3 ? 12 : 14;
  static_assert(!SPLIT || (G == 32), "SPLIT is built for G = 32");
  static_assert(!OUTER || (!SPLIT && CPI == 1 && KM == 4 && VM == 4 && KB != 3 && VB != 3), "OUTER: plain variant only");
  constexpr int VBASE = 4;                      // OUTER: p * S enters the value MMA scaled by 2^(VBASE - field position)
  static_assert((NST & (NST - 1)) == 0, "stage count must be a power of two");
  static_assert(CPI == 1 || CPI == 2, "one or two chunks per iteration");

  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, j = lane & 3;
  const int split = blockIdx.y;
  if (split >= a.grid_y) return;      // batched launch: this sequence uses fewer grid rows than the longest one
  const int b = u / L.Hkv, hkv = u % L.Hkv;
  const int nh = min(SPLIT ? 1 : kHeads, L.r * a.n_q - a.head0);
  // Row of q / out of column h of this launch: head h' = (head0 + h) % r of query token i = (head0 + h) / r
  // (q, out: [B, n_q, Hq, D]; n_q = 1: the pass's heads are consecutive rows), and the row of its split partials.
  auto q_row = [&](int h) {
    const int v = a.head0 + h, i = a.n_q > 1 ? v / L.r : 0;
    return (b * a.n_q + i) * L.Hq + hkv * L.r + (v - i * L.r);
  };
  const int prow0 = a.n_q > 1 ? u * kHeads : q_row(0);
  const int n_parts = a.grid_y;
  const bool fast = split < a.n_splits;
  // ---------------- this warp's work: tail tiles and a range of packed chunks ----------------------
  // Tail tiles of the unit are dealt round-robin to CTAs, then to warps.  A tile costs about as much as
  // `tail_cost_units` range units, so packed ranges are shortened accordingly (contiguous, ordered).
  const int Gy = a.grid_y, cst = a.tail_cost_units;
  const int n_chunks_total = (OUTER ? cn.n_qk : cn.n_qv) / kChunk;   // chunks in which keys AND values are packed
  const int n_units_total = (n_chunks_total + RU - 1) / RU;
  const int q_cta = a.tiles_q0 + (split < a.tiles_rem ? 1 : 0);                 // tail tiles of this CTA
  const int tiles_before = split * a.tiles_q0 + min(split, a.tiles_rem);         // ... of the CTAs before it
  auto tiles_of_warp = [&](int q, int w) { return (q >> 3) + (w < (q & 7) ? 1 : 0); };
  const int u_lo = max(0, min(n_units_total, split * a.units_per_split - cst * tiles_before));
  const int u_hi = split == a.n_splits - 1
                       ? n_units_total
                       : max(u_lo, min(n_units_total, (split + 1) * a.units_per_split - cst * (tiles_before + q_cta)));
  const int n_u = fast ? u_hi - u_lo : 0;
  const int n_virtual = n_u + cst * q_cta;
  const int tw_before = warp * (q_cta >> 3) + min(warp, q_cta & 7);
  const int tw = tiles_of_warp(q_cta, warp);                        // tail tiles of this warp
  const int wu_lo = u_lo + max(0, min(n_u, ((n_virtual * warp) >> 3) - cst * tw_before));
  const int wu_hi = warp == kWarps - 1
                        ? u_lo + n_u
                        : max(wu_lo, u_lo + max(0, min(n_u, ((n_virtual * (warp + 1)) >> 3) - cst * (tw_before + tw))));
  const int c_lo = wu_lo * RU;                                  // first chunk
  const int n_chunks_w = (wu_hi - wu_lo) * RU;                  // chunks of this warp (may be odd when CPI = 2)
  const int n_iters = (n_chunks_w + CPI - 1) / CPI;

  unsigned char* ring = smem + (size_t)warp * SL::kWarpBytes;
  uint32_t* side = reinterpret_cast<uint32_t*>(smem + SL::kOffSide + (size_t)warp * SL::kSideBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::kOffBars) + warp * NST;
  const uint32_t ring_u32 = smem_u32(ring), bars_u32 = smem_u32(bars);
  // Group record g of this unit (a paged cache looks the group's page up in the cache's page table).
  // (ptab: the table as a kernel parameter, when the launcher could pass it; else it is read from the cache buffer)
  [[maybe_unused]] auto page_of = [&](int slot) -> uint32_t {
    return ptab ? ptab->id[slot] : reinterpret_cast<const uint32_t*>(a.cache + L.page_table_off)[slot];
  };
  [[maybe_unused]] auto page_start = [&](uint32_t page) -> const unsigned char* {
    return L.pool + (size_t)page * L.page_bytes + (size_t)u * L.k.rec_unit_stride;
  };
  auto group_rec = [&](int g) -> const unsigned char* {
    if constexpr (PAGED) {
      const int slot = g / L.page_groups;
      return page_start(page_of(slot)) + (size_t)(g - slot * L.page_groups) * SL::kGroupRec;
    } else {
      return a.cache + L.k.rec_off + (size_t)u * L.k.rec_unit_stride + (size_t)g * SL::kGroupRec;
    }
  };

  // Copies of consecutive iterations read consecutive byte ranges of the record area: keep a running source.
  // In a paged cache (PAGED) that holds inside a page (2^k chunks): the copy that starts a page is re-based, and the
  // copy whose two chunks lie in two pages is split.  The table entry of the page after the current one is loaded
  // one page ahead (page_next), so that no copy waits for a table lookup except a warp's first one.
  const unsigned char* nx_src = n_iters > 0 ? group_rec(c_lo / CH) + (size_t)(c_lo % CH) * SL::kRec : nullptr;
  int nx_ci = c_lo;
  [[maybe_unused]] uint32_t page_next = 0;
  [[maybe_unused]] auto load_page_next = [&](int ci) {      // ci: a chunk of the page that is current from now on
    const int slot = (ci >> L.page_chunk_shift) + 1;
    if ((slot << L.page_chunk_shift) < c_lo + n_chunks_w)   // this warp will read that page: it exists
      page_next = page_of(slot);
  };
  if constexpr (PAGED) {
    if (n_iters > 0) load_page_next(c_lo);
  }
  auto issue = [&](int st) {   // one lane: arm the barrier, start the copy of the next iteration into stage st
    // the value group's scale/zero words sit right behind its last chunk
    // (OUTER: the key group's words sit in front of its first chunk)
    const int n_meta = OUTER ? ((nx_ci & (CH - 1)) == 0 ? 1 : 0)
                             : (CPI >= CH ? CPI / CH : (((nx_ci + CPI) & (CH - 1)) == 0 ? 1 : 0));
    const uint32_t bytes = CPI * SL::kRec + n_meta * SL::kVMeta;
    mbar_expect_tx(bars_u32 + 8 * st, bytes);
    if constexpr (PAGED) {
      const int in_page = nx_ci & L.page_chunk_mask;
      if (in_page == 0 && nx_ci != c_lo) {
        nx_src = page_start(page_next);
        load_page_next(nx_ci);
      } else if (in_page + CPI > L.page_chunk_mask + 1) {
        // CPI = 2 with one chunk per group, first chunk at the end of a page: two copies of one group record each.
        // A second chunk beyond this warp's range is not used (and its page may not exist): the first one again.
        const bool used = nx_ci + 1 < c_lo + n_chunks_w;
        const unsigned char* second = used ? page_start(page_next) : nx_src;
        bulk_g2s(ring_u32 + st * SL::kBytes, nx_src, bytes / 2, bars_u32 + 8 * st);
        bulk_g2s(ring_u32 + st * SL::kBytes + bytes / 2, second, bytes / 2, bars_u32 + 8 * st);
        nx_src = second + bytes / 2;
        if (used) load_page_next(nx_ci + 1);
        nx_ci += CPI;
        return;
      }
    }
    bulk_g2s(ring_u32 + st * SL::kBytes, nx_src, bytes, bars_u32 + 8 * st);
    nx_src += bytes;
    nx_ci += CPI;
  };
  // Tail tile x: up to 16 tokens outside the range where both K and V are packed.  Skew tiles
  // (x < n_skew_tiles): keys are packed rows n_qv + 16x .. of one chunk record, values fp16 ring rows.
  // Other tiles: entries of the list [sink tokens, recent key tokens], keys and values fp16.
  // (OUTER: the skew zone has packed values and fp16 keys, and the list ends with the recent VALUE tokens)
  const int n_skew = OUTER ? cn.n_qv - cn.n_qk : cn.n_qk - cn.n_qv;
  const int n_list = cn.n_sink + (OUTER ? cn.n_v_recent : cn.n_k_recent);
  auto tail_tile = [&](int k, bool& skew, int& e0, int& cnt) {
    const int x = split + Gy * (warp + kWarps * k);
    skew = x < a.n_skew_tiles;
    e0 = 16 * (skew ? x : x - a.n_skew_tiles);
    cnt = min(16, (skew ? n_skew : n_list) - e0);
  };
  // fp16 row of list entry e: sink rows, else ring slot = (first slot + offset), wrapped once
  const uint4* v_sink4 = reinterpret_cast<const uint4*>(a.cache + L.v.sink_off + (size_t)u * L.v.sink_stride);
  const uint4* v_ring4 = reinterpret_cast<const uint4*>(a.cache + L.v.ring_off + (size_t)u * L.v.ring_stride);
  const uint4* k_sink4 = reinterpret_cast<const uint4*>(a.cache + L.k.sink_off + (size_t)u * L.k.sink_stride);
  const uint4* k_ring4 = reinterpret_cast<const uint4*>(a.cache + L.k.ring_off + (size_t)u * L.k.ring_stride);
  // the tensor that is still fp16 in the skew zone (values; OUTER: keys) has the zone's tokens at the head of its ring
  auto v_row = [&](bool skew, int e) -> const uint4* {
    if (!skew && e < cn.n_sink) return v_sink4 + (size_t)e * 16;
    int slot = a.v_ring_pos0 + (OUTER ? e - cn.n_sink : (skew ? e : n_skew + (e - cn.n_sink)));
    if (slot >= L.v.ring_cap) slot -= L.v.ring_cap;
    return v_ring4 + (size_t)slot * 16;
  };
  auto k_row = [&](bool skew, int e) -> const uint4* {
    if (!skew && e < cn.n_sink) return k_sink4 + (size_t)e * 16;
    int slot = a.k_ring_pos0 + (OUTER ? (skew ? e : n_skew + (e - cn.n_sink)) : e - cn.n_sink);
    if (slot >= L.k.ring_cap) slot -= L.k.ring_cap;
    return k_ring4 + (size_t)slot * 16;
  };
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < NST; ++s) mbar_init(bars_u32 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // Everything above touches no global memory: under a programmatic dependent launch it runs while the kernels
  // before this one in the stream (the step's append, the previous decode's merge) are still running.  What they may
  // still be writing is known: the fp16 rings, and packed rows / groups that did not exist when the previous decode
  // of this cache was launched (that decode made sure of its own predecessors before it let this one start).  So
  // this kernel waits for its predecessors (dep_wait) only before it touches those: the tail tiles and the chunks
  // from safe_chunks on.  q and the norms are inputs that are complete before the call (see innerq.h); the chunks
  // below safe_chunks are streamed, and the q tables built, while the append is still running.
  bool dep_waited = false;
  auto dep_wait = [&]() {
    if (!dep_waited) { grid_dependency_wait(); dep_waited = true; }
  };
  // What the step's append writes for this unit (rings, newest packed rows) is complete when the unit's counter in
  // the cache buffer holds this decode's N: the append publishes it (release) after its last write, long before the
  // append kernel ends (one of its CTAs stays until the previous decode has ended).  A warp looks for a bounded time
  // (acquire; see append_count_is): when the count is there it goes on, while the append's other units and the
  // previous decode may still be running; if it never shows, it waits for its predecessor's completion, which is
  // always right.
  auto wait_for_append = [&]() {
    if (dep_waited) return;
    const uint32_t* flag = reinterpret_cast<const uint32_t*>(a.cache + L.appended_off) + u;
    if (!append_count_is(flag, (uint32_t)cn.N)) dep_wait();
    // what was acquired is ordered ahead of bulk async copies too (this kernel's later ones, and through
    // launch_dependents the next kernel's, which stream the rows that append packed)
    asm volatile("fence.proxy.async.global;" ::: "memory");
  };
  auto ld_tail = [&](const uint4* p) -> uint4 { return dep_waited ? __ldg(p) : __ldcg(p); };
  // an iteration's copy covers the chunks [c_lo + i * CPI, c_lo + (i + 1) * CPI)
  auto dep_wait_for_iteration = [&](int i) {
    if (c_lo + (i + 1) * CPI > a.safe_chunks) dep_wait();
  };
  // q and the key norms are requested first of all, ahead of the bulk copies below: behind several
  // hundred KB of queued chunk data per SM they would take microseconds to arrive.
  // Only requested here: nothing may USE the loaded values before the copies below are issued (a warp issues in
  // order, so a conversion or a select on them would hold the copies back until q has arrived from memory).
  unsigned short q_bits[2];
  float n_raw[2];
  {
    const float* norm_g = reinterpret_cast<const float*>(a.cache + L.norm_off) + (size_t)u * kD;
    const unsigned short* q16 = reinterpret_cast<const unsigned short*>(a.q);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int i = tid + e * kThreads, h = i >> 7, c = i & (kD - 1);
      q_bits[e] = q16[(size_t)q_row(h < nh ? h : 0) * kD + c];
      n_raw[e] = norm_g[c];
    }
  }
#pragma unroll
  for (int s = 0; s < NST; ++s)
    if (s < n_iters) {
      dep_wait_for_iteration(s);
      if (lane == 0) issue(s);
    }
  float q_early[2], n_early[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int h = (tid + e * kThreads) >> 7;
    q_early[e] = h < nh ? __half2float(__ushort_as_half(q_bits[e])) : 0.f;
    n_early[e] = L.k_normalize ? n_raw[e] : 1.0f;
  }

  __shared__ unsigned int s_past_tail;      // warps of this CTA that are past their tail tiles (see the main loop's head)
  if (tid == 0) s_past_tail = 0u;           // ordered before its first use by the barriers of the prologue
  // ---------------- prologue: q'' = q * sm_scale * log2(e) (* norm for packed key rows) -------------
  float* q_nrm_s = reinterpret_cast<float*>(smem + SL::kOffSide);  // [4][128]   (the side area is not in use yet)
  float* q_raw_s = q_nrm_s + kHeads * kD;                          // [4][128]
  float* qg_s = q_raw_s + kHeads * kD;                             // [4][4]
  int* qe_s = reinterpret_cast<int*>(qg_s + kHeads * 4);           // [4] exponent of max|q''|
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int i = tid + e * kThreads;
    const float v = q_early[e] * (L.sm_scale * kLog2e);
    q_raw_s[i] = v;
    q_nrm_s[i] = v * n_early[e];
  }
  __syncthreads();
  if (warp < kHeads) {      // warp h: group sums and max |q''| of head h
    float v[4], am = 0.f, amr = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[e] = q_nrm_s[warp * kD + e * 32 + lane];
      am = fmaxf(am, fabsf(v[e]));
      amr = fmaxf(amr, fabsf(q_raw_s[warp * kD + e * 32 + lane]));
    }
    // channel c = e * 32 + lane belongs to group c / G
    float gs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int e = 0; e < 4; ++e) gs[(e * 32) / G] += v[e];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
      amr = fmaxf(amr, __shfl_xor_sync(0xffffffffu, amr, o));
#pragma unroll
      for (int g = 0; g < 4; ++g) gs[g] += __shfl_xor_sync(0xffffffffu, gs[g], o);
    }
    if (lane == 0) {
#pragma unroll
      for (int g = 0; g < 4; ++g) qg_s[warp * 4 + g] = gs[g];
      int e = 0;
      if (am > 0.f && am < INFINITY) e = ((__float_as_int(am) >> 23) & 0xff) - 126;
      qe_s[warp] = e;     // am < 2^e
      int er = 0;
      if (amr > 0.f && amr < INFINITY) er = ((__float_as_int(amr) >> 23) & 0xff) - 126;
      qe_s[4 + warp] = er;
    }
  }
  __syncthreads();

  {
    // ======================= fast path: packed keys and values ===================================
    // ---- per-thread constants.  As owner of B-fragment column gid: (head, hi|lo) or, in SPLIT, (group, hi|lo).
    const int col_head = SPLIT ? 0 : (gid >> 1), col_group = gid >> 1, col_part = gid & 1;
    // The fragment values depend on (lane, k-step, register) only, not on the warp: warp w computes the
    // k-step-w entries for every lane once, all warps then read their 16 registers from shared memory.
    uint32_t* bq_s = reinterpret_cast<uint32_t*>(qe_s + 16);      // [8 k-steps][2][32 lanes]
    uint32_t* bqr_s = bq_s + 512;                                  // same for raw q against fp16 key rows
    {
      const float bscale = pow2i(QE - qe_s[col_head]);   // |q''| * bscale < 2^QE
      const int s = warp;
      const int kk = (s % (2 * KPW)) % KPW;
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int pos = 2 * kk + rr;
        const float scl = bscale * pow2i(-KP * pos);
        const int c0 = 16 * s + 2 * j + 8 * rr;
        const uint32_t v0 = split_hi_lo(q_nrm_s[col_head * kD + c0] * scl);
        const uint32_t v1 = split_hi_lo(q_nrm_s[col_head * kD + c0 + 1] * scl);
        uint32_t v = col_part ? ((v0 >> 16) | (v1 & 0xFFFF0000u)) : ((v0 & 0xFFFFu) | (v1 << 16));
        if (SPLIT && (s / KS_PER_G) != col_group) v = 0u;
        bq_s[(s * 2 + rr) * 32 + lane] = v;
      }
      // raw q'' for fp16 key rows: k rows follow the 16-byte-piece order of a row load (piece tid4 + 4*i holds
      // the column pairs of k-steps 2i and 2i+1); one head per column pair also in SPLIT (pair 0 only)
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int c0 = 8 * (j + 4 * (s >> 1)) + 4 * (s & 1) + 2 * rr;
        const int h = gid >> 1;
        const float bs = pow2i(14 - qe_s[4 + h]);
        const uint32_t v0 = split_hi_lo(q_raw_s[h * kD + c0] * bs), v1 = split_hi_lo(q_raw_s[h * kD + c0 + 1] * bs);
        bqr_s[(s * 2 + rr) * 32 + lane] = col_part ? ((v0 >> 16) | (v1 & 0xFFFF0000u)) : ((v0 & 0xFFFFu) | (v1 << 16));
      }
    }
    __syncthreads();
    uint32_t Bq[8][2];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      Bq[s][0] = bq_s[(s * 2) * 32 + lane];
      Bq[s][1] = bq_s[(s * 2 + 1) * 32 + lane];
    }
    // ---- as owner of C-fragment columns 2j, 2j+1: head j, or in SPLIT (head 0, key group j)
    const int my_head = SPLIT ? 0 : j;
    // first absolute token position this lane's query row must not see (all tokens for the newest query)
    const int pos_end = cn.n_sink + cn.n_qk + cn.n_k_recent - (a.n_q - 1 - (a.head0 + my_head) / L.r);
    const int e_c = qe_s[my_head];
    const float kfac = pow2i(24 - (QE - e_c));       // undoes the 2^-24 of the subnormal codes and bscale
    const float inv_kfac = pow2i(-(24 - (QE - e_c)));
    float Qg[SPLIT ? 1 : NG];
    if constexpr (SPLIT) {
      Qg[0] = qg_s[j] * inv_kfac;                     // NG == 4: every lane of the quad owns one group
    } else {
#pragma unroll
      for (int g = 0; g < NG; ++g) Qg[g] = qg_s[j * 4 + g] * inv_kfac;
    }
    const float neg_half = -(float)(1 << (KB - 1)), neg_half_v = -(float)(1 << (VB - 1));
    // Raw scores (still carrying 1/kfac) of the 16 packed key rows r0 .. r0+15 of a chunk: this lane's rows are
    // r0 + gid and r0 + gid + 8.  kc / km: packed rows and metadata rows of the chunk (shared or global memory).
    auto k_mtile = [&](const uint32_t* kc, const uint32_t* km, int r0, float& sA_out, float& sB_out) {
      const int rA = r0 + gid, rB = rA + 8;
      uint32_t wa[RWL], wb[RWL];
      if constexpr (RWL == 2) {
        const uint2 xa = *reinterpret_cast<const uint2*>(kc + rA * RW + j * RWL);
        const uint2 xb = *reinterpret_cast<const uint2*>(kc + rB * RW + j * RWL);
        wa[0] = xa.x; wa[1] = xa.y; wb[0] = xb.x; wb[1] = xb.y;
      } else {
        const uint4 xa = *reinterpret_cast<const uint4*>(kc + rA * RW + j * RWL);
        const uint4 xb = *reinterpret_cast<const uint4*>(kc + rB * RW + j * RWL);
        wa[0] = xa.x; wa[1] = xa.y; wa[2] = xa.z; wa[3] = xa.w;
        wb[0] = xb.x; wb[1] = xb.y; wb[2] = xb.z; wb[3] = xb.w;
      }
      uint32_t ha = 0u, hb = 0u;                      // 1-bit plane of 3-bit codes: one word per lane and row
      if constexpr (KB == 3) { ha = kc[rA * RW + 8 + j]; hb = kc[rB * RW + 8 + j]; }
      auto kstep = [&](float (&c4)[4], int ks, bool zero_c) {
        const int wi = ks / (2 * KPW), sw = ks % (2 * KPW);
        const int window = sw / KPW, kk = sw % KPW;
        const uint32_t xa = window ? (wa[wi] >> 8) : wa[wi];
        const uint32_t xb = window ? (wb[wi] >> 8) : wb[wi];
        const uint32_t m0 = F::kField << (KP * (2 * kk)), m1 = F::kField << (KP * (2 * kk + 1));
        if (zero_c) mma16816_z(c4, xa & m0, xb & m0, xa & m1, xb & m1, Bq[ks][0], Bq[ks][1]);
        else mma16816(c4, xa & m0, xb & m0, xa & m1, xb & m1, Bq[ks][0], Bq[ks][1]);
        if constexpr (KB == 3) {
          // top bit of the code: weight 4, field 2*ks + odd of each half-word; the operand is the same q''
          // fragment rescaled (exactly, by a power of two) for this plane's field position
          const uint32_t ya = (ks >> 2) ? (ha >> 8) : ha, yb = (ks >> 2) ? (hb >> 8) : hb;
          const int p0 = (2 * ks) & 7, p1 = (2 * ks + 1) & 7;
          const uint32_t h0 = 0x00010001u << p0, h1 = 0x00010001u << p1;
          const __half2 f0 = __float2half2_rn(pow2i(KP * (2 * kk) + 2 - p0)), f1 = __float2half2_rn(pow2i(KP * (2 * kk + 1) + 2 - p1));
          const __half2 b0 = __hmul2(*reinterpret_cast<const __half2*>(&Bq[ks][0]), f0);
          const __half2 b1 = __hmul2(*reinterpret_cast<const __half2*>(&Bq[ks][1]), f1);
          mma16816(c4, ya & h0, yb & h0, ya & h1, yb & h1, *reinterpret_cast<const uint32_t*>(&b0),
                   *reinterpret_cast<const uint32_t*>(&b1));
        }
      };
      auto kmeta = [&](int row, int g, float& s_, float& z_) {      // decoder parameters of (row, group)
        if constexpr (KM == 4) decode_fast(km[row * NG + g], neg_half, s_, z_);
        else {
          s_ = h2f_bits(reinterpret_cast<const uint16_t*>(km)[row * NG + g] & 0x7FFFu);
          z_ = neg_half * s_;
        }
      };
      float sA, sB;
      if constexpr (OUTER) {          // the scales are inside Bq: the sums over all 128 channels are the scores
        float c4[4];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) kstep(c4, ks, ks == 0);
        sA = c4[0] + c4[1];
        sB = c4[2] + c4[3];
      } else if constexpr (SPLIT) {
        float c4[4];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) kstep(c4, ks, ks == 0);
        float s_, z_;
        kmeta(rA, j, s_, z_);
        sA = fmaf(s_, c4[0] + c4[1], z_ * Qg[0]);
        kmeta(rB, j, s_, z_);
        sB = fmaf(s_, c4[2] + c4[3], z_ * Qg[0]);
        sA += __shfl_xor_sync(0xffffffffu, sA, 1);
        sB += __shfl_xor_sync(0xffffffffu, sB, 1);
        sA += __shfl_xor_sync(0xffffffffu, sA, 2);
        sB += __shfl_xor_sync(0xffffffffu, sB, 2);
      } else {
        sA = 0.f; sB = 0.f;
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          float c4[4];
#pragma unroll
          for (int ks = 0; ks < KS_PER_G; ++ks) kstep(c4, g * KS_PER_G + ks, ks == 0);
          float s_, z_;
          kmeta(rA, g, s_, z_);
          sA = fmaf(s_, c4[0] + c4[1], fmaf(z_, Qg[g], sA));
          kmeta(rB, g, s_, z_);
          sB = fmaf(s_, c4[2] + c4[3], fmaf(z_, Qg[g], sB));
        }
      }
      sA_out = sA;
      sB_out = sB;
    };

    // OUTER: operand fragments and constants of one key group (G tokens) from its 128 metadata words `kmj` (scale |
    // zero-point << 16, ordered like block_meta_index): Bq <- q'' * S_j, hi / lo split, scaled below 2^QE by the
    // group's largest scale; kconst <- sum_c q''_c Z_jc of this lane's accumulator head; kfac_cur undoes the scaling.
    float kconst = 0.f, kfac_cur = 0.f;
    auto outer_group = [&](const uint32_t* kmj) {
      auto entry = [&](int ks, int rr) { return ((2 * ks + rr) & 7) * 16 + (ks >> 2) * 8 + 2 * j; };   // channels 16ks+2j+8rr, +1
      float smax = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          const uint2 w = *reinterpret_cast<const uint2*>(kmj + entry(ks, rr));
          smax = fmaxf(smax, fmaxf(fabsf(__low2float(*reinterpret_cast<const __half2*>(&w.x))),
                                   fabsf(__low2float(*reinterpret_cast<const __half2*>(&w.y)))));
        }
      smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, 1));
      smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, 2));
      const int eS = smax > 0.f ? ((__float_as_int(smax) >> 23) & 0xff) - 126 : 0;     // smax < 2^eS
      const int bexp = QE - qe_s[4 + (gid >> 1)] - eS;          // qe_s[4 + h]: exponent of max |q''| of head h
      float zc = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          const uint2 w = *reinterpret_cast<const uint2*>(kmj + entry(ks, rr));
          const __half2 h0 = *reinterpret_cast<const __half2*>(&w.x), h1 = *reinterpret_cast<const __half2*>(&w.y);
          const int c0 = 16 * ks + 2 * j + 8 * rr;
          const float q0 = q_raw_s[(gid >> 1) * kD + c0], q1 = q_raw_s[(gid >> 1) * kD + c0 + 1];
          const int kk = (ks % (2 * KPW)) % KPW;
          const float scl = pow2i(bexp - KP * (2 * kk + rr));
          const uint32_t v0 = split_hi_lo(q0 * fabsf(__low2float(h0)) * scl);
          const uint32_t v1 = split_hi_lo(q1 * fabsf(__low2float(h1)) * scl);
          Bq[ks][rr] = (gid & 1) ? ((v0 >> 16) | (v1 & 0xFFFF0000u)) : ((v0 & 0xFFFFu) | (v1 << 16));
          zc = fmaf(q0, __high2float(h0), fmaf(q1, __high2float(h1), zc));
        }
      zc += __shfl_xor_sync(0xffffffffu, zc, 1);
      zc += __shfl_xor_sync(0xffffffffu, zc, 2);
      kconst = __shfl_sync(0xffffffffu, zc, 8 * j);          // lanes 8j .. 8j+7 hold head j's sum
      kfac_cur = pow2i(24 - (QE - qe_s[4 + j] - eS));
    };

    // Fragments of raw q'' for the fp16 key rows of this warp's tail tiles (registers only while those run).
    // SPLIT reuses the table area for its side ring, so the tables are released now, while all warps are in step.
    uint32_t Bqr[8][2];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      Bqr[s][0] = tw > 0 ? bqr_s[(s * 2) * 32 + lane] : 0u;
      Bqr[s][1] = tw > 0 ? bqr_s[(s * 2 + 1) * 32 + lane] : 0u;
    }
    const float kfac_raw = pow2i(-(14 - qe_s[4 + my_head]));       // fp16 key rows: accumulator * kfac_raw
    // From here on every warp uses its slice of the table area as scratch (the side ring of SPLIT, the exchange of
    // decoded value metadata otherwise): all warps have taken their table entries into registers by now.
    __syncthreads();
    if constexpr (SPLIT) {
      for (int i = lane; i < SL::kSideBytes / 4; i += 32) side[i] = 0u;
      __syncwarp();
    }

    float m_run = -INFINITY, l_part = 0.f, psum = 0.f;
    float out_acc[8][2];
    float accg[8][4];
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      out_acc[m][0] = out_acc[m][1] = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) accg[m][e] = 0.f;
    }
    bool failed = false;
    // OUTER: sum_t p_t Z_{t,g} per channel group (this lane's tokens, head tid4), and the value operand of 16 tokens:
    // p * S_{t,g} as fp16, one set per half of the m-tiles when there is more than one channel group (G = 32: the
    // two groups an m-tile's rows fall into share a set as its two column variants).
    constexpr int NSET = OUTER && NG > 1 ? 2 : 1;
    float zacc[OUTER ? NG : 1];
#pragma unroll
    for (int g = 0; g < (OUTER ? NG : 1); ++g) zacc[g] = 0.f;
    // meta_rows: the chunk's value metadata rows [token][NG]; tok: token inside the chunk; pos: field position
    auto outer_v_operand = [&](const uint32_t* meta_rows, int tok, float p, int pos, uint32_t (&pk)[NSET]) {
      float ps[NG];
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        const uint32_t w = meta_rows[tok * NG + g];
        const __half2 h2 = *reinterpret_cast<const __half2*>(&w);
        zacc[g] = fmaf(p, __high2float(h2), zacc[g]);
        ps[g] = p * fabsf(__low2float(h2)) * pow2i(VBASE - VP * pos);
      }
#pragma unroll
      for (int st_ = 0; st_ < NSET; ++st_) {
        if constexpr (NG == 4)
          pk[st_] = pack_half2_rn(ps[2 * st_], ps[2 * st_ + 1]);
        else
          pk[st_] = pack_half2_rn(ps[NG == 2 ? st_ : 0], 0.f);
      }
    };

    // ---------------- tail tiles of this warp: fp16 windows and the K/V skew zone -------------------
    // 16 tokens at a time, operands straight from global memory (coalesced 128-bit loads), into the warp's
    // running soft-max state.  Keys: fp16 rows against raw q'' (pieces tid4 + 4i of rows gid, gid + 8), or the
    // packed rows of the skew zone through the same path as the main loop.  Values: fp16 rows, pieces gid and
    // gid + 8 of token rows 2*tid4, 2*tid4 + 1 (+8), byte-permuted into (channel; token pair) fragments.
    // After the wait for the predecessor kernel these rows go through the read-only path; a warp that went on after
    // its look at the append's counter reads them at the L2 cache (the acquire covers ordinary loads, and this SM's
    // read-only cache may still hold the rows as an earlier decode saw them).
    if (tw > 0) wait_for_append();   // the rings and the newest packed rows are what the append writes
    for (int k = 0; k < tw; ++k) {
      bool skew; int e0, cnt;
      tail_tile(k, skew, e0, cnt);
      float sA, sB;                                            // true log2-domain scores of entries e0+gid, e0+gid+8
      if (skew && !OUTER) {
        const int iq = cn.n_qv + e0;                           // first packed key row of the tile (16-aligned)
        const unsigned char* rec = group_rec((iq / kChunk) / CH) + (size_t)((iq / kChunk) % CH) * SL::kRec;
        k_mtile(reinterpret_cast<const uint32_t*>(rec), reinterpret_cast<const uint32_t*>(rec + SL::kOffKMeta),
                iq % kChunk, sA, sB);
        sA *= kfac;
        sB *= kfac;
      } else {
        const uint4* ra = k_row(skew, e0 + min(gid, cnt - 1));
        const uint4* rb = k_row(skew, e0 + min(gid + 8, cnt - 1));
        uint4 ka[4], kb[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { ka[i] = ld_tail(ra + j + 4 * i); kb[i] = ld_tail(rb + j + 4 * i); }
        float c4[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (i == 0) mma16816_z(c4, ka[i].x, kb[i].x, ka[i].y, kb[i].y, Bqr[0][0], Bqr[0][1]);
          else mma16816(c4, ka[i].x, kb[i].x, ka[i].y, kb[i].y, Bqr[2 * i][0], Bqr[2 * i][1]);
          mma16816(c4, ka[i].z, kb[i].z, ka[i].w, kb[i].w, Bqr[2 * i + 1][0], Bqr[2 * i + 1][1]);
        }
        sA = (c4[0] + c4[1]) * kfac_raw;
        sB = (c4[2] + c4[3]) * kfac_raw;
        if constexpr (SPLIT) {       // only column pair 0 carries the head: hand its sums to the whole quad
          sA = __shfl_sync(0xffffffffu, sA, lane & ~3);
          sB = __shfl_sync(0xffffffffu, sB, lane & ~3);
        }
      }
      if (gid >= cnt) sA = -INFINITY;
      if (gid + 8 >= cnt) sB = -INFINITY;
      if (a.n_q > 1) {
        // causal mask of this lane's query row: entries at absolute positions >= pos_end are newer than its token
        auto pos = [&](int e) {
          return skew ? cn.n_sink + min(cn.n_qk, cn.n_qv) + e
                      : (e < cn.n_sink ? e : max(cn.n_qk, cn.n_qv) + e);      // n_sink + n_packed + (e - n_sink)
        };
        if (pos(e0 + gid) >= pos_end) sA = -INFINITY;
        if (pos(e0 + gid + 8) >= pos_end) sB = -INFINITY;
      }
      float cmax = fmaxf(sA, sB);
      cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 4));
      cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
      cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));
      const float m_new = fmaxf(m_run, cmax);
      // 0 while m_run = -inf; a tile that is masked completely for this row leaves the state as it is
      const float alpha = m_new == -INFINITY ? 1.f : ex2_approx(m_run - m_new);
      m_run = m_new;
      l_part *= alpha;
#pragma unroll
      for (int m = 0; m < 8; ++m) { out_acc[m][0] *= alpha; out_acc[m][1] *= alpha; }
      if constexpr (OUTER) {
#pragma unroll
        for (int g = 0; g < NG; ++g) zacc[g] *= alpha;
#pragma unroll
        for (int m = 0; m < 8; ++m)
#pragma unroll
          for (int e = 0; e < 4; ++e) accg[m][e] *= alpha;
      }
      const float pA = sA == -INFINITY ? 0.f : ex2_approx(sA - m_new), pB = sB == -INFINITY ? 0.f : ex2_approx(sB - m_new);
      l_part += pA + pB;
      if (OUTER && skew) {
        // values of the skew zone are packed (half a chunk: one k-step of 16 tokens), read straight from global memory
        const int iq = cn.n_qk + e0, ci = iq / kChunk, ks = (iq % kChunk) / 16;
        const unsigned char* rec = group_rec(ci / CH) + SL::kVMeta + (size_t)(ci % CH) * SL::kRec;
        const uint32_t* vmr = reinterpret_cast<const uint32_t*>(rec + SL::kOffKMeta);
        const uint32_t* vcg = reinterpret_cast<const uint32_t*>(rec + SL::kOffVCodes);
        uint32_t Bt[NSET][2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t pk[NSET];
          outer_v_operand(vmr, 16 * ks + gid + 8 * h, h ? pB : pA, h, pk);   // fields are shifted down to position h below
#pragma unroll
          for (int st_ = 0; st_ < NSET; ++st_) Bt[st_][h] = movmatrix_trans(pk[st_]);
        }
        if constexpr (VP == 2) {
          const uint4 v0 = ld_tail(reinterpret_cast<const uint4*>(vcg + lane * 4));
          const uint4 v1 = ld_tail(reinterpret_cast<const uint4*>(vcg + 128 + lane * 4));
          const uint32_t vw[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
          for (int m = 0; m < 8; ++m) {
            const uint32_t w0 = vw[m] >> (4 * ks), w1 = w0 >> 8;          // this k-step's fields at positions 0 and 1
            const uint32_t m0 = FV::kField, m1 = FV::kField << 2;
            mma16816(accg[m], w0 & m0, w1 & m0, w0 & m1, w1 & m1, Bt[NSET > 1 ? m >> 2 : 0][0], Bt[NSET > 1 ? m >> 2 : 0][1]);
          }
        } else {
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const uint4 v = ld_tail(reinterpret_cast<const uint4*>(vcg + ks * 256 + hh * 128 + lane * 4));
            const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int mm = 0; mm < 4; ++mm) {
              const uint32_t w0 = vw[mm], w1 = vw[mm] >> 8;
              const uint32_t m0 = FV::kField, m1 = FV::kField << 4;
              mma16816(accg[hh * 4 + mm], w0 & m0, w1 & m0, w0 & m1, w1 & m1, Bt[NSET > 1 ? hh : 0][0], Bt[NSET > 1 ? hh : 0][1]);
            }
          }
        }
        continue;
      }
      uint32_t pkA = split_hi_lo(pA * 1024.f), pkB = split_hi_lo(pB * 1024.f);
      if (SPLIT && j != 0) { pkA = 0u; pkB = 0u; }              // SPLIT: lane 0 of each quad takes the tail's sums
      const uint32_t b0 = movmatrix_trans(pkA), b1 = movmatrix_trans(pkB);
      const uint4* vr[4] = {v_row(skew, e0 + min(2 * j, cnt - 1)), v_row(skew, e0 + min(2 * j + 1, cnt - 1)),
                            v_row(skew, e0 + min(2 * j + 8, cnt - 1)), v_row(skew, e0 + min(2 * j + 9, cnt - 1))};
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint4 v4[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) v4[r] = ld_tail(vr[r] + gid + 8 * hh);
        const uint32_t* T0 = reinterpret_cast<const uint32_t*>(&v4[0]);
        const uint32_t* T1 = reinterpret_cast<const uint32_t*>(&v4[1]);
        const uint32_t* T8 = reinterpret_cast<const uint32_t*>(&v4[2]);
        const uint32_t* T9 = reinterpret_cast<const uint32_t*>(&v4[3]);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {                        // m-tile 4*hh + kk: channels 64*hh + 8*gid + 2*kk (+1)
          float c4[4];
          mma16816_z(c4, __byte_perm(T0[kk], T1[kk], 0x5410), __byte_perm(T0[kk], T1[kk], 0x7632),
                     __byte_perm(T8[kk], T9[kk], 0x5410), __byte_perm(T8[kk], T9[kk], 0x7632), b0, b1);
          // out_acc is kept in units of 2^-14; these sums carry p * 2^10
          out_acc[4 * hh + kk][0] = fmaf(c4[0] + c4[1], 0x1p-24f, out_acc[4 * hh + kk][0]);
          out_acc[4 * hh + kk][1] = fmaf(c4[2] + c4[3], 0x1p-24f, out_acc[4 * hh + kk][1]);
        }
      }
    }

    // From here on this warp reads nothing that the next step's append writes (the fp16 rings and packed rows /
    // groups that do not exist yet).  When that holds for every warp of the CTA, the CTA lets the next kernel in the
    // stream start (one call per CTA counts, so the last warp to get here makes it); dependents start when every
    // CTA has.  One warp per unit gets here only after it has seen the unit's last append complete, so the next
    // append (which works first and waits afterwards) finds its predecessor's writes in place and nobody reading
    // what it is about to overwrite.  The step's append thus runs while this kernel streams, not after it.
    if (split == 0 && warp == 0) wait_for_append();
    __syncwarp();
    if (lane == 0 && atomicAdd(&s_past_tail, 1u) == kWarps - 1) grid_launch_dependents();

    // The loop body is deliberately not unrolled over iterations: two CTAs of eight warps walk it at
    // different phases, so it has to stay resident in the instruction cache.
#pragma unroll 1
    for (int it = 0; it < n_iters; ++it) {
      const int st = it & (NST - 1);
      const uint32_t parity = (uint32_t)(it / NST) & 1u;
      if (!mbar_wait(bars_u32 + 8 * st, parity)) { failed = true; break; }
      const unsigned char* sp = ring + st * SL::kBytes;
      const int ci0 = c_lo + it * CPI;                           // first chunk of this iteration (unit-relative)
      const bool last_valid = CPI == 1 || (it * CPI + 1 < n_chunks_w);   // odd chunk count: the last half is empty

      // ---------------- raw scores: CPI * 2 m-tiles of 16 tokens -------------------------------------
      float sc[CPI][2][2];
#pragma unroll
      for (int cc = 0; cc < CPI; ++cc) {
        if (cc > 0 && !last_valid) {      // nothing there: this warp's range ends in the middle of the iteration
          sc[cc][0][0] = sc[cc][0][1] = sc[cc][1][0] = sc[cc][1][1] = -INFINITY;
          continue;
        }
        // OUTER: a group's first chunk is preceded in the stage by the key group's metadata
        const int lead = OUTER && ((ci0 + cc) & (CH - 1)) == 0 ? SL::kVMeta : 0;
        if constexpr (OUTER) {
          if (lead) outer_group(reinterpret_cast<const uint32_t*>(sp));
        }
        const uint32_t* kc = reinterpret_cast<const uint32_t*>(sp + lead + SL::off(cc));
        const uint32_t* km = reinterpret_cast<const uint32_t*>(sp + lead + SL::off(cc) + SL::kOffKMeta);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          float sA = 0.f, sB = 0.f;
          if constexpr (!(ABL & 1)) k_mtile(kc, km, 16 * mt, sA, sB);      // (else: timing experiment, no key side)
          if constexpr (OUTER) {       // true log2-domain scores right away (the scaling changes from group to group)
            sA = fmaf(sA, kfac_cur, kconst);
            sB = fmaf(sB, kfac_cur, kconst);
          }
          const bool valid = cc == 0 || last_valid;
          sc[cc][mt][0] = valid ? sA : -INFINITY;
          sc[cc][mt][1] = valid ? sB : -INFINITY;
        }
      }

      // ---------------- online softmax (log2 domain; raw scores still carry 1/kfac) -------------------
      // The reference m_run of the running sums is any value within kLazy of the largest score so far, not the
      // maximum itself: it only moves (with the cross-lane reduction and the rescaling that takes) when a score of
      // this iteration exceeds it by more than kLazy, so p <= 2^kLazy and the usual iteration needs one vote.
      constexpr float kLazy = OUTER ? 0.f : 4.f;
      float cmax = -INFINITY;
#pragma unroll
      for (int cc = 0; cc < CPI; ++cc)
        cmax = fmaxf(cmax, fmaxf(fmaxf(sc[cc][0][0], sc[cc][0][1]), fmaxf(sc[cc][1][0], sc[cc][1][1])));
      const float kf = OUTER ? 1.0f : kfac;                    // what the raw scores still have to be multiplied by
      float m_new = m_run;
      if (__any_sync(0xffffffffu, cmax * kf > m_run + kLazy)) {
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 4));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));
        m_new = fmaxf(m_run, cmax * kf);
        const float alpha = ex2_approx(m_run - m_new);     // 0 on the first iteration (m_run = -inf)
        l_part *= alpha;
        psum *= alpha;
        if constexpr (OUTER) {
#pragma unroll
          for (int g = 0; g < NG; ++g) zacc[g] *= alpha;
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          out_acc[m][0] *= alpha; out_acc[m][1] *= alpha;
#pragma unroll
          for (int e = 0; e < 4; ++e) accg[m][e] *= alpha;
        }
      }
      m_run = m_new;

#pragma unroll
      for (int cc = 0; cc < CPI; ++cc) {
        if (cc > 0 && !last_valid) continue;
        const int ci = ci0 + cc;
        const int lead = OUTER && (ci & (CH - 1)) == 0 ? SL::kVMeta : 0;
        const uint32_t* vc = reinterpret_cast<const uint32_t*>(sp + lead + SL::off(cc) + SL::kOffVCodes);
        const uint32_t* vm = reinterpret_cast<const uint32_t*>(sp + SL::off(cc) + SL::kRec);
        // slot: position of this chunk's value group in the SPLIT window / position of the chunk in its group
        const int slot = SPLIT ? (ci - c_lo) & (WIN - 1) : ci % CH;
        const bool group_start = slot == 0;
        const bool group_end = SPLIT ? (slot == WIN - 1 || (it == n_iters - 1 && (cc == CPI - 1 || !last_valid)))
                                     : (slot == CH - 1);
        constexpr bool kFreshEveryChunk = !SPLIT && !OUTER && CH == 1;   // then the first value mma takes a zero C
        if (!OUTER && !kFreshEveryChunk && group_start) {
#pragma unroll
          for (int m = 0; m < 8; ++m)
#pragma unroll
            for (int e = 0; e < 4; ++e) accg[m][e] = 0.f;
        }
        uint32_t Bps[NSET][2][2];
        uint32_t (&Bp)[2][2] = Bps[0];
        float psum_c = 0.f;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const float p = ex2_approx(fmaf(sc[cc][mt][h], kf, -m_new));
            psum_c += p;
            const int pos = VP == 2 ? 2 * mt + h : h;
            if constexpr (OUTER) {
              uint32_t pks[NSET];
              outer_v_operand(reinterpret_cast<const uint32_t*>(sp + lead + SL::off(cc) + SL::kOffKMeta), 16 * mt + gid + 8 * h, p,
                              pos, pks);
#pragma unroll
              for (int st_ = 0; st_ < NSET; ++st_) Bps[st_][mt][h] = movmatrix_trans(pks[st_]);
              continue;
            }
            // p goes in as one fp16 (the lo column stays zero): its 2^-12 relative rounding is random per token and
            // far inside the output tolerance, and it saves the hi/lo split of every probability
            uint32_t pk = pack_half2_rn(p * pow2i(10 - VP * pos), 0.f);
            if (SPLIT && j != slot) pk = 0u;                 // column pair of this chunk's window slot only
            Bp[mt][h] = movmatrix_trans(pk);
          }
        }
        l_part += psum_c;
        if constexpr (SPLIT) psum += (j == slot) ? psum_c : 0.f;
        else psum += psum_c;

        // ---------------- values: 8 m-tiles of 16 channels x 2 k-steps of 16 tokens ------------------
        if constexpr (ABL & 2) {
          // timing experiment: no value side
        } else if constexpr (VP == 2) {
          const uint4 v0 = *reinterpret_cast<const uint4*>(vc + lane * 4);
          const uint4 v1 = *reinterpret_cast<const uint4*>(vc + 128 + lane * 4);
          const uint32_t vw[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
          for (int m = 0; m < 8; ++m) {
            const uint32_t w0 = vw[m], w1 = vw[m] >> 8;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
              const uint32_t m0 = FV::kField << (2 * (2 * ks)), m1 = FV::kField << (2 * (2 * ks + 1));
              if (kFreshEveryChunk && ks == 0) mma16816_z(accg[m], w0 & m0, w1 & m0, w0 & m1, w1 & m1, Bp[ks][0], Bp[ks][1]);
              else mma16816(accg[m], w0 & m0, w1 & m0, w0 & m1, w1 & m1, Bps[NSET > 1 ? m >> 2 : 0][ks][0], Bps[NSET > 1 ? m >> 2 : 0][ks][1]);
            }
          }
        } else {
#pragma unroll
          for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              const uint4 v = *reinterpret_cast<const uint4*>(vc + ks * 256 + hh * 128 + lane * 4);
              const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int mm = 0; mm < 4; ++mm) {
                const uint32_t w0 = vw[mm], w1 = vw[mm] >> 8;
                const uint32_t m0 = FV::kField, m1 = FV::kField << 4;
                if (kFreshEveryChunk && ks == 0)
                  mma16816_z(accg[hh * 4 + mm], w0 & m0, w1 & m0, w0 & m1, w1 & m1, Bp[ks][0], Bp[ks][1]);
                else
                  mma16816(accg[hh * 4 + mm], w0 & m0, w1 & m0, w0 & m1, w1 & m1, Bps[NSET > 1 ? hh : 0][ks][0], Bps[NSET > 1 ? hh : 0][ks][1]);
              }
            }
          }
        }

        if constexpr (VB == 3 && !(ABL & 2)) {
          // 1-bit plane (weight 4): 4 words per lane, word m/2 holds fields ((m%2)*2 + rh)*4 + 2*ks + kh
          const uint4 hv = *reinterpret_cast<const uint4*>(vc + 256 + lane * 4);
          const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w};
          uint32_t Bh[2][2];
#pragma unroll
          for (int ks = 0; ks < 2; ++ks)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const __half2 f = __float2half2_rn(pow2i(2 * ks + h + 2));      // 4^pos * 4 / 2^pos of the p fragment
              const __half2 bb = __hmul2(*reinterpret_cast<const __half2*>(&Bp[ks][h]), f);
              Bh[ks][h] = *reinterpret_cast<const uint32_t*>(&bb);
            }
#pragma unroll
          for (int m = 0; m < 8; ++m) {
            const uint32_t x0 = hw[m >> 1] >> (8 * (m & 1)), x1 = hw[m >> 1] >> (8 * (m & 1) + 4);
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
              const uint32_t h0 = 0x00010001u << (2 * ks), h1 = 0x00010001u << (2 * ks + 1);
              mma16816(accg[m], x0 & h0, x1 & h0, x0 & h1, x1 & h1, Bh[ks][0], Bh[ks][1]);
            }
          }
        }

        // ---------------- end of a value group: apply scale / zero-point once per channel -----------
        const bool chunk_valid = cc == 0 || last_valid;
        if constexpr (SPLIT) {
          // keep this group's metadata for the end of the window (the stage will be refilled)
          if (chunk_valid && lane * 16 < SL::kVMeta)
            *reinterpret_cast<uint4*>(side + slot * (SL::kVMeta / 4) + lane * 4) = *reinterpret_cast<const uint4*>(vm + lane * 4);
        }
        if (!OUTER && group_end && chunk_valid) {
          if constexpr (SPLIT) __syncwarp();
          float pg = psum;
          pg += __shfl_xor_sync(0xffffffffu, pg, 4);
          pg += __shfl_xor_sync(0xffffffffu, pg, 8);
          pg += __shfl_xor_sync(0xffffffffu, pg, 16);
          pg *= 0x1p-14f;                               // accumulators carry p * 2^10 * 2^-24
          const uint32_t* vmg = SPLIT ? side + j * (SL::kVMeta / 4) : vm;    // this group's entries (slot j's in SPLIT)
          // The value sums of a lane sit in the even accumulator columns (p enters as one fp16 per token, the lo
          // column of its pair is zero), except in the outer-grouped variant.
          auto acc_sum = [&](int m, int rh) { return OUTER ? accg[m][2 * rh] + accg[m][2 * rh + 1] : accg[m][2 * rh]; };
          if constexpr (!SPLIT && VM == 4) {
            // The four lanes of a quad need the same 16 entries: every lane decodes 4 of the group's 128 once, the
            // warp exchanges (scale, zero-point) pairs through its side area (rows of 16 pairs, padded to 36 words
            // so that the 128-bit reads of the eight lane groups fall into different banks), each lane reads its 16.
            float* ds = reinterpret_cast<float*>(side);
            {
              const uint4 mw = *reinterpret_cast<const uint4*>(vmg + lane * 4);
              const uint32_t mws[4] = {mw.x, mw.y, mw.z, mw.w};
              float sz[8];
#pragma unroll
              for (int e = 0; e < 4; ++e) decode_fast(mws[e], neg_half_v, sz[2 * e], sz[2 * e + 1]);
              float* dst = ds + (lane >> 2) * 36 + (lane & 3) * 8;       // entries 4*lane .. 4*lane+3 = row lane/4
              *reinterpret_cast<float4*>(dst) = make_float4(sz[0], sz[1], sz[2], sz[3]);
              *reinterpret_cast<float4*>(dst + 4) = make_float4(sz[4], sz[5], sz[6], sz[7]);
            }
            __syncwarp();
            const float4* row = reinterpret_cast<const float4*>(ds + gid * 36);
#pragma unroll
            for (int q8 = 0; q8 < 8; ++q8) {
              const float4 v = row[q8];                                   // entries 2*q8, 2*q8 + 1: (s, z, s, z)
              const int m = q8;                                           // entry idx = 2 * m + rh
              out_acc[m][0] = fmaf(v.x, acc_sum(m, 0), fmaf(v.y, pg, out_acc[m][0]));
              out_acc[m][1] = fmaf(v.z, acc_sum(m, 1), fmaf(v.w, pg, out_acc[m][1]));
            }
            __syncwarp();                                                 // the side area is reused at the next group end
          } else if constexpr (VM == 4) {
            const uint4* vm4 = reinterpret_cast<const uint4*>(vmg + gid * 16);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const uint4 mw = vm4[q4];
              const uint32_t mws[4] = {mw.x, mw.y, mw.z, mw.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int idx = q4 * 4 + e, m = idx >> 1, rh = idx & 1;    // fragment row (m, rh) of lane group gid
                float s_, z_;
                decode_fast(mws[e], neg_half_v, s_, z_);
                out_acc[m][rh] = fmaf(s_, acc_sum(m, rh), fmaf(z_, pg, out_acc[m][rh]));
              }
            }
          } else {
            const uint4* vm4 = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(vmg) + gid * 16);
#pragma unroll
            for (int q4 = 0; q4 < 2; ++q4) {
              const uint4 mw = vm4[q4];
              const uint32_t mws[4] = {mw.x, mw.y, mw.z, mw.w};
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const int idx = q4 * 8 + e, m = idx >> 1, rh = idx & 1;
                const float s_ = h2f_bits((uint16_t)((mws[e >> 1] >> (16 * (e & 1))) & 0x7FFFu));
                out_acc[m][rh] = fmaf(s_, acc_sum(m, rh), fmaf(neg_half_v * s_, pg, out_acc[m][rh]));
              }
            }
          }
          psum = 0.f;
        }
      }

      __syncwarp();
      if (it + NST < n_iters) {
        dep_wait_for_iteration(it + NST);
        if (lane == 0) issue(st);
      }
    }

    // the partials and tickets written below are also shared with the previous decode
    dep_wait();
    if (failed) {
      // a copy never arrived: flag it for the host and contribute nothing
      if (lane == 0) atomicExch(reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off) + L.U, 1u);
      m_run = -INFINITY;
      l_part = 0.f;
    }

    // ---------------- warp result -> shared memory -> CTA partial ---------------------------------
    l_part += __shfl_xor_sync(0xffffffffu, l_part, 4);
    l_part += __shfl_xor_sync(0xffffffffu, l_part, 8);
    l_part += __shfl_xor_sync(0xffffffffu, l_part, 16);
    if constexpr (SPLIT) {
      // the four lanes of a quad hold the contributions of different window slots: add them up
#pragma unroll
      for (int m = 0; m < 8; ++m)
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
          float v = out_acc[m][rh];
          v += __shfl_xor_sync(0xffffffffu, v, 1);
          v += __shfl_xor_sync(0xffffffffu, v, 2);
          out_acc[m][rh] = v;
        }
    }
    if constexpr (OUTER) {
      // the value accumulators carry sum p S u * 2^(VBASE - 24); zero-points: lanes of the same head add their tokens
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        zacc[g] += __shfl_xor_sync(0xffffffffu, zacc[g], 4);
        zacc[g] += __shfl_xor_sync(0xffffffffu, zacc[g], 8);
        zacc[g] += __shfl_xor_sync(0xffffffffu, zacc[g], 16);
      }
      const bool up = (gid >> 2) != 0;                 // G = 32: rows of lanes 16..31 belong to the m-tile's second group
#pragma unroll
      for (int m = 0; m < 8; ++m)
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
          float sel, zz;
          if constexpr (NG == 4) {
            sel = up ? accg[m][2 * rh + 1] : accg[m][2 * rh];
            zz = up ? zacc[2 * (m >> 2) + 1] : zacc[2 * (m >> 2)];
          } else {
            sel = accg[m][2 * rh];
            zz = zacc[NG == 2 ? (m >> 2) : 0];
          }
          out_acc[m][rh] += sel * pow2i(10 - VBASE) + zz * 0x1p-14f;
        }
    }
    __syncthreads();                                   // every warp is done with its ring
    float* wres = reinterpret_cast<float*>(smem);      // [warp][head][kD + 2]
    const bool writer = SPLIT ? (j == 0) : true;
    const bool any = n_iters > 0 || tw > 0;
    if (writer) {
      float* mine = wres + ((size_t)warp * kHeads + (SPLIT ? 0 : j)) * (kD + 2);
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        mine[block_row_channel(m, 0, gid)] = any ? out_acc[m][0] * 0x1p14f : 0.f;
        mine[block_row_channel(m, 1, gid)] = any ? out_acc[m][1] * 0x1p14f : 0.f;
      }
      if (gid == 0) {
        mine[kD] = any ? m_run : -INFINITY;
        mine[kD + 1] = any ? l_part : 0.f;
      }
    }
    __syncthreads();
    float* partials = a.partials;
    for (int i = tid; i < nh * kD; i += kThreads) {
      const int h = i >> 7, c = i & (kD - 1);
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) M = fmaxf(M, wres[((size_t)w * kHeads + h) * (kD + 2) + kD]);
      float num = 0.f, den = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float* r_ = wres + ((size_t)w * kHeads + h) * (kD + 2);
        const float wgt = r_[kD] == -INFINITY ? 0.f : ex2_approx(r_[kD] - M);
        num = fmaf(r_[c], wgt, num);
        den = fmaf(r_[kD + 1], wgt, den);
      }
      float* P = partials + ((size_t)(prow0 + h) * L.max_splits + split) * kPartialStride;
      P[c] = num;
      if (c == 0) { P[kD] = M; P[kD + 1] = den; }
    }
  }

  // ---------------- cross-CTA merge: the last CTA of the unit to arrive combines all parts -----------
  __shared__ unsigned int s_ticket;
  __syncthreads();                 // all partial writes of this CTA happen-before thread 0's ticket below
  if (tid == 0) {
    // release: publishes the whole CTA's partial (ordered before this thread by the barrier) with the ticket;
    // acquire: the CTA that draws the last ticket sees every other CTA's partial
    unsigned int t;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;"
                 : "=r"(t) : "l"(reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off) + u) : "memory");
    s_ticket = t;
  }
  __syncthreads();
  if (s_ticket != a.grid_y - 1) return;
  merge_parts(a.partials, reinterpret_cast<float*>(smem), a.out, nh, n_parts, prow0,
              make_int4(q_row(0), q_row(1), q_row(2), q_row(3)), L.max_splits);
  if (tid == 0) reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off)[u] = 0u;   // ready for the next launch
}

// One cache: block x = unit.
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false, bool PAGED = false, int ABL = 0>
__global__ void __launch_bounds__(kThreads, 2)
decode_mma_kernel(const Layout L, const Counts cn, const DecodeArgs a) {
  decode_mma_body<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, PAGED, ABL>(L, cn, a, blockIdx.x);
}

// One paged cache with its page table in the parameter space (read in place: no look-up in device memory).
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false>
__global__ void __launch_bounds__(kThreads, 2)
decode_mma_paged_kernel(const Layout L, const Counts cn, const DecodeArgs a, const __grid_constant__ PageIds P) {
  decode_mma_body<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, true>(L, cn, a, blockIdx.x, &P);
}
// Several caches of one configuration: block x = sequence * U + unit, the sequence's counts and parameters come
// from its table entry (read in place from the parameter space).
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false, bool PAGED = false>
__global__ void __launch_bounds__(kThreads, 2)
decode_mma_batched_kernel(const __grid_constant__ Layout L, const __grid_constant__ SeqTable T) {
  const int seq = blockIdx.x / L.U;
  decode_mma_body<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, PAGED>(L, T.s[seq].cn, T.s[seq].a, blockIdx.x - seq * L.U);
}

// Split-dependent launch parameters of one cache for a grid of grid_y rows (0: choose it): how many of the rows
// stream packed chunks, the range units per row, the tail tiles per row.  Returns grid_y.
template <int RU>
int fill_split_args(const Layout& L, const Counts& cn, DecodeArgs& a, bool outer, int n_splits, int grid_y) {
  const int n_chunks = (outer ? cn.n_qk : cn.n_qv) / kChunk;
  const int n_units = (n_chunks + RU - 1) / RU;
  const int by_work = (n_units + kWarps - 1) / kWarps;      // at least one range unit per warp
  if (n_splits > by_work) n_splits = by_work;
  if (n_units == 0) n_splits = 0;
  if (grid_y <= 0) {
    // without packed chunks the CTAs only share the tail tiles (eight per CTA)
    grid_y = n_splits > 0 ? n_splits : (a.n_tail_tiles + kWarps - 1) / kWarps;
    if (grid_y < 1) grid_y = 1;
    if (grid_y > L.max_splits) grid_y = L.max_splits;
  }
  if (n_splits > grid_y) n_splits = grid_y;
  a.grid_y = grid_y;
  a.n_splits = n_splits;
  a.tail_cost_units = n_splits ? 1 : 0;     // a tail tile costs a warp about as much as one value group's chunks
  const int virt = n_units + a.tail_cost_units * a.n_tail_tiles;
  a.units_per_split = n_splits ? (virt + n_splits - 1) / n_splits : 0;
  a.tiles_q0 = a.n_tail_tiles / grid_y;
  a.tiles_rem = a.n_tail_tiles % grid_y;
  return grid_y;
}

template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false, bool PAGED = false>
int launch_one_p(const Layout& L, const Counts& cn, DecodeArgs a, int n_splits, cudaStream_t st) {
  using SL = StageLayout<KB, VB, G, KM, VM, CPI>;
  constexpr int kSmem = SL::kCtaBytes;
  constexpr int RU = SL::kCH;
  static std::atomic<unsigned long long> configured{0};
  if (!opt_in_dynamic_smem(decode_mma_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, PAGED>, kSmem, configured)) return -1;
  // a paged cache whose page list fits the parameter space: the kernel that takes the table as a parameter
  [[maybe_unused]] PageIds ids;
  bool table_in_params = false;
  if constexpr (PAGED) {
    static std::atomic<unsigned long long> configured_p{0};
    if (a.pages_host && a.n_pages_host <= kParamPages) {
      if (!opt_in_dynamic_smem(decode_mma_paged_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER>, kSmem, configured_p)) return -1;
      for (int i = 0; i < a.n_pages_host; ++i) ids.id[i] = a.pages_host[i];
      table_in_params = true;
    }
  }
  const int grid_y = fill_split_args<RU>(L, cn, a, OUTER, n_splits, 0);
  dim3 grid(L.U, grid_y);
  int launches = 0;
  const int step = SPLIT ? 1 : kHeads;
  for (int h0 = 0; h0 < L.r * a.n_q; h0 += step) {
    a.head0 = h0;
    // launched as a programmatic dependent of whatever precedes it in the stream: its set-up overlaps that
    // kernel's tail, its first global access waits for it (grid_dependency_wait)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t err;
    if constexpr (PAGED) {
      if (a.ablation) return -2;      // the timing instances exist for contiguous caches only
      err = table_in_params ? cudaLaunchKernelEx(&cfg, decode_mma_paged_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER>, L, cn, a, ids)
                            : cudaLaunchKernelEx(&cfg, decode_mma_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, PAGED>, L, cn, a);
    } else if (a.ablation == 1 || a.ablation == 2) {
#ifdef IQ_WITH_TIMING_INSTANCES      // defined by the translation units of the formats the latency study times
      static std::atomic<unsigned long long> configured_a1{0}, configured_a2{0};
      if (a.ablation == 1) {
        if (!opt_in_dynamic_smem(decode_mma_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, false, 1>, kSmem, configured_a1)) return -1;
        err = cudaLaunchKernelEx(&cfg, decode_mma_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, false, 1>, L, cn, a);
      } else {
        if (!opt_in_dynamic_smem(decode_mma_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, false, 2>, kSmem, configured_a2)) return -1;
        err = cudaLaunchKernelEx(&cfg, decode_mma_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, false, 2>, L, cn, a);
      }
#else
      return -2;
#endif
    } else {
      err = cudaLaunchKernelEx(&cfg, decode_mma_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, PAGED>, L, cn, a);
    }
    if (err != cudaSuccess) return -1;
    ++launches;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// The same kernel over a table of caches.  Every sequence splits its own chunks over as many of the launch's
// grid rows as it has work for; the rows beyond that only take their share of its tail tiles.
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false, bool PAGED = false>
int launch_one_batched_p(const Layout& L, SeqTable& T, int n_seqs, int n_splits, cudaStream_t st) {
  using SL = StageLayout<KB, VB, G, KM, VM, CPI>;
  constexpr int kSmem = SL::kCtaBytes;
  constexpr int RU = SL::kCH;
  static std::atomic<unsigned long long> configured{0};
  if (!opt_in_dynamic_smem(decode_mma_batched_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, PAGED>, kSmem, configured)) return -1;
  // Grid rows per sequence: the fewest chunks per row T such that all sequences together, each cut into rows of at
  // most T chunks, need no more than n_splits rows in total (so the longest row, which sets the time, is as short
  // as one wave of CTAs allows, and short sequences hold few CTAs).
  long long chunks[kMaxSeqs], longest = 1;
  for (int i = 0; i < n_seqs; ++i) {
    chunks[i] = (OUTER ? T.s[i].cn.n_qk : T.s[i].cn.n_qv) / kChunk;
    if (chunks[i] > longest) longest = chunks[i];
  }
  const long long budget = n_splits;                    // rows of all sequences together (each row is U CTAs)
  auto rows_needed = [&](long long t) {
    long long r = 0;
    for (int i = 0; i < n_seqs; ++i) r += chunks[i] > 0 ? (chunks[i] + t - 1) / t : 1;
    return r;
  };
  long long lo = 1, hi = longest;                       // smallest t with rows_needed(t) <= budget (hi always fits)
  while (lo < hi) {
    const long long mid = (lo + hi) / 2;
    if (rows_needed(mid) <= budget) hi = mid; else lo = mid + 1;
  }
  int grid_y = 1;
  for (int i = 0; i < n_seqs; ++i) {
    int want = chunks[i] > 0 ? (int)((chunks[i] + lo - 1) / lo) : 1;
    if (want > L.max_splits) want = L.max_splits;
    if (want > 128) want = 128;
    const int gy = fill_split_args<RU>(L, T.s[i].cn, T.s[i].a, OUTER, want, 0);
    if (gy > grid_y) grid_y = gy;
  }
  dim3 grid(n_seqs * L.U, grid_y);
  int launches = 0;
  const int step = SPLIT ? 1 : kHeads;
  for (int h0 = 0; h0 < L.r; h0 += step) {
    for (int i = 0; i < n_seqs; ++i) T.s[i].a.head0 = h0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_mma_batched_kernel<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, PAGED>, L, T) != cudaSuccess) return -1;
    ++launches;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// Contiguous or paged record area: two instances of every kernel, so that the contiguous one carries none of the
// page arithmetic.
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false>
int launch_one(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits, cudaStream_t st) {
  return L.page_groups > 0 ? launch_one_p<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, true>(L, cn, a, n_splits, st)
                           : launch_one_p<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, false>(L, cn, a, n_splits, st);
}
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool OUTER = false>
int launch_one_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, cudaStream_t st) {
  return L.page_groups > 0 ? launch_one_batched_p<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, true>(L, T, n_seqs, n_splits, st)
                           : launch_one_batched_p<KB, VB, G, KM, VM, SPLIT, CPI, OUTER, false>(L, T, n_seqs, n_splits, st);
}

template <int KB, int VB>
int launch_format_outer_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, cudaStream_t st) {
  if (L.G == 32) return launch_one_batched<KB, VB, 32, 4, 4, false, 1, true>(L, T, n_seqs, n_splits, st);
  if (L.G == 64) return launch_one_batched<KB, VB, 64, 4, 4, false, 1, true>(L, T, n_seqs, n_splits, st);
  if (L.G == 128) return launch_one_batched<KB, VB, 128, 4, 4, false, 1, true>(L, T, n_seqs, n_splits, st);
  return -2;
}

// The outer-grouped comparison cache with KB-bit keys and VB-bit values at every group size.
template <int KB, int VB>
int launch_format_outer(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits, cudaStream_t st) {
  if (L.G == 32) return launch_one<KB, VB, 32, 4, 4, false, 1, true>(L, cn, a, n_splits, st);
  if (L.G == 64) return launch_one<KB, VB, 64, 4, 4, false, 1, true>(L, cn, a, n_splits, st);
  if (L.G == 128) return launch_one<KB, VB, 128, 4, 4, false, 1, true>(L, cn, a, n_splits, st);
  return -2;
}

}  // namespace

// Names of the externally visible launchers of one inner-grouped format (defined by the integer-operand kernel's
// translation units), and the definition of the outer-grouped ones in the translation unit that compiles their kernels.
#define IQ_MMA_FORMAT_NAME(KB, VB, KM, VM) launch_decode_mma_k##KB##v##VB##_m##KM##VM
#define IQ_MMA_FORMAT_NAME_BATCHED(KB, VB, KM, VM) launch_decode_mma_k##KB##v##VB##_m##KM##VM##_batched
#define IQ_DEFINE_MMA_OUTER_FORMAT(KB, VB)                                                                          \
  int launch_decode_mma_outer_k##KB##v##VB(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits,    \
                                           int, cudaStream_t st) {                                                   \
    return launch_format_outer<KB, VB>(L, cn, a, n_splits, st);                                                      \
  }                                                                                                                  \
  int launch_decode_mma_outer_k##KB##v##VB##_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, int,    \
                                                     cudaStream_t st) {                                              \
    return launch_format_outer_batched<KB, VB>(L, T, n_seqs, n_splits, st);                                          \
  }

}  // namespace iq
