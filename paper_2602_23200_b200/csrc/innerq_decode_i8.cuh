// Fused decode attention over the inner-grouped packed InnerQ cache (2-, 3- or 4-bit keys, 2-, 3- or 4-bit values) on
// the 8-bit integer tensor-core instruction (mma.sync m16n8k32, u8 x s8 / u8 x u8, s32 accumulate).
//
// Same launch shape, pipeline, tail tiles and merge as the fp16-operand kernel of the outer-grouped comparison cache
// (innerq_decode_mma.cuh, whose helpers this file uses); what differs is the arithmetic core.  The cache keeps its
// codes in byte order (Store::perm = 1, see row_pos_i8 / block_pos_i8), so `word & (0x03030303 << 2p)` (2-bit codes;
// 4-bit: `word & 0x0F0F0F0F`, `word & 0xF0F0F0F0`) is four operand bytes at once: half the unpack instructions and
// half the MMAs of the fp16 path per cached element.  3-bit codes are a 2-bit and a 1-bit plane that one bit-select
// per pair of bit positions joins into 3-bit fields (see row_pos_i8_3): 1.5 logic instructions per operand word.
//   Keys.   q'' (scaled, normalised query) is split into two signed base-128 digits per channel; columns of the
//           second operand are (head, digit), or (channel group, digit) when there is one query head per KV head and
//           G = 32 (SPLIT).  The integer code sums come out exact; scale and zero-point are applied once per
//           (token, group) in fp32, as the method's inner grouping allows (Section "InnerQ").
//   Values. p = 2^(s - m) with an INTEGER reference m >= every score so far (so p <= 1 and a change of reference is
//           an exact shift of the integer accumulators) is split into two unsigned base-256 digits (16 bits); scale
//           and zero-point once per (group, channel).
// Integer accumulators start from the bit pattern of a float constant (2^23 or 1.5 * 2^23), so that reading them
// as floats and subtracting the constant converts them exactly with one fp32 addition instead of a conversion.
#pragma once
#include <type_traits>

#include "innerq_decode_mma.cuh"

namespace iq {

namespace {

__device__ __forceinline__ void imma_us(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {      // unsigned codes x signed digits
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void imma_uu(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {      // unsigned codes x unsigned digits
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the same with a constant accumulator input (every element = c0): no registers to set up for a fresh sum
__device__ __forceinline__ void imma_us_init(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1, int c0) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c0));
}
__device__ __forceinline__ void imma_uu_init(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1, int c0) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c0));
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

constexpr int kMagicS = 0x4B400000;          // bits of 1.5 * 2^23: signed sums |S| < 2^22
constexpr float kMagicSf = 12582912.0f;
constexpr int kMagicU = 0x4B000000;          // bits of 2^23: unsigned sums S < 2^23
constexpr float kMagicUf = 8388608.0f;
constexpr float kQDigits = 16256.0f;         // |q'' * bscale| <= 127 * 128: two signed base-128 digits
constexpr float kPScale = 65535.0f;          // p <= 1 as 16 bits: two unsigned base-256 digits

// G: group size; KM / VM: bytes of a metadata entry (4: scale|zero, 2: scale only); SPLIT (one query head per KV
// head, G = 32): the 8 columns are 4 groups x 2 digits for keys and 4 value groups of a window x 2 digits for
// values, which removes the 4x redundancy a quad otherwise has in decoding per-group metadata; CPI: chunks of 32
// tokens per loop iteration.
// ABL (timing experiments only, results wrong on purpose): bit 0 leaves out the key side's unpack + MMA work of the
// streaming loop (scores taken as 0), bit 1 the value side's; all bytes are still streamed.
// KB / VB: bits per key / value code (2, 3 or 4).
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool PAGED = false, int ABL = 0>
__device__ __forceinline__ void decode_i8_body(const Layout& L, const Counts& cn, const DecodeArgs& a, const int u,
                                               const PageIds* ptab = nullptr) {
  using SL = StageLayout<KB, VB, G, KM, VM, CPI>;
  static_assert(KB >= 2 && KB <= 4 && VB >= 2 && VB <= 4, "2-, 3- and 4-bit codes");
  constexpr int NG = SL::kNG;                   // key groups per token
  constexpr int CH = SL::kCH;                   // chunks per value group
  constexpr int NST = SL::kStages;
  constexpr int RW = 4 * KB;                    // 32-bit words per packed key row
  constexpr int RU = CH;                        // chunks per range unit: one value group
  constexpr int WIN = 4;                        // SPLIT: value groups per window (one per lane of a quad)
  static_assert(!SPLIT || (G == 32), "SPLIT is built for G = 32");
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
  const int n_chunks_total = cn.n_qv / kChunk;   // chunks in which keys AND values are packed
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
    const int n_meta = CPI >= CH ? CPI / CH : (((nx_ci + CPI) & (CH - 1)) == 0 ? 1 : 0);
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
  const int n_skew = cn.n_qk - cn.n_qv;
  const int n_list = cn.n_sink + cn.n_k_recent;
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
  // the values, still fp16 in the skew zone, have the zone's tokens at the head of their ring
  auto v_row = [&](bool skew, int e) -> const uint4* {
    if (!skew && e < cn.n_sink) return v_sink4 + (size_t)e * 16;
    int slot = a.v_ring_pos0 + (skew ? e : n_skew + (e - cn.n_sink));
    if (slot >= L.v.ring_cap) slot -= L.v.ring_cap;
    return v_ring4 + (size_t)slot * 16;
  };
  auto k_row = [&](bool skew, int e) -> const uint4* {
    if (!skew && e < cn.n_sink) return k_sink4 + (size_t)e * 16;
    int slot = a.k_ring_pos0 + e - cn.n_sink;
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
  float* qg_s = q_raw_s + kHeads * kD;                             // [4][4] per-group sums of the integer q''
  int* qe_s = reinterpret_cast<int*>(qg_s + kHeads * 4);           // [4] exponent of max|q''|, [4] of max |raw q''|
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int i = tid + e * kThreads;
    const float v = q_early[e] * (L.sm_scale * kLog2e);
    q_raw_s[i] = v;
    q_nrm_s[i] = v * n_early[e];
  }
  __syncthreads();
  if (warp < kHeads) {      // warp h: exponent of max |q''| of head h, then the group sums of its integer image
    float v[4], am = 0.f, amr = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[e] = q_nrm_s[warp * kD + e * 32 + lane];
      am = fmaxf(am, fabsf(v[e]));
      amr = fmaxf(amr, fabsf(q_raw_s[warp * kD + e * 32 + lane]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
      amr = fmaxf(amr, __shfl_xor_sync(0xffffffffu, amr, o));
    }
    int ex = 0;
    if (am > 0.f && am < INFINITY) ex = ((__float_as_int(am) >> 23) & 0xff) - 126;      // am < 2^ex
    const float bs = kQDigits * pow2i(-ex);
    // channel c = e * 32 + lane belongs to group c / G; the keys' zero-points meet the sum of the SAME integers the
    // MMAs see, so that the score is the dot product of one (quantised) q'' with the dequantised row
    float gs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int e = 0; e < 4; ++e) gs[(e * 32) / G] += rintf(v[e] * bs);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
      for (int g = 0; g < 4; ++g) gs[g] += __shfl_xor_sync(0xffffffffu, gs[g], o);
    if (lane == 0) {
#pragma unroll
      for (int g = 0; g < 4; ++g) qg_s[warp * 4 + g] = gs[g];
      qe_s[warp] = ex;
      int er = 0;
      if (amr > 0.f && amr < INFINITY) er = ((__float_as_int(amr) >> 23) & 0xff) - 126;
      qe_s[4 + warp] = er;
    }
  }
  __syncthreads();

  {
    // ======================= fast path: packed keys and values ===================================
    // ---- per-thread constants.  As owner of B-fragment column gid: (head, digit) or, in SPLIT, (group, digit).
    const int col_head = SPLIT ? 0 : (gid >> 1), col_group = gid >> 1, col_part = gid & 1;
    // The fragment values depend on (lane, k-step, register) only, not on the warp: warp w computes the entries of
    // k-step (bit position) w % 4, register w / 4 for every lane once, all warps then read their 8 registers.
    uint32_t* bq_s = reinterpret_cast<uint32_t*>(qe_s + 16);      // [4 positions][2][32 lanes]
    uint32_t* bqr_s = bq_s + 256;                                  // [8 k-steps][2][32 lanes]: raw q against fp16 key rows
    {
      const float bs = kQDigits * pow2i(-qe_s[col_head]);
      const int g = warp & 3, rr = warp >> 2;
      uint32_t v = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // byte i of B register rr at k-step g: k = 16 rr + 4 j + i, i.e. channel 32 g + k
        const int Qi = __float2int_rn(q_nrm_s[col_head * kD + 32 * g + 16 * rr + 4 * j + i] * bs);
        const int hi = (Qi + 64) >> 7, lo = Qi - (hi << 7);         // Qi = 128 hi + lo, -64 <= lo < 64, |hi| <= 127
        v |= (uint32_t)((col_part ? lo : hi) & 0xff) << (8 * i);
      }
      if (SPLIT && g != col_group) v = 0u;
      bq_s[(g * 2 + rr) * 32 + lane] = v;
      // raw q'' for fp16 key rows: k rows follow the 16-byte-piece order of a row load (piece tid4 + 4*i holds
      // the column pairs of k-steps 2i and 2i+1); fp16 hi / lo pairs, one head per column pair (pair 0 only in SPLIT)
      const int s = warp;
#pragma unroll
      for (int r2 = 0; r2 < 2; ++r2) {
        const int c0 = 8 * (j + 4 * (s >> 1)) + 4 * (s & 1) + 2 * r2;
        const int h = gid >> 1;
        const float bsr = pow2i(14 - qe_s[4 + h]);
        const uint32_t v0 = split_hi_lo(q_raw_s[h * kD + c0] * bsr), v1 = split_hi_lo(q_raw_s[h * kD + c0 + 1] * bsr);
        bqr_s[(s * 2 + r2) * 32 + lane] = col_part ? ((v0 >> 16) | (v1 & 0xFFFF0000u)) : ((v0 & 0xFFFFu) | (v1 << 16));
      }
    }
    __syncthreads();
    uint32_t Bq[4][2];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      Bq[g][0] = bq_s[(g * 2) * 32 + lane];
      Bq[g][1] = bq_s[(g * 2 + 1) * 32 + lane];
    }
    // ---- as owner of C-fragment columns 2j, 2j+1: head j, or in SPLIT (head 0, key group j)
    const int my_head = SPLIT ? 0 : j;
    // first absolute token position this lane's query row must not see (all tokens for the newest query)
    const int pos_end = cn.n_sink + cn.n_qk + cn.n_k_recent - (a.n_q - 1 - (a.head0 + my_head) / L.r);
    const float kfac = pow2i(qe_s[my_head]) * (1.0f / kQDigits);      // raw integer score sums -> log2-domain scores
    float Qg[SPLIT ? 1 : NG];
    if constexpr (SPLIT) {
      Qg[0] = qg_s[j];                                // NG == 4: every lane of the quad owns one group
    } else {
#pragma unroll
      for (int g = 0; g < NG; ++g) Qg[g] = qg_s[j * 4 + g];
    }
    // SPLIT: group j sits at bit position j of a byte (weight 4^j), with 4-bit codes in nibble j % 2 (weight
    // 16^(j % 2)), with 3-bit codes in the field of position j (weight 1, 2, 16, 32)
    const float wj = KB == 2 ? pow2i(-2 * j) : KB == 4 ? pow2i(-4 * (j & 1)) : pow2i(-(4 * (j >> 1) + (j & 1)));
    const float wjm = -wj * kMagicSf;
    const float neg_half = -(float)(1 << (KB - 1)), neg_half_v = -(float)(1 << (VB - 1));               // -2^(b-1)
    // 128 * hi + lo of one accumulator pair (bit patterns of kMagicSf + sum), times the power of two w (wm = -w *
    // kMagicSf).  The inner product, 128 w H - w kMagicSf, is a multiple of 128 w below 2^24 of them: exact; the outer one
    // rounds w (128 H + L) once.
    auto digits = [&](int hi, int lo, float w, float wm) {
      return fmaf(w, __int_as_float(lo), fmaf(128.f * w, __int_as_float(hi), 129.f * wm));
    };
    // Raw scores (integer units: multiply by kfac) of the 16 packed key rows r0 .. r0+15 of a chunk: this lane's rows
    // are r0 + gid and r0 + gid + 8.  kc / km: packed rows and metadata rows of the chunk (shared or global memory).
    // decoded: std::true_type when km points to decoder parameters that the warp has already worked out for the whole
    // chunk ((scale, zero-point) float pairs, see kShareKMeta below), std::false_type for the stored metadata words.
    auto k_mtile = [&](auto decoded, const uint32_t* kc, const uint32_t* km, int r0, float& sA_out, float& sB_out) {
      const int rA = r0 + gid, rB = rA + 8;
      auto kmeta = [&](int row, int g, float& s_, float& z_) {      // decoder parameters of (row, group)
        if constexpr (decltype(decoded)::value) {
          const float2 v = reinterpret_cast<const float2*>(km)[row * NG + g];
          s_ = v.x; z_ = v.y;
        } else if constexpr (KM == 4) decode_fast(km[row * NG + g], neg_half, s_, z_);
        else {
          s_ = h2f_bits(reinterpret_cast<const uint16_t*>(km)[row * NG + g] & 0x7FFFu);
          z_ = neg_half * s_;
        }
      };
      float sA, sB, s_, z_;
      if constexpr (KB == 3) {
        // 3-bit codes: one bit-select of a 2-bit plane word and the 1-bit plane word (as it is for the row's first
        // half, shifted by one for the second) per parity of the bit position gives the 3-bit fields of two positions
        const uint2 la = *reinterpret_cast<const uint2*>(kc + rA * RW + 2 * j);
        const uint2 lb = *reinterpret_cast<const uint2*>(kc + rB * RW + 2 * j);
        const uint32_t ha = kc[rA * RW + 8 + j], hb = kc[rB * RW + 8 + j];
        const uint32_t lo[4] = {la.x, lb.x, la.y, lb.y};                        // operand registers a0 .. a3
        const uint32_t ze[4] = {ha, hb, ha >> 1, hb >> 1}, zo[4] = {ha, hb, ha << 1, hb << 1};
        uint32_t we[4], wo[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          we[r] = (lo[r] & 0x33333333u) | (ze[r] & 0xCCCCCCCCu);                // positions 0, 2: bits 0-2, 4-6
          wo[r] = (lo[r] & 0xCCCCCCCCu) | (zo[r] & 0x33333333u);                // positions 1, 3: bits 1-3, 5-7
        }
        auto areg = [&](int p, int r) {
          return (p & 1) ? (wo[r] & (0x0E0E0E0Eu << (4 * (p >> 1)))) : (we[r] & (0x07070707u << (4 * (p >> 1))));
        };
        if constexpr (SPLIT) {
          int c4[4];
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            if (g == 0) imma_us_init(c4, areg(g, 0), areg(g, 1), areg(g, 2), areg(g, 3), Bq[g][0], Bq[g][1], kMagicS);
            else imma_us(c4, areg(g, 0), areg(g, 1), areg(g, 2), areg(g, 3), Bq[g][0], Bq[g][1]);
          }
          kmeta(rA, j, s_, z_);
          sA = fmaf(s_, digits(c4[0], c4[1], wj, wjm), z_ * Qg[0]);
          kmeta(rB, j, s_, z_);
          sB = fmaf(s_, digits(c4[2], c4[3], wj, wjm), z_ * Qg[0]);
          sA += __shfl_xor_sync(0xffffffffu, sA, 1);
          sB += __shfl_xor_sync(0xffffffffu, sB, 1);
          sA += __shfl_xor_sync(0xffffffffu, sA, 2);
          sB += __shfl_xor_sync(0xffffffffu, sB, 2);
        } else {
          // the four positions carry different weights: one accumulator each, joined per group in fp32
          float tA[NG], tB[NG];
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            int c4[4];
            imma_us_init(c4, areg(p, 0), areg(p, 1), areg(p, 2), areg(p, 3), Bq[p][0], Bq[p][1], kMagicS);
            const float w = pow2i(-(4 * (p >> 1) + (p & 1))), wm = -w * kMagicSf;
            const float dA = digits(c4[0], c4[1], w, wm), dB = digits(c4[2], c4[3], w, wm);
            constexpr int PG = G / 32;                      // bit positions per group
            if (p % PG == 0) { tA[p / PG] = dA; tB[p / PG] = dB; }
            else { tA[p / PG] += dA; tB[p / PG] += dB; }
          }
          sA = 0.f; sB = 0.f;
#pragma unroll
          for (int g = 0; g < NG; ++g) {
            kmeta(rA, g, s_, z_);
            sA = fmaf(s_, tA[g], fmaf(z_, Qg[g], sA));
            kmeta(rB, g, s_, z_);
            sB = fmaf(s_, tB[g], fmaf(z_, Qg[g], sB));
          }
        }
      } else if constexpr (KB == 2) {
      const uint2 xa = *reinterpret_cast<const uint2*>(kc + rA * RW + 2 * j);      // bytes 4j.. and 16+4j.. of row rA
      const uint2 xb = *reinterpret_cast<const uint2*>(kc + rB * RW + 2 * j);
      if constexpr (SPLIT) {
        // column pair g carries q'' of group g only, so one accumulator chain leaves group j's sums with lane j
        int c4[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const uint32_t mk = 0x03030303u << (2 * g);
          if (g == 0) imma_us_init(c4, xa.x & mk, xb.x & mk, xa.y & mk, xb.y & mk, Bq[g][0], Bq[g][1], kMagicS);
          else imma_us(c4, xa.x & mk, xb.x & mk, xa.y & mk, xb.y & mk, Bq[g][0], Bq[g][1]);
        }
        kmeta(rA, j, s_, z_);
        sA = fmaf(s_, digits(c4[0], c4[1], wj, wjm), z_ * Qg[0]);
        kmeta(rB, j, s_, z_);
        sB = fmaf(s_, digits(c4[2], c4[3], wj, wjm), z_ * Qg[0]);
        sA += __shfl_xor_sync(0xffffffffu, sA, 1);
        sB += __shfl_xor_sync(0xffffffffu, sB, 1);
        sA += __shfl_xor_sync(0xffffffffu, sA, 2);
        sB += __shfl_xor_sync(0xffffffffu, sB, 2);
      } else if constexpr (G == 32) {
        sA = 0.f; sB = 0.f;
#pragma unroll
        for (int g = 0; g < 4; ++g) {                 // bit position g = group g: its own accumulator
          int c4[4];
          const uint32_t mk = 0x03030303u << (2 * g);
          imma_us_init(c4, xa.x & mk, xb.x & mk, xa.y & mk, xb.y & mk, Bq[g][0], Bq[g][1], kMagicS);
          const float w = pow2i(-2 * g), wm = -w * kMagicSf;
          kmeta(rA, g, s_, z_);
          sA = fmaf(s_, digits(c4[0], c4[1], w, wm), fmaf(z_, Qg[g], sA));
          kmeta(rB, g, s_, z_);
          sB = fmaf(s_, digits(c4[2], c4[3], w, wm), fmaf(z_, Qg[g], sB));
        }
      } else {
        // G = 64 / 128: bit positions 2c and 2c+1 share an accumulator (the odd one shifted down by two bits, so both
        // carry the weight 16^c)
        const uint32_t ya0 = xa.x >> 2, ya1 = xa.y >> 2, yb0 = xb.x >> 2, yb1 = xb.y >> 2;
        float tA[2], tB[2];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          int c4[4];
          const uint32_t mk = 0x03030303u << (4 * c);
          imma_us_init(c4, xa.x & mk, xb.x & mk, xa.y & mk, xb.y & mk, Bq[2 * c][0], Bq[2 * c][1], kMagicS);
          imma_us(c4, ya0 & mk, yb0 & mk, ya1 & mk, yb1 & mk, Bq[2 * c + 1][0], Bq[2 * c + 1][1]);
          const float w = pow2i(-4 * c), wm = -w * kMagicSf;
          tA[c] = digits(c4[0], c4[1], w, wm);
          tB[c] = digits(c4[2], c4[3], w, wm);
        }
        if constexpr (G == 64) {
          kmeta(rA, 0, s_, z_);
          sA = fmaf(s_, tA[0], z_ * Qg[0]);
          kmeta(rB, 0, s_, z_);
          sB = fmaf(s_, tB[0], z_ * Qg[0]);
          kmeta(rA, 1, s_, z_);
          sA = fmaf(s_, tA[1], fmaf(z_, Qg[1], sA));
          kmeta(rB, 1, s_, z_);
          sB = fmaf(s_, tB[1], fmaf(z_, Qg[1], sB));
        } else {
          kmeta(rA, 0, s_, z_);
          sA = fmaf(s_, tA[0] + tA[1], z_ * Qg[0]);
          kmeta(rB, 0, s_, z_);
          sB = fmaf(s_, tB[0] + tB[1], z_ * Qg[0]);
        }
      }
      } else {
        // 4-bit codes: words [2 h2 + h] = bytes 16 h + 4 j .. of row half h2; channel run s = low (s even) or high
        // (s odd) nibbles of half s / 2
        const uint4 xa4 = *reinterpret_cast<const uint4*>(kc + rA * RW + 4 * j);
        const uint4 xb4 = *reinterpret_cast<const uint4*>(kc + rB * RW + 4 * j);
        const uint32_t xa[4] = {xa4.x, xa4.y, xa4.z, xa4.w}, xb[4] = {xb4.x, xb4.y, xb4.z, xb4.w};
        if constexpr (SPLIT || G == 32) {
          int cs[SPLIT ? 1 : 4][4];
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            int (&c4)[4] = cs[SPLIT ? 0 : g];
            const uint32_t mk = (g & 1) ? 0xF0F0F0F0u : 0x0F0F0F0Fu;
            const int h2 = g >> 1;
            if (!SPLIT || g == 0)
              imma_us_init(c4, xa[2 * h2] & mk, xb[2 * h2] & mk, xa[2 * h2 + 1] & mk, xb[2 * h2 + 1] & mk, Bq[g][0], Bq[g][1], kMagicS);
            else
              imma_us(c4, xa[2 * h2] & mk, xb[2 * h2] & mk, xa[2 * h2 + 1] & mk, xb[2 * h2 + 1] & mk, Bq[g][0], Bq[g][1]);
          }
          if constexpr (SPLIT) {
            kmeta(rA, j, s_, z_);
            sA = fmaf(s_, digits(cs[0][0], cs[0][1], wj, wjm), z_ * Qg[0]);
            kmeta(rB, j, s_, z_);
            sB = fmaf(s_, digits(cs[0][2], cs[0][3], wj, wjm), z_ * Qg[0]);
            sA += __shfl_xor_sync(0xffffffffu, sA, 1);
            sB += __shfl_xor_sync(0xffffffffu, sB, 1);
            sA += __shfl_xor_sync(0xffffffffu, sA, 2);
            sB += __shfl_xor_sync(0xffffffffu, sB, 2);
          } else {
            sA = 0.f; sB = 0.f;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const float w = pow2i(-4 * (g & 1)), wm = -w * kMagicSf;
              kmeta(rA, g, s_, z_);
              sA = fmaf(s_, digits(cs[SPLIT ? 0 : g][0], cs[SPLIT ? 0 : g][1], w, wm), fmaf(z_, Qg[SPLIT ? 0 : g], sA));
              kmeta(rB, g, s_, z_);
              sB = fmaf(s_, digits(cs[SPLIT ? 0 : g][2], cs[SPLIT ? 0 : g][3], w, wm), fmaf(z_, Qg[SPLIT ? 0 : g], sB));
            }
          }
        } else {
          // G = 64 / 128: the high nibbles are shifted down, so that the two channel runs of a row half (G = 64: one
          // group) or all four (G = 128) share an accumulator at weight 1
          float tA[2], tB[2];
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            int c4[4];
            const uint32_t mk = 0x0F0F0F0Fu;
            imma_us_init(c4, xa[2 * h2] & mk, xb[2 * h2] & mk, xa[2 * h2 + 1] & mk, xb[2 * h2 + 1] & mk, Bq[2 * h2][0], Bq[2 * h2][1], kMagicS);
            imma_us(c4, (xa[2 * h2] >> 4) & mk, (xb[2 * h2] >> 4) & mk, (xa[2 * h2 + 1] >> 4) & mk, (xb[2 * h2 + 1] >> 4) & mk,
                    Bq[2 * h2 + 1][0], Bq[2 * h2 + 1][1]);
            tA[h2] = digits(c4[0], c4[1], 1.0f, -kMagicSf);
            tB[h2] = digits(c4[2], c4[3], 1.0f, -kMagicSf);
          }
          if constexpr (G == 64) {
            kmeta(rA, 0, s_, z_);
            sA = fmaf(s_, tA[0], z_ * Qg[0]);
            kmeta(rB, 0, s_, z_);
            sB = fmaf(s_, tB[0], z_ * Qg[0]);
            kmeta(rA, 1, s_, z_);
            sA = fmaf(s_, tA[1], fmaf(z_, Qg[1], sA));
            kmeta(rB, 1, s_, z_);
            sB = fmaf(s_, tB[1], fmaf(z_, Qg[1], sB));
          } else {
            kmeta(rA, 0, s_, z_);
            sA = fmaf(s_, tA[0] + tA[1], z_ * Qg[0]);
            kmeta(rB, 0, s_, z_);
            sB = fmaf(s_, tB[0] + tB[1], z_ * Qg[0]);
          }
        }
      }
      sA_out = sA;
      sB_out = sB;
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
    int accg[8][4];          // value code sums of the current group: bit patterns of kMagicUf + sum (see the file header)
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      out_acc[m][0] = out_acc[m][1] = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) accg[m][e] = kMagicU;
    }
    bool failed = false;

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
      if (skew) {
        const int iq = cn.n_qv + e0;                           // first packed key row of the tile (16-aligned)
        const unsigned char* rec = group_rec((iq / kChunk) / CH) + (size_t)((iq / kChunk) % CH) * SL::kRec;
        k_mtile(std::false_type{}, reinterpret_cast<const uint32_t*>(rec), reinterpret_cast<const uint32_t*>(rec + SL::kOffKMeta),
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
      // The reference of the running sums is an integer (log2 domain) that no score so far exceeds: see the main loop.
      const float m_new = fmaxf(m_run, ceilf(cmax));
      // 0 while m_run = -inf; a tile that is masked completely for this row leaves the state as it is
      const float alpha = m_new == -INFINITY ? 1.f : ex2_approx(m_run - m_new);
      m_run = m_new;
      l_part *= alpha;
#pragma unroll
      for (int m = 0; m < 8; ++m) { out_acc[m][0] *= alpha; out_acc[m][1] *= alpha; }
      const float pA = sA == -INFINITY ? 0.f : ex2_approx(sA - m_new), pB = sB == -INFINITY ? 0.f : ex2_approx(sB - m_new);
      l_part += pA + pB;
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
          // out_acc is kept in units of 1 / kPScale (the integer image of p); these sums carry p * 2^10
          out_acc[4 * hh + kk][0] = fmaf(c4[0] + c4[1], kPScale * 0x1p-10f, out_acc[4 * hh + kk][0]);
          out_acc[4 * hh + kk][1] = fmaf(c4[2] + c4[3], kPScale * 0x1p-10f, out_acc[4 * hh + kk][1]);
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

    constexpr bool kFreshEveryChunk = !SPLIT && CH == 1;      // a value group is one chunk: nothing is carried over
    constexpr bool kStaticSlots = !SPLIT && CH == CPI && CH > 1;   // a value group is one iteration (G = 64, two chunks)
    // see the raw scores below; measured: 2.4 % faster in a chain where an iteration holds two chunks of four groups per
    // row (one exchange for 256 entries), 0-2 % SLOWER with one chunk per iteration (3- and 4-bit keys) or two groups
    constexpr bool kShareKMeta = !SPLIT && NG == 4 && CPI == 2;
    static_assert(!kShareKMeta || CPI * kChunk * NG * 8 <= SL::kSideBytes, "decoded key metadata of an iteration fit the side area");
    // 256 * hi + lo of a value accumulator pair (bit patterns of kMagicUf + sum), times the power of two w: the inner
    // product, 256 w H - w kMagicUf, is exact (a multiple of 256 w), the outer one rounds w (256 H + L) once
    auto vdigits = [&](int hi, int lo, float w) {
      return fmaf(w, __int_as_float(lo), fmaf(256.f * w, __int_as_float(hi), -257.f * w * kMagicUf));
    };
    // lanes this lane fetches its value-side B registers from: the lane that holds the probabilities of tokens
    // k = 4j .. 4j+3 (register 0) and 16 + 4j .. (register 1) for this column's head
    const int src0 = 4 * j + (SPLIT ? 0 : (gid >> 1)), src1 = src0 + 16;

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
      // With several key groups per token and several heads per pass, the four lanes of a quad need the decoder
      // parameters of the same (row, group) entries: lane = row decodes its row's NG entries once, the warp exchanges
      // them through its side area (free between the value groups' ends), each lane reads its two rows per m-tile.
      if constexpr (kShareKMeta && !(ABL & 1)) {
#pragma unroll
        for (int cc = 0; cc < CPI; ++cc) {
          if (cc > 0 && !last_valid) continue;
          const unsigned char* kmb = sp + SL::off(cc) + SL::kOffKMeta + lane * (NG * KM);
          float* dst = reinterpret_cast<float*>(side) + cc * (kChunk * NG * 2) + lane * (NG * 2);
          float sz[2 * NG];
          if constexpr (KM == 4) {
            uint32_t mw[NG];
            if constexpr (NG == 4) {
              const uint4 t = *reinterpret_cast<const uint4*>(kmb);
              mw[0] = t.x; mw[1] = t.y; mw[2] = t.z; mw[3] = t.w;
            } else {
              const uint2 t = *reinterpret_cast<const uint2*>(kmb);
              mw[0] = t.x; mw[1] = t.y;
            }
#pragma unroll
            for (int g = 0; g < NG; ++g) decode_fast(mw[g], neg_half, sz[2 * g], sz[2 * g + 1]);
          } else {
            uint32_t hw[NG / 2];
            if constexpr (NG == 4) {
              const uint2 t = *reinterpret_cast<const uint2*>(kmb);
              hw[0] = t.x; hw[1] = t.y;
            } else {
              hw[0] = *reinterpret_cast<const uint32_t*>(kmb);
            }
#pragma unroll
            for (int g = 0; g < NG; ++g) {
              sz[2 * g] = h2f_bits((hw[g >> 1] >> (16 * (g & 1))) & 0x7FFFu);
              sz[2 * g + 1] = neg_half * sz[2 * g];
            }
          }
#pragma unroll
          for (int g = 0; g < NG; g += 2)
            *reinterpret_cast<float4*>(dst + 2 * g) = make_float4(sz[2 * g], sz[2 * g + 1], sz[2 * g + 2], sz[2 * g + 3]);
        }
        __syncwarp();
      }
      float sc[CPI][2][2];
#pragma unroll
      for (int cc = 0; cc < CPI; ++cc) {
        if (cc > 0 && !last_valid) {      // nothing there: this warp's range ends in the middle of the iteration
          sc[cc][0][0] = sc[cc][0][1] = sc[cc][1][0] = sc[cc][1][1] = -INFINITY;
          continue;
        }
        const uint32_t* kc = reinterpret_cast<const uint32_t*>(sp + SL::off(cc));
        const uint32_t* km = reinterpret_cast<const uint32_t*>(sp + SL::off(cc) + SL::kOffKMeta);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          if constexpr (ABL & 1) sc[cc][mt][0] = sc[cc][mt][1] = 0.f;      // timing experiment: no key side
          else if constexpr (kShareKMeta)
            k_mtile(std::true_type{}, kc, side + cc * (kChunk * NG * 2), 16 * mt, sc[cc][mt][0], sc[cc][mt][1]);
          else k_mtile(std::false_type{}, kc, km, 16 * mt, sc[cc][mt][0], sc[cc][mt][1]);
        }
      }
      if constexpr (kShareKMeta && !(ABL & 1)) __syncwarp();      // the side area goes back to the value groups' ends

      // ---------------- online softmax (log2 domain; raw scores are in integer units: times kfac) -----
      // The reference m_run of the running sums is an INTEGER that no score so far exceeds (the ceiling of the
      // largest one when it last moved): p = 2^(s - m_run) <= 1 fills the 16 bits of its integer image, and a move of
      // the reference rescales the integer accumulators of the open value group by an exact shift.
      float cmax = -INFINITY;
#pragma unroll
      for (int cc = 0; cc < CPI; ++cc)
        cmax = fmaxf(cmax, fmaxf(fmaxf(sc[cc][0][0], sc[cc][0][1]), fmaxf(sc[cc][1][0], sc[cc][1][1])));
      float m_new = m_run;
      if (__any_sync(0xffffffffu, cmax * kfac > m_run)) {
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 4));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
        cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));
        m_new = fmaxf(m_run, ceilf(cmax * kfac));
        const float alpha = ex2_approx(m_run - m_new);     // 2^-k exactly; 0 on the first iteration (m_run = -inf)
        l_part *= alpha;
        psum *= alpha;
#pragma unroll
        for (int m = 0; m < 8; ++m) { out_acc[m][0] *= alpha; out_acc[m][1] *= alpha; }
        if constexpr (!kFreshEveryChunk && !kStaticSlots) {      // (else no value group is open between iterations)
          // sums of the open value group: (256 hi + lo) >> k, the bits that leave hi carried into lo (they weigh 256)
          const int k = m_run == -INFINITY ? 23 : min(23, (int)(m_new - m_run));
          const int keep = k < 23 ? -1 : 0, low = (1 << k) - 1;
#pragma unroll
          for (int m = 0; m < 8; ++m)
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
              const int hi = (accg[m][2 * rh] - kMagicU) & keep, lo = (accg[m][2 * rh + 1] - kMagicU) & keep;
              accg[m][2 * rh] = kMagicU + (hi >> k);
              accg[m][2 * rh + 1] = kMagicU + ((lo + ((hi & low) << 8)) >> k);
            }
        }
      }
      m_run = m_new;

#pragma unroll
      for (int cc = 0; cc < CPI; ++cc) {
        if (cc > 0 && !last_valid) continue;
        const int ci = ci0 + cc;
        const uint32_t* vc = reinterpret_cast<const uint32_t*>(sp + SL::off(cc) + SL::kOffVCodes);
        const uint32_t* vm = reinterpret_cast<const uint32_t*>(sp + SL::off(cc) + SL::kRec);
        // slot: position of this chunk's value group in the SPLIT window / position of the chunk in its group
        // (kStaticSlots: an iteration is exactly one value group, so the position is the chunk's index in the iteration)
        const int slot = SPLIT ? (ci - c_lo) & (WIN - 1) : (kStaticSlots ? cc : ci % CH);
        const bool group_start = slot == 0;
        // the first MMA of a sum takes the constant as its accumulator input instead of registers set up for it
        const bool init_here = kFreshEveryChunk || (kStaticSlots && cc == 0);
        const bool group_end = SPLIT ? (slot == WIN - 1 || (it == n_iters - 1 && (cc == CPI - 1 || !last_valid)))
                                     : (slot == CH - 1);
        if (!kFreshEveryChunk && !kStaticSlots && group_start) {
#pragma unroll
          for (int m = 0; m < 8; ++m)
#pragma unroll
            for (int e = 0; e < 4; ++e) accg[m][e] = kMagicU;
        }
        // ---------------- probabilities as 16-bit integers, two base-256 digits -------------------------
        // This lane's four tokens of the chunk are rows gid + 8 i (i = 2 mt + h), which the value chunk stores at
        // k = 4 gid + i: its digit words are exactly one B register of the lanes that need them.
        uint32_t Pb[4];
        float psum_c = 0.f;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const float p = ex2_approx(fmaf(sc[cc][mt][h], kfac, -m_new));
            psum_c += p;
            Pb[2 * mt + h] = __float_as_uint(fmaf(p, kPScale, kMagicUf));      // low 16 bits: rint(p * 65535)
          }
        l_part += psum_c;
        if constexpr (SPLIT) psum += (j == slot) ? psum_c : 0.f;
        else psum += psum_c;
        const uint32_t x01 = prmt(Pb[0], Pb[1], 0x5140u), x23 = prmt(Pb[2], Pb[3], 0x5140u);   // (lo0, lo1, hi0, hi1)
        const uint32_t Plo = prmt(x01, x23, 0x5410u), Phi = prmt(x01, x23, 0x7632u);
        const uint32_t h0 = __shfl_sync(0xffffffffu, Phi, src0), l0 = __shfl_sync(0xffffffffu, Plo, src0);
        const uint32_t h1 = __shfl_sync(0xffffffffu, Phi, src1), l1 = __shfl_sync(0xffffffffu, Plo, src1);
        uint32_t b0 = (gid & 1) ? l0 : h0, b1 = (gid & 1) ? l1 : h1;
        if (SPLIT && (gid >> 1) != slot) { b0 = 0u; b1 = 0u; }      // column pair of this chunk's window slot only

        // ---------------- values: 8 m-tiles of 16 channels x one k-step of 32 tokens --------------------
        if constexpr (!(ABL & 2) && VB == 3) {
          // 3-bit codes: word sets W = 0, 1 of the 2-bit plane (as with 2-bit codes) and one set of the 1-bit plane,
          // as it is for W = 0 and shifted by one for W = 1
          const uint4 l0 = *reinterpret_cast<const uint4*>(vc + lane * 4);
          const uint4 l1 = *reinterpret_cast<const uint4*>(vc + 128 + lane * 4);
          const uint4 h4 = *reinterpret_cast<const uint4*>(vc + 256 + lane * 4);
          const uint32_t lw[2][4] = {{l0.x, l0.y, l0.z, l0.w}, {l1.x, l1.y, l1.z, l1.w}};
          const uint32_t hw[4] = {h4.x, h4.y, h4.z, h4.w};
#pragma unroll
          for (int W = 0; W < 2; ++W) {
            uint32_t we[4], wo[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              const uint32_t ze = W ? hw[r] >> 1 : hw[r], zo = W ? hw[r] << 1 : hw[r];
              we[r] = (lw[W][r] & 0x33333333u) | (ze & 0xCCCCCCCCu);
              wo[r] = (lw[W][r] & 0xCCCCCCCCu) | (zo & 0x33333333u);
            }
#pragma unroll
            for (int pos = 0; pos < 4; ++pos) {
              const uint32_t mk = (pos & 1) ? (0x0E0E0E0Eu << (4 * (pos >> 1))) : (0x07070707u << (4 * (pos >> 1)));
              const uint32_t* src = (pos & 1) ? wo : we;
              if (init_here)
                imma_uu_init(accg[4 * W + pos], src[0] & mk, src[1] & mk, src[2] & mk, src[3] & mk, b0, b1, kMagicU);
              else
                imma_uu(accg[4 * W + pos], src[0] & mk, src[1] & mk, src[2] & mk, src[3] & mk, b0, b1);
            }
          }
        } else if constexpr (!(ABL & 2) && VB == 4) {
          // 4-bit codes: word set W = m / 2 (four words: the roles a0 .. a3), nibble m % 2
#pragma unroll
          for (int W = 0; W < 4; ++W) {
            const uint4 v = *reinterpret_cast<const uint4*>(vc + W * 128 + lane * 4);
#pragma unroll
            for (int pos = 0; pos < 2; ++pos) {
              const uint32_t mk = pos ? 0xF0F0F0F0u : 0x0F0F0F0Fu;
              if (init_here)
                imma_uu_init(accg[2 * W + pos], v.x & mk, v.y & mk, v.z & mk, v.w & mk, b0, b1, kMagicU);
              else
                imma_uu(accg[2 * W + pos], v.x & mk, v.y & mk, v.z & mk, v.w & mk, b0, b1);
            }
          }
        } else if constexpr (!(ABL & 2)) {
          const uint4 v0 = *reinterpret_cast<const uint4*>(vc + lane * 4);
          const uint4 v1 = *reinterpret_cast<const uint4*>(vc + 128 + lane * 4);
          const uint32_t vw[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
          for (int W = 0; W < 2; ++W)
#pragma unroll
            for (int pos = 0; pos < 4; ++pos) {
              const uint32_t mk = 0x03030303u << (2 * pos);
              if (init_here)
                imma_uu_init(accg[4 * W + pos], vw[4 * W] & mk, vw[4 * W + 1] & mk, vw[4 * W + 2] & mk, vw[4 * W + 3] & mk,
                             b0, b1, kMagicU);
              else
                imma_uu(accg[4 * W + pos], vw[4 * W] & mk, vw[4 * W + 1] & mk, vw[4 * W + 2] & mk, vw[4 * W + 3] & mk, b0, b1);
            }
        }

        // ---------------- end of a value group: apply scale / zero-point once per channel -----------
        const bool chunk_valid = cc == 0 || last_valid;
        if constexpr (SPLIT) {
          // keep this group's metadata for the end of the window (the stage will be refilled)
          if (chunk_valid && lane * 16 < SL::kVMeta)
            *reinterpret_cast<uint4*>(side + slot * (SL::kVMeta / 4) + lane * 4) = *reinterpret_cast<const uint4*>(vm + lane * 4);
        }
        if (group_end && chunk_valid) {
          if constexpr (SPLIT) __syncwarp();
          float pg = psum;
          pg += __shfl_xor_sync(0xffffffffu, pg, 4);
          pg += __shfl_xor_sync(0xffffffffu, pg, 8);
          pg += __shfl_xor_sync(0xffffffffu, pg, 16);
          pg *= kPScale;                                // out_acc is in units of 1 / kPScale
          const uint32_t* vmg = SPLIT ? side + j * (SL::kVMeta / 4) : vm;    // this group's entries (slot j's in SPLIT)
          // code sum of fragment row (m, rh): m-tile m sits at bit position m % 4 of its words (weight 4^(m % 4);
          // 3-bit fields: 1, 2, 16, 32), with 4-bit codes in nibble m % 2
          auto acc_sum = [&](int m, int rh) {
            return vdigits(accg[m][2 * rh], accg[m][2 * rh + 1],
                           VB == 2 ? pow2i(-2 * (m & 3)) : VB == 4 ? pow2i(-4 * (m & 1)) : pow2i(-(2 * (m & 2) + (m & 1))));
          };
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
    __syncthreads();                                   // every warp is done with its ring
    float* wres = reinterpret_cast<float*>(smem);      // [warp][head][kD + 2]
    const bool writer = SPLIT ? (j == 0) : true;
    const bool any = n_iters > 0 || tw > 0;
    if (writer) {
      float* mine = wres + ((size_t)warp * kHeads + (SPLIT ? 0 : j)) * (kD + 2);
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        mine[block_row_channel(m, 0, gid)] = any ? out_acc[m][0] * (1.0f / kPScale) : 0.f;
        mine[block_row_channel(m, 1, gid)] = any ? out_acc[m][1] * (1.0f / kPScale) : 0.f;
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
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool PAGED = false, int ABL = 0>
__global__ void __launch_bounds__(kThreads, 2)
decode_i8_kernel(const Layout L, const Counts cn, const DecodeArgs a) {
  decode_i8_body<KB, VB, G, KM, VM, SPLIT, CPI, PAGED, ABL>(L, cn, a, blockIdx.x);
}
// One paged cache with its page table in the parameter space (read in place: no look-up in device memory).
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI>
__global__ void __launch_bounds__(kThreads, 2)
decode_i8_paged_kernel(const Layout L, const Counts cn, const DecodeArgs a, const __grid_constant__ PageIds P) {
  decode_i8_body<KB, VB, G, KM, VM, SPLIT, CPI, true>(L, cn, a, blockIdx.x, &P);
}
// Several caches of one configuration: block x = sequence * U + unit.
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool PAGED = false>
__global__ void __launch_bounds__(kThreads, 2)
decode_i8_batched_kernel(const __grid_constant__ Layout L, const __grid_constant__ SeqTable T) {
  const int seq = blockIdx.x / L.U;
  decode_i8_body<KB, VB, G, KM, VM, SPLIT, CPI, PAGED>(L, T.s[seq].cn, T.s[seq].a, blockIdx.x - seq * L.U);
}

// ---- host side: the launchers of one metadata format (KM, VM) at every group size ---------------------------
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool PAGED>
int launch_i8_one_p(const Layout& L, const Counts& cn, DecodeArgs a, int n_splits, cudaStream_t st) {
  using SL = StageLayout<KB, VB, G, KM, VM, CPI>;
  constexpr int kSmem = SL::kCtaBytes;
  constexpr int RU = SL::kCH;
  static std::atomic<unsigned long long> configured{0};
  if (!opt_in_dynamic_smem(decode_i8_kernel<KB, VB, G, KM, VM, SPLIT, CPI, PAGED>, kSmem, configured)) return -1;
  // a paged cache whose page list fits the parameter space: the kernel that takes the table as a parameter
  [[maybe_unused]] PageIds ids;
  bool table_in_params = false;
  if constexpr (PAGED) {
    static std::atomic<unsigned long long> configured_p{0};
    if (a.pages_host && a.n_pages_host <= kParamPages) {
      if (!opt_in_dynamic_smem(decode_i8_paged_kernel<KB, VB, G, KM, VM, SPLIT, CPI>, kSmem, configured_p)) return -1;
      for (int i = 0; i < a.n_pages_host; ++i) ids.id[i] = a.pages_host[i];
      table_in_params = true;
    }
  }
  const int grid_y = fill_split_args<RU>(L, cn, a, false, n_splits, 0);
  dim3 grid(L.U, grid_y);
  int launches = 0;
  const int step = SPLIT ? 1 : kHeads;
  for (int h0 = 0; h0 < L.r * a.n_q; h0 += step) {
    a.head0 = h0;
    // launched as a programmatic dependent of whatever precedes it in the stream (see the kernel's dep_wait)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t err;
    if constexpr (PAGED) {
      if (a.ablation) return -2;      // the timing instances exist for contiguous caches only
      err = table_in_params ? cudaLaunchKernelEx(&cfg, decode_i8_paged_kernel<KB, VB, G, KM, VM, SPLIT, CPI>, L, cn, a, ids)
                            : cudaLaunchKernelEx(&cfg, decode_i8_kernel<KB, VB, G, KM, VM, SPLIT, CPI, PAGED>, L, cn, a);
    } else if (a.ablation == 1 || a.ablation == 2) {
#ifdef IQ_WITH_TIMING_INSTANCES      // defined by the translation units of the formats the latency study and the bench time
      static std::atomic<unsigned long long> configured_a1{0}, configured_a2{0};
      if (a.ablation == 1) {
        if (!opt_in_dynamic_smem(decode_i8_kernel<KB, VB, G, KM, VM, SPLIT, CPI, false, 1>, kSmem, configured_a1)) return -1;
        err = cudaLaunchKernelEx(&cfg, decode_i8_kernel<KB, VB, G, KM, VM, SPLIT, CPI, false, 1>, L, cn, a);
      } else {
        if (!opt_in_dynamic_smem(decode_i8_kernel<KB, VB, G, KM, VM, SPLIT, CPI, false, 2>, kSmem, configured_a2)) return -1;
        err = cudaLaunchKernelEx(&cfg, decode_i8_kernel<KB, VB, G, KM, VM, SPLIT, CPI, false, 2>, L, cn, a);
      }
#else
      return -2;
#endif
    } else {
      err = cudaLaunchKernelEx(&cfg, decode_i8_kernel<KB, VB, G, KM, VM, SPLIT, CPI, PAGED>, L, cn, a);
    }
    if (err != cudaSuccess) return -1;
    ++launches;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// The same kernel over a table of caches (rows per sequence: see launch_one_batched_p of the fp16-operand kernel).
template <int KB, int VB, int G, int KM, int VM, bool SPLIT, int CPI, bool PAGED>
int launch_i8_batched_p(const Layout& L, SeqTable& T, int n_seqs, int n_splits, cudaStream_t st) {
  using SL = StageLayout<KB, VB, G, KM, VM, CPI>;
  constexpr int kSmem = SL::kCtaBytes;
  constexpr int RU = SL::kCH;
  static std::atomic<unsigned long long> configured{0};
  if (!opt_in_dynamic_smem(decode_i8_batched_kernel<KB, VB, G, KM, VM, SPLIT, CPI, PAGED>, kSmem, configured)) return -1;
  long long chunks[kMaxSeqs], longest = 1;
  for (int i = 0; i < n_seqs; ++i) {
    chunks[i] = T.s[i].cn.n_qv / kChunk;
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
    const int gy = fill_split_args<RU>(L, T.s[i].cn, T.s[i].a, false, want, 0);
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
    if (cudaLaunchKernelEx(&cfg, decode_i8_batched_kernel<KB, VB, G, KM, VM, SPLIT, CPI, PAGED>, L, T) != cudaSuccess) return -1;
    ++launches;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// cpi: chunks of 32 tokens per loop iteration, 0 = automatic: two for 2-bit codes (4-bit stages are twice the size:
// always one), unless a warp gets so few chunks that the second half of an iteration would often be empty (G = 32,
// where a warp's range may be an odd number of chunks, and fewer than four chunks per warp: short contexts split
// over many CTAs).
template <int KB, int VB, int G, int KM, int VM, bool SPLIT>
int launch_i8_cpi(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits, int cpi, cudaStream_t st) {
  const bool paged = L.page_groups > 0;
  if (cpi == 0 && G == 32 && cn.n_qv / kChunk < 4 * kWarps * (n_splits > 0 ? n_splits : 1)) cpi = 1;
  if constexpr (KB == 2 && VB == 2) {
    if (cpi != 1)
      return paged ? launch_i8_one_p<KB, VB, G, KM, VM, SPLIT, 2, true>(L, cn, a, n_splits, st)
                   : launch_i8_one_p<KB, VB, G, KM, VM, SPLIT, 2, false>(L, cn, a, n_splits, st);
  }
  return paged ? launch_i8_one_p<KB, VB, G, KM, VM, SPLIT, 1, true>(L, cn, a, n_splits, st)
               : launch_i8_one_p<KB, VB, G, KM, VM, SPLIT, 1, false>(L, cn, a, n_splits, st);
}
template <int KB, int VB, int G, int KM, int VM, bool SPLIT>
int launch_i8_cpi_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, int cpi, cudaStream_t st) {
  const bool paged = L.page_groups > 0;
  if constexpr (KB == 2 && VB == 2) {
    if (cpi != 1)
      return paged ? launch_i8_batched_p<KB, VB, G, KM, VM, SPLIT, 2, true>(L, T, n_seqs, n_splits, st)
                   : launch_i8_batched_p<KB, VB, G, KM, VM, SPLIT, 2, false>(L, T, n_seqs, n_splits, st);
  }
  return paged ? launch_i8_batched_p<KB, VB, G, KM, VM, SPLIT, 1, true>(L, T, n_seqs, n_splits, st)
               : launch_i8_batched_p<KB, VB, G, KM, VM, SPLIT, 1, false>(L, T, n_seqs, n_splits, st);
}

template <int KB, int VB, int KM, int VM>
int launch_i8_format(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits, int cpi, cudaStream_t st) {
  if (L.G == 32 && L.r == 1 && a.n_q == 1) return launch_i8_cpi<KB, VB, 32, KM, VM, true>(L, cn, a, n_splits, cpi, st);
  if (L.G == 32) return launch_i8_cpi<KB, VB, 32, KM, VM, false>(L, cn, a, n_splits, cpi, st);
  if (L.G == 64) return launch_i8_cpi<KB, VB, 64, KM, VM, false>(L, cn, a, n_splits, cpi, st);
  if (L.G == 128) return launch_i8_cpi<KB, VB, 128, KM, VM, false>(L, cn, a, n_splits, cpi, st);
  return -2;
}
template <int KB, int VB, int KM, int VM>
int launch_i8_format_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, int cpi, cudaStream_t st) {
  if (L.G == 32 && L.r == 1) return launch_i8_cpi_batched<KB, VB, 32, KM, VM, true>(L, T, n_seqs, n_splits, cpi, st);
  if (L.G == 32) return launch_i8_cpi_batched<KB, VB, 32, KM, VM, false>(L, T, n_seqs, n_splits, cpi, st);
  if (L.G == 64) return launch_i8_cpi_batched<KB, VB, 64, KM, VM, false>(L, T, n_seqs, n_splits, cpi, st);
  if (L.G == 128) return launch_i8_cpi_batched<KB, VB, 128, KM, VM, false>(L, T, n_seqs, n_splits, cpi, st);
  return -2;
}

}  // namespace

// Defines the externally visible launchers of one metadata format in the translation unit that compiles its kernels
// (same names as the fp16-operand kernel's: the host dispatch does not change).
#define IQ_DEFINE_I8_FORMAT(KB, VB, KM, VM)                                                                           \
  int IQ_MMA_FORMAT_NAME(KB, VB, KM, VM)(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits,   \
                                             int cpi, cudaStream_t st) {                                              \
    return launch_i8_format<KB, VB, KM, VM>(L, cn, a, n_splits, cpi, st);                                               \
  }                                                                                                                   \
  int IQ_MMA_FORMAT_NAME_BATCHED(KB, VB, KM, VM)(const Layout& L, SeqTable& T, int n_seqs, int n_splits, int cpi, \
                                                     cudaStream_t st) {                                               \
    return launch_i8_format_batched<KB, VB, KM, VM>(L, T, n_seqs, n_splits, cpi, st);                                   \
  }

}  // namespace iq
