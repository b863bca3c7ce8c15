// Decode attention over the packed InnerQ cache with the 5th-generation tensor cores (tcgen05.mma, accumulators
// and the code operand in tensor memory), for the format of the 7B-class MHA workload: 2-bit keys and values,
// group 32, one query head per KV head, scale|zero metadata.
//
// Why a second kernel: in the warp-level kernel (innerq_decode_mma.cuh) every MMA is issued by the warp that also
// unpacks the codes, and on this GPU the legacy mma.sync and the ALU-pipe unpacking do not overlap.  Here a CTA of
// 128 threads works on tiles of 128 tokens (four 32-token chunk records):
//   keys:   thread t expands the packed row of token t to fp16 pairs (one LOP3 per pair: `word & mask` is a pair of
//           subnormals scaled by the field position) and stores them as row t of the A operand in tensor memory;
//           one thread issues D_k[128 tokens x 16] = A_k[128 x 128 channels] * B_q, where the columns of B_q are
//           (channel group, hi | lo part) of q'' with zeros outside the group, so D_k holds the per-group code sums;
//           thread t reads its row of D_k and applies the four scale / zero-point pairs of its token.
//   values: thread c expands the codes of channel c for the tile's 128 tokens as row c of A_v; B_p has one column
//           per chunk (= value group) holding p of that chunk's tokens; D_v[128 channels x 16] are the per-group
//           sums, to which thread c applies the group's scale / zero-point of its channel.
// The MMAs run asynchronously; the expansion of the next operand overlaps them.  A fifth warp starts the bulk copies
// and issues the MMAs; it and the four compute warps hand work to each other through mbarriers only.  Same records,
// same bulk-copy pipeline, same split merge as the warp-level kernel; the fp16 windows and the K/V skew zone are
// handled with plain SIMT code, a slice per CTA, before its first tile.
#include "innerq_device.cuh"
#include "innerq_kernels.h"

namespace iq {

namespace {

constexpr int kT5Threads = 128;
constexpr int kTile = 128;                         // tokens per tile
constexpr int kChunksPerTile = kTile / kChunk;     // 4
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kWaitLimit = 1u << 22;

// one chunk record of this format: [key rows 32 x 32 B][key metadata 32 x 16 B][value chunk 1024 B][value metadata 512 B]
constexpr int kKRow = 32, kKCodes = kChunk * kKRow, kKMetaRow = 16, kKMeta = kChunk * kKMetaRow;
constexpr int kVCodes = 1024, kVMeta = 512;
constexpr int kOffKMeta = kKCodes, kOffVCodes = kKCodes + kKMeta, kOffVMeta = kOffVCodes + kVCodes;
constexpr int kRecBytes = kOffVMeta + kVMeta;      // 3072
constexpr int kTileBytes = kChunksPerTile * kRecBytes;
constexpr int kStages = 3;

// shared memory map
constexpr int kOffBq = kStages * kTileBytes;       // B_q: 16 columns x 128 channels fp16, canonical K-major layout
constexpr int kOffBp = kOffBq + 4096;              // B_p: 16 columns x 128 tokens
constexpr int kOffMisc = kOffBp + 4096;            // barriers, reductions, tensor-memory base address
constexpr int kOffScratch = kOffMisc + 512;        // q'' raw and normalised, result of the fp16 / skew token slice
constexpr int kT5Smem = kOffScratch + 2048;

// tensor memory (32-bit columns, 128 lanes), two allocations so that three CTAs fit into the SM's 512 columns:
// operands A_k 64 + A_v 64, accumulators D_k 16 + D_v 16
constexpr int kColAk = 0, kColAv = 64, kTmemColsA = 128;
constexpr int kColDk = 0, kColDv = 16, kTmemColsD = 32;

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
// bounded wait: false after kWaitLimit polls (the caller flags an error and stops using the data)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kWaitLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float pow2i(int e) { return __int_as_float((e + 127) << 23); }
__device__ __forceinline__ uint32_t split_hi_lo(float x) {
  const __half hi = __float2half_rn(x);
  const __half lo = __float2half_rn(x - __half2float(hi));
  return (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
}

// ---- tensor memory and tcgen05 ---------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {       // one full warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_alloc_done() {                                  // after the CTA's last allocation
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {        // the same warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* d) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
  tc_wait_ld();
#pragma unroll
  for (int i = 0; i < 8; ++i) d[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, float* d) {
  uint32_t r[4];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
  tc_wait_ld();
#pragma unroll
  for (int i = 0; i < 4; ++i) d[i] = __uint_as_float(r[i]);
}
// Shared-memory operand descriptor: K-major, no swizzle.  Core matrix = 8 rows x 16 bytes, stored contiguously;
// `lbo`: bytes between the two 16-byte K-halves of one MMA (K = 16 fp16); `sbo`: bytes between 8-row groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// Instruction descriptor of kind::f16: fp16 x fp16 -> fp32, both operands K-major, M = 128, N = 16.
constexpr uint32_t kIdesc = (1u << 4) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
// D[128 x 16] (+)= A[128 x 16 (tensor memory)] * B[16 x 16 (shared memory)]; issued by ONE thread
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
// arrive on `bar` when every MMA issued so far by this thread has completed
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

struct T5Args {
  const unsigned char* cache;
  unsigned char* ws;
  const __half* q;
  __half* out;
  int n_splits;        // CTAs per unit (= gridDim.y)
  int k_ring_pos0, v_ring_pos0;
};

// Position of channel c inside the expanded key row (the K index of A_k / B_q): the thread expands word wi = 0..7 of
// the packed row into pairs fld = 0..7 (field 2*fld of both half-words), pair index wi * 8 + fld.
__device__ __forceinline__ int key_k_index(int c) {
  const int s = c >> 4, col = c & 15, j = (col & 7) >> 1, hf = col & 1, odd = col >> 3;
  const int wi = 2 * j + (s >> 2), fld = 2 * (s & 3) + odd;
  return 2 * (wi * 8 + fld) + hf;
}
__device__ __forceinline__ int key_field(int c) { return (2 * ((c >> 4) & 3) + ((c & 15) >> 3)) & 3; }   // after the window shift
// Position of token tau (0..31) of chunk ch inside the expanded value row (the K index of A_v / B_p), and its field.
__device__ __forceinline__ int val_field(int tau) { return 2 * (tau >> 4) + ((tau >> 3) & 1); }
__device__ __forceinline__ int val_k_index(int ch, int tau) {
  const int jj = (tau & 7) >> 1, tp = tau & 1;
  return 2 * (ch * 16 + jj * 4 + val_field(tau)) + tp;
}
// byte offset of element (column n, K index k) in the canonical K-major operand (lbo 256, sbo 128)
__device__ __forceinline__ int b_offset(int n, int k) { return (k >> 3) * 256 + (n >> 3) * 128 + (n & 7) * 16 + (k & 7) * 2; }

// Log-sum-exp merge of the partial results of a unit (see innerq_decode_mma.cuh); four warps.
__device__ __noinline__ void merge_parts4(const float* __restrict__ partials, float* wm, __half* __restrict__ out,
                                          int n_parts, int head, int max_splits) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;       // warps 0..3 work, a fifth only joins the barrier
  float M = -INFINITY, den = 0.f, n0 = 0.f, n1 = 0.f, n2 = 0.f, n3 = 0.f;
  const float* Ph = partials + (size_t)head * max_splits * kPartialStride;
#pragma unroll 1
  for (int s0 = warp; s0 < n_parts && warp < 4; s0 += 4 * 4) {
    float4 v[4];
    float2 ml[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int s = s0 + e * 4;
      const float* P = Ph + (size_t)(s < n_parts ? s : s0) * kPartialStride;
      v[e] = __ldcg(reinterpret_cast<const float4*>(P) + lane);
      ml[e] = __ldcg(reinterpret_cast<const float2*>(P + kD));
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
  if (warp < 4) {
    float* mine = wm + warp * (kD + 2);
    *reinterpret_cast<float2*>(mine + 4 * lane) = make_float2(n0, n1);
    *reinterpret_cast<float2*>(mine + 4 * lane + 2) = make_float2(n2, n3);
    if (lane == 0) { mine[kD] = M; mine[kD + 1] = den; }
  }
  __syncthreads();
  if (warp >= 4) return;
  const int c = tid;
  float Mx = -INFINITY;
#pragma unroll
  for (int w = 0; w < 4; ++w) Mx = fmaxf(Mx, wm[w * (kD + 2) + kD]);
  float num = 0.f, dn = 0.f;
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const float* r_ = wm + w * (kD + 2);
    const float wgt = r_[kD] == -INFINITY ? 0.f : ex2_approx(r_[kD] - Mx);
    num = fmaf(r_[c], wgt, num);
    dn = fmaf(r_[kD + 1], wgt, dn);
  }
  out[(size_t)head * kD + c] = __float2half_rn(num / dn);
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// warp-wide maximum of floats / sum of non-negative floats <= 1 with one redux instruction each
__device__ __forceinline__ float warp_max(float v) {
  int b = __float_as_int(v);
  b ^= (b >> 31) & 0x7fffffff;                       // order-preserving map to signed integers (an involution)
  b = __reduce_max_sync(0xffffffffu, b);
  b ^= (b >> 31) & 0x7fffffff;
  return __int_as_float(b);
}
__device__ __forceinline__ float warp_sum_unit(float v) {      // 24 fractional bits
  return (float)__reduce_add_sync(0xffffffffu, (unsigned)__float2uint_rn(v * 0x1p24f)) * 0x1p-24f;
}

// The tokens outside the range where keys and values are both packed (at most a few hundred per unit): the K/V skew
// zone (packed key rows n_qv .., fp16 values from the value ring), the sink window and the recent window (fp16
// both), as one list of entries.  Every CTA of a unit takes a slice [e_lo, e_hi) of the list; ONE warp works it off
// with plain SIMT code while the others stream the packed tiles: lane = entry for the scores (32 per round), lane =
// four channels for the values.  qs / qn: q'' and q'' * norm in shared memory.  res: [128] channel sums, max, sum.
__device__ void tail_slice_warp(const Layout& L, const Counts& cn, const T5Args& a, int u, int e_lo, int e_hi,
                                const float* qs, const float* qn, float* res) {
  const int lane = threadIdx.x & 31;
  const int n_skew = cn.n_qk - cn.n_qv;
  const Rec rec = unit_rec(L, a.cache, u);
  const __half* k_sink = reinterpret_cast<const __half*>(a.cache + L.k.sink_off + (size_t)u * L.k.sink_stride);
  const __half* k_ring = reinterpret_cast<const __half*>(a.cache + L.k.ring_off + (size_t)u * L.k.ring_stride);
  const __half* v_sink = reinterpret_cast<const __half*>(a.cache + L.v.sink_off + (size_t)u * L.v.sink_stride);
  const __half* v_ring = reinterpret_cast<const __half*>(a.cache + L.v.ring_off + (size_t)u * L.v.ring_stride);
  auto v_row = [&](int e) -> const __half* {          // entry e of [skew tokens, sink tokens, recent key tokens]
    if (e >= n_skew && e - n_skew < cn.n_sink) return v_sink + (size_t)(e - n_skew) * kD;
    int slot = a.v_ring_pos0 + (e < n_skew ? e : n_skew + (e - n_skew - cn.n_sink));
    if (slot >= L.v.ring_cap) slot -= L.v.ring_cap;
    return v_ring + (size_t)slot * kD;
  };
  float m_run = -INFINITY, l_run = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int e0 = e_lo; e0 < e_hi; e0 += 32) {
    const int e = e0 + lane;
    float s = -INFINITY;
    if (e < n_skew && e < e_hi) {                       // packed key row
      const int i = cn.n_qv + e;
      const uint4* row4 = reinterpret_cast<const uint4*>(row_code_ptr(rec, L.k, i));
      const uint4 r0 = __ldg(row4), r1 = __ldg(row4 + 1);
      const uint32_t w[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
      const uint4 mw = __ldg(reinterpret_cast<const uint4*>(row_meta_ptr(rec, L.k, i)));
      const uint32_t mws[4] = {mw.x, mw.y, mw.z, mw.w};
      float d = 0.f;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        float sc, zc;
        decode_meta(mws[g], 2, sc, zc);
        float dg = 0.f, qg = 0.f;
#pragma unroll
        for (int cc = 0; cc < 32; ++cc) {
          const int c = 32 * g + cc, k = key_k_index(c);            // word (k / 2) / 8, field (k / 2) % 8, half k % 2
          const uint32_t code = (w[k >> 4] >> (16 * (k & 1) + 2 * ((k >> 1) & 7))) & 3u;
          dg = fmaf(qn[c], (float)code, dg);
          qg += qn[c];
        }
        d = fmaf(sc, dg, fmaf(zc, qg, d));
      }
      s = d;
    } else if (e < e_hi) {
      const int le = e - n_skew;
      const __half* kr;
      if (le < cn.n_sink) kr = k_sink + (size_t)le * kD;
      else {
        int slot = a.k_ring_pos0 + (le - cn.n_sink);
        if (slot >= L.k.ring_cap) slot -= L.k.ring_cap;
        kr = k_ring + (size_t)slot * kD;
      }
      float d = 0.f;
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(kr) + i);
        const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 f = __half22float2(h[k]);
          d = fmaf(f.x, qs[8 * i + 2 * k], fmaf(f.y, qs[8 * i + 2 * k + 1], d));
        }
      }
      s = d;
    }
    const float m_new = fmaxf(m_run, warp_max(s));
    const float alpha = m_run == -INFINITY ? 0.f : ex2_approx(m_run - m_new);
    const float p = e < e_hi ? ex2_approx(s - m_new) : 0.f;
    float ps = p;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    l_run = l_run * alpha + ps;
    m_run = m_new;
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] *= alpha;
    const int n = min(32, e_hi - e0);
    for (int ee = 0; ee < n; ++ee) {
      const float pe = __shfl_sync(0xffffffffu, p, ee);
      const uint2 v = __ldg(reinterpret_cast<const uint2*>(v_row(e0 + ee)) + lane);
      const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
      const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
      acc[0] = fmaf(pe, f0.x, acc[0]); acc[1] = fmaf(pe, f0.y, acc[1]);
      acc[2] = fmaf(pe, f1.x, acc[2]); acc[3] = fmaf(pe, f1.y, acc[3]);
    }
  }
  *reinterpret_cast<float4*>(res + 4 * lane) = make_float4(acc[0], acc[1], acc[2], acc[3]);
  if (lane == 0) { res[kD] = m_run; res[kD + 1] = l_run; }
}

constexpr int kT5Block = kT5Threads + 64;            // four compute warps, the issuing warp, the warp of the fp16 tokens

// Compute warps 0..3: thread t is token t of the tile on the key side and channel t on the value side.  Warp 4:
// its lane 0 starts the bulk copies and issues the MMAs.  They talk through mbarriers only (no CTA barrier in the
// loop):   ak_ready / avbp_ready (128 arrivals: the operands of the key / value MMA are complete),
//          dk_done / dv_done (the MMA's commit), full[s] / empty[s] (a stage's data has arrived / been consumed).
// Software pipeline of a compute thread:  MMA-K(i) || expand V(i);  MMA-V(i) || expand K(i+1);  MMA-K(i+1) || output(i).
__global__ void __launch_bounds__(kT5Block, 3) decode_tc5_kernel(const Layout L, const Counts cn, const T5Args a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool compute = warp < 4;
  const int u = blockIdx.x, split = blockIdx.y;
  unsigned char* misc = smem + kOffMisc;
  const uint32_t bar_full = smem_u32(misc), bar_empty = bar_full + 8 * kStages, bar_ak = bar_empty + 8 * kStages,
                 bar_avbp = bar_ak + 8, bar_dk = bar_avbp + 8, bar_dv = bar_dk + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 96);       // [0] operands, [1] accumulators
  float* redmax = reinterpret_cast<float*>(misc + 128);
  float* redsum = reinterpret_cast<float*>(misc + 144);
  float* qg_s = reinterpret_cast<float*>(misc + 160);
  float* red4 = reinterpret_cast<float*>(misc + 176);
  __shared__ unsigned int s_ticket;
  const int n_parts = gridDim.y;
  float out_c = 0.f, m_run = -INFINITY, l_run = 0.f;      // this thread's channel of the partial result
  bool failed = false;

  {
    const int n_chunks = cn.n_qv / kChunk, n_tiles = (n_chunks + kChunksPerTile - 1) / kChunksPerTile;
    const int t_lo = (int)((long long)split * n_tiles / a.n_splits), t_hi = (int)((long long)(split + 1) * n_tiles / a.n_splits);
    const int n_my = t_hi - t_lo;
    const unsigned char* g_rec = a.cache + L.k.rec_off + (size_t)u * L.k.rec_unit_stride;
    auto issue = [&](int it) {      // issuing lane: tile t_lo + it into stage it % kStages
      const int ti = t_lo + it, st = it % kStages;
      const int nv = min(kChunksPerTile, n_chunks - kChunksPerTile * ti);
      const uint32_t bytes = (uint32_t)nv * kRecBytes;
      mbar_expect_tx(bar_full + 8 * st, bytes);
      bulk_g2s(smem_u32(smem + st * kTileBytes), g_rec + (size_t)ti * kTileBytes, bytes, bar_full + 8 * st);
    };
    // ---------------- set-up that touches no global memory -------------------------------------------------------
    if (tid == 0) {
#pragma unroll
      for (int s = 0; s < kStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, kT5Threads); }
      mbar_init(bar_ak, kT5Threads);
      mbar_init(bar_avbp, kT5Threads);
      mbar_init(bar_dk, 1);
      mbar_init(bar_dv, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 4) {
      tmem_alloc(smem_u32(tmem_slot), kTmemColsA);
      tmem_alloc(smem_u32(tmem_slot + 1), kTmemColsD);
      tmem_alloc_done();
    }
    for (int i = tid; i < 8192 / 16; i += kT5Block) reinterpret_cast<uint4*>(smem + kOffBq)[i] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // ---------------- q'' and the B_q operand ---------------------------------------------------------------------
    const float* norm = reinterpret_cast<const float*>(a.cache + L.norm_off) + (size_t)u * kD;
    float qv = 0.f;
    float* qs_s = reinterpret_cast<float*>(smem + kOffScratch);       // q'' raw, q'' * norm, result of the fp16 tokens
    float* qn_s = qs_s + kD;
    float* tail_res = qn_s + kD;
    if (compute) {
      qv = __half2float(a.q[(size_t)u * kD + tid]) * (L.sm_scale * kLog2e);
      qs_s[tid] = qv;
      if (L.k_normalize) qv *= norm[tid];
      qn_s[tid] = qv;
    }
    __syncthreads();                 // barrier init, zero fill and the tensor-memory address are visible
    if (warp == 4 && lane == 0)
      for (int it = 0; it < kStages && it < n_my; ++it) issue(it);
    float amax = warp_max(fabsf(qv));
    if (compute && lane == 0) red4[warp] = amax;
    __syncthreads();
    amax = fmaxf(fmaxf(red4[0], red4[1]), fmaxf(red4[2], red4[3]));
    int e_q = 0;
    if (amax > 0.f && amax < INFINITY) e_q = ((__float_as_int(amax) >> 23) & 0xff) - 126;     // amax < 2^e_q
    if (compute) {
      const int k = key_k_index(tid), g = tid >> 5;
      const uint32_t v = split_hi_lo(qv * pow2i(14 - e_q - 2 * key_field(tid)));
      *reinterpret_cast<uint16_t*>(smem + kOffBq + b_offset(2 * g, k)) = (uint16_t)(v & 0xFFFFu);
      *reinterpret_cast<uint16_t*>(smem + kOffBq + b_offset(2 * g + 1, k)) = (uint16_t)(v >> 16);
      float gs = qv;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) gs += __shfl_xor_sync(0xffffffffu, gs, o);
      if (lane == 0) qg_s[warp] = gs;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // B_q is read by the tensor core (async proxy)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot[0], tbase_d = tmem_slot[1];

    if (warp == 5) {
      // ======================= the unit's fp16 / skew tokens: this CTA's slice =====================================
      const int total = (cn.n_qk - cn.n_qv) + cn.n_sink + cn.n_k_recent;
      const int e_lo = (int)((long long)split * total / gridDim.y), e_hi = (int)((long long)(split + 1) * total / gridDim.y);
      tail_slice_warp(L, cn, a, u, e_lo, e_hi, qs_s, qn_s, tail_res);
    } else if (!compute) {
      // ======================= issuing warp ======================================================================
      if (lane == 0) {
        auto issue_mma = [&](int col_d, int col_a, int off_b, uint32_t bar) {
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_ts(tbase_d + col_d, tbase + col_a + 8 * ks, smem_desc(smem_u32(smem + off_b) + 512 * ks, 256, 128), ks > 0);
          mma_commit(bar);
        };
        for (int it = 0; it < n_my && !failed; ++it) {
          if (!mbar_wait(bar_ak, (uint32_t)it & 1u)) { failed = true; break; }
          issue_mma(kColDk, kColAk, kOffBq, bar_dk);
          if (it >= 1 && it - 1 + kStages < n_my) {                  // the stage of tile it-1 has been consumed: refill it
            if (!mbar_wait(bar_empty + 8 * ((it - 1) % kStages), (uint32_t)((it - 1) / kStages) & 1u)) { failed = true; break; }
            issue(it - 1 + kStages);
          }
          if (!mbar_wait(bar_avbp, (uint32_t)it & 1u)) { failed = true; break; }
          issue_mma(kColDv, kColAv, kOffBp, bar_dv);
        }
      }
      __syncwarp();
    } else {
      // ======================= compute warps =====================================================================
      const uint32_t t_lane = tbase + ((uint32_t)(32 * warp) << 16);   // this warp's quarter of the 128 lanes
      const uint32_t t_lane_d = tbase_d + ((uint32_t)(32 * warp) << 16);
      const float kfac = pow2i(24 - (14 - e_q)), inv_kfac = pow2i(-(24 - (14 - e_q)));
      const float Qg[4] = {qg_s[0] * inv_kfac, qg_s[1] * inv_kfac, qg_s[2] * inv_kfac, qg_s[3] * inv_kfac};
      // this thread as a channel of the value side
      const int vm_ = 4 * (tid >> 6) + ((tid >> 1) & 3), vgid = (tid >> 3) & 7, vrh = tid & 1;
      const int v_word0 = (vm_ >> 2) * 128 + 16 * vgid + (vm_ & 3);          // + 4 * jj
      const int v_meta_idx = block_meta_index(tid);
      // this thread as a token of the key side: where its probability goes in B_p
      const int p_off = b_offset(warp, val_k_index(warp, lane));
      const float p_scale = pow2i(10 - 2 * val_field(lane));
      auto expand_keys = [&](const unsigned char* sp) {       // packed row of token `tid` -> row `tid` of A_k
        const uint4* row = reinterpret_cast<const uint4*>(sp + warp * kRecBytes + lane * kKRow);
        const uint4 r0 = row[0], r1 = row[1];
        const uint32_t w[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t regs[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int wi = 2 * q4 + (i >> 3), fld = i & 7;
            const uint32_t x = fld >= 4 ? (w[wi] >> 8) : w[wi];
            regs[i] = x & (0x00030003u << (2 * (fld & 3)));
          }
          tmem_st16(t_lane + kColAk + 16 * q4, regs);
        }
      };
      auto expand_values = [&](const unsigned char* sp) {     // codes of channel `tid` for the tile's tokens -> A_v
#pragma unroll
        for (int ch = 0; ch < kChunksPerTile; ++ch) {
          const uint32_t* vc = reinterpret_cast<const uint32_t*>(sp + ch * kRecBytes + kOffVCodes);
          uint32_t regs[16];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const uint32_t x = vc[v_word0 + 4 * jj] >> (8 * vrh);
#pragma unroll
            for (int fld = 0; fld < 4; ++fld) regs[4 * jj + fld] = x & (0x00030003u << (2 * fld));
          }
          tmem_st16(t_lane + kColAv + 16 * ch, regs);
        }
      };
      // (A wait that runs out does not leave the loop; later waits are skipped and the result is discarded.)
      if (n_my > 0) {
        if (!mbar_wait(bar_full, 0u)) failed = true;
        expand_keys(smem);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_ak);
      }
      for (int it = 0; it < n_my; ++it) {
        const int st = it % kStages, ti = t_lo + it;
        const int nv = min(kChunksPerTile, n_chunks - kChunksPerTile * ti);
        const unsigned char* sp = smem + st * kTileBytes;
        expand_values(sp);                                                       // || MMA-K(it)
        // ---------------- scores of token `tid`; probabilities relative to the chunk's own maximum -----------------
        if (!failed && !mbar_wait(bar_dk, (uint32_t)it & 1u)) failed = true;
        tc_fence_after();
        float d[8];
        tmem_ld8(t_lane_d + kColDk, d);
        float s;
        {
          const uint4 mw = *reinterpret_cast<const uint4*>(sp + warp * kRecBytes + kOffKMeta + lane * kKMetaRow);
          const uint32_t mws[4] = {mw.x, mw.y, mw.z, mw.w};
          float acc = 0.f;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const __half2 h2 = *reinterpret_cast<const __half2*>(&mws[g]);
            const float sg = __low2float(h2);
            const float z = fmaf(-2.0f, fmaxf(sg, 0.f), __high2float(h2));       // symmetric groups: -s * 2^(b-1)
            acc = fmaf(fabsf(sg), d[2 * g] + d[2 * g + 1], fmaf(z, Qg[g], acc));
          }
          s = warp < nv ? acc * kfac : -INFINITY;
        }
        const float wmax = warp_max(s);
        const float p = warp < nv ? ex2_approx(s - wmax) : 0.f;                  // chunk = warp = one column of B_p
        const float wsum = warp_sum_unit(p);
        if (lane == 0) { redmax[warp] = wmax; redsum[warp] = wsum; }
        *reinterpret_cast<__half*>(smem + kOffBp + p_off) = __float2half_rn(p * p_scale);
        tc_wait_st();                                                            // A_v
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");             // B_p
        tc_fence_before();
        mbar_arrive(bar_avbp);
        // value metadata of channel `tid` (the stage is handed back before it is used)
        uint32_t vmeta[4];
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
          vmeta[ch] = *reinterpret_cast<const uint32_t*>(sp + ch * kRecBytes + kOffVMeta + 4 * v_meta_idx);
        if (it + 1 < n_my) {                                                     // || MMA-V(it)
          const int st1 = (it + 1) % kStages;
          if (!failed && !mbar_wait(bar_full + 8 * st1, (uint32_t)((it + 1) / kStages) & 1u)) failed = true;
          expand_keys(smem + st1 * kTileBytes);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(bar_ak);
        }
        // the chunks' maxima and sums (all four warps have written theirs once avbp_ready has completed)
        if (!failed && !mbar_wait(bar_avbp, (uint32_t)it & 1u)) failed = true;
        float cm[4], cs[4];
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) { cm[ch] = redmax[ch]; cs[ch] = redsum[ch]; }
        const float m_new = fmaxf(m_run, fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3])));
        const float alpha = m_run == -INFINITY ? 0.f : ex2_approx(m_run - m_new);
        float cw[4];
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) cw[ch] = cm[ch] == -INFINITY ? 0.f : ex2_approx(cm[ch] - m_new);
        l_run = l_run * alpha + ((cs[0] * cw[0] + cs[1] * cw[1]) + (cs[2] * cw[2] + cs[3] * cw[3]));
        m_run = m_new;
        if (!failed && !mbar_wait(bar_dv, (uint32_t)it & 1u)) failed = true;
        tc_fence_after();
        float dv[4];
        tmem_ld4(t_lane_d + kColDv, dv);
        tc_fence_before();
        mbar_arrive(bar_empty + 8 * st);                                         // stage, D_v and B_p are free again
        // ---------------- output channel `tid` ------------------------------------------------- || MMA-K(it+1) ----
        out_c *= alpha;
#pragma unroll
        for (int ch = 0; ch < kChunksPerTile; ++ch) {
          if (ch < nv) {
            const __half2 h2 = *reinterpret_cast<const __half2*>(&vmeta[ch]);
            const float sg = __low2float(h2);
            const float z = fmaf(-2.0f, fmaxf(sg, 0.f), __high2float(h2));
            out_c = fmaf(cw[ch], fmaf(fabsf(sg), dv[ch] * 0x1p14f, z * cs[ch]), out_c);
          }
        }
      }
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    failed = __syncthreads_or(failed ? 1 : 0) != 0;
    if (warp == 4) {
      tmem_dealloc(tmem_slot[0], kTmemColsA);
      tmem_dealloc(tmem_slot[1], kTmemColsD);
    }
    if (failed) {
      if (tid == 0) atomicExch(reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off) + L.U, 1u);
      m_run = -INFINITY; l_run = 0.f; out_c = 0.f;
    } else if (compute) {          // add the slice of fp16 tokens (its results were published by the barrier above)
      const float mt = tail_res[kD], lt = tail_res[kD + 1];
      const float m_new = fmaxf(m_run, mt);
      const float wa = m_run == -INFINITY ? 0.f : ex2_approx(m_run - m_new), wb = mt == -INFINITY ? 0.f : ex2_approx(mt - m_new);
      out_c = out_c * wa + tail_res[tid] * wb;
      l_run = l_run * wa + lt * wb;
      m_run = m_new;
    }
  }

  // ---------------- partial result, ticket, merge by the last CTA of the unit ------------------------------------
  float* partials = reinterpret_cast<float*>(a.ws + L.ws_partial_off);
  if (compute) {
    float* P = partials + ((size_t)u * L.max_splits + split) * kPartialStride;
    P[tid] = m_run == -INFINITY ? 0.f : out_c;
    if (tid == 0) { P[kD] = m_run; P[kD + 1] = l_run; }
  }
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    s_ticket = atomicAdd(reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off) + u, 1u);
  }
  __syncthreads();
  if (s_ticket != (unsigned int)(n_parts - 1)) return;
  __threadfence();
  merge_parts4(partials, reinterpret_cast<float*>(smem), a.out, n_parts, u, L.max_splits);
  if (tid == 0) reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off)[u] = 0u;
}

}  // namespace

// The format this kernel is built for.
bool decode_tc5_supported(const Layout& L) {
  return L.page_groups == 0 && L.grouping == 0 && L.r == 1 && L.G == 32 && L.k.kind == kRow && L.v.kind == kBlock && L.k.bits == 2 &&
         L.v.bits == 2 && L.k.meta_bytes == 4 && L.v.meta_bytes == 4;
}

int launch_decode_tc5(const Layout& L, const unsigned char* cache, unsigned char* ws, int N, const __half* q, __half* out,
                      int n_splits, cudaStream_t st) {
  if (!decode_tc5_supported(L)) return -2;
  const Counts cn = counts_for(L, N);
  static std::atomic<unsigned long long> configured{0};
  if (!opt_in_dynamic_smem(decode_tc5_kernel, kT5Smem, configured)) return -1;
  const int n_tiles = (cn.n_qv / kChunk + kChunksPerTile - 1) / kChunksPerTile;
  if (n_splits <= 0) n_splits = (3 * 148) / L.U;         // three CTAs per SM
  if (n_splits > n_tiles) n_splits = n_tiles;
  if (n_splits > L.max_splits) n_splits = L.max_splits;
  if (n_splits < 1) n_splits = 1;                        // short contexts: the fp16 tokens only
  T5Args a;
  a.cache = cache; a.ws = ws; a.q = q; a.out = out;
  a.n_splits = n_splits;
  a.k_ring_pos0 = L.k.ring_cap ? cn.n_qk % L.k.ring_cap : 0;
  a.v_ring_pos0 = L.v.ring_cap ? cn.n_qv % L.v.ring_cap : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(L.U, n_splits); cfg.blockDim = dim3(kT5Block); cfg.dynamicSmemBytes = kT5Smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_tc5_kernel, L, cn, a) == cudaSuccess ? 1 : -1;
}

}  // namespace iq
