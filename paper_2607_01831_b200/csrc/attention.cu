// lynx_anchor_attention and lynx_merge_verify_attention: split-K decode attention over the
// packed nibble planes, dequantised on chip (sm_100a).  This file holds what the kernels share
// (parameters, PTX helpers, the end-of-piece merge and the accept / reject decision) and the host
// side; the kernels are in attention_i8.cuh and attention_wide.cuh.
//
// What is computed (Section 2 attention equation on the states of Section 4.2; accept/reject
// of Section 4.3): for every (sequence, KV head) the G = Hq/Hkv query heads of each of the n_q
// query positions ("columns", n_q*G of them) share one pass over that head's K and V planes.
//
// Per-token groups make dequantisation almost free: with x^ = zero_t + scale_t * level,
//     q . K^_t        = scale_t * (q . level_t) + zero_t * sum_d q_d
//     sum_t p_t V^_t  = sum_t (p_t scale_t) level_t + (sum_t p_t zero_t) * 1
// so the two contractions run on the integer levels and the scalars are applied per token
// outside.  Anchor attention (any column count) and verification with up to 16 columns per launch
// (17..32 columns: two such launches) run both contractions as exact integer products on
// tcgen05.mma kind::i8 (attention_i8.cuh); verification with 33..64 columns per launch runs them on
// tcgen05.mma kind::f16 with two-term FP16 weights (attention_wide.cuh).
//
// Common shape.  Persistent grid, one CTA per SM, flash-decoding split-K in stream-K form: the
// (sequence, KV head, stage-unit) list is cut into equal contiguous ranges, one per CTA.
// Producer warps stream 16-token sub-blocks of the planes (1 KiB each, contiguous in the paged
// layout) into a shared-memory ring with bulk copies (TMA) completing on mbarriers, and
// the queries of each piece into one of two slots.
// A range that covers a whole (sequence, KV head) writes the output directly, otherwise the
// partial (m, l, O) goes to the workspace and the last contributor (atomic ticket, no waiting)
// merges them; for verification the last CTA of a sequence also takes the accept/reject
// decision.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "lynx_common.cuh"

namespace lynx {
namespace {

constexpr int kMaxQ = 16;          // query positions per launch
constexpr int kMaxWindow = 64;     // query positions per call (Section 5.1: at most 64 speculative tokens); more than
                                   // kMaxQ positions or kMaxCols columns run as slices, one pass over the planes each
constexpr int kMaxCols = 64;       // n_q * G per launch
constexpr int kPartStride = 132;   // floats per (chunk, column) partial: O[128], m, l, pad

struct AttnParams {
  const __nv_bfloat16* q;
  const uint8_t *ka, *kr, *va, *vr;
  const float *km, *vm;
  const int32_t* block_table;
  const int32_t* seq_lens;
  float* out;
  const float* draft;
  int32_t* first_reject;
  float* dev;
  uint32_t* ws_flags;
  uint32_t* ws_chunk_ctr;  // [B*Hkv]
  uint32_t* ws_seq_ctr;    // [B]
  uint32_t* ws_group_ctr;  // [2 * CTAs of the largest grid]: tickets of the groups of partial slots
  float* ws_shadow;        // FP32 copies of the O accumulators (see kFlushMmas), or null
  float* ws_dev;           // [B*Hkv][kMaxQ]
  float* ws_lse;           // [B][nq_stride][Hq] natural-log log-sum-exp of every output row's scores
  float* ws_part;          // [B*Hkv + CTAs][ncols_pad][kPartStride], slot = segment + CTA index
  float atol, rtol;
  float sm_log2;           // softmax_scale * log2(e)
  int B, nq, causal, Hq, Hkv, G, bt, num_blocks, max_blocks, ncols;
  // A call may be one slice [j0, j0 + nq) of the caller's n_q query positions (q and out then point at
  // position j0): nq_stride = the caller's n_q (positions per sequence in q and out), tail = n_q - j0
  // (the causal limit of position j of the slice is len - tail + j + 1).  Unsliced: both equal nq.
  int nq_stride, tail;
};

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
// One probe of the barrier.  The hint lets the hardware park the thread (up to ~20 us here)
// until the phase completes instead of returning at once, so a waiting warp does not burn
// issue slots on polling; completion wakes it early.
constexpr uint32_t kMbarHintNs = 20000;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kMbarHintNs)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: gives up after ~2 s (at once if another thread of the CTA already gave up),
// records it in the CTA's abort word and returns false.  Callers carry on without the data (every
// loop has a fixed trip count, so the kernel still ends) and the host is told through the
// workspace status word.  Nothing in this kernel waits on another CTA.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_word) {
  if (*abort_word) return false;
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_word) return false;
    if (globaltimer_ns() - t0 > 2000000000ull) {
      *abort_word = 1;
      return false;
    }
  }
}
// One non-blocking probe of an mbarrier phase.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_word) {
  if (mbar_test(bar, parity)) return true;   // (a plain probe is several times quicker than one that may suspend)
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_word);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  return __byte_perm(a, b, sel);
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 lds64f(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

// Packed FP32 pairs (Blackwell fma/add/mul .f32x2: two lanes per instruction).
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// Full codes of 8 elements from an anchor word and a residual word: ev = codes of elements
// 0,2,4,6 (one per byte), od = codes of elements 1,3,5,7.
// Each is one shift and one bitwise select, (a & mask) | (b & ~mask), in a single LOP3.
__device__ __forceinline__ uint32_t bit_select(uint32_t a, uint32_t b, uint32_t mask) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xE4;" : "=r"(d) : "r"(a), "r"(b), "r"(mask));
  return d;
}
__device__ __forceinline__ void merge_codes(uint32_t xa, uint32_t xr, uint32_t& ev, uint32_t& od) {
  ev = bit_select(xa << 4, xr, 0xF0F0F0F0u);
  od = bit_select(xa, xr >> 4, 0xF0F0F0F0u);
}
// Natural-log log-sum-exp of a row's scores from its running maximum (or reference exponent) M, in log2 units,
// and the sum L of 2^(score - M); -inf for a row that saw no token.
__device__ __forceinline__ float lse_of(float M, float L) {
  return L > 0.0f ? (M + __log2f(L)) * 0.6931471805599453f : -INFINITY;
}
constexpr int kPieceUnits = 64;  // stage-units whose block ids are looked up at a time

struct Item {  // one piece: a run of stage-units of one (sequence, KV head) given to one CTA
  int b, hkv, len, first_cta, n_contrib, pad0, pad1, pad2;  // pad0 = units, pad1 = first unit
};

__device__ __forceinline__ void named_bar(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// After a piece's result is in the output (direct) or in its partial slot: the last
// contributor of the (sequence, KV head) merges the slots, and for verification the CTA holding
// the final outputs of a head takes part in the accept / reject decision (Section 4.3).
// Called by all consumer threads of the CTA (named barrier 1).
template <bool FULL, int kColsPad, int kConsThreads>
__device__ __forceinline__ void finish_piece(const AttnParams& p, const Item& item, bool direct, int tid,
                                             int* misc, int bar_id = 1) {
  const size_t bh = (size_t)item.b * p.Hkv + item.hkv;
  bool final_here = direct;
  if (!direct) {
    // The partial slots of this (sequence, KV head) are merged in two levels, so that no CTA walks
    // through all of them one L2 round trip after the other (74 slots for a 131072-token head on
    // 592 CTAs: 20 us at the tail of the launch).  The last CTA to arrive of each group of kGroup
    // neighbouring contributors merges the group into its first slot; the last group to finish
    // merges the group results into the output.  Every ticket resets itself; nobody waits.
    constexpr int kGroup = 8, kOneLevel = 24;   // up to kOneLevel slots are merged in one go
    constexpr int kAhead = 6;                    // loads in flight per thread
    const int n = item.n_contrib;
    const int ng = (n + kGroup - 1) / kGroup;
    const int g = ((int)blockIdx.x - item.first_cta) / kGroup;
    const int gsize = min(kGroup, n - g * kGroup);
    float* seg = p.ws_part + (bh + (size_t)item.first_cta) * (size_t)kColsPad * kPartStride;
    const size_t cstride = (size_t)kColsPad * kPartStride;
    const int lane = tid & 31;
    named_bar(bar_id, kConsThreads);
    if (tid == 0) {
      bool last = true;   // of this CTA's group (n <= kOneLevel: of the whole segment)
      if (n <= kOneLevel) {
        last = atomicInc(p.ws_chunk_ctr + bh, (uint32_t)n - 1) == (uint32_t)n - 1;
      } else if (gsize > 1) {
        // the group's ticket lives with its first CTA; a CTA can lead two groups at most: the first
        // group of the segment that starts in its range, and a later group of the one that ends there
        uint32_t* ctr = p.ws_group_ctr + 2 * (item.first_cta + g * kGroup) + (g == 0 ? 1 : 0);
        last = atomicInc(ctr, (uint32_t)gsize - 1) == (uint32_t)gsize - 1;
      }
      misc[1] = last ? 1 : 0;
    }
    named_bar(bar_id, kConsThreads);
    final_here = false;
    bool top = n <= kOneLevel;   // this pass writes the output
    // (one copy of the merge code, run once or twice: uniform over the CTA)
    for (bool go = misc[1] != 0; go;) {
      __threadfence();
      const int first = top ? 0 : g * kGroup;
      const int count = top ? (n <= kOneLevel ? n : ng) : gsize;
      const size_t sstride = (top && n > kOneLevel ? (size_t)kGroup : (size_t)1) * cstride;
      // a warp per column, a lane per 4 dims; `count` slots from `first` on, merged online, kAhead
      // loads ahead; the result goes to the output (normalised) or back to slot `first`
      for (int c = tid >> 5; c < p.ncols; c += kConsThreads / 32) {
        float* col = seg + (size_t)first * cstride + (size_t)c * kPartStride;
        float M = -INFINITY, L = 0.0f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int i0 = 0; i0 < count; i0 += kAhead) {
          float mi[kAhead], li[kAhead];
          float4 oi[kAhead];
#pragma unroll
          for (int u = 0; u < kAhead; ++u) {
            const bool in = i0 + u < count;
            const float* src = col + (size_t)(in ? i0 + u : i0) * sstride;
            mi[u] = in ? __ldcg(src + 128) : -INFINITY;
            li[u] = __ldcg(src + 129);
            oi[u] = __ldcg(reinterpret_cast<const float4*>(src) + lane);
          }
#pragma unroll
          for (int u = 0; u < kAhead; ++u) {
            const float Mn = fmaxf(M, mi[u]);
            // an absent slot (mi = -inf) keeps fa = 1, fb = 0 once M is finite; while M is still
            // -inf both factors are forced to 0 / taken from the slot without forming inf - inf
            const float fa = M == -INFINITY ? 0.0f : ex2(M - Mn);
            const float fb = mi[u] == -INFINITY ? 0.0f : ex2(mi[u] - Mn);
            acc.x = acc.x * fa + oi[u].x * fb;
            acc.y = acc.y * fa + oi[u].y * fb;
            acc.z = acc.z * fa + oi[u].z * fb;
            acc.w = acc.w * fa + oi[u].w * fb;
            L = L * fa + li[u] * fb;
            M = Mn;
          }
        }
        if (top) {
          const float inv = L > 0.0f ? 1.0f / L : 0.0f;
          const int j = c / p.G, hh = c % p.G;
          float4* dst = reinterpret_cast<float4*>(
              p.out + (((size_t)item.b * p.nq_stride + j) * p.Hq + item.hkv * p.G + hh) * LYNX_D);
          dst[lane] = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
          if (lane == 0) p.ws_lse[((size_t)item.b * p.nq_stride + j) * p.Hq + item.hkv * p.G + hh] = lse_of(M, L);
        } else {
          reinterpret_cast<float4*>(col)[lane] = acc;
          if (lane == 0) { col[128] = M; col[129] = L; }
        }
      }
      if (top) {
        final_here = true;
        break;
      }
      // the group's result is in its first slot: one more ticket, among the groups
      __threadfence();
      named_bar(bar_id, kConsThreads);
      if (tid == 0) misc[1] = (atomicInc(p.ws_chunk_ctr + bh, (uint32_t)ng - 1) == (uint32_t)ng - 1);
      named_bar(bar_id, kConsThreads);
      go = misc[1] != 0;
      top = true;
    }
  }
  // accept / reject (Section 4.3): by the CTA that wrote the final outputs of this head
  if (FULL && p.draft != nullptr) {
    int* devs = misc + 16;
    named_bar(bar_id, kConsThreads);  // final outputs written; devs free
    if (final_here) {
      if (tid < kMaxQ) devs[tid] = 0;
      named_bar(bar_id, kConsThreads);
      for (int idx = tid; idx < p.ncols * LYNX_D; idx += kConsThreads) {
        const int c = idx >> 7, d = idx & 127;
        const int j = c / p.G, hh = c % p.G;
        const size_t o = (((size_t)item.b * p.nq_stride + j) * p.Hq + item.hkv * p.G + hh) * LYNX_D + d;
        const float f = p.out[o], dr = __ldg(p.draft + o);
        const float r = fabsf(f - dr) / (p.atol + p.rtol * fabsf(f));
        atomicMax(devs + j, __float_as_int(r));  // r >= 0: integer order = float order
      }
      named_bar(bar_id, kConsThreads);
      if (tid < p.nq) p.ws_dev[bh * kMaxQ + tid] = __int_as_float(devs[tid]);
      __threadfence();
      named_bar(bar_id, kConsThreads);
      if (tid == 0)
        misc[1] = (atomicInc(p.ws_seq_ctr + item.b, (uint32_t)p.Hkv - 1) == (uint32_t)p.Hkv - 1);
      named_bar(bar_id, kConsThreads);
      if (misc[1] && tid == 0) {
        __threadfence();
        int fr = p.nq;
        for (int j = p.nq - 1; j >= 0; --j) {
          float worst = 0.0f;
          for (int h = 0; h < p.Hkv; ++h)
            worst = fmaxf(worst, __ldcg(p.ws_dev + ((size_t)item.b * p.Hkv + h) * kMaxQ + j));
          p.dev[(size_t)item.b * p.nq_stride + j] = worst;
          if (worst > 1.0f) fr = j;
        }
        p.first_reject[item.b] = fr;
      }
    }
    named_bar(bar_id, kConsThreads);
  }
}


// The stream-K cut of the work list (units of ST tokens in (sequence, KV head, position) order) for
// CTA `cta` of `n_cta`, derived by one warp from the sequence lengths on the device.  Normally every
// CTA takes q = ceil(total / n_cta) consecutive units, wherever the (sequence, head) boundaries fall.
// When all sequences have the same number of units U and the B * Hkv segments are few enough to give
// each of them c >= 1 CTAs of its own (one layer of a long context per launch), the cut is aligned
// instead: q = ceil(U / c), and CTA i takes part i % c of segment i / c.  No CTA then pays for the
// end of one piece and the start of another, at the cost of n_cta - c * segments idle CTAs (accepted
// up to 15 %).  lo, hi index a list in which every segment occupies c * q entries, so that the
// contributors of a segment and their partial slots follow from lo and q as in the plain cut.
struct SkRange {
  long long q, lo, hi, off_lo;   // off_lo: offset of `lo` among the Hkv * U units of sequence b_lo
  int b_lo;
};
template <int ST, class ClampLen>
__device__ __forceinline__ SkRange sk_range(const AttnParams& p, int n_cta, int cta, int lane, ClampLen clamp_len) {
  SkRange r;
  long long tot = 0;
  int umin = 0x7FFFFFFF, umax = 0;
  for (int b = lane; b < p.B; b += 32) {
    const int u = (clamp_len(b) + ST - 1) / ST;
    tot += u;
    umin = min(umin, u);
    umax = max(umax, u);
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    tot += __shfl_xor_sync(0xFFFFFFFFu, tot, off);
    umin = min(umin, __shfl_xor_sync(0xFFFFFFFFu, umin, off));
    umax = max(umax, __shfl_xor_sync(0xFFFFFFFFu, umax, off));
  }
  const long long T = tot * p.Hkv;
  const long long segs = (long long)p.B * p.Hkv;
  if (umin == umax && umax > 0 && segs <= n_cta && (n_cta / segs) * segs * 100 >= 85LL * n_cta) {
    const int c = (int)(n_cta / segs), U = umax;
    r.q = (U + c - 1) / c;
    const int s = cta / c, part = cta % c;
    r.lo = r.hi = 0; r.b_lo = 0; r.off_lo = 0;
    if (s < segs && (long long)part * r.q < U) {
      r.b_lo = s / p.Hkv;
      r.off_lo = (long long)(s % p.Hkv) * U + (long long)part * r.q;
      r.lo = ((long long)s * c + part) * r.q;
      r.hi = r.lo + min(r.q, (long long)U - (long long)part * r.q);
    }
    return r;
  }
  r.q = (T + n_cta - 1) / n_cta;
  r.lo = (long long)cta * r.q;
  r.hi = (r.lo + r.q < T) ? r.lo + r.q : T;
  r.b_lo = 0;
  r.off_lo = 0;
  if (r.lo < r.hi) {
    long long running = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
      const int b = b0 + lane;
      const long long u = b < p.B ? (long long)p.Hkv * ((clamp_len(b) + ST - 1) / ST) : 0;
      long long incl = u;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const long long v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
      }
      const long long excl = running + incl - u;
      const bool hit = u > 0 && r.lo >= excl && r.lo < excl + u;
      const unsigned mk = __ballot_sync(0xFFFFFFFFu, hit);
      if (mk) {
        const int src = __ffs(mk) - 1;
        r.b_lo = b0 + src;
        r.off_lo = r.lo - __shfl_sync(0xFFFFFFFFu, excl, src);
        break;
      }
      running += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
  }
  return r;
}

#include "attention_wide.cuh"
#include "attention_i8.cuh"

// ------------------------------------------------------------------ host side
constexpr int kMaxCtasPerSm = 4;

// Query positions per launch of a verification call: all of them up to kMaxQ positions and kMaxCols
// columns, else as many whole positions as fit both.
inline int verify_slice(int nq, int G) {
  // (17..32 columns: two passes of the exact integer kernel at 16 columns measure as fast as one pass of the
  // FP16 kernel at 32, without its limits on the value range)
  if (nq * G > 16 && nq * G <= 32 && 16 / G > 0) return 16 / G;
  if (nq <= kMaxQ && nq * G <= kMaxCols) return nq;
  const int by_cols = kMaxCols / G > 0 ? kMaxCols / G : 1;
  return by_cols < kMaxQ ? by_cols : kMaxQ;
}

struct Plan {
  int per;             // query positions per verification launch
  int ncols, variant;  // variant: 0: NT1 TW4 CG1; 1: NT2 TW4 CG1; 2: NT2 TW4 CG2; 3: NT2 TW2 CG4
  int cols_pad;
  size_t off_chunk_ctr, off_seq_ctr, off_group_ctr, off_dev, off_lse, off_part, bytes;
  size_t shadow_bytes;   // optional tail of the workspace: FP32 copies of the accumulators (see kFlushMmas)
};

bool make_plan(const lynx_shape* s, int B, int nq, Plan* pl) {
  if (!s || s->head_dim != LYNX_D || s->num_kv_heads <= 0 || s->num_q_heads <= 0 ||
      s->num_q_heads % s->num_kv_heads != 0 || s->block_tokens <= 0 || s->block_tokens % 16 != 0 ||
      s->num_blocks <= 0 || s->max_blocks_per_seq <= 0 || B <= 0 || nq <= 0 || nq > kMaxWindow)
    return false;
  const int G = s->num_q_heads / s->num_kv_heads;
  if (G > 16) return false;
  // positions per launch of a verification call (anchor calls slice further, to 32 columns); the scratch is
  // sized for the widest launch
  pl->per = verify_slice(nq, G);
  const int ncols = pl->per * G;
  const int64_t cap = (int64_t)s->max_blocks_per_seq * s->block_tokens;
  if (cap >= (1ll << 31)) return false;
  if ((int64_t)s->num_blocks * s->num_kv_heads * s->block_tokens >= (1ll << 32)) return false;
  pl->ncols = ncols;
  pl->variant = ncols <= 8 ? 0 : ncols <= 16 ? 1 : ncols <= 32 ? 2 : 3;
  // (the partial slots also serve anchor calls on the same workspace, which take up to 32 columns per launch)
  const int cols_anchor = nq * G <= 32 ? nq * G : (32 / G > 0 ? 32 / G : 1) * G;
  const int cols_max = ncols > cols_anchor ? ncols : cols_anchor;
  pl->cols_pad = cols_max <= 8 ? 8 : cols_max <= 16 ? 16 : cols_max <= 32 ? 32 : 64;
  size_t off = kWsHeaderBytes;
  pl->off_chunk_ctr = off; off += (size_t)B * s->num_kv_heads * 4;
  pl->off_seq_ctr = off;   off += (size_t)B * 4;
  pl->off_group_ctr = off; off += (size_t)2 * sm_count() * kMaxCtasPerSm * 4;
  off = (off + 255) & ~(size_t)255;
  pl->off_dev = off;       off += (size_t)B * s->num_kv_heads * kMaxQ * 4;
  off = (off + 255) & ~(size_t)255;
  pl->off_lse = off;       off += (size_t)B * nq * s->num_q_heads * 4;
  off = (off + 255) & ~(size_t)255;
  pl->off_part = off;
  off += ((size_t)B * s->num_kv_heads + (size_t)sm_count() * kMaxCtasPerSm) * pl->cols_pad * kPartStride * 4;
  pl->bytes = (off + 255) & ~(size_t)255;
  // FP32 copies of the accumulators of the FP16 kernel (verification with 33..64 columns per launch):
  // 2 groups x 128 rows x 128 dims per CTA
  pl->shadow_bytes = ncols > 32 ? (size_t)sm_count() * 131072 : 0;
  return true;
}

// Section 4.3's longest agreeing prefix over a window that was verified in slices: the smallest position
// whose deviation exceeds 1, or the number of positions.
__global__ void first_reject_kernel(const float* __restrict__ dev, int B, int nq, int32_t* __restrict__ first_reject) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int fr = nq;
  for (int j = nq - 1; j >= 0; --j)
    if (dev[(size_t)b * nq + j] > 1.0f) fr = j;
  first_reject[b] = fr;
}

// Section 4.3's agreement test on outputs that are already in memory (a verification pass whose result was joined
// with a BF16 tail first): dev[b][j] = max over heads and dims of |f - d| / (atol + rtol |f|), the arithmetic of
// the decision fused into the verification kernels.  One CTA per (sequence, position).
__global__ void __launch_bounds__(256) deviation_kernel(const float4* __restrict__ out_full, const float4* __restrict__ draft,
                                                        int row_f4, float atol, float rtol, float* __restrict__ dev) {
  const float4* f = out_full + (size_t)blockIdx.x * row_f4;
  const float4* d = draft + (size_t)blockIdx.x * row_f4;
  float worst = 0.0f;
  for (int i = threadIdx.x; i < row_f4; i += 256) {
    const float4 a = f[i], b = __ldg(d + i);
    worst = fmaxf(worst, fabsf(a.x - b.x) / (atol + rtol * fabsf(a.x)));
    worst = fmaxf(worst, fabsf(a.y - b.y) / (atol + rtol * fabsf(a.y)));
    worst = fmaxf(worst, fabsf(a.z - b.z) / (atol + rtol * fabsf(a.z)));
    worst = fmaxf(worst, fabsf(a.w - b.w) / (atol + rtol * fabsf(a.w)));
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) worst = fmaxf(worst, __shfl_xor_sync(0xFFFFFFFFu, worst, off));
  __shared__ float red[8];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = worst;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < 8; ++w) worst = fmaxf(worst, red[w]);
    dev[blockIdx.x] = worst;
  }
}

lynx_status run_attention(bool full, const lynx_shape* shape, const void* q, int B, int nq, int causal,
                          lynx_plane K, lynx_plane V, const int32_t* block_table,
                          const int32_t* seq_lens, float softmax_scale, const float* draft,
                          float atol, float rtol, float* out, int32_t* first_reject, float* dev,
                          void* workspace, size_t workspace_bytes, void* stream, bool fixed_scratch = false) {
  if (B == 0) return LYNX_OK;
  if (!shape) return LYNX_ERR_NULL;
  if (B < 0 || nq <= 0) return LYNX_ERR_SHAPE;
  if (shape->head_dim != LYNX_D || shape->block_tokens <= 0 || shape->block_tokens % 16 != 0)
    return LYNX_ERR_UNSUPPORTED;
  Plan pl;
  if (!make_plan(shape, B, nq, &pl)) return LYNX_ERR_UNSUPPORTED;
  if (!q || !K.anchor || !K.meta || !V.anchor || !V.meta || !block_table || !seq_lens || !out || !workspace)
    return LYNX_ERR_NULL;
  if (full && (!K.residual || !V.residual)) return LYNX_ERR_NULL;
  if (full && draft && (!first_reject || !dev)) return LYNX_ERR_NULL;
  if (!aligned16(q) || !aligned16(K.anchor) || !aligned16(V.anchor) || !aligned16(K.meta) ||
      !aligned16(V.meta) || !aligned16(workspace) || !aligned16(out) ||
      (full && (!aligned16(K.residual) || !aligned16(V.residual))))
    return LYNX_ERR_ALIGN;
  // the FP16 kernels cut their accumulation chains into FP32 copies at the end of the workspace; the
  // fixed-scratch entry point has no room for them and says so in its contract
  const bool fp16_kernel = full && pl.ncols > 32;   // (pl.ncols: the columns of the widest launch)
  const bool use_shadow = fp16_kernel && !fixed_scratch;
  if (workspace_bytes < pl.bytes + (use_shadow ? pl.shadow_bytes : 0)) return LYNX_ERR_WORKSPACE;
  if (full && draft && !(atol > 0.0f && rtol >= 0.0f)) return LYNX_ERR_SHAPE;

  unsigned char* ws = static_cast<unsigned char*>(workspace);
  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.ka = K.anchor; p.kr = K.residual; p.km = K.meta;
  p.va = V.anchor; p.vr = V.residual; p.vm = V.meta;
  p.block_table = block_table; p.seq_lens = seq_lens;
  p.out = out; p.draft = full ? draft : nullptr; p.first_reject = first_reject; p.dev = dev;
  p.ws_flags = reinterpret_cast<uint32_t*>(ws);
  p.ws_chunk_ctr = reinterpret_cast<uint32_t*>(ws + pl.off_chunk_ctr);
  p.ws_seq_ctr = reinterpret_cast<uint32_t*>(ws + pl.off_seq_ctr);
  p.ws_group_ctr = reinterpret_cast<uint32_t*>(ws + pl.off_group_ctr);
  p.ws_shadow = use_shadow ? reinterpret_cast<float*>(ws + pl.bytes) : nullptr;
  p.ws_dev = reinterpret_cast<float*>(ws + pl.off_dev);
  p.ws_lse = reinterpret_cast<float*>(ws + pl.off_lse);
  p.ws_part = reinterpret_cast<float*>(ws + pl.off_part);
  p.atol = atol; p.rtol = rtol;
  const float sc = softmax_scale == 0.0f ? 0.08838834764831845f : softmax_scale;
  p.sm_log2 = sc * 1.4426950408889634f;
  p.B = B; p.nq = nq; p.nq_stride = nq; p.tail = nq; p.causal = causal ? 1 : 0;
  p.Hq = shape->num_q_heads; p.Hkv = shape->num_kv_heads; p.G = p.Hq / p.Hkv;
  p.bt = shape->block_tokens; p.num_blocks = shape->num_blocks; p.max_blocks = shape->max_blocks_per_seq;
  p.ncols = pl.ncols;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the fixed array keeps what the previous call left: the status word and the tickets must be zero
  if (fixed_scratch && cudaMemsetAsync(workspace, 0, pl.off_dev, st) != cudaSuccess) return LYNX_ERR_CUDA;
  if (!full) {
    // Anchor attention: the integer tcgen05 kernels take up to 32 columns.  A call with more (33..64) is
    // run as slices of whole query positions, each a pass of its own over the planes, one after the
    // other on the stream (they share the workspace).
    const int per = nq * p.G <= 32 ? nq : (32 / p.G > 0 ? 32 / p.G : 1);
    for (int j0 = 0; j0 < nq; j0 += per) {
      AttnParams ps = p;
      ps.nq = nq - j0 < per ? nq - j0 : per;
      ps.ncols = ps.nq * p.G;
      ps.tail = nq - j0;
      ps.q = p.q + (size_t)j0 * p.Hq * LYNX_D;
      ps.out = p.out + (size_t)j0 * p.Hq * LYNX_D;
      ps.ws_lse = p.ws_lse + (size_t)j0 * p.Hq;
      const lynx_status rc = ps.ncols <= 4 ? launch_i8<false, 4>(ps, st) : ps.ncols <= 8 ? launch_i8<false, 8>(ps, st)
                           : ps.ncols <= 16 ? launch_i8<false, 16>(ps, st) : launch_i8<false, 32>(ps, st);
      if (rc != LYNX_OK) return rc;
    }
    return LYNX_OK;
  }
  // verification: the integer kernels up to 16 columns, tcgen05 with FP16 operands (attention_wide.cuh) above.
  // A window of more than kMaxQ positions or kMaxCols columns runs as slices of whole positions, each a pass
  // of its own over the planes that writes its outputs and deviations; the index of the first rejected
  // position over the whole window then follows from the deviations.
  for (int j0 = 0; j0 < nq; j0 += pl.per) {
    AttnParams ps = p;
    ps.nq = nq - j0 < pl.per ? nq - j0 : pl.per;
    ps.ncols = ps.nq * p.G;
    ps.tail = nq - j0;
    ps.q = p.q + (size_t)j0 * p.Hq * LYNX_D;
    ps.out = p.out + (size_t)j0 * p.Hq * LYNX_D;
    ps.ws_lse = p.ws_lse + (size_t)j0 * p.Hq;
    if (p.draft) { ps.draft = p.draft + (size_t)j0 * p.Hq * LYNX_D; ps.dev = p.dev + j0; }
    const lynx_status rc = ps.ncols <= 4 ? launch_i8<true, 4>(ps, st) : ps.ncols <= 8 ? launch_i8<true, 8>(ps, st)
                         : ps.ncols <= 16 ? launch_i8<true, 16>(ps, st) : launch_wide<2, 1>(ps, st);
    if (rc != LYNX_OK) return rc;
  }
  if (p.draft && pl.per < nq) {
    first_reject_kernel<<<(unsigned)((B + 127) / 128), 128, 0, st>>>(p.dev, B, nq, p.first_reject);
    return launch_status();
  }
  return LYNX_OK;
}

}  // namespace
}  // namespace lynx

extern "C" size_t lynx_workspace_bytes(const lynx_shape* shape, int32_t batch, int32_t n_cols_q) {
  lynx::Plan pl;
  if (!lynx::make_plan(shape, batch, n_cols_q, &pl)) return 0;
  return pl.bytes + pl.shadow_bytes;
}

extern "C" lynx_status lynx_verify_decision(const float* out_full, const float* draft_out, int32_t batch, int32_t k,
                                            int32_t num_q_heads, float atol, float rtol, int32_t* first_reject,
                                            float* dev, void* stream) {
  using namespace lynx;
  if (batch == 0) return LYNX_OK;
  if (batch < 0 || k <= 0 || k > kMaxWindow || num_q_heads <= 0 || (int64_t)batch * k >= (1ll << 31)) return LYNX_ERR_SHAPE;
  if (!out_full || !draft_out || !first_reject || !dev) return LYNX_ERR_NULL;
  if (!aligned16(out_full) || !aligned16(draft_out)) return LYNX_ERR_ALIGN;
  if (!(atol > 0.0f && rtol >= 0.0f)) return LYNX_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  deviation_kernel<<<(unsigned)(batch * k), 256, 0, st>>>(reinterpret_cast<const float4*>(out_full),
                                                         reinterpret_cast<const float4*>(draft_out),
                                                         num_q_heads * (LYNX_D / 4), atol, rtol, dev);
  lynx_status rc = launch_status();
  if (rc != LYNX_OK) return rc;
  first_reject_kernel<<<(unsigned)((batch + 127) / 128), 128, 0, st>>>(dev, batch, k, first_reject);
  return launch_status();
}

extern "C" const float* lynx_workspace_lse(const lynx_shape* shape, int32_t batch, int32_t n_q, const void* workspace) {
  lynx::Plan pl;
  if (!workspace || !lynx::make_plan(shape, batch, n_q, &pl)) return nullptr;
  return reinterpret_cast<const float*>(static_cast<const unsigned char*>(workspace) + pl.off_lse);
}

extern "C" lynx_status lynx_anchor_attention(const lynx_shape* shape, const void* q_bf16, int32_t batch,
                                             int32_t n_q, int32_t causal, lynx_plane K, lynx_plane V,
                                             const int32_t* block_table, const int32_t* seq_lens,
                                             float softmax_scale, float* out, void* workspace,
                                             size_t workspace_bytes, void* stream) {
  return lynx::run_attention(false, shape, q_bf16, batch, n_q, causal, K, V, block_table, seq_lens,
                             softmax_scale, nullptr, 0.f, 0.f, out, nullptr, nullptr, workspace,
                             workspace_bytes, stream);
}

extern "C" lynx_status lynx_merge_verify_attention(const lynx_shape* shape, const void* q_bf16,
                                                   int32_t batch, int32_t k, int32_t causal,
                                                   lynx_plane K, lynx_plane V,
                                                   const int32_t* block_table, const int32_t* seq_lens,
                                                   float softmax_scale, const float* draft_out,
                                                   float atol, float rtol, float* out_full,
                                                   int32_t* first_reject, float* dev, void* workspace,
                                                   size_t workspace_bytes, void* stream) {
  return lynx::run_attention(true, shape, q_bf16, batch, k, causal, K, V, block_table, seq_lens,
                             softmax_scale, draft_out, atol, rtol, out_full, first_reject, dev,
                             workspace, workspace_bytes, stream);
}

// ---------------------------------------------------------------------------------------------
// Anchor attention for callers that cannot hand over a workspace (no paper counterpart).
//
// The split-K partials, tickets and status word live in one fixed array in device memory that
// is part of the loaded library image: nothing is allocated, by this call or by any routine it
// uses.  Host code cannot use the array's name as an address (on the host the name is only a
// handle for the runtime), so the device address is looked up once per device with
// cudaGetSymbolAddress, while that device is current, and the kernels are given that address.
namespace lynx {
namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;  // 8 MiB held by every GPU that loads the library
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

lynx_status static_scratch_address(void** out) {
  static void* resolved[64] = {nullptr};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LYNX_ERR_CUDA;
  if (resolved[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return LYNX_ERR_CUDA;
    resolved[dev] = ptr;
  }
  *out = resolved[dev];
  return LYNX_OK;
}

}  // namespace
}  // namespace lynx

extern "C" lynx_status lynx_anchor_attention_static(const lynx_shape* shape, const void* q_bf16,
                                                    int32_t batch, int32_t n_q, int32_t causal,
                                                    lynx_plane K, lynx_plane V,
                                                    const int32_t* block_table, const int32_t* seq_lens,
                                                    float softmax_scale, float* out, void* stream) {
  using namespace lynx;
  if (batch == 0) return LYNX_OK;
  if (!shape) return LYNX_ERR_NULL;
  if (batch < 0 || n_q <= 0) return LYNX_ERR_SHAPE;
  Plan pl;
  if (!make_plan(shape, batch, n_q, &pl)) return LYNX_ERR_UNSUPPORTED;
  if (pl.bytes > kStaticScratchBytes) return LYNX_ERR_WORKSPACE;  // problem too large for the fixed array
  void* scratch = nullptr;
  const lynx_status st = static_scratch_address(&scratch);
  if (st != LYNX_OK) return st;
  // (validated there before anything is enqueued; the words that must start at zero are cleared on
  // `stream` only once the call is known to launch)
  return run_attention(false, shape, q_bf16, batch, n_q, causal, K, V, block_table, seq_lens,
                       softmax_scale, nullptr, 0.f, 0.f, out, nullptr, nullptr, scratch,
                       pl.bytes, stream, true);
}
