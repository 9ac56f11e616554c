// lynx_anchor_attention and lynx_merge_verify_attention: split-K decode attention over the
// packed nibble planes, dequantised in registers (sm_100a).
//
// What is computed (Section 2 attention equation on the states of Section 4.2; accept/reject
// of Section 4.3): for every (sequence, KV head) the G = Hq/Hkv query heads of each of the n_q
// query positions ("columns", n_q*G of them) share one pass over that head's K and V planes.
//
// Per-token groups make dequantisation almost free: with x^ = zero_t + scale_t * level,
//     q . K^_t        = scale_t * (q . level_t) + zero_t * sum_d q_d
//     sum_t p_t V^_t  = sum_t (p_t scale_t) level_t + (sum_t p_t zero_t) * 1
// so the two contractions run on the integer levels and the scalars are applied per token
// outside.  Q.K^T is exact integer arithmetic on the int8 tensor-core path (u8 levels times two
// s8 digit planes of the query).  P.V runs in FP16 with the levels as FP16 subnormals (the bit
// pattern 0x00cc is code * 2^-24: no conversion arithmetic) and the weights p * scale as the sum
// of two FP16 numbers (the rounded weight and the rounding's remainder, each with its own MMA), so
// the weights carry about 22 bits.  From 17 columns on the verify pass runs on tcgen05
// (attention_wide.cuh).
//
// Kernel shape.  Persistent grid (a few CTAs per SM), flash-decoding split-K in stream-K form:
// the (sequence, KV head, stage-unit) list is cut into equal contiguous ranges, one per CTA.
// A CTA has DS*TEAMS consumer warps and one producer warp.  The producer streams 16-token
// sub-blocks (1 KiB per plane + 128 B of meta, each contiguous in the paged layout) into a
// shared-memory ring with cp.async.bulk (TMA, 1-D) completing on mbarriers, and the queries of
// each piece into one of two slots.  A team of DS consumer warps takes DS 16-token tiles of
// every stage; warp d of the team does, for ALL columns,
//   S^T[16 tok x 8 col] = level(K)[16 x 128] . Q^T        mma.m16n8k32 u8 x s8, tokens are M
//   online softmax with a lazily updated maximum shared by the team
//   P^T -> B operand by movmatrix (8x8 b16 transpose), published in shared memory (DS > 1)
// for tile d, and then, for every tile of the team,
//   O^T[slice x 8 col] += level(V)^T[slice x 16 tok] . P^T  mma.m16n8k16 f16, dims are M
// for its own slice of 128/DS output dims: the nibbles of a tile are dequantised once however
// many columns there are, and the accumulators shrink with DS.
// K operands are the nibbles / merged codes themselves (one or two logic ops per 4 levels);
// V operands are built from the nibbles with LOP3/PRMT alone.
// A range that covers a whole (sequence, KV head) writes the output directly, otherwise the
// partial (m, l, O) goes to the workspace and the last contributor (atomic ticket, no waiting)
// merges them; for verification the last CTA of a sequence also takes the accept/reject
// decision.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "lynx_common.cuh"

namespace lynx {
namespace {

constexpr int kMaxQ = 16;          // query positions per call
constexpr int kMaxCols = 64;       // n_q * G
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
  float* ws_part;          // [B*Hkv + CTAs][ncols_pad][kPartStride], slot = segment + CTA index
  float atol, rtol;
  float sm_log2;           // softmax_scale * log2(e)
  int B, nq, causal, Hq, Hkv, G, bt, num_blocks, max_blocks, ncols;
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
#ifndef LYNX_MBAR_HINT_NS
#define LYNX_MBAR_HINT_NS 20000
#endif
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"((uint32_t)LYNX_MBAR_HINT_NS)
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_word) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_word);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
// the two FP16 halves of h as FP32 (exact)
__device__ __forceinline__ void unpack_f16x2(uint32_t h, float& lo, float& hi) {
  asm("{\n\t.reg .b16 l, u;\n\tmov.b32 {l, u}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, u;\n\t}"
      : "=f"(lo), "=f"(hi) : "r"(h));
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

// Four FP16 pairs from the low 16 bits of each half of u, with no arithmetic at all: a 16-bit
// pattern 0x000n is the FP16 subnormal n * 2^-24 and 0x00n0 is 16 n * 2^-24, both exact, and the
// tensor core takes subnormal FP16 operands as they are.  r[0], r[2] hold nibbles 0 and 2 of
// each half (scale 2^-24), r[1], r[3] nibbles 1 and 3 (scale 2^-20); the scales are undone
// when the accumulators are written out.  (Full codes use the same idea with one byte per
// 16-bit lane: 0x00cc = code * 2^-24.)
__device__ __forceinline__ void nib4_to_h2(uint32_t u, uint32_t (&r)[4]) {
  const uint32_t s = u >> 8;
  r[0] = u & 0x000F000Fu;
  r[1] = u & 0x00F000F0u;
  r[2] = s & 0x000F000Fu;
  r[3] = s & 0x00F000F0u;
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
// token row permutation inside a 16-token tile (keeps the shared-memory reads of both the
// K fragments and the V fragments at <= 2-way bank conflicts)
__device__ __forceinline__ int pi_row(int r) { return r ^ ((r >> 1) & 1); }

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
    constexpr int kGroup = 8, kOneLevel = 16;   // up to kOneLevel slots are merged in one go
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
      // a warp per column, a lane per 4 dims; `count` slots from `first` on, merged online, four
      // loads ahead; the result goes to the output (normalised) or back to slot `first`
      for (int c = tid >> 5; c < p.ncols; c += kConsThreads / 32) {
        float* col = seg + (size_t)first * cstride + (size_t)c * kPartStride;
        float M = -INFINITY, L = 0.0f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int i0 = 0; i0 < count; i0 += 4) {
          float mi[4], li[4];
          float4 oi[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const bool in = i0 + u < count;
            const float* src = col + (size_t)(in ? i0 + u : i0) * sstride;
            mi[u] = in ? __ldcg(src + 128) : -INFINITY;
            li[u] = __ldcg(src + 129);
            oi[u] = __ldcg(reinterpret_cast<const float4*>(src) + lane);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
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
              p.out + (((size_t)item.b * p.nq + j) * p.Hq + item.hkv * p.G + hh) * LYNX_D);
          dst[lane] = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
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
        const size_t o = (((size_t)item.b * p.nq + j) * p.Hq + item.hkv * p.G + hh) * LYNX_D + d;
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
          p.dev[(size_t)item.b * p.nq + j] = worst;
          if (worst > 1.0f) fr = j;
        }
        p.first_reject[item.b] = fr;
      }
    }
    named_bar(bar_id, kConsThreads);
  }
}

// The producer warp: works out this CTA's range of stage-units (and handles sequences with no
// token), then streams the pieces of the range: queries of each piece into one of two slots,
// 16-token sub-blocks of the planes into the ring.  `C` supplies the shared-memory geometry.
template <class C, bool FULL, int TW, int NSTAGE>
__device__ __forceinline__ void producer_warp(const AttnParams& p, int lane, uint32_t ring_u32,
                                              uint32_t full0, uint32_t empty0, uint32_t qfull0,
                                              uint32_t qempty0, __nv_bfloat16* q_s, uint32_t* blk_s,
                                              int4* info_s, Item* items, int* misc,
                                              volatile int* abort_word) {
  constexpr int ST = C::kST;
  const int n_cta = gridDim.x, cta = blockIdx.x;
  const int cap = p.max_blocks * p.bt;
  auto clamp_len = [&](int b) {
    int len = __ldg(p.seq_lens + b);
    return len < 0 ? 0 : (len > cap ? cap : len);
  };
  // ---- prologue (producer warp): total work, this CTA's range, empty sequences ----------
  long long tot = 0;
  for (int b = lane; b < p.B; b += 32) tot += (clamp_len(b) + ST - 1) / ST;
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) tot += __shfl_xor_sync(0xFFFFFFFFu, tot, off);
  const long long T = tot * p.Hkv;
  const long long q = (T + n_cta - 1) / n_cta;
  const long long lo = (long long)cta * q, hi = (lo + q < T) ? lo + q : T;
  int b_lo = 0;
  long long off_lo = 0;
  if (lo < hi) {
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
      const bool hit = u > 0 && lo >= excl && lo < excl + u;
      const unsigned m = __ballot_sync(0xFFFFFFFFu, hit);
      if (m) {
        const int src = __ffs(m) - 1;
        b_lo = b0 + src;
        off_lo = lo - __shfl_sync(0xFFFFFFFFu, excl, src);
        break;
      }
      running += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
  }
  if (lane == 0) {
    misc[4] = (int)(q > 0x7FFFFFFF ? 0x7FFFFFFF : q);
    misc[7] = lo < hi ? (int)(hi - lo) : 0;
  }
  // sequences with no token: outputs are zero, nothing is rejected unless the draft is not zero
  for (int b = cta; b < p.B; b += n_cta) {
    if (clamp_len(b) != 0) continue;
    const size_t n = (size_t)p.nq * p.Hq * LYNX_D;
    for (size_t i = lane; i < n; i += 32) p.out[(size_t)b * n + i] = 0.0f;
    if (FULL && p.draft != nullptr) {
      int fr = p.nq;
      for (int j = p.nq - 1; j >= 0; --j) {
        float worst = 0.0f;
        for (int i = lane; i < p.Hq * LYNX_D; i += 32)
          worst = fmaxf(worst, fabsf(__ldg(p.draft + ((size_t)b * p.nq + j) * p.Hq * LYNX_D + i)) / p.atol);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) worst = fmaxf(worst, __shfl_xor_sync(0xFFFFFFFFu, worst, off));
        if (lane == 0) p.dev[(size_t)b * p.nq + j] = worst;
        if (worst > 1.0f) fr = j;
      }
      if (lane == 0) p.first_reject[b] = fr;
    }
  }
  __syncthreads();  // (A) the range is published
  const int n_units = (int)(lo < hi ? hi - lo : 0);
  if (n_units == 0) return;

  // =============================== producer loop ===============================
  // every lane has fixed roles: role r = lane + 32 i copies one array of one 16-token sub-block
  constexpr int NARR = FULL ? 6 : 4;
  constexpr int NROLE = (TW * NARR + 31) / 32;
  int my_sub[NROLE];
  const unsigned char* my_src[NROLE];
  uint32_t my_mul[NROLE], my_dst[NROLE], my_bytes[NROLE];
#pragma unroll
  for (int i = 0; i < NROLE; ++i) {
    const int r = lane + 32 * i;
    my_sub[i] = r < TW * NARR ? r / NARR : TW;  // TW = no role
    const int arr = r % NARR;
    const bool is_meta = arr == 2 || arr == 3;
    my_src[i] = arr == 0 ? p.ka : arr == 1 ? p.va
              : arr == 2 ? reinterpret_cast<const unsigned char*>(p.km)
              : arr == 3 ? reinterpret_cast<const unsigned char*>(p.vm)
              : arr == 4 ? p.kr : p.vr;
    const uint32_t dst0 = arr == 0 ? 0u : arr == 1 ? ST * 64u
                        : arr == 2 ? (FULL ? ST * 256u : ST * 128u)
                        : arr == 3 ? (FULL ? ST * 264u : ST * 136u)
                        : arr == 4 ? ST * 128u : ST * 192u;
    my_mul[i] = is_meta ? 8u : 64u;
    my_bytes[i] = is_meta ? 128u : 1024u;
    my_dst[i] = dst0 + (uint32_t)(my_sub[i] < TW ? my_sub[i] : 0) * my_bytes[i];
  }
  int b = b_lo, len = clamp_len(b), U = (len + ST - 1) / ST;
  int hkv = (int)(off_lo / U), u = (int)(off_lo % U);
  int remaining = n_units, gs = 0, ic = 0;
  while (remaining > 0) {
    const int n = min(remaining, U - u);
    const int qi = ic & 1;
    if (ic >= 2) mbar_wait(qempty0 + qi * 8, ((ic >> 1) - 1) & 1, abort_word);
    const long long seg0 = lo + (n_units - remaining) - u;  // first unit of this segment
    if (lane == 0) {
      Item it;
      it.b = b; it.hkv = hkv; it.len = len;
      it.first_cta = (int)(seg0 / q);
      it.n_contrib = (int)((seg0 + U - 1) / q) - it.first_cta + 1;
      it.pad0 = n;   // units of this piece
      it.pad1 = u;   // index of its first unit within the sequence
      it.pad2 = 0;
      items[qi] = it;
      mbar_expect_tx(qfull0 + qi * 8, (uint32_t)(p.nq * p.G * LYNX_D * 2));
    }
    __syncwarp();
    for (int j = lane; j < p.nq; j += 32)
      bulk_g2s(smem_u32(q_s + ((size_t)qi * C::kColsPad + j * p.G) * LYNX_D),
               p.q + (((size_t)b * p.nq + j) * p.Hq + (size_t)hkv * p.G) * LYNX_D,
               (uint32_t)(p.G * LYNX_D * 2), qfull0 + qi * 8);
    for (int c0 = 0; c0 < n; c0 += kPieceUnits) {
      const int cn = min(kPieceUnits, n - c0);
      for (int i = lane; i < cn * TW; i += 32) {
        const int t0 = (u + c0) * ST + i * 16;
        uint32_t row = 0;
        if (t0 < len) {
          int blk = __ldg(p.block_table + (size_t)b * p.max_blocks + t0 / p.bt);
          if (blk < 0 || blk >= p.num_blocks) {
            atomicOr(p.ws_flags, kFlagBadBlock);
            blk = blk < 0 ? 0 : p.num_blocks - 1;
          }
          row = (uint32_t)(((size_t)blk * p.Hkv + hkv) * p.bt + (t0 % p.bt));
        }
        blk_s[i] = row;
      }
      __syncwarp();
      for (int k = 0; k < cn; ++k, ++gs) {
        const int slot = gs % NSTAGE;
        if (gs >= NSTAGE) mbar_wait(empty0 + slot * 8, ((gs / NSTAGE) - 1) & 1, abort_word);
        const int uu = u + c0 + k;
        const int nsub = min(TW, (len - uu * ST + 15) >> 4);
        const uint32_t bar = full0 + slot * 8;
        if (lane == 0) {
          info_s[slot] = make_int4(qi, uu, (c0 + k == 0 ? 1 : 0) | (c0 + k == n - 1 ? 2 : 0), 0);
          mbar_expect_tx(bar, nsub * C::kSubBytes);
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < NROLE; ++i)
          if (my_sub[i] < nsub)
            bulk_g2s(ring_u32 + slot * C::kStageBytes + my_dst[i],
                     my_src[i] + (size_t)blk_s[k * TW + my_sub[i]] * my_mul[i], my_bytes[i], bar);
      }
      __syncwarp();  // blk_s is rewritten by the next round
    }
    remaining -= n;
    u += n;
    ++ic;
    if (u == U && remaining > 0) {
      u = 0;
      if (++hkv == p.Hkv) {
        hkv = 0;
        do {
          ++b;
          len = b < p.B ? clamp_len(b) : 0;
          U = (len + ST - 1) / ST;
        } while (b < p.B && U == 0);
        if (b >= p.B) break;  // cannot happen: the range ends inside the list
      }
    }
  }
}

// =============================================================================================
// Shared-memory geometry of one kernel variant.  NT = 8-column tiles (all of them in every
// warp), DS = warps per team = tiles per team and step = slices of the output dims,
// TEAMS = teams per CTA.  The query fragments (two s8 digit planes) and sum-of-q live in shared
// memory, built once per piece.
// With DS > 1 a team keeps one running maximum per column: two named barriers per step, growth
// agreed through shared memory.  With DS == 1 a warp is its own team and nothing is exchanged.
// =============================================================================================
template <bool FULL, int NT, int DS, int TEAMS, int NSTAGE, int TPW = 1>
struct TeamCfg {
  static_assert(TPW == 1 || DS == 1, "several tiles per warp and stage only without teams");
  static constexpr int kTW = DS * TEAMS * TPW;              // tiles per stage (TPW per consumer warp)
  static constexpr int kST = kTW * 16;
  static constexpr int kSubBytes = FULL ? 16 * 272 : 16 * 144;
  static constexpr int kStageBytes = kST * (FULL ? 272 : 144);
  static constexpr int kConsWarps = DS * TEAMS;
  static constexpr int kConsThreads = kConsWarps * 32;
  static constexpr int kThreads = (kConsWarps + 1) * 32;
  static constexpr int kColsPad = NT * 8;
  static constexpr int kMT = 8 / DS;                        // m-tiles (16 dims) per warp
  static constexpr int kRing = NSTAGE * kStageBytes;
  static constexpr int kMailRegs = NT * kMT * 4 + NT * 6;   // o slice + m, l, zs
  static constexpr int kMailBytes = TEAMS > 1 ? kMailRegs * 32 * 4 : 0;  // one box, used slice by slice
  static constexpr int kXchgBytes = DS > 1 ? kConsWarps * (16 + kColsPad * 4 + NT * 4 * 32 * 4) : 0;  // flag, colmax, P^T (two terms)
  static constexpr int kLzBytes = DS * kColsPad * 2 * 4 + 16;
  static constexpr int kQfBytes = NT * 2 * 4 * 32 * 8 + kColsPad * 4;  // query fragments, sum of q
  static constexpr int kQBytes = 2 * kColsPad * LYNX_D * 2;
  static constexpr int kBlkBytes = kPieceUnits * kTW * 4;
  static constexpr int kInfoBytes = NSTAGE * 16 + 2 * 32;
  static constexpr int kBarBytes = (2 * NSTAGE + 4) * 8;
  static constexpr int kMiscBytes = 256;
  static constexpr int kSmem = kRing + kMailBytes + kXchgBytes + kLzBytes + kQfBytes + kQBytes +
                               kBlkBytes + kInfoBytes + kBarBytes + kMiscBytes;
};

// K operand fragments of one tile for all four k32 steps: a[wd] = {ev(row g), ev(row g+8),
// od(row g), od(row g+8)} (ev/od: levels of the even / odd elements of word wd).
template <bool FULL, int ST>
__device__ __forceinline__ void k_fragments(uint32_t st, int r0, int t, uint32_t (&a)[4][4]) {
  constexpr uint32_t KA = 0, KR = ST * 128;
  const uint4 a_lo = lds128(st + KA + r0 * 64 + t * 16);
  const uint4 a_hi = lds128(st + KA + (r0 + 8) * 64 + t * 16);
  const uint32_t xl[4] = {a_lo.x, a_lo.y, a_lo.z, a_lo.w};
  const uint32_t xh[4] = {a_hi.x, a_hi.y, a_hi.z, a_hi.w};
  if (FULL) {
    const uint4 b_lo = lds128(st + KR + r0 * 64 + t * 16);
    const uint4 b_hi = lds128(st + KR + (r0 + 8) * 64 + t * 16);
    const uint32_t yl[4] = {b_lo.x, b_lo.y, b_lo.z, b_lo.w};
    const uint32_t yh[4] = {b_hi.x, b_hi.y, b_hi.z, b_hi.w};
#pragma unroll
    for (int wd = 0; wd < 4; ++wd) {
      merge_codes(xl[wd], yl[wd], a[wd][0], a[wd][2]);
      merge_codes(xh[wd], yh[wd], a[wd][1], a[wd][3]);
    }
  } else {
#pragma unroll
    for (int wd = 0; wd < 4; ++wd) {
      a[wd][0] = xl[wd] & 0x0F0F0F0Fu; a[wd][2] = (xl[wd] >> 4) & 0x0F0F0F0Fu;
      a[wd][1] = xh[wd] & 0x0F0F0F0Fu; a[wd][3] = (xh[wd] >> 4) & 0x0F0F0F0Fu;
    }
  }
}

// O^T slice += level(V)^T[slice dims x 16 tokens] . P^T for one tile (stage rows row0..row0+15).
// Slice d of DS covers the m-tiles (word, half) of every lane's 16 dims: DS=1 all eight, DS=2
// word d, DS=4 word d>>1 / half d&1.
template <bool FULL, int NT, int ST, int DS, bool TWO>
__device__ __forceinline__ void pv_slice(float (&o)[NT][8 / DS][4], uint32_t st, int row0, int g, int t,
                                         int d, const uint32_t (&pb)[NT][4]) {
  constexpr uint32_t VA = ST * 64, VR = ST * 192;
  constexpr int NW = DS == 1 ? 2 : 1;  // words of the lane's 8 V bytes this warp touches
  constexpr int NH = DS == 4 ? 1 : 2;  // halves of each word
  const int ta = row0 + pi_row(2 * t), tb = row0 + pi_row(2 * t + 1);
  uint32_t A[NW], Bw[NW], C[NW], Dw[NW], RA[NW], RB[NW], RC[NW], RD[NW];
  const uint32_t wofs = DS == 1 ? 0u : (DS == 2 ? (uint32_t)d * 4u : (uint32_t)(d >> 1) * 4u);
  if constexpr (DS == 1) {  // both words of the lane's 8 bytes: one 64-bit load per token row
    const uint32_t off = g * 8;
    const uint2 va = lds64(st + VA + ta * 64 + off), vb = lds64(st + VA + tb * 64 + off);
    const uint2 vc = lds64(st + VA + (ta + 8) * 64 + off), vd = lds64(st + VA + (tb + 8) * 64 + off);
    A[0] = va.x; A[NW - 1] = va.y; Bw[0] = vb.x; Bw[NW - 1] = vb.y;
    C[0] = vc.x; C[NW - 1] = vc.y; Dw[0] = vd.x; Dw[NW - 1] = vd.y;
    if (FULL) {
      const uint2 ra = lds64(st + VR + ta * 64 + off), rb = lds64(st + VR + tb * 64 + off);
      const uint2 rc = lds64(st + VR + (ta + 8) * 64 + off), rd = lds64(st + VR + (tb + 8) * 64 + off);
      RA[0] = ra.x; RA[NW - 1] = ra.y; RB[0] = rb.x; RB[NW - 1] = rb.y;
      RC[0] = rc.x; RC[NW - 1] = rc.y; RD[0] = rd.x; RD[NW - 1] = rd.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < NW; ++i) {
      const uint32_t off = g * 8 + wofs + i * 4;
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(A[i]) : "r"(st + VA + ta * 64 + off));
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(Bw[i]) : "r"(st + VA + tb * 64 + off));
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(C[i]) : "r"(st + VA + (ta + 8) * 64 + off));
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(Dw[i]) : "r"(st + VA + (tb + 8) * 64 + off));
      if (FULL) {
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(RA[i]) : "r"(st + VR + ta * 64 + off));
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(RB[i]) : "r"(st + VR + tb * 64 + off));
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(RC[i]) : "r"(st + VR + (ta + 8) * 64 + off));
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(RD[i]) : "r"(st + VR + (tb + 8) * 64 + off));
      }
    }
  }
#pragma unroll
  for (int i = 0; i < NW; ++i) {
    uint32_t ea = 0, oa = 0, eb = 0, ob = 0, ec = 0, oc = 0, ed = 0, od = 0;
    if (FULL) {
      merge_codes(A[i], RA[i], ea, oa);
      merge_codes(Bw[i], RB[i], eb, ob);
      merge_codes(C[i], RC[i], ec, oc);
      merge_codes(Dw[i], RD[i], ed, od);
    }
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      const int half = DS == 4 ? (d & 1) : hh;
      const uint32_t sel = half ? 0x7632u : 0x5410u;
      uint32_t ab[4], cd[4];
      if (!FULL) {
        nib4_to_h2(prmt(A[i], Bw[i], sel), ab);  // dims e(4half+0..3), token pair (a, b)
        nib4_to_h2(prmt(C[i], Dw[i], sel), cd);  // same dims, token pair (c, d)
      } else {
        const uint32_t uab = prmt(ea, eb, sel), vab = prmt(oa, ob, sel);
        const uint32_t ucd = prmt(ec, ed, sel), vcd = prmt(oc, od, sel);
        // a 16-bit pattern 0x00cc is the FP16 subnormal code * 2^-24: one byte per 16-bit lane
        ab[0] = uab & 0x00FF00FFu; ab[1] = vab & 0x00FF00FFu;
        ab[2] = prmt(uab, 0u, 0x4341); ab[3] = prmt(vab, 0u, 0x4341);
        cd[0] = ucd & 0x00FF00FFu; cd[1] = vcd & 0x00FF00FFu;
        cd[2] = prmt(ucd, 0u, 0x4341); cd[3] = prmt(vcd, 0u, 0x4341);
      }
#pragma unroll
      for (int qd = 0; qd < 2; ++qd) {
        const int lm = (DS == 1 ? i * 4 : 0) + (DS == 4 ? 0 : hh * 2) + qd;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
        {  // the rounded weights, then the remainders of their rounding
          mma16816(o[nt][lm], ab[2 * qd], ab[2 * qd + 1], cd[2 * qd], cd[2 * qd + 1], pb[nt][0], pb[nt][1]);
          if (TWO) mma16816(o[nt][lm], ab[2 * qd], ab[2 * qd + 1], cd[2 * qd], cd[2 * qd + 1], pb[nt][2], pb[nt][3]);
        }
      }
    }
  }
}

template <bool FULL, int NT, int DS, int TEAMS, int NSTAGE, int TPW, bool PACK>
__device__ __forceinline__ void attn_team_body(const AttnParams& p) {
  // PACK (at most four query columns): columns 4..7 of the n-tile repeat columns 0..3 and carry the
  // remainders of the weights' rounding, so one MMA per operand does the work of two
  static_assert(!PACK || (NT == 1 && DS == 1), "column packing is for the single n-tile kernels");
  using C = TeamCfg<FULL, NT, DS, TEAMS, NSTAGE, TPW>;
  constexpr int ST = C::kST, TW = C::kTW, MT = C::kMT;
  constexpr uint32_t KM = FULL ? ST * 256 : ST * 128, VM = KM + ST * 8;
  constexpr float kMidK = FULL ? 0.0f : 8.0f;
  constexpr float kMidV = FULL ? 0.0f : 8.0f;      // V levels: plain codes (full) / plain nibbles (anchor)
  constexpr float kLevelScaleV = FULL ? 1.0f : 16.0f;
  // The FP16 weights are p * scale_v * 256 (p <= 16 against the lazily raised maximum): FP16 has no
  // room below 2^-24, and weights that vanish there would still count in the softmax sum and in the
  // zero-point term.  With the factor a weight vanishes only below 2^-27 of the running maximum
  // (typical scale 2^-5); weights overflow from scale_v = 16 on, a value row with a range above 4080.
  constexpr float kWeightUp = FULL ? 256.0f : 16.0f;
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* ring = smem;
  float* mail = reinterpret_cast<float*>(smem + C::kRing);
  unsigned char* xchg = smem + C::kRing + C::kMailBytes;
  float* lz = reinterpret_cast<float*>(xchg + C::kXchgBytes);
  unsigned char* qf_s = xchg + C::kXchgBytes + C::kLzBytes;   // [nt][plane][wd][lane] uint2, then qs[col]
  float* qs_s = reinterpret_cast<float*>(qf_s + NT * 2 * 4 * 32 * 8);
  __nv_bfloat16* q_s = reinterpret_cast<__nv_bfloat16*>(xchg + C::kXchgBytes + C::kLzBytes + C::kQfBytes);
  uint32_t* blk_s = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(q_s) + C::kQBytes);
  int4* info_s = reinterpret_cast<int4*>(reinterpret_cast<unsigned char*>(blk_s) + C::kBlkBytes);
  Item* items = reinterpret_cast<Item*>(info_s + NSTAGE);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(info_s) + C::kInfoBytes);
  int* misc = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(bars) + C::kBarBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x;
  const uint32_t ring_u32 = smem_u32(ring);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + NSTAGE * 8;
  const uint32_t qfull0 = empty0 + NSTAGE * 8, qempty0 = qfull0 + 16;
  volatile int* abort_word = misc;

  if (tid == 0) {
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(full0 + i * 8, 1);
      mbar_init(empty0 + i * 8, C::kConsWarps);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(qfull0 + i * 8, 1);
      mbar_init(qempty0 + i * 8, C::kConsWarps);
    }
    misc[0] = 0; misc[1] = 0; misc[7] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < C::kQBytes / 16; i += C::kThreads) reinterpret_cast<uint4*>(q_s)[i] = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  if (warp == C::kConsWarps) {
    producer_warp<C, FULL, TW, NSTAGE>(p, lane, ring_u32, full0, empty0, qfull0, qempty0, q_s, blk_s,
                                       info_s, items, misc, abort_word);
    return;
  }
  __syncthreads();  // (A)
  const int n_units = misc[7];
  if (n_units == 0) return;

  // per-warp exchange area: [flag (16 B)] [column maxima: kColsPad floats] [P^T: NT x 2 x 32 words]
  constexpr int kXW = 16 + C::kColsPad * 4 + NT * 4 * 32 * 4;
  const int g = lane >> 2, t = lane & 3;
  const int team = warp / DS, d = warp % DS;
  const float cb = p.sm_log2;
  // m holds MINUS the running maximum inside the stage loop (it enters the score FMA directly)
  // The tensor core truncates when it adds into its FP32 accumulators: every MMA loses half a unit
  // in the last place of the accumulator on average, about 0.4 * 2^-23 of its value (measured; mantissas spread
  // log-uniformly).  Over the thousands of MMAs of a long piece that is a relative bias of some
  // 1e-4 on the uncentred level sums, which are large against the outputs they cancel into.  The
  // MMAs into each accumulator are counted and the expected loss is put back at the end of a piece.
  // The estimate is good to some 30 %, which is not enough for the longest chains (a CTA that
  // works through a whole 131072-token head adds 16 000 MMAs into an accumulator) on rows whose
  // level sums are a hundred times their outputs.  So the chains are cut: every kFlushMmas MMAs the
  // accumulators are added in FP32 (round to nearest, by the L2's reduction unit: no load, nothing
  // to wait for) into a copy of the O slice in the workspace and start again from zero.  Without
  // that part of the workspace (see lynx_workspace_bytes) the chains are not cut.
  constexpr float kTruncPerMma = 0.40f * 1.1920929e-7f;
  constexpr int kFlushMmas = 1024;
  int n_mma = 0;          // MMAs into each accumulator since the last flush
  bool flushed = false;   // the copy holds earlier parts of this piece
  float* shadow = p.ws_shadow == nullptr ? nullptr
      : p.ws_shadow + ((size_t)cta * C::kConsWarps + warp) * (NT * MT * 4 * 32) + lane;
  float m[NT][2], l[NT][2], zs[NT][2], o[NT][MT][4];
  const uint32_t qf_u32 = smem_u32(qf_s), qs_u32 = smem_u32(qs_s);
  auto col_limit = [&](int col, int len_) {
    if (PACK) col &= 3;
    return col < p.ncols ? (p.causal ? len_ - p.nq + col / p.G + 1 : len_) : 0;
  };
  bool fresh = true;
  float ca = 0.0f;
  int len = 0, full_lim = 0, ic = 0;
  Item item;
  item.b = 0; item.hkv = 0; item.len = 0; item.first_cta = 0; item.n_contrib = 1;

  for (int gs = 0; gs < n_units; ++gs) {
    const int slot = gs % NSTAGE;
    mbar_wait(full0 + slot * 8, (gs / NSTAGE) & 1, abort_word);
    const int4 info = info_s[slot];
    if (info.z & 1) {
      const int qi = info.x & 1;
      mbar_wait(qfull0 + qi * 8, (ic >> 1) & 1, abort_word);
      item = items[qi];
      len = item.len;
      full_lim = p.causal ? len - p.nq + 1 : len;
      const __nv_bfloat16* qb = q_s + (size_t)qi * C::kColsPad * LYNX_D;
      float amax = 0.0f;
      for (int i = lane; i < C::kColsPad * (LYNX_D / 8); i += 32) {
        const uint4 v = reinterpret_cast<const uint4*>(qb)[i];
        const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          amax = fmaxf(amax, fabsf(__uint_as_float(ww[k] << 16)));
          amax = fmaxf(amax, fabsf(__uint_as_float(ww[k] & 0xFFFF0000u)));
        }
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, off));
      // two balanced s8 digit planes of q: q_int = rint(q * 2^e) = 256 * hi + lo, |q_int| < 2^15
      int e = 0;
      if (amax > 0.0f && amax < INFINITY) e = 14 - (((__float_as_int(amax) >> 23) & 0xFF) - 127);
      e = max(-100, min(100, e));
      const float up = __int_as_float((127 + e) << 23), down = __int_as_float((127 - e) << 23);
      ca = p.sm_log2 * down * (FULL ? 1.0f : 16.0f);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        // warp w builds the shared fragments of the n-tiles nt = w, w + (consumer warps), ... for everybody
        const bool mine = (nt % C::kConsWarps) == warp;
        if (mine) {
          const int c = PACK ? (g & 3) : nt * 8 + g;
#pragma unroll
          for (int wd = 0; wd < 4; ++wd) {
            const uint4 v = *reinterpret_cast<const uint4*>(qb + c * LYNX_D + 32 * t + 8 * wd);
            const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
            int qv[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              // (32640, the largest BF16 mantissa at the top exponent, would need hi = 128)
              qv[2 * k] = min(__float2int_rn(__uint_as_float(ww[k] << 16) * up), 32639);
              qv[2 * k + 1] = min(__float2int_rn(__uint_as_float(ww[k] & 0xFFFF0000u) * up), 32639);
            }
            uint32_t hi_e = 0, hi_o = 0, lo_e = 0, lo_o = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int he = (qv[2 * k] + 128) >> 8, ho = (qv[2 * k + 1] + 128) >> 8;   // lo in [-128, 127]
              hi_e |= (uint32_t)(he & 0xFF) << (8 * k);
              lo_e |= (uint32_t)((qv[2 * k] - (he << 8)) & 0xFF) << (8 * k);
              hi_o |= (uint32_t)(ho & 0xFF) << (8 * k);
              lo_o |= (uint32_t)((qv[2 * k + 1] - (ho << 8)) & 0xFF) << (8 * k);
            }
            reinterpret_cast<uint2*>(qf_s)[((nt * 2 + 0) * 4 + wd) * 32 + lane] = make_uint2(hi_e, hi_o);
            reinterpret_cast<uint2*>(qf_s)[((nt * 2 + 1) * 4 + wd) * 32 + lane] = make_uint2(lo_e, lo_o);
          }
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int col = nt * 8 + 2 * t + cc;
            const uint4* qq = reinterpret_cast<const uint4*>(qb + (PACK ? (col & 3) : col) * LYNX_D + 16 * g);
            float sum = 0.0f;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const uint4 v = qq[h];
              const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int k = 0; k < 4; ++k)
                sum += __uint_as_float(ww[k] << 16) + __uint_as_float(ww[k] & 0xFFFF0000u);
            }
            sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 4);
            sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 8);
            sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 16);
            if (g == 0) qs_s[col] = sum;
          }
        }
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          m[nt][cc] = 0.0f; l[nt][cc] = 0.0f; zs[nt][cc] = 0.0f;
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int i = 0; i < 4; ++i) o[nt][mt][i] = 0.0f;
      }
      named_bar(1, C::kConsThreads);  // the shared fragments are complete
      fresh = true;
      n_mma = 0;
      flushed = false;
    }

    const uint32_t st = ring_u32 + slot * C::kStageBytes;
    const int unit_t0 = info.y * ST;
#pragma unroll
    for (int tp = 0; tp < TPW; ++tp) {   // the tiles of this warp in the stage
    const int wt = warp + tp * C::kConsWarps;
    const int tile_t0 = unit_t0 + wt * 16;
    const bool in_range = tile_t0 < len;                          // this warp's own tile
    const bool team_valid = unit_t0 + (DS == 1 ? wt : team * DS) * 16 < len;   // the team's first tile
    if (DS > 1 || in_range) {  // a lone warp (DS == 1) has nothing to do for a tile beyond the end
    const bool valid = DS == 1 ? true : in_range;
    unsigned char* my_x = xchg + (size_t)warp * kXW;
    float s[NT][4];
    float cmx[DS > 1 ? 1 : NT][2];  // column maxima of this tile (kept in registers when DS == 1)
    float2 vm_lo = make_float2(0.f, 0.f), vm_hi = make_float2(0.f, 0.f);
    const int r0 = wt * 16 + pi_row(g);
    const int tok_lo = tile_t0 + pi_row(g), tok_hi = tok_lo + 8;
    const bool masked = tile_t0 + 16 > full_lim;
    // ---- phase A: scores of this warp's tile, growth vote -------------------------------
    bool gw = false;
    if (valid) {
      {
        uint32_t a[4][4];
        k_fragments<FULL, ST>(st, r0, t, a);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          int shi[4] = {0, 0, 0, 0}, slo[4] = {0, 0, 0, 0};
#pragma unroll
          for (int wd = 0; wd < 4; ++wd) {
            const uint2 bh = lds64(qf_u32 + (((nt * 2 + 0) * 4 + wd) * 32 + lane) * 8);
            const uint2 bl = lds64(qf_u32 + (((nt * 2 + 1) * 4 + wd) * 32 + lane) * 8);
            mma_u8s8(shi, a[wd][0], a[wd][1], a[wd][2], a[wd][3], bh.x, bh.y);
            mma_u8s8(slo, a[wd][0], a[wd][1], a[wd][2], a[wd][3], bl.x, bl.y);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) s[nt][i] = (float)(shi[i] * 256 + slo[i]);
        }
      }
      float2 km_lo = lds64f(st + KM + r0 * 8), km_hi = lds64f(st + KM + (r0 + 8) * 8);
      vm_lo = lds64f(st + VM + r0 * 8); vm_hi = lds64f(st + VM + (r0 + 8) * 8);
      if (masked) {
        int maxlim = 0;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
          maxlim = max(maxlim, max(col_limit(nt * 8 + 2 * t, len), col_limit(nt * 8 + 2 * t + 1, len)));
        maxlim = max(maxlim, __shfl_xor_sync(0xFFFFFFFFu, maxlim, 1));
        maxlim = max(maxlim, __shfl_xor_sync(0xFFFFFFFFu, maxlim, 2));
        if (tok_lo >= maxlim) { km_lo = make_float2(0.f, 0.f); vm_lo = make_float2(0.f, 0.f); }
        if (tok_hi >= maxlim) { km_hi = make_float2(0.f, 0.f); vm_hi = make_float2(0.f, 0.f); }
      }
      const float al_lo = km_lo.x * ca, al_hi = km_hi.x * ca;
      const float be_lo = fmaf(km_lo.x, kMidK, km_lo.y) * cb, be_hi = fmaf(km_hi.x, kMidK, km_hi.y) * cb;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const float2 qq = lds64f(qs_u32 + (nt * 8 + 2 * t) * 4);
        const float q0 = qq.x, q1 = qq.y;
        {  // score - max for the lane's 2 rows x 2 columns, two lanes of FP32 per instruction
          const uint64_t qq2 = pk2(q0, q1), nm2 = pk2(m[nt][0], m[nt][1]);  // m = minus the maximum
          const uint64_t lo2 = ffma2(pk2(al_lo, al_lo), pk2(s[nt][0], s[nt][1]), ffma2(pk2(be_lo, be_lo), qq2, nm2));
          const uint64_t hi2 = ffma2(pk2(al_hi, al_hi), pk2(s[nt][2], s[nt][3]), ffma2(pk2(be_hi, be_hi), qq2, nm2));
          upk2(lo2, s[nt][0], s[nt][1]);
          upk2(hi2, s[nt][2], s[nt][3]);
        }
        if (masked) {
          const int l0 = col_limit(nt * 8 + 2 * t, len), l1 = col_limit(nt * 8 + 2 * t + 1, len);
          if (tok_lo >= l0) s[nt][0] = -INFINITY;
          if (tok_lo >= l1) s[nt][1] = -INFINITY;
          if (tok_hi >= l0) s[nt][2] = -INFINITY;
          if (tok_hi >= l1) s[nt][3] = -INFINITY;
        }
        gw |= fmaxf(fmaxf(s[nt][0], s[nt][2]), fmaxf(s[nt][1], s[nt][3])) > 4.0f;
      }
      gw = __any_sync(0xFFFFFFFFu, gw) || fresh;
      if (gw) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            float mx = fmaxf(s[nt][cc], s[nt][cc + 2]);
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 16));
            if constexpr (DS > 1) {
              if (g == 0) reinterpret_cast<float*>(my_x + 16)[nt * 8 + 2 * t + cc] = mx;
            } else {
              cmx[nt][cc] = mx;
            }
          }
      }
    }
    if constexpr (DS > 1) {
      if (lane == 0) *reinterpret_cast<int*>(my_x) = gw ? 1 : 0;
      named_bar(2 + team, DS * 32);
    }
    // ---- agree on the running maxima ----------------------------------------------------
    {
      bool any = gw;
      int flags[DS];
      if constexpr (DS > 1) {
        any = false;
#pragma unroll
        for (int dd = 0; dd < DS; ++dd) {
          flags[dd] = *reinterpret_cast<const volatile int*>(xchg + (size_t)(team * DS + dd) * kXW);
          any |= flags[dd] != 0;
        }
      }
      if (any) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            float mx = -INFINITY;
            if constexpr (DS > 1) {
#pragma unroll
              for (int dd = 0; dd < DS; ++dd)
                if (flags[dd])
                  mx = fmaxf(mx, reinterpret_cast<const volatile float*>(xchg + (size_t)(team * DS + dd) * kXW + 16)[nt * 8 + 2 * t + cc]);
            } else {
              mx = cmx[nt][cc];
            }
            const float up = fresh ? fmaxf(mx, -1.0e4f) : fmaxf(mx, 0.0f);
            const float f = fresh ? 0.0f : ex2(-up);
            m[nt][cc] -= up;  // minus the maximum
            s[nt][cc] -= up;
            s[nt][cc + 2] -= up;
            l[nt][cc] *= f;
            zs[nt][cc] *= f;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              o[nt][mt][cc] *= f;
              o[nt][mt][cc + 2] *= f;
              if (flushed) {   // rare: the copy follows the new maximum
                float* s0 = shadow + ((nt * MT + mt) * 4 + cc) * 32;
                __stcg(s0, __ldcg(s0) * f);
                __stcg(s0 + 64, __ldcg(s0 + 64) * f);
              }
            }
          }
      }
      if (team_valid) fresh = false;
    }
    // ---- weights of this warp's tile, P^T fragments to shared memory ---------------------
    uint32_t pown[DS > 1 ? 1 : NT][4];  // P^T fragments of the own tile (DS == 1): rounded weights, remainders
    if (valid) {
      const float sv_lo = vm_lo.x * (kLevelScaleV * kWeightUp), sv_hi = vm_hi.x * (kLevelScaleV * kWeightUp);
      const float zv_lo = fmaf(vm_lo.x, kMidV, vm_lo.y), zv_hi = fmaf(vm_hi.x, kMidV, vm_hi.y);
      uint32_t* pf = reinterpret_cast<uint32_t*>(my_x + 16 + C::kColsPad * 4) + lane;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const float p0 = ex2(s[nt][0]), p1 = ex2(s[nt][1]);
        const float p2 = ex2(s[nt][2]), p3 = ex2(s[nt][3]);
        const uint64_t plo = pk2(p0, p1), phi = pk2(p2, p3);
        upk2(fadd2(pk2(l[nt][0], l[nt][1]), fadd2(plo, phi)), l[nt][0], l[nt][1]);
        upk2(ffma2(plo, pk2(zv_lo, zv_lo), ffma2(phi, pk2(zv_hi, zv_hi), pk2(zs[nt][0], zs[nt][1]))),
             zs[nt][0], zs[nt][1]);
        float w0, w1, w2, w3;
        upk2(fmul2(plo, pk2(sv_lo, sv_lo)), w0, w1);
        upk2(fmul2(phi, pk2(sv_hi, sv_hi)), w2, w3);
        // w = h + r: h the FP16 rounding of w, r its remainder (exact in FP32, rounded to FP16)
        const uint32_t h01 = pack_f16x2(w0, w1), h23 = pack_f16x2(w2, w3);
        float b0, b1, b2, b3;
        unpack_f16x2(h01, b0, b1);
        unpack_f16x2(h23, b2, b3);
        const uint32_t r01 = pack_f16x2(w0 - b0, w1 - b1), r23 = pack_f16x2(w2 - b2, w3 - b3);
        if constexpr (PACK) {   // columns 0..3: the rounded weights; their repeats 4..7: the remainders
          pown[nt][0] = movmatrix_trans(t >= 2 ? r01 : h01);
          pown[nt][1] = movmatrix_trans(t >= 2 ? r23 : h23);
          pown[nt][2] = 0u; pown[nt][3] = 0u;
          continue;
        }
        const uint32_t f0 = movmatrix_trans(h01), f1 = movmatrix_trans(h23);
        const uint32_t f2 = movmatrix_trans(r01), f3 = movmatrix_trans(r23);
        if constexpr (DS > 1) {
          pf[(nt * 4 + 0) * 32] = f0;
          pf[(nt * 4 + 1) * 32] = f1;
          pf[(nt * 4 + 2) * 32] = f2;
          pf[(nt * 4 + 3) * 32] = f3;
        } else {
          pown[nt][0] = f0; pown[nt][1] = f1; pown[nt][2] = f2; pown[nt][3] = f3;
        }
      }
    }
    if constexpr (DS > 1) named_bar(2 + team, DS * 32);
    // ---- phase C: P.V of the team's tiles for this warp's slice of the output dims --------
    if constexpr (DS == 1) {
      if (valid) {
        pv_slice<FULL, NT, ST, 1, !PACK>(o, st, wt * 16, g, t, 0, pown);
        n_mma += PACK ? 1 : 2;   // into every accumulator: the rounded weights and their remainders
      }
    }
#pragma unroll
    for (int tau = 0; tau < (DS > 1 ? DS : 0); ++tau) {
      const int src = team * DS + tau;
      if (unit_t0 + src * 16 >= len) break;  // uniform: later tiles of the unit are beyond len too
      uint32_t pb[NT][4];
      const uint32_t* pf = reinterpret_cast<const uint32_t*>(xchg + (size_t)src * kXW + 16 + C::kColsPad * 4) + lane;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int i = 0; i < 4; ++i) pb[nt][i] = *reinterpret_cast<const volatile uint32_t*>(pf + (nt * 4 + i) * 32);
      }
      pv_slice<FULL, NT, ST, DS, true>(o, st, src * 16, g, t, d, pb);
      n_mma += 2;
    }
    }  // if (DS > 1 || in_range)
    }  // tiles of this warp
    if (shadow != nullptr && n_mma >= kFlushMmas) {   // uniform over the warp
      const float back = 1.0f + (float)n_mma * kTruncPerMma;   // the expected truncation loss, put back
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float* sh = shadow + ((nt * MT + mt) * 4 + i) * 32;
            const float v = o[nt][mt][i] * back;
            if (flushed) atomicAdd(sh, v); else __stcg(sh, v);
            o[nt][mt][i] = 0.0f;
          }
      flushed = true;
      n_mma = 0;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty0 + slot * 8);
    if (!(info.z & 2)) continue;

    // ---- end of the piece -----------------------------------------------------------------
    {
      const float back = 1.0f + (float)n_mma * kTruncPerMma;   // the expected truncation loss, put back
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            o[nt][mt][i] *= back;
            if (flushed) o[nt][mt][i] += __ldcg(shadow + ((nt * MT + mt) * 4 + i) * 32);
            // the remainders' part, accumulated under the repeated columns, joins its column
            if (PACK) o[nt][mt][i] += __shfl_xor_sync(0xFFFFFFFFu, o[nt][mt][i], 2);
          }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { m[nt][0] = -m[nt][0]; m[nt][1] = -m[nt][1]; }  // back to the maximum
    if (fresh) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) m[nt][0] = m[nt][1] = -1.0e30f;
    }
    // teams 1.. are absorbed into team 0, slice by slice, through lane-private mailboxes
    for (int src = 1; src < TEAMS; ++src) {
      for (int dd = 0; dd < DS; ++dd) {
        float* box = mail + lane;
        if (team == src && d == dd) {
          int r = 0;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
              for (int i = 0; i < 4; ++i) box[(r++) * 32] = o[nt][mt][i];
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              box[(r++) * 32] = m[nt][cc];
              box[(r++) * 32] = l[nt][cc];
              box[(r++) * 32] = zs[nt][cc];
            }
          }
        }
        named_bar(1, C::kConsThreads);
        if (team == 0 && d == dd) {
          int r = 0;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            float f1[2], f2[2];
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              const float m2 = box[((MT * 4 + 6) * nt + MT * 4 + 3 * cc) * 32];
              const float M = fmaxf(m[nt][cc], m2);
              f1[cc] = ex2(m[nt][cc] - M);
              f2[cc] = ex2(m2 - M);
              m[nt][cc] = M;
            }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float o2 = box[(r++) * 32];
                o[nt][mt][i] = o[nt][mt][i] * f1[i & 1] + o2 * f2[i & 1];
              }
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              r++;
              const float l2 = box[(r++) * 32];
              const float z2 = box[(r++) * 32];
              l[nt][cc] = l[nt][cc] * f1[cc] + l2 * f2[cc];
              zs[nt][cc] = zs[nt][cc] * f1[cc] + z2 * f2[cc];
            }
          }
        }
        named_bar(1, C::kConsThreads);
      }
    }
    // team 0: totals of l and zs over its DS warps (each saw different tokens)
    if (team == 0) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          float lv = l[nt][cc], z = zs[nt][cc];
#pragma unroll
          for (int off = 4; off <= 16; off <<= 1) {
            lv += __shfl_xor_sync(0xFFFFFFFFu, lv, off);
            z += __shfl_xor_sync(0xFFFFFFFFu, z, off);
          }
          if (g == 0)
            *reinterpret_cast<float2*>(lz + ((size_t)d * C::kColsPad + nt * 8 + 2 * t + cc) * 2) = make_float2(lv, z);
        }
    }
    named_bar(1, C::kConsThreads);
    const bool direct = item.n_contrib == 1;
    if (team == 0) {
      const size_t bh = (size_t)item.b * p.Hkv + item.hkv;
      float* part = p.ws_part + (bh + (size_t)cta) * (size_t)C::kColsPad * kPartStride;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int c = nt * 8 + 2 * t + cc;
          float lt = 0.0f, z = 0.0f;
#pragma unroll
          for (int dd = 0; dd < DS; ++dd) {
            const float2 v = *reinterpret_cast<const float2*>(lz + ((size_t)dd * C::kColsPad + c) * 2);
            lt += v.x; z += v.y;
          }
          if (c >= p.ncols) continue;
          const int j = c / p.G, hh = c % p.G;
          float* dst = direct ? p.out + (((size_t)item.b * p.nq + j) * p.Hq + item.hkv * p.G + hh) * LYNX_D
                              : part + (size_t)c * kPartStride;
          const float inv = direct ? (lt > 0.0f ? 1.0f / lt : 0.0f) : 1.0f;
          // undo the subnormal scales of the V operands (2^-24; odd dims of the anchor 2^-20) and kWeightUp
          constexpr float fix_even = 16777216.0f / kWeightUp, fix_odd = (FULL ? 16777216.0f : 1048576.0f) / kWeightUp;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const int gmt = d * MT + mt;  // m-tile index among the eight of a lane's 16 dims
            const int dim = 16 * g + 8 * (gmt >> 2) + 2 * (gmt & 3);
            *reinterpret_cast<float2*>(dst + dim) =
                make_float2(fmaf(o[nt][mt][cc], fix_even, z) * inv, fmaf(o[nt][mt][cc + 2], fix_odd, z) * inv);
          }
          if (!direct && d == 0 && g == 0) { dst[128] = m[nt][cc]; dst[129] = lt; }
        }
      }
      __threadfence();
    }
    finish_piece<FULL, C::kColsPad, C::kConsThreads>(p, item, direct, tid, misc);
    __syncwarp();
    if (lane == 0) mbar_arrive(qempty0 + (info.x & 1) * 8);
    ++ic;
  }
  if (tid == 0 && misc[0]) atomicOr(p.ws_flags, kFlagTimeout);
}

// At least MINB CTAs per SM (the compiler caps registers accordingly).  Nine warps cannot
// have more than 168 registers each: three of them share one SM sub-partition's 16 K registers.
template <bool FULL, int NT, int DS, int TEAMS, int NSTAGE, int MINB, int TPW, bool PACK>
__global__ void __launch_bounds__((DS * TEAMS + 1) * 32, MINB)
attn_team_kernel(const AttnParams p) {
  attn_team_body<FULL, NT, DS, TEAMS, NSTAGE, TPW, PACK>(p);
}
#ifndef LYNX_WIDE_VERIFY
#define LYNX_WIDE_VERIFY 2   // comparison builds: 1 = mma.sync kernel for 17..32 verify columns, 0 = for 33..64 too
#endif
#include "attention_wide.cuh"
#include "attention_i8.cuh"

// ------------------------------------------------------------------ host side
constexpr int kMaxCtasPerSm = 4;

struct Plan {
  int ncols, variant;  // variant: 0: NT1 TW4 CG1; 1: NT2 TW4 CG1; 2: NT2 TW4 CG2; 3: NT2 TW2 CG4
  int cols_pad;
  size_t off_chunk_ctr, off_seq_ctr, off_group_ctr, off_dev, off_part, bytes;
  size_t shadow_bytes;   // optional tail of the workspace: FP32 copies of the accumulators (see kFlushMmas)
};

bool make_plan(const lynx_shape* s, int B, int nq, Plan* pl) {
  if (!s || s->head_dim != LYNX_D || s->num_kv_heads <= 0 || s->num_q_heads <= 0 ||
      s->num_q_heads % s->num_kv_heads != 0 || s->block_tokens <= 0 || s->block_tokens % 16 != 0 ||
      s->num_blocks <= 0 || s->max_blocks_per_seq <= 0 || B <= 0 || nq <= 0 || nq > kMaxQ)
    return false;
  const int G = s->num_q_heads / s->num_kv_heads;
  const int ncols = nq * G;
  if (ncols > kMaxCols) return false;
  const int64_t cap = (int64_t)s->max_blocks_per_seq * s->block_tokens;
  if (cap >= (1ll << 31)) return false;
  if ((int64_t)s->num_blocks * s->num_kv_heads * s->block_tokens >= (1ll << 32)) return false;
  pl->ncols = ncols;
  pl->variant = ncols <= 8 ? 0 : ncols <= 16 ? 1 : ncols <= 32 ? 2 : 3;
  pl->cols_pad = ncols <= 8 ? 8 : ncols <= 16 ? 16 : ncols <= 32 ? 32 : 64;
  size_t off = kWsHeaderBytes;
  pl->off_chunk_ctr = off; off += (size_t)B * s->num_kv_heads * 4;
  pl->off_seq_ctr = off;   off += (size_t)B * 4;
  pl->off_group_ctr = off; off += (size_t)2 * sm_count() * kMaxCtasPerSm * 4;
  off = (off + 255) & ~(size_t)255;
  pl->off_dev = off;       off += (size_t)B * s->num_kv_heads * kMaxQ * 4;
  off = (off + 255) & ~(size_t)255;
  pl->off_part = off;
  off += ((size_t)B * s->num_kv_heads + (size_t)sm_count() * kMaxCtasPerSm) * pl->cols_pad * kPartStride * 4;
  pl->bytes = (off + 255) & ~(size_t)255;
  // mma.sync kernels: one O slice per consumer warp, 16 KB per CTA (64 KB with 64 columns, one CTA per
  // SM); tcgen05 kernels: 2 groups x 128 rows x 128 dims per CTA
  pl->shadow_bytes = (size_t)sm_count() * (ncols > 16 && ncols <= 64 ? 131072 : kMaxCtasPerSm * 16384);
  if (pl->shadow_bytes < (size_t)sm_count() * kMaxCtasPerSm * 16384) pl->shadow_bytes = (size_t)sm_count() * kMaxCtasPerSm * 16384;
  return true;
}

template <bool FULL, int NT, int DS, int TEAMS, int NSTAGE, int MINB, int TPW = 1, bool PACK = false>
lynx_status launch_team(const AttnParams& p, cudaStream_t st) {
  using C = TeamCfg<FULL, NT, DS, TEAMS, NSTAGE, TPW>;
  static_assert(MINB <= kMaxCtasPerSm, "partial slots are sized for kMaxCtasPerSm CTAs per SM");
  constexpr int kCtasPerSm = MINB;
  static_assert(kCtasPerSm * (C::kSmem + 1024) <= 228 * 1024, "shared memory budget per SM");
  static_assert(2 + TEAMS <= 16, "named barriers");
  auto kern = attn_team_kernel<FULL, NT, DS, TEAMS, NSTAGE, MINB, TPW, PACK>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmem) != cudaSuccess)
      return LYNX_ERR_CUDA;
    configured[dev] = true;
  }
  // small problems: no more CTAs than ranges of at least 8 stage-units (an upper bound from the
  // table capacity: the lengths live on the device)
  const long long cap_units = (long long)p.B * p.Hkv * (((long long)p.max_blocks * p.bt + C::kST - 1) / C::kST);
  long long grid = (cap_units + 7) / 8;
  const long long full = (long long)sm_count() * kCtasPerSm;
  grid = grid < 1 ? 1 : (grid > full ? full : grid);
  kern<<<(unsigned)grid, C::kThreads, C::kSmem, st>>>(p);
  return launch_status();
}

lynx_status run_attention(bool full, const lynx_shape* shape, const void* q, int B, int nq, int causal,
                          lynx_plane K, lynx_plane V, const int32_t* block_table,
                          const int32_t* seq_lens, float softmax_scale, const float* draft,
                          float atol, float rtol, float* out, int32_t* first_reject, float* dev,
                          void* workspace, size_t workspace_bytes, void* stream) {
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
  if (workspace_bytes < pl.bytes) return LYNX_ERR_WORKSPACE;
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
  p.ws_shadow = workspace_bytes >= pl.bytes + pl.shadow_bytes ? reinterpret_cast<float*>(ws + pl.bytes) : nullptr;
  p.ws_dev = reinterpret_cast<float*>(ws + pl.off_dev);
  p.ws_part = reinterpret_cast<float*>(ws + pl.off_part);
  p.atol = atol; p.rtol = rtol;
  const float sc = softmax_scale == 0.0f ? 0.08838834764831845f : softmax_scale;
  p.sm_log2 = sc * 1.4426950408889634f;
  p.B = B; p.nq = nq; p.causal = causal ? 1 : 0;
  p.Hq = shape->num_q_heads; p.Hkv = shape->num_kv_heads; p.G = p.Hq / p.Hkv;
  p.bt = shape->block_tokens; p.num_blocks = shape->num_blocks; p.max_blocks = shape->max_blocks_per_seq;
  p.ncols = pl.ncols;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // up to 32 columns: the integer tcgen05 kernels
  if (pl.ncols <= 32) {
    if (!full) {
      if (pl.ncols <= 4) return launch_i8<false, 4>(p, st);
      if (pl.ncols <= 8) return launch_i8<false, 8>(p, st);
      if (pl.ncols <= 16) return launch_i8<false, 16>(p, st);
      return launch_i8<false, 32>(p, st);
    }
    if (pl.ncols <= 4) return launch_i8<true, 4>(p, st);
    if (pl.ncols <= 8) return launch_i8<true, 8>(p, st);
    if (pl.ncols <= 16) return launch_i8<true, 16>(p, st);
    return launch_i8<true, 32>(p, st);
  }
  // <FULL, NT, DS, TEAMS, stages, CTAs/SM>
  if (!full) {
    switch (pl.variant) {
      case 0:   // two tiles per warp and stage
        if (pl.ncols <= 4) return launch_team<false, 1, 1, 4, 2, 4, 2, true>(p, st);
        return launch_team<false, 1, 1, 4, 2, 4, 2>(p, st);
      case 1: return launch_team<false, 2, 2, 2, 4, 3>(p, st);
      case 2: return launch_team<false, 4, 4, 1, 3, 3>(p, st);
      default: return launch_team<false, 8, 4, 2, 3, 1>(p, st);
    }
  }
  switch (pl.variant) {
    case 0:
      if (pl.ncols <= 4) return launch_team<true, 1, 1, 4, 3, 3, 1, true>(p, st);
      return launch_team<true, 1, 1, 4, 3, 3>(p, st);
    case 1: return launch_team<true, 2, 2, 2, 3, 3>(p, st);
    // 17..64 columns: tcgen05.  (The mma.sync kernels for them are built in comparison builds only.)
#if LYNX_WIDE_VERIFY > 1
    case 2: return launch_wide<2, 2>(p, st);
#else
    case 2: return launch_team<true, 4, 4, 1, 2, 3>(p, st);
#endif
#if LYNX_WIDE_VERIFY
    default: return launch_wide<2, 1>(p, st);
#else
    default: return launch_team<true, 8, 4, 2, 3, 1>(p, st);
#endif
  }
}

}  // namespace
}  // namespace lynx

extern "C" size_t lynx_workspace_bytes(const lynx_shape* shape, int32_t batch, int32_t n_cols_q) {
  lynx::Plan pl;
  if (!lynx::make_plan(shape, batch, n_cols_q, &pl)) return 0;
  return pl.bytes + pl.shadow_bytes;
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
  // the array keeps what the previous call left: the status word and the tickets must be zero
  if (cudaMemsetAsync(scratch, 0, pl.off_dev, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return LYNX_ERR_CUDA;
  return run_attention(false, shape, q_bf16, batch, n_q, causal, K, V, block_table, seq_lens,
                       softmax_scale, nullptr, 0.f, 0.f, out, nullptr, nullptr, scratch,
                       kStaticScratchBytes, stream);
}
