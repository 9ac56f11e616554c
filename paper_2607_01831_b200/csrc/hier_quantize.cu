// lynx_hier_quantize / lynx_hier_dequantize: the paper's own quantiser, Algorithm 1 "Lynx Hierarchical
// Quantization" (Section 4.1), and its inverse (the inverse alpha-law of stage 3), on sm_100a.
//
// A page is P = 256 consecutive tokens of one KV head, 128 channels each, BF16, contiguous
// ([n_pages][256][128]).  Every channel is treated on its own: stage 1 normalises it by its minimum
// and range over the page, stage 2 centres and scales every chunk of C = 32 consecutive tokens by the
// chunk's mean and largest deviation, stage 3 compands the magnitudes with the alpha-law to integers,
// stage 4 splits them into a 4-bit Anchor (sign-aware two's complement) and a 4-bit centred Residual.
// Constants and readings (alpha = 255, epsilon = 1e-6, magnitude scale 120, Sign of the centred value,
// round to nearest even) are those of the CPU oracle; arithmetic here is binary32.
//
// One CTA per page: the page (64 KB) is staged in shared memory once, the statistics are computed
// from there by channel pairs (a 32-bit word holds two channels of a token: conflict-free column
// walks), the codes leave as packed nibbles, byte j of a token row = channel 2j | channel 2j+1 << 4,
// the same packing as the linear planes.  HBM-bound by construction (64 KB read, 32 KB + 9 KB written
// per page), with ~25 ALU operations per element on top.
#include <cuda_bf16.h>

#include "lynx_common.cuh"

namespace lynx {
namespace {

constexpr int kP = 256, kC = 32, kChunks = kP / kC;
constexpr float kAlpha = 255.0f, kEps = 1.0e-6f, kYmax = 120.0f;
constexpr float kLog2_1pAlpha = 8.0f;            // log2(1 + 255)

__device__ __forceinline__ float lo_bf16(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_bf16(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t lop3_sel(uint32_t a, uint32_t b, uint32_t mask) {   // (a & mask) | (b & ~mask)
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(d) : "r"(mask), "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf2_min(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf2_max(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float rcp_fast(float x) {
  float r;
  asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ void cp_async16(uint32_t saddr, const void* g) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(saddr), "l"(g) : "memory");
}

// Stages 3 and 4 for the two channels of a word (packed FP32 pairs): x_final = (x - mean) * A (stages 1 and 2
// folded: the difference first, which is exact where it is small; one multiply-add x * A - mean * A would carry the
// rounding of mean * A, a large error for a channel whose offset dwarfs its chunk deviation), the alpha-law magnitude
// y = log2(1 + 255 |x_final|) * 15 rounded to the nearest even integer I (0..120) by the magic-number
// addition, whose sum keeps the integer in its low mantissa bits; the magic number carries the +7 of stage 4,
// so the low byte of r is J = I + 7 (7..127).  t keeps the sign of x_final.
__device__ __forceinline__ void hier_code2(uint32_t w, uint64_t A2, uint64_t M2, uint32_t& r0, uint32_t& r1,
                                           uint32_t& t0, uint32_t& t1) {
  uint64_t d2, t2;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d2) : "l"(pack2(lo_bf16(w), hi_bf16(w))), "l"(M2));
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(t2) : "l"(d2), "l"(A2));
  float f0, f1;
  unpack2(t2, f0, f1);
  float l0, l1;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l0) : "f"(fmaf(kAlpha, fabsf(f0), 1.0f)));
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l1) : "f"(fmaf(kAlpha, fabsf(f1), 1.0f)));
  const uint64_t k2 = pack2(kYmax / kLog2_1pAlpha, kYmax / kLog2_1pAlpha), m2 = pack2(12582919.0f, 12582919.0f);
  const uint64_t r2 = f2_fma(pack2(l0, l1), k2, m2);   // 0x4B400007 + I
  asm("mov.b64 {%0, %1}, %2;" : "=r"(r0), "=r"(r1) : "l"(r2));
  t0 = __float_as_uint(f0);
  t1 = __float_as_uint(f1);
}

// Stage 4 for four channels at once, one byte per channel.  J = I + 7 in the low bytes of r[0..3], the signs in
// the top bytes of t[0..3].  v_mag = J >> 4; the Anchor nibble is v_mag for S = +1 and -v_mag - 1 = ~v_mag for
// S = -1, i.e. bits 4..7 of J ^ (sign mask); the Residual nibble 16 v_mag - I modulo 16 = (7 - J) modulo 16 is
// the low nibble of J ^ 7.  Returned: the nibble pairs of channels (0, 1) in byte 0 and of (2, 3) in byte 2
// (the other bytes are not used); the Residual still lacks its ^ 0x77.
__device__ __forceinline__ void hier_nibbles4(const uint32_t* r, const uint32_t* t, uint32_t& anc, uint32_t& res) {
  const uint32_t J = prmt(prmt(r[0], r[1], 0x0040u), prmt(r[2], r[3], 0x0040u), 0x5410u);
  const uint32_t S = prmt(prmt(t[0], t[1], 0x00FBu), prmt(t[2], t[3], 0x00FBu), 0x5410u);   // 0xFF where negative
  const uint32_t X = J ^ S;
  anc = lop3_sel(X >> 4, X >> 8, 0x000F000Fu);
  res = lop3_sel(J, J >> 4, 0x000F000Fu);
}

// One CTA per page: the page (64 KB) is staged in shared memory by asynchronous 16-byte copies.  A thread owns
// eight channels (four 32-bit words of a token row: 16-byte shared-memory loads, 4-byte plane stores) of half a
// chunk (16 tokens); the two halves of a chunk are lanes l and l ^ 16 of one warp.  First the chunk statistics
// (minimum, maximum as packed BF16 pairs; sums in FP32 pairs), from which the page's minimum and range follow
// (stage 1) and, with them, every chunk's mean and largest deviation (stage 2: max |x - mean| =
// max(max - mean, mean - min)); then the codes.  The reciprocals are split between the two halves of a chunk and
// exchanged by shuffles.
__global__ void __launch_bounds__(256, 3) hier_quantize_kernel(const __nv_bfloat16* __restrict__ src, int n_pages,
                                                               uint8_t* __restrict__ q_anc, uint8_t* __restrict__ q_res,
                                                               float* __restrict__ g_min, float* __restrict__ g_scale,
                                                               float* __restrict__ mu, float* __restrict__ sigma) {
  extern __shared__ __align__(16) unsigned char smem[];
  const uint4* page = reinterpret_cast<const uint4*>(smem);           // [256 tokens][16 quads of channel pairs]
  uint4* c_min = reinterpret_cast<uint4*>(smem + kP * 256);           // [8 chunks][16 quads] packed BF16 pairs
  uint4* c_max = c_min + kChunks * 16;
  const uint32_t page_s = (uint32_t)__cvta_generic_to_shared(smem);
  const int tid = threadIdx.x, q = tid & 15, half = (tid >> 4) & 1, ch = tid >> 5;
  const int row0 = ch * kC + half * (kC / 2);
  for (int pg = blockIdx.x; pg < n_pages; pg += gridDim.x) {
    const uint4* gsrc = reinterpret_cast<const uint4*>(src + (size_t)pg * kP * LYNX_D);
    __syncthreads();                                                  // the previous page is done with shared memory
#pragma unroll 8
    for (int i = tid; i < kP * LYNX_D / 8; i += 256) cp_async16(page_s + (uint32_t)i * 16u, gsrc + i);
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // ---- chunk statistics of the thread's 16 tokens, then of the chunk (both halves) --------------------------
    uint32_t mn[4], mx[4];
    uint64_t sm2[4];
    {
      const uint4 v = page[row0 * 16 + q];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) { mn[j] = w[j]; mx[j] = w[j]; sm2[j] = pack2(lo_bf16(w[j]), hi_bf16(w[j])); }
    }
#pragma unroll 5
    for (int t = 1; t < kC / 2; ++t) {
      const uint4 v = page[(row0 + t) * 16 + q];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mn[j] = bf2_min(mn[j], w[j]);
        mx[j] = bf2_max(mx[j], w[j]);
        sm2[j] = f2_add(sm2[j], pack2(lo_bf16(w[j]), hi_bf16(w[j])));
      }
    }
    float mean[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      mn[j] = bf2_min(mn[j], __shfl_xor_sync(0xFFFFFFFFu, mn[j], 16));
      mx[j] = bf2_max(mx[j], __shfl_xor_sync(0xFFFFFFFFu, mx[j], 16));
      float s0, s1;
      unpack2(sm2[j], s0, s1);
      mean[2 * j] = (s0 + __shfl_xor_sync(0xFFFFFFFFu, s0, 16)) * (1.0f / kC);
      mean[2 * j + 1] = (s1 + __shfl_xor_sync(0xFFFFFFFFu, s1, 16)) * (1.0f / kC);
    }
    if (half == 0) {
      c_min[ch * 16 + q] = make_uint4(mn[0], mn[1], mn[2], mn[3]);
      c_max[ch * 16 + q] = make_uint4(mx[0], mx[1], mx[2], mx[3]);
    }
    __syncthreads();
    // ---- stage 1: the page's minimum and range per channel (each half reduces four chunks) --------------------
    uint32_t pmn[4], pmx[4];
    {
      const uint4 a = c_min[(4 * half) * 16 + q], b = c_max[(4 * half) * 16 + q];
      pmn[0] = a.x; pmn[1] = a.y; pmn[2] = a.z; pmn[3] = a.w;
      pmx[0] = b.x; pmx[1] = b.y; pmx[2] = b.z; pmx[3] = b.w;
#pragma unroll
      for (int c = 1; c < 4; ++c) {
        const uint4 a2 = c_min[(4 * half + c) * 16 + q], b2 = c_max[(4 * half + c) * 16 + q];
        pmn[0] = bf2_min(pmn[0], a2.x); pmn[1] = bf2_min(pmn[1], a2.y);
        pmn[2] = bf2_min(pmn[2], a2.z); pmn[3] = bf2_min(pmn[3], a2.w);
        pmx[0] = bf2_max(pmx[0], b2.x); pmx[1] = bf2_max(pmx[1], b2.y);
        pmx[2] = bf2_max(pmx[2], b2.z); pmx[3] = bf2_max(pmx[3], b2.w);
      }
    }
    float gmn[8], gsc[8], inv[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      pmn[j] = bf2_min(pmn[j], __shfl_xor_sync(0xFFFFFFFFu, pmn[j], 16));
      pmx[j] = bf2_max(pmx[j], __shfl_xor_sync(0xFFFFFFFFu, pmx[j], 16));
      gmn[2 * j] = lo_bf16(pmn[j]);
      gmn[2 * j + 1] = hi_bf16(pmn[j]);
      gsc[2 * j] = lo_bf16(pmx[j]) - gmn[2 * j];
      gsc[2 * j + 1] = hi_bf16(pmx[j]) - gmn[2 * j + 1];
    }
    // reciprocals: this half computes those of channels 4 half .. 4 half + 3, the other half the rest
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float mine = rcp_fast((half ? gsc[4 + i] : gsc[i]) + kEps);
      const float other = __shfl_xor_sync(0xFFFFFFFFu, mine, 16);
      inv[i] = half ? other : mine;
      inv[4 + i] = half ? mine : other;
    }
    if (ch == 0) {
      float* dstp = (half ? g_scale : g_min) + (size_t)pg * LYNX_D + q * 8;
      const float* v = half ? gsc : gmn;
      reinterpret_cast<float4*>(dstp)[0] = make_float4(v[0], v[1], v[2], v[3]);
      reinterpret_cast<float4*>(dstp)[1] = make_float4(v[4], v[5], v[6], v[7]);
    }
    // ---- stage 2 in the page-normalised scale: mean and largest deviation of the chunk -------------------------
    float sg[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      sg[2 * j] = fmaxf(lo_bf16(mx[j]) - mean[2 * j], mean[2 * j] - lo_bf16(mn[j])) * inv[2 * j];
      sg[2 * j + 1] = fmaxf(hi_bf16(mx[j]) - mean[2 * j + 1], mean[2 * j + 1] - hi_bf16(mn[j])) * inv[2 * j + 1];
    }
    {
      float o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] = half ? sg[i] : (mean[i] - gmn[i]) * inv[i];
      float* dstp = (half ? sigma : mu) + ((size_t)pg * kChunks + ch) * LYNX_D + q * 8;
      reinterpret_cast<float4*>(dstp)[0] = make_float4(o[0], o[1], o[2], o[3]);
      reinterpret_cast<float4*>(dstp)[1] = make_float4(o[4], o[5], o[6], o[7]);
    }
    // x_final = ((x - gmin) inv - mu) / (sigma + eps) = (x - mean) * A,  A = inv / (sigma + eps)
    uint64_t A2[4], M2[4];
    {
      float A[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float mine = rcp_fast((half ? sg[4 + i] : sg[i]) + kEps);
        const float other = __shfl_xor_sync(0xFFFFFFFFu, mine, 16);
        A[i] = (half ? other : mine) * inv[i];
        A[4 + i] = (half ? mine : other) * inv[4 + i];
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        A2[j] = pack2(A[2 * j], A[2 * j + 1]);
        M2[j] = pack2(mean[2 * j], mean[2 * j + 1]);
      }
    }
    // ---- stages 3 and 4: the codes of the thread's 16 tokens x 8 channels ---------------------------------------
    uint32_t* pa = reinterpret_cast<uint32_t*>(q_anc + ((size_t)pg * kP + row0) * 64) + q;
    uint32_t* pr_ = reinterpret_cast<uint32_t*>(q_res + ((size_t)pg * kP + row0) * 64) + q;
#pragma unroll 4
    for (int t = 0; t < kC / 2; ++t) {
      const uint4 v = page[(row0 + t) * 16 + q];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      uint32_t r[8], s[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) hier_code2(w[j], A2[j], M2[j], r[2 * j], r[2 * j + 1], s[2 * j], s[2 * j + 1]);
      uint32_t a_lo, r_lo, a_hi, r_hi;
      hier_nibbles4(r, s, a_lo, r_lo);
      hier_nibbles4(r + 4, s + 4, a_hi, r_hi);
      pa[(size_t)t * 16] = prmt(a_lo, a_hi, 0x6420u);
      pr_[(size_t)t * 16] = prmt(r_lo, r_hi, 0x6420u) ^ 0x77777777u;
    }
  }
}

// Inverse: packed nibbles + metadata -> BF16 page.  The 16 x 16 pairs (Anchor nibble, Residual nibble) index a
// table of x_final values (sign-extended nibbles, v_mag, I = 16 v_mag - q_res, inverse alpha-law, sign), built
// by every CTA in shared memory with the same arithmetic a per-element evaluation would use (FULL = false, the
// Anchor-only case, uses the 16 entries with a zero Residual).  A thread owns eight channels (four bytes of each
// plane row) of a chunk; the two scalings of the inverse (chunk, then page) are folded into one multiply-add per
// channel, x = x_final * S + T with S = (sigma + eps)(gamma_scale + eps), T = mu (gamma_scale + eps) + gamma_min.
// Per token: one 32-bit load per plane (issued eight tokens ahead: the loop is bound by their latency otherwise),
// the table indices of four channels at a time by one bit-select, eight look-ups, four packed multiply-adds, one
// 16-byte store.
template <bool FULL>
__global__ void __launch_bounds__(128, FULL ? 4 : 6) hier_dequantize_kernel(const uint8_t* __restrict__ q_anc,
                                                              const uint8_t* __restrict__ q_res, int n_pages,
                                                              const float* __restrict__ g_min,
                                                              const float* __restrict__ g_scale,
                                                              const float* __restrict__ mu,
                                                              const float* __restrict__ sigma,
                                                              __nv_bfloat16* __restrict__ dst) {
  // FULL: every lane has its own copy of the 256 entries (entry e of lane l at e * 32 + l), so that the eight
  // look-ups of a token never meet in a bank; the 16 entries of the Anchor-only case sit in 16 banks anyway.
  constexpr int kEntries = FULL ? 256 : 16, kCopies = FULL ? 32 : 1;
  __shared__ float table[kEntries * kCopies];
  const int tid = threadIdx.x;
  for (int e = tid; e < kEntries; e += 128) {
    const int i = FULL ? e : e << 4;
    const int qa = ((i >> 4) ^ 8) - 8, qr = ((i & 15) ^ 8) - 8;             // sign-extend the nibbles
    const int v_mag = qa < 0 ? -qa - 1 : qa;
    const int I = (v_mag << 4) - qr;
    const float mag = (exp2f((float)I * (kLog2_1pAlpha / kYmax)) - 1.0f) * (1.0f / kAlpha);
    table[e * kCopies] = qa < 0 ? -mag : mag;
  }
  __syncthreads();
  if (FULL) {
    for (int i = tid; i < kEntries * kCopies; i += 128) table[i] = table[i & ~(kCopies - 1)];
    __syncthreads();
  }
  const uint32_t lane4 = (uint32_t)(tid & 31) << 2;
  const int ch = tid >> 4, oc = tid & 15;                                     // chunk, octet of channels
  constexpr int kB = 8;                                                       // tokens per batch of loads
  for (int pg = blockIdx.x; pg < n_pages; pg += gridDim.x) {
    const uint32_t* pa = reinterpret_cast<const uint32_t*>(q_anc + ((size_t)pg * kP + ch * kC) * 64) + oc;
    const uint32_t* prr = reinterpret_cast<const uint32_t*>(q_res + ((size_t)pg * kP + ch * kC) * 64) + oc;
    uint32_t wa[2][kB], wr[2][kB];
#pragma unroll
    for (int i = 0; i < kB; ++i) {
      wa[0][i] = __ldcs(pa + (size_t)i * 16);
      wr[0][i] = FULL ? __ldcs(prr + (size_t)i * 16) : 0u;
    }
    uint64_t S2[4], T2[4];
    {
      const float4* a = reinterpret_cast<const float4*>(sigma + ((size_t)pg * kChunks + ch) * LYNX_D) + oc * 2;
      const float4* b = reinterpret_cast<const float4*>(mu + ((size_t)pg * kChunks + ch) * LYNX_D) + oc * 2;
      const float4* c = reinterpret_cast<const float4*>(g_scale + (size_t)pg * LYNX_D) + oc * 2;
      const float4* d = reinterpret_cast<const float4*>(g_min + (size_t)pg * LYNX_D) + oc * 2;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float4 va = __ldg(a + h), vb = __ldg(b + h), vc = __ldg(c + h), vd = __ldg(d + h);
        const float sc0 = vc.x + kEps, sc1 = vc.y + kEps, sc2 = vc.z + kEps, sc3 = vc.w + kEps;
        S2[2 * h] = pack2((va.x + kEps) * sc0, (va.y + kEps) * sc1);
        S2[2 * h + 1] = pack2((va.z + kEps) * sc2, (va.w + kEps) * sc3);
        T2[2 * h] = pack2(fmaf(vb.x, sc0, vd.x), fmaf(vb.y, sc1, vd.y));
        T2[2 * h + 1] = pack2(fmaf(vb.z, sc2, vd.z), fmaf(vb.w, sc3, vd.w));
      }
    }
    uint4* out = reinterpret_cast<uint4*>(dst + ((size_t)pg * kP + ch * kC) * LYNX_D) + oc;
#pragma unroll
    for (int bt = 0; bt < kC / kB; ++bt) {
      const int cur = bt & 1;
      if (bt + 1 < kC / kB) {
#pragma unroll
        for (int i = 0; i < kB; ++i) {
          wa[cur ^ 1][i] = __ldcs(pa + (size_t)((bt + 1) * kB + i) * 16);
          wr[cur ^ 1][i] = FULL ? __ldcs(prr + (size_t)((bt + 1) * kB + i) * 16) : 0u;
        }
      }
#pragma unroll
      for (int i = 0; i < kB; ++i) {
        // table indices of the even channels (low nibbles) and the odd channels (high nibbles), a byte each
        const uint32_t a = wa[cur][i], r = wr[cur][i];
        const uint32_t L = FULL ? lop3_sel(a << 4, r, 0xF0F0F0F0u) : a & 0x0F0F0F0Fu;
        const uint32_t H = FULL ? lop3_sel(a, r >> 4, 0xF0F0F0F0u) : (a >> 4) & 0x0F0F0F0Fu;
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float x0, x1;
          if (FULL) {   // byte offset of entry e of this lane: e * 128 + lane * 4, one shift and one bit-select
            const uint32_t o0 = lop3_sel(j == 0 ? L << 7 : L >> (8 * j - 7), lane4, 0x7F80u);
            const uint32_t o1 = lop3_sel(j == 0 ? H << 7 : H >> (8 * j - 7), lane4, 0x7F80u);
            x0 = *reinterpret_cast<const float*>(reinterpret_cast<const char*>(table) + o0);
            x1 = *reinterpret_cast<const float*>(reinterpret_cast<const char*>(table) + o1);
          } else {
            x0 = table[(L >> (8 * j)) & 0xFFu];
            x1 = table[(H >> (8 * j)) & 0xFFu];
          }
          float y0, y1;
          unpack2(f2_fma(pack2(x0, x1), S2[j], T2[j]), y0, y1);
          asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[j]) : "f"(y1), "f"(y0));
        }
        __stcs(out + (size_t)(bt * kB + i) * 16, make_uint4(o[0], o[1], o[2], o[3]));
      }
    }
  }
}

}  // namespace
}  // namespace lynx

extern "C" lynx_status lynx_hier_quantize(const void* src_bf16, int64_t n_pages, uint8_t* q_anc, uint8_t* q_res,
                                          float* gamma_min, float* gamma_scale, float* mu, float* sigma,
                                          void* stream) {
  using namespace lynx;
  if (n_pages == 0) return LYNX_OK;
  if (n_pages < 0 || n_pages > (1ll << 30)) return LYNX_ERR_SHAPE;
  if (!src_bf16 || !q_anc || !q_res || !gamma_min || !gamma_scale || !mu || !sigma) return LYNX_ERR_NULL;
  if (!aligned16(src_bf16) || !aligned16(gamma_min) || !aligned16(gamma_scale) || !aligned16(mu) || !aligned16(sigma))
    return LYNX_ERR_ALIGN;
  constexpr int kSmem = kP * 256 + 2 * kChunks * 64 * 4;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(hier_quantize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess)
      return LYNX_ERR_CUDA;
    configured[dev] = true;
  }
  const int64_t grid = n_pages < (int64_t)sm_count() * 3 ? n_pages : (int64_t)sm_count() * 3;
  hier_quantize_kernel<<<(unsigned)grid, 256, kSmem, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(src_bf16), (int)n_pages, q_anc, q_res, gamma_min, gamma_scale, mu, sigma);
  return launch_status();
}

extern "C" lynx_status lynx_hier_dequantize(const uint8_t* q_anc, const uint8_t* q_res, int64_t n_pages,
                                            const float* gamma_min, const float* gamma_scale, const float* mu,
                                            const float* sigma, void* dst_bf16, void* stream) {
  using namespace lynx;
  if (n_pages == 0) return LYNX_OK;
  if (n_pages < 0 || n_pages > (1ll << 30)) return LYNX_ERR_SHAPE;
  if (!q_anc || !gamma_min || !gamma_scale || !mu || !sigma || !dst_bf16) return LYNX_ERR_NULL;
  if (!aligned16(dst_bf16) || !aligned16(gamma_min) || !aligned16(gamma_scale) || !aligned16(mu) || !aligned16(sigma))
    return LYNX_ERR_ALIGN;
  if (!aligned16(q_anc) || (q_res && !aligned16(q_res))) return LYNX_ERR_ALIGN;
  const int64_t grid = n_pages < (int64_t)sm_count() * 16 ? n_pages : (int64_t)sm_count() * 16;
  if (q_res)
    hier_dequantize_kernel<true><<<(unsigned)grid, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        q_anc, q_res, (int)n_pages, gamma_min, gamma_scale, mu, sigma, static_cast<__nv_bfloat16*>(dst_bf16));
  else
    hier_dequantize_kernel<false><<<(unsigned)grid, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        q_anc, q_anc, (int)n_pages, gamma_min, gamma_scale, mu, sigma, static_cast<__nv_bfloat16*>(dst_bf16));
  return launch_status();
}
