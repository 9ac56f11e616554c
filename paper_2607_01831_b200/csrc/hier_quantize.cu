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
__device__ __forceinline__ float hi_or_lo(uint32_t w, int hi) { return hi ? hi_bf16(w) : lo_bf16(w); }

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
// Stages 3 and 4 for the two channels of a word (the multiply-adds as packed FP32 pairs):
// x_final = fma(x, A, B) (stages 1 and 2 folded into one multiply-add), the alpha-law magnitude
// y = log2(1 + 255 |x_final|) * 15 rounded to the nearest even integer I (0..120) by the magic-number
// addition, whose sum keeps I in its low mantissa bits.  Returned per channel: (I + 7) ^ sign mask, whose
// bits 4..7 are the Anchor nibble (v_mag = (I + 7) >> 4; two's complement -v_mag - 1 = ~v_mag for negative
// values), and -I, whose low nibble is the Residual (16 v_mag - I modulo 16).
__device__ __forceinline__ void hier_code2(uint32_t w, uint64_t A2, uint64_t B2, uint32_t& anc4_0, uint32_t& negI_0,
                                           uint32_t& anc4_1, uint32_t& negI_1) {
  const uint64_t x2 = pack2(lo_bf16(w), hi_bf16(w));
  uint64_t t2;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(t2) : "l"(x2), "l"(A2), "l"(B2));
  float t0, t1;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(t0), "=f"(t1) : "l"(t2));
  float l0, l1;
  asm("lg2.approx.f32 %0, %1;" : "=f"(l0) : "f"(fmaf(kAlpha, fabsf(t0), 1.0f)));
  asm("lg2.approx.f32 %0, %1;" : "=f"(l1) : "f"(fmaf(kAlpha, fabsf(t1), 1.0f)));
  uint64_t r2;
  const uint64_t k2 = pack2(kYmax / kLog2_1pAlpha, kYmax / kLog2_1pAlpha), m2 = pack2(12582912.0f, 12582912.0f);
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r2) : "l"(pack2(l0, l1)), "l"(k2), "l"(m2));
  uint32_t r0, r1;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(r0), "=r"(r1) : "l"(r2));   // 0x4B400000 + I
  anc4_0 = (r0 + 7u) ^ (uint32_t)(__float_as_int(t0) >> 31);
  anc4_1 = (r1 + 7u) ^ (uint32_t)(__float_as_int(t1) >> 31);
  negI_0 = 0u - r0;
  negI_1 = 0u - r1;
}

// One CTA per page: the page (64 KB) is staged in shared memory; a thread owns a channel pair (one 32-bit word
// of a token row: conflict-free column walks) of two chunks.  First the chunk statistics (minimum, maximum as
// packed BF16 pairs; sums in FP32), from which the page's minimum and range follow (stage 1) and, with them,
// every chunk's mean and largest deviation (stage 2: max |x - mean| = max(max - mean, mean - min)); then the
// codes.
__global__ void __launch_bounds__(256, 3) hier_quantize_kernel(const __nv_bfloat16* __restrict__ src, int n_pages,
                                                               uint8_t* __restrict__ q_anc, uint8_t* __restrict__ q_res,
                                                               float* __restrict__ g_min, float* __restrict__ g_scale,
                                                               float* __restrict__ mu, float* __restrict__ sigma) {
  extern __shared__ __align__(16) unsigned char smem[];
  uint32_t* page = reinterpret_cast<uint32_t*>(smem);                 // [256 tokens][64 channel pairs]
  uint32_t* c_min = reinterpret_cast<uint32_t*>(smem + kP * 256);     // [8 chunks][64 pairs] packed BF16 pairs
  uint32_t* c_max = c_min + kChunks * 64;
  float2* s_min = reinterpret_cast<float2*>(c_max + kChunks * 64);    // [64] page minimum per channel pair
  float2* s_inv = s_min + 64;                                         // 1 / (range + eps)
  const int tid = threadIdx.x, pr = tid & 63, ch0 = tid >> 6;         // chunks ch0 and ch0 + 4
  for (int pg = blockIdx.x; pg < n_pages; pg += gridDim.x) {
    const uint4* gsrc = reinterpret_cast<const uint4*>(src + (size_t)pg * kP * LYNX_D);
    __syncthreads();                                                  // the previous page is done with shared memory
#pragma unroll 4
    for (int i = tid; i < kP * LYNX_D / 8; i += 256) reinterpret_cast<uint4*>(page)[i] = __ldcs(gsrc + i);
    __syncthreads();
    float sum[2][2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int ch = ch0 + 4 * k;
      uint32_t mn = page[ch * kC * 64 + pr], mx = mn;
      float s0 = 0.0f, s1 = 0.0f;
#pragma unroll 8
      for (int t = 0; t < kC; ++t) {
        const uint32_t w = page[(ch * kC + t) * 64 + pr];
        mn = bf2_min(mn, w);
        mx = bf2_max(mx, w);
        s0 += lo_bf16(w);
        s1 += hi_bf16(w);
      }
      c_min[ch * 64 + pr] = mn;
      c_max[ch * 64 + pr] = mx;
      sum[k][0] = s0;
      sum[k][1] = s1;
    }
    __syncthreads();
    if (tid < 64) {   // stage 1: the page's minimum and range per channel
      uint32_t mn = c_min[tid], mx = c_max[tid];
#pragma unroll
      for (int ch = 1; ch < kChunks; ++ch) {
        mn = bf2_min(mn, c_min[ch * 64 + tid]);
        mx = bf2_max(mx, c_max[ch * 64 + tid]);
      }
      const float2 lo = make_float2(lo_bf16(mn), hi_bf16(mn));
      const float2 sc = make_float2(lo_bf16(mx) - lo.x, hi_bf16(mx) - lo.y);
      s_min[tid] = lo;
      s_inv[tid] = make_float2(1.0f / (sc.x + kEps), 1.0f / (sc.y + kEps));
      reinterpret_cast<float2*>(g_min + (size_t)pg * LYNX_D)[tid] = lo;
      reinterpret_cast<float2*>(g_scale + (size_t)pg * LYNX_D)[tid] = sc;
    }
    __syncthreads();
    const float2 gmn = s_min[pr], inv = s_inv[pr];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int ch = ch0 + 4 * k;
      const uint32_t mn = c_min[ch * 64 + pr], mx = c_max[ch * 64 + pr];
      // stage 2 in the page-normalised scale: mean and largest deviation of the chunk
      const float mean0 = sum[k][0] * (1.0f / kC), mean1 = sum[k][1] * (1.0f / kC);
      const float sg0 = fmaxf(hi_or_lo(mx, 0) - mean0, mean0 - hi_or_lo(mn, 0)) * inv.x;
      const float sg1 = fmaxf(hi_or_lo(mx, 1) - mean1, mean1 - hi_or_lo(mn, 1)) * inv.y;
      reinterpret_cast<float2*>(mu + ((size_t)pg * kChunks + ch) * LYNX_D)[pr] =
          make_float2((mean0 - gmn.x) * inv.x, (mean1 - gmn.y) * inv.y);
      reinterpret_cast<float2*>(sigma + ((size_t)pg * kChunks + ch) * LYNX_D)[pr] = make_float2(sg0, sg1);
      // x_final = ((x - gmin) inv - mu) / (sigma + eps) = (x - mean) * A
      const float A0 = inv.x / (sg0 + kEps), A1 = inv.y / (sg1 + kEps);
      const float B0 = -mean0 * A0, B1 = -mean1 * A1;
      const uint64_t A2 = pack2(A0, A1), B2 = pack2(B0, B1);
      uint8_t* pa = q_anc + ((size_t)pg * kP + ch * kC) * 64 + pr;
      uint8_t* pr_ = q_res + ((size_t)pg * kP + ch * kC) * 64 + pr;
#pragma unroll 8
      for (int t = 0; t < kC; ++t) {
        const uint32_t w = page[(ch * kC + t) * 64 + pr];
        uint32_t a0, n0, a1, n1;
        hier_code2(w, A2, B2, a0, n0, a1, n1);
        pa[(size_t)t * 64] = (uint8_t)lop3_sel(a0 >> 4, a1, 0x0Fu);
        pr_[(size_t)t * 64] = (uint8_t)lop3_sel(n0, n1 << 4, 0x0Fu);
      }
    }
  }
}

// Inverse: packed nibbles + metadata -> BF16 page.  The 16 x 16 pairs (Anchor nibble, Residual nibble) index a
// table of x_final values (sign-extended nibbles, v_mag, I = 16 v_mag - q_res, inverse alpha-law, sign), built
// by every CTA in shared memory with the same arithmetic a per-element evaluation would use (a second table of
// 16 entries serves the Anchor-only case, whose indices would otherwise fall into two banks).  A thread owns
// eight channels (four bytes of each plane row) of a chunk: per token one 32-bit load per plane, eight look-ups,
// sixteen multiply-adds, one 16-byte store.
__global__ void __launch_bounds__(128) hier_dequantize_kernel(const uint8_t* __restrict__ q_anc,
                                                              const uint8_t* __restrict__ q_res, int n_pages,
                                                              const float* __restrict__ g_min,
                                                              const float* __restrict__ g_scale,
                                                              const float* __restrict__ mu,
                                                              const float* __restrict__ sigma,
                                                              __nv_bfloat16* __restrict__ dst) {
  __shared__ float table[256], table_a[16];
  const int tid = threadIdx.x;
  for (int i = tid; i < 256; i += 128) {
    const int qa = ((i >> 4) ^ 8) - 8, qr = ((i & 15) ^ 8) - 8;             // sign-extend the nibbles
    const int v_mag = qa < 0 ? -qa - 1 : qa;
    const int I = (v_mag << 4) - qr;
    const float mag = (exp2f((float)I * (kLog2_1pAlpha / kYmax)) - 1.0f) * (1.0f / kAlpha);
    const float v = qa < 0 ? -mag : mag;
    table[i] = v;
    if ((i & 15) == 0) table_a[i >> 4] = v;
  }
  __syncthreads();
  const int ch = tid >> 4, oc = tid & 15;                                     // chunk, octet of channels
  for (int pg = blockIdx.x; pg < n_pages; pg += gridDim.x) {
    float sg[8], mm[8], sc[8], mn[8];
    {
      const float4* a = reinterpret_cast<const float4*>(sigma + ((size_t)pg * kChunks + ch) * LYNX_D) + oc * 2;
      const float4* b = reinterpret_cast<const float4*>(mu + ((size_t)pg * kChunks + ch) * LYNX_D) + oc * 2;
      const float4* c = reinterpret_cast<const float4*>(g_scale + (size_t)pg * LYNX_D) + oc * 2;
      const float4* d = reinterpret_cast<const float4*>(g_min + (size_t)pg * LYNX_D) + oc * 2;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float4 va = __ldg(a + h), vb = __ldg(b + h), vc = __ldg(c + h), vd = __ldg(d + h);
        sg[4 * h] = va.x + kEps; sg[4 * h + 1] = va.y + kEps; sg[4 * h + 2] = va.z + kEps; sg[4 * h + 3] = va.w + kEps;
        mm[4 * h] = vb.x; mm[4 * h + 1] = vb.y; mm[4 * h + 2] = vb.z; mm[4 * h + 3] = vb.w;
        sc[4 * h] = vc.x + kEps; sc[4 * h + 1] = vc.y + kEps; sc[4 * h + 2] = vc.z + kEps; sc[4 * h + 3] = vc.w + kEps;
        mn[4 * h] = vd.x; mn[4 * h + 1] = vd.y; mn[4 * h + 2] = vd.z; mn[4 * h + 3] = vd.w;
      }
    }
    const uint32_t* pa = reinterpret_cast<const uint32_t*>(q_anc + ((size_t)pg * kP + ch * kC) * 64) + oc;
    const uint32_t* prr = q_res ? reinterpret_cast<const uint32_t*>(q_res + ((size_t)pg * kP + ch * kC) * 64) + oc : nullptr;
    uint4* out = reinterpret_cast<uint4*>(dst + ((size_t)pg * kP + ch * kC) * LYNX_D) + oc;
#pragma unroll 4
    for (int t = 0; t < kC; ++t) {
      const uint32_t wa = __ldcs(pa + (size_t)t * 16), wr = prr ? __ldcs(prr + (size_t)t * 16) : 0u;
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {   // byte j: channels 2j (low nibbles) and 2j + 1 (high nibbles)
        const uint32_t ba = (wa >> (8 * j)) & 0xFFu, br = (wr >> (8 * j)) & 0xFFu;
        float x0, x1;
        if (prr) { x0 = table[((ba & 15u) << 4) | (br & 15u)]; x1 = table[(ba & 0xF0u) | (br >> 4)]; }
        else { x0 = table_a[ba & 15u]; x1 = table_a[ba >> 4]; }
        const float y0 = fmaf(fmaf(x0, sg[2 * j], mm[2 * j]), sc[2 * j], mn[2 * j]);
        const float y1 = fmaf(fmaf(x1, sg[2 * j + 1], mm[2 * j + 1]), sc[2 * j + 1], mn[2 * j + 1]);
        const __nv_bfloat162 v = __floats2bfloat162_rn(y0, y1);
        o[j] = *reinterpret_cast<const uint32_t*>(&v);
      }
      __stcs(out + (size_t)t * 16, make_uint4(o[0], o[1], o[2], o[3]));
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
  constexpr int kSmem = kP * 256 + 2 * kChunks * 64 * 4 + 2 * 64 * 8;
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
  hier_dequantize_kernel<<<(unsigned)grid, 128, 0, static_cast<cudaStream_t>(stream)>>>(
      q_anc, q_res, (int)n_pages, gamma_min, gamma_scale, mu, sigma, static_cast<__nv_bfloat16*>(dst_bf16));
  return launch_status();
}
