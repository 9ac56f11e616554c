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

// alpha-law magnitude code of a normalised value x in [-1, 1] and the two nibbles of stage 4
__device__ __forceinline__ void hier_code(float x, uint32_t& anc, uint32_t& res) {
  const float y = __log2f(fmaf(kAlpha, fabsf(x), 1.0f)) * (kYmax / kLog2_1pAlpha);
  const int I = __float2int_rn(y);                 // raw integer, 0..120
  const int v_mag = (I + 7) >> 4;                  // round-half-down bias, magnitude (Anchor)
  const int q_res = (v_mag << 4) - I;              // centred correction, -8..7
  const int q_anc = x < 0.0f ? -v_mag - 1 : v_mag; // sign-aware two's complement, -8..7
  anc = (uint32_t)q_anc & 15u;
  res = (uint32_t)q_res & 15u;
}

__global__ void __launch_bounds__(256) hier_quantize_kernel(const __nv_bfloat16* __restrict__ src, int n_pages,
                                                            uint8_t* __restrict__ q_anc, uint8_t* __restrict__ q_res,
                                                            float* __restrict__ g_min, float* __restrict__ g_scale,
                                                            float* __restrict__ mu, float* __restrict__ sigma) {
  extern __shared__ __align__(16) unsigned char smem[];
  uint32_t* page = reinterpret_cast<uint32_t*>(smem);                 // [256 tokens][64 channel pairs]
  float2* s_min = reinterpret_cast<float2*>(smem + kP * 256);         // [64] per channel pair
  float2* s_inv = s_min + 64;                                         // 1 / (range + eps)
  float2* red = s_inv + 64;                                           // [4][64][2]: partial min, max
  const int tid = threadIdx.x;
  for (int pg = blockIdx.x; pg < n_pages; pg += gridDim.x) {
    const uint4* gsrc = reinterpret_cast<const uint4*>(src + (size_t)pg * kP * LYNX_D);
    __syncthreads();                                                  // the previous page is done with shared memory
    for (int i = tid; i < kP * LYNX_D / 8; i += 256) reinterpret_cast<uint4*>(page)[i] = __ldg(gsrc + i);
    __syncthreads();
    // ---- stage 1: per-channel minimum and range over the page's 256 tokens --------------------------
    {
      const int pr = tid & 63, qt = tid >> 6;                         // channel pair, quarter of the tokens
      float mn0 = INFINITY, mn1 = INFINITY, mx0 = -INFINITY, mx1 = -INFINITY;
      for (int t = qt * 64; t < qt * 64 + 64; ++t) {
        const uint32_t w = page[t * 64 + pr];
        mn0 = fminf(mn0, lo_bf16(w)); mx0 = fmaxf(mx0, lo_bf16(w));
        mn1 = fminf(mn1, hi_bf16(w)); mx1 = fmaxf(mx1, hi_bf16(w));
      }
      red[(qt * 64 + pr) * 2] = make_float2(mn0, mn1);
      red[(qt * 64 + pr) * 2 + 1] = make_float2(mx0, mx1);
    }
    __syncthreads();
    if (tid < 64) {
      float2 mn = red[tid * 2], mx = red[tid * 2 + 1];
      for (int qt = 1; qt < 4; ++qt) {
        const float2 a = red[(qt * 64 + tid) * 2], b = red[(qt * 64 + tid) * 2 + 1];
        mn.x = fminf(mn.x, a.x); mn.y = fminf(mn.y, a.y);
        mx.x = fmaxf(mx.x, b.x); mx.y = fmaxf(mx.y, b.y);
      }
      const float2 sc = make_float2(mx.x - mn.x, mx.y - mn.y);
      s_min[tid] = mn;
      s_inv[tid] = make_float2(1.0f / (sc.x + kEps), 1.0f / (sc.y + kEps));
      reinterpret_cast<float2*>(g_min + (size_t)pg * LYNX_D)[tid] = mn;
      reinterpret_cast<float2*>(g_scale + (size_t)pg * LYNX_D)[tid] = sc;
    }
    __syncthreads();
    // ---- stages 2-4 per (chunk, channel pair): 512 tasks, two per thread -------------------------------
    for (int task = tid; task < kChunks * 64; task += 256) {
      const int ch = task >> 6, pr = task & 63;
      const float2 mn = s_min[pr], inv = s_inv[pr];
      float sum0 = 0.0f, sum1 = 0.0f;
      for (int t = ch * kC; t < ch * kC + kC; ++t) {
        const uint32_t w = page[t * 64 + pr];
        sum0 += (lo_bf16(w) - mn.x) * inv.x;
        sum1 += (hi_bf16(w) - mn.y) * inv.y;
      }
      const float m0 = sum0 * (1.0f / kC), m1 = sum1 * (1.0f / kC);
      float s0 = 0.0f, s1 = 0.0f;
      for (int t = ch * kC; t < ch * kC + kC; ++t) {
        const uint32_t w = page[t * 64 + pr];
        s0 = fmaxf(s0, fabsf((lo_bf16(w) - mn.x) * inv.x - m0));
        s1 = fmaxf(s1, fabsf((hi_bf16(w) - mn.y) * inv.y - m1));
      }
      reinterpret_cast<float2*>(mu + ((size_t)pg * kChunks + ch) * LYNX_D)[pr] = make_float2(m0, m1);
      reinterpret_cast<float2*>(sigma + ((size_t)pg * kChunks + ch) * LYNX_D)[pr] = make_float2(s0, s1);
      const float i0 = 1.0f / (s0 + kEps), i1 = 1.0f / (s1 + kEps);
      uint8_t* pa = q_anc + ((size_t)pg * kP + ch * kC) * 64 + pr;
      uint8_t* pr_ = q_res + ((size_t)pg * kP + ch * kC) * 64 + pr;
      for (int t = 0; t < kC; ++t) {
        const uint32_t w = page[(ch * kC + t) * 64 + pr];
        uint32_t a0, r0, a1, r1;
        hier_code(((lo_bf16(w) - mn.x) * inv.x - m0) * i0, a0, r0);
        hier_code(((hi_bf16(w) - mn.y) * inv.y - m1) * i1, a1, r1);
        pa[(size_t)t * 64] = (uint8_t)(a0 | (a1 << 4));
        pr_[(size_t)t * 64] = (uint8_t)(r0 | (r1 << 4));
      }
    }
  }
}

// Inverse: packed nibbles + metadata -> BF16 page.  A thread owns a channel pair of a chunk.
__global__ void __launch_bounds__(256) hier_dequantize_kernel(const uint8_t* __restrict__ q_anc,
                                                              const uint8_t* __restrict__ q_res, int n_pages,
                                                              const float* __restrict__ g_min,
                                                              const float* __restrict__ g_scale,
                                                              const float* __restrict__ mu,
                                                              const float* __restrict__ sigma,
                                                              __nv_bfloat16* __restrict__ dst) {
  const int tid = threadIdx.x;
  for (int pg = blockIdx.x; pg < n_pages; pg += gridDim.x) {
    for (int task = tid; task < kChunks * 64; task += 256) {
      const int ch = task >> 6, pr = task & 63;
      const float2 mn = reinterpret_cast<const float2*>(g_min + (size_t)pg * LYNX_D)[pr];
      const float2 sc = reinterpret_cast<const float2*>(g_scale + (size_t)pg * LYNX_D)[pr];
      const float2 m = reinterpret_cast<const float2*>(mu + ((size_t)pg * kChunks + ch) * LYNX_D)[pr];
      const float2 sg = reinterpret_cast<const float2*>(sigma + ((size_t)pg * kChunks + ch) * LYNX_D)[pr];
      const uint8_t* pa = q_anc + ((size_t)pg * kP + ch * kC) * 64 + pr;
      const uint8_t* prr = q_res ? q_res + ((size_t)pg * kP + ch * kC) * 64 + pr : nullptr;
      uint32_t* out = reinterpret_cast<uint32_t*>(dst + ((size_t)pg * kP + ch * kC) * LYNX_D) + pr;
      for (int t = 0; t < kC; ++t) {
        const uint32_t ba = pa[(size_t)t * 64], br = prr ? prr[(size_t)t * 64] : 0u;
        float x[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int qa = ((int)((ba >> (4 * h)) & 15u) ^ 8) - 8;          // sign-extend the nibbles
          const int qr = ((int)((br >> (4 * h)) & 15u) ^ 8) - 8;
          const int v_mag = qa < 0 ? -qa - 1 : qa;
          const int I = (v_mag << 4) - qr;
          const float mag = (exp2f((float)I * (kLog2_1pAlpha / kYmax)) - 1.0f) * (1.0f / kAlpha);
          const float xf = qa < 0 ? -mag : mag;
          const float sgm = h ? sg.y : sg.x, mm = h ? m.y : m.x, scl = h ? sc.y : sc.x, mnn = h ? mn.y : mn.x;
          x[h] = fmaf(fmaf(xf, sgm + kEps, mm), scl + kEps, mnn);
        }
        const __nv_bfloat162 v = __floats2bfloat162_rn(x[0], x[1]);
        out[(size_t)t * 64] = *reinterpret_cast<const uint32_t*>(&v);
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
  constexpr int kSmem = kP * 256 + 64 * 8 * 2 + 4 * 64 * 2 * 8;
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
  const int64_t grid = n_pages < (int64_t)sm_count() * 8 ? n_pages : (int64_t)sm_count() * 8;
  hier_dequantize_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      q_anc, q_res, (int)n_pages, gamma_min, gamma_scale, mu, sigma, static_cast<__nv_bfloat16*>(dst_bf16));
  return launch_status();
}
