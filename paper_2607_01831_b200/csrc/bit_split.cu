// lynx_split_quantize_bits and lynx_recombine_bits: the Anchor / Residual split at other bit positions (sm_100a).
//
// The paper splits the 8-bit code of the linear grouped quantiser (Section 2.3; one group = one token's
// 128-element head vector) into its top 4 and bottom 4 bits (Section 4.1 stage 4) and names other splits as a
// direction (Conclusion).  Here the Anchor is the top A bits and the Residual the bottom R = 8 - A bits,
// A in {2, 4, 6}; code, scale and zero are those of lynx_split_quantize (the same arithmetic, operation for
// operation), so (anchor << R) | residual is that code for every A and A = 4 writes the same planes.
// Packing per row and stream: element e's field at bits [e w, (e + 1) w) of the row's 16 w bytes, least
// significant bit first (w = A or R).  Recombine is the refinement to the full code of Section 4.2 or, on the
// Anchor alone, the bucket mid-point (anchor << R) + 2^(R-1), then level * scale + zero rounded once to FP32
// and to BF16.
//
// Streaming kernels, HBM-bound: a quarter-warp owns a row, a lane 16 consecutive elements (two 128-bit loads),
// min / max on packed BF16 pairs and three xor-shuffles, 16 fields of each stream packed into w / 2 words.
#include <cuda_bf16.h>

#include "lynx_common.cuh"

namespace lynx {
namespace {

constexpr int kBsThreads = 256;
constexpr int kBsRows = 4;   // rows in flight per quarter-warp

__device__ __forceinline__ uint32_t bs_min2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bs_max2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// 32 contiguous bytes per lane in one instruction (the address must be 32-byte aligned)
__device__ __forceinline__ void ld256_cs(const void* p, uint4& a, uint4& b) {
  asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p));
}
__device__ __forceinline__ void st256_cs(void* p, const uint4& a, const uint4& b) {
  asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

// 16 fields of W bits, element order, least significant bit first, into W / 2 words
template <int W>
__device__ __forceinline__ void pack16(const uint32_t (&f)[16], uint32_t (&w)[W / 2]) {
#pragma unroll
  for (int i = 0; i < W / 2; ++i) w[i] = 0u;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int bit = i * W, word = bit >> 5, sh = bit & 31;
    w[word] |= f[i] << sh;
    if (sh + W > 32) w[word + 1] |= f[i] >> (32 - sh);
  }
}
template <int W>
__device__ __forceinline__ uint32_t field16(const uint32_t (&w)[W / 2], int i) {
  const int bit = i * W, word = bit >> 5, sh = bit & 31;
  uint32_t v = w[word] >> sh;
  if (sh + W > 32) v |= w[word + 1] << (32 - sh);
  return v & ((1u << W) - 1u);
}

template <int A>
__global__ void __launch_bounds__(kBsThreads) split_bits_kernel(const uint4* __restrict__ src, int64_t n_rows,
                                                                uint32_t* __restrict__ anchor,
                                                                uint32_t* __restrict__ residual,
                                                                float2* __restrict__ meta, bool wide) {
  constexpr int R = 8 - A;
  const int ln = threadIdx.x & 7;
  const int64_t grp = (int64_t)blockIdx.x * (kBsThreads / 8) + (threadIdx.x >> 3);
  const int64_t grp_total = (int64_t)gridDim.x * (kBsThreads / 8);
  for (int64_t r0 = grp * kBsRows; r0 < n_rows; r0 += grp_total * kBsRows) {
    uint4 lo[kBsRows], hi[kBsRows];
#pragma unroll
    for (int u = 0; u < kBsRows; ++u) {
      lo[u] = hi[u] = make_uint4(0, 0, 0, 0);
      if (r0 + u < n_rows) {   // elements 16 ln .. 16 ln + 7 and 16 ln + 8 .. 16 ln + 15
        if (wide) {
          ld256_cs(src + (r0 + u) * 16 + 2 * ln, lo[u], hi[u]);
        } else {
          lo[u] = __ldcs(src + (r0 + u) * 16 + 2 * ln);
          hi[u] = __ldcs(src + (r0 + u) * 16 + 2 * ln + 1);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kBsRows; ++u) {
      // (the shuffles are executed by every lane of the warp, valid row or not)
      const uint32_t w[8] = {lo[u].x, lo[u].y, lo[u].z, lo[u].w, hi[u].x, hi[u].y, hi[u].z, hi[u].w};
      uint32_t mn2 = w[0], mx2 = w[0];
#pragma unroll
      for (int i = 1; i < 8; ++i) { mn2 = bs_min2(mn2, w[i]); mx2 = bs_max2(mx2, w[i]); }
      // one register (min, -max) through three xor-shuffles of the 8 lanes that own the row
      uint32_t v = bs_min2(__byte_perm(mn2, mx2, 0x5410) ^ 0x80000000u, __byte_perm(mn2, mx2, 0x7632) ^ 0x80000000u);
#pragma unroll
      for (int off = 4; off >= 1; off >>= 1) v = bs_min2(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
      const float mn = __uint_as_float(v << 16);
      const float mx = __uint_as_float((v & 0xFFFF0000u) ^ 0x80000000u);
      const float range = __fsub_rn(mx, mn);
      const bool live = range >= 0x1p-100f;
      const float scale = live ? __fdiv_rn(range, 255.0f) : 0.0f;
      const float inv = live ? __fdiv_rn(255.0f, range) : 0.0f;
      const float zero = __fadd_rn(mn, 0.0f);   // -0 -> +0
      uint32_t fa[16], fr[16];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        // code = round-half-even of the exact product (x - mn) inv: the low byte of fma(u, inv, 1.5 * 2^23)
        const uint32_t c0 = __float_as_uint(__fmaf_rn(__fsub_rn(__uint_as_float(w[i] << 16), mn), inv, 12582912.0f)) & 0xFFu;
        const uint32_t c1 = __float_as_uint(__fmaf_rn(__fsub_rn(__uint_as_float(w[i] & 0xFFFF0000u), mn), inv, 12582912.0f)) & 0xFFu;
        fa[2 * i] = c0 >> R;  fr[2 * i] = c0 & ((1u << R) - 1u);
        fa[2 * i + 1] = c1 >> R;  fr[2 * i + 1] = c1 & ((1u << R) - 1u);
      }
      uint32_t wa[A / 2], wr[R / 2];
      pack16<A>(fa, wa);
      pack16<R>(fr, wr);
      if (r0 + u < n_rows) {
        uint32_t* pa = anchor + (r0 + u) * (4 * A) + ln * (A / 2);
        uint32_t* pr = residual + (r0 + u) * (4 * R) + ln * (R / 2);
#pragma unroll
        for (int i = 0; i < A / 2; ++i) __stcs(pa + i, wa[i]);
#pragma unroll
        for (int i = 0; i < R / 2; ++i) __stcs(pr + i, wr[i]);
        if (ln == 0) __stcs(meta + r0 + u, make_float2(scale, zero));
      }
    }
  }
}

template <int A, bool kFull, bool kCodes, bool kBf16>
__global__ void __launch_bounds__(kBsThreads) recombine_bits_kernel(const uint32_t* __restrict__ anchor,
                                                                    const uint32_t* __restrict__ residual,
                                                                    const float2* __restrict__ meta, int64_t n_rows,
                                                                    uint4* __restrict__ codes, uint4* __restrict__ deq,
                                                                    bool wide) {
  constexpr int R = 8 - A;
  const int64_t n_items = n_rows * 8;   // 8 lanes per row, 16 elements per lane
  const int64_t stride = (int64_t)gridDim.x * kBsThreads;
  for (int64_t i = (int64_t)blockIdx.x * kBsThreads + threadIdx.x; i < n_items; i += stride) {
    const int64_t row = i >> 3;
    const int ln = (int)(i & 7);
    uint32_t wa[A / 2], wr[R / 2];
#pragma unroll
    for (int j = 0; j < A / 2; ++j) wa[j] = __ldcs(anchor + row * (4 * A) + ln * (A / 2) + j);
#pragma unroll
    for (int j = 0; j < R / 2; ++j) wr[j] = kFull ? __ldcs(residual + row * (4 * R) + ln * (R / 2) + j) : 0u;
    uint32_t lv[16];
#pragma unroll
    for (int e = 0; e < 16; ++e)
      lv[e] = (field16<A>(wa, e) << R) | (kFull ? field16<R>(wr, e) : (1u << (R - 1)));
    if (kCodes) {
      uint32_t c[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) c[j] = lv[4 * j] | (lv[4 * j + 1] << 8) | (lv[4 * j + 2] << 16) | (lv[4 * j + 3] << 24);
      __stcs(codes + i, make_uint4(c[0], c[1], c[2], c[3]));
    }
    if (kBf16) {
      const float2 m = __ldg(meta + row);
      uint32_t o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const __nv_bfloat162 p = __floats2bfloat162_rn(__fmaf_rn((float)lv[2 * j], m.x, m.y),
                                                       __fmaf_rn((float)lv[2 * j + 1], m.x, m.y));
        o[j] = *reinterpret_cast<const uint32_t*>(&p);
      }
      if (wide) {
        st256_cs(deq + 2 * i, make_uint4(o[0], o[1], o[2], o[3]), make_uint4(o[4], o[5], o[6], o[7]));
      } else {
        __stcs(deq + 2 * i, make_uint4(o[0], o[1], o[2], o[3]));
        __stcs(deq + 2 * i + 1, make_uint4(o[4], o[5], o[6], o[7]));
      }
    }
  }
}

inline unsigned bs_grid(int64_t ctas) {
  const int64_t cap = (int64_t)sm_count() * 8;
  return (unsigned)(ctas < 1 ? 1 : ctas < cap ? ctas : cap);
}

template <int A>
lynx_status launch_recombine_bits(const uint32_t* a, const uint32_t* r, const float2* m, int64_t n_rows, uint4* c,
                                  uint4* d, cudaStream_t st) {
  const unsigned grid = bs_grid((n_rows * 8 + kBsThreads - 1) / kBsThreads);
  const bool wide = (reinterpret_cast<uintptr_t>(d) & 31u) == 0;   // 256-bit stores of the BF16 rows
#define LYNX_RB(F, C, B) recombine_bits_kernel<A, F, C, B><<<grid, kBsThreads, 0, st>>>(a, r, m, n_rows, c, d, wide)
  if (r) {
    if (c && d) LYNX_RB(true, true, true); else if (c) LYNX_RB(true, true, false); else LYNX_RB(true, false, true);
  } else {
    if (c && d) LYNX_RB(false, true, true); else if (c) LYNX_RB(false, true, false); else LYNX_RB(false, false, true);
  }
#undef LYNX_RB
  return launch_status();
}

}  // namespace
}  // namespace lynx

extern "C" lynx_status lynx_split_quantize_bits(const void* src_bf16, int64_t n_rows, int32_t anchor_bits,
                                                uint8_t* anchor, uint8_t* residual, float* meta, void* stream) {
  using namespace lynx;
  if (n_rows < 0) return LYNX_ERR_SHAPE;
  if (anchor_bits != 2 && anchor_bits != 4 && anchor_bits != 6) return LYNX_ERR_UNSUPPORTED;
  if (n_rows == 0) return LYNX_OK;
  if (!src_bf16 || !anchor || !residual || !meta) return LYNX_ERR_NULL;
  if (!aligned16(src_bf16) || !aligned16(anchor) || !aligned16(residual) || (reinterpret_cast<uintptr_t>(meta) & 7u))
    return LYNX_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int rows_per_trip = (kBsThreads / 8) * kBsRows;
  const unsigned grid = bs_grid((n_rows + rows_per_trip - 1) / rows_per_trip);
  const uint4* s = static_cast<const uint4*>(src_bf16);
  uint32_t* a = reinterpret_cast<uint32_t*>(anchor);
  uint32_t* r = reinterpret_cast<uint32_t*>(residual);
  float2* m = reinterpret_cast<float2*>(meta);
  const bool wide = (reinterpret_cast<uintptr_t>(src_bf16) & 31u) == 0;   // 256-bit loads of the source rows
  if (anchor_bits == 2) split_bits_kernel<2><<<grid, kBsThreads, 0, st>>>(s, n_rows, a, r, m, wide);
  else if (anchor_bits == 4) split_bits_kernel<4><<<grid, kBsThreads, 0, st>>>(s, n_rows, a, r, m, wide);
  else split_bits_kernel<6><<<grid, kBsThreads, 0, st>>>(s, n_rows, a, r, m, wide);
  return launch_status();
}

extern "C" lynx_status lynx_recombine_bits(const uint8_t* anchor, const uint8_t* residual, const float* meta,
                                           int64_t n_rows, int32_t anchor_bits, uint8_t* codes_u8, void* dequant_bf16,
                                           void* stream) {
  using namespace lynx;
  if (n_rows < 0) return LYNX_ERR_SHAPE;
  if (anchor_bits != 2 && anchor_bits != 4 && anchor_bits != 6) return LYNX_ERR_UNSUPPORTED;
  if (n_rows == 0) return LYNX_OK;
  if (!anchor || (!codes_u8 && !dequant_bf16)) return LYNX_ERR_NULL;
  if (dequant_bf16 && !meta) return LYNX_ERR_NULL;
  if (!aligned16(anchor) || !aligned16(residual) || !aligned16(codes_u8) || !aligned16(dequant_bf16) ||
      (reinterpret_cast<uintptr_t>(meta) & 7u))
    return LYNX_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint32_t* a = reinterpret_cast<const uint32_t*>(anchor);
  const uint32_t* r = reinterpret_cast<const uint32_t*>(residual);
  const float2* m = reinterpret_cast<const float2*>(meta);
  uint4* c = reinterpret_cast<uint4*>(codes_u8);
  uint4* d = static_cast<uint4*>(dequant_bf16);
  if (anchor_bits == 2) return launch_recombine_bits<2>(a, r, m, n_rows, c, d, st);
  if (anchor_bits == 4) return launch_recombine_bits<4>(a, r, m, n_rows, c, d, st);
  return launch_recombine_bits<6>(a, r, m, n_rows, c, d, st);
}
