// lynx_split_quantize and lynx_recombine: streaming codec kernels (HBM-bound).
//
// Split-quantise follows the linear grouped quantiser of Section 2.3 (one group = one token's
// 128-element head vector), the MSB/LSB split of Section 4.1 stage 4 and the two-nibbles-per-
// byte, one-contiguous-buffer-per-stream packing of the Compression Kernel paragraph.
// Recombine is the Residual-phase refinement to Q_full of Section 4.2.
//
// Mapping: a row is 256 B of BF16; a quarter-warp (8 lanes) owns a row: two 128-bit streaming
// loads per lane (each instruction covers 128 contiguous bytes of the row), min/max on packed
// BF16 pairs and three xor-shuffles, 16 codes per lane, 2 x 4 B of each plane per lane.
// Eight rows are in flight per quarter-warp.
#include <cuda_bf16.h>

#include "lynx_common.cuh"

namespace lynx {

namespace {

constexpr int kThreads = 256;
constexpr int kLanesPerRow = 8;   // a quarter-warp owns a row: 2 x 16 B per lane
// rows per quarter-warp per loop trip: dense rows 8 (2: 0.84, 4: 0.87, 8: 0.90 of the copy rate; 12:
// spills); rows of listed blocks 4 (2: 0.81, 4: 0.87, 8: 0.77: the block lookups cost registers)
constexpr int kRowsInFlight = 8;
constexpr int kRowsInFlightIds = 4;

// Round-half-even of the exact product u*inv, as the low byte of an FP32 whose ulp is 1:
// fma(u, inv, 1.5 * 2^23) rounds the exact sum once, to an integer, ties to even.
__device__ __forceinline__ uint32_t code_bits(float x, float mn, float inv) {
  return __float_as_uint(__fmaf_rn(__fsub_rn(x, mn), inv, 12582912.0f));
}
__device__ __forceinline__ uint32_t bf2min(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf2max(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// Two FP32 values in a register pair, one instruction for both (IEEE round-to-nearest per element, as the
// scalar forms)
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
// Codes of 8 consecutive elements (4 BF16 pairs in w) -> 4 bytes of each nibble plane.
__device__ __forceinline__ void codes8(const uint32_t (&w)[4], float mn, float inv, uint32_t& a,
                                       uint32_t& r) {
  uint32_t c[8];
  const uint64_t mn2 = pack2(mn, mn), inv2 = pack2(inv, inv), magic2 = pack2(12582912.0f, 12582912.0f);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    // (x - mn) rounded, then fma(u, inv, 1.5 * 2^23): the two elements of a word at once
    const uint64_t x2 = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
    uint64_t u2, y2;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(u2) : "l"(x2), "l"(mn2));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(y2) : "l"(u2), "l"(inv2), "l"(magic2));
    asm("mov.b64 {%0, %1}, %2;" : "=r"(c[2 * i]), "=r"(c[2 * i + 1]) : "l"(y2));
  }
  // low bytes gathered: w0 = codes 0..3, w1 = codes 4..7
  const uint32_t w0 = __byte_perm(__byte_perm(c[0], c[1], 0x0040), __byte_perm(c[2], c[3], 0x0040), 0x5410);
  const uint32_t w1 = __byte_perm(__byte_perm(c[4], c[5], 0x0040), __byte_perm(c[6], c[7], 0x0040), 0x5410);
  // bytes 0 and 2 of each combination hold two packed nibbles (the other bytes are unused)
  const uint32_t s0 = w0 >> 4, s1 = w1 >> 4;
  const uint32_t a0 = (s0 & 0x0F0F0F0Fu) | ((w0 >> 8) & 0xF0F0F0F0u);
  const uint32_t a1 = (s1 & 0x0F0F0F0Fu) | ((w1 >> 8) & 0xF0F0F0F0u);
  const uint32_t r0 = (w0 & 0x0F0F0F0Fu) | (s0 & 0xF0F0F0F0u);
  const uint32_t r1 = (w1 & 0x0F0F0F0Fu) | (s1 & 0xF0F0F0F0u);
  a = __byte_perm(a0, a1, 0x6420);
  r = __byte_perm(r0, r1, 0x6420);
}

template <bool kIds>
__global__ void __launch_bounds__(kThreads)
split_quantize_kernel(const uint4* __restrict__ src, int64_t n_logical_rows,
                      const int32_t* __restrict__ block_ids, uint32_t rows_per_block,
                      int64_t n_blocks_total, uint32_t* __restrict__ anchor,
                      uint32_t* __restrict__ residual, float2* __restrict__ meta) {
  const int ln = threadIdx.x & (kLanesPerRow - 1);
  const int64_t grp = (int64_t)blockIdx.x * (kThreads / kLanesPerRow) + (threadIdx.x / kLanesPerRow);
  const int64_t grp_total = (int64_t)gridDim.x * (kThreads / kLanesPerRow);

  constexpr int kRows = kIds ? kRowsInFlightIds : kRowsInFlight;
  for (int64_t r0 = grp * kRows; r0 < n_logical_rows; r0 += grp_total * kRows) {
    uint4 lo[kRows], hi[kRows];
    int64_t row[kRows];
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      int64_t lr = r0 + u;
      row[u] = -1;
      if (lr < n_logical_rows) {
        if (kIds) {
          uint32_t lb = (uint32_t)lr / rows_per_block;
          uint32_t in = (uint32_t)lr - lb * rows_per_block;
          int32_t blk = __ldg(block_ids + lb);
          if (blk >= 0 && blk < n_blocks_total) row[u] = (int64_t)blk * rows_per_block + in;
        } else {
          row[u] = lr;
        }
      }
      lo[u] = hi[u] = make_uint4(0, 0, 0, 0);
      if (row[u] >= 0) {
        lo[u] = __ldcs(src + row[u] * 16 + ln);      // elements 8*ln .. 8*ln+7
        hi[u] = __ldcs(src + row[u] * 16 + 8 + ln);  // elements 64+8*ln .. 64+8*ln+7
      }
    }
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      // the shuffles below are executed by every lane of the warp, valid row or not
      const uint32_t wl[4] = {lo[u].x, lo[u].y, lo[u].z, lo[u].w};
      const uint32_t wh[4] = {hi[u].x, hi[u].y, hi[u].z, hi[u].w};
      // packed BF16 min / max over the lane's 16 values, then one register (min, -max) through
      // three xor-shuffles of the 8 lanes that own the row
      const uint32_t mn2 = bf2min(bf2min(bf2min(wl[0], wl[1]), bf2min(wl[2], wl[3])),
                                  bf2min(bf2min(wh[0], wh[1]), bf2min(wh[2], wh[3])));
      const uint32_t mx2 = bf2max(bf2max(bf2max(wl[0], wl[1]), bf2max(wl[2], wl[3])),
                                  bf2max(bf2max(wh[0], wh[1]), bf2max(wh[2], wh[3])));
      uint32_t v = bf2min(__byte_perm(mn2, mx2, 0x5410) ^ 0x80000000u,
                          __byte_perm(mn2, mx2, 0x7632) ^ 0x80000000u);
#pragma unroll
      for (int off = 4; off >= 1; off >>= 1) v = bf2min(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
      const float mn = __uint_as_float(v << 16);
      const float mx = __uint_as_float((v & 0xFFFF0000u) ^ 0x80000000u);
      const float range = __fsub_rn(mx, mn);
      const bool live = range >= 0x1p-100f;
      const float scale = live ? __fdiv_rn(range, 255.0f) : 0.0f;
      const float inv = live ? __fdiv_rn(255.0f, range) : 0.0f;
      const float zero = __fadd_rn(mn, 0.0f);  // -0 -> +0

      uint32_t a_lo, r_lo, a_hi, r_hi;
      codes8(wl, mn, inv, a_lo, r_lo);
      codes8(wh, mn, inv, a_hi, r_hi);
      if (row[u] >= 0) {
        __stcs(anchor + row[u] * 16 + ln, a_lo);
        __stcs(anchor + row[u] * 16 + 8 + ln, a_hi);
        __stcs(residual + row[u] * 16 + ln, r_lo);
        __stcs(residual + row[u] * 16 + 8 + ln, r_hi);
        if (ln == 0) __stcs(meta + row[u], make_float2(scale, zero));
      }
    }
  }
}

template <bool kCodes, bool kBf16>
__global__ void __launch_bounds__(kThreads)
recombine_kernel(const uint32_t* __restrict__ anchor, const uint32_t* __restrict__ residual,
                 const float2* __restrict__ meta, int64_t n_rows, uint2* __restrict__ codes,
                 uint4* __restrict__ deq) {
  const int64_t n_items = n_rows * 16;  // 16 lanes per row, 8 elements per lane
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  constexpr int kAhead = 4;             // items per thread and trip: their loads are issued together
  for (int64_t i0 = (int64_t)blockIdx.x * kThreads + threadIdx.x; i0 < n_items; i0 += stride * kAhead) {
    uint32_t xas[kAhead], xrs[kAhead];
#pragma unroll
    for (int u = 0; u < kAhead; ++u) {
      const int64_t i = i0 + u * stride;
      xas[u] = i < n_items ? __ldcs(anchor + i) : 0u;
      xrs[u] = i < n_items ? __ldcs(residual + i) : 0u;
    }
#pragma unroll
    for (int u = 0; u < kAhead; ++u) {
    const int64_t i = i0 + u * stride;
    if (i >= n_items) break;
    const uint32_t xa = xas[u], xr = xrs[u];
    // even elements: (a << 4) | r from the low nibbles; odd elements from the high nibbles
    const uint32_t ev = ((xa << 4) & 0xF0F0F0F0u) | (xr & 0x0F0F0F0Fu);
    const uint32_t od = (xa & 0xF0F0F0F0u) | ((xr >> 4) & 0x0F0F0F0Fu);
    const uint32_t c0 = __byte_perm(ev, od, 0x5140);  // elements 0..3
    const uint32_t c1 = __byte_perm(ev, od, 0x7362);  // elements 4..7
    if (kCodes) __stcs(codes + i, make_uint2(c0, c1));
    if (kBf16) {
      const float2 m = __ldg(meta + (i >> 4));
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t cw = j < 2 ? c0 : c1;
        const float lo = __fmaf_rn((float)((cw >> ((j & 1) * 16)) & 0xFFu), m.x, m.y);
        const float hi = __fmaf_rn((float)((cw >> ((j & 1) * 16 + 8)) & 0xFFu), m.x, m.y);
        const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
        o[j] = *reinterpret_cast<const uint32_t*>(&p);
      }
      __stcs(deq + i, make_uint4(o[0], o[1], o[2], o[3]));
    }
    }
  }
}

int grid_for(int64_t items_per_block_unit, int blocks_per_sm) {
  int64_t cap = (int64_t)sm_count() * blocks_per_sm;
  int64_t g = items_per_block_unit < cap ? items_per_block_unit : cap;
  return (int)(g < 1 ? 1 : g);
}

}  // namespace
}  // namespace lynx

extern "C" lynx_status lynx_split_quantize(const void* src_bf16, int64_t n_rows,
                                           const int32_t* block_ids, int32_t n_block_ids,
                                           int32_t rows_per_block, uint8_t* anchor,
                                           uint8_t* residual, float* meta, void* stream) {
  using namespace lynx;
  if (n_rows < 0) return LYNX_ERR_SHAPE;
  if (n_rows == 0) return LYNX_OK;
  if (!src_bf16 || !anchor || !residual || !meta) return LYNX_ERR_NULL;
  if (!aligned16(src_bf16) || !aligned16(anchor) || !aligned16(residual) ||
      (reinterpret_cast<uintptr_t>(meta) & 7u))
    return LYNX_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int rows_per_cta_trip = (kThreads / kLanesPerRow) * (block_ids ? kRowsInFlightIds : kRowsInFlight);
  if (block_ids) {
    if (n_block_ids < 0 || rows_per_block <= 0 || n_rows % rows_per_block != 0) return LYNX_ERR_SHAPE;
    if (n_block_ids == 0) return LYNX_OK;
    const int64_t logical = (int64_t)n_block_ids * rows_per_block;
    if (logical >= (1ll << 31)) return LYNX_ERR_UNSUPPORTED;
    const int grid = grid_for((logical + rows_per_cta_trip - 1) / rows_per_cta_trip, 8);
    split_quantize_kernel<true><<<grid, kThreads, 0, st>>>(
        static_cast<const uint4*>(src_bf16), logical, block_ids, (uint32_t)rows_per_block,
        n_rows / rows_per_block, reinterpret_cast<uint32_t*>(anchor),
        reinterpret_cast<uint32_t*>(residual), reinterpret_cast<float2*>(meta));
  } else {
    const int grid = grid_for((n_rows + rows_per_cta_trip - 1) / rows_per_cta_trip, 8);
    split_quantize_kernel<false><<<grid, kThreads, 0, st>>>(
        static_cast<const uint4*>(src_bf16), n_rows, nullptr, 1u, n_rows,
        reinterpret_cast<uint32_t*>(anchor), reinterpret_cast<uint32_t*>(residual),
        reinterpret_cast<float2*>(meta));
  }
  return launch_status();
}

extern "C" lynx_status lynx_recombine(const uint8_t* anchor, const uint8_t* residual,
                                      const float* meta, int64_t n_rows, uint8_t* codes_u8,
                                      void* dequant_bf16, void* stream) {
  using namespace lynx;
  if (n_rows < 0) return LYNX_ERR_SHAPE;
  if (n_rows == 0) return LYNX_OK;
  if (!anchor || !residual || (!codes_u8 && !dequant_bf16)) return LYNX_ERR_NULL;
  if (dequant_bf16 && !meta) return LYNX_ERR_NULL;
  if (!aligned16(anchor) || !aligned16(residual) || !aligned16(codes_u8) ||
      !aligned16(dequant_bf16) || (reinterpret_cast<uintptr_t>(meta) & 7u))
    return LYNX_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int grid = grid_for((n_rows * 16 + kThreads - 1) / kThreads, 8);
  const uint32_t* a = reinterpret_cast<const uint32_t*>(anchor);
  const uint32_t* r = reinterpret_cast<const uint32_t*>(residual);
  const float2* m = reinterpret_cast<const float2*>(meta);
  uint2* c = reinterpret_cast<uint2*>(codes_u8);
  uint4* d = static_cast<uint4*>(dequant_bf16);
  if (codes_u8 && dequant_bf16)
    recombine_kernel<true, true><<<grid, kThreads, 0, st>>>(a, r, m, n_rows, c, d);
  else if (codes_u8)
    recombine_kernel<true, false><<<grid, kThreads, 0, st>>>(a, r, m, n_rows, c, d);
  else
    recombine_kernel<false, true><<<grid, kThreads, 0, st>>>(a, r, m, n_rows, c, d);
  return launch_status();
}
