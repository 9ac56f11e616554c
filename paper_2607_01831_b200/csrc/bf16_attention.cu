// lynx_bf16_attention: decode attention over dequantised BF16 KV pages (sm_100a).
//
// The paper's own decode path (Section 4.2): the dequantisation kernel scatters BF16 pages into the
// paged KV memory and the engine's stock attention reads them, 256 bytes per row of K or V.  This is
// that second half, hand-written, as the baseline the fused kernels (72 / 136 bytes per row) are
// measured against: softmax(q K^T scale) V of Section 2 on pages [num_blocks][Hkv][block_tokens][128]
// BF16, as lynx_recombine writes them.
//
// Flash-decoding split-K: a CTA takes a chunk of kChunk tokens of one (sequence, KV head) and writes a
// partial (m, l, O) to the workspace; a second kernel merges the chunks.  Nothing waits on anything.
// Two kernels for the chunk: on the BF16 tensor cores (mma.sync m16n8k16, K and V tiles through a cp.async
// ring per warp) for block sizes that are multiples of 16 tokens -- it streams the pages at the rate of a
// plain copy -- and on the FP32 pipes for any other block size (8 or 16 lanes own a token, each 16 or 8 of
// its 128 dims; partial dot products reduced with shuffles), which runs out of multiply-adds at 8 columns.
#include <cuda_bf16.h>

#include "lynx_common.cuh"

namespace lynx {
namespace {

constexpr int kChunk = 2048;        // tokens per CTA
constexpr int kWarps = 8;           // warps per CTA: 256 tokens each
constexpr int kPartStrideB = 132;   // floats per (chunk, column) partial: O[128], m, l, pad

struct BfParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16 *k, *v;
  const int32_t* block_table;
  const int32_t* seq_lens;
  float* out;
  float* part;      // [B][Hkv][chunks][cols][kPartStrideB]
  float* lse;       // [B][nq][Hq] natural-log log-sum-exp of every output row's scores
  float sm_log2;
  int B, nq, causal, Hq, Hkv, G, bt, num_blocks, max_blocks, ncols, chunks;
  // A launch may be one slice [j0, j0 + nq) of the caller's n_q query positions (q, out and lse then point at
  // position j0): nq_stride = the caller's n_q, tail = n_q - j0 (the causal limit of position j of the slice is
  // len - tail + j + 1).  Unsliced: both equal nq.
  int nq_stride, tail;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// COLS query columns (padded), LPT lanes per token
template <int COLS, int LPT>
__global__ void __launch_bounds__(kWarps * 32, COLS <= 4 ? 2 : 1) bf16_decode_kernel(const BfParams p) {
  constexpr int DPL = LYNX_D / LPT;      // dims per lane: 16 or 8
  constexpr int TPP = 32 / LPT;          // tokens per pass of a warp: 4 or 2
  constexpr int NV = DPL / 8;            // 128-bit loads per row and lane
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = lane / LPT, sl = lane % LPT;
  const int chunk = blockIdx.x % p.chunks;
  const int bh = blockIdx.x / p.chunks;
  const int b = bh / p.Hkv, hkv = bh % p.Hkv;
  const int cap = p.max_blocks * p.bt;
  int len = __ldg(p.seq_lens + b);
  len = len < 0 ? 0 : (len > cap ? cap : len);
  float* part = p.part + ((size_t)bh * p.chunks + chunk) * (size_t)COLS * kPartStrideB;
  const int t_begin = chunk * kChunk, t_end = min(len, t_begin + kChunk);

  // this lane's slice of the queries, pre-multiplied by the softmax scale (log2 units)
  float q[COLS][DPL];
  int lim[COLS];
#pragma unroll
  for (int c = 0; c < COLS; ++c) {
    const int j = c / p.G, hh = c % p.G;
    const bool in = c < p.ncols;
    lim[c] = in ? (p.causal ? len - p.tail + j + 1 : len) : 0;
    const __nv_bfloat16* qp = p.q + (((size_t)b * p.nq_stride + (in ? j : 0)) * p.Hq + hkv * p.G + (in ? hh : 0)) * LYNX_D + sl * DPL;
#pragma unroll
    for (int d = 0; d < DPL; ++d) q[c][d] = in ? __bfloat162float(qp[d]) * p.sm_log2 : 0.0f;
  }
  float m[COLS], l[COLS], o[COLS][DPL];
#pragma unroll
  for (int c = 0; c < COLS; ++c) {
    m[c] = -1.0e30f; l[c] = 0.0f;
#pragma unroll
    for (int d = 0; d < DPL; ++d) o[c][d] = 0.0f;
  }

  // tokens of this warp: t_begin + warp * 256 + pass * TPP + grp
  const int w_begin = t_begin + warp * (kChunk / kWarps), w_end = min(t_end, w_begin + kChunk / kWarps);
  constexpr int U = COLS <= 4 ? 4 : 2;   // passes whose loads are issued together
  for (int t00 = w_begin; t00 < w_end; t00 += U * TPP) {
    uint4 kxu[U][NV], vxu[U][NV];
    bool validu[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = t00 + u * TPP + grp;
      validu[u] = t < w_end;
#pragma unroll
      for (int i = 0; i < NV; ++i) { kxu[u][i] = make_uint4(0, 0, 0, 0); vxu[u][i] = kxu[u][i]; }
      if (validu[u]) {
        int blk = __ldg(p.block_table + (size_t)b * p.max_blocks + t / p.bt);
        blk = min(max(blk, 0), p.num_blocks - 1);
        const size_t row = ((size_t)blk * p.Hkv + hkv) * p.bt + (t % p.bt);
        const uint4* kp = reinterpret_cast<const uint4*>(p.k + row * LYNX_D + sl * DPL);
        const uint4* vp = reinterpret_cast<const uint4*>(p.v + row * LYNX_D + sl * DPL);
#pragma unroll
        for (int i = 0; i < NV; ++i) { kxu[u][i] = __ldg(kp + i); vxu[u][i] = __ldg(vp + i); }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
    const int t = t00 + u * TPP + grp;
    const bool valid = validu[u];
    const uint4 (&kx)[NV] = kxu[u];
    const uint4 (&vx)[NV] = vxu[u];
    // scores of this token for every column: partial over this lane's dims, then over the LPT lanes
    float s[COLS];
#pragma unroll
    for (int c = 0; c < COLS; ++c) s[c] = 0.0f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const uint32_t w[4] = {kx[i].x, kx[i].y, kx[i].z, kx[i].w};
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        const float lo = __uint_as_float(w[k2] << 16), hi = __uint_as_float(w[k2] & 0xFFFF0000u);
#pragma unroll
        for (int c = 0; c < COLS; ++c) s[c] = fmaf(q[c][i * 8 + 2 * k2 + 1], hi, fmaf(q[c][i * 8 + 2 * k2], lo, s[c]));
      }
    }
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
#pragma unroll
      for (int off = LPT / 2; off >= 1; off >>= 1) s[c] += __shfl_xor_sync(0xFFFFFFFFu, s[c], off);
      if (!valid || t >= lim[c]) s[c] = -INFINITY;
    }
    // online softmax of the token group, O accumulation
    float pw[COLS];
    bool grew = false;
#pragma unroll
    for (int c = 0; c < COLS; ++c) grew |= s[c] > m[c];
    if (__any_sync(0xFFFFFFFFu, grew)) {   // the running maxima rise rarely: rescale only then
#pragma unroll
      for (int c = 0; c < COLS; ++c) {
        const float mn = fmaxf(m[c], s[c]);
        const float f = ex2f(m[c] - mn);
        l[c] *= f;
        m[c] = mn;
#pragma unroll
        for (int d = 0; d < DPL; ++d) o[c][d] *= f;
      }
    }
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
      pw[c] = ex2f(s[c] - m[c]);
      l[c] += pw[c];
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const uint32_t w[4] = {vx[i].x, vx[i].y, vx[i].z, vx[i].w};
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        const float lo = __uint_as_float(w[k2] << 16), hi = __uint_as_float(w[k2] & 0xFFFF0000u);
#pragma unroll
        for (int c = 0; c < COLS; ++c) {
          o[c][i * 8 + 2 * k2] = fmaf(pw[c], lo, o[c][i * 8 + 2 * k2]);
          o[c][i * 8 + 2 * k2 + 1] = fmaf(pw[c], hi, o[c][i * 8 + 2 * k2 + 1]);
        }
      }
    }
  }
  }
  // merge the token groups of the warp (lanes with the same dim slice), then the warps through shared memory
#pragma unroll
  for (int off = LPT; off < 32; off <<= 1) {
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
      const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m[c], off), l2 = __shfl_xor_sync(0xFFFFFFFFu, l[c], off);
      const float mn = fmaxf(m[c], m2);
      const float f1 = ex2f(m[c] - mn), f2 = ex2f(m2 - mn);
      l[c] = l[c] * f1 + l2 * f2;
      m[c] = mn;
#pragma unroll
      for (int d = 0; d < DPL; ++d) o[c][d] = o[c][d] * f1 + __shfl_xor_sync(0xFFFFFFFFu, o[c][d], off) * f2;
    }
  }
  __shared__ float sm_o[kWarps][COLS][LYNX_D];
  __shared__ float sm_ml[kWarps][COLS][2];
  if (grp == 0) {
#pragma unroll
    for (int c = 0; c < COLS; ++c) {
#pragma unroll
      for (int d = 0; d < DPL; ++d) sm_o[warp][c][sl * DPL + d] = o[c][d];
      if (sl == 0) { sm_ml[warp][c][0] = m[c]; sm_ml[warp][c][1] = l[c]; }
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < COLS * LYNX_D; idx += kWarps * 32) {
    const int c = idx / LYNX_D, d = idx % LYNX_D;
    float M = -1.0e30f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_ml[w][c][0]);
    float acc = 0.0f, L = 0.0f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float f = ex2f(sm_ml[w][c][0] - M);
      acc = fmaf(sm_o[w][c][d], f, acc);
      L = fmaf(sm_ml[w][c][1], f, L);
    }
    part[(size_t)c * kPartStrideB + d] = acc;
    if (d == 0) { part[(size_t)c * kPartStrideB + 128] = M; part[(size_t)c * kPartStrideB + 129] = L; }
  }
}

// ---------------------------------------------------------------------------------------------------
// The same split-K decode on the BF16 tensor cores (mma.sync m16n8k16), for block sizes that are multiples
// of 16 tokens: with 8 columns the FP32 pipes above need more multiply-adds per byte than they have.
// A warp takes every fourth 16-token tile of the CTA's chunk: the tile's K and V rows (4 KB each, contiguous
// in a block) go through a three-stage cp.async ring of the warp's own in shared memory, 16-byte chunks
// XOR-swizzled by the row so that ldmatrix reads them without bank conflicts.
//   S[columns x 16 tokens] = Q K^T    A = Q (rows = query columns, 8 of 16 used), B = K rows as stored
//   O[columns x 128 dims] += P V      A = P (the S accumulators, exponentiated, as BF16 pairs), B = V rows
//                                     through ldmatrix.trans
// The weights enter P.V as two BF16 terms (p = hi + lo, the remainder of the rounding): with one term their
// 8-bit mantissa would show in the outputs.
constexpr int kTcWarps = 4, kTcStages = 3, kTcTile = 16;
constexpr int kTcStageBytes = 2 * kTcTile * 256;   // K rows, then V rows

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t bf16x2_of(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

template <int COLS>
__global__ void __launch_bounds__(kTcWarps * 32, 2) bf16_decode_tc_kernel(const BfParams p) {
  extern __shared__ __align__(128) unsigned char smem_tc[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int chunk = blockIdx.x % p.chunks, bh = blockIdx.x / p.chunks;
  const int b = bh / p.Hkv, hkv = bh % p.Hkv;
  const int cap = p.max_blocks * p.bt;
  int len = __ldg(p.seq_lens + b);
  len = len < 0 ? 0 : (len > cap ? cap : len);
  float* part = p.part + ((size_t)bh * p.chunks + chunk) * (size_t)COLS * kPartStrideB;
  const int t_begin = chunk * kChunk, t_end = min(len, t_begin + kChunk);
  const int n_tiles = t_end > t_begin ? (t_end - t_begin + kTcTile - 1) / kTcTile : 0;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(smem_tc) + (uint32_t)warp * kTcStages * kTcStageBytes;

  // Q fragments: row g = column g (rows 8..15 of the tile are zero), k = dims
  uint32_t qa[8][2];
  int lim = 0;
  {
    const int c = g, j = c / p.G, hh = c % p.G;
    const bool in = c < p.ncols;
    lim = in ? (p.causal ? len - p.tail + j + 1 : len) : 0;
    const uint32_t* qp = reinterpret_cast<const uint32_t*>(
        p.q + (((size_t)b * p.nq_stride + (in ? j : 0)) * p.Hq + hkv * p.G + (in ? hh : 0)) * LYNX_D);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = in ? __ldg(qp + 8 * ks + t) : 0u;
      qa[ks][1] = in ? __ldg(qp + 8 * ks + 4 + t) : 0u;
    }
  }
  float o[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) { o[j][0] = 0.f; o[j][1] = 0.f; o[j][2] = 0.f; o[j][3] = 0.f; }
  float m = -1.0e30f, l = 0.0f;

  // tile i of this warp = tile warp + 4 i of the chunk; its rows: 16 consecutive rows of one block
  auto issue = [&](int i) {
    const int tile = warp + kTcWarps * i;
    if (tile < n_tiles) {
      const int t0 = t_begin + tile * kTcTile;
      int blk = __ldg(p.block_table + (size_t)b * p.max_blocks + t0 / p.bt);
      blk = min(max(blk, 0), p.num_blocks - 1);
      const size_t row0 = ((size_t)blk * p.Hkv + hkv) * p.bt + (t0 % p.bt);
      const uint32_t st = ring + (uint32_t)(i % kTcStages) * kTcStageBytes;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int idx = lane + 32 * k, row = idx >> 4, c = idx & 15;
        const uint32_t dst = (uint32_t)(row * 256 + ((c ^ (row & 7)) << 4));
        const uint32_t sz = t0 + row < len ? 16u : 0u;   // rows past the end of the sequence are zero-filled
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(st + dst),
                     "l"(p.k + (row0 + row) * LYNX_D + c * 8), "r"(sz) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(st + kTcTile * 256 + dst),
                     "l"(p.v + (row0 + row) * LYNX_D + c * 8), "r"(sz) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  const int my_tiles = n_tiles > warp ? (n_tiles - warp + kTcWarps - 1) / kTcWarps : 0;
  issue(0);
  issue(1);
  for (int i = 0; i < my_tiles; ++i) {
    issue(i + 2);
    asm volatile("cp.async.wait_group 2;" ::: "memory");
    __syncwarp();
    const uint32_t st = ring + (uint32_t)(i % kTcStages) * kTcStageBytes;
    const int t0 = t_begin + (warp + kTcWarps * i) * kTcTile;
    // ---- S = Q K^T: two n-tiles of 8 tokens, eight k-steps of 16 dims
    float s[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      s[j][0] = 0.f; s[j][1] = 0.f; s[j][2] = 0.f; s[j][3] = 0.f;
      const int tok = 8 * j + (lane & 7), mi = lane >> 3;   // ldmatrix: this lane's row of matrix mi
#pragma unroll
      for (int kp = 0; kp < 4; ++kp) {   // pairs of k-steps
        uint32_t kb[4];
        ldsm4(st + (uint32_t)(tok * 256 + (((4 * kp + mi) ^ (tok & 7)) << 4)), kb);
        const uint32_t a0[4] = {qa[2 * kp][0], 0u, qa[2 * kp][1], 0u};
        const uint32_t a1[4] = {qa[2 * kp + 1][0], 0u, qa[2 * kp + 1][1], 0u};
        mma_bf16(s[j], a0, kb[0], kb[1]);
        mma_bf16(s[j], a1, kb[2], kb[3]);
      }
    }
    // ---- online softmax of row g (column g) over the tile's 16 tokens
    float x[4];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int tk = t0 + 8 * j + 2 * t + e;
        x[2 * j + e] = tk < lim ? s[j][e] * p.sm_log2 : -INFINITY;
        mx = fmaxf(mx, x[2 * j + e]);
      }
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
    if (__any_sync(0xFFFFFFFFu, mx > m)) {
      const float mn = fmaxf(m, mx), f = ex2f(m - mn);
      l *= f;
      m = mn;
#pragma unroll
      for (int j = 0; j < 16; ++j) { o[j][0] *= f; o[j][1] *= f; }
    }
    uint32_t ph[4] = {0u, 0u, 0u, 0u}, pl[4] = {0u, 0u, 0u, 0u};   // P as A fragments: hi and lo terms
    {
      float pw[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) { pw[k] = ex2f(x[k] - m); l += pw[k]; }
      ph[0] = bf16x2_of(pw[0], pw[1]);
      ph[2] = bf16x2_of(pw[2], pw[3]);
      const float r0 = pw[0] - __uint_as_float(ph[0] << 16), r1 = pw[1] - __uint_as_float(ph[0] & 0xFFFF0000u);
      const float r2 = pw[2] - __uint_as_float(ph[2] << 16), r3 = pw[3] - __uint_as_float(ph[2] & 0xFFFF0000u);
      pl[0] = bf16x2_of(r0, r1);
      pl[2] = bf16x2_of(r2, r3);
    }
    // ---- O += P V: sixteen n-tiles of 8 dims, one k-step of 16 tokens
    {
      const int tok = 8 * ((lane >> 3) & 1) + (lane & 7), cj = lane >> 4;
#pragma unroll
      for (int jp = 0; jp < 8; ++jp) {   // pairs of n-tiles
        uint32_t vb[4];
        ldsm4_t(st + kTcTile * 256 + (uint32_t)(tok * 256 + (((2 * jp + cj) ^ (tok & 7)) << 4)), vb);
        mma_bf16(o[2 * jp], ph, vb[0], vb[1]);
        mma_bf16(o[2 * jp], pl, vb[0], vb[1]);
        mma_bf16(o[2 * jp + 1], ph, vb[2], vb[3]);
        mma_bf16(o[2 * jp + 1], pl, vb[2], vb[3]);
      }
    }
    __syncwarp();   // the stage is rewritten two iterations from now
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 1);
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 2);
  // the warps' partial results through shared memory (the ring is idle now), then the chunk's partial
  __syncthreads();
  float* sm_o = reinterpret_cast<float*>(smem_tc);                    // [warps][COLS][128]
  float* sm_ml = sm_o + kTcWarps * COLS * LYNX_D;                     // [warps][COLS][2]
  if (g < COLS) {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      sm_o[(warp * COLS + g) * LYNX_D + 8 * j + 2 * t] = o[j][0];
      sm_o[(warp * COLS + g) * LYNX_D + 8 * j + 2 * t + 1] = o[j][1];
    }
    if (t == 0) { sm_ml[(warp * COLS + g) * 2] = m; sm_ml[(warp * COLS + g) * 2 + 1] = l; }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < COLS * LYNX_D; idx += kTcWarps * 32) {
    const int c = idx / LYNX_D, d = idx % LYNX_D;
    float M = -1.0e30f;
#pragma unroll
    for (int w = 0; w < kTcWarps; ++w) M = fmaxf(M, sm_ml[(w * COLS + c) * 2]);
    float acc = 0.0f, L = 0.0f;
#pragma unroll
    for (int w = 0; w < kTcWarps; ++w) {
      const float f = ex2f(sm_ml[(w * COLS + c) * 2] - M);
      acc = fmaf(sm_o[(w * COLS + c) * LYNX_D + d], f, acc);
      L = fmaf(sm_ml[(w * COLS + c) * 2 + 1], f, L);
    }
    part[(size_t)c * kPartStrideB + d] = acc;
    if (d == 0) { part[(size_t)c * kPartStrideB + 128] = M; part[(size_t)c * kPartStrideB + 129] = L; }
  }
}

// One CTA per (sequence, KV head, column): merges the chunk partials, normalises, writes the output.
template <int COLS>
__global__ void __launch_bounds__(LYNX_D) bf16_combine_kernel(const BfParams p) {
  const int c = blockIdx.x % COLS, bh = blockIdx.x / COLS;
  if (c >= p.ncols) return;
  const int b = bh / p.Hkv, hkv = bh % p.Hkv, d = threadIdx.x;
  const int cap = p.max_blocks * p.bt;
  int len = __ldg(p.seq_lens + b);
  len = len < 0 ? 0 : (len > cap ? cap : len);
  const int n = (len + kChunk - 1) / kChunk;
  const float* part = p.part + (size_t)bh * p.chunks * (size_t)COLS * kPartStrideB + (size_t)c * kPartStrideB;
  float M = -1.0e30f, L = 0.0f, acc = 0.0f;
  constexpr int kAhead = 8;   // partials whose loads are issued together (one L2 round trip per batch, not per chunk)
  for (int i0 = 0; i0 < n; i0 += kAhead) {
    float mi[kAhead], li[kAhead], oi[kAhead];
#pragma unroll
    for (int u = 0; u < kAhead; ++u) {
      const bool in = i0 + u < n;
      const float* src = part + (size_t)(in ? i0 + u : i0) * COLS * kPartStrideB;
      mi[u] = in ? src[128] : -1.0e30f;
      li[u] = in ? src[129] : 0.0f;
      oi[u] = in ? src[d] : 0.0f;
    }
#pragma unroll
    for (int u = 0; u < kAhead; ++u) {
      const float mn = fmaxf(M, mi[u]);
      const float fa = ex2f(M - mn), fb = ex2f(mi[u] - mn);
      acc = acc * fa + oi[u] * fb;
      L = L * fa + li[u] * fb;
      M = mn;
    }
  }
  const int j = c / p.G, hh = c % p.G;
  p.out[(((size_t)b * p.nq_stride + j) * p.Hq + hkv * p.G + hh) * LYNX_D + d] = L > 0.0f ? acc / L : 0.0f;
  if (d == 0) p.lse[((size_t)b * p.nq_stride + j) * p.Hq + hkv * p.G + hh] = L > 0.0f ? (M + __log2f(L)) * 0.6931471805599453f : -INFINITY;
}

template <int COLS, int LPT>
lynx_status launch_bf16(const BfParams& p, cudaStream_t st) {
  bf16_decode_kernel<COLS, LPT><<<(unsigned)(p.B * p.Hkv * p.chunks), kWarps * 32, 0, st>>>(p);
  lynx_status rc = launch_status();
  if (rc != LYNX_OK) return rc;
  bf16_combine_kernel<COLS><<<(unsigned)(p.B * p.Hkv * COLS), LYNX_D, 0, st>>>(p);
  return launch_status();
}

template <int COLS>
lynx_status launch_bf16_tc(const BfParams& p, cudaStream_t st) {
  constexpr int kSmem = kTcWarps * kTcStages * kTcStageBytes;   // 96 KB: two CTAs per SM
  static_assert(kSmem >= (int)((kTcWarps * COLS * LYNX_D + kTcWarps * COLS * 2) * sizeof(float)), "merge scratch");
  auto kern = bf16_decode_tc_kernel<COLS>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess) return LYNX_ERR_CUDA;
    configured[dev] = true;
  }
  kern<<<(unsigned)(p.B * p.Hkv * p.chunks), kTcWarps * 32, kSmem, st>>>(p);
  lynx_status rc = launch_status();
  if (rc != LYNX_OK) return rc;
  bf16_combine_kernel<COLS><<<(unsigned)(p.B * p.Hkv * COLS), LYNX_D, 0, st>>>(p);
  return launch_status();
}

// bytes of the chunk partials, rounded up to 256: the log-sum-exps follow them in the workspace
size_t bf16_part_bytes(const lynx_shape* s, int B, int ncols, int chunks) {
  const int cols_pad = ncols <= 1 ? 1 : ncols <= 2 ? 2 : ncols <= 4 ? 4 : 8;
  const size_t b = (size_t)B * s->num_kv_heads * chunks * cols_pad * kPartStrideB * sizeof(float);
  return (b + 255) & ~(size_t)255;
}

bool bf16_shape_ok(const lynx_shape* s, int B, int nq, int* ncols, int* chunks) {
  if (!s || s->head_dim != LYNX_D || s->num_kv_heads <= 0 || s->num_q_heads <= 0 ||
      s->num_q_heads % s->num_kv_heads != 0 || s->block_tokens <= 0 || s->num_blocks <= 0 ||
      s->max_blocks_per_seq <= 0 || B <= 0 || nq <= 0)
    return false;
  const int G = s->num_q_heads / s->num_kv_heads;
  if (G > 8 || nq > 64) return false;
  const int64_t cap = (int64_t)s->max_blocks_per_seq * s->block_tokens;
  if (cap >= (1ll << 31) || (int64_t)B * s->num_kv_heads * ((cap + kChunk - 1) / kChunk) >= (1ll << 31)) return false;
  *ncols = nq * G <= 8 ? nq * G : (8 / G) * G;   // columns of the widest launch: whole positions, 8 columns at most
  *chunks = (int)((cap + kChunk - 1) / kChunk);
  return true;
}

}  // namespace
}  // namespace lynx

extern "C" size_t lynx_bf16_workspace_bytes(const lynx_shape* shape, int32_t batch, int32_t n_q) {
  int ncols = 0, chunks = 0;
  if (!lynx::bf16_shape_ok(shape, batch, n_q, &ncols, &chunks)) return 0;
  return lynx::bf16_part_bytes(shape, batch, ncols, chunks) + (size_t)batch * n_q * shape->num_q_heads * sizeof(float);
}

extern "C" const float* lynx_bf16_workspace_lse(const lynx_shape* shape, int32_t batch, int32_t n_q, const void* workspace) {
  int ncols = 0, chunks = 0;
  if (!workspace || !lynx::bf16_shape_ok(shape, batch, n_q, &ncols, &chunks)) return nullptr;
  return reinterpret_cast<const float*>(static_cast<const unsigned char*>(workspace) +
                                        lynx::bf16_part_bytes(shape, batch, ncols, chunks));
}

extern "C" lynx_status lynx_bf16_attention(const lynx_shape* shape, const void* q_bf16, int32_t batch, int32_t n_q,
                                           int32_t causal, const void* k_pages_bf16, const void* v_pages_bf16,
                                           const int32_t* block_table, const int32_t* seq_lens,
                                           float softmax_scale, float* out, void* workspace,
                                           size_t workspace_bytes, void* stream) {
  using namespace lynx;
  if (batch == 0) return LYNX_OK;
  if (!shape) return LYNX_ERR_NULL;
  if (batch < 0 || n_q <= 0) return LYNX_ERR_SHAPE;
  BfParams p;
  if (!bf16_shape_ok(shape, batch, n_q, &p.ncols, &p.chunks)) return LYNX_ERR_UNSUPPORTED;
  if (!q_bf16 || !k_pages_bf16 || !v_pages_bf16 || !block_table || !seq_lens || !out || !workspace) return LYNX_ERR_NULL;
  if (!aligned16(q_bf16) || !aligned16(k_pages_bf16) || !aligned16(v_pages_bf16) || !aligned16(out) || !aligned16(workspace))
    return LYNX_ERR_ALIGN;
  if (workspace_bytes < lynx_bf16_workspace_bytes(shape, batch, n_q)) return LYNX_ERR_WORKSPACE;
  p.q = static_cast<const __nv_bfloat16*>(q_bf16);
  p.k = static_cast<const __nv_bfloat16*>(k_pages_bf16);
  p.v = static_cast<const __nv_bfloat16*>(v_pages_bf16);
  p.block_table = block_table; p.seq_lens = seq_lens; p.out = out;
  p.part = static_cast<float*>(workspace);
  p.lse = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + bf16_part_bytes(shape, batch, p.ncols, p.chunks));
  const float sc = softmax_scale == 0.0f ? 0.08838834764831845f : softmax_scale;
  p.sm_log2 = sc * 1.4426950408889634f;
  p.B = batch; p.nq = n_q; p.causal = causal ? 1 : 0;
  p.Hq = shape->num_q_heads; p.Hkv = shape->num_kv_heads; p.G = p.Hq / p.Hkv;
  p.bt = shape->block_tokens; p.num_blocks = shape->num_blocks; p.max_blocks = shape->max_blocks_per_seq;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // a launch takes up to 8 query columns; a call with more runs as slices of whole positions, each a pass of its
  // own over the pages, one after the other on the stream (they share the partials)
  const int per = n_q * p.G <= 8 ? n_q : 8 / p.G;
  for (int j0 = 0; j0 < n_q; j0 += per) {
    BfParams ps = p;
    ps.nq = n_q - j0 < per ? n_q - j0 : per;
    ps.ncols = ps.nq * p.G;
    ps.nq_stride = n_q;
    ps.tail = n_q - j0;
    ps.q = p.q + (size_t)j0 * p.Hq * LYNX_D;
    ps.out = p.out + (size_t)j0 * p.Hq * LYNX_D;
    ps.lse = p.lse + (size_t)j0 * p.Hq;
    lynx_status rc;
    if (p.bt % 16 == 0) {   // the tensor-core kernel (tiles of 16 tokens inside a block)
      rc = ps.ncols <= 1 ? launch_bf16_tc<1>(ps, st) : ps.ncols <= 2 ? launch_bf16_tc<2>(ps, st)
         : ps.ncols <= 4 ? launch_bf16_tc<4>(ps, st) : launch_bf16_tc<8>(ps, st);
    } else {
      rc = ps.ncols <= 1 ? launch_bf16<1, 8>(ps, st) : ps.ncols <= 2 ? launch_bf16<2, 8>(ps, st)
         : ps.ncols <= 4 ? launch_bf16<4, 16>(ps, st) : launch_bf16<8, 16>(ps, st);
    }
    if (rc != LYNX_OK) return rc;
  }
  return LYNX_OK;
}
