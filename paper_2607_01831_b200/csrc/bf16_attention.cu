// lynx_bf16_attention: decode attention over dequantised BF16 KV pages (sm_100a).
//
// The paper's own decode path (Section 4.2): the dequantisation kernel scatters BF16 pages into the
// paged KV memory and the engine's stock attention reads them, 256 bytes per row of K or V.  This is
// that second half, hand-written, as the baseline the fused kernels (72 / 136 bytes per row) are
// measured against: softmax(q K^T scale) V of Section 2 on pages [num_blocks][Hkv][block_tokens][128]
// BF16, as lynx_recombine writes them.
//
// The kernel is HBM-bound by construction (no reuse beyond the n_q * G query columns of a KV head) and
// small enough in arithmetic for the FP32 pipes: 8 (or 16) lanes own a token, each 16 (8) of its 128
// dims, so every row is read with fully used 128-bit loads; the partial dot products are reduced with
// shuffles, the softmax is online per token group, and O is accumulated in registers.  Flash-decoding
// split-K: a CTA takes a chunk of kChunk tokens of one (sequence, KV head) and writes a partial
// (m, l, O) to the workspace; a second kernel merges the chunks.  Nothing waits on anything.
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
  float sm_log2;
  int B, nq, causal, Hq, Hkv, G, bt, num_blocks, max_blocks, ncols, chunks;
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
    lim[c] = in ? (p.causal ? len - p.nq + j + 1 : len) : 0;
    const __nv_bfloat16* qp = p.q + (((size_t)b * p.nq + (in ? j : 0)) * p.Hq + hkv * p.G + (in ? hh : 0)) * LYNX_D + sl * DPL;
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
  for (int i = 0; i < n; ++i) {
    const float* src = part + (size_t)i * COLS * kPartStrideB;
    const float mi = src[128], li = src[129], oi = src[d];
    const float mn = fmaxf(M, mi);
    const float fa = ex2f(M - mn), fb = ex2f(mi - mn);
    acc = acc * fa + oi * fb;
    L = L * fa + li * fb;
    M = mn;
  }
  const int j = c / p.G, hh = c % p.G;
  p.out[(((size_t)b * p.nq + j) * p.Hq + hkv * p.G + hh) * LYNX_D + d] = L > 0.0f ? acc / L : 0.0f;
}

template <int COLS, int LPT>
lynx_status launch_bf16(const BfParams& p, cudaStream_t st) {
  bf16_decode_kernel<COLS, LPT><<<(unsigned)(p.B * p.Hkv * p.chunks), kWarps * 32, 0, st>>>(p);
  lynx_status rc = launch_status();
  if (rc != LYNX_OK) return rc;
  bf16_combine_kernel<COLS><<<(unsigned)(p.B * p.Hkv * COLS), LYNX_D, 0, st>>>(p);
  return launch_status();
}

bool bf16_shape_ok(const lynx_shape* s, int B, int nq, int* ncols, int* chunks) {
  if (!s || s->head_dim != LYNX_D || s->num_kv_heads <= 0 || s->num_q_heads <= 0 ||
      s->num_q_heads % s->num_kv_heads != 0 || s->block_tokens <= 0 || s->num_blocks <= 0 ||
      s->max_blocks_per_seq <= 0 || B <= 0 || nq <= 0)
    return false;
  const int G = s->num_q_heads / s->num_kv_heads;
  if ((int64_t)nq * G > 8) return false;
  const int64_t cap = (int64_t)s->max_blocks_per_seq * s->block_tokens;
  if (cap >= (1ll << 31) || (int64_t)B * s->num_kv_heads * ((cap + kChunk - 1) / kChunk) >= (1ll << 31)) return false;
  *ncols = nq * G;
  *chunks = (int)((cap + kChunk - 1) / kChunk);
  return true;
}

}  // namespace
}  // namespace lynx

extern "C" size_t lynx_bf16_workspace_bytes(const lynx_shape* shape, int32_t batch, int32_t n_q) {
  int ncols = 0, chunks = 0;
  if (!lynx::bf16_shape_ok(shape, batch, n_q, &ncols, &chunks)) return 0;
  const int cols_pad = ncols <= 1 ? 1 : ncols <= 2 ? 2 : ncols <= 4 ? 4 : 8;
  return (size_t)batch * shape->num_kv_heads * chunks * cols_pad * lynx::kPartStrideB * sizeof(float);
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
  const float sc = softmax_scale == 0.0f ? 0.08838834764831845f : softmax_scale;
  p.sm_log2 = sc * 1.4426950408889634f;
  p.B = batch; p.nq = n_q; p.causal = causal ? 1 : 0;
  p.Hq = shape->num_q_heads; p.Hkv = shape->num_kv_heads; p.G = p.Hq / p.Hkv;
  p.bt = shape->block_tokens; p.num_blocks = shape->num_blocks; p.max_blocks = shape->max_blocks_per_seq;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (p.ncols <= 1) return launch_bf16<1, 8>(p, st);
  if (p.ncols <= 2) return launch_bf16<2, 8>(p, st);
  if (p.ncols <= 4) return launch_bf16<4, 16>(p, st);
  return launch_bf16<8, 16>(p, st);
}
