/*
 * CPU oracle for the Lynx split-stream quantisation hot path.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, obviously-correct
 * restatement of what the path computes, used only to check the CUDA library
 * (tests, the smoke check, and the benchmark's timed CPU baseline).  It shares
 * no code, header, table or constant with the CUDA sources and the product
 * never calls it.
 *
 * What it follows in the paper:
 *   - linear grouped quantisation Q(X) = round(X/S + Z), S from the group's
 *     min-max range (Section 2.3, "Standard & Grouped Quantization");
 *   - the 8-bit code is split into its top 4 bits (Anchor stream) and bottom
 *     4 bits (Residual stream), INT4 + INT4 = INT8 (Section 4.1 stage 4 and
 *     the Conclusion); two 4-bit values are packed per byte, each stream in a
 *     contiguous buffer, scalars travelling with the Anchor stream
 *     (Section "Implementation", Compression Kernel);
 *   - attention O = softmax(Q K^T / sqrt(d_k)) V (Section 2, un-numbered
 *     equation) evaluated on the Anchor-only state (Section 4.2, Anchor Phase)
 *     and on the refined full state Q_full (Section 4.2, Residual Phase);
 *   - verification: one parallel pass over the speculated positions on Q_full,
 *     accept the longest agreeing prefix (Section 4.3).
 *
 * Readings taken where the paper is silent (group = one token's 128-element
 * head vector, unsigned codes, real-valued zero point, tie rule, nibble
 * order, bucket mid-point for the Anchor-only value, attention-level
 * agreement test) are listed in the design notes of the repository; each
 * function below states the one it uses.
 *
 * Arithmetic: quantisation in IEEE binary32 exactly as stated (one rounding
 * per stated operation; the code is the round-half-even of the EXACT product);
 * attention and the agreement test in binary64.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (no fast-math).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define LYNX_D 128 /* head_dim = quantisation group size */

static float bf16_to_f32(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* binary32 -> bfloat16, round to nearest even (finite inputs). */
static uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------------
 * Split quantisation of n_rows rows of 128 BF16 values (Section 2.3 linear
 * grouped quantisation; Section 4.1 stage 4 bit split; packing as in the
 * Compression Kernel paragraph).
 *
 * Per row:  mn = min, mx = max;  range = fl(mx - mn);
 *           scale = fl(range / 255), inv = fl(255 / range), zero = mn (+0);
 *           a row whose range is below 2^-100 is treated as constant:
 *           scale = 0, inv = 0, every code 0.
 *           u = fl(x - mn);  code = round_half_even(u * inv) exactly, clamped
 *           to [0, 255];  a = code >> 4;  r = code & 15.
 * Byte j of the Anchor row holds a[2j] in its low nibble and a[2j+1] in its
 * high nibble; the Residual row likewise.  meta[row] = {scale, zero}.
 * codes (optional, may be NULL) receives the unsplit 8-bit codes.
 * ---------------------------------------------------------------------- */
void lynx_oracle_split_quantize(const uint16_t* src_bf16, int64_t n_rows,
                                uint8_t* anchor, uint8_t* residual, float* meta,
                                uint8_t* codes) {
#pragma omp parallel for schedule(static)
  for (int64_t row = 0; row < n_rows; ++row) {
    const uint16_t* x = src_bf16 + row * LYNX_D;
    float v[LYNX_D];
    float mn = bf16_to_f32(x[0]), mx = mn;
    for (int d = 0; d < LYNX_D; ++d) {
      v[d] = bf16_to_f32(x[d]);
      if (v[d] < mn) mn = v[d];
      if (v[d] > mx) mx = v[d];
    }
    float range = mx - mn;
    float scale = 0.0f, inv = 0.0f;
    if (range >= 0x1p-100f) {
      scale = range / 255.0f;
      inv = 255.0f / range;
    }
    float zero = mn + 0.0f; /* -0 becomes +0 */
    meta[row * 2 + 0] = scale;
    meta[row * 2 + 1] = zero;
    uint8_t c[LYNX_D];
    for (int d = 0; d < LYNX_D; ++d) {
      float u = v[d] - mn;
      double prod = (double)u * (double)inv; /* exact: 24 x 24 bit product */
      double rn = nearbyint(prod);           /* default mode: half to even */
      if (rn < 0.0) rn = 0.0;
      if (rn > 255.0) rn = 255.0;
      c[d] = (uint8_t)rn;
      if (codes) codes[row * LYNX_D + d] = c[d];
    }
    for (int j = 0; j < LYNX_D / 2; ++j) {
      uint8_t lo = c[2 * j], hi = c[2 * j + 1];
      anchor[row * 64 + j] = (uint8_t)((lo >> 4) | ((hi >> 4) << 4));
      residual[row * 64 + j] = (uint8_t)((lo & 15) | ((hi & 15) << 4));
    }
  }
}

/* ------------------------------------------------------------------------
 * Recombine (Section 4.2 Residual Phase: the Residual stream refines the
 * state to full precision Q_full).  code = (a << 4) | r.  Optional outputs:
 * codes [n_rows][128] u8 and the dequantised value rounded to BF16,
 * x_hat = bf16_rne(fl(code * scale + zero)) with the multiply-add rounded once.
 * ---------------------------------------------------------------------- */
void lynx_oracle_recombine(const uint8_t* anchor, const uint8_t* residual,
                           const float* meta, int64_t n_rows, uint8_t* codes,
                           uint16_t* dequant_bf16) {
#pragma omp parallel for schedule(static)
  for (int64_t row = 0; row < n_rows; ++row) {
    float scale = meta[row * 2 + 0], zero = meta[row * 2 + 1];
    for (int d = 0; d < LYNX_D; ++d) {
      uint8_t ab = anchor[row * 64 + d / 2], rb = residual[row * 64 + d / 2];
      int a = (d & 1) ? (ab >> 4) : (ab & 15);
      int r = (d & 1) ? (rb >> 4) : (rb & 15);
      int code = (a << 4) | r;
      if (codes) codes[row * LYNX_D + d] = (uint8_t)code;
      if (dequant_bf16)
        dequant_bf16[row * LYNX_D + d] = f32_to_bf16_rne(fmaf((float)code, scale, zero));
    }
  }
}

/* Integer level of element d of a plane row: the Anchor-only state uses the
 * mid-point of the 16-wide bucket (16 a + 8); the full state uses 16 a + r. */
static double level(const uint8_t* anchor_row, const uint8_t* residual_row, int d, int full) {
  uint8_t ab = anchor_row[d / 2];
  int a = (d & 1) ? (ab >> 4) : (ab & 15);
  if (!full) return (double)(16 * a + 8);
  uint8_t rb = residual_row[d / 2];
  int r = (d & 1) ? (rb >> 4) : (rb & 15);
  return (double)(16 * a + r);
}

/* ------------------------------------------------------------------------
 * Decode attention over quantised, paged K and V (Section 2 attention
 * equation; Section 4.2 Anchor / Residual phases), in binary64.
 *
 * Plane layout: anchor/residual [num_blocks][Hkv][block_tokens][64] bytes,
 * meta [num_blocks][Hkv][block_tokens][2] floats.  Token t of sequence b is
 * row t % block_tokens of block block_table[b][t / block_tokens].
 * q is BF16 [B][n_q][Hq][128]; query head h reads KV head h / (Hq / Hkv).
 * x_hat = zero + scale * level.  score = (q . K_hat) * softmax_scale;
 * softmax with max subtraction over the visible tokens;  O = sum p V_hat.
 * causal != 0: query j sees tokens [0, len - n_q + j + 1); else [0, len).
 * A query that sees no token gets an all-zero output.
 * out: binary64 [B][n_q][Hq][128].
 * ---------------------------------------------------------------------- */
void lynx_oracle_attention(int full, int32_t Hq, int32_t Hkv, int32_t block_tokens,
                           int32_t max_blocks_per_seq, const uint16_t* q_bf16, int32_t B,
                           int32_t n_q, int32_t causal, const uint8_t* k_anchor,
                           const uint8_t* k_residual, const float* k_meta,
                           const uint8_t* v_anchor, const uint8_t* v_residual,
                           const float* v_meta, const int32_t* block_table,
                           const int32_t* seq_lens, float softmax_scale, double* out) {
  const int G = Hq / Hkv;
  const double sm = (double)softmax_scale;
  const int64_t n_prob = (int64_t)B * n_q * Hq;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t prob = 0; prob < n_prob; ++prob) {
    const int h = (int)(prob % Hq);
    const int j = (int)((prob / Hq) % n_q);
    const int b = (int)(prob / ((int64_t)Hq * n_q));
    const int hkv = h / G;
    const int len = seq_lens[b];
    int64_t vis = causal ? (int64_t)len - n_q + j + 1 : (int64_t)len;
    double* o = out + prob * LYNX_D;
    for (int d = 0; d < LYNX_D; ++d) o[d] = 0.0;
    if (vis <= 0) continue;
    double qv[LYNX_D];
    for (int d = 0; d < LYNX_D; ++d) qv[d] = (double)bf16_to_f32(q_bf16[prob * LYNX_D + d]);
    double* s = (double*)malloc(sizeof(double) * (size_t)vis);
    /* pass 1: scores and their maximum */
    double smax = -INFINITY;
    for (int64_t t = 0; t < vis; ++t) {
      int64_t blk = block_table[(int64_t)b * max_blocks_per_seq + t / block_tokens];
      int64_t row = (blk * Hkv + hkv) * block_tokens + t % block_tokens;
      double scale = (double)k_meta[row * 2], zero = (double)k_meta[row * 2 + 1];
      const uint8_t* ar = k_anchor + row * 64;
      const uint8_t* rr = full ? k_residual + row * 64 : NULL;
      double dot = 0.0;
      for (int d = 0; d < LYNX_D; ++d) dot += qv[d] * (zero + scale * level(ar, rr, d, full));
      s[t] = dot * sm;
      if (s[t] > smax) smax = s[t];
    }
    /* pass 2: weights and weighted sum of V_hat */
    double denom = 0.0;
    for (int64_t t = 0; t < vis; ++t) {
      double p = exp(s[t] - smax);
      denom += p;
      int64_t blk = block_table[(int64_t)b * max_blocks_per_seq + t / block_tokens];
      int64_t row = (blk * Hkv + hkv) * block_tokens + t % block_tokens;
      double scale = (double)v_meta[row * 2], zero = (double)v_meta[row * 2 + 1];
      const uint8_t* ar = v_anchor + row * 64;
      const uint8_t* rr = full ? v_residual + row * 64 : NULL;
      for (int d = 0; d < LYNX_D; ++d) o[d] += p * (zero + scale * level(ar, rr, d, full));
    }
    for (int d = 0; d < LYNX_D; ++d) o[d] /= denom;
    free(s);
  }
}

/* ------------------------------------------------------------------------
 * Accept / reject over k speculated positions (Section 4.3: accept the
 * longest prefix, the first divergence is corrected by the full result).
 * Attention-level agreement test (a reading; the paper verifies tokens):
 *   dev[b][j] = max over heads h and dims d of
 *               |O_full - O_draft| / (atol + rtol * |O_full|)
 *   first_reject[b] = smallest j with dev[b][j] > 1, or k when none.
 * out_full is binary64 [B][k][Hq][128]; draft is binary32, same shape.
 * ---------------------------------------------------------------------- */
void lynx_oracle_verify_decision(const double* out_full, const float* draft, int32_t B,
                                 int32_t k, int32_t Hq, double atol, double rtol,
                                 int32_t* first_reject, double* dev) {
  for (int b = 0; b < B; ++b) {
    int32_t fr = k;
    for (int j = k - 1; j >= 0; --j) {
      double worst = 0.0;
      int64_t base = ((int64_t)b * k + j) * Hq * LYNX_D;
      for (int64_t e = 0; e < (int64_t)Hq * LYNX_D; ++e) {
        double f = out_full[base + e], g = (double)draft[base + e];
        double r = fabs(f - g) / (atol + rtol * fabs(f));
        if (r > worst) worst = r;
      }
      dev[(int64_t)b * k + j] = worst;
      if (worst > 1.0) fr = j;
    }
    first_reject[b] = fr;
  }
}

int lynx_oracle_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp master
    n = omp_get_num_threads();
  }
#endif
  return n;
}
