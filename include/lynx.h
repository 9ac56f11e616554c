/*
 * lynx.h -- C interface of the B200 (sm_100a) library for the data-parallel hot path of
 * Lynx's progressive speculative quantisation of the KV cache.
 *
 * The path (paper sections in brackets):
 *   1. split-quantise: BF16 K or V rows -> 8-bit linear per-group codes (Section 2.3,
 *      "Standard & Grouped Quantization": Q(X) = round(X/S + Z), S from the group's min-max
 *      range) split into an Anchor plane (top 4 bits) and a Residual plane (bottom 4 bits),
 *      two 4-bit values per byte, each stream contiguous, the scalars travelling with the
 *      Anchor stream (Section 4.1 stage 4; Section "Implementation", Compression Kernel).
 *   2. anchor attention: decode attention softmax(Q K^T / sqrt(d)) V (Section 2) evaluated on
 *      the Anchor plane alone, which is what the decode instance has when it starts drafting
 *      (Section 4.2, Anchor Phase).
 *   3. merge-verify attention: Anchor and Residual recombined into the full 8-bit state
 *      Q_full (Section 4.2, Residual Phase), the k drafted positions scored in one pass and the
 *      longest agreeing prefix reported (Section 4.3).
 *   4. recombine: the stand-alone Residual-phase refinement to full codes / BF16 pages.
 *
 * Group = one token's head vector of 128 elements (a "row").  Per row:
 *   mn = min, mx = max, range = fl(mx - mn), scale = fl(range/255), inv = fl(255/range),
 *   zero = mn (with -0 stored as +0); range < 2^-100 -> scale = inv = 0 (constant row);
 *   code = round-half-even of the exact product fl(x - mn) * inv, in [0, 255];
 *   anchor nibble a = code >> 4, residual nibble r = code & 15;
 *   byte j of a plane row = nibble of element 2j (low half) | nibble of element 2j+1 << 4.
 * Reconstruction: full state x^ = zero + scale * (16 a + r); Anchor-only state
 * x^ = zero + scale * (16 a + 8) (bucket mid-point).  Inputs must be finite.
 *
 * Memory layout of a quantised K (or V) cache of one layer, paged:
 *   anchor, residual : uint8 [num_blocks][num_kv_heads][block_tokens][64]
 *   meta             : float [num_blocks][num_kv_heads][block_tokens][2] = {scale, zero}
 * Token t of sequence b lives in row (t % block_tokens) of block
 * block_table[b][t / block_tokens].  A contiguous cache is the identity block table.
 * Several layers may be flattened into the batch dimension (each (layer, sequence) pair is an
 * independent problem with its own block-table row).
 *
 * Conventions for every call:
 *   - every pointer is a DEVICE pointer owned by the caller unless stated otherwise; the
 *     library never allocates, frees or synchronises (lynx_check is the one exception);
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream); calls
 *     only enqueue work and return;
 *   - arguments are validated on the host before any launch; an invalid call launches
 *     nothing and returns a status other than LYNX_OK;
 *   - device code never traps: block ids outside [0, num_blocks) are clamped and recorded in
 *     the workspace's status word, which lynx_check turns into LYNX_ERR_BAD_BLOCK_TABLE.
 */
#ifndef LYNX_H_
#define LYNX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LYNX_OK = 0,
  LYNX_ERR_NULL = 1,            /* a required pointer is NULL */
  LYNX_ERR_SHAPE = 2,           /* negative / zero / inconsistent size */
  LYNX_ERR_ALIGN = 3,           /* a pointer is not 16-byte aligned */
  LYNX_ERR_UNSUPPORTED = 4,     /* head_dim != 128, block_tokens % 16 != 0, too many columns */
  LYNX_ERR_WORKSPACE = 5,       /* workspace too small (see lynx_workspace_bytes) */
  LYNX_ERR_CUDA = 6,            /* a CUDA runtime call failed */
  LYNX_ERR_BAD_BLOCK_TABLE = 7, /* (lynx_check) a kernel saw a block id out of range */
  LYNX_ERR_TIMEOUT = 8,         /* (lynx_check) a bounded on-chip wait ran out */
  LYNX_ERR_RANGE = 9            /* (lynx_check) a value row outside the range a kernel can represent */
} lynx_status;

/* One of K or V of one layer (or of several flattened layers), quantised and paged. */
typedef struct {
  const uint8_t* anchor;   /* [num_blocks][Hkv][block_tokens][64] */
  const uint8_t* residual; /* same shape; ignored (may be NULL) by lynx_anchor_attention */
  const float* meta;       /* [num_blocks][Hkv][block_tokens][2] = {scale, zero} */
} lynx_plane;

typedef struct {
  int32_t num_q_heads;        /* Hq, a multiple of num_kv_heads; Hq/Hkv in 1..16 */
  int32_t num_kv_heads;       /* Hkv */
  int32_t head_dim;           /* must be 128 */
  int32_t block_tokens;       /* tokens per block, a multiple of 16 */
  int32_t num_blocks;         /* blocks in the pool the planes cover */
  int32_t max_blocks_per_seq; /* row length of block_table */
} lynx_shape;

/* Steps 1 (Section 2.3 quantiser; Section 4.1 stage 4 split; Compression Kernel packing).
 * src_bf16 : [n_rows][128] BF16, 16-byte aligned.  Row i of src produces row i of anchor
 *            ([n_rows][64] u8), residual ([n_rows][64] u8) and meta ([n_rows][2] float).
 * block_ids: NULL -> all rows 0..n_rows-1 are quantised.  Otherwise int32 [n_block_ids]:
 *            only rows block_ids[i]*rows_per_block .. +rows_per_block-1 are quantised (newly
 *            arrived blocks); ids outside [0, n_rows/rows_per_block) are skipped.  n_rows must
 *            then be a multiple of rows_per_block.
 * n_rows == 0 (or n_block_ids == 0) is a valid no-op. */
lynx_status lynx_split_quantize(const void* src_bf16, int64_t n_rows, const int32_t* block_ids,
                                int32_t n_block_ids, int32_t rows_per_block, uint8_t* anchor,
                                uint8_t* residual, float* meta, void* stream);

/* Step 4 (Section 4.2 Residual Phase refinement to Q_full).  For each of n_rows rows:
 * code = (a << 4) | r.  codes_u8 ([n_rows][128] u8) and dequant_bf16 ([n_rows][128] BF16 =
 * bf16_rne(fl(fma(code, scale, zero)))) are optional outputs; at least one must be given. */
lynx_status lynx_recombine(const uint8_t* anchor, const uint8_t* residual, const float* meta,
                           int64_t n_rows, uint8_t* codes_u8, void* dequant_bf16, void* stream);

/* Bytes of workspace the two attention calls need for `batch` sequences, `n_cols_q` query
 * positions (n_q or k) and sequences of at most max_blocks_per_seq * block_tokens tokens.
 * Returns 0 for an unsupported shape.  The workspace must be zero-filled once before its first
 * use (lynx_workspace_init, or cudaMemsetAsync of the whole buffer); each call leaves it ready
 * for the next.  Calls sharing a workspace must be ordered on one stream.
 * A buffer smaller than this figure is rejected by the attention calls (LYNX_ERR_WORKSPACE): nothing
 * degrades silently.  For verification with more than 32 columns (k * Hq/Hkv in 33..64) the figure
 * includes about 19 MB for FP32 copies of the accumulators of the FP16 tensor-core kernels used there
 * (their accumulation chains are cut every 256 units of 64 tokens, which bounds what the tensor
 * cores lose by truncating when they accumulate, whatever the context length).  Anchor attention and
 * verification with up to 16 columns run on exact integer tensor-core products and need no such copies. */
size_t lynx_workspace_bytes(const lynx_shape* shape, int32_t batch, int32_t n_cols_q);
lynx_status lynx_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Step 2 (Section 2 attention equation on the Anchor-only state of Section 4.2).
 * q_bf16 : [batch][n_q][Hq][128] BF16; query head h reads KV head h / (Hq/Hkv).
 * Query j of sequence b attends tokens [0, seq_lens[b]) (causal == 0) or
 * [0, seq_lens[b] - n_q + j + 1) (causal != 0); a query that sees no token gets zeros.
 * softmax_scale 0 means 1/sqrt(128).  out : [batch][n_q][Hq][128] float.
 * n_q must be <= 64 (the cap on speculated positions of Section 5.1).  A kernel launch takes up to 32
 * query columns n_q * (Hq/Hkv); a call with more runs as slices of whole positions, each a pass of its own
 * over the planes, one after the other on the stream.  seq_lens[b] is clamped to the table's capacity.
 * Value rows of any finite scale are handled (the weights are fixed-point numbers relative to a
 * per-column reference exponent).  Queries enter as fixed-point numbers with 22 bits below the largest
 * |q| among the columns of a (sequence, KV head): whatever their magnitude, entries are exact to
 * 2^-22 of that largest one. */
lynx_status lynx_anchor_attention(const lynx_shape* shape, const void* q_bf16, int32_t batch,
                                  int32_t n_q, int32_t causal, lynx_plane K, lynx_plane V,
                                  const int32_t* block_table, const int32_t* seq_lens,
                                  float softmax_scale, float* out, void* workspace,
                                  size_t workspace_bytes, void* stream);

/* Step 3 (Section 4.2 Residual Phase + Section 4.3 verification).  Same attention on the
 * recombined full codes for the k drafted positions in one pass over the context, then per
 * sequence   dev[b][j] = max over heads, dims of |out_full - draft| / (atol + rtol*|out_full|)
 * and first_reject[b] = smallest j with dev[b][j] > 1, or k if none (the longest agreeing
 * prefix; out_full at that position is the correction).
 * draft_out : [batch][k][Hq][128] float, the Anchor-state results being verified; may be NULL,
 * then dev / first_reject are not written (and may be NULL).  out_full : same shape, float.
 * k must be <= 64.  Up to 16 columns k * (Hq/Hkv) are one launch of the exact integer kernel and 17..32 two
 * passes of it; 33..64 columns (up to 16 positions) are one launch of a kernel whose weights are FP16
 * numbers; a longer window runs as slices of whole positions (a pass over the planes each).  With several
 * launches first_reject is taken over the whole window from the deviations.  In the FP16 kernel a value
 * row whose scale reaches 16 (a range of 4080 or more) would overflow the weights; such rows are recorded
 * in the status word and lynx_check returns LYNX_ERR_RANGE (the outputs of that call are then not
 * to be used).  Up to 32 columns there is no such limit. */
lynx_status lynx_merge_verify_attention(const lynx_shape* shape, const void* q_bf16,
                                        int32_t batch, int32_t k, int32_t causal, lynx_plane K,
                                        lynx_plane V, const int32_t* block_table,
                                        const int32_t* seq_lens, float softmax_scale,
                                        const float* draft_out, float atol, float rtol,
                                        float* out_full, int32_t* first_reject, float* dev,
                                        void* workspace, size_t workspace_bytes, void* stream);

/* Anchor attention without a caller workspace (the paper has no counterpart; this exists for
 * deployments where the calling code may not allocate device memory: a plug-in running inside
 * another framework's memory plan, a latency-critical serving loop that has frozen its
 * allocations, or a host that must not touch the allocator while other streams are being
 * captured).  Same computation, arguments and result as lynx_anchor_attention, but the scratch
 * memory is a fixed 8 MiB array inside the library image (every GPU that loads the library
 * holds it until the process exits); the call itself allocates nothing.
 *  - Problems whose scratch need (lynx_workspace_bytes for the same shape) exceeds 8 MiB are rejected
 *    with LYNX_ERR_WORKSPACE; nothing is launched and the array is not touched.
 *  - The first call on each device looks up the array's device address (a one-time set-up,
 *    done with that device current); make that first call before any stream capture begins.
 *  - All calls share the one array.  Each call clears the words that must start at zero, on
 *    `stream`; two calls that overlap on the GPU (different streams, or different host threads
 *    without ordering) race on it and produce wrong results.  Order them on one stream.
 *  - Out-of-range block ids are clamped as usual but cannot be reported (there is no workspace
 *    for lynx_check to read). */
lynx_status lynx_anchor_attention_static(const lynx_shape* shape, const void* q_bf16, int32_t batch,
                                         int32_t n_q, int32_t causal, lynx_plane K, lynx_plane V,
                                         const int32_t* block_table, const int32_t* seq_lens,
                                         float softmax_scale, float* out, void* stream);

/* The paper's own quantiser (Section 4.1, Algorithm 1 "Lynx Hierarchical Quantization"; inverse: the
 * inverse alpha-law of its stage 3, eq. 4) as a second scheme beside the linear one above.
 * src_bf16 : BF16 [n_pages][256][128]: pages of P = 256 consecutive tokens of one KV head (contiguous).
 * Per channel: page minimum and range (gamma_min, gamma_scale: float [n_pages][128]); per chunk of
 * C = 32 consecutive tokens its mean and largest deviation (mu, sigma: float [n_pages][8][128]);
 * magnitudes companded with the alpha-law (alpha = 255) to integers 0..120, split into a 4-bit
 * sign-aware two's-complement Anchor and a 4-bit centred Residual, packed two per byte like the linear
 * planes (q_anc, q_res: uint8 [n_pages][256][64], byte j = channel 2j | channel 2j+1 << 4).
 * Arithmetic is binary32; the readings of the algorithm's open points (alpha, epsilon = 1e-6, the scale
 * 120, the sign taken from the centred value) are stated in the library's design notes.  All pointers
 * 16-byte aligned (LYNX_ERR_ALIGN otherwise); n_pages == 0 is a valid no-op.
 * lynx_hier_dequantize reconstructs BF16 pages [n_pages][256][128] from both streams, or from the
 * Anchor alone when q_res is NULL (the Residual, a centred correction, taken as zero); the pages can be
 * attended to with lynx_bf16_attention (block_tokens = 256). */
lynx_status lynx_hier_quantize(const void* src_bf16, int64_t n_pages, uint8_t* q_anc, uint8_t* q_res,
                               float* gamma_min, float* gamma_scale, float* mu, float* sigma, void* stream);
lynx_status lynx_hier_dequantize(const uint8_t* q_anc, const uint8_t* q_res, int64_t n_pages,
                                 const float* gamma_min, const float* gamma_scale, const float* mu,
                                 const float* sigma, void* dst_bf16, void* stream);

/* Token-level verification of a speculated window (Section 4.3; the acceptance rule of speculative sampling
 * the paper builds on, Section 2.4).  The k draft tokens s_i were drawn from the Anchor-state distributions
 * p_i; the verification pass yields the distributions q_1 .. q_{k+1}.  Token i is accepted iff
 * u_i * p_i(s_i) < q_i(s_i), i.e. with probability min(1, q_i(s_i) / p_i(s_i)); n_accepted[b] is the length of
 * the accepted prefix.  next_token[b] is the correction drawn from norm(max(0, q_j - p_j)) at the first
 * rejected position j (from q_j itself should that residual be zero everywhere), or the bonus token drawn
 * from q_{k+1} when all k are accepted: the smallest vocabulary index whose cumulative weight exceeds
 * r[b] * total.  The outputs are then distributed as samples of q alone.
 * p_probs : float [batch][k][vocab]; q_probs : float [batch][k+1][vocab]; draft_tokens : int32 [batch][k]
 * (clamped to the vocabulary); u : float [batch][k] and r : float [batch], uniform in [0, 1), supplied by the
 * caller; n_accepted, next_token : int32 [batch].  1 <= k <= 64; vocab <= 1572864 (LYNX_ERR_UNSUPPORTED
 * beyond).  Sums are FP32: a decision within rounding of its threshold may differ from a higher-precision
 * evaluation. */
lynx_status lynx_token_verify(const float* p_probs, const float* q_probs, const int32_t* draft_tokens,
                              const float* u, const float* r, int32_t batch, int32_t k, int32_t vocab,
                              int32_t* n_accepted, int32_t* next_token, void* stream);

/* Decode attention over dequantised BF16 pages: the path the paper itself describes (Section 4.2: the
 * dequantisation kernel scatters BF16 pages into the paged KV memory, the engine's attention reads
 * them; Section 2 attention equation), here as the baseline the fused calls above are measured
 * against (256 bytes per row of K or V instead of 72 / 136).
 * k_pages_bf16, v_pages_bf16 : BF16 [num_blocks][Hkv][block_tokens][128], as lynx_recombine writes
 * them (dequant_bf16).  q_bf16, block_table, seq_lens, causal, softmax_scale, out as for
 * lynx_anchor_attention.  Hq/Hkv must be <= 8 and n_q <= 64; a launch takes up to 8 query columns
 * n_q * (Hq/Hkv), a call with more runs as slices of whole positions, each a pass of its own over the pages.
 * Any block_tokens.
 * workspace : lynx_bf16_workspace_bytes(shape, batch, n_q) bytes of scratch (split-K partials and the rows'
 * log-sum-exps), no initialisation needed.  Out-of-range block ids are clamped and not reported. */
size_t lynx_bf16_workspace_bytes(const lynx_shape* shape, int32_t batch, int32_t n_q);
lynx_status lynx_bf16_attention(const lynx_shape* shape, const void* q_bf16, int32_t batch, int32_t n_q,
                                int32_t causal, const void* k_pages_bf16, const void* v_pages_bf16,
                                const int32_t* block_table, const int32_t* seq_lens,
                                float softmax_scale, float* out, void* workspace,
                                size_t workspace_bytes, void* stream);

/* A quantised prefix followed by a BF16 tail (no paper counterpart as a call; Section 4.2 keeps the tokens the
 * decode node generates itself out of the quantiser, and Section 2's softmax runs over prefix and tail alike).
 * Every attention call above leaves, next to its output, the natural-log log-sum-exp of each output row's scaled
 * scores in its workspace: lse[b][j][h] = log sum_t exp(softmax_scale * q[b][j][h] . K_hat[t]) over the tokens the
 * query saw, -inf where it saw none.  lynx_workspace_lse / lynx_bf16_workspace_lse return the DEVICE address of
 * that array, float [batch][n_q][Hq], inside `workspace`, for the (shape, batch, n_q) of the call that wrote it
 * (NULL for an unsupported shape or a NULL workspace); it is valid once that call has completed on its stream and
 * until the next call on the workspace.  Nothing is launched, allocated or copied.
 *
 * lynx_lse_merge joins two results over disjoint key sets into the attention over their union:
 *   out[r] = (e^lse_a[r] out_a[r] + e^lse_b[r] out_b[r]) / (e^lse_a[r] + e^lse_b[r]),  lse_out[r] = log of that sum,
 * for n_rows rows of 128 floats (n_rows = batch * n_q * Hq for two attention calls on the same queries: the
 * prefix through lynx_anchor_attention or lynx_merge_verify_attention, non-causal, the tail through
 * lynx_bf16_attention, causal among the tail's own tokens).  A row with lse = -inf contributes nothing, whatever
 * its out row holds; two such rows give zeros and -inf.  All pointers are DEVICE pointers; out_* and out 16-byte
 * aligned; out may be out_a or out_b; lse_out may be NULL.  Asynchronous on `stream`.
 *
 * lynx_verify_decision is Section 4.3's agreement test on outputs that are already in memory -- the full-state
 * result of a window after it has been joined with the tail: out_full, draft_out float [batch][k][Hq][128],
 * dev[b][j] = max over heads and dims of |f - d| / (atol + rtol |f|), first_reject[b] = the smallest j with
 * dev[b][j] > 1, else k: the decision lynx_merge_verify_attention takes when it is given a draft.  k <= 64,
 * atol > 0, rtol >= 0; out_full and draft_out 16-byte aligned.  Asynchronous on `stream`. */
const float* lynx_workspace_lse(const lynx_shape* shape, int32_t batch, int32_t n_q, const void* workspace);
const float* lynx_bf16_workspace_lse(const lynx_shape* shape, int32_t batch, int32_t n_q, const void* workspace);
lynx_status lynx_lse_merge(const float* out_a, const float* lse_a, const float* out_b, const float* lse_b,
                           int64_t n_rows, float* out, float* lse_out, void* stream);
lynx_status lynx_verify_decision(const float* out_full, const float* draft_out, int32_t batch, int32_t k,
                                 int32_t num_q_heads, float atol, float rtol, int32_t* first_reject, float* dev,
                                 void* stream);

/* The Anchor / Residual split at other bit positions (Conclusion: splits other than INT4 + INT4; Section 4.1
 * stage 4 for the split itself, Section 2.3 for the code).  anchor_bits = A in {2, 4, 6}; R = 8 - A.  The 8-bit
 * code, scale and zero are exactly those of lynx_split_quantize; the Anchor plane holds the top A bits of every
 * code, the Residual plane the bottom R bits: (anchor << R) | residual is the code, and A = 4 writes the planes
 * lynx_split_quantize writes.  Packing per 128-element row and stream: element e's field occupies bits
 * [e w, (e + 1) w) of the row's 16 w bytes, least significant bit first (w = A or R).
 *   src_bf16 : [n_rows][128] BF16;  anchor : [n_rows][16 A] bytes;  residual : [n_rows][16 R] bytes;
 *   meta : [n_rows][2] float (scale, zero).  All DEVICE pointers, 16-byte aligned (meta: 8).
 * lynx_recombine_bits: levels = (anchor << R) | residual, or with residual NULL the middle of the Anchor's
 * bucket, (anchor << R) + 2^(R-1) (Section 4.2, Anchor phase); codes_u8 [n_rows][128] and / or dequant_bf16
 * [n_rows][128] BF16 = bf16(fl(level * scale + zero)), as lynx_recombine; at least one output.  The pages it
 * writes feed lynx_bf16_attention: that is how these splits reach attention (the fused attention calls read
 * the 4 + 4 planes only).  LYNX_ERR_UNSUPPORTED for any other anchor_bits. */
lynx_status lynx_split_quantize_bits(const void* src_bf16, int64_t n_rows, int32_t anchor_bits, uint8_t* anchor,
                                     uint8_t* residual, float* meta, void* stream);
lynx_status lynx_recombine_bits(const uint8_t* anchor, const uint8_t* residual, const float* meta, int64_t n_rows,
                                int32_t anchor_bits, uint8_t* codes_u8, void* dequant_bf16, void* stream);

/* Synchronises `stream`, reads and clears the workspace's status word.  Test / debug use. */
lynx_status lynx_check(void* workspace, void* stream);

const char* lynx_status_string(lynx_status s);
int lynx_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LYNX_H_ */
