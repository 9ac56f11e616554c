// Merge-verify attention for 17..64 columns on the fifth-generation tensor cores (tcgen05, TMEM).
// Included by attention.cu inside its namespace: shares the stream-K cut of the work, the piece
// bookkeeping and finish_piece with the mma.sync kernels.
//
// With this many query rows per KV head the verify pass of Section 4.3 is a dense contraction
// (about 120 flop per plane byte at 64 columns), which the mma.sync kernels cannot feed: their
// tensor pipe would have to be busier than 100 % at the HBM roofline.  Here the two
// contractions of a 64-token stage-unit are two tcgen05.mma groups with M = 128:
//   S[128 rows x 64 tokens]  = Q[128 x 128 dims] . codes(K)^T      A = Q in TMEM, B in shared memory
//   O[128 rows x 128 dims]  += P[128 x 64 tokens] . codes(V)       A = P in TMEM, B in shared memory
// The weights go in as two FP16 terms, p * scale_v = h + r (the rounded weight and the rounding's
// remainder).  With up to 32 columns the two terms have rows of their own in the M = 128 and one
// pass does both; with 64 columns P holds h for a first pass and r for a second pass over the
// same V tile.
// Row r of the M = 128 is (term, copy, column): the k*G columns (padded to 32 or 64) are replicated
// NCOPY times and copy i owns tokens [i*64/NCOPY, (i+1)*64/NCOPY) of the unit: its P
// entries for the other tokens stay zero, so every row is an independent flash-decoding split
// with its own running maximum and all 128 TMEM lanes (threads) have softmax work.  Rows are
// merged at the end of a piece.
//
// Warp roles of a CTA (one CTA per SM: it owns all 512 TMEM columns):
//   2 softmax warpgroups (4 warps each) alternate over the units of a piece; each has its own
//     S, P, O regions in TMEM (64 + 32 + 128 columns; Q takes the other 64) and its own K and V
//     operand tiles.  Per unit a group reads its rows' scores from TMEM, applies the per-token
//     scale / zero point, the causal limit and the lazily raised running maximum, and writes FP16
//     weights p * scale_v to its part of P.  It also expands the NEXT unit's K planes into the
//     K tile (so that S of the next unit is computed under this unit's softmax) and, in the
//     64-column variant, its own V tile.
//   (4 V converter warps expand the V planes in instantiations with four token copies.)
//   3 producer warps stream the raw planes into a shared-memory ring (cp.async.bulk, 8 of the
//     24 copies of a unit each: one warp issuing all of them caps at about 2.7 TB/s).
//   1 MMA warp: one thread polls the "operands ready" mbarriers and issues every tcgen05.mma
//     and its commit, so that no softmax warp stalls on the tensor pipe's queue.
// The expansion writes FP16 code tiles as subnormal patterns (0x00cc = code * 2^-24, one
// PRMT/LOP3 per word) in the canonical 128-byte-swizzled layout; the same bytes serve as K-major
// B operand (K) and as MN-major B operand (V).  All hand-offs are mbarriers (tcgen05.commit for
// the MMAs); every wait is bounded.  Element order along head_dim inside each group of 8 is
// {0,4,2,6,1,5,3,7} in all operand tiles (what the nibble expansion produces for free); it is
// undone when O is written out.

// position -> element within a group of 8: {0,4,2,6,1,5,3,7}, the 3-bit reversal
__host__ __device__ constexpr int wide_perm(int pos) { return ((pos & 1) << 2) | (pos & 2) | ((pos >> 2) & 1); }

// NCOPY: token slices of a unit, each with its own rows.  TERMS = 1: a row's weights go in as two
// P.V passes (rounded weights, then remainders); TERMS = 2: the rounded weights and the remainders
// have rows of their own and one pass does both (half as many columns fit).
template <int NCOPY, int TERMS>
struct WideCfg {
  static constexpr int kRows = NCOPY * TERMS;    // rows of the M = 128 per column
  static constexpr int kST = 64;                 // tokens per stage-unit
  static constexpr int kTW = 4;                  // 16-token sub-blocks per stage
  static constexpr int kNStage = TERMS == 2 ? 6 : 5;   // what fits beside the operand tiles and the query slots
  static constexpr int kSubBytes = 16 * 272;
  static constexpr int kStageBytes = kST * 272;  // KA, VA, KR, VR (4 KiB each), KM, VM (512 B each)
  static constexpr int kColsPad = 128 / kRows;
  static constexpr int kTok = kST / NCOPY;       // tokens of a unit that one row owns
  static constexpr int kConsWarps = 8;
  static constexpr int kConsThreads = 256;
  static constexpr int kProdWarps = 3;           // each issues 8 of the 24 plane copies of a unit
  static constexpr int kMmaWarp = kConsWarps + kProdWarps;   // one thread of it issues every tcgen05.mma
  static constexpr int kVWarp0 = kMmaWarp + 1;    // warps that expand the V tiles; without them the softmax groups do it
  static constexpr int kVWarps = NCOPY == 4 ? 4 : 0;   // (16 warps leave 128 registers per thread: too few for 32 tokens per row)
  static constexpr int kThreads = (kConsWarps + kProdWarps + 1 + kVWarps) * 32;
  // shared memory map (offsets from a 1024-byte aligned base)
  static constexpr int kTileBytes = 2 * 64 * 128;              // [2 dim blocks][64 tokens][128 B]
  static constexpr int kOffCanon = 0;                          // [wg][K tile, V tile 0, V tile 1]
  static constexpr int kOffRing = 6 * kTileBytes;
  static constexpr int kOffScal = kOffRing + kNStage * kStageBytes;  // [group][3 sets][256 floats]
  static constexpr int kOffQs = kOffScal + 2 * 3 * 4 * 64 * 4;       // sum of q per column
  static constexpr int kOffQ = kOffQs + kColsPad * 4;                // raw BF16 queries, 2 slots
  static constexpr int kOffBlk = kOffQ + 2 * kColsPad * LYNX_D * 2;
  static constexpr int kOffInfo = kOffBlk + kProdWarps * 2 * kPieceUnits * 4;
  static constexpr int kOffBars = kOffInfo + kNStage * 16 + 2 * 32;
  static constexpr int kOffMisc = kOffBars + (2 * kNStage + 22) * 8;  // full, empty, q full/empty, sready, odone, kready, pready, rready, rdone (x2), vready (x2)
  static constexpr int kSmem = kOffMisc + 256 + 1024;                // + alignment slack
  // TMEM columns of a warpgroup
  static constexpr int kTmemQ = 0, kTmemWg0 = 64, kTmemS = 0, kTmemP = 64, kTmemO = 96, kTmemWg = 224, kTmemCols = 512;
  static_assert(kOffRing % 16 == 0 && kTileBytes % 1024 == 0, "operand tiles are 1024-byte aligned");
  static_assert(kOffQ % 16 == 0 && kOffBars % 8 == 0, "alignment");
  static_assert(kSmem <= 227 * 1024, "shared memory");
  // scratch of the end-of-piece merge lives in the operand tiles (idle by then)
  static constexpr int kMergeStride = 129;                     // floats per column (odd: no bank conflicts)
  static_assert(kColsPad * kMergeStride * 4 + 3 * 256 * 4 <= 6 * kTileBytes, "merge scratch");
};

// ---- tcgen05 wrappers -------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] . B[smem]
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
// D[tmem] (+)= A[tmem] . B[smem]
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading / stride byte
// offsets (16-byte units), descriptor version 1, layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t tc_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: FP32 accumulate, FP16 A and B, A K-major, M = 128.
__host__ __device__ constexpr uint32_t tc_idesc(int n, bool b_mn_major) {
  return (1u << 4) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

template <int N>
struct TmemRegs;  // loads / stores of N consecutive 32-bit columns of the thread's own lane
template <>
struct TmemRegs<8> {
  static __device__ __forceinline__ void ld(uint32_t a, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(a) : "memory");
  }
  static __device__ __forceinline__ void st(uint32_t a, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(a), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
  }
};
template <>
struct TmemRegs<16> {
  static __device__ __forceinline__ void ld(uint32_t a, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(a) : "memory");
  }
  static __device__ __forceinline__ void st(uint32_t a, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(a), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
  }
};
template <>
struct TmemRegs<32> {
  static __device__ __forceinline__ void ld(uint32_t a, uint32_t* r) {
    TmemRegs<16>::ld(a, r);
    TmemRegs<16>::ld(a + 16, r + 16);
  }
  static __device__ __forceinline__ void st(uint32_t a, const uint32_t* r) {
    TmemRegs<16>::st(a, r);
    TmemRegs<16>::st(a + 16, r + 16);
  }
};

// Expand the nibble planes of one tensor of a 64-token raw stage into the FP16 code tile.
// Thread i of the warpgroup converts the 16-byte chunk i & 3 (32 elements) of rows i >> 2 and
// (i >> 2) + 32: two 128-bit loads, per word two merges and four expansions, four 128-bit
// stores at the swizzled chunk positions.
__device__ __forceinline__ void wide_expand(uint32_t raw_a, uint32_t raw_r, uint32_t tile, int i) {
  const int cc = i & 3, row0 = i >> 2;
  // Half of the threads take the two 8-byte halves of their 16 bytes in the other order (sw = 2):
  // cc >= 2 xor an odd row pair.  The four threads of a row then store to four different chunk
  // positions in every store instruction (conflict-free 128-bit stores), and rows r and r + 2, which
  // share their banks in the raw stage, read different halves (conflict-free 64-bit loads).
  const uint32_t sw = (uint32_t)(((cc >> 1) ^ (row0 >> 1)) & 1) * 2u;
  // all loads first: the shared-memory accesses are volatile asm and keep their order
  uint2 xa[2][2], xr[2][2];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const uint32_t off = (uint32_t)((row0 + 32 * j) * 64 + cc * 16);
    xa[j][0] = lds64(raw_a + off + sw * 4u); xa[j][1] = lds64(raw_a + off + (sw ^ 2u) * 4u);
    xr[j][0] = lds64(raw_r + off + sw * 4u); xr[j][1] = lds64(raw_r + off + (sw ^ 2u) * 4u);
  }
  // rows row0 and row0 + 32 have the same row & 7: one set of swizzled chunk offsets
  const uint32_t base = tile + (uint32_t)(cc >> 1) * 8192u + (uint32_t)row0 * 128u;
  const uint32_t swz = (uint32_t)(((cc & 1) * 4) ^ (row0 & 7) ^ (int)sw) * 16u;
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const uint32_t wa[4] = {xa[j][0].x, xa[j][0].y, xa[j][1].x, xa[j][1].y};
    const uint32_t wr[4] = {xr[j][0].x, xr[j][0].y, xr[j][1].x, xr[j][1].y};
#pragma unroll
    for (int k = 0; k < 4; ++k) {   // register k holds word k ^ sw of the chunk
      uint32_t ev, od;
      merge_codes(wa[k], wr[k], ev, od);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + (uint32_t)j * 4096u + (swz ^ (uint32_t)(k * 16))),
                   "r"(ev & 0x00FF00FFu), "r"(prmt(ev, 0u, 0x4341)), "r"(od & 0x00FF00FFu),
                   "r"(prmt(od, 0u, 0x4341)) : "memory");
    }
  }
}

// One of the producer warps of the wide kernel: the stream-K bookkeeping of producer_warp (every
// warp derives the same range and pieces; warp 0 alone publishes them, loads the queries and
// handles empty sequences), and per unit its share of the 24 plane copies (4 sub-blocks of 16
// tokens x 6 arrays).  One warp issuing all 24 copies of a unit sustains only about 2.7 TB/s
// over the GPU; three warps with eight copies each lift that limit.
template <class C>
__device__ __forceinline__ void wide_producer(const AttnParams& p, int pw, int lane, uint32_t ring_u32,
                                              uint32_t full0, uint32_t empty0, uint32_t qfull0, uint32_t qempty0,
                                              __nv_bfloat16* q_s, uint32_t* blk_s, Item* items, int* misc,
                                              volatile int* abort_word) {
  constexpr int ST = C::kST, NSTAGE = C::kNStage;
  const int n_cta = gridDim.x, cta = blockIdx.x;
  const int cap = p.max_blocks * p.bt;
  auto clamp_len = [&](int b) {
    int len = __ldg(p.seq_lens + b);
    return len < 0 ? 0 : (len > cap ? cap : len);
  };
  const SkRange rng = sk_range<ST>(p, n_cta, cta, lane, clamp_len);
  const long long q = rng.q, lo = rng.lo, hi = rng.hi, off_lo = rng.off_lo;
  const int b_lo = rng.b_lo;
  if (pw == 0) {
    if (lane == 0) misc[7] = lo < hi ? (int)(hi - lo) : 0;
    // sequences with no token: outputs are zero, nothing is rejected unless the draft is not zero
    for (int b = cta; b < p.B; b += n_cta) {
      if (clamp_len(b) != 0) continue;
      const size_t n = (size_t)p.nq * p.Hq * LYNX_D;
      for (size_t i = lane; i < n; i += 32) p.out[(size_t)b * p.nq_stride * p.Hq * LYNX_D + i] = 0.0f;
      for (int i = lane; i < p.nq * p.Hq; i += 32) p.ws_lse[(size_t)b * p.nq_stride * p.Hq + i] = -INFINITY;
      if (p.draft != nullptr) {
        int fr = p.nq;
        for (int j = p.nq - 1; j >= 0; --j) {
          float worst = 0.0f;
          for (int i = lane; i < p.Hq * LYNX_D; i += 32)
            worst = fmaxf(worst, fabsf(__ldg(p.draft + ((size_t)b * p.nq_stride + j) * p.Hq * LYNX_D + i)) / p.atol);
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) worst = fmaxf(worst, __shfl_xor_sync(0xFFFFFFFFu, worst, off));
          if (lane == 0) p.dev[(size_t)b * p.nq_stride + j] = worst;
          if (worst > 1.0f) fr = j;
        }
        if (lane == 0) p.first_reject[b] = fr;
      }
    }
  }
  __syncthreads();  // (A) the range is published
  const int n_units = (int)(lo < hi ? hi - lo : 0);
  if (n_units == 0) return;

  // role = (sub-block, array) of a unit's 24 copies; arrays: K anchor, V anchor, K meta, V meta, K residual,
  // V residual.  Warp pw has the roles 8 pw .. 8 pw + 7 (lanes 0..7), which lie in two sub-blocks.
  constexpr int RP = 24 / C::kProdWarps;
  const int role = pw * RP + (lane < RP ? lane : 0);
  const int sub = role / 6, arr = role % 6, sub_first = (pw * RP) / 6;
  const bool is_meta = arr == 2 || arr == 3;
  const unsigned char* my_src = arr == 0 ? p.ka : arr == 1 ? p.va
                              : arr == 2 ? reinterpret_cast<const unsigned char*>(p.km)
                              : arr == 3 ? reinterpret_cast<const unsigned char*>(p.vm)
                              : arr == 4 ? p.kr : p.vr;
  const uint32_t my_bytes = is_meta ? 128u : 1024u, my_mul = is_meta ? 8u : 64u;
  const uint32_t my_dst = (arr == 0 ? 0u : arr == 1 ? ST * 64u : arr == 2 ? ST * 256u : arr == 3 ? ST * 264u
                           : arr == 4 ? ST * 128u : ST * 192u) + (uint32_t)sub * my_bytes;
  uint32_t bytes_sub[2];   // bytes this warp copies of its first / second sub-block
#pragma unroll
  for (int s2 = 0; s2 < 2; ++s2) {
    uint32_t v = (lane < RP && sub == sub_first + s2) ? my_bytes : 0u;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    bytes_sub[s2] = v;
  }
  uint32_t* my_blk = blk_s + pw * 2 * kPieceUnits;   // [2 sub-blocks][kPieceUnits]
  int b = b_lo, len = clamp_len(b), U = (len + ST - 1) / ST;
  int hkv = (int)(off_lo / U), u = (int)(off_lo % U);
  int remaining = n_units, gs = 0, ic = 0;
  while (remaining > 0) {
    const int n = min(remaining, U - u);
    const int qi = ic & 1;
    if (pw == 0) {
      if (ic >= 2) mbar_wait(qempty0 + qi * 8, ((ic >> 1) - 1) & 1, abort_word);
      const long long seg0 = lo + (n_units - remaining) - u;  // first unit of this segment
      if (lane == 0) {
        Item it;
        it.b = b; it.hkv = hkv; it.len = len;
        it.first_cta = (int)(seg0 / q);
        it.n_contrib = (int)((seg0 + U - 1) / q) - it.first_cta + 1;
        it.pad0 = n; it.pad1 = u; it.pad2 = 0;
        items[qi] = it;
        mbar_expect_tx(qfull0 + qi * 8, (uint32_t)(p.nq * p.G * LYNX_D * 2));
      }
      __syncwarp();
      for (int j = lane; j < p.nq; j += 32)
        bulk_g2s(smem_u32(q_s + ((size_t)qi * C::kColsPad + j * p.G) * LYNX_D),
                 p.q + (((size_t)b * p.nq_stride + j) * p.Hq + (size_t)hkv * p.G) * LYNX_D,
                 (uint32_t)(p.G * LYNX_D * 2), qfull0 + qi * 8);
    }
    for (int c0 = 0; c0 < n; c0 += kPieceUnits) {
      const int cn = min(kPieceUnits, n - c0);
      for (int i2 = lane; i2 < 2 * cn; i2 += 32) {
        const int i = i2 >> 1;
        const int t0 = (u + c0 + i) * ST + (sub_first + (i2 & 1)) * 16;
        uint32_t row = 0xFFFFFFFFu;  // sub-block beyond the end of the sequence: nothing to copy
        if (t0 < len) {
          int blk = __ldg(p.block_table + (size_t)b * p.max_blocks + t0 / p.bt);
          if (blk < 0 || blk >= p.num_blocks) {
            atomicOr(p.ws_flags, kFlagBadBlock);
            blk = blk < 0 ? 0 : p.num_blocks - 1;
          }
          row = (uint32_t)(((size_t)blk * p.Hkv + hkv) * p.bt + (t0 % p.bt));
        }
        my_blk[(i2 & 1) * kPieceUnits + i] = row;
      }
      __syncwarp();
      for (int k = 0; k < cn; ++k, ++gs) {
        const int slot = gs % NSTAGE;
        if (gs >= NSTAGE) mbar_wait(empty0 + slot * 8, ((gs / NSTAGE) - 1) & 1, abort_word);
        const uint32_t row0 = my_blk[k], row1 = my_blk[kPieceUnits + k];
        const uint32_t row = sub == sub_first ? row0 : row1;
        const uint32_t bar = full0 + slot * 8;
        if (lane == 0) {
          const uint32_t bytes = (row0 != 0xFFFFFFFFu ? bytes_sub[0] : 0u) + (row1 != 0xFFFFFFFFu ? bytes_sub[1] : 0u);
          if (bytes) mbar_expect_tx(bar, bytes);
          else mbar_arrive(bar);
        }
        __syncwarp();
        if (lane < RP && row != 0xFFFFFFFFu)
          bulk_g2s(ring_u32 + slot * C::kStageBytes + my_dst, my_src + (size_t)row * my_mul, my_bytes, bar);
      }
      __syncwarp();  // my_blk is rewritten by the next round
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

// Moves a row of O (128 FP32 columns of tensor memory, lane = row) to its FP32 copy in the
// workspace and zeroes it; see the call.  Out of line: it runs once in hundreds of units.
__device__ __noinline__ void wide_flush_row(uint32_t tm_row, float* wsh, float corr, bool add) {
#pragma unroll
  for (int cch = 0; cch < 4; ++cch) {
    uint32_t o[32];
    TmemRegs<32>::ld(tm_row + cch * 32, o);
    tc_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      float* sh = wsh + (cch * 32 + i) * 128;
      const float v = __uint_as_float(o[i]) * corr;
      if (add) atomicAdd(sh, v); else __stcg(sh, v);
      o[i] = 0u;
    }
    TmemRegs<32>::st(tm_row + cch * 32, o);
  }
}

// The FP16 weights are p * scale_v * 64 (p <= 64 against the lazily raised maximum): FP16 has no
// room below 2^-24, and weights that vanish there would still count in the softmax sum and the
// zero-point term.  Weights overflow from scale_v = 16 on (a value row with a range above 4080).
constexpr float kWideWeightUp = 64.0f;
// Truncation loss per MMA that adds rounded weights into a row of O: 0.46 * 2^-23 of the sum
// (measured on long pieces).  The estimate is good to some 30 %; so that this is enough for the
// longest pieces, a row of O is moved to an FP32 copy in the workspace every kWideFlushUnits units.
constexpr float kWideTruncPerMma = 0.46f * 1.1920929e-7f;
constexpr int kWideFlushUnits = 256;

template <int NCOPY, int TERMS>
__global__ void __launch_bounds__(WideCfg<NCOPY, TERMS>::kThreads, 1) attn_wide_kernel(const AttnParams p) {
  using C = WideCfg<NCOPY, TERMS>;
  constexpr int NR = C::kRows;
  constexpr int NSTAGE = C::kNStage, KT = C::kTok, CP = C::kColsPad;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  float* scal = reinterpret_cast<float*>(smem + C::kOffScal);
  float* qs_s = reinterpret_cast<float*>(smem + C::kOffQs);
  __nv_bfloat16* q_s = reinterpret_cast<__nv_bfloat16*>(smem + C::kOffQ);
  uint32_t* blk_s = reinterpret_cast<uint32_t*>(smem + C::kOffBlk);
  int4* info_s = reinterpret_cast<int4*>(smem + C::kOffInfo);
  Item* items = reinterpret_cast<Item*>(info_s + NSTAGE);
  int* misc = reinterpret_cast<int*>(smem + C::kOffMisc);
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);   // (broadcast: the compiler may keep what follows from it in uniform registers)
  const int cta = blockIdx.x;
  const uint32_t ring_u32 = sbase + C::kOffRing;
  const uint32_t full0 = sbase + C::kOffBars, empty0 = full0 + NSTAGE * 8;
  const uint32_t qfull0 = empty0 + NSTAGE * 8, qempty0 = qfull0 + 16;
  const uint32_t sready0 = qempty0 + 16, odone0 = sready0 + 16, kready0 = odone0 + 16, pready0 = kready0 + 16,
                 rready0 = pready0 + 16, rdone0 = rready0 + 16, vready0 = rdone0 + 32;
  volatile int* abort_word = misc;

  if (tid == 0) {
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(full0 + i * 8, C::kProdWarps);
      mbar_init(empty0 + i * 8, 4 + C::kVWarps);  // the owning group (K side) and the V converters
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(qfull0 + i * 8, 1);
      mbar_init(qempty0 + i * 8, C::kConsWarps);
      mbar_init(sready0 + i * 8, 1);
      mbar_init(odone0 + i * 8, 1);
      mbar_init(kready0 + i * 8, 4);   // K tile and scalars of group i written, its previous scores in registers
      mbar_init(pready0 + i * 8, 4);   // P of group i written (and its V tile, when the group expands it itself)
      mbar_init(vready0 + (2 * i) * 8, C::kVWarps > 0 ? C::kVWarps : 1);       // V tile written by the V converters,
      mbar_init(vready0 + (2 * i + 1) * 8, C::kVWarps > 0 ? C::kVWarps : 1);   // one barrier per V tile of the group
      mbar_init(rready0 + i * 8, 4);   // the remainders of the weights' FP16 rounding are in P
      mbar_init(rdone0 + (2 * i) * 8, 1);       // P.V of the remainders complete (tcgen05.commit), one barrier
      mbar_init(rdone0 + (2 * i + 1) * 8, 1);   // per V tile of the group (units alternate between them)
    }
    misc[0] = 0; misc[1] = 0; misc[7] = 0; misc[8] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < 2 * CP * LYNX_D * 2 / 16; i += C::kThreads)
    reinterpret_cast<uint4*>(q_s)[i] = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  if (warp >= C::kConsWarps && warp < C::kMmaWarp) {
    wide_producer<C>(p, warp - C::kConsWarps, lane, ring_u32, full0, empty0, qfull0, qempty0, q_s, blk_s, items,
                     misc, abort_word);
    return;
  }
  __syncthreads();  // (A)
  const int n_units = misc[7];
  if (n_units == 0) return;

  // ---- tensor memory: all 512 columns of the SM (one CTA per SM) -------------------------------
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(misc + 8)),
                 "r"((uint32_t)C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  uint32_t tmem0 = 0;
  if (warp < C::kVWarp0) {
    tc_fence_before();
    named_bar(5, C::kConsThreads + 32);
    tc_fence_after();
    tmem0 = __shfl_sync(0xFFFFFFFFu, *reinterpret_cast<volatile uint32_t*>(misc + 8), 0);
  }
  // =============================================================================================
  // V converters (4 warps): expand the V planes of every unit into the V tile of the group that
  // owns the unit, as soon as that group's previous P.V has released the tile
  // =============================================================================================
  if (C::kVWarps > 0 && warp >= C::kVWarp0) {
    const int vt = tid - C::kVWarp0 * 32;  // 0..127
    uint32_t nv[2] = {0, 0};               // V tiles so far, per group
    int gs_base = 0, ic = 0;
    while (gs_base < n_units) {
      const int qi = ic & 1;
      mbar_wait(qfull0 + qi * 8, (ic >> 1) & 1, abort_word);
      const int n_piece = items[qi].pad0;
      named_bar(6, C::kConsThreads + C::kVWarps * 32);   // the end-of-piece merge no longer uses the tiles
      for (int u = 0; u < n_piece; ++u) {
        const int w = u & 1;
        const int gs = gs_base + u, slot = gs % NSTAGE;
        const uint32_t nvw = w ? nv[1] : nv[0];
        const uint32_t tile_v = sbase + C::kOffCanon + w * 3 * C::kTileBytes + (1 + (nvw & 1)) * C::kTileBytes;
        mbar_wait(full0 + slot * 8, (gs / NSTAGE) & 1, abort_word);
        // the group's V tiles alternate: this one is free once both P.V passes of the unit before last are done
        if (nvw > 1) mbar_wait(rdone0 + (w * 2 + (nvw & 1)) * 8, ((nvw >> 1) - 1) & 1, abort_word);
        const uint32_t st = ring_u32 + slot * C::kStageBytes;
        wide_expand(st + 4096u, st + 12288u, tile_v, vt);   // VA, VR
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(empty0 + slot * 8);
          mbar_arrive(vready0 + (w * 2 + (nvw & 1)) * 8);
        }
        if (w) ++nv[1]; else ++nv[0];
      }
      gs_base += n_piece;
      ++ic;
    }
    return;
  }
  constexpr uint32_t kIdescS = tc_idesc(64, false), kIdescO = tc_idesc(128, true);
  // =============================================================================================
  // The MMA warp: one thread issues every tcgen05.mma, so that no softmax warp stalls on the
  // tensor pipe's queue.  It polls the "operands ready" barriers and issues what is ready, the P.V
  // passes (which a group waits for soonest) before the next unit's Q.K^T.
  // =============================================================================================
  if (warp == C::kMmaWarp) {
    if (lane == 0) {
      const uint32_t tm_q = tmem0 + C::kTmemQ;
      uint32_t gk[2] = {0, 0}, gp[2] = {0, 0}, gr[2] = {0, 0};   // Q.K^T / P.V / remainder P.V issued so far, per group
      int gs_base = 0, ic = 0;
      while (gs_base < n_units) {
        const int qi = ic & 1;
        mbar_wait(qfull0 + qi * 8, (ic >> 1) & 1, abort_word);
        const int n_piece = items[qi].pad0;
        int todo_k[2] = {(n_piece + 1) >> 1, n_piece >> 1}, todo_p[2] = {(n_piece + 1) >> 1, n_piece >> 1};
        int todo_r[2] = {TERMS == 1 ? (n_piece + 1) >> 1 : 0, TERMS == 1 ? n_piece >> 1 : 0};
        int first_p[2] = {1, 1};
        uint64_t t0 = globaltimer_ns();
        uint32_t idle = 0;   // the clock is read once in 1024 idle rounds: reading it every round slows the polling
        while (todo_k[0] + todo_k[1] + todo_p[0] + todo_p[1] + todo_r[0] + todo_r[1] > 0) {
          bool progress = false;
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            const uint32_t tile_k = sbase + C::kOffCanon + w * 3 * C::kTileBytes;
            const uint32_t tile_vp = tile_k + (1 + (gp[w] & 1)) * C::kTileBytes;   // V tile of the unit whose P.V comes next
            const uint32_t tile_vr = tile_k + (1 + (gr[w] & 1)) * C::kTileBytes;   // ... whose remainder pass comes next
            const uint32_t tm_w = tmem0 + C::kTmemWg0 + w * C::kTmemWg;
            if (todo_r[w] > 0 && mbar_test(rready0 + w * 8, gr[w] & 1)) {   // the same P.V on the remainders
              tc_fence_after();
#pragma unroll
              for (int ks = 0; ks < 4; ++ks)
                tc_mma_ts(tm_w + C::kTmemO, tm_w + C::kTmemP + (uint32_t)ks * 8u,
                          tc_desc(tile_vr + (uint32_t)ks * 2048u, 8192u, 1024u), kIdescO, 1u);
              tc_commit(rdone0 + (w * 2 + (gr[w] & 1)) * 8);
              ++gr[w]; --todo_r[w]; progress = true;
            }
            if (todo_p[w] > 0 && mbar_test(pready0 + w * 8, gp[w] & 1) &&
                (C::kVWarps == 0 || mbar_test(vready0 + (w * 2 + (gp[w] & 1)) * 8, (gp[w] >> 1) & 1))) {
              tc_fence_after();
#pragma unroll
              for (int ks = 0; ks < 4; ++ks)
                tc_mma_ts(tm_w + C::kTmemO, tm_w + C::kTmemP + (uint32_t)ks * 8u,
                          tc_desc(tile_vp + (uint32_t)ks * 2048u, 8192u, 1024u), kIdescO,
                          (!first_p[w] || ks > 0) ? 1u : 0u);
              tc_commit(odone0 + w * 8);
              if (TERMS == 2) {   // no second pass: the V tile is free with this one
                tc_commit(rdone0 + (w * 2 + (gr[w] & 1)) * 8);
                ++gr[w];
              }
              first_p[w] = 0;
              ++gp[w]; --todo_p[w]; progress = true;
            }
            if (todo_k[w] > 0 && mbar_test(kready0 + w * 8, gk[w] & 1)) {
              tc_fence_after();
#pragma unroll
              for (int ks = 0; ks < 8; ++ks)
                tc_mma_ts(tm_w + C::kTmemS, tm_q + (uint32_t)ks * 8u,
                          tc_desc(tile_k + (uint32_t)(ks >> 2) * 8192u + (uint32_t)(ks & 3) * 32u, 16u, 1024u),
                          kIdescS, ks > 0 ? 1u : 0u);
              tc_commit(sready0 + w * 8);
              ++gk[w]; --todo_k[w]; progress = true;
            }
          }
          if (progress) {
            idle = 0;
          } else if ((++idle & 1023u) == 0) {
            if (idle == 1024u) t0 = globaltimer_ns();
            if (*abort_word || globaltimer_ns() - t0 > 2000000000ull) {
              *abort_word = 1;   // give up: the waiting groups see the abort word and run out their loops
              break;
            }
          }
        }
        gs_base += n_piece;
        ++ic;
      }
    }
    return;
  }
  const int wg = warp >> 2, w4 = warp & 3;
  const int r = tid & 127;                       // row of the M = 128 = TMEM lane
  const int copy = (r / CP) % NCOPY, term = r / (CP * NCOPY), c = r % CP;   // warp-uniform copy and term
  const uint32_t lane_sel = (uint32_t)(w4 * 32) << 16;
  const uint32_t tm_q = tmem0 + C::kTmemQ;
  const uint32_t tm_s = tmem0 + C::kTmemWg0 + wg * C::kTmemWg + C::kTmemS;
  const uint32_t tm_p = tmem0 + C::kTmemWg0 + wg * C::kTmemWg + C::kTmemP;
  const uint32_t tm_o = tmem0 + C::kTmemWg0 + wg * C::kTmemWg + C::kTmemO;
  // FP32 copy of this row of O in the workspace: [CTA][group][dim][row] (worked out where it is
  // used: the address is not worth two registers in the unit loop)
  auto shadow_row = [&]() { return p.ws_shadow + (((size_t)cta * 2 + wg) * 128) * 128 + r; };
  {  // P starts as zero: a row only ever writes its own tokens
    uint32_t z[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) z[i] = 0u;
    TmemRegs<32>::st(tm_p + lane_sel, z);
    tc_wait_st();
  }
  const uint32_t tile_k = sbase + C::kOffCanon + wg * 3 * C::kTileBytes;
  float* my_scal = scal + wg * 768;
  const float cb = p.sm_log2;

  int gs_base = 0, ic = 0;
  uint32_t n_u = 0;            // units of this group so far (selects the scalar set)
  uint32_t n_s = 0, n_o = 0, n_r = 0;   // commits so far on this group's MMA barriers (scores, P.V, remainder P.V)
  bool r_todo = false;         // the remainders of the last unit's weights are still in registers
  bool r_pending = false;      // the last remainder P.V has not been waited for yet
  uint32_t pr_prev[KT / 2];    // those remainders (FP16 pairs)

  while (gs_base < n_units) {
    const int qi = ic & 1;
    mbar_wait(qfull0 + qi * 8, (ic >> 1) & 1, abort_word);
    const Item item = items[qi];
    const int len = item.len, n_piece = item.pad0;
    const int full_lim = p.causal ? len - p.tail + 1 : len;   // (a slice of a longer window: tail positions to its end)
    const int lim_c = c < p.ncols ? (p.causal ? len - p.tail + c / p.G + 1 : len) : 0;
    const __nv_bfloat16* qb = q_s + (size_t)qi * CP * LYNX_D;
    // ---- the piece's queries: common power-of-two scale, FP16 A operand, sum of q ------------
    float amax = 0.0f;
    for (int i = lane; i < CP * (LYNX_D / 8); i += 32) {
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
    int e = 0;  // |q * 2^e| < 2^14: exact in FP16 down to 2^-24 of the largest entry
    if (amax > 0.0f && amax < INFINITY) e = 13 - (((__float_as_int(amax) >> 23) & 0xFF) - 127);
    e = max(-100, min(100, e));
    const float up = __int_as_float((127 + e) << 23), down = __int_as_float((127 - e) << 23);
    const float ca = p.sm_log2 * down * 16777216.0f;  // undoes 2^e of q and 2^-24 of the K codes
    {
      // A operand of Q.K^T in TMEM: lane = row, column j = K positions 2j, 2j+1 (FP16 pairs); this
      // group writes the half of head_dim it is numbered after (32 columns)
      const int half = wg;
      uint32_t h[32];
#pragma unroll
      for (int g8 = 0; g8 < 8; ++g8) {
        h[4 * g8] = h[4 * g8 + 1] = h[4 * g8 + 2] = h[4 * g8 + 3] = 0u;
        if (c < p.ncols) {
          const uint4 v = *reinterpret_cast<const uint4*>(qb + c * LYNX_D + 64 * half + 8 * g8);
          const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
          float f[8];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            f[2 * k] = __uint_as_float(ww[k] << 16) * up;
            f[2 * k + 1] = __uint_as_float(ww[k] & 0xFFFF0000u) * up;
          }
          h[4 * g8] = pack_f16x2(f[0], f[4]); h[4 * g8 + 1] = pack_f16x2(f[2], f[6]);
          h[4 * g8 + 2] = pack_f16x2(f[1], f[5]); h[4 * g8 + 3] = pack_f16x2(f[3], f[7]);
        }
      }
      TmemRegs<32>::st(tm_q + lane_sel + (uint32_t)half * 32u, h);
      tc_wait_st();
      if (tid < CP) {
        float sum = 0.0f;
        if (tid < p.ncols) {
          const uint4* qq = reinterpret_cast<const uint4*>(qb + tid * LYNX_D);
          for (int i = 0; i < 16; ++i) {
            const uint4 v = qq[i];
            const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) sum += __uint_as_float(ww[k] << 16) + __uint_as_float(ww[k] & 0xFFFF0000u);
          }
        }
        qs_s[tid] = sum;
      }
    }
    tc_fence_before();
    named_bar(6, C::kConsThreads + C::kVWarps * 32);
    const float qsum = qs_s[c];

    float m = 0.0f, l = 0.0f, zs = 0.0f;  // m: the running maximum (log2 units)
    bool fresh = true;
    int my_units = 0;
    int units_since = 0;      // units added into this row of O since it was last moved to the copy
    bool w_flushed = false;   // the copy in the workspace holds earlier units of this piece ...
    float m_sh = 0.0f;        // ... relative to this running maximum

    // K side of unit k of this piece: code tile, per-token scalars (set `set`), S = Q . K^T.  The K
    // tile is free: the previous Q.K^T of this group has been waited for.
    auto prefetch = [&](int k, int set) {
      const int gs = gs_base + k;
      const int slot = gs % NSTAGE;
      mbar_wait(full0 + slot * 8, (gs / NSTAGE) & 1, abort_word);
      const uint32_t st = ring_u32 + slot * C::kStageBytes;
      float2 km = make_float2(0.f, 0.f), vm = km;
      if (r < 64) { km = lds64f(st + 16384u + r * 8); vm = lds64f(st + 16896u + r * 8); }
      wide_expand(st, st + 8192u, tile_k, r);            // KA, KR
      if (r < 64) {
        const int unit_t0 = (item.pad1 + k) * C::kST;
        const bool in = unit_t0 + r < len;
        // [pair][alpha0, alpha1, beta0, beta1] and [pair][zero0, zero1, scale0, scale1]
        float* sc = my_scal + set * 256 + (r >> 1) * 4 + (r & 1);
        sc[0] = in ? km.x * ca : 0.0f;     // alpha: score per unit of the raw dot product
        sc[2] = in ? km.y * cb : 0.0f;     // beta: score per unit of sum(q)
        sc[128] = in ? vm.y : 0.0f;        // zero point of the V row
        sc[130] = in ? vm.x * kWideWeightUp : 0.0f;   // scale of the V row, times the weights' factor
        if (in && !(vm.x < 16.0f)) atomicOr(p.ws_flags, kFlagRange);   // FP16 weights would overflow: reported, not hidden
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (C::kVWarps > 0) mbar_arrive(empty0 + slot * 8);   // the V converters release the slot too
        mbar_arrive(kready0 + wg * 8);    // this warp's part of the K side is ready and its S is in registers
      }
      ++n_s;
    };
    // The weights go to the tensor core as two FP16 numbers: the rounded weight (P.V issued at the
    // end of the unit) and the rounding's remainder, whose pass over the same V tile is issued
    // from here once the first has completed (P holds one of the two at a time).
    auto flush_remainders = [&]() {
      if (!r_todo) return;
      r_todo = false;
      if (TERMS == 2) {   // one pass: only its completion is still to be waited for
        ++n_r;
        r_pending = true;
        return;
      }
      mbar_wait(odone0 + wg * 8, (n_o - 1) & 1, abort_word);   // the pass on the rounded weights is done with P
      tc_fence_after();
      TmemRegs<KT / 2>::st(tm_p + lane_sel + (uint32_t)(copy * (KT / 2)), pr_prev);
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(rready0 + wg * 8);
      ++n_r;
      r_todo = false;
      r_pending = true;
    };
    auto wait_remainders = [&]() {
      if (!r_pending) return;
      mbar_wait(rdone0 + (wg * 2 + ((n_r - 1) & 1)) * 8, ((n_r - 1) >> 1) & 1, abort_word);
      r_pending = false;
    };
    if (wg < n_piece) prefetch(wg, (int)(n_u % 3u));

    for (int k = wg; k < n_piece; k += 2, ++my_units, ++units_since) {
      const int set = (int)(n_u % 3u);
      const int slot = (gs_base + k) % NSTAGE;
      const int unit_t0 = (item.pad1 + k) * C::kST;
      const uint32_t scal_u32 = smem_u32(my_scal + set * 256);
      // the scores of this unit (the only outstanding Q.K^T commit of the group)
      mbar_wait(sready0 + wg * 8, (n_s - 1) & 1, abort_word);
      tc_fence_after();
      float x[KT];
      {
        uint32_t raw[KT];
        TmemRegs<KT>::ld(tm_s + lane_sel + (uint32_t)(copy * KT), raw);
        tc_wait_ld();
        const uint64_t qs2 = pk2(qsum, qsum), nm2 = pk2(-m, -m);
#pragma unroll
        for (int i = 0; i < KT; i += 2) {
          const uint4 ab = lds128(scal_u32 + (uint32_t)(copy * KT + i) * 8u);  // alpha0, alpha1, beta0, beta1
          const uint64_t s2 = pk2(__uint_as_float(raw[i]), __uint_as_float(raw[i + 1]));
          upk2(ffma2(pk2(__uint_as_float(ab.x), __uint_as_float(ab.y)), s2,
                     ffma2(pk2(__uint_as_float(ab.z), __uint_as_float(ab.w)), qs2, nm2)), x[i], x[i + 1]);
        }
      }
      // the next unit's K side runs on the tensor core while this unit's softmax is computed
      if (k + 2 < n_piece) prefetch(k + 2, (set + 1) % 3);
      flush_remainders();   // of the previous unit
      // ---- softmax of this row's tokens ----------------------------------------------------------
      const int tok0 = unit_t0 + copy * KT;
      if (unit_t0 + C::kST > full_lim) {
#pragma unroll
        for (int i = 0; i < KT; ++i)
          if (tok0 + i >= lim_c) x[i] = -INFINITY;
      }
      // ---- weights: fast path without the maximum; redone when a weight may have grown too large -----
      uint32_t ph[KT / 2], pr[KT / 2];   // rounded weights and remainders, FP16 pairs
      float l_n, zs_n;
      auto weights = [&]() {
        uint64_t l2 = pk2(l, 0.0f), z2 = pk2(zs, 0.0f);
#pragma unroll
        for (int i = 0; i < KT; i += 2) {
          const uint4 zv = lds128(scal_u32 + 512u + (uint32_t)(copy * KT + i) * 8u);  // zero0, zero1, scale0, scale1
          const uint64_t p2 = pk2(ex2(x[i]), ex2(x[i + 1]));
          l2 = fadd2(l2, p2);
          z2 = ffma2(p2, pk2(__uint_as_float(zv.x), __uint_as_float(zv.y)), z2);
          float w0, w1, b0, b1;
          upk2(fmul2(p2, pk2(__uint_as_float(zv.z), __uint_as_float(zv.w))), w0, w1);
          const uint32_t hh = pack_f16x2(w0, w1);
          asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tcvt.f32.f16 %0, lo;\n\tcvt.f32.f16 %1, hi;\n\t}"
              : "=f"(b0), "=f"(b1) : "r"(hh));
          const uint32_t rr = pack_f16x2(w0 - b0, w1 - b1);   // w = h + r, r exact in FP32 and then rounded to FP16
          if (TERMS == 2) {
            ph[i / 2] = term ? rr : hh;   // the rows of the second term carry the remainders
          } else {
            ph[i / 2] = hh;
            pr[i / 2] = rr;
          }
        }
        float a0, a1;
        upk2(l2, a0, a1); l_n = a0 + a1;
        upk2(z2, a0, a1); zs_n = a0 + a1;
      };
      weights();
      // every weight of the unit is below 64 unless the unit's sum says otherwise
      const bool grow = fresh || !(l_n - l <= 64.0f);
      if (__any_sync(0xFFFFFFFFu, grow)) {
        float f = 1.0f;
        if (grow) {
          float mx = x[0];
#pragma unroll
          for (int i = 1; i < KT; ++i) mx = fmaxf(mx, x[i]);
          const float upm = fresh ? fmaxf(mx, -1.0e4f) : fmaxf(mx, 0.0f);
          f = fresh ? 0.0f : ex2(-upm);
          m += upm;
          l *= f; zs *= f;
#pragma unroll
          for (int i = 0; i < KT; ++i) x[i] -= upm;
        }
        weights();
        if (my_units > 0) {  // O holds earlier units of this piece: rescale the row in TMEM
          wait_remainders();   // both passes of the previous unit have been accumulated
          tc_fence_after();
#pragma unroll
          for (int cch = 0; cch < 4; ++cch) {
            uint32_t o[32];
            TmemRegs<32>::ld(tm_o + lane_sel + cch * 32, o);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
            TmemRegs<32>::st(tm_o + lane_sel + cch * 32, o);
          }
        }
      }
      fresh = false;
      l = l_n; zs = zs_n;
      {
        // P and the V tile are free once both P.V passes of the previous unit are complete
        wait_remainders();
        tc_fence_after();
        if (units_since >= kWideFlushUnits && p.ws_shadow != nullptr) {
          float* wsh = shadow_row();
          // cut the accumulation chain: this row of O is added in FP32 (reductions in L2, round to
          // nearest: no load, nothing to wait for), with the expected truncation loss put back, to
          // its copy and starts again from zero.  The copy stays relative to the running maximum
          // m_sh of the row's first flush, so a later rise of the maximum does not touch it; what is
          // added is scaled up by 2^(m - m_sh) (a rise of more than 60 moves the copy instead).
          float up = w_flushed ? m - m_sh : 0.0f;
          if (!w_flushed) m_sh = m;
          if (up > 60.0f) {   // rare, per row
            const float down = ex2(-up);
#pragma unroll 8
            for (int col = 0; col < 128; ++col) __stcg(wsh + col * 128, __ldcg(wsh + col * 128) * down);
            m_sh = m;
            up = 0.0f;
          }
          const float corr = (1.0f + (float)(4 * units_since) * kWideTruncPerMma) * ex2(up);
          wide_flush_row(tm_o + lane_sel, wsh, corr, w_flushed);
          w_flushed = true;
          units_since = 0;
        }
        TmemRegs<KT / 2>::st(tm_p + lane_sel + (uint32_t)(copy * (KT / 2)), ph);
#pragma unroll
        for (int i = 0; i < KT / 2; ++i) pr_prev[i] = TERMS == 1 ? pr[i] : 0u;
      }
      if constexpr (C::kVWarps == 0) {  // this group expands its own V tile (free: the odone wait above)
        const uint32_t st = ring_u32 + slot * C::kStageBytes;
        // (its V tiles alternate; this one was last read by the unit before last, both passes long done)
        wide_expand(st + 4096u, st + 12288u, tile_k + (1 + (n_o & 1)) * C::kTileBytes, r);   // VA, VR
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + slot * 8);
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(pready0 + wg * 8);   // this warp's rows of P and part of the V tile are ready
      ++n_u;
      ++n_o;
      r_todo = true;
    }

    // ---- end of the piece: merge the 2 * NR partial rows of every column ----------------------------
    flush_remainders();
    wait_remainders();
    tc_fence_after();
    float* msc = reinterpret_cast<float*>(smem + C::kOffCanon);        // [CP][kMergeStride]
    float* sc_m = msc + CP * C::kMergeStride;                          // [256] maxima, then [256] l, [256] zs
    float* sc_l = sc_m + 256;
    float* sc_z = sc_l + 256;
    const bool have = my_units > 0;
    named_bar(1, C::kConsThreads);  // both groups are done with the operand tiles the scratch overlays
    sc_m[tid] = have ? m : -INFINITY;
    named_bar(1, C::kConsThreads);
    float M = -INFINITY;
#pragma unroll
    for (int i = 0; i < 2 * NR; ++i) M = fmaxf(M, sc_m[(i / NR) * 128 + (i % NR) * CP + c]);
    const float f = (have && m > -INFINITY && M > -INFINITY) ? ex2(m - M) : 0.0f;
    sc_l[tid] = term == 0 ? l * f : 0.0f;   // the rows of the second term repeat the first term's sums
    sc_z[tid] = term == 0 ? zs * f : 0.0f;
    // undoes the 2^-24 of the V codes and the weights' factor, and puts back what the tensor core's
    // truncating accumulation lost on average: kWideTruncPerMma of the sum for each of the four
    // MMAs (token slices) with which a unit adds rounded weights into a row of O (the remainders of
    // a second pass are too small to lose more than themselves)
    const float coef = f * (16777216.0f / kWideWeightUp);
    const float corr = 1.0f + (float)(4 * units_since) * kWideTruncPerMma;
    const float keep_sh = w_flushed ? ex2(m_sh - m) : 0.0f;   // the copy, brought to the row's final maximum
    const float* wsh = shadow_row();
    const int part = wg * NR + r / CP;
    for (int round = 0; round < 2 * NR; ++round) {
      if (part == round && have) {   // warp-uniform
#pragma unroll
        for (int cch = 0; cch < 4; ++cch) {
          uint32_t o[32];
          TmemRegs<32>::ld(tm_o + lane_sel + cch * 32, o);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int d = cch * 32 + (i & ~7) + wide_perm(i & 7);   // logical head dim of column i
            float* dst = msc + c * C::kMergeStride + d;
            float part_o = __uint_as_float(o[i]) * corr;
            if (w_flushed) part_o = fmaf(__ldcg(wsh + (cch * 32 + i) * 128), keep_sh, part_o);   // earlier units of the piece
            const float v = coef * part_o;
            *dst = round == 0 ? v : *dst + v;
          }
        }
      } else if (round == 0 && part == 0) {  // group 0 had no unit: cannot happen (k starts at wg = 0)
#pragma unroll 4
        for (int d = 0; d < LYNX_D; ++d) msc[c * C::kMergeStride + d] = 0.0f;
      }
      named_bar(1, C::kConsThreads);
    }
    const bool direct = item.n_contrib == 1;
    {
      const size_t bh = (size_t)item.b * p.Hkv + item.hkv;
      float* part_dst = p.ws_part + (bh + (size_t)cta) * (size_t)CP * kPartStride;
      for (int idx = tid; idx < p.ncols * LYNX_D; idx += C::kConsThreads) {
        const int cc = idx >> 7, d = idx & 127;
        float lt = 0.0f, z = 0.0f;
#pragma unroll
        for (int i = 0; i < 2 * NR; ++i) {
          lt += sc_l[(i / NR) * 128 + (i % NR) * CP + cc];
          z += sc_z[(i / NR) * 128 + (i % NR) * CP + cc];
        }
        const float v = msc[cc * C::kMergeStride + d] + z;
        if (direct) {
          const int j = cc / p.G, hh = cc % p.G;
          p.out[(((size_t)item.b * p.nq_stride + j) * p.Hq + item.hkv * p.G + hh) * LYNX_D + d] =
              lt > 0.0f ? v / lt : 0.0f;
          if (d == 0) {
            float Mc = -INFINITY;
#pragma unroll
            for (int i = 0; i < 2 * NR; ++i) Mc = fmaxf(Mc, sc_m[(i / NR) * 128 + (i % NR) * CP + cc]);
            p.ws_lse[((size_t)item.b * p.nq_stride + j) * p.Hq + item.hkv * p.G + hh] = lse_of(Mc, lt);
          }
        } else {
          part_dst[(size_t)cc * kPartStride + d] = v;
          if (d == 0) {
            float Mc = -INFINITY;
#pragma unroll
            for (int i = 0; i < 2 * NR; ++i) Mc = fmaxf(Mc, sc_m[(i / NR) * 128 + (i % NR) * CP + cc]);
            part_dst[(size_t)cc * kPartStride + 128] = Mc > -INFINITY ? Mc : -1.0e30f;
            part_dst[(size_t)cc * kPartStride + 129] = lt;
          }
        }
      }
      __threadfence();
    }
    finish_piece<true, CP, C::kConsThreads>(p, item, direct, tid, misc);
    __syncwarp();
    if (lane == 0) mbar_arrive(qempty0 + qi * 8);
    gs_base += n_piece;
    ++ic;
  }
  // ---- release the tensor memory ---------------------------------------------------------------
  tc_fence_before();
  named_bar(1, C::kConsThreads);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem0), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
  if (tid == 0 && misc[0]) atomicOr(p.ws_flags, kFlagTimeout);
}

template <int NCOPY, int TERMS>
lynx_status launch_wide(const AttnParams& p, cudaStream_t st) {
  using C = WideCfg<NCOPY, TERMS>;
  auto kern = attn_wide_kernel<NCOPY, TERMS>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmem) != cudaSuccess)
      return LYNX_ERR_CUDA;
    configured[dev] = true;
  }
  const long long cap_units = (long long)p.B * p.Hkv * (((long long)p.max_blocks * p.bt + C::kST - 1) / C::kST);
  long long grid = (cap_units + 7) / 8;
  const long long full = sm_count();   // one CTA per SM: it owns all of the SM's tensor memory
  grid = grid < 1 ? 1 : (grid > full ? full : grid);
  kern<<<(unsigned)grid, C::kThreads, C::kSmem, st>>>(p);
  return launch_status();
}
