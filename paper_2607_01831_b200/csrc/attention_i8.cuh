// Anchor and merge-verify attention on the integer path of the fifth-generation tensor cores
// (tcgen05.mma kind::i8, accumulators in tensor memory).  Included by attention.cu inside its
// namespace: shares AttnParams, the stream-K cut of the work and finish_piece with the other
// kernels.
//
// With one (scale, zero) per token row the two contractions of Section 2's attention run on the
// integer levels themselves (see attention.cu).  Here both are exact integer tensor-core
// products over a 128-token stage-unit:
//   S^T[128 tokens x 3 CP]   = level(K)[128 x 128 dims] . Qd^T     A = K levels (u8, in tensor memory),
//                                                                   B = three balanced s8 digit planes
//                                                                       of the fixed-point query
//   O^T[128 dims x 4 CP]    += level(V)^T[128 x 128 tokens] . Wd    A = V tile (u8, MN-major),
//                                                                   B = the four bytes of the u32
//                                                                       fixed-point weights (MN-major)
// CP = query columns (n_q * G) padded to 4, 8, 16 or 32 (anchor calls with more are run in slices).  The int32 accumulators are exact, so
// there is no rounding in either product: the query is good to 2^-22 of its largest entry and a
// weight to 2^-28 of the largest weight seen so far.
//
// Weights.  For token t and column c,  x = s * log2(e) + log2(scale_v(t))  and  W = 2^(x - ref[c])
// rounded to a u32, with ref[c] chosen so that the largest W of the first unit is 2^28; a later x
// that would push W beyond 2^31.5 raises ref[c] (rare), which ends the current accumulation: the
// int32 accumulators are added, scaled, into an FP32 copy (also in tensor memory) and restart
// from zero.  The same happens before they could overflow.  The softmax sums use the unrounded
// W / scale_v, so a single attended token reproduces its value row to FP32 rounding.
//
// Warp roles of a CTA (one CTA per SM):
//   Teams of four warps (eight with 32 columns) each take every kTeams-th unit of the CTA's range
//     and do everything for it, so that no hand-off between warps with different jobs lies on the
//     path of a unit and the teams hide one another's latencies:
//       K levels into tensor memory (a thread owns a token = a TMEM lane; Q.K^T takes its A
//         operand from there, so the K levels never pass through shared memory again);
//       Q.K^T (one thread issues four tcgen05.mma and a commit);
//       V level tile into shared memory (128-byte-swizzled canonical layout, MN-major);
//       scores -> weights: S read back (TMEM lane = token), per-token scale / zero point / causal
//         limit applied, weights written to the team's P tile;
//       P.V (one thread issues), accumulators and their FP32 copy in the team's tensor memory.
//     The team that owns a piece's first unit also writes the piece's query digit planes; at the
//     end of a piece the teams' partial results are merged by the team that owns its last unit.
//   Producer warps stream the raw planes into a shared-memory ring (cp.async.bulk).  The per-token
//     (scale, zero) pairs do not travel with them (the copy engine takes ~35 cycles per copy
//     whatever its size): every thread reads its own, two units ahead.
// All hand-offs are mbarriers or sequence counters with bounded waits; nothing waits on another CTA.
//
// Element order along head_dim inside operand tiles: byte 16 (2 j + parity) + 4 w + i of a row
// holds dim 32 j + 8 w + 2 i + parity (what the nibble expansion yields with two logic
// operations per word); the query planes use the same order and O is un-permuted at write-out.

// Tensor maps of the K planes ([rows][64 bytes] u8, box = one 16-token sub-block, 64-byte swizzle): the
// copy engine stores 16-byte chunk c of row r at position c ^ ((r >> 1) & 3), which is the order in which
// the threads of a quarter-warp can read their rows (64 bytes apart) without bank conflicts; read back at
// position i ^ ((r >> 1) & 3), chunk i arrives in place with no reordering in registers.
// The V planes go through maps of the same shape without swizzle, so that one instruction of a producer warp
// issues all its copies of a unit (the map is a per-lane operand).
struct alignas(64) I8Maps {
  CUtensorMap m[4];   // K Anchor, V Anchor, K Residual, V Residual (the order of the stage's arrays)
};
inline bool i8_plane_map(CUtensorMap* m, const uint8_t* base, uint64_t rows, bool swizzle) {
  using Fn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                          const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                          CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static Fn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<Fn>(f);
  }();
  if (!fn || !base || rows == 0) return false;
  const cuuint64_t dims[2] = {64, rows};
  const cuuint64_t strides[1] = {64};
  const cuuint32_t box[2] = {64, 16}, es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// one 16-row box of a plane (rows row .. row + 15, all 64 bytes) into shared memory
__device__ __forceinline__ void tma_rows16(uint32_t dst, const CUtensorMap* map, int row, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(row), "r"(bar)
      : "memory");
}

constexpr int kI8PieceUnits = 32;  // stage-units whose block ids a producer warp looks up at a time

template <bool FULL, int CP>
struct I8Cfg {
  static_assert(CP == 4 || CP == 8 || CP == 16 || CP == 32, "padded column counts");
  static constexpr int kST = 128;                   // tokens per stage-unit
  static constexpr int kNArr = FULL ? 4 : 2;        // plane arrays copied per 16-token sub-block (the metadata is
                                                    // read with plain loads: the copy engine takes ~35 cycles per copy)
  static constexpr int kStageBytes = kST * (FULL ? 256 : 128);
  static constexpr int kOffKA = 0, kOffVA = kST * 64, kOffKR = kST * 128, kOffVR = kST * 192;
  // Anchor decode with 4 columns feeds the K planes to Q.K^T as they are: a token's 64 raw bytes
  // b_m = a_2m + 16 a_2m+1 followed by the 64 masked bytes a_2m, against the query values Q_2m+1 and
  // 16 Q_2m - Q_2m+1 (four digit planes instead of three: they fit the padding of N), which gives
  // 16 sum_d Q_d a_d with a third of the logic operations of a full nibble expansion.
  // (with more columns the fourth plane's share of the score arithmetic costs more registers than the
  // expansion saves: 8 columns measured 20 % slower with it)
  static constexpr bool kRawK = !FULL && CP == 4;
  static constexpr bool kVoteFirst = FULL || CP > 4;   // restart question before the weights (see the unit loop)
  static constexpr int kQPlanes = kRawK ? 4 : 3;
  static constexpr int kNQK = (kQPlanes * CP + 15) / 16 * 16;   // N of the Q.K^T product
  static constexpr int kNPV = 4 * CP;                    // N of the P.V product
  static constexpr int kPartCols = CP < 8 ? 8 : CP;      // column stride of the partial slots
  static constexpr int kColsPad = CP;
  // warps: kTeams teams, then the producers.  A team is one warpgroup per column group: with 32 columns
  // two warpgroups share the tokens of a unit, each scoring 16 columns (and one expanding K, the other V).
  static constexpr int kGroups = CP == 32 ? 2 : 1;
  static constexpr int kCG = CP / kGroups;               // columns of a column group
  static constexpr int kTeamWarps = 4 * kGroups, kTeamThreads = 32 * kTeamWarps;
  // (4 columns: four teams at 95 registers without spills and an 8-stage ring measure 2 % below five teams at
  // 80 registers on one launch over 32 flattened layers, but 11 % faster on one launch per layer and 3-12 %
  // faster on short and ragged contexts, where pieces end often)
  static constexpr int kTeams = CP == 32 ? 2 : (FULL || CP == 16) ? 3 : CP == 4 ? 4 : 5;
  static constexpr int kProdWarps = CP == 32 ? 2 : 4;
  static constexpr int kProdWarp0 = kTeamWarps * kTeams;
  static constexpr int kThreads = (kProdWarp0 + kProdWarps) * 32;
  // shared memory map (offsets from a 1024-byte aligned base)
  static constexpr int kTile = 16384;                    // V level tile: [128 tokens][128 B]
  static constexpr int kPRow = 4 * CP < 32 ? 32 : 4 * CP;   // bytes of a P tile row (one token)
  static constexpr int kPTile = 128 * kPRow;
  static constexpr int kPLayout = kPRow == 32 ? 6 : kPRow == 64 ? 4 : 2;   // descriptor swizzle mode of the P tile
  static constexpr int kTeamBytes = kTile + kPTile;      // V tile, P tile (the K levels live in tensor memory)
  static constexpr int kQTile = (kNQK * 128 + 1023) / 1024 * 1024;
  static constexpr int kMail = CP * 128 * 4;             // end-of-piece deposit of a team: O in its V tile, (l, zs, ref) in its P tile
  static_assert(kMail <= kTile, "the deposit lives in the team's V tile");
  static constexpr int kOffQT = kTeams * kTeamBytes;
  static constexpr int kOffRing = kOffQT + 2 * kQTile;
  static constexpr int kTeamScal = (8 * CP + 4 * 2 * CP + 2 * CP) * 4;   // qs, ref, factor, limits, maxima; reduce scratch; totals
  static constexpr int kFixedTail = 2 * CP * 256 + kTeams * kTeamScal +
                                    8 * kI8PieceUnits * 4 + 2 * 32 + 64 * 8 + (1 + kTeams) * 256 + 64;
  static constexpr int kAvail = 227 * 1024 - 1024 - kOffRing - kFixedTail;
  static constexpr int kNStage = kAvail / kStageBytes > 8 ? 8 : kAvail / kStageBytes;
  static_assert(kNStage >= 2, "ring too small");
  static constexpr int kOffQRaw = kOffRing + kNStage * kStageBytes;
  static constexpr int kOffScal = kOffQRaw + 2 * CP * 256;
  static constexpr int kOffBlk = kOffScal + kTeams * kTeamScal;
  static constexpr int kOffItems = kOffBlk + 8 * kI8PieceUnits * 4;
  static constexpr int kOffBars = kOffItems + 2 * 32;
  static constexpr int kOffMisc = kOffBars + 64 * 8;             // [1 + teams][64] ints
  static constexpr int kSmem = kOffMisc + (1 + kTeams) * 256 + 64 + 1024;   // + alignment slack
  static_assert(kSmem <= 227 * 1024, "shared memory");
  static_assert(kOffScal % 16 == 0 && kTeamScal % 16 == 0 && kOffBars % 8 == 0, "alignment");
  // tensor memory columns of a team: S, O accumulators, FP32 copy of O, K levels (128 bytes per token)
  // (with 32 columns there is no room for the copy: it stays in registers)
  static constexpr bool kOfInTmem = CP <= 16 && !(CP == 8 && !FULL);
  static constexpr int kTmS = 0, kTmO = kNQK, kTmOF = kNQK + kNPV, kTmK = kOfInTmem ? (kTmOF + CP + 7) / 8 * 8 : kTmOF;
  static constexpr int kTmTeam = CP == 32 ? 256 : CP == 16 ? 160 : (CP == 4 || !FULL) ? 96 : 128;
  static constexpr int kTmCols = 512;
  static_assert(kTmK + 32 <= kTmTeam && kTeams * kTmTeam <= 512, "tensor memory");
  static constexpr int kDrainUnits = FULL ? 256 : 4096;  // own units after which the int32 sums could overflow
};

template <>
struct TmemRegs<4> {
  static __device__ __forceinline__ void ld(uint32_t a, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a) : "memory");
  }
  static __device__ __forceinline__ void st(uint32_t a, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};"
                 ::"r"(a), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
  }
};

// Instruction descriptor of kind::i8: int32 accumulate, u8 A, u8 or s8 B, M = 128.
__host__ __device__ constexpr uint32_t i8_idesc(int n, bool mn_major, bool b_signed) {
  return (2u << 4) | ((b_signed ? 1u : 0u) << 10) | ((mn_major ? 1u : 0u) << 15) | ((mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void i8_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void i8_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
// barrier among `n` threads that also ORs a predicate over them
__device__ __forceinline__ bool bar_or(int id, int n, bool pred) {
  uint32_t res;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t"
      "barrier.cta.red.or.pred q, %2, %3, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(res) : "r"(pred ? 1u : 0u), "r"(id), "r"(n) : "memory");
  return res != 0;
}
__device__ __forceinline__ void bar_arrive(int id, int n) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory");
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ex2_ftz(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Packed pairs of FP32 values (one 64-bit register pair, one instruction per pair of operations)
__device__ __forceinline__ uint64_t f2_pack(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float ex2_full(float x) {   // no flush of small results
  float y;
  asm("ex2.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Expand the nibble planes of one tensor of a 128-token raw stage into its u8 level tile.  A warp
// takes 8 token rows per step (512 contiguous raw bytes): lane = (row & 7) * 4 + 16-byte chunk.
template <bool FULL>
__device__ __forceinline__ void i8_expand(uint32_t raw_a, uint32_t raw_r, uint32_t tile, int w4, int lane) {
  const int row8 = lane >> 2, j = lane & 3;
  uint4 xa[4], xr[4];
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const uint32_t off = (uint32_t)(((w4 + 4 * s) * 8 + row8) * 64 + j * 16);
    xa[s] = lds128(raw_a + off);
    if (FULL) xr[s] = lds128(raw_r + off);
  }
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const int row = (w4 + 4 * s) * 8 + row8;
    const uint32_t a[4] = {xa[s].x, xa[s].y, xa[s].z, xa[s].w};
    uint32_t ev[4], od[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (FULL) {
        const uint32_t r[4] = {xr[s].x, xr[s].y, xr[s].z, xr[s].w};
        merge_codes(a[k], r[k], ev[k], od[k]);
      } else {
        ev[k] = a[k] & 0x0F0F0F0Fu;
        od[k] = (a[k] >> 4) & 0x0F0F0F0Fu;
      }
    }
    const uint32_t base = tile + (uint32_t)row * 128u;
    const uint32_t c0 = (uint32_t)((2 * j) ^ (row & 7)) << 4, c1 = (uint32_t)((2 * j + 1) ^ (row & 7)) << 4;
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + c0), "r"(ev[0]), "r"(ev[1]), "r"(ev[2]),
                 "r"(ev[3]) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + c1), "r"(od[0]), "r"(od[1]), "r"(od[2]),
                 "r"(od[3]) : "memory");
  }
}

// K levels of a 128-token raw stage into tensor memory: thread r owns token r (TMEM lane r) and writes
// its 128 level bytes to 32 columns, byte 4 col + b in the order of the operand tiles (see the header).
// The four 16-byte chunks of the row are read in a lane-dependent order (chunk i ^ s, s = (r >> 1) & 3:
// rows are 64 bytes apart, so a fixed order would put a quarter-warp on two bank groups) and put back
// in order with two levels of selects.
template <bool FULL, bool RAW>
__device__ __forceinline__ void i8_expand_k_tmem(uint32_t raw_a, uint32_t raw_r, int r, uint32_t tm_k) {
  const uint32_t s = ((uint32_t)r >> 1) & 3u;
  uint4 xa[4], xr[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t off = (uint32_t)r * 64u + (((uint32_t)i ^ s) << 4);
    xa[i] = lds128(raw_a + off);
    if (FULL) xr[i] = lds128(raw_r + off);
  }
  uint32_t regs[32];
#pragma unroll
  for (int j = 0; j < 4; ++j) {   // (position j ^ s holds chunk j: the copy engine's 64-byte swizzle)
    const uint32_t a[4] = {xa[j].x, xa[j].y, xa[j].z, xa[j].w};
    uint32_t rr[4] = {0, 0, 0, 0};
    if (FULL) { rr[0] = xr[j].x; rr[1] = xr[j].y; rr[2] = xr[j].z; rr[3] = xr[j].w; }
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      if (FULL) {
        merge_codes(a[w], rr[w], regs[8 * j + w], regs[8 * j + 4 + w]);
      } else if (RAW) {   // bytes 16 j + 4 w .. + 3 of the row as they are, and their low nibbles 64 bytes further on
        regs[4 * j + w] = a[w];
        regs[16 + 4 * j + w] = a[w] & 0x0F0F0F0Fu;
      } else {
        regs[8 * j + w] = a[w] & 0x0F0F0F0Fu;
        regs[8 * j + 4 + w] = (a[w] >> 4) & 0x0F0F0F0Fu;
      }
    }
  }
  TmemRegs<32>::st(tm_k, regs);
}

// One of the producer warps: the stream-K bookkeeping (every warp derives the same range and
// pieces; warp 0 alone publishes them, loads the queries and handles empty sequences) and, per
// unit, its share of the plane copies: 8 sub-blocks of 16 tokens x kNArr arrays, two sub-blocks
// per warp.
template <class C, bool FULL>
__device__ __forceinline__ void i8_producer(const AttnParams& p, int pw, int lane, uint32_t ring_u32,
                                            uint32_t full0, uint32_t empty0, uint32_t qfull0, uint32_t qempty0,
                                            uint32_t qraw_u32, uint32_t* blk_s, Item* items, int* misc,
                                            volatile int* abort_word, const I8Maps* maps) {
  constexpr int ST = C::kST, NSTAGE = C::kNStage, NARR = C::kNArr;
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
      if (FULL && p.draft != nullptr) {
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

  constexpr int SPW = 8 / C::kProdWarps;       // 16-token sub-blocks per warp: 1, 2 or 4
  constexpr int RP = SPW * NARR;               // roles of this warp: (sub-block, array)
  const int role = pw * RP + (lane < RP ? lane : 0);
  const int sub = role / NARR, arr = role % NARR, sub_first = SPW * pw;
  const uint32_t my_bytes = 1024u;
  const uint32_t my_dst = (uint32_t)(arr == 0 ? C::kOffKA : arr == 1 ? C::kOffVA : arr == 2 ? C::kOffKR : C::kOffVR) +
                          (uint32_t)sub * my_bytes;
  constexpr uint32_t kBytesSub = (FULL ? 4u : 2u) * 1024u;   // bytes of one sub-block
  uint32_t* my_blk = blk_s + pw * SPW * kI8PieceUnits;   // [SPW sub-blocks][kI8PieceUnits]
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
        bulk_g2s(qraw_u32 + (uint32_t)((qi * C::kColsPad + j * p.G) * LYNX_D * 2),
                 p.q + (((size_t)b * p.nq_stride + j) * p.Hq + (size_t)hkv * p.G) * LYNX_D,
                 (uint32_t)(p.G * LYNX_D * 2), qfull0 + qi * 8);
    }
    for (int c0 = 0; c0 < n; c0 += kI8PieceUnits) {
      const int cn = min(kI8PieceUnits, n - c0);
      for (int i2 = lane; i2 < SPW * cn; i2 += 32) {
        const int i = i2 / SPW;
        const int t0 = (u + c0 + i) * ST + (sub_first + (i2 % SPW)) * 16;
        uint32_t row = 0xFFFFFFFFu;  // sub-block beyond the end of the sequence: nothing to copy
        if (t0 < len) {
          int blk = __ldg(p.block_table + (size_t)b * p.max_blocks + t0 / p.bt);
          if (blk < 0 || blk >= p.num_blocks) {
            atomicOr(p.ws_flags, kFlagBadBlock);
            blk = blk < 0 ? 0 : p.num_blocks - 1;
          }
          row = (uint32_t)(((size_t)blk * p.Hkv + hkv) * p.bt + (t0 % p.bt));
        }
        my_blk[(i2 % SPW) * kI8PieceUnits + i] = row;
      }
      __syncwarp();
      for (int k = 0; k < cn; ++k, ++gs) {
        const int slot = gs % NSTAGE;
        if (gs >= NSTAGE) mbar_wait(empty0 + slot * 8, ((gs / NSTAGE) - 1) & 1, abort_word);
        const uint32_t row = my_blk[(sub - sub_first) * kI8PieceUnits + k];
        const uint32_t bar = full0 + slot * 8;
        if (lane == 0) {
          uint32_t bytes = 0;
#pragma unroll
          for (int i = 0; i < SPW; ++i) bytes += my_blk[i * kI8PieceUnits + k] != 0xFFFFFFFFu ? kBytesSub : 0u;
          if (bytes) mbar_expect_tx(bar, bytes);
          else mbar_arrive(bar);
        }
        __syncwarp();
        if (lane < RP && row != 0xFFFFFFFFu)
          tma_rows16(ring_u32 + slot * C::kStageBytes + my_dst, &maps->m[arr], (int)row, bar);
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

// Largest |q| of a piece's raw queries, by 128 threads (index i of 0..127), reduced over the
// warp; the caller combines the warps.
template <int CP>
__device__ __forceinline__ float i8_q_absmax(const unsigned char* qraw, int i, int nthr) {
  float amax = 0.0f;
  for (int k = i; k < CP * 16; k += nthr) {
    const uint4 v = reinterpret_cast<const uint4*>(qraw)[k];
    const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      amax = fmaxf(amax, fabsf(__uint_as_float(ww[j] << 16)));
      amax = fmaxf(amax, fabsf(__uint_as_float(ww[j] & 0xFFFF0000u)));
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, off));
  return amax;
}
// Fixed-point exponent of a piece's queries: |q * 2^e| < 2^22.
__device__ __forceinline__ int i8_q_exponent(float amax) {
  int e = 0;
  if (amax > 0.0f && amax < INFINITY) e = 21 - (((__float_as_int(amax) >> 23) & 0xFF) - 127);
  return max(-100, min(100, e));
}

// The two halves of a shared-memory matrix descriptor (the MMA-issuing thread keeps the low words of
// its operands in registers and adds the K-step offset: building descriptors is a chain of dependent
// instructions in the one thread everybody waits for).
__host__ __device__ constexpr uint32_t i8_desc_hi(uint32_t sbo_bytes, uint32_t layout) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (layout << 29);
}
__device__ __forceinline__ uint32_t i8_desc_lo(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ uint64_t i8_pack(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
// Shared-memory matrix descriptor with the swizzle mode given (2 = 128 B, 4 = 64 B, 6 = 32 B).
__device__ __forceinline__ uint64_t i8_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}

// Bounded wait until a shared-memory sequence counter has reached `need` (a counter, unlike an mbarrier
// phase, cannot be misread by a waiter that is ahead of the writer).  Gives up after ~2 s like mbar_wait.
__device__ __noinline__ bool seq_wait(const volatile int* ctr, int need, volatile int* abort_word) {
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i) {
      if (*ctr >= need) { __threadfence_block(); return true; }
      __nanosleep(40);
    }
    if (*abort_word) return false;
    if (globaltimer_ns() - t0 > 2000000000ull) { *abort_word = 1; return false; }
  }
}

template <bool FULL, int CP>
__global__ void __launch_bounds__(I8Cfg<FULL, CP>::kThreads, 1) attn_i8_kernel(const AttnParams p,
                                                                               const __grid_constant__ I8Maps maps) {
  using C = I8Cfg<FULL, CP>;
  constexpr int NSTAGE = C::kNStage, T = C::kTeams, G = C::kGroups, CG = C::kCG, TT = C::kTeamThreads;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  unsigned char* qraw = smem + C::kOffQRaw;
  uint32_t* blk_s = reinterpret_cast<uint32_t*>(smem + C::kOffBlk);
  Item* items = reinterpret_cast<Item*>(smem + C::kOffItems);
  int* misc = reinterpret_cast<int*>(smem + C::kOffMisc);
  const int tid = threadIdx.x, lane = tid & 31;
  // (broadcast from lane 0 so that the compiler knows the warp index, and all that follows from it -- team, tiles,
  // operand descriptors -- to be the same for every lane: such values can live in uniform registers)
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);
  const uint32_t ring_u32 = sbase + C::kOffRing;
  const uint32_t full0 = sbase + C::kOffBars, empty0 = full0 + NSTAGE * 8;
  const uint32_t qfull0 = empty0 + NSTAGE * 8, qempty0 = qfull0 + 16;
  const uint32_t qready0 = qempty0 + 16;          // [query slot]  the digit planes of the piece are written
  const uint32_t sfull0 = qready0 + 16;           // [team]  Q.K^T complete: scores valid, K tile free
  const uint32_t pvdone0 = sfull0 + T * 8;        // [team]  P.V complete: P and V tiles free, accumulators current
  volatile int* abort_word = misc;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent grid may be scheduled as SMs become free
  // misc[8] = tensor memory base; misc[16 + t] = deposits written by team t, misc[24 + t] = deposits of team t read;
  // misc[32 + s] = completed phases of raw stage s

  if (tid == 0) {
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(full0 + i * 8, C::kProdWarps);
      mbar_init(empty0 + i * 8, C::kTeamWarps);   // the warps of the team that owns the unit
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(qfull0 + i * 8, 1);
      mbar_init(qempty0 + i * 8, C::kTeamWarps * T);
      mbar_init(qready0 + i * 8, C::kTeamWarps);
    }
    for (int i = 0; i < T; ++i) {
      mbar_init(sfull0 + i * 8, 1);
      mbar_init(pvdone0 + i * 8, 1);
    }
    for (int i = 0; i < (1 + T) * 64 + 16; ++i) misc[i] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // raw query slots (their padding columns stay zero) and query digit planes (their padding rows too)
  for (int i = tid; i < 2 * CP * 256 / 16; i += C::kThreads) reinterpret_cast<uint4*>(qraw)[i] = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < 2 * C::kQTile / 16; i += C::kThreads)
    reinterpret_cast<uint4*>(smem + C::kOffQT)[i] = make_uint4(0, 0, 0, 0);
  // the teams' scalars (the reference exponents must be finite numbers before their first use)
  for (int i = tid; i < T * C::kTeamScal / 4; i += C::kThreads) reinterpret_cast<float*>(smem + C::kOffScal)[i] = 0.0f;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  // nothing in global memory has been touched so far: wait for the grids this one depends on
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp >= C::kProdWarp0) {
    i8_producer<C, FULL>(p, warp - C::kProdWarp0, lane, ring_u32, full0, empty0, qfull0, qempty0,
                         sbase + C::kOffQRaw, blk_s, items, misc, abort_word, &maps);
    return;
  }
  __syncthreads();  // (A)
  const int n_units = misc[7];
  if (n_units == 0) return;

  // ---- tensor memory ---------------------------------------------------------------------------
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(misc + 8)),
                 "r"((uint32_t)C::kTmCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  named_bar(8, T * TT);
  tc_fence_after();
  const uint32_t tmem0 = __shfl_sync(0xFFFFFFFFu, *reinterpret_cast<volatile uint32_t*>(misc + 8), 0);   // (known to be uniform)
  constexpr uint32_t kIdescS = i8_idesc(C::kNQK, false, true), kIdescO = i8_idesc(C::kNPV, true, false);

  // =============================================================================================
  // Teams.  Team t takes the units gs = t, t + T, ... of the CTA's range and does everything for
  // them: K tile, Q.K^T, V tile, scores -> weights, P.V.
  // =============================================================================================
  const int tm = warp / C::kTeamWarps, grp = (warp >> 2) % G, w4 = warp & 3;
  const int r = tid & 127;                        // token of the unit (S), output dim position (O): TMEM lane
  const int tt = r + 128 * grp;                   // thread of the team
  const int c0 = grp * CG;                        // first column of this thread's column group
  const uint32_t lane_sel = (uint32_t)(w4 * 32) << 16;
  const uint32_t tm_s = tmem0 + tm * C::kTmTeam + C::kTmS + c0 + lane_sel;        // + plane * CP
  const uint32_t tm_o = tmem0 + tm * C::kTmTeam + C::kTmO + 4 * c0 + lane_sel;
  const uint32_t tm_of = tmem0 + tm * C::kTmTeam + C::kTmOF + c0 + lane_sel;
  float* my_scal = reinterpret_cast<float*>(smem + C::kOffScal + tm * C::kTeamScal);
  float* qs_s = my_scal, *ref_s = my_scal + CP, *fac_s = my_scal + 2 * CP;
  int* lim_s = reinterpret_cast<int*>(my_scal + 3 * CP);
  float* amax_s = my_scal + 4 * CP;               // [team warps]
  const float* zero_s = my_scal + 5 * CP;         // [CP] zeros (never written after the set-up)
  float* my_red = my_scal + 8 * CP;               // [team warps][2 CG]
  float* my_lz = my_scal + 16 * CP;               // [2 CP]
  const int tw = grp * 4 + w4;                    // warp of the team
  int* my_misc = misc + 64 * (1 + tm);
  const int bar_tm = 1 + tm;                      // named barrier of this team
  const uint32_t vtile = sbase + tm * C::kTeamBytes, ptile = vtile + C::kTile;
  float* my_hdr = reinterpret_cast<float*>(smem + tm * C::kTeamBytes + C::kTile);   // [3 CP] l, zs, ref of this team's deposit (in its idle P tile)
  const uint32_t tm_k = tmem0 + tm * C::kTmTeam + C::kTmK;
  const int dim_out = 32 * (r >> 5) + 8 * ((r >> 2) & 3) + 2 * (r & 3) + ((r >> 4) & 1);   // head dim of lane r of O
  // this thread's row of the P tile: 16-byte chunk j goes to position j ^ p_swz
  const uint32_t p_swz = C::kPRow == 32 ? ((uint32_t)r >> 2) & 1u : C::kPRow == 64 ? ((uint32_t)r >> 1) & 3u : (uint32_t)r & 7u;
  const uint32_t p_row = ptile + (uint32_t)r * C::kPRow;
  const float cb = p.sm_log2;
  // descriptor low words of the MMA operands (used by the team's issuing thread)
  const uint32_t qd_lo0 = i8_desc_lo(sbase + C::kOffQT, 16u), vd_lo = i8_desc_lo(vtile, 16384u), pd_lo = i8_desc_lo(ptile, 16384u);
  constexpr uint32_t kQdHi = i8_desc_hi(1024u, 2u), kVdHi = i8_desc_hi(1024u, 2u),
                     kPdHi = i8_desc_hi(8u * C::kPRow, (uint32_t)C::kPLayout);
  uint32_t dep_cnt[T];                            // deposits made so far, per team (every team keeps the same count)
#pragma unroll
  for (int i = 0; i < T; ++i) dep_cnt[i] = 0;
  uint32_t my_deps = 0;                           // this team's own deposits
  bool ack_pending = false;                       // this team's last deposit (in its V tile) may not have been read yet

  int gs_base = 0, ic = 0;
  while (gs_base < n_units) {
    const int qi = ic & 1;
    mbar_wait(qfull0 + qi * 8, (ic >> 1) & 1, abort_word);
    const Item item = items[qi];
    const int len = item.len, n_piece = item.pad0;
    const int team0 = gs_base % T;                        // team of the piece's first unit
    const int u_first = (tm - team0 + T) % T;             // this team's units of the piece: u_first, u_first + T, ...
    const int team_f = (gs_base + n_piece - 1) % T;       // team of the piece's last unit: it writes the piece's result
    if (u_first < n_piece) {
      const bool finisher = tm == team_f;
      const int full_lim = p.causal ? len - p.tail + 1 : len;
      // ---- the piece's queries: fixed-point exponent, sum of q per column, causal limits ----------
      const unsigned char* qb = qraw + qi * CP * 256;
      {
        const float am = i8_q_absmax<CP>(qb, tt, TT);
        if (lane == 0) amax_s[tw] = am;
        for (int c = tw; c < CP; c += C::kTeamWarps) {
          const uint2 v = *reinterpret_cast<const uint2*>(qb + c * 256 + lane * 8);
          float sum = (__uint_as_float(v.x << 16) + __uint_as_float(v.x & 0xFFFF0000u)) +
                      (__uint_as_float(v.y << 16) + __uint_as_float(v.y & 0xFFFF0000u));
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
          if (lane == 0) qs_s[c] = sum;
        }
        if (tt < CP) lim_s[tt] = tt < p.ncols ? (p.causal ? len - p.tail + tt / p.G + 1 : len) : 0;
        named_bar(bar_tm, TT);
      }
      float amax = 0.0f;
#pragma unroll
      for (int i = 0; i < C::kTeamWarps; ++i) amax = fmaxf(amax, amax_s[i]);
      const int e = i8_q_exponent(amax);
      const float ca = p.sm_log2 * __int_as_float((127 - e) << 23) * ((FULL || C::kRawK) ? 1.0f : 16.0f);
      const uint32_t qt = sbase + C::kOffQT + qi * C::kQTile;
      if (u_first == 0 && tt < CP * 4) {
        // this team owns the piece's first unit: it writes the three balanced s8 digit planes of
        // q_int = rint(q 2^e), rows plane * CP + column.  (The slot's previous planes belong to the piece
        // before last, which every team has left: the queries of this piece were loaded after that.)
        const float up = __int_as_float((127 + e) << 23);
        const int c = tt >> 2, j = tt & 3;
        constexpr int NP = C::kQPlanes;
        uint32_t pl[NP][2][4];   // [plane][half][word]
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const uint4 v = *reinterpret_cast<const uint4*>(qb + c * 256 + j * 64 + w * 16);
          const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
          uint32_t acc[NP][2];
#pragma unroll
          for (int pln = 0; pln < NP; ++pln) { acc[pln][0] = 0; acc[pln][1] = 0; }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            int qv2[2];
#pragma unroll
            for (int par = 0; par < 2; ++par) {
              const float f = par ? __uint_as_float(ww[i] & 0xFFFF0000u) : __uint_as_float(ww[i] << 16);
              const int qv = __float2int_rn(f * up);
              qv2[par] = max(-4194303, min(4194303, qv));
            }
            // half 0 / 1 of the row: even / odd dims -- or, where K goes in as raw bytes, what multiplies the
            // byte pair m (dims 2m, 2m+1; odd value) and its low nibble (16 x even value - odd value)
            int val[2] = {qv2[0], qv2[1]};
            if (C::kRawK) { val[0] = qv2[1]; val[1] = 16 * qv2[0] - qv2[1]; }
#pragma unroll
            for (int par = 0; par < 2; ++par) {
              int qv = val[par];
#pragma unroll
              for (int pln = 0; pln < NP; ++pln) {
                const int dgt = (int)(signed char)(qv & 0xFF);
                acc[pln][par] |= (uint32_t)(dgt & 0xFF) << (8 * i);
                qv = (qv - dgt) >> 8;
              }
            }
          }
#pragma unroll
          for (int pln = 0; pln < NP; ++pln) { pl[pln][0][w] = acc[pln][0]; pl[pln][1][w] = acc[pln][1]; }
        }
#pragma unroll
        for (int pln = 0; pln < NP; ++pln) {
          const int n = pln * CP + c;
#pragma unroll
          for (int par = 0; par < 2; ++par) {
            const int chunk = C::kRawK ? 4 * par + j : 2 * j + par;   // 16 bytes of the row's 128
            const uint32_t a = qt + (uint32_t)n * 128u + ((uint32_t)(chunk ^ (n & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pl[pln][par][0]),
                         "r"(pl[pln][par][1]), "r"(pl[pln][par][2]), "r"(pl[pln][par][3]) : "memory");
          }
        }
      }
      if (u_first == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(qready0 + qi * 8);
      }

      uint64_t l2[CG / 2], zs2[CG / 2];   // softmax sums, two columns per register pair
      float of_r[C::kOfInTmem ? 1 : CG];   // FP32 copy of O where tensor memory has no room for it
#pragma unroll
      for (int c = 0; c < CG / 2; ++c) { l2[c] = 0ull; zs2[c] = 0ull; }
      bool fresh = true, have_of = false;
      int units_in_acc = 0;
      uint32_t n_own = (uint32_t)((gs_base + u_first) / T);   // index of the unit among this team's units

      // Ends the current accumulation (the team's last P.V is complete): the int32 accumulators, four
      // byte planes per column, are added to the FP32 copy and the sum is scaled by fac_s[] (the change
      // of the reference exponents).
      auto drain = [&](bool scale) {
        if (units_in_acc > 0) {
          tc_fence_after();
#pragma unroll
          for (int c4 = 0; c4 < CG / 4; ++c4) {
            uint32_t a[16], of[4];
            TmemRegs<16>::ld(tm_o + c4 * 16, a);
            if (C::kOfInTmem && have_of) TmemRegs<4>::ld(tm_of + c4 * 4, of);
            tc_wait_ld();
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float v = fmaf(fmaf(fmaf((float)(int)a[4 * k + 3], 256.0f, (float)(int)a[4 * k + 2]), 256.0f,
                                        (float)(int)a[4 * k + 1]), 256.0f, (float)(int)a[4 * k]);
              const float old = !have_of ? 0.0f : C::kOfInTmem ? __uint_as_float(of[k]) : of_r[C::kOfInTmem ? 0 : c4 * 4 + k];
              const float nw = (old + v) * (scale ? fac_s[c0 + c4 * 4 + k] : 1.0f);
              of[k] = __float_as_uint(nw);
              if (!C::kOfInTmem) of_r[C::kOfInTmem ? 0 : c4 * 4 + k] = nw;
            }
            if (C::kOfInTmem) TmemRegs<4>::st(tm_of + c4 * 4, of);
          }
          if (C::kOfInTmem) tc_wait_st();
          have_of = true;
          units_in_acc = 0;
        } else if (have_of && scale) {
#pragma unroll
          for (int c4 = 0; c4 < CG / 4; ++c4) {
            if (C::kOfInTmem) {
              uint32_t of[4];
              TmemRegs<4>::ld(tm_of + c4 * 4, of);
              tc_wait_ld();
#pragma unroll
              for (int k = 0; k < 4; ++k) of[k] = __float_as_uint(__uint_as_float(of[k]) * fac_s[c0 + c4 * 4 + k]);
              TmemRegs<4>::st(tm_of + c4 * 4, of);
            } else {
#pragma unroll
              for (int k = 0; k < 4; ++k) of_r[C::kOfInTmem ? 0 : c4 * 4 + k] *= fac_s[c0 + c4 * 4 + k];
            }
          }
          if (C::kOfInTmem) tc_wait_st();
        }
      };

      // Metadata of this thread's token, read with plain loads two steps ahead: the block id of the unit
      // after next (a block-table look-up whose result is first touched one step later, so that nothing
      // waits for it), the (scale, zero) pairs of the next unit.
      const int bt_shift = (p.bt & (p.bt - 1)) == 0 ? 31 - __clz(p.bt) : -1;   // block size a power of two?
      auto blk_of = [&](int uu) -> int {      // the raw table entry (0 where there is no such token)
        const int t = (item.pad1 + uu) * C::kST + r;
        if (uu >= n_piece || t >= len) return 0;
        const int bi = bt_shift >= 0 ? t >> bt_shift : t / p.bt;
        return __ldg(p.block_table + (size_t)item.b * p.max_blocks + bi);
      };
      auto row_of = [&](int uu, int blk) -> uint32_t {
        const int t = (item.pad1 + uu) * C::kST + r;
        if (uu >= n_piece || t >= len) return 0xFFFFFFFFu;
        const int in_blk = bt_shift >= 0 ? t & (p.bt - 1) : t % p.bt;
        blk = min(max(blk, 0), p.num_blocks - 1);     // (out-of-range ids are reported by the producer)
        return (uint32_t)(((size_t)blk * p.Hkv + item.hkv) * p.bt + in_blk);
      };
      auto meta_of = [&](uint32_t row, float2& k2, float2& v2) {
        k2 = make_float2(0.f, 0.f); v2 = k2;
        if (row != 0xFFFFFFFFu) {
          k2 = __ldg(reinterpret_cast<const float2*>(p.km) + row);
          v2 = __ldg(reinterpret_cast<const float2*>(p.vm) + row);
        }
      };
      int blk_n1 = blk_of(u_first + T), blk_n2 = blk_of(u_first + 2 * T);
      float2 km_c, vm_c;
      meta_of(row_of(u_first, blk_of(u_first)), km_c, vm_c);

      for (int u = u_first; u < n_piece; u += T, ++n_own) {
        const int gs = gs_base + u, slot = gs % NSTAGE;
        const int unit_t0 = (item.pad1 + u) * C::kST;
        const int tok = unit_t0 + r;
        const uint32_t st = ring_u32 + slot * C::kStageBytes;
        // stages are shared between the teams: the wait for this stage's phase gs / NSTAGE is only well
        // defined once the phase before it is known to be complete (its owner says so in misc[32 + slot])
        if (gs >= NSTAGE && *reinterpret_cast<volatile int*>(misc + 32 + slot) < gs / NSTAGE)
          seq_wait(misc + 32 + slot, gs / NSTAGE, abort_word);
        mbar_wait(full0 + slot * 8, (gs / NSTAGE) & 1, abort_word);
        if (tt == 0) *reinterpret_cast<volatile int*>(misc + 32 + slot) = gs / NSTAGE + 1;
        float2 km = km_c, vm = vm_c;
        meta_of(row_of(u + T, blk_n1), km_c, vm_c);   // for this team's next unit
        blk_n1 = blk_n2;
        blk_n2 = blk_of(u + 3 * T);                   // and the block id of the one after the one after
        if (ack_pending) {   // uniform over the team: its last deposit (in the V tile) has been read
          if (tt == 0) seq_wait(misc + 24 + tm, (int)my_deps, abort_word);
          named_bar(bar_tm, TT);
          ack_pending = false;
        }
        // ---- K levels (free: the team's previous Q.K^T has been waited for), then Q.K^T; V tile (free
        // once the team's previous P.V is complete).  With two column groups one expands K, the other V.
        if (G == 1 || grp == 0) {
          i8_expand_k_tmem<FULL, C::kRawK>(st + C::kOffKA, st + C::kOffKR, r, tm_k + lane_sel);
          tc_wait_st();
        } else {
          if (n_own > 0) mbar_wait(pvdone0 + tm * 8, (n_own - 1) & 1, abort_word);
          i8_expand<FULL>(st + C::kOffVA, st + C::kOffVR, vtile, w4, lane);
        }
        tc_fence_before();
        named_bar(bar_tm, TT);
        if (tt == 0) {
          if (u == u_first) mbar_wait(qready0 + qi * 8, (ic >> 1) & 1, abort_word);   // the piece's query planes
          tc_fence_after();
          const uint32_t d = tmem0 + tm * C::kTmTeam + C::kTmS;
          const uint32_t qd_lo = qd_lo0 + (uint32_t)qi * (C::kQTile >> 4);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            i8_mma_ts(d, tm_k + (uint32_t)k4 * 8u, i8_pack(qd_lo + (uint32_t)k4 * 2u, kQdHi), kIdescS, k4 > 0 ? 1u : 0u);
          tc_commit(sfull0 + tm * 8);
        }
        __syncwarp();
        if (G == 1 || grp == 0) {   // (the other group has waited already)
          if (n_own > 0) mbar_wait(pvdone0 + tm * 8, (n_own - 1) & 1, abort_word);
        }
        if (G == 1) i8_expand<FULL>(st + C::kOffVA, st + C::kOffVR, vtile, w4, lane);
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + slot * 8);
        const bool valid = tok < len;
        if (!valid) { km = make_float2(0.f, 0.f); vm = make_float2(0.f, 0.f); }
        const float sve = fmaxf(FULL ? vm.x : 16.0f * vm.x, 9.094947e-13f);   // floor 2^-40
        const float al = km.x * ca;
        const float be = (FULL ? km.y : fmaf(km.x, 8.0f, km.y)) * cb;
        const float lsv = lg2_approx(sve);
        const float ia = valid ? rcp_approx(sve) : 0.0f;
        const float ib = (FULL ? vm.y : fmaf(vm.x, 8.0f, vm.y)) * ia;

        // ---- scores of this thread's token -------------------------------------------------------
        mbar_wait(sfull0 + tm * 8, n_own & 1, abort_word);
        tc_fence_after();
        // y = log2 of the weight relative to the column's reference exponent, two columns per register pair
        uint64_t y2[CG / 2];
        {
          uint32_t s0[CG], s1[CG], s2[CG], s3[C::kRawK ? CG : 1];
          TmemRegs<CG>::ld(tm_s, s0);
          TmemRegs<CG>::ld(tm_s + CP, s1);
          TmemRegs<CG>::ld(tm_s + 2 * CP, s2);
          if (C::kRawK) TmemRegs<CG>::ld(tm_s + 3 * CP, s3);
          tc_wait_ld();
          const uint64_t al2 = f2_pack(al, al), be2 = f2_pack(be, be), lsv2 = f2_pack(lsv, lsv);
          const uint64_t k256 = C::kRawK ? f2_pack(65536.0f, 65536.0f) : f2_pack(256.0f, 256.0f);
          const float* ref_r = fresh ? zero_s : ref_s;   // (a piece's first unit: relative to zero)
#pragma unroll
          for (int c = 0; c < CG / 2; ++c) {
            uint64_t hi, lo;   // the digit-plane sums put together: exact in int32 two planes at a time
            if (C::kRawK) {
              hi = f2_pack((float)((int)s3[2 * c] * 256 + (int)s2[2 * c]), (float)((int)s3[2 * c + 1] * 256 + (int)s2[2 * c + 1]));
              lo = f2_pack((float)((int)s1[2 * c] * 256 + (int)s0[2 * c]), (float)((int)s1[2 * c + 1] * 256 + (int)s0[2 * c + 1]));
            } else {
              hi = f2_pack((float)((int)s2[2 * c] * 256 + (int)s1[2 * c]), (float)((int)s2[2 * c + 1] * 256 + (int)s1[2 * c + 1]));
              lo = f2_pack((float)(int)s0[2 * c], (float)(int)s0[2 * c + 1]);
            }
            const uint64_t qs2 = *reinterpret_cast<const uint64_t*>(qs_s + c0 + 2 * c);
            const uint64_t rf2 = *reinterpret_cast<const uint64_t*>(ref_r + c0 + 2 * c);
            y2[c] = f2_fma(f2_fma(hi, k256, lo), al2, f2_fma(be2, qs2, f2_sub(lsv2, rf2)));
          }
        }
        if (unit_t0 + C::kST > full_lim) {
#pragma unroll
          for (int c = 0; c < CG / 2; ++c) {
            float a, b;
            f2_unpack(y2[c], a, b);
            if (tok >= lim_s[c0 + 2 * c]) a = -INFINITY;
            if (tok >= lim_s[c0 + 2 * c + 1]) b = -INFINITY;
            y2[c] = f2_pack(a, b);
          }
        }
        // ---- reference exponents: raised when a weight would leave the u32 range -----------------------
        float ymax = -INFINITY;
#pragma unroll
        for (int c = 0; c < CG / 2; ++c) {
          float a, b;
          f2_unpack(y2[c], a, b);
          ymax = max3(ymax, a, b);
        }
        // A restart of the accumulation (new reference exponents, the int32 sums drained into the FP32 copy)
        // is a decision of the whole team: one P.V covers all columns.  Where it is known beforehand (first
        // unit of a piece, sums about to overflow) it is taken first.  Otherwise every thread writes its
        // weights at once and a thread whose weight would leave the u32 range raises a flag, which all
        // look at after the barrier that completes the P tile anyway: the common case has no barrier of
        // its own for the question.
        const bool forced = fresh || units_in_acc >= C::kDrainUnits;   // uniform over the team
        const bool over = ymax > 31.5f;
        volatile int* raise_flag = my_misc + 2;
        auto restart = [&]() {
#pragma unroll
          for (int c = 0; c < CG; ++c) {   // (rare path: back to absolute exponents x = y + ref)
            float a, b;
            f2_unpack(y2[c >> 1], a, b);
            float mx = ((c & 1) ? b : a) + (fresh ? 0.0f : ref_s[c0 + c]);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
            if (lane == 0) my_red[tw * CG + c] = mx;
          }
          named_bar(bar_tm, TT);
          if (tt == 0) *raise_flag = 0;
          if (tt < CP) {
            const float* mr = my_red + (tt / CG) * 4 * CG + (tt % CG);   // the four warps of the column's group
            const float mx = fmaxf(fmaxf(mr[0], mr[CG]), fmaxf(mr[2 * CG], mr[3 * CG]));
            const float old = fresh ? 0.0f : ref_s[tt];
            float nw = old, f = 1.0f;
            if (fresh) { nw = fmaxf(mx, -1.0e4f) - 28.0f; f = 0.0f; }
            else if (mx - old > 31.5f) { nw = mx - 28.0f; f = ex2_full(old - nw); }
            ref_s[tt] = nw;
            fac_s[tt] = f;
            my_red[C::kTeamWarps * CG + tt] = nw - old;   // what the change takes off every exponent of the column
          }
          named_bar(bar_tm, TT);
#pragma unroll
          for (int c = 0; c < CG / 2; ++c) {
            const uint64_t f2 = *reinterpret_cast<const uint64_t*>(fac_s + c0 + 2 * c);
            l2[c] = f2_mul(l2[c], f2);
            zs2[c] = f2_mul(zs2[c], f2);
            // the exponents again, relative to the new references
            const uint64_t od = *reinterpret_cast<const uint64_t*>(my_red + C::kTeamWarps * CG + c0 + 2 * c);
            y2[c] = f2_sub(y2[c], od);
          }
          drain(true);   // (the team's previous P.V has been waited for)
          fresh = false;
        };
        // weights of this thread's token into its row of the P tile; `commit`: add them to the softmax sums
        auto weights = [&](bool commit) {
          uint32_t wi[CG];
          const uint64_t ia2 = f2_pack(ia, ia), ib2 = f2_pack(ib, ib);
#pragma unroll
          for (int c = 0; c < CG / 2; ++c) {
            float a, b;
            f2_unpack(y2[c], a, b);
            const float wa = ex2_ftz(a), wb = ex2_ftz(b);
            asm("cvt.rni.u32.f32 %0, %1;" : "=r"(wi[2 * c]) : "f"(wa));
            asm("cvt.rni.u32.f32 %0, %1;" : "=r"(wi[2 * c + 1]) : "f"(wb));
            if (commit) {   // (not for weights beyond the range: they may be infinite)
              const uint64_t w2 = f2_pack(wa, wb);
              l2[c] = f2_fma(w2, ia2, l2[c]);
              zs2[c] = f2_fma(w2, ib2, zs2[c]);
            }
          }
#pragma unroll
          for (int j = 0; j < CG / 4; ++j)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                         ::"r"(p_row + (((uint32_t)(grp * (CG / 4) + j) ^ p_swz) << 4)), "r"(wi[4 * j]), "r"(wi[4 * j + 1]),
                           "r"(wi[4 * j + 2]), "r"(wi[4 * j + 3]) : "memory");
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          tc_fence_before();
          named_bar(bar_tm, TT);     // the P tile and the V tile are complete, S has been read
        };
        if (C::kVoteFirst) {   // (every instance but the 4-column anchor one measures faster with the question asked first)
          if (bar_or(bar_tm, TT, forced || over)) restart();
          weights(true);
        } else {
          if (forced) restart();
          else if (over) *raise_flag = 1;
          // (a thread beyond the range keeps its weights out of the sums: after the restart they are different ones)
          weights(forced || !over);
          if (!forced && *raise_flag != 0) {   // uniform: read after the barrier; cleared inside restart()
            restart();
            weights(over);
          }
        }
        if (tt == 0) {
          tc_fence_after();
          const uint32_t d = tmem0 + tm * C::kTmTeam + C::kTmO;
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            i8_mma_ss(d, i8_pack(vd_lo + (uint32_t)k4 * (4096u >> 4), kVdHi),
                      i8_pack(pd_lo + (uint32_t)k4 * ((32u * C::kPRow) >> 4), kPdHi),
                      kIdescO, (units_in_acc > 0 || k4 > 0) ? 1u : 0u);
          tc_commit(pvdone0 + tm * 8);
        }
        __syncwarp();
        ++units_in_acc;
      }
      // ---- end of the piece for this team -----------------------------------------------------------
      mbar_wait(pvdone0 + tm * 8, (n_own - 1) & 1, abort_word);   // the last P.V
      drain(false);   // the FP32 copy now holds this team's part of O
      float of[CG];
#pragma unroll
      for (int c4 = 0; c4 < CG / 4; ++c4) {
        if (C::kOfInTmem) {
          uint32_t t[4];
          TmemRegs<4>::ld(tm_of + c4 * 4, t);
          tc_wait_ld();
#pragma unroll
          for (int k = 0; k < 4; ++k) of[c4 * 4 + k] = __uint_as_float(t[k]);
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k) of[c4 * 4 + k] = of_r[C::kOfInTmem ? 0 : c4 * 4 + k];
        }
      }
      tc_fence_before();
      // totals of l and zs over the 128 token lanes of every column group
#pragma unroll
      for (int c = 0; c < CG; ++c) {
        float a, b;
        {
          float l_lo, l_hi, z_lo, z_hi;
          f2_unpack(l2[c >> 1], l_lo, l_hi);
          f2_unpack(zs2[c >> 1], z_lo, z_hi);
          a = (c & 1) ? l_hi : l_lo;
          b = (c & 1) ? z_hi : z_lo;
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          a += __shfl_xor_sync(0xFFFFFFFFu, a, off);
          b += __shfl_xor_sync(0xFFFFFFFFu, b, off);
        }
        if (lane == 0) { my_red[tw * 2 * CG + c] = a; my_red[tw * 2 * CG + CG + c] = b; }
      }
      named_bar(bar_tm, TT);
      if (tt < 2 * CP) {   // my_lz: l of the CP columns, then zs
        const int which = tt / CP, c = tt % CP;
        const float* mr = my_red + (c / CG) * 4 * 2 * CG + which * CG + (c % CG);   // the four warps of the column's group
        my_lz[tt] = (mr[0] + mr[2 * CG]) + (mr[4 * CG] + mr[6 * CG]);
      }
      named_bar(bar_tm, TT);
      if (!finisher) {
        // deposit O in this team's V tile and (l, zs, ref) in its P tile (both idle: its last P.V is
        // complete), for the team that owns the piece's last unit
        float* mail = reinterpret_cast<float*>(smem + tm * C::kTeamBytes);
#pragma unroll
        for (int c = 0; c < CG; ++c) mail[(c0 + c) * 128 + r] = of[c];
        if (tt < CP) {
          my_hdr[tt] = my_lz[tt];
          my_hdr[CP + tt] = my_lz[CP + tt];
          my_hdr[2 * CP + tt] = ref_s[tt];
        }
        __threadfence_block();
        named_bar(bar_tm, TT);
        ++my_deps;
        if (tt == 0) *reinterpret_cast<volatile int*>(misc + 16 + tm) = (int)my_deps;
        ack_pending = true;
      } else {
        float lt[CG], zt[CG], mt[CG];
#pragma unroll
        for (int c = 0; c < CG; ++c) { lt[c] = my_lz[c0 + c]; zt[c] = my_lz[CP + c0 + c]; mt[c] = ref_s[c0 + c]; }
#pragma unroll
        for (int d = 0; d < T; ++d) {
          if (d == tm || (d - team0 + T) % T >= n_piece) continue;   // itself; a team without a unit in the piece
          if (tt == 0) seq_wait(misc + 16 + d, (int)dep_cnt[d] + 1, abort_word);   // its deposit is complete
          named_bar(bar_tm, TT);
          const float* mo = reinterpret_cast<const float*>(smem + d * C::kTeamBytes);
          const float* mh = reinterpret_cast<const float*>(smem + d * C::kTeamBytes + C::kTile);
#pragma unroll
          for (int c = 0; c < CG; ++c) {
            const float o2 = mo[(c0 + c) * 128 + r], l2 = mh[c0 + c];
            const float z2 = mh[CP + c0 + c], m2 = mh[2 * CP + c0 + c];
            const float M = fmaxf(mt[c], m2);
            const float f1 = ex2_full(mt[c] - M), f2 = ex2_full(m2 - M);
            of[c] = of[c] * f1 + o2 * f2;
            lt[c] = lt[c] * f1 + l2 * f2;
            zt[c] = zt[c] * f1 + z2 * f2;
            mt[c] = M;
          }
          __threadfence_block();
          named_bar(bar_tm, TT);
          if (tt == 0) *reinterpret_cast<volatile int*>(misc + 24 + d) = (int)dep_cnt[d] + 1;   // it may deposit again
        }
        const bool direct = item.n_contrib == 1;
        const size_t bh = (size_t)item.b * p.Hkv + item.hkv;
        float* part = p.ws_part + (bh + (size_t)blockIdx.x) * (size_t)C::kPartCols * kPartStride;
#pragma unroll
        for (int cc = 0; cc < CG; ++cc) {
          const int c = c0 + cc;
          if (c >= p.ncols) break;
          const float v = of[cc] + zt[cc];
          if (direct) {
            const int j = c / p.G, hh = c % p.G;
            p.out[(((size_t)item.b * p.nq_stride + j) * p.Hq + item.hkv * p.G + hh) * LYNX_D + dim_out] =
                lt[cc] > 0.0f ? v / lt[cc] : 0.0f;
            if (r == 0) p.ws_lse[((size_t)item.b * p.nq_stride + j) * p.Hq + item.hkv * p.G + hh] = lse_of(mt[cc], lt[cc]);
          } else {
            part[(size_t)c * kPartStride + dim_out] = v;
            if (r == 0) { part[(size_t)c * kPartStride + 128] = mt[cc]; part[(size_t)c * kPartStride + 129] = lt[cc]; }
          }
        }
        __threadfence();
        finish_piece<FULL, C::kPartCols, TT>(p, item, direct, tt, my_misc, bar_tm);
      }
    }
    // every team keeps count of every team's deposits (the phase of its deposit barrier)
#pragma unroll
    for (int d = 0; d < T; ++d)
      if (d != team_f && (d - team0 + T) % T < n_piece) ++dep_cnt[d];
    __syncwarp();
    if (lane == 0) mbar_arrive(qempty0 + qi * 8);
    gs_base += n_piece;
    ++ic;
  }
  // ---- release the tensor memory ---------------------------------------------------------------
  tc_fence_before();
  named_bar(9, T * TT);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem0), "r"((uint32_t)C::kTmCols)
                 : "memory");
  }
  if (tid == 0 && misc[0]) atomicOr(p.ws_flags, kFlagTimeout);
}

template <bool FULL, int CP>
lynx_status launch_i8(const AttnParams& p, cudaStream_t st) {
  using C = I8Cfg<FULL, CP>;
  auto kern = attn_i8_kernel<FULL, CP>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmem) != cudaSuccess)
      return LYNX_ERR_CUDA;
    configured[dev] = true;
  }
  const long long cap_units = (long long)p.B * p.Hkv * (((long long)p.max_blocks * p.bt + C::kST - 1) / C::kST);
  long long grid = (cap_units + 3) / 4;
  const long long full = sm_count();   // one CTA per SM
  grid = grid < 1 ? 1 : (grid > full ? full : grid);
  // Programmatic dependent launch: when the kernel before this one in the stream is of the same kind (one
  // launch per layer of a decoder), this grid's CTAs may become resident, and set up their shared and tensor
  // memory, while the last CTAs of that kernel are still merging; they read nothing before
  // griddepcontrol.wait, i.e. before that kernel has completed and its memory is visible.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(C::kThreads);
  cfg.dynamicSmemBytes = C::kSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  I8Maps maps;
  const uint64_t plane_rows = (uint64_t)p.num_blocks * p.Hkv * p.bt;
  if (!i8_plane_map(&maps.m[0], p.ka, plane_rows, true) || !i8_plane_map(&maps.m[1], p.va, plane_rows, false))
    return LYNX_ERR_CUDA;
  if (FULL) {
    if (!i8_plane_map(&maps.m[2], p.kr, plane_rows, true) || !i8_plane_map(&maps.m[3], p.vr, plane_rows, false))
      return LYNX_ERR_CUDA;
  } else {
    maps.m[2] = maps.m[0];
    maps.m[3] = maps.m[1];
  }
  if (cudaLaunchKernelEx(&cfg, kern, p, maps) != cudaSuccess) return LYNX_ERR_CUDA;
  return launch_status();
}
