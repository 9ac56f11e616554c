// lynx_token_verify: token-level verification of a speculated window (Section 4.3; the acceptance rule of
// speculative sampling that Section 2.4 refers to), on sm_100a.
//
// Draft tokens s_1..s_k were drawn from the Anchor-state distributions p_i; the verification pass gives the
// full-precision distributions q_1..q_{k+1}.  Token i is accepted iff u_i p_i(s_i) < q_i(s_i) (probability
// min(1, q/p), no division); the first rejected position j is corrected by a token drawn from
// norm(max(0, q_j - p_j)), and if all are accepted a bonus token is drawn from q_{k+1} -- both by inverse CDF
// in vocabulary order with the uniform r.  The random numbers are inputs.
//
// One CTA per sequence.  The acceptance scan touches k values (a lane per position); the correction reads one or two vocabulary rows
// (4 or 8 bytes per entry) once, with coalesced loads: the 32 warps sum the row in chunks of 128 entries
// (four chunks of a warp in flight) into shared memory, one warp scans the chunk sums for the chunk that
// holds r * total and walks that chunk with a warp scan per step.  HBM-bound by construction, and small: the
// point of this kernel is that the decision stays on the device.
#include "lynx_common.cuh"

namespace lynx {
namespace {

constexpr int kTvThreads = 512, kTvWarps = kTvThreads / 32;
constexpr int kCh = 4;   // chunks of a warp in flight

__global__ void __launch_bounds__(kTvThreads) token_verify_kernel(const float* __restrict__ p_probs,
                                                                  const float* __restrict__ q_probs,
                                                                  const int32_t* __restrict__ draft,
                                                                  const float* __restrict__ u,
                                                                  const float* __restrict__ r, int k, int V,
                                                                  int32_t* __restrict__ n_accepted,
                                                                  int32_t* __restrict__ next_token) {
  extern __shared__ float csum[];   // [chunks of 128 entries]
  __shared__ int j_s, again_s;
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float* p = p_probs + (size_t)b * k * V;
  const float* q = q_probs + (size_t)b * (k + 1) * V;
  if (warp == 0) {   // the acceptance scan: a lane per position, all loads in flight together (k <= 64: two rounds)
    int j = k;
    for (int base = 0; base < k && j == k; base += 32) {
      const int i = base + lane;
      bool reject = false;
      if (i < k) {
        int s = draft[(size_t)b * k + i];
        s = s < 0 ? 0 : (s >= V ? V - 1 : s);
        reject = !(u[(size_t)b * k + i] * p[(size_t)i * V + s] < q[(size_t)i * V + s]);
      }
      const unsigned hit = __ballot_sync(0xFFFFFFFFu, reject);
      if (hit != 0u) j = base + __ffs(hit) - 1;
    }
    if (lane == 0) {
      j_s = j;
      n_accepted[b] = j;
    }
  }
  __syncthreads();
  const int j = j_s;
  const float* qj = q + (size_t)j * V;
  const float* pj = j < k ? p + (size_t)j * V : nullptr;
  const int n_chunks = (V + 127) / 128;
  bool residual = pj != nullptr;
  // rows start on 16-byte boundaries when the arrays do and V is a multiple of 4
  const bool vec = (V & 3) == 0 && ((reinterpret_cast<uintptr_t>(p_probs) | reinterpret_cast<uintptr_t>(q_probs)) & 15u) == 0;
  auto weight = [&](int x) -> float {
    if (x >= V) return 0.0f;
    return residual ? fmaxf(__ldg(qj + x) - __ldg(pj + x), 0.0f) : __ldg(qj + x);
  };
  for (int pass = 0; pass < 2; ++pass) {   // a second pass only if the residual is zero everywhere: w = q_j
    // chunk sums: four chunks of a warp in flight at a time, all their loads issued before the first use
    // (branch-free: an index beyond the row is clamped and its value masked).  With 16-byte alignment a lane takes
    // four consecutive entries of a chunk in one load, else entry 32 e + lane in step e.
    for (int c = warp * kCh; c < n_chunks; c += kTvWarps * kCh) {
      float s[kCh];
      if (vec) {
        float4 a[kCh], d[kCh];
#pragma unroll
        for (int i = 0; i < kCh; ++i) {
          const int x = (c + i) * 128 + lane * 4;
          const int xx = x < V ? x : 0;
          a[i] = __ldg(reinterpret_cast<const float4*>(qj + xx));
          d[i] = residual ? __ldg(reinterpret_cast<const float4*>(pj + xx)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int i = 0; i < kCh; ++i) {
          const float v = residual ? (fmaxf(a[i].x - d[i].x, 0.0f) + fmaxf(a[i].y - d[i].y, 0.0f)) +
                                         (fmaxf(a[i].z - d[i].z, 0.0f) + fmaxf(a[i].w - d[i].w, 0.0f))
                                   : (a[i].x + a[i].y) + (a[i].z + a[i].w);
          s[i] = (c + i) * 128 + lane * 4 < V ? v : 0.0f;
        }
      } else {
#pragma unroll
        for (int i = 0; i < kCh; ++i) {
          float a[4], d[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int x = (c + i) * 128 + e * 32 + lane;
            const int xx = x < V ? x : 0;
            a[e] = __ldg(qj + xx);
            d[e] = residual ? __ldg(pj + xx) : 0.0f;
          }
          s[i] = 0.0f;
#pragma unroll
          for (int e = 0; e < 4; ++e)
            s[i] += (c + i) * 128 + e * 32 + lane < V ? (residual ? fmaxf(a[e] - d[e], 0.0f) : a[e]) : 0.0f;
        }
      }
#pragma unroll
      for (int i = 0; i < kCh; ++i) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) s[i] += __shfl_xor_sync(0xFFFFFFFFu, s[i], off);
        if (lane == 0 && c + i < n_chunks) csum[c + i] = s[i];
      }
    }
    __syncthreads();
    if (warp == 0) {
      float total = 0.0f;
      for (int c = lane; c < n_chunks; c += 32) total += csum[c];
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, off);
      if (residual && !(total > 0.0f)) {
        if (lane == 0) again_s = 1;
      } else {
        if (lane == 0) again_s = 0;
        const float t = r[b] * total;
        // the chunk that holds t: inclusive scan of the chunk sums, 32 at a time
        float run = 0.0f, before = 0.0f;
        int chunk = -1;
        for (int base = 0; base < n_chunks && chunk < 0; base += 32) {
          const float v = base + lane < n_chunks ? csum[base + lane] : 0.0f;
          float inc = v;
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) {
            const float o = __shfl_up_sync(0xFFFFFFFFu, inc, off);
            if (lane >= off) inc += o;
          }
          const unsigned hit = __ballot_sync(0xFFFFFFFFu, base + lane < n_chunks && run + inc > t);
          if (hit != 0u) {
            const int l = __ffs(hit) - 1;
            chunk = base + l;
            before = run + __shfl_sync(0xFFFFFFFFu, inc - v, l);
          }
          run += __shfl_sync(0xFFFFFFFFu, inc, 31);
        }
        if (chunk < 0) {   // rounding left t at or above the total: the last chunk with weight, from its start
          chunk = n_chunks - 1;
          before = run - csum[n_chunks - 1];
        }
        // walk the chunk in vocabulary order
        float c = before;
        int pick = min(V, (chunk + 1) * 128) - 1;
        bool found = false;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int x = chunk * 128 + e * 32 + lane;
          const float v = weight(x);
          float inc = v;
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) {
            const float o = __shfl_up_sync(0xFFFFFFFFu, inc, off);
            if (lane >= off) inc += o;
          }
          const unsigned hit = __ballot_sync(0xFFFFFFFFu, x < V && c + inc > t);
          if (hit != 0u && !found) {
            pick = chunk * 128 + e * 32 + (__ffs(hit) - 1);
            found = true;
          }
          c += __shfl_sync(0xFFFFFFFFu, inc, 31);
        }
        if (lane == 0) next_token[b] = pick;
      }
    }
    __syncthreads();
    if (!again_s) break;   // (uniform over the CTA)
    residual = false;
  }
}

}  // namespace
}  // namespace lynx

extern "C" lynx_status lynx_token_verify(const float* p_probs, const float* q_probs, const int32_t* draft_tokens,
                                         const float* u, const float* r, int32_t batch, int32_t k, int32_t vocab,
                                         int32_t* n_accepted, int32_t* next_token, void* stream) {
  using namespace lynx;
  if (batch == 0) return LYNX_OK;
  if (batch < 0 || k <= 0 || k > 64 || vocab <= 0) return LYNX_ERR_SHAPE;
  if (!p_probs || !q_probs || !draft_tokens || !u || !r || !n_accepted || !next_token) return LYNX_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t smem = (size_t)((vocab + 127) / 128) * sizeof(float);
  if (smem > 48 * 1024) return LYNX_ERR_UNSUPPORTED;   // vocabularies beyond 1.5 M entries
  token_verify_kernel<<<(unsigned)batch, kTvThreads, smem, st>>>(p_probs, q_probs, draft_tokens, u, r, k, vocab,
                                                                 n_accepted, next_token);
  return launch_status();
}
