// lynx_lse_merge: joins two attention results over disjoint key sets (sm_100a).
//
// The decode node's KV cache is the transferred prefix, held in the Lynx planes (Section 4.1 stage 4), followed by
// the tokens it generated itself, which were never quantised and stay BF16 pages.  Section 2's
// softmax(q K^T scale) V over the concatenation is the average of the two parts' own attentions weighted by
// e^lse of their scores: the attention kernels leave the natural-log log-sum-exp of every output row in their
// workspace (lynx_workspace_lse, lynx_bf16_workspace_lse), and this kernel forms the weighted average.
// One warp per output row of 128 floats; HBM-bound and tiny next to the attention passes.
#include "lynx_common.cuh"

namespace lynx {
namespace {

__global__ void __launch_bounds__(256) lse_merge_kernel(const float4* __restrict__ out_a, const float* __restrict__ lse_a,
                                                        const float4* __restrict__ out_b, const float* __restrict__ lse_b,
                                                        int64_t n_rows, float4* out, float* lse_out) {
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const int lane = threadIdx.x & 31;
  const float la = __ldg(lse_a + row), lb = __ldg(lse_b + row);
  const float m = fmaxf(la, lb);
  float wa = 0.0f, wb = 0.0f, l = -INFINITY;
  if (m > -INFINITY) {   // (an empty part has lse = -inf and weight 0; two empty parts give a zero row)
    const float ea = expf(la - m), eb = expf(lb - m);
    const float inv = 1.0f / (ea + eb);
    wa = ea * inv;
    wb = eb * inv;
    l = m + logf(ea + eb);
  }
  // (weight 0 must also silence whatever an empty part's row holds)
  const float4 a = wa > 0.0f ? out_a[row * 32 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
  const float4 b = wb > 0.0f ? out_b[row * 32 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
  out[row * 32 + lane] = make_float4(a.x * wa + b.x * wb, a.y * wa + b.y * wb, a.z * wa + b.z * wb, a.w * wa + b.w * wb);
  if (lse_out && lane == 0) lse_out[row] = l;
}

}  // namespace
}  // namespace lynx

extern "C" lynx_status lynx_lse_merge(const float* out_a, const float* lse_a, const float* out_b, const float* lse_b,
                                      int64_t n_rows, float* out, float* lse_out, void* stream) {
  using namespace lynx;
  if (n_rows == 0) return LYNX_OK;
  if (n_rows < 0 || n_rows > (1ll << 40)) return LYNX_ERR_SHAPE;
  if (!out_a || !lse_a || !out_b || !lse_b || !out) return LYNX_ERR_NULL;
  if (!aligned16(out_a) || !aligned16(out_b) || !aligned16(out)) return LYNX_ERR_ALIGN;
  lse_merge_kernel<<<(unsigned)((n_rows + 7) / 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const float4*>(out_a), lse_a, reinterpret_cast<const float4*>(out_b), lse_b, n_rows,
      reinterpret_cast<float4*>(out), lse_out);
  return launch_status();
}
