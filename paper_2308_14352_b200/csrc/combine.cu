// Gather / weighted combine (paper Sections 1/2.1: a token's output is the gate-weighted sum
// of its Top-K experts' outputs):  y[t] = sum_j gates[t][j] * o[slot of pair (t,j)], j ascending.
// Expert outputs arrive in expert-sorted order and possibly as several split-K partial sums,
// which are added first, in a fixed order.  Pure streaming: one float4 of y per thread, a row of
// blocks per token.
#include "common.cuh"

namespace emoe {
namespace {

__global__ void __launch_bounds__(256)
    combine_kernel(const float* __restrict__ o_part, int ksplit, size_t part_stride, const float* __restrict__ gates,
                   const int32_t* __restrict__ slot_of_pair, int T, int top_k, int d, float* __restrict__ y) {
  // a block row per token: no index division in front of the first load
  const int d4 = d >> 2;
  const int t = blockIdx.x;
  const int c = blockIdx.y * blockDim.x + threadIdx.x;
  pdl_wait();
  pdl_trigger();
  if (c >= d4) return;
  const size_t idx = static_cast<size_t>(t) * d4 + c;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j = 0; j < top_k; ++j) {
    const int slot = slot_of_pair[t * top_k + j];
    if (slot < 0) continue;
    const float g = gates[t * top_k + j];
    const float4* src = reinterpret_cast<const float4*>(o_part + static_cast<size_t>(slot) * d) + c;
    float4 v = src[0];
#pragma unroll 4
    for (int z = 1; z < ksplit; ++z) {
      const float4 u = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(src) + z * part_stride);
      v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
    }
    acc.x = fmaf(g, v.x, acc.x);
    acc.y = fmaf(g, v.y, acc.y);
    acc.z = fmaf(g, v.z, acc.z);
    acc.w = fmaf(g, v.w, acc.w);
  }
  reinterpret_cast<float4*>(y)[idx] = acc;
}

}  // namespace

cudaError_t launch_combine(const float* o_part, int ksplit, size_t n_pairs_stride, const float* gates,
                           const int32_t* slot_of_pair, int T, int top_k, int d, float* y, cudaStream_t st) {
  const int d4 = d >> 2;
  const int threads = d4 >= 256 ? 256 : (d4 + 31) / 32 * 32;
  return launch_chain(combine_kernel, dim3(T, (d4 + threads - 1) / threads), dim3(threads), 0, st, o_part, ksplit, n_pairs_stride * d * sizeof(float), gates,
                      slot_of_pair, T, top_k, d, y);
}

}  // namespace emoe
