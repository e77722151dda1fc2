// Router logits and Top-K gating as device functions (paper Section 2.1: a trained router sends
// every token to its Top-K experts), shared by the kernels that route: the router kernel, the
// one-launch routing kernel and the one-launch decode layer.
#pragma once
#include <math_constants.h>

#include "common.cuh"

namespace emoe {

constexpr int ROUTER_THREADS = 256;
constexpr int ROUTER_DC = 1024;  // d_model chunk held in shared memory (1 and 8 tokens per CTA)
// tokens per CTA -> chunk: 32 tokens take chunks of 256 so that their rows still fit shared memory
__host__ __device__ constexpr int router_dc(int tt) { return tt > 8 ? 256 : ROUTER_DC; }

// Logits of the CTA's TT tokens into zs[TT][EP] (shared memory).  x and the router weights are
// inputs of the call: the logits are computed while the kernels in front drain; the wait on
// them comes before the first write to global memory (ids / gates may still be read there).
template <int TT>
__device__ __forceinline__ void router_logits(float* smem, const void* __restrict__ x, int x_bf16, int T, int d,
                                              const float* __restrict__ Wr, const float* __restrict__ bias,
                                              int bias_stride, int E, int EP, int ep_shift, float* __restrict__ logits) {
  constexpr int DC = router_dc(TT);
  float* xs = smem;                          // [TT][DC]
  float* red = xs + TT * DC;                 // [S][TT][EP]
  float* zs = red + ROUTER_THREADS * TT;     // [TT][EP]
  const int tid = threadIdx.x;
  const int e = tid & (EP - 1);
  const int slice = tid >> ep_shift;
  const int S = ROUTER_THREADS >> ep_shift;
  const int t0 = blockIdx.x * TT;

  float acc[TT];
#pragma unroll
  for (int tt = 0; tt < TT; ++tt) acc[tt] = 0.0f;

  for (int c0 = 0; c0 < d; c0 += DC) {
    const int dc = min(DC, d - c0);
    __syncthreads();
    for (int tt = 0; tt < TT; ++tt) {
      const int t = t0 + tt;
      for (int i = tid; i < dc; i += ROUTER_THREADS) {
        float v = 0.0f;
        if (t < T) {
          const size_t src = static_cast<size_t>(t) * d + c0 + i;
          v = x_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[src])
                     : reinterpret_cast<const float*>(x)[src];
        }
        xs[tt * DC + i] = v;
      }
    }
    __syncthreads();
    if (e < E) {
      // many independent router-weight loads in flight per thread (the loop is L2-latency bound;
      // with one token per CTA the registers allow 24)
      constexpr int U = TT == 1 ? 24 : 8;
      for (int i = slice; i < dc; i += U * S) {
        float w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int ii = i + u * S;
          w[u] = ii < dc ? __ldg(Wr + static_cast<size_t>(c0 + ii) * E + e) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int ii = min(i + u * S, dc - 1);
#pragma unroll
          for (int tt = 0; tt < TT; ++tt) acc[tt] = fmaf(xs[tt * DC + ii], w[u], acc[tt]);
        }
      }
    }
  }
#pragma unroll
  for (int tt = 0; tt < TT; ++tt) red[(slice * TT + tt) * EP + e] = acc[tt];
  __syncthreads();
  pdl_wait();
  for (int idx = tid; idx < TT * EP; idx += ROUTER_THREADS) {
    const int tt = idx >> ep_shift, ee = idx & (EP - 1);
    const int t = t0 + tt;
    float z = 0.0f;
    for (int s = 0; s < S; ++s) z += red[(s * TT + tt) * EP + ee];
    if (ee < E && t < T) {
      if (bias) z += bias[static_cast<size_t>(t) * bias_stride + ee];
      if (logits) logits[static_cast<size_t>(t) * E + ee] = z;
    }
    zs[idx] = z;
  }
  __syncthreads();
}

// Softmax and Top-K of one token by one warp from its row of logits zrow[EP] (shared memory):
// K rounds of arg-max, ties to the lower expert index.  Lane r < top_k returns the r-th pick.
__device__ __forceinline__ void router_pick(const float* zrow, int E, int top_k, int renorm, int lane, int& out_id,
                                            float& out_gate) {
  constexpr int MAXJ = EMOE_MAX_EXPERTS / 32;
  float zv[MAXJ], pe[MAXJ];
  float m = -CUDART_INF_F;
#pragma unroll
  for (int j = 0; j < MAXJ; ++j) {
    const int ee = lane + 32 * j;
    zv[j] = ee < E ? zrow[ee] : -CUDART_INF_F;
    m = fmaxf(m, zv[j]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float denom = 0.0f;
#pragma unroll
  for (int j = 0; j < MAXJ; ++j) {
    pe[j] = (lane + 32 * j) < E ? expf(zv[j] - m) : 0.0f;
    denom += pe[j];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, o);

  unsigned taken = 0;
  float psel = 0.0f;
  int my_id = 0;     // lane r keeps the r-th pick
  float my_p = 0.0f;
  for (int r = 0; r < top_k; ++r) {
    float bv = -CUDART_INF_F;
    int bi = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < MAXJ; ++j) {
      const int ee = lane + 32 * j;
      if (ee < E && !((taken >> j) & 1u) && (zv[j] > bv || bi == 0x7fffffff)) {
        bv = zv[j];
        bi = ee;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (oi != 0x7fffffff && (bi == 0x7fffffff || ov > bv || (ov == bv && oi < bi))) {
        bv = ov;
        bi = oi;
      }
    }
    float p = 0.0f;
#pragma unroll
    for (int j = 0; j < MAXJ; ++j)
      if (lane + 32 * j == bi) {
        taken |= 1u << j;
        p = pe[j];
      }
    p = __shfl_sync(0xffffffffu, p, bi & 31) / denom;
    psel += p;
    if (lane == r) {
      my_id = bi;
      my_p = p;
    }
  }
  out_id = my_id;
  out_gate = renorm ? my_p / psel : my_p;
}

}  // namespace emoe
