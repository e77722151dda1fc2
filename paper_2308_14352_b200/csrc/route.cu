// Router + Top-K gating and the token -> expert permutation (paper Sections 1 and 2.1: a
// trained router sends every token to its Top-K experts).
//
// router_topk_kernel: a CTA owns TT tokens.  Threads are laid out as (expert, slice of the
// d_model axis); router_W is streamed once per CTA with expert-contiguous (coalesced) reads
// while the tokens' activations sit in shared memory.  One warp per token then does the
// softmax and the K rounds of arg-max with shuffles (ties go to the lower expert index).
//
// permute_kernel: one CTA, deterministic.  Histogram (integer shared-memory atomics),
// warp-scan of the histogram, then a stable scatter: pairs are visited in chunks of 1024
// in index order, ranks inside a warp come from match/ballot, ranks across warps from a
// per-warp count table, so no order-dependent atomics decide a position.
#include <math_constants.h>

#include "common.cuh"

namespace emoe {
namespace {

constexpr int ROUTER_THREADS = 256;
constexpr int ROUTER_DC = 1024;  // d_model chunk held in shared memory

template <int TT>
__global__ void __launch_bounds__(ROUTER_THREADS)
    router_topk_kernel(const void* __restrict__ x, int x_bf16, int T, int d, const float* __restrict__ Wr,
                       const float* __restrict__ bias, int bias_stride, int E, int EP, int ep_shift, int top_k,
                       int renorm, int32_t* __restrict__ ids, float* __restrict__ gates,
                       float* __restrict__ logits) {
  extern __shared__ float smem[];
  float* xs = smem;                          // [TT][ROUTER_DC]
  float* red = xs + TT * ROUTER_DC;          // [S][TT][EP]
  float* zs = red + ROUTER_THREADS * TT;     // [TT][EP]
  const int tid = threadIdx.x;
  const int e = tid & (EP - 1);
  const int slice = tid >> ep_shift;
  const int S = ROUTER_THREADS >> ep_shift;
  const int t0 = blockIdx.x * TT;

  // x and the router weights are inputs of the call: the logits are computed while the kernels
  // in front drain; the wait comes before the first write (ids / gates may still be read there)
  pdl_trigger();
  float acc[TT];
#pragma unroll
  for (int tt = 0; tt < TT; ++tt) acc[tt] = 0.0f;

  for (int c0 = 0; c0 < d; c0 += ROUTER_DC) {
    const int dc = min(ROUTER_DC, d - c0);
    __syncthreads();
    for (int idx = tid; idx < TT * dc; idx += ROUTER_THREADS) {
      const int tt = idx / dc, i = idx - tt * dc;
      const int t = t0 + tt;
      float v = 0.0f;
      if (t < T) {
        const size_t src = static_cast<size_t>(t) * d + c0 + i;
        v = x_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[src])
                   : reinterpret_cast<const float*>(x)[src];
      }
      xs[tt * ROUTER_DC + i] = v;
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
          for (int tt = 0; tt < TT; ++tt) acc[tt] = fmaf(xs[tt * ROUTER_DC + ii], w[u], acc[tt]);
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

  const int warp = tid >> 5, lane = tid & 31;
  if (warp >= TT) return;
  const int t = t0 + warp;
  if (t >= T) return;

  constexpr int MAXJ = EMOE_MAX_EXPERTS / 32;
  float zv[MAXJ], pe[MAXJ];
  float m = -CUDART_INF_F;
#pragma unroll
  for (int j = 0; j < MAXJ; ++j) {
    const int ee = lane + 32 * j;
    zv[j] = ee < E ? zs[warp * EP + ee] : -CUDART_INF_F;
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
  if (lane < top_k) {
    ids[static_cast<size_t>(t) * top_k + lane] = my_id;
    gates[static_cast<size_t>(t) * top_k + lane] = renorm ? my_p / psel : my_p;
  }
}

__global__ void __launch_bounds__(1024)
    permute_kernel(const int32_t* __restrict__ ids, int n, int E, int32_t* __restrict__ counts,
                   int32_t* __restrict__ off, int32_t* __restrict__ perm, int32_t* __restrict__ slot_of_pair,
                   int* __restrict__ check_word) {
  extern __shared__ int sm[];
  int* cnt = sm;          // [E]
  int* cursor = cnt + E;  // [E]
  int* wcnt = cursor + E; // [32][E]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  pdl_wait();
  pdl_trigger();
  for (int e = tid; e < E; e += 1024) cnt[e] = 0;
  __syncthreads();
  bool bad = false;
  for (int p = tid; p < n; p += 1024) {
    const int e = ids[p];
    if (e >= 0 && e < E) atomicAdd(&cnt[e], 1);
    else bad = true;
  }
  if (bad) atomicOr(check_word, CHECK_BAD_EXPERT_ID);
  __syncthreads();
  if (warp == 0) {
    const int ch = (E + 31) / 32;
    int local = 0;
    for (int i = 0; i < ch; ++i) {
      const int e = lane * ch + i;
      if (e < E) local += cnt[e];
    }
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    int run = incl - local;
    for (int i = 0; i < ch; ++i) {
      const int e = lane * ch + i;
      if (e < E) {
        cursor[e] = run;
        off[e] = run;
        counts[e] = cnt[e];
        run += cnt[e];
      }
    }
    if (lane == 31) off[E] = incl;
  }
  __syncthreads();
  // pairs with an id outside [0, E) own no slot: the slots behind the last valid one read as "no pair"
  for (int p = off[E] + tid; p < n; p += 1024) perm[p] = -1;

  for (int base = 0; base < n; base += 1024) {
    for (int i = tid; i < 32 * E; i += 1024) wcnt[i] = 0;
    __syncthreads();
    const int p = base + tid;
    const int e = p < n ? ids[p] : -1;
    const bool ok = e >= 0 && e < E;
    const unsigned act = __ballot_sync(0xffffffffu, ok);
    int rank = 0;
    if (ok) {
      const unsigned same = __match_any_sync(act, e);
      rank = __popc(same & ((1u << lane) - 1u));
      if (rank == 0) wcnt[warp * E + e] = __popc(same);
    }
    __syncthreads();
    if (ok) {
      int prefix = 0;
      for (int w = 0; w < warp; ++w) prefix += wcnt[w * E + e];
      const int pos = cursor[e] + prefix + rank;
      perm[pos] = p;
      if (slot_of_pair) slot_of_pair[p] = pos;
    } else if (p < n && slot_of_pair) {
      slot_of_pair[p] = -1;
    }
    __syncthreads();
    for (int ee = tid; ee < E; ee += 1024) {
      int tot = 0;
      for (int w = 0; w < 32; ++w) tot += wcnt[w * E + ee];
      cursor[ee] += tot;
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_router_topk(const void* x, int x_bf16, int T, int d, const float* Wr, const float* bias,
                               int bias_stride, int E, int top_k, int renorm, int32_t* ids, float* gates,
                               float* logits, cudaStream_t st) {
  int EP = 1, sh = 0;
  while (EP < E) {
    EP <<= 1;
    ++sh;
  }
  // 8 tokens per CTA once there are enough tokens to fill the GPU that way, else 1
  if (T >= 8 * 64) {
    constexpr int TT = 8;
    const size_t smem = sizeof(float) * (TT * ROUTER_DC + ROUTER_THREADS * TT + TT * EP);  // <= 48 KB
    return launch_chain(router_topk_kernel<TT>, dim3((T + TT - 1) / TT), dim3(ROUTER_THREADS), smem, st, x, x_bf16, T, d, Wr, bias,
                        bias_stride, E, EP, sh, top_k, renorm, ids, gates, logits);
  } else {
    constexpr int TT = 1;
    const size_t smem = sizeof(float) * (TT * ROUTER_DC + ROUTER_THREADS * TT + TT * EP);
    return launch_chain(router_topk_kernel<TT>, dim3(T), dim3(ROUTER_THREADS), smem, st, x, x_bf16, T, d, Wr, bias, bias_stride, E,
                        EP, sh, top_k, renorm, ids, gates, logits);
  }
  return cudaGetLastError();
}

cudaError_t launch_permute(const int32_t* ids, int n_pairs, int E, int32_t* counts, int32_t* off, int32_t* perm,
                           int32_t* slot_of_pair, int* check_word, cudaStream_t st) {
  const size_t smem = sizeof(int) * (2 * E + 32 * E);
  return launch_chain(permute_kernel, dim3(1), dim3(1024), smem, st, ids, n_pairs, E, counts, off, perm, slot_of_pair, check_word);
}

}  // namespace emoe
