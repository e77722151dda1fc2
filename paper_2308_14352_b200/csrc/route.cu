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
#include "router.cuh"
#include "scatter.cuh"

namespace emoe {
namespace {

template <int TT>
__global__ void __launch_bounds__(ROUTER_THREADS)
    router_topk_kernel(const void* __restrict__ x, int x_bf16, int T, int d, const float* __restrict__ Wr,
                       const float* __restrict__ bias, int bias_stride, int E, int EP, int ep_shift, int top_k,
                       int renorm, int32_t* __restrict__ ids, float* __restrict__ gates,
                       float* __restrict__ logits) {
  extern __shared__ float smem[];
  pdl_trigger();
  router_logits<TT>(smem, x, x_bf16, T, d, Wr, bias, bias_stride, E, EP, ep_shift, logits);
  const float* zs = smem + TT * router_dc(TT) + ROUTER_THREADS * TT;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int tt = warp; tt < TT; tt += ROUTER_THREADS / 32) {  // a warp per token, in turns when the CTA owns more tokens than warps
    const int t = blockIdx.x * TT + tt;
    if (t >= T) return;
    int my_id;
    float my_gate;
    router_pick(zs + tt * EP, E, top_k, renorm, lane, my_id, my_gate);
    if (lane < top_k) {
      ids[static_cast<size_t>(t) * top_k + lane] = my_id;
      gates[static_cast<size_t>(t) * top_k + lane] = my_gate;
    }
  }
}

// Router, Top-K, permutation, scatter and work plan in one launch for small batches: one CTA per
// token.  A CTA computes its token's picks, publishes them, and waits until every CTA of the grid
// has done so (an arrival counter in global memory; the host launches this kernel only with a
// grid that is resident at once, and the wait is bounded).  Then it works out the slots of its
// own pairs exactly as permute_scatter_kernel does and copies its row into them; CTA 0 also
// writes counts, offsets and the plan.  sync[0] counts arrivals, sync[1] departures; the last CTA
// to leave sets both back to zero for the next launch.
constexpr int RPS_MAX_PAIRS = 1024;
__global__ void __launch_bounds__(ROUTER_THREADS)
    route_permute_scatter_kernel(const __nv_bfloat16* __restrict__ x, int T, int d, const float* __restrict__ Wr,
                                 const float* __restrict__ bias, int bias_stride, int E, int EP, int ep_shift, int top_k,
                                 int renorm, int32_t* ids, float* __restrict__ gates,
                                 const ExpertDev* __restrict__ experts, int fmt, int32_t* __restrict__ counts,
                                 int32_t* __restrict__ off, int32_t* __restrict__ perm,
                                 int32_t* __restrict__ slot_of_pair, int* __restrict__ plan, int* __restrict__ check_word,
                                 __nv_bfloat16* __restrict__ xs_out, float* __restrict__ xsc, unsigned* sync,
                                 unsigned wait_limit, int extra_arrivals) {
  extern __shared__ float smem[];
  __shared__ int s_ids[RPS_MAX_PAIRS];
  __shared__ int s_off[EMOE_MAX_EXPERTS + 1];
  __shared__ int s_red[2][ROUTER_THREADS / 32];
  __shared__ int s_ok;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = blockIdx.x;
  const int n_pairs = T * top_k;
  // The next kernel of the chain is scheduled once every CTA of this grid has executed this, i.e.
  // once the whole grid is resident: it cannot take the room of a CTA the wait below needs.
  pdl_trigger();
  router_logits<1>(smem, x, 1, T, d, Wr, bias, bias_stride, E, EP, ep_shift, nullptr);  // waits on the kernels in front
  // should this CTA's wait run out, the expert kernel behind must find an empty plan, not an old one
  if (t == 0 && tid == 0) plan[0] = 0;
  if (warp == 0) {
    int my_id;
    float my_gate;
    router_pick(smem + ROUTER_DC + ROUTER_THREADS, E, top_k, renorm, lane, my_id, my_gate);
    if (lane < top_k) {
      ids[static_cast<size_t>(t) * top_k + lane] = my_id;
      gates[static_cast<size_t>(t) * top_k + lane] = my_gate;
    }
  }
  __syncthreads();
  if (tid == 0 && gridDim.x == 1) s_ok = 1;  // a single CTA has nobody to wait for
  if (tid == 0 && gridDim.x > 1) {
    __threadfence();
    atomicAdd(&sync[0], 1u);
    unsigned seen = 0, polls = 0;
    int ok = 1;
    for (;;) {
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(sync) : "memory");
      if (seen >= static_cast<unsigned>(T + extra_arrivals)) break;
      if (++polls > wait_limit) {
        ok = 0;
        break;
      }
    }
    if (ok) {
      if (atomicAdd(&sync[1], 1u) == static_cast<unsigned>(T) - 1u) {  // every CTA has passed its wait
        sync[0] = 0;
        sync[1] = 0;
        __threadfence();
      }
    } else {
      atomicOr(check_word, CHECK_WAIT_TIMEOUT);
    }
    s_ok = ok;
  }
  __syncthreads();
  if (!s_ok) return;
  for (int q = tid; q < n_pairs; q += ROUTER_THREADS) s_ids[q] = __ldcg(ids + q);
  __syncthreads();
  if (t == 0) {
    // counts, offsets, plan (this CTA only); invalid ids cannot occur here: the picks lie in [0, E)
    for (int ee = tid; ee <= E; ee += ROUTER_THREADS) s_off[ee] = 0;
    __syncthreads();
    for (int q = tid; q < n_pairs; q += ROUTER_THREADS) atomicAdd(&s_off[s_ids[q] + 1], 1);
    __syncthreads();
    if (warp == 0) counts_to_offsets(s_off, counts, E, lane);
    __syncthreads();
    for (int ee = tid; ee <= E; ee += ROUTER_THREADS) off[ee] = s_off[ee];
    if (warp == 0) build_plan(plan, experts, s_off, E, 1, 0x7fffffff, lane);
  }
  for (int j = 0; j < top_k; ++j) {
    const int p = t * top_k + j;
    const int e = s_ids[p];
    int before = 0;
    for (int q = tid; q < n_pairs; q += ROUTER_THREADS) {
      const int eq = s_ids[q];
      before += eq < e || (eq == e && q < p);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
    __syncthreads();  // s_red of the previous pair has been read
    if (lane == 0) s_red[0][warp] = before;
    __syncthreads();
    int slot = 0;
#pragma unroll
    for (int w = 0; w < ROUTER_THREADS / 32; ++w) slot += s_red[0][w];
    if (tid == 0) {
      perm[slot] = p;
      slot_of_pair[p] = slot;
    }
    scatter_any(x + static_cast<size_t>(t) * d, xs_out, xsc, slot, d, experts[e].bits, fmt, check_word);
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
  // 8 tokens per CTA once there are enough tokens to fill the GPU that way, else 1 (32 tokens per CTA, which
  // would cut the re-reads of the router matrix from L2, was measured three times slower at 2048 tokens: 64 CTAs,
  // each bound by its shared-memory reads)
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

bool route_permute_scatter_supported(const LayerDims& L, int T, int resident_ctas) {
  return L.act_bf16 && T * L.top_k <= RPS_MAX_PAIRS && L.E <= EMOE_MAX_EXPERTS && 2 * T <= resident_ctas;
}

int route_permute_scatter_resident_ctas(int device) {
  int per_sm = 0, sms = 0;
  const size_t smem = sizeof(float) * (ROUTER_DC + ROUTER_THREADS + EMOE_MAX_EXPERTS);
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, route_permute_scatter_kernel, ROUTER_THREADS, smem) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return 0;
  return per_sm * sms;
}

cudaError_t launch_route_permute_scatter(const LayerDims& L, const ExpertDev* experts, const void* x, int T, const float* Wr,
                                         const float* bias, int bias_stride, int32_t* ids, float* gates, int32_t* counts,
                                         int32_t* off, int32_t* perm, int32_t* slot_of_pair, int* plan, __nv_bfloat16* xs,
                                         float* xsc, int fmt, unsigned* sync, unsigned wait_limit, int extra_arrivals,
                                         int* check_word, cudaStream_t st) {
  int EP = 1, sh = 0;
  while (EP < L.E) {
    EP <<= 1;
    ++sh;
  }
  const size_t smem = sizeof(float) * (ROUTER_DC + ROUTER_THREADS + EP);
  return launch_chain(route_permute_scatter_kernel, dim3(T), dim3(ROUTER_THREADS), smem, st,
                      reinterpret_cast<const __nv_bfloat16*>(x), T, L.d_model, Wr, bias, bias_stride, L.E, EP, sh, L.top_k,
                      static_cast<int>(L.gate_mode == EMOE_GATE_SOFTMAX_RENORM), ids, gates, experts, fmt, counts, off, perm,
                      slot_of_pair, plan, check_word, xs, xsc, sync, wait_limit, extra_arrivals);
}

cudaError_t launch_permute(const int32_t* ids, int n_pairs, int E, int32_t* counts, int32_t* off, int32_t* perm,
                           int32_t* slot_of_pair, int* check_word, cudaStream_t st) {
  const size_t smem = sizeof(int) * (2 * E + 32 * E);
  return launch_chain(permute_kernel, dim3(1), dim3(1024), smem, st, ids, n_pairs, E, counts, off, perm, slot_of_pair, check_word);
}

}  // namespace emoe
