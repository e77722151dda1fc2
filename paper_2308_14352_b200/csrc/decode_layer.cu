// A whole MoE layer in ONE launch for a handful of tokens on a small layer (paper Sections 2.1 and
// 3.2: router, Top-K, the activated experts' FFNs on their packed codes, gate-weighted sum; the
// paper's target is single-request decoding, where every step of the layer is a few microseconds
// of work and the launches and dependencies between kernels are most of the time).
//
// The grid is resident at once (the host sizes it from the device's capacity and the call's
// work: one to three CTAs per SM), so its CTAs may wait for one another; every such wait is bounded.
//   1. The d_model axis of every token's router product is cut into slices, one CTA each; a CTA
//      writes its partial logits and counts itself in.  Every CTA waits until all slices have
//      arrived, adds the partial logits up in slice order and makes the picks itself (the Top-K
//      device function of the router kernel), so that no second wait is needed to spread them.
//      Each warp then asks for the rows of the second projection it will need (L2 prefetch).
//   2. First projection: one warp per (pair, four hidden channels) streams its packed rows
//      with 128-bit loads, all started before the first is used, decodes in registers, reads
//      the activations once for all of them, accumulates in fp32 and stores the activated values
//      in the activation type.  The CTAs then meet at a grid-wide arrival counter.
//   3. Second projection and gate-weighted sum: four, two or one warps share one (token, four
//      output channels), each takes its part of the hidden axis of every expert of the token; the
//      parts are added in a fixed order, so the result does not depend on timing.
// The last CTA also writes the bookkeeping the library keeps per call (counts, offsets, permutation).
// sync[0] counts the routing arrivals, sync[1] the arrivals after the first projection, sync[2]
// the departures; the last CTA to leave sets all three back to zero for the next launch.
#include "common.cuh"
#include "router.cuh"

namespace emoe {
namespace {

constexpr int DL_THREADS = ROUTER_THREADS;
constexpr int DL_WARPS = DL_THREADS / 32;
constexpr int DL_MAX_PAIRS = 16;
constexpr int DL_WPR_MAX = 4;                // most warps that share a row block of the second projection (a.wpr: 1, 2 or 4)
constexpr int DL_R_MAX = 4;                  // consecutive rows of a matrix one warp takes at once
constexpr long long DL_MAX_WEIGHTS = 8LL << 20;  // per matrix: beyond this a layer is bandwidth-bound and streams better

struct DecodeLayerArgs {
  LayerDims L;
  const ExpertDev* experts;
  const void* x;
  int T;
  const float* Wr;       // null: the picks are given (ids_in / gates_in)
  const float* bias;
  int bias_stride, EP, ep_shift, renorm;
  int rsplit;            // slices of the d_model axis per token in the router product
  int wpr;               // warps per row block in the second projection: 1, 2 or 4
  float* zpart;          // [T][rsplit][EP] partial logits
  const int32_t* ids_in;
  const float* gates_in;
  int32_t* ids;
  float* gates;
  int32_t *counts, *off, *perm, *slot_of_pair;
  void* hidden;  // [pairs][d_ff], activation type
  float* y;      // [T][d_model]
  unsigned* sync;
  unsigned wait_limit;
  int extra_arrivals;  // test hook: arrivals the grid-wide wait expects beyond the grid's CTAs
  int* check_word;
};

// 8 consecutive activations as fp32
__device__ __forceinline__ void x8(const void* row, bool bf16, int k, bool coherent, float (&v)[8]) {
  if (bf16) {
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(row) + k);
    const uint4 r = coherent ? __ldcg(p) : __ldg(p);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  } else {
    const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(row) + k);
    const float4 a = coherent ? __ldcg(p) : __ldg(p);
    const float4 b = coherent ? __ldcg(p + 1) : __ldg(p + 1);
    v[0] = a.x, v[1] = a.y, v[2] = a.z, v[3] = a.w;
    v[4] = b.x, v[5] = b.y, v[6] = b.z, v[7] = b.w;
  }
}

// The lane's share of  sum_k q[r][k] * s[r][k / G] * x[k]  for DL_R consecutive rows r of one packed
// matrix over their 128-bit words j0 .. j1-1 (two's-complement fields, low bits first); the caller
// adds the lanes up.  The rows' loads are all started before the first is used, and the
// activations are read once for all of them.  `coherent`: x was written by other CTAs of this
// launch and must not come from the read-only cache.
template <int BITS, int DL_R>
__device__ __forceinline__ void dot_rows(const uint8_t* __restrict__ row0, size_t row_bytes, const char* __restrict__ srow0,
                                         size_t srow_bytes, bool scale_f16, int gshift, const void* xrow, bool x_bf16,
                                         bool coherent, int j0, int j1, int lane, float (&acc)[DL_R]) {
  constexpr int WPV = 128 / BITS;  // weights per 128-bit word
  constexpr int PER32 = 32 / BITS;
  for (int j = j0 + lane; j < j1; j += 32) {
    uint32_t w[DL_R][4];
    float sc[DL_R], part[DL_R];
    const int k0 = j * WPV;
    const int g = gshift < 0 ? 0 : k0 >> gshift;
#pragma unroll
    for (int r = 0; r < DL_R; ++r) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(row0 + r * row_bytes) + j);
      w[r][0] = v.x, w[r][1] = v.y, w[r][2] = v.z, w[r][3] = v.w;
      const char* sp = srow0 + r * srow_bytes;
      sc[r] = scale_f16 ? __half2float(reinterpret_cast<const __half*>(sp)[g]) : reinterpret_cast<const float*>(sp)[g];
      part[r] = 0.0f;
    }
#pragma unroll
    for (int blk = 0; blk < WPV / 8; ++blk) {
      float xv[8];
      x8(xrow, x_bf16, k0 + 8 * blk, coherent, xv);
#pragma unroll
      for (int r = 0; r < DL_R; ++r) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int c = 8 * blk + i;  // code index inside the 128-bit word
          const int q = static_cast<int>(w[r][c / PER32] << (32 - BITS * (c % PER32 + 1))) >> (32 - BITS);
          // the integer as a float without the conversion unit: 1.5 * 2^23 + q has q in its low mantissa bits
          part[r] = fmaf(__int_as_float(0x4B400000 + q) - 12582912.0f, xv[i], part[r]);
        }
      }
    }
#pragma unroll
    for (int r = 0; r < DL_R; ++r) acc[r] = fmaf(sc[r], part[r], acc[r]);
  }
}

template <int DL_R>
__device__ __forceinline__ void dot_bits(int bits, const uint8_t* row0, size_t row_bytes, const char* srow0, size_t srow_bytes,
                                         bool scale_f16, int gshift, const void* xrow, bool x_bf16, bool coherent, int j0,
                                         int j1, int lane, float (&acc)[DL_R]) {
  switch (bits) {
    case 8: dot_rows<8, DL_R>(row0, row_bytes, srow0, srow_bytes, scale_f16, gshift, xrow, x_bf16, coherent, j0, j1, lane, acc); break;
    case 4: dot_rows<4, DL_R>(row0, row_bytes, srow0, srow_bytes, scale_f16, gshift, xrow, x_bf16, coherent, j0, j1, lane, acc); break;
    default: dot_rows<2, DL_R>(row0, row_bytes, srow0, srow_bytes, scale_f16, gshift, xrow, x_bf16, coherent, j0, j1, lane, acc); break;
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Thread 0 of the CTA counts the CTA in and polls until `target` CTAs have arrived (at most
// `limit` polls); the CTA's earlier global writes are visible to whoever sees its arrival.
// Returns to every thread whether the wait ended in time.
__device__ __forceinline__ bool grid_arrive_wait(unsigned* counter, unsigned target, bool arrive, unsigned limit,
                                                 int* check_word, int* s_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    if (arrive) {
      __threadfence();
      atomicAdd(counter, 1u);
    }
    unsigned seen = 0, polls = 0;
    int ok = 1;
    for (;;) {
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
      if (seen >= target) break;
      if (++polls > limit) {
        ok = 0;
        atomicOr(check_word, CHECK_WAIT_TIMEOUT);
        break;
      }
      __nanosleep(40);
    }
    *s_flag = ok;
  }
  __syncthreads();
  return *s_flag != 0;
}

template <int DL_R>
__global__ void __launch_bounds__(DL_THREADS, 3) decode_layer_kernel(const DecodeLayerArgs a) {
  __shared__ int s_ids[DL_MAX_PAIRS];
  __shared__ float s_gates[DL_MAX_PAIRS];
  __shared__ float s_part[DL_WARPS][DL_R_MAX];  // [row block of the CTA][warp of the block][row]
  __shared__ float s_red[DL_THREADS];            // router product: [parts][EP]
  __shared__ float s_z[DL_WARPS][EMOE_MAX_EXPERTS];  // logits of the token a warp picks for
  __shared__ int s_flag;
  const LayerDims& L = a.L;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = a.T * L.top_k;
  const bool bf16 = L.act_bf16 != 0;
  const size_t xsz = bf16 ? 2 : 4;
  const int gshift = L.group > 0 ? 31 - __clz(L.group) : -1;
  // The next kernel of the chain is scheduled once every CTA of this grid has executed this, i.e.
  // once the whole grid is resident: it cannot take the room of a CTA the waits below need.
  pdl_trigger();

  // ---- 1. routing ----
  if (a.Wr) {
    const int RS = a.rsplit, EP = a.EP, d = L.d_model;
    const int n_route = a.T * RS;
    if (static_cast<int>(blockIdx.x) < n_route) {
      // partial logits of one token over one slice of the d_model axis: thread = (expert, interleaved part of the slice)
      const int t = static_cast<int>(blockIdx.x) / RS, r = static_cast<int>(blockIdx.x) - t * RS;
      const int kb = static_cast<int>(static_cast<long long>(d) * r / RS), ke = static_cast<int>(static_cast<long long>(d) * (r + 1) / RS);
      const int e = tid & (EP - 1), part = tid >> a.ep_shift, S = DL_THREADS >> a.ep_shift;
      float acc = 0.0f;
      if (e < L.E) {
        constexpr int U = 8;  // independent loads in flight per thread
        for (int i = kb + part; i < ke; i += U * S) {
          float w[U], xv[U];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const int ii = i + u * S;
            const bool in = ii < ke;
            w[u] = in ? __ldg(a.Wr + static_cast<size_t>(ii) * L.E + e) : 0.0f;
            const size_t xi = static_cast<size_t>(t) * d + (in ? ii : kb);
            xv[u] = bf16 ? __bfloat162float(__ldg(reinterpret_cast<const __nv_bfloat16*>(a.x) + xi))
                         : __ldg(reinterpret_cast<const float*>(a.x) + xi);
          }
#pragma unroll
          for (int u = 0; u < U; ++u) acc = fmaf(xv[u], w[u], acc);
        }
      }
      s_red[part * EP + e] = acc;
      __syncthreads();
      pdl_wait();  // the kernels in front may still read what is written from here on
      if (tid < EP) {
        float z = 0.0f;
        for (int sidx = 0; sidx < S; ++sidx) z += s_red[sidx * EP + tid];
        a.zpart[(static_cast<size_t>(t) * RS + r) * EP + tid] = z;
      }
    } else {
      pdl_wait();
    }
    if (!grid_arrive_wait(a.sync, static_cast<unsigned>(n_route + a.extra_arrivals), static_cast<int>(blockIdx.x) < n_route,
                          a.wait_limit, a.check_word, &s_flag))
      return;
    // every CTA makes the picks of every token from the same numbers in the same order
    for (int t = warp; t < a.T; t += DL_WARPS) {
      float* zrow = s_z[warp];
      for (int e = lane; e < EP; e += 32) {
        float z = 0.0f;
        if (e < L.E) {
          for (int r = 0; r < RS; ++r) z += __ldcg(a.zpart + (static_cast<size_t>(t) * RS + r) * EP + e);
          if (a.bias) z += a.bias[static_cast<size_t>(t) * a.bias_stride + e];
        }
        zrow[e] = z;
      }
      __syncwarp();
      int my_id;
      float my_gate;
      router_pick(zrow, L.E, L.top_k, a.renorm, lane, my_id, my_gate);
      if (lane < L.top_k) {
        s_ids[t * L.top_k + lane] = my_id;
        s_gates[t * L.top_k + lane] = my_gate;
        if (blockIdx.x == 0) {
          a.ids[static_cast<size_t>(t) * L.top_k + lane] = my_id;
          a.gates[static_cast<size_t>(t) * L.top_k + lane] = my_gate;
        }
      }
      __syncwarp();
    }
  } else {
    pdl_wait();
    if (tid < P) {
      int id = __ldcg(a.ids_in + tid);
      if (id < 0 || id >= L.E) {  // only a caller's picks can be out of range
        atomicOr(a.check_word, CHECK_BAD_EXPERT_ID);
        id = -1;
      }
      s_ids[tid] = id;
      s_gates[tid] = __ldcg(a.gates_in + tid);
    }
  }
  __syncthreads();

  // the rows of the second projection this warp will read: ask for them now, so that they are in
  // L2 by the time the first projection is done
  {
    const int N = L.d_model, K = L.d_ff;
    const int m_last = L.act == EMOE_ACT_RELU ? 1 : 2;
    const int NB = N / DL_R;  // blocks of DL_R rows
    const long long units = static_cast<long long>(a.T) * NB;
    const int wpr = a.wpr, blocks_cta = DL_WARPS / a.wpr;
    const long long stride = static_cast<long long>(gridDim.x) * blocks_cta;
    const int rs = warp / wpr, sub = warp % wpr;
    for (long long u = static_cast<long long>(blockIdx.x) * blocks_cta + rs; u < units; u += stride) {
      const int t = static_cast<int>(u / NB);
      const int n = static_cast<int>(u - static_cast<long long>(t) * NB) * DL_R;
      for (int j = 0; j < L.top_k; ++j) {
        const int e = s_ids[t * L.top_k + j];
        if (e < 0) continue;
        const ExpertDev ex = a.experts[e];
        const int nvec = K * ex.bits / 128;
        const size_t b0 = static_cast<size_t>(static_cast<long long>(nvec) * sub / wpr) * 16;
        const size_t b1 = static_cast<size_t>(static_cast<long long>(nvec) * (sub + 1) / wpr) * 16;
        const size_t row_bytes = static_cast<size_t>(K) * ex.bits / 8;
        for (int r = 0; r < DL_R; ++r) {
          const uint8_t* row = ex.packed[m_last] + static_cast<size_t>(n + r) * row_bytes;
          for (size_t b = (b0 & ~static_cast<size_t>(127)) + 128 * lane; b < b1; b += 128 * 32)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(row + b));
        }
      }
    }
  }

  if (blockIdx.x == gridDim.x - 1) {
    // per-call bookkeeping, by the CTA with the least work in the projections: counts, exclusive
    // offsets, pairs in expert order (stable) and the inverse; every entry on its own
    for (int e = tid; e <= L.E; e += DL_THREADS) {
      int below = 0, same = 0;
      for (int p = 0; p < P; ++p) {
        below += s_ids[p] >= 0 && s_ids[p] < e;
        same += s_ids[p] == e;
      }
      a.off[e] = below;
      if (e < L.E) a.counts[e] = same;
    }
    if (tid < P && s_ids[tid] >= 0) {
      int slot = 0;
      for (int q = 0; q < P; ++q) slot += s_ids[q] >= 0 && (s_ids[q] < s_ids[tid] || (s_ids[q] == s_ids[tid] && q < tid));
      a.perm[slot] = tid;
      a.slot_of_pair[tid] = slot;
    }
  }

  // ---- 2. first projection: hidden[p][n] = act(W1[e_p][n] . x_t), DL_R hidden channels per warp ----
  {
    const int N = L.d_ff, K = L.d_model, NB = N / DL_R;
    const int ngroups = gshift < 0 ? 1 : K >> gshift;
    const size_t srow_bytes = static_cast<size_t>(ngroups) * (L.scale_f16 ? 2 : 4);
    const long long units = static_cast<long long>(P) * NB;
    const long long stride = static_cast<long long>(gridDim.x) * DL_WARPS;
    // a warp with more than one unit asks for the rows of the later ones now: their loads then
    // come from L2 instead of starting a trip to HBM only when the unit before is done
    for (long long u = static_cast<long long>(blockIdx.x) * DL_WARPS + warp + stride; u < units; u += stride) {
      const int p = static_cast<int>(u / NB);
      const int n = static_cast<int>(u - static_cast<long long>(p) * NB) * DL_R;
      const int e = s_ids[p];
      if (e < 0) continue;
      const ExpertDev ex = a.experts[e];
      const size_t bytes = static_cast<size_t>(K) * ex.bits / 8 * DL_R;  // the unit's rows follow each other
      const int n_mat = L.act == EMOE_ACT_RELU ? 1 : 2;
      for (int m = 0; m < n_mat; ++m) {
        const uint8_t* rows = ex.packed[m] + static_cast<size_t>(n) * (bytes / DL_R);
        for (size_t b = 128 * static_cast<size_t>(lane); b < bytes; b += 128 * 32)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(rows + b));
      }
    }
    for (long long u = static_cast<long long>(blockIdx.x) * DL_WARPS + warp; u < units; u += stride) {
      const int p = static_cast<int>(u / NB);
      const int n = static_cast<int>(u - static_cast<long long>(p) * NB) * DL_R;
      const int e = s_ids[p];
      float h[DL_R];
#pragma unroll
      for (int r = 0; r < DL_R; ++r) h[r] = 0.0f;
      if (e >= 0) {
        const ExpertDev ex = a.experts[e];
        const int nvec = K * ex.bits / 128;
        const size_t row_bytes = static_cast<size_t>(K) * ex.bits / 8;
        const void* xrow = static_cast<const char*>(a.x) + static_cast<size_t>(p / L.top_k) * K * xsz;
        float v1[DL_R];
#pragma unroll
        for (int r = 0; r < DL_R; ++r) v1[r] = 0.0f;
        dot_bits<DL_R>(ex.bits, ex.packed[0] + n * row_bytes, row_bytes, static_cast<const char*>(ex.scales[0]) + n * srow_bytes, srow_bytes,
                 L.scale_f16, gshift, xrow, bf16, false, 0, nvec, lane, v1);
        if (L.act == EMOE_ACT_RELU) {
#pragma unroll
          for (int r = 0; r < DL_R; ++r) h[r] = fmaxf(warp_sum(v1[r]), 0.0f);
        } else {
          float v3[DL_R];
#pragma unroll
          for (int r = 0; r < DL_R; ++r) v3[r] = 0.0f;
          dot_bits<DL_R>(ex.bits, ex.packed[1] + n * row_bytes, row_bytes, static_cast<const char*>(ex.scales[1]) + n * srow_bytes, srow_bytes,
                   L.scale_f16, gshift, xrow, bf16, false, 0, nvec, lane, v3);
#pragma unroll
          for (int r = 0; r < DL_R; ++r) {
            const float g1 = warp_sum(v1[r]), g3 = warp_sum(v3[r]);
            h[r] = g1 / (1.0f + expf(-g1)) * g3;
          }
        }
      }
      if (lane == 0) {
        const size_t o = static_cast<size_t>(p) * N + n;
#pragma unroll
        for (int r = 0; r < DL_R; ++r) {
          if (bf16) reinterpret_cast<__nv_bfloat16*>(a.hidden)[o + r] = __float2bfloat16_rn(h[r]);
          else reinterpret_cast<float*>(a.hidden)[o + r] = h[r];
        }
      }
    }
  }
  if (!grid_arrive_wait(a.sync + 1, gridDim.x + static_cast<unsigned>(a.extra_arrivals), true, a.wait_limit, a.check_word,
                        &s_flag))
    return;

  // ---- 3. second projection and gate-weighted sum: y[t][n] = sum_j gate_j * (W2[e_j][n] . hidden_j),
  //         DL_R output channels per group of a.wpr warps ----
  {
    const int N = L.d_model, K = L.d_ff, NB = N / DL_R;
    const int ngroups = gshift < 0 ? 1 : K >> gshift;
    const size_t srow_bytes = static_cast<size_t>(ngroups) * (L.scale_f16 ? 2 : 4);
    const int m_last = L.act == EMOE_ACT_RELU ? 1 : 2;
    const long long units = static_cast<long long>(a.T) * NB;
    const int wpr = a.wpr, blocks_cta = DL_WARPS / a.wpr;
    const long long stride = static_cast<long long>(gridDim.x) * blocks_cta;
    const int rs = warp / wpr, sub = warp % wpr;
    for (long long u0 = static_cast<long long>(blockIdx.x) * blocks_cta; u0 < units; u0 += stride) {  // same trip count for the whole CTA
      const long long u = u0 + rs;
      float acc[DL_R];
#pragma unroll
      for (int r = 0; r < DL_R; ++r) acc[r] = 0.0f;
      int t = 0, n = 0;
      if (u < units) {
        t = static_cast<int>(u / NB);
        n = static_cast<int>(u - static_cast<long long>(t) * NB) * DL_R;
        for (int j = 0; j < L.top_k; ++j) {
          const int p = t * L.top_k + j;
          const int e = s_ids[p];
          if (e < 0) continue;
          const ExpertDev ex = a.experts[e];
          const int nvec = K * ex.bits / 128;
          const int j0 = static_cast<int>(static_cast<long long>(nvec) * sub / wpr);
          const int j1 = static_cast<int>(static_cast<long long>(nvec) * (sub + 1) / wpr);
          const size_t row_bytes = static_cast<size_t>(K) * ex.bits / 8;
          const void* hrow = static_cast<const char*>(a.hidden) + static_cast<size_t>(p) * K * xsz;
          float d[DL_R];
#pragma unroll
          for (int r = 0; r < DL_R; ++r) d[r] = 0.0f;
          dot_bits<DL_R>(ex.bits, ex.packed[m_last] + n * row_bytes, row_bytes, static_cast<const char*>(ex.scales[m_last]) + n * srow_bytes,
                   srow_bytes, L.scale_f16, gshift, hrow, bf16, true, j0, j1, lane, d);
#pragma unroll
          for (int r = 0; r < DL_R; ++r) acc[r] = fmaf(s_gates[p], d[r], acc[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < DL_R; ++r) {
        const float v = warp_sum(acc[r]);
        if (lane == 0) s_part[warp][r] = v;
      }
      __syncthreads();
      if (sub == 0 && lane < DL_R && u < units) {
        float v = s_part[warp][lane];  // the block's warps follow each other: a fixed order of additions
        for (int i = 1; i < wpr; ++i) v += s_part[warp + i][lane];
        a.y[static_cast<size_t>(t) * N + n + lane] = v;
      }
      __syncthreads();
    }
  }
  // the last CTA to leave clears the counters for the next launch
  if (tid == 0 && atomicAdd(a.sync + 2, 1u) == gridDim.x - 1u) {
    a.sync[0] = 0;
    a.sync[1] = 0;
    a.sync[2] = 0;
    __threadfence();
  }
}

size_t decode_layer_smem() { return 0; }

}  // namespace

bool decode_layer_supported(const LayerDims& L, int T) {
  const bool group_ok = L.group == 0 || L.group == 64 || L.group == 128;
  return T * L.top_k <= DL_MAX_PAIRS && L.E <= EMOE_MAX_EXPERTS && L.d_model % 64 == 0 && L.d_ff % 64 == 0 && group_ok &&
         static_cast<long long>(L.d_model) * L.d_ff <= DL_MAX_WEIGHTS;
}

int decode_layer_resident_ctas(int device) {
  int per_sm = 0, sms = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_layer_kernel<DL_R_MAX>, DL_THREADS, decode_layer_smem()) != cudaSuccess)
    return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return 0;
  return per_sm * sms;
}

cudaError_t launch_decode_layer(const LayerDims& L, const ExpertDev* experts, const void* x, int T, const float* Wr,
                                const float* bias, int bias_stride, const int32_t* ids_in, const float* gates_in,
                                int32_t* ids, float* gates, int32_t* counts, int32_t* off, int32_t* perm,
                                int32_t* slot_of_pair, void* hidden, float* y, float* zpart, size_t zpart_floats,
                                int resident_ctas, int sms, unsigned* sync, unsigned wait_limit, int extra_arrivals,
                                int* check_word, cudaStream_t st) {
  DecodeLayerArgs a;
  a.L = L;
  a.experts = experts;
  a.x = x;
  a.T = T;
  a.Wr = Wr;
  a.bias = bias;
  a.bias_stride = bias_stride;
  a.EP = 1;
  a.ep_shift = 0;
  while (a.EP < L.E) {
    a.EP <<= 1;
    ++a.ep_shift;
  }
  a.renorm = L.gate_mode == EMOE_GATE_SOFTMAX_RENORM;
  // slices of the router product: as many as the scratch array holds and as leave a slice 64 inputs or more
  a.rsplit = 8;
  while (a.rsplit > 1 && (static_cast<size_t>(T) * a.rsplit * a.EP > zpart_floats || L.d_model / a.rsplit < 64)) a.rsplit >>= 1;
  if (Wr && static_cast<size_t>(T) * a.rsplit * a.EP > zpart_floats) return cudaErrorInvalidValue;
  a.zpart = zpart;
  a.ids_in = ids_in;
  a.gates_in = gates_in;
  a.ids = ids;
  a.gates = gates;
  a.counts = counts;
  a.off = off;
  a.perm = perm;
  a.slot_of_pair = slot_of_pair;
  a.hidden = hidden;
  a.y = y;
  a.sync = sync;
  a.wait_limit = wait_limit;
  a.extra_arrivals = extra_arrivals;
  a.check_word = check_word;
  // Every CTA must be resident at once.  As few CTAs as give every block of four rows of the
  // first projection a warp of its own (one, two or three per SM): each further CTA makes the two
  // grid-wide waits longer (as measured, one token: 0.139 ms per 12-layer step with one CTA per
  // SM, 0.154 with two, 0.173 with three; four tokens: 0.307 / 0.259 / 0.224).
  const long long blocks = static_cast<long long>(T) * L.top_k * L.d_ff / DL_R_MAX;
  const int max_per_sm = resident_ctas / sms < 3 ? resident_ctas / sms : 3;
  int per_sm = 1;
  while (per_sm < max_per_sm && static_cast<long long>(per_sm) * sms * DL_WARPS < blocks) ++per_sm;
  const int grid = per_sm * sms;
  // second projection: four warps share a block of four output rows while every block then finds its warps in
  // one pass; else two, else one (eight tokens: 0.361 -> 0.304 ms per 12-layer step with two)
  a.wpr = DL_WPR_MAX;
  while (a.wpr > 1 && static_cast<long long>(T) * (L.d_model / DL_R_MAX) > static_cast<long long>(grid) * (DL_WARPS / a.wpr)) a.wpr >>= 1;
  while (a.rsplit > 1 && T * a.rsplit > grid) a.rsplit >>= 1;  // a small device: fewer slices than CTAs
  if (per_sm < 1 || grid < T) return cudaErrorInvalidConfiguration;
  return launch_chain(decode_layer_kernel<DL_R_MAX>, dim3(grid), dim3(DL_THREADS), decode_layer_smem(), st, a);
}

}  // namespace emoe
