// Grouped GEMV on packed expert weights, CUDA-core path (paper Sections 1/2.1: each
// activated expert is an independent FFN; Section 3.2: weights are stored as b-bit codes
// with a scale channel and decompressed as q * s — here in registers).
//
// One warp owns one output channel of one expert: its 32 lanes stream the packed row with
// 128-bit loads (16 / 32 / 64 weights per load at 8 / 4 / 2 bits), decode the codes with a
// bitwidth-specialised unpack, accumulate sum(q * x) in fp32, apply the group scale to each
// load's partial sum, and finish with a shuffle reduction.  Up to GEMV_MTOK tokens of the
// expert share one pass over the row.  This is the path for fp32 activations (fp32
// accumulation throughout) and the fallback for shapes the tensor-core path does not take.
#include "common.cuh"

namespace emoe {
namespace {

constexpr int GEMV_WARPS = 8;
constexpr int GEMV_MTOK = 4;

// 8 consecutive activations as fp32
__device__ __forceinline__ void load_x8(const void* base, bool bf16, size_t idx, float (&v)[8]) {
  if (bf16) {
    const uint4 r = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(base) + idx);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  } else {
    const float4 a = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + idx);
    const float4 b = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + idx + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}

// a small integer as fp32 without the conversion unit: 1.5 * 2^23 + i has i in its low mantissa bits
__device__ __forceinline__ float small_int_to_float(int i) { return __int_as_float(0x4B400000 + i) - 12582912.0f; }

// codes 8*blk .. 8*blk+7 of a 128-bit load, as fp32 (two's-complement fields, low bits first)
template <int BITS>
__device__ __forceinline__ void unpack8(const uint32_t (&w)[4], int blk, float (&q)[8]);

template <>
__device__ __forceinline__ void unpack8<8>(const uint32_t (&w)[4], int blk, float (&q)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t word = w[2 * blk + (i >> 2)];
    q[i] = small_int_to_float(static_cast<int>(word << (24 - 8 * (i & 3))) >> 24);
  }
}
template <>
__device__ __forceinline__ void unpack8<4>(const uint32_t (&w)[4], int blk, float (&q)[8]) {
  const uint32_t word = w[blk];
#pragma unroll
  for (int i = 0; i < 8; ++i) q[i] = small_int_to_float(static_cast<int>(word << (28 - 4 * i)) >> 28);
}
template <>
__device__ __forceinline__ void unpack8<2>(const uint32_t (&w)[4], int blk, float (&q)[8]) {
  const uint32_t word = w[blk >> 1] >> (16 * (blk & 1));
#pragma unroll
  for (int i = 0; i < 8; ++i) q[i] = small_int_to_float(static_cast<int>(word << (30 - 2 * i)) >> 30);
}

__device__ __forceinline__ float load_scale(const void* scales, bool f16, size_t idx) {
  return f16 ? __half2float(reinterpret_cast<const __half*>(scales)[idx]) : reinterpret_cast<const float*>(scales)[idx];
}

// acc[m] += sum_k q[n][k] * s[n][k/G] * xrow_m[k] for the lane's share of the row
template <int BITS>
__device__ __forceinline__ void row_dot(const uint8_t* __restrict__ packed, const void* __restrict__ scales,
                                        bool scale_f16, int n, int K, int G, const void* (&xrow)[GEMV_MTOK],
                                        int ntok, bool x_bf16, int lane, float (&acc)[GEMV_MTOK]) {
  constexpr int WPV = 128 / BITS;  // weights per 128-bit load
  const int nvec = K / WPV;
  const int ngroups = K / G;
  const int gshift = (G & (G - 1)) == 0 ? 31 - __clz(G) : -1;  // log2(G) when G is a power of two
  const uint4* row = reinterpret_cast<const uint4*>(packed + static_cast<size_t>(n) * (static_cast<size_t>(K) * BITS / 8));
  for (int j = lane; j < nvec; j += 32) {
    const uint4 r = __ldg(row + j);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    const int k0 = j * WPV;
    const int g = ngroups == 1 ? 0 : (gshift >= 0 ? k0 >> gshift : k0 / G);
    const float s = load_scale(scales, scale_f16, static_cast<size_t>(n) * ngroups + g);
    float part[GEMV_MTOK];
#pragma unroll
    for (int m = 0; m < GEMV_MTOK; ++m) part[m] = 0.0f;
#pragma unroll
    for (int blk = 0; blk < WPV / 8; ++blk) {
      float q[8];
      unpack8<BITS>(w, blk, q);
#pragma unroll
      for (int m = 0; m < GEMV_MTOK; ++m) {
        if (m < ntok) {
          float xv[8];
          load_x8(xrow[m], x_bf16, static_cast<size_t>(k0 + 8 * blk), xv);
#pragma unroll
          for (int i = 0; i < 8; ++i) part[m] = fmaf(q[i], xv[i], part[m]);
        }
      }
    }
#pragma unroll
    for (int m = 0; m < GEMV_MTOK; ++m) acc[m] = fmaf(s, part[m], acc[m]);
  }
}

template <int BITS>
__device__ __forceinline__ void expert_rows(int phase, const LayerDims& L, const ExpertDev& ex, const void* x,
                                            const int32_t* perm, int begin, int cnt, void* hidden, float* o) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const int K = phase == 0 ? L.d_model : L.d_ff;
  const int G = L.group > 0 ? L.group : K;
  const int n = blockIdx.x * GEMV_WARPS + warp;
  if (n >= N) return;
  const bool bf16 = L.act_bf16 != 0;
  const size_t xsz = bf16 ? 2 : 4;
  const int m_last = L.act == EMOE_ACT_RELU ? 1 : 2;
  for (int c0 = 0; c0 < cnt; c0 += GEMV_MTOK) {
    const int ntok = min(GEMV_MTOK, cnt - c0);
    const void* xrow[GEMV_MTOK];
#pragma unroll
    for (int m = 0; m < GEMV_MTOK; ++m) {
      const int slot = begin + c0 + min(m, ntok - 1);
      const size_t r = phase == 0 ? static_cast<size_t>(L.top_k == 1 ? perm[slot] : perm[slot] / L.top_k) : static_cast<size_t>(slot);
      const char* base = reinterpret_cast<const char*>(phase == 0 ? x : hidden);
      xrow[m] = base + r * static_cast<size_t>(K) * xsz;
    }
    float a[GEMV_MTOK], b[GEMV_MTOK];
#pragma unroll
    for (int m = 0; m < GEMV_MTOK; ++m) a[m] = b[m] = 0.0f;
    if (phase == 0) {
      row_dot<BITS>(ex.packed[0], ex.scales[0], L.scale_f16, n, K, G, xrow, ntok, bf16, lane, a);
      if (L.act == EMOE_ACT_SWIGLU)
        row_dot<BITS>(ex.packed[1], ex.scales[1], L.scale_f16, n, K, G, xrow, ntok, bf16, lane, b);
    } else {
      row_dot<BITS>(ex.packed[m_last], ex.scales[m_last], L.scale_f16, n, K, G, xrow, ntok, bf16, lane, a);
    }
#pragma unroll
    for (int m = 0; m < GEMV_MTOK; ++m) {
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        a[m] += __shfl_xor_sync(0xffffffffu, a[m], s);
        b[m] += __shfl_xor_sync(0xffffffffu, b[m], s);
      }
    }
    if (lane == 0) {
      for (int m = 0; m < ntok; ++m) {
        const size_t slot = static_cast<size_t>(begin + c0 + m);
        if (phase == 0) {
          float h;
          if (L.act == EMOE_ACT_RELU) h = fmaxf(a[m], 0.0f);
          else h = a[m] / (1.0f + expf(-a[m])) * b[m];
          if (bf16) reinterpret_cast<__nv_bfloat16*>(hidden)[slot * N + n] = __float2bfloat16_rn(h);
          else reinterpret_cast<float*>(hidden)[slot * N + n] = h;
        } else {
          o[slot * N + n] = a[m];
        }
      }
    }
  }
}

__global__ void __launch_bounds__(GEMV_WARPS * 32)
    ffn_gemv_kernel(int phase, LayerDims L, const ExpertDev* __restrict__ experts, const void* __restrict__ x,
                    const int32_t* __restrict__ perm, const int32_t* __restrict__ off, void* hidden,
                    float* __restrict__ o) {
  pdl_wait();
  pdl_trigger();
  const int e = blockIdx.y;
  const int begin = off[e];
  const int cnt = off[e + 1] - begin;
  if (cnt <= 0) return;  // only activated experts are touched
  const ExpertDev ex = experts[e];
  switch (ex.bits) {
    case 2: expert_rows<2>(phase, L, ex, x, perm, begin, cnt, hidden, o); break;
    case 4: expert_rows<4>(phase, L, ex, x, perm, begin, cnt, hidden, o); break;
    case 8: expert_rows<8>(phase, L, ex, x, perm, begin, cnt, hidden, o); break;
    default: break;
  }
}

}  // namespace

cudaError_t launch_ffn_gemv(int phase, const LayerDims& L, const ExpertDev* experts, const void* x,
                            const int32_t* perm, const int32_t* off, void* hidden, float* o, int n_pairs,
                            cudaStream_t st) {
  (void)n_pairs;
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const dim3 grid((N + GEMV_WARPS - 1) / GEMV_WARPS, L.E);
  return launch_chain(ffn_gemv_kernel, grid, dim3(GEMV_WARPS * 32), 0, st, phase, L, experts, x, perm, off, hidden, o);
}

}  // namespace emoe
