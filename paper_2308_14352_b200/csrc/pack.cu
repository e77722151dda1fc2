// Expert-wise quantisation kernels (paper Section 3.2, "Choosing the algorithm"):
// channel-wise linear quantisation to INT2/INT4/INT8 codes plus a scale channel, from an fp32
// matrix (emoe_pack_expert) or from a matrix already stored at another width
// (emoe_requantize_expert: the bitwidth selection of Section 3.2 lowers the width of chosen
// experts; the weight is decompressed in registers, w~ = q * s rounded once to fp32, and the fp32
// original is not needed).  One warp owns one (output channel, group) unit at a time: it finds
// the unit's max-abs, derives the scale, then quantises and packs, each lane emitting the codes
// of 4 consecutive weights.  Groups of 128 weights, the usual case, are taken UNITS at a time so
// that a warp has several independent loads in flight.  HBM-bound by definition: 4 (or
// b_in / 8) bytes read and b_out / 8 bytes written per weight.
#include "common.cuh"

namespace emoe {
namespace {

template <int BITS>
struct PackWord;  // the codes of 4 consecutive weights
template <>
struct PackWord<8> { typedef uint32_t type; };
template <>
struct PackWord<4> { typedef uint16_t type; };
template <>
struct PackWord<2> { typedef uint8_t type; };

// Where the weights come from.  load4(n, k): weights k .. k+3 of row n (k a multiple of 4);
// `unit` is the row's group index n * ngroups + g.
struct SourceF32 {
  const float* W;
  int K;
  __device__ __forceinline__ float4 load4(int n, int k, long long) const {
    return *reinterpret_cast<const float4*>(W + static_cast<size_t>(n) * K + k);
  }
};
template <int BIN>
struct SourcePacked {
  const uint8_t* packed;
  const void* scales;
  int K, scale_f16;
  __device__ __forceinline__ float4 load4(int n, int k, long long unit) const {
    const uint8_t* row = packed + static_cast<size_t>(n) * (static_cast<size_t>(K) * BIN / 8);
    uint32_t w;  // the codes of the 4 weights, low fields first
    if (BIN == 8) w = *reinterpret_cast<const uint32_t*>(row + k);
    else if (BIN == 4) w = *reinterpret_cast<const uint16_t*>(row + (k >> 1));
    else w = row[k >> 2];
    const float s = scale_f16 ? __half2float(reinterpret_cast<const __half*>(scales)[unit])
                              : reinterpret_cast<const float*>(scales)[unit];
    float v[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int q = static_cast<int>(w << (32 - BIN * (c + 1))) >> (32 - BIN);  // sign-extended field
      v[c] = __fmul_rn(static_cast<float>(q), s);
    }
    return make_float4(v[0], v[1], v[2], v[3]);
  }
};

// scale = max-abs / representable range, IEEE division; stored in the scale channel's type
__device__ __forceinline__ float store_scale(float amax, float qmax, int scale_f16, void* scales, long long unit, int lane) {
  float s = __fdiv_rn(amax, qmax);
  if (scale_f16) {
    const __half h = __float2half_rn(s);
    s = __half2float(h);
    if (lane == 0) reinterpret_cast<__half*>(scales)[unit] = h;
  } else if (lane == 0) {
    reinterpret_cast<float*>(scales)[unit] = s;
  }
  return s;
}

// codes of 4 weights: round half to even on the quotient by the stored scale, clamp, pack
template <int BITS>
__device__ __forceinline__ uint32_t quantise4(const float4& v, float s, float qmax) {
  constexpr int MASK = (1 << BITS) - 1;
  const float e[4] = {v.x, v.y, v.z, v.w};
  uint32_t word = 0;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    int q = 0;
    if (s != 0.0f) {
      float r = rintf(__fdiv_rn(e[c], s));
      r = fminf(fmaxf(r, -qmax), qmax);
      q = static_cast<int>(r);
    }
    word |= static_cast<uint32_t>(q & MASK) << (BITS * c);
  }
  return word;
}

__device__ __forceinline__ float amax4(const float4& v) {
  return fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
}

constexpr int UNITS = 4;  // 128-weight units a warp works on at once

template <int BITS, typename Source>
__global__ void __launch_bounds__(256) quantise_kernel(const Source src, int N, int K, int G, int ngroups, int scale_f16,
                                                       uint8_t* __restrict__ packed, void* __restrict__ scales) {
  typedef typename PackWord<BITS>::type word_t;
  const float qmax = static_cast<float>((1 << (BITS - 1)) - 1);
  const int lane = threadIdx.x & 31;
  const long long n_units = static_cast<long long>(N) * ngroups;
  const long long warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
  const long long warp = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const size_t row_bytes = static_cast<size_t>(K) * BITS / 8;

  if (G == 128) {
    // one step per unit: the unit's weights stay in registers, UNITS units in flight
    for (long long u0 = warp * UNITS; u0 < n_units; u0 += warps * UNITS) {
      float4 v[UNITS];
      float amax[UNITS];
#pragma unroll
      for (int u = 0; u < UNITS; ++u) {
        const long long unit = u0 + u;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (unit < n_units)
          v[u] = src.load4(static_cast<int>(unit / ngroups), static_cast<int>(unit % ngroups) * 128 + lane * 4, unit);
        amax[u] = amax4(v[u]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int u = 0; u < UNITS; ++u) amax[u] = fmaxf(amax[u], __shfl_xor_sync(0xffffffffu, amax[u], o));
#pragma unroll
      for (int u = 0; u < UNITS; ++u) {
        const long long unit = u0 + u;
        if (unit >= n_units) break;
        const float s = store_scale(amax[u], qmax, scale_f16, scales, unit, lane);
        word_t* out = reinterpret_cast<word_t*>(packed + static_cast<size_t>(unit / ngroups) * row_bytes +
                                                static_cast<size_t>(unit % ngroups) * 128 * BITS / 8);
        out[lane] = static_cast<word_t>(quantise4<BITS>(v[u], s, qmax));
      }
    }
    return;
  }

  for (long long unit = warp; unit < n_units; unit += warps) {
    const int n = static_cast<int>(unit / ngroups);
    const int g = static_cast<int>(unit % ngroups);
    const int k_first = g * G;
    // every lane owns 4 consecutive weights per 128-weight step; the first step stays in registers
    float4 first = make_float4(0.f, 0.f, 0.f, 0.f);
    float amax = 0.0f;
    for (int i = lane * 4; i < G; i += 128) {
      const float4 v = src.load4(n, k_first + i, unit);
      if (i < 128) first = v;
      amax = fmaxf(amax, amax4(v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float s = store_scale(amax, qmax, scale_f16, scales, unit, lane);
    word_t* out = reinterpret_cast<word_t*>(packed + static_cast<size_t>(n) * row_bytes + static_cast<size_t>(g) * G * BITS / 8);
    for (int i = lane * 4; i < G; i += 128) {
      const float4 v = i < 128 ? first : src.load4(n, k_first + i, unit);  // later steps come from L1/L2
      out[i >> 2] = static_cast<word_t>(quantise4<BITS>(v, s, qmax));
    }
  }
}

template <typename Source>
cudaError_t launch_quantise(const Source& src, int N, int K, int bits, int group, int scale_f16, uint8_t* packed,
                            void* scales, cudaStream_t st) {
  const int G = group > 0 ? group : K;
  const int ngroups = K / G;
  const long long units = static_cast<long long>(N) * ngroups;
  const long long warps_needed = G == 128 ? (units + UNITS - 1) / UNITS : units;
  const int threads = 256;
  long long blocks = (warps_needed * 32 + threads - 1) / threads;
  const long long cap = 148LL * 8 * 4;  // a few waves of resident blocks; each warp then loops over its units
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const dim3 grid(static_cast<unsigned>(blocks));
  switch (bits) {
    case 2: quantise_kernel<2, Source><<<grid, threads, 0, st>>>(src, N, K, G, ngroups, scale_f16, packed, scales); break;
    case 4: quantise_kernel<4, Source><<<grid, threads, 0, st>>>(src, N, K, G, ngroups, scale_f16, packed, scales); break;
    case 8: quantise_kernel<8, Source><<<grid, threads, 0, st>>>(src, N, K, G, ngroups, scale_f16, packed, scales); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_pack(const float* W, int N, int K, int bits, int group, int scale_f16, uint8_t* packed,
                        void* scales, cudaStream_t st) {
  return launch_quantise(SourceF32{W, K}, N, K, bits, group, scale_f16, packed, scales, st);
}

cudaError_t launch_requant(const uint8_t* in_packed, const void* in_scales, int N, int K, int bits_in, int bits_out,
                           int group, int scale_f16, uint8_t* packed, void* scales, cudaStream_t st) {
  switch (bits_in) {
    case 2: return launch_quantise(SourcePacked<2>{in_packed, in_scales, K, scale_f16}, N, K, bits_out, group, scale_f16, packed, scales, st);
    case 4: return launch_quantise(SourcePacked<4>{in_packed, in_scales, K, scale_f16}, N, K, bits_out, group, scale_f16, packed, scales, st);
    case 8: return launch_quantise(SourcePacked<8>{in_packed, in_scales, K, scale_f16}, N, K, bits_out, group, scale_f16, packed, scales, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace emoe
