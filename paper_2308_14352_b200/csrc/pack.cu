// Expert-wise quantisation kernel (paper Section 3.2, "Choosing the algorithm"):
// channel-wise linear quantisation of an fp32 matrix to INT2/INT4/INT8 codes plus a scale
// channel.  One warp owns one (output channel, group) unit: it finds the unit's max-abs,
// derives the scale, then quantises and packs, each lane emitting the codes of 4 consecutive weights.
// HBM-bound: 4 bytes read and bits/8 bytes written per weight (the second read of a unit
// comes from L1/L2).
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

template <int BITS>
__global__ void __launch_bounds__(256) pack_kernel(const float* __restrict__ W, int N, int K, int G, int ngroups,
                                                   int scale_f16, uint8_t* __restrict__ packed,
                                                   void* __restrict__ scales) {
  typedef typename PackWord<BITS>::type word_t;
  constexpr int MASK = (1 << BITS) - 1;
  const float qmax = static_cast<float>((1 << (BITS - 1)) - 1);
  const int lane = threadIdx.x & 31;
  const long long n_units = static_cast<long long>(N) * ngroups;
  const long long warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
  for (long long unit = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; unit < n_units; unit += warps) {
  const int n = static_cast<int>(unit / ngroups);
  const int g = static_cast<int>(unit % ngroups);
  const float* w = W + static_cast<size_t>(n) * K + static_cast<size_t>(g) * G;

  // every lane owns 4 consecutive weights per 128-weight step; with 128-weight groups the
  // weights stay in registers between the two passes
  float4 first = make_float4(0.f, 0.f, 0.f, 0.f);
  float amax = 0.0f;
  for (int i = lane * 4; i < G; i += 128) {
    const float4 v = *reinterpret_cast<const float4*>(w + i);
    if (i < 128) first = v;
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));

  // scale = max-abs / representable range, IEEE division; stored in the scale channel's type
  float s = __fdiv_rn(amax, qmax);
  if (scale_f16) {
    const __half h = __float2half_rn(s);
    s = __half2float(h);
    if (lane == 0) reinterpret_cast<__half*>(scales)[unit] = h;
  } else if (lane == 0) {
    reinterpret_cast<float*>(scales)[unit] = s;
  }

  word_t* out = reinterpret_cast<word_t*>(packed + static_cast<size_t>(n) * (static_cast<size_t>(K) * BITS / 8) +
                                          static_cast<size_t>(g) * G * BITS / 8);
  for (int i = lane * 4; i < G; i += 128) {
    const float4 v = i < 128 ? first : *reinterpret_cast<const float4*>(w + i);
    const float e[4] = {v.x, v.y, v.z, v.w};
    uint32_t word = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      int q = 0;
      if (s != 0.0f) {
        float r = rintf(__fdiv_rn(e[c], s));  // round half to even on the quotient by the stored scale
        r = fminf(fmaxf(r, -qmax), qmax);
        q = static_cast<int>(r);
      }
      word |= static_cast<uint32_t>(q & MASK) << (BITS * c);
    }
    out[i >> 2] = static_cast<word_t>(word);
  }
  }
}

// ---- a stored matrix to another bitwidth (Section 3.2: the bitwidth selection lowers the width
// of chosen experts; the fp32 original is not needed) ------------------------------------------
// Same unit ownership and the same arithmetic as pack_kernel; the only difference is where a
// weight comes from: it is decompressed in registers (w~ = q * s, rounded once to fp32; exact
// with fp16 scales), never written to memory.  HBM-bound on packed bytes: BIN/8 bytes read and
// BOUT/8 bytes written per weight.
template <int BIN>
__device__ __forceinline__ float4 decompress4(const uint8_t* __restrict__ row, int k, float s) {
  // the codes of the 4 consecutive weights k .. k+3 (k a multiple of 4), low fields first
  uint32_t w;
  if (BIN == 8) w = *reinterpret_cast<const uint32_t*>(row + k);
  else if (BIN == 4) w = *reinterpret_cast<const uint16_t*>(row + (k >> 1));
  else w = row[k >> 2];
  float v[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int q = static_cast<int>(w << (32 - BIN * (c + 1))) >> (32 - BIN);  // sign-extended field
    v[c] = __fmul_rn(static_cast<float>(q), s);
  }
  return make_float4(v[0], v[1], v[2], v[3]);
}

template <int BIN, int BOUT>
__global__ void __launch_bounds__(256) requant_kernel(const uint8_t* __restrict__ in_packed,
                                                      const void* __restrict__ in_scales, int N, int K, int G,
                                                      int ngroups, int scale_f16, uint8_t* __restrict__ packed,
                                                      void* __restrict__ scales) {
  typedef typename PackWord<BOUT>::type word_t;
  constexpr int MASK = (1 << BOUT) - 1;
  const float qmax = static_cast<float>((1 << (BOUT - 1)) - 1);
  const int lane = threadIdx.x & 31;
  const long long n_units = static_cast<long long>(N) * ngroups;
  const long long warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
  for (long long unit = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; unit < n_units;
       unit += warps) {
    const int n = static_cast<int>(unit / ngroups);
    const int g = static_cast<int>(unit % ngroups);
    const uint8_t* row = in_packed + static_cast<size_t>(n) * (static_cast<size_t>(K) * BIN / 8);
    const float s_in = scale_f16 ? __half2float(reinterpret_cast<const __half*>(in_scales)[unit])
                                 : reinterpret_cast<const float*>(in_scales)[unit];
    const int k_first = g * G;

    float4 first = make_float4(0.f, 0.f, 0.f, 0.f);
    float amax = 0.0f;
    for (int i = lane * 4; i < G; i += 128) {
      const float4 v = decompress4<BIN>(row, k_first + i, s_in);
      if (i < 128) first = v;
      amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));

    float s = __fdiv_rn(amax, qmax);
    if (scale_f16) {
      const __half h = __float2half_rn(s);
      s = __half2float(h);
      if (lane == 0) reinterpret_cast<__half*>(scales)[unit] = h;
    } else if (lane == 0) {
      reinterpret_cast<float*>(scales)[unit] = s;
    }

    word_t* out = reinterpret_cast<word_t*>(packed + static_cast<size_t>(n) * (static_cast<size_t>(K) * BOUT / 8) +
                                            static_cast<size_t>(g) * G * BOUT / 8);
    for (int i = lane * 4; i < G; i += 128) {
      const float4 v = i < 128 ? first : decompress4<BIN>(row, k_first + i, s_in);
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
        word |= static_cast<uint32_t>(q & MASK) << (BOUT * c);
      }
      out[i >> 2] = static_cast<word_t>(word);
    }
  }
}

template <int BIN>
cudaError_t launch_requant_in(const uint8_t* in_packed, const void* in_scales, int N, int K, int G, int ngroups,
                              int bits_out, int scale_f16, uint8_t* packed, void* scales, dim3 grid, cudaStream_t st) {
  switch (bits_out) {
    case 2: requant_kernel<BIN, 2><<<grid, 256, 0, st>>>(in_packed, in_scales, N, K, G, ngroups, scale_f16, packed, scales); break;
    case 4: requant_kernel<BIN, 4><<<grid, 256, 0, st>>>(in_packed, in_scales, N, K, G, ngroups, scale_f16, packed, scales); break;
    case 8: requant_kernel<BIN, 8><<<grid, 256, 0, st>>>(in_packed, in_scales, N, K, G, ngroups, scale_f16, packed, scales); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_requant(const uint8_t* in_packed, const void* in_scales, int N, int K, int bits_in, int bits_out,
                           int group, int scale_f16, uint8_t* packed, void* scales, cudaStream_t st) {
  const int G = group > 0 ? group : K;
  const int ngroups = K / G;
  const long long units = static_cast<long long>(N) * ngroups;
  long long blocks = (units * 32 + 255) / 256;
  const long long cap = 148LL * 8 * 4;
  if (blocks > cap) blocks = cap;
  const dim3 grid(static_cast<unsigned>(blocks));
  switch (bits_in) {
    case 2: return launch_requant_in<2>(in_packed, in_scales, N, K, G, ngroups, bits_out, scale_f16, packed, scales, grid, st);
    case 4: return launch_requant_in<4>(in_packed, in_scales, N, K, G, ngroups, bits_out, scale_f16, packed, scales, grid, st);
    case 8: return launch_requant_in<8>(in_packed, in_scales, N, K, G, ngroups, bits_out, scale_f16, packed, scales, grid, st);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_pack(const float* W, int N, int K, int bits, int group, int scale_f16, uint8_t* packed,
                        void* scales, cudaStream_t st) {
  const int G = group > 0 ? group : K;
  const int ngroups = K / G;
  const long long units = static_cast<long long>(N) * ngroups;
  const int threads = 256;
  long long blocks = (units * 32 + threads - 1) / threads;
  const long long cap = 148LL * 8 * 4;  // a few waves of resident blocks; each warp then loops over its units
  if (blocks > cap) blocks = cap;
  const dim3 grid(static_cast<unsigned>(blocks));
  switch (bits) {
    case 2: pack_kernel<2><<<grid, threads, 0, st>>>(W, N, K, G, ngroups, scale_f16, packed, scales); break;
    case 4: pack_kernel<4><<<grid, threads, 0, st>>>(W, N, K, G, ngroups, scale_f16, packed, scales); break;
    case 8: pack_kernel<8><<<grid, threads, 0, st>>>(W, N, K, G, ngroups, scale_f16, packed, scales); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace emoe
