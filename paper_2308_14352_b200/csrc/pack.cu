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

}  // namespace

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
