// Expert-wise quantisation kernels (paper Section 3.2, "Choosing the algorithm"):
// channel-wise linear quantisation to INT2/INT4/INT8 codes plus a scale channel, from an fp32
// matrix (emoe_pack_expert) or from a matrix already stored at another width
// (emoe_requantize_expert: the bitwidth selection of Section 3.2 lowers the width of chosen
// experts; the weight is decompressed in registers, w~ = q * s rounded once to fp32, and the fp32
// original is not needed).  One warp owns one (output channel, group) unit at a time: it finds
// the unit's max-abs, derives the scale, then quantises and packs, each lane emitting the codes
// of 4 consecutive weights.  Groups of 128 weights, the usual case, take another route: the
// matrix is dense, so its units follow each other in memory; a warp takes four consecutive units
// at a time, eight lanes per unit and sixteen consecutive weights per lane (64 bytes read, 4 / 8 /
// 16 bytes written by one store), two such steps in flight.  HBM-bound by definition: 4 (or
// b_in / 8) bytes read and b_out / 8 bytes written per weight.
//
// Two readings of "the range expressible by the bitwidth" (Section 3.2): symmetric codes
// -qmax .. qmax with qmax = 2^(b-1) - 1 and scale = max-abs / qmax (the default), or every code of
// the field, -2^(b-1) .. 2^(b-1) - 1, with scale = max-abs / 2^(b-1) ("full range": four levels at
// 2 bits instead of three).
//
// The quotient w / s is an IEEE division in the definition.  The kernels multiply by 1 / s
// instead and keep the result when it cannot differ from the definition's: the product lies
// within 1.8e-7 relative of the rounded quotient, so unless it comes within 1e-4 of a half-integer
// (or leaves the range where that bound holds) both round to the same integer; otherwise the
// division is carried out.  Bit-exact with the definition either way.
#include "common.cuh"

namespace emoe {
namespace {

constexpr float ROUND_MAGIC = 12582912.0f;  // 1.5 * 2^23, bit pattern 0x4B400000

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
  static constexpr int IN_BITS = 32;
  const float* W;
  int K;
  __device__ __forceinline__ float4 load4(int n, int k, long long) const {
    return *reinterpret_cast<const float4*>(W + static_cast<size_t>(n) * K + k);
  }
  // 16 consecutive weights from linear index w0 (a multiple of 16) of the dense matrix: first the
  // loads (several steps are requested before the first is used), then the values
  static constexpr int STEPS = 2;  // four-unit steps a warp has in flight
  struct Raw {
    float4 f[4];
  };
  __device__ __forceinline__ void load_raw(long long w0, long long, Raw& r, float&) const {
    const float4* p = reinterpret_cast<const float4*>(W + w0);
#pragma unroll
    for (int i = 0; i < 4; ++i) r.f[i] = p[i];
  }
  __device__ __forceinline__ void zero_raw(Raw& r, float&) const {
#pragma unroll
    for (int i = 0; i < 4; ++i) r.f[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  __device__ __forceinline__ void decode(const Raw& r, float, float (&v)[16]) const {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[4 * i] = r.f[i].x;
      v[4 * i + 1] = r.f[i].y;
      v[4 * i + 2] = r.f[i].z;
      v[4 * i + 3] = r.f[i].w;
    }
  }
};
template <int BIN>
struct SourcePacked {
  static constexpr int IN_BITS = BIN;
  const uint8_t* packed;
  const void* scales;
  int K, scale_f16;
  __device__ __forceinline__ float scale_of(long long unit) const {
    return scale_f16 ? __half2float(reinterpret_cast<const __half*>(scales)[unit]) : reinterpret_cast<const float*>(scales)[unit];
  }
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
  static constexpr int STEPS = 2;  // as measured: more steps in flight buy nothing here (the kernel is bound by its instruction count)
  struct Raw {
    uint32_t w[BIN / 2];  // the 16 codes, low fields first
  };
  __device__ __forceinline__ void load_raw(long long w0, long long unit, Raw& r, float& s) const {
    const uint8_t* p = packed + w0 * BIN / 8;
    if (BIN == 8) {
      const uint4 q = *reinterpret_cast<const uint4*>(p);
      r.w[0] = q.x, r.w[1] = q.y, r.w[2] = q.z, r.w[3] = q.w;
    } else if (BIN == 4) {
      const uint2 q = *reinterpret_cast<const uint2*>(p);
      r.w[0] = q.x, r.w[1] = q.y;
    } else {
      r.w[0] = *reinterpret_cast<const uint32_t*>(p);
    }
    s = scale_of(unit);
  }
  __device__ __forceinline__ void zero_raw(Raw& r, float& s) const {
#pragma unroll
    for (int i = 0; i < BIN / 2; ++i) r.w[i] = 0u;
    s = 0.0f;
  }
  __device__ __forceinline__ void decode(const Raw& r, float s, float (&v)[16]) const {
    constexpr int PER_WORD = 32 / BIN;
    if constexpr (BIN == 8) {
      // a byte with its sign bit flipped is q + 128; dropped into the low mantissa byte of
      // 1.5 * 2^23 it is the float 12582912 + 128 + q, exactly
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint32_t word = r.w[c >> 2] ^ 0x80808080u;
        const uint32_t f = __byte_perm(word, 0x4B400000u, 0x7640u | (c & 3));
        v[c] = __fmul_rn(__uint_as_float(f) - (ROUND_MAGIC + 128.0f), s);
      }
    } else {
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint32_t word = r.w[c / PER_WORD];
        const int q = static_cast<int>(word << (32 - BIN * (c % PER_WORD + 1))) >> (32 - BIN);
        v[c] = __fmul_rn(__int_as_float(0x4B400000 + q) - ROUND_MAGIC, s);  // the integer as a float, exactly
      }
    }
  }
};

// scale = max-abs / representable range, IEEE division; stored in the scale channel's type
__device__ __forceinline__ float store_scale(float amax, float range, int scale_f16, void* scales, long long unit, bool writer) {
  float s = __fdiv_rn(amax, range);
  if (scale_f16) {
    const __half h = __float2half_rn(s);
    s = __half2float(h);
    if (writer) reinterpret_cast<__half*>(scales)[unit] = h;
  } else if (writer) {
    reinterpret_cast<float*>(scales)[unit] = s;
  }
  return s;
}

// What the codes of one unit are made with: the stored scale, its reciprocal for the fast
// quotient (NaN where the error bound of the product does not hold: the division then decides
// every code), and the clamp.
struct QuantParams {
  float s, r, qlo, qhi;
};
__device__ __forceinline__ QuantParams quant_params(float s, float amax, float qlo, float qhi) {
  QuantParams p;
  p.s = s;
  // scale 0: reciprocal 0, every product is 0 and every code is 0, as the definition says
  p.r = s == 0.0f ? 0.0f : ((s > 1e-30f && s < 1e30f) ? __frcp_rn(s) : __int_as_float(0x7fc00000));
  // The rounding by addition needs |w * r| well below 2^22.  No weight of the unit exceeds its
  // max-abs and the product is monotone, so one test per unit covers them all (it fails only
  // where the stored scale lost its precision to fp16's subnormal range).
  if (!(__fmul_rn(amax, p.r) < 200.0f)) p.r = __int_as_float(0x7fc00000);
  p.qlo = qlo;
  p.qhi = qhi;
  return p;
}
// Adding and subtracting 1.5 * 2^23 rounds a float of magnitude below 2^22 to the nearest integer,
// ties to even (the addition's own rounding); after the addition the integer sits in the low
// mantissa bits in two's complement.
// one code (its low bits are the field): round-half-even of the fp32 quotient e / s, clamped
__device__ __forceinline__ uint32_t quantise1(float e, const QuantParams& p) {
  const float t = __fmul_rn(e, p.r);  // never contracted into the addition below
  float q = __fsub_rn(__fadd_rn(t, ROUND_MAGIC), ROUND_MAGIC);
  const float d = fabsf(fabsf(t - q) - 0.5f);
  if (!(d >= 1e-4f)) q = rintf(__fdiv_rn(e, p.s));  // also every weight of a unit whose reciprocal is NaN
  q = fminf(fmaxf(q, p.qlo), p.qhi);
  return __float_as_uint(__fadd_rn(q, ROUND_MAGIC));
}

// codes of 4 weights: round half to even on the quotient by the stored scale, clamp, pack
template <int BITS>
__device__ __forceinline__ uint32_t quantise4(const float4& v, const QuantParams& p) {
  constexpr int MASK = (1 << BITS) - 1;
  const float e[4] = {v.x, v.y, v.z, v.w};
  uint32_t word = 0;
#pragma unroll
  for (int c = 0; c < 4; ++c) word |= (quantise1(e[c], p) & MASK) << (BITS * c);
  return word;
}

__device__ __forceinline__ float amax4(const float4& v) {
  return fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
}

template <int BITS, typename Source>
__global__ void __launch_bounds__(256) quantise_kernel(const Source src, int N, int K, int G, int ngroups, int scale_f16,
                                                       int full_range, uint8_t* __restrict__ packed,
                                                       void* __restrict__ scales) {
  typedef typename PackWord<BITS>::type word_t;
  constexpr int MASK = (1 << BITS) - 1;
  const float qhi = static_cast<float>((1 << (BITS - 1)) - 1);
  const float qlo = full_range ? -static_cast<float>(1 << (BITS - 1)) : -qhi;
  const float range = full_range ? static_cast<float>(1 << (BITS - 1)) : qhi;  // max-abs is divided by this
  const int lane = threadIdx.x & 31;
  const long long n_units = static_cast<long long>(N) * ngroups;
  const long long warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;
  const long long warp = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const size_t row_bytes = static_cast<size_t>(K) * BITS / 8;

  if constexpr (Source::IN_BITS == 4 && BITS == 2) {
    if (G == 128) {
      // A 4-bit unit holds at most 16 different weights: the unit's 8 lanes quantise two of the 16
      // possible codes each (with the very function every other path uses), share the results as a
      // table of 16 x 2 bits, and every stored code is then a table lookup.  The unit's max-abs is
      // s * max |q| (rounding is monotone), found on the integer codes.
      constexpr int STEPS = Source::STEPS;
      const long long n_steps = (n_units + 3) >> 2;
      for (long long st0 = warp * STEPS; st0 < n_steps; st0 += warps * STEPS) {
        typename Source::Raw raws[STEPS];
        float s_ins[STEPS];
#pragma unroll
        for (int u = 0; u < STEPS; ++u) {
          const long long unit = (st0 + u) * 4 + (lane >> 3);
          if (unit < n_units) src.load_raw(unit * 128 + (lane & 7) * 16, unit, raws[u], s_ins[u]);
          else src.zero_raw(raws[u], s_ins[u]);
        }
#pragma unroll
        for (int u = 0; u < STEPS; ++u) {
          const long long unit = (st0 + u) * 4 + (lane >> 3);
          const bool live = unit < n_units;
          const uint32_t rx = raws[u].w[0], ry = raws[u].w[1];
          const float s_in = s_ins[u];
          int m = 0;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const uint32_t word = c < 8 ? rx : ry;
            const int q = static_cast<int>(word << (28 - 4 * (c & 7))) >> 28;
            m = max(m, abs(q));
          }
#pragma unroll
          for (int o = 4; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
          const float amax = __fmul_rn(static_cast<float>(m), s_in);
          const QuantParams p = quant_params(store_scale(amax, range, scale_f16, scales, unit, live && (lane & 7) == 0), amax, qlo, qhi);
          uint32_t lut = 0;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const int nib = 2 * (lane & 7) + i;
            const int q = (nib ^ 8) - 8;  // the field's value
            lut |= (quantise1(__fmul_rn(static_cast<float>(q), s_in), p) & 3u) << (2 * nib);
          }
#pragma unroll
          for (int o = 4; o > 0; o >>= 1) lut |= __shfl_xor_sync(0xffffffffu, lut, o);
          uint32_t out = 0;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const uint32_t word = c < 8 ? rx : ry;
            const uint32_t nib2 = ((word >> (4 * (c & 7))) << 1) & 30u;
            out |= ((lut >> nib2) & 3u) << (2 * c);
          }
          if (live) *reinterpret_cast<uint32_t*>(packed + (unit * 128 + (lane & 7) * 16) / 4) = out;
        }
      }
      return;
    }
  }
  if (G == 128) {
    // K is a whole number of units, so unit u holds the weights 128 u .. 128 u + 127 of the dense
    // matrix and the bytes 16 b u .. of the packed one, whatever its row
    constexpr int STEPS = Source::STEPS;
    const long long n_steps = (n_units + 3) >> 2;
    for (long long st0 = warp * STEPS; st0 < n_steps; st0 += warps * STEPS) {
      typename Source::Raw raws[STEPS];
      float s_ins[STEPS];
#pragma unroll
      for (int u = 0; u < STEPS; ++u) {
        const long long unit = (st0 + u) * 4 + (lane >> 3);
        if (unit < n_units) src.load_raw(unit * 128 + (lane & 7) * 16, unit, raws[u], s_ins[u]);
        else src.zero_raw(raws[u], s_ins[u]);
      }
#pragma unroll
      for (int u = 0; u < STEPS; ++u) {
        const long long unit = (st0 + u) * 4 + (lane >> 3);
        const bool live = unit < n_units;
        float v[16];
        src.decode(raws[u], s_ins[u], v);
        float amax = 0.0f;
#pragma unroll
        for (int c = 0; c < 16; ++c) amax = fmaxf(amax, fabsf(v[c]));
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        const QuantParams p = quant_params(store_scale(amax, range, scale_f16, scales, unit, live && (lane & 7) == 0), amax, qlo, qhi);
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        constexpr int PER_WORD = 32 / BITS;
#pragma unroll
        for (int c = 0; c < 16; ++c) w[c / PER_WORD] |= (quantise1(v[c], p) & MASK) << (BITS * (c % PER_WORD));
        if (live) {
          uint8_t* out = packed + (unit * 128 + (lane & 7) * 16) * BITS / 8;
          if (BITS == 8) *reinterpret_cast<uint4*>(out) = make_uint4(w[0], w[1], w[2], w[3]);
          else if (BITS == 4) *reinterpret_cast<uint2*>(out) = make_uint2(w[0], w[1]);
          else *reinterpret_cast<uint32_t*>(out) = w[0];
        }
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
    const QuantParams p = quant_params(store_scale(amax, range, scale_f16, scales, unit, lane == 0), amax, qlo, qhi);
    word_t* out = reinterpret_cast<word_t*>(packed + static_cast<size_t>(n) * row_bytes + static_cast<size_t>(g) * G * BITS / 8);
    for (int i = lane * 4; i < G; i += 128) {
      const float4 v = i < 128 ? first : src.load4(n, k_first + i, unit);  // later steps come from L1/L2
      out[i >> 2] = static_cast<word_t>(quantise4<BITS>(v, p));
    }
  }
}

template <typename Source>
cudaError_t launch_quantise(const Source& src, int N, int K, int bits, int group, int scale_f16, int full_range,
                            uint8_t* packed, void* scales, cudaStream_t st) {
  const int G = group > 0 ? group : K;
  const int ngroups = K / G;
  const long long units = static_cast<long long>(N) * ngroups;
  const long long warps_needed = G == 128 ? (units + 4 * Source::STEPS - 1) / (4 * Source::STEPS) : units;
  const int threads = 256;
  long long blocks = (warps_needed * 32 + threads - 1) / threads;
  const long long cap = 148LL * 8 * 4;  // a few waves of resident blocks; each warp then loops over its units
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const dim3 grid(static_cast<unsigned>(blocks));
  switch (bits) {
    case 2: quantise_kernel<2, Source><<<grid, threads, 0, st>>>(src, N, K, G, ngroups, scale_f16, full_range, packed, scales); break;
    case 4: quantise_kernel<4, Source><<<grid, threads, 0, st>>>(src, N, K, G, ngroups, scale_f16, full_range, packed, scales); break;
    case 8: quantise_kernel<8, Source><<<grid, threads, 0, st>>>(src, N, K, G, ngroups, scale_f16, full_range, packed, scales); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_pack(const float* W, int N, int K, int bits, int group, int scale_f16, int full_range, uint8_t* packed,
                        void* scales, cudaStream_t st) {
  return launch_quantise(SourceF32{W, K}, N, K, bits, group, scale_f16, full_range, packed, scales, st);
}

cudaError_t launch_requant(const uint8_t* in_packed, const void* in_scales, int N, int K, int bits_in, int bits_out,
                           int group, int scale_f16, int full_range, uint8_t* packed, void* scales, cudaStream_t st) {
  switch (bits_in) {
    case 2: return launch_quantise(SourcePacked<2>{in_packed, in_scales, K, scale_f16}, N, K, bits_out, group, scale_f16, full_range, packed, scales, st);
    case 4: return launch_quantise(SourcePacked<4>{in_packed, in_scales, K, scale_f16}, N, K, bits_out, group, scale_f16, full_range, packed, scales, st);
    case 8: return launch_quantise(SourcePacked<8>{in_packed, in_scales, K, scale_f16}, N, K, bits_out, group, scale_f16, full_range, packed, scales, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace emoe
