// Activations of the int8 tensor-core expert kernel (ffn_i8.cu): block-scaled two-limb integers.
//
// The expert kernel multiplies the packed codes (Section 3.2 of the paper: b-bit integers q with a
// scale channel, w~ = q * s) as 8-bit integer tensor-core operands, so the other operand, the
// activations, must be 8-bit integers too.  A bf16 activation has 8 significant bits; two signed
// 8-bit limbs under a power-of-two scale shared by a block of 128 inputs hold 15:
//     x  ~=  2^(E-13) * (128 * hi + lo),     2^E <= max |x| of the block < 2^(E+1),
//     v = rint(x * 2^(13-E)) in (-2^14, 2^14),  hi = v >> 7 in [-128, 127],  lo = v & 127 in [0, 127].
// Every element within a factor 2^6 of the block maximum is represented exactly, the others with
// an absolute error of at most 2^(E-14): far below the bf16 rounding the values already carry.
// The tensor core then forms sum_k q_k * hi_k and sum_k q_k * lo_k exactly in 32-bit integers.
//
// Layout in global memory, per slot (token in expert order): two rows of K signed bytes (hi, then
// lo) and K/128 fp32 block scales 2^(E-13) (0 is never needed: an all-zero block has v = 0).
// Inside each block of 128 inputs the bytes are stored in the order in which the unpack of the
// owning expert's bitwidth emits its codes (act_q_pos), so that both operands enumerate the
// reduction index alike.
#pragma once
#include "common.cuh"

namespace emoe {

// Position of input k (natural order) inside the activation rows for an expert of `BITS` bits.
//   8 bits: codes are used as they lie: identity;
//   4 bits: a 32-bit word of eight nibbles is split into (even nibbles, odd nibbles):
//           inside each 8: order 0 2 4 6 1 3 5 7;
//   2 bits: a word of sixteen fields is split into four words of fields (r, r+4, r+8, r+12):
//           inside each 16: order 0 4 8 12 1 5 9 13 2 6 10 14 3 7 11 15.
template <int BITS>
__host__ __device__ __forceinline__ int act_q_pos(int k) {
  if (BITS == 8) return k;
  if (BITS == 4) return (k & ~7) + ((k & 1) << 2) + ((k & 7) >> 1);
  return (k & ~15) + ((k & 3) << 2) + ((k & 15) >> 2);
}
__host__ __device__ __forceinline__ int act_q_pos_rt(int bits, int k) {
  return bits == 8 ? act_q_pos<8>(k) : (bits == 4 ? act_q_pos<4>(k) : act_q_pos<2>(k));
}

constexpr int ACT_Q_MIN_EXP = -100;  // blocks whose maximum lies below 2^-100 are scaled as if it were 2^-100

// exponent E of a block from the largest |x| of the block given as fp32 bits (sign cleared)
__device__ __forceinline__ int act_q_block_exp(uint32_t max_abs_bits) {
  const int e = static_cast<int>(max_abs_bits >> 23) - 127;
  return e < ACT_Q_MIN_EXP ? ACT_Q_MIN_EXP : e;
}
__device__ __forceinline__ float act_q_inv_scale(int E) { return __uint_as_float(static_cast<uint32_t>(140 - E) << 23); }  // 2^(13-E)
__device__ __forceinline__ float act_q_scale(int E) { return __uint_as_float(static_cast<uint32_t>(E + 114) << 23); }      // 2^(E-13)

// the integer v of one value; hi = v >> 7, lo = v & 127
__device__ __forceinline__ int act_q_int(float x, float inv_scale) { return __float2int_rn(x * inv_scale); }

__device__ __forceinline__ uint32_t redux_max_u32(uint32_t v) {
  uint32_t r;
  asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
  return r;
}

// One activation row (bf16, natural order) -> limb rows + block scales, by the threads of a CTA
// (any multiple of 32): a warp takes one 128-input block at a time; a lane produces the four
// bytes of output positions 4*lane .. 4*lane+3 of the block, i.e. it picks the four inputs that
// the order above puts there, and writes them with one 32-bit store per limb.
__device__ __forceinline__ void act_q_row(const __nv_bfloat16* __restrict__ src, int8_t* __restrict__ dst_hi,
                                          int8_t* __restrict__ dst_lo, float* __restrict__ dst_scale, int K, int bits) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  for (int blk = warp; blk < K / 128; blk += nwarps) {
    const __nv_bfloat16* b = src + blk * 128;
    float x[4];
    if (bits == 8) {
      const uint2 v = *reinterpret_cast<const uint2*>(b + 4 * lane);
      x[0] = __uint_as_float(v.x << 16);
      x[1] = __uint_as_float(v.x & 0xffff0000u);
      x[2] = __uint_as_float(v.y << 16);
      x[3] = __uint_as_float(v.y & 0xffff0000u);
    } else if (bits == 4) {
      // positions 4*lane + i of the block: the 8 inputs 8*(lane/2) ..., even ones for even lanes, odd for odd
      const uint4 v = *reinterpret_cast<const uint4*>(b + 8 * (lane >> 1));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) x[i] = __uint_as_float((lane & 1) ? (w[i] & 0xffff0000u) : (w[i] << 16));
    } else {
      // positions 4*lane + i: inputs 16*(lane/4) + (lane%4) + 4*i
      const uint4 v0 = *reinterpret_cast<const uint4*>(b + 16 * (lane >> 2));
      const uint4 v1 = *reinterpret_cast<const uint4*>(b + 16 * (lane >> 2) + 8);
      const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
      const int r = lane & 3;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // element r + 4i sits in word (r + 4i) / 2 = 2i + r/2, half r & 1
        const uint32_t ww = (r >> 1) ? w[2 * i + 1] : w[2 * i];
        x[i] = __uint_as_float((r & 1) ? (ww & 0xffff0000u) : (ww << 16));
      }
    }
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) m = max(m, __float_as_uint(x[i]) & 0x7fffffffu);
    const int E = act_q_block_exp(redux_max_u32(m));
    const float inv = act_q_inv_scale(E);
    uint32_t hi = 0, lo = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int v = act_q_int(x[i], inv);
      hi |= static_cast<uint32_t>((v >> 7) & 0xff) << (8 * i);
      lo |= static_cast<uint32_t>(v & 127) << (8 * i);
    }
    *reinterpret_cast<uint32_t*>(dst_hi + blk * 128 + 4 * lane) = hi;
    *reinterpret_cast<uint32_t*>(dst_lo + blk * 128 + 4 * lane) = lo;
    if (lane == 0) dst_scale[blk] = act_q_scale(E);
  }
}

}  // namespace emoe
