// Device helpers shared by the tensor-core expert-FFN kernels: the bitwidth-specialised unpack
// of packed codes into exact bf16 integers, the MMA wrapper, and the activation layout.
//
// Activation layout ("k-interleave").  An MMA does not care in which order the reduction index
// is enumerated as long as A and B agree, so the activations (x rows and the hidden vector) are
// stored once in the order that makes both operands cheap:
//   * inside a 128-input segment, lane t of a quad owns inputs [32t, 32t+32);
//   * the unpack emits code pairs (c, c+4) of an 8-code word at 4 bits, (c, c+8) of a 16-code
//     word at 2 bits and (2c, 2c+1) at 8 bits, so the lane's 32 activations are stored in that
//     pair order (position 2r, 2r+1 <- the two inputs of pair r);
//   * the lane's four 16-byte pieces q are stored piece-major, at (q*4 + t)*16 bytes of the
//     segment, so that the four lanes of a quad read adjacent 16-byte columns of shared memory.
#pragma once
#include "common.cuh"

namespace emoe {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// (a & b) ^ c in one LOP3
__device__ __forceinline__ uint32_t and_xor(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0x6a;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

__device__ __forceinline__ uint32_t bf16x2_fma(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t a0, const uint32_t a1, const uint32_t a2,
                                         const uint32_t a3, const uint32_t b0, const uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---- per-bitwidth unpack: 32 codes of one output channel -> 16 bf16x2 registers -------------
// P[r] holds the codes with local index (a_r, b_r); the interleaved activation layout puts
// x[a_r] at position 2r and x[b_r] at 2r+1 of the lane's 32-element block.
template <int BITS>
struct Raw;  // the lane's raw bytes for one row of one segment
template <>
struct Raw<8> { uint4 v[2]; };
template <>
struct Raw<4> { uint4 v[1]; };
template <>
struct Raw<2> { uint2 v[1]; };

template <int BITS>
__device__ __forceinline__ Raw<BITS> load_raw(const uint8_t* p);
template <>
__device__ __forceinline__ Raw<8> load_raw<8>(const uint8_t* p) {
  Raw<8> r;
  r.v[0] = __ldg(reinterpret_cast<const uint4*>(p));
  r.v[1] = __ldg(reinterpret_cast<const uint4*>(p) + 1);
  return r;
}
template <>
__device__ __forceinline__ Raw<4> load_raw<4>(const uint8_t* p) {
  Raw<4> r;
  r.v[0] = __ldg(reinterpret_cast<const uint4*>(p));
  return r;
}
template <>
__device__ __forceinline__ Raw<2> load_raw<2>(const uint8_t* p) {
  Raw<2> r;
  r.v[0] = __ldg(reinterpret_cast<const uint2*>(p));
  return r;
}

// 8 bits: byte -> 2^23 + (q+128) as fp32 by byte permute, subtract, keep the high halves
// (integers of magnitude <= 128 are exact in bf16).  Natural pair order (2r, 2r+1).
__device__ __forceinline__ void unpack(const Raw<8>& raw, uint32_t (&P)[16]) {
  const uint32_t w[8] = {raw.v[0].x, raw.v[0].y, raw.v[0].z, raw.v[0].w, raw.v[1].x, raw.v[1].y, raw.v[1].z, raw.v[1].w};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t u = w[i] ^ 0x80808080u;
    const float f0 = __uint_as_float(prmt(u, 0x4B000000u, 0x7540u)) - 8388736.0f;
    const float f1 = __uint_as_float(prmt(u, 0x4B000000u, 0x7541u)) - 8388736.0f;
    const float f2 = __uint_as_float(prmt(u, 0x4B000000u, 0x7542u)) - 8388736.0f;
    const float f3 = __uint_as_float(prmt(u, 0x4B000000u, 0x7543u)) - 8388736.0f;
    P[2 * i] = prmt(__float_as_uint(f0), __float_as_uint(f1), 0x7632u);
    P[2 * i + 1] = prmt(__float_as_uint(f2), __float_as_uint(f3), 0x7632u);
  }
}

// 4 bits: nibble c of a 16-bit half lands in the mantissa of bf16 128.0 (ulp 1), with its
// sign bit flipped (two's complement -> offset binary): value 128 + (q + 8); subtract 136.
// Pair order (c, c+4) inside each 8-code word.
__device__ __forceinline__ void unpack(const Raw<4>& raw, uint32_t (&P)[16]) {
  const uint32_t w[4] = {raw.v[0].x, raw.v[0].y, raw.v[0].z, raw.v[0].w};
  const uint32_t one = 0x3F803F80u;   // bf16x2 (1, 1)
  const uint32_t m136 = 0xC308C308u;  // bf16x2 (-136, -136)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint32_t v = and_xor(w[i] >> (4 * c), 0x000F000Fu, 0x43084308u);
      P[4 * i + c] = bf16x2_fma(v, one, m136);
    }
  }
}

// 2 bits: field at mantissa bit p in {0,2,4} of bf16 128.0: value 128 + (q + 2) * 2^p;
// q = v * 2^-p - (128 * 2^-p + 2).  Pair order (c, c+8) inside each 16-code word.
__device__ __forceinline__ void unpack(const Raw<2>& raw, uint32_t (&P)[16]) {
  const uint32_t w[2] = {raw.v[0].x, raw.v[0].y};
  // bf16: 1 = 0x3F80, 0.25 = 0x3E80, 0.0625 = 0x3D80; -130 = 0xC302, -34 = 0xC208, -10 = 0xC120
  const uint32_t mul[3] = {0x3F803F80u, 0x3E803E80u, 0x3D803D80u};
  const uint32_t add[3] = {0xC302C302u, 0xC208C208u, 0xC120C120u};
  const uint32_t msk[3] = {0x00030003u, 0x000C000Cu, 0x00300030u};
  const uint32_t mag[3] = {0x43024302u, 0x43084308u, 0x43204320u};  // 128 with the field's sign bit set
#pragma unroll
  for (int i = 0; i < 2; ++i) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int sh = 6 * (c / 3), p = c % 3;
      const uint32_t v = and_xor(w[i] >> sh, msk[p], mag[p]);
      P[8 * i + c] = bf16x2_fma(v, mul[p], add[p]);
    }
  }
}

// One k16-pair step of the unpack: the four registers (code pairs 4q .. 4q+3 of the lane's
// row) that feed the two MMAs of step q, so that a tile can be consumed step by step without
// holding all 16 registers of a row at once.
__device__ __forceinline__ void unpack_step(const Raw<8>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[8] = {raw.v[0].x, raw.v[0].y, raw.v[0].z, raw.v[0].w, raw.v[1].x, raw.v[1].y, raw.v[1].z, raw.v[1].w};
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const uint32_t u = w[2 * q + j] ^ 0x80808080u;
    const float f0 = __uint_as_float(prmt(u, 0x4B000000u, 0x7540u)) - 8388736.0f;
    const float f1 = __uint_as_float(prmt(u, 0x4B000000u, 0x7541u)) - 8388736.0f;
    const float f2 = __uint_as_float(prmt(u, 0x4B000000u, 0x7542u)) - 8388736.0f;
    const float f3 = __uint_as_float(prmt(u, 0x4B000000u, 0x7543u)) - 8388736.0f;
    o[2 * j] = prmt(__float_as_uint(f0), __float_as_uint(f1), 0x7632u);
    o[2 * j + 1] = prmt(__float_as_uint(f2), __float_as_uint(f3), 0x7632u);
  }
}
__device__ __forceinline__ void unpack_step(const Raw<4>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[4] = {raw.v[0].x, raw.v[0].y, raw.v[0].z, raw.v[0].w};
#pragma unroll
  for (int c = 0; c < 4; ++c)
    o[c] = bf16x2_fma(and_xor(w[q] >> (4 * c), 0x000F000Fu, 0x43084308u), 0x3F803F80u, 0xC308C308u);
}
__device__ __forceinline__ void unpack_step(const Raw<2>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[2] = {raw.v[0].x, raw.v[0].y};
  const uint32_t mul[3] = {0x3F803F80u, 0x3E803E80u, 0x3D803D80u};
  const uint32_t add[3] = {0xC302C302u, 0xC208C208u, 0xC120C120u};
  const uint32_t msk[3] = {0x00030003u, 0x000C000Cu, 0x00300030u};
  const uint32_t mag[3] = {0x43024302u, 0x43084308u, 0x43204320u};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = 4 * (q & 1) + j;
    const int sh = 6 * (c / 3), p = c % 3;
    o[j] = bf16x2_fma(and_xor(w[q >> 1] >> sh, msk[p], mag[p]), mul[p], add[p]);
  }
}

// ---- offset codes: the unpack of the streaming kernel -------------------------------------------
// fp16 has a 10-bit mantissa, so a code field that sits at bit p of a 16-bit half can be read in
// place as mantissa bits of the fp16 number 2^(10-p) (whose mantissa bit p weighs 1): masking the
// field, flipping its sign bit (two's complement -> offset binary) and setting the exponent is
// ONE logic instruction, and the result is the exact fp16 integer c + q with the constant
// c = 2^(10-p) + 2^(b-1).  The constant is not subtracted per code:
//   sum_k (c + q_k) x_k  =  sum_k q_k x_k  +  c * sum_k x_k,
// and the second sum does not depend on the output channel, so one extra MMA per step, with the
// constants as its A operand, yields it for all channels of the warp at once.  Products of two
// fp16 numbers are exact in fp32; what the subtraction costs is cancellation inside the tensor
// core's accumulation, which grows with c / rms(q).  The fields are therefore moved (one shift
// per word of fields) to the highest position that holds them, where c is smallest:
//   8 bits: no constant is carried: byte ^ 0x80 under the exponent byte 0x64 is 1152 + q, and one
//           fp16x2 subtraction makes it q (the only position that holds 8 bits is p = 0, where
//           c = 1152 costs more accuracy than the subtraction costs time), pairs (2c, 2c+1);
//   4 bits: pairs (c, c+4) of an 8-code word, every field at p = 4: 72 + q;
//   2 bits: pairs (c, c+8) of a 16-code word, odd c at p = 8 (6 + q), even c at p = 6 (18 + q),
//           two neighbouring pairs per shifted word.
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t a0, const uint32_t a1, const uint32_t a2,
                                        const uint32_t a3, const uint32_t b0, const uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t f16x2_sub(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// fp16x2 constant c of register j (0..3) of a step, per bitwidth (both halves equal)
template <int BITS>
__device__ __forceinline__ constexpr uint32_t offset_const(int j) {
  if (BITS == 8) return 0u;                      // exact codes, nothing to take out
  if (BITS == 4) return 0x54805480u;             // 72
  return (j & 1) ? 0x46004600u : 0x4C804C80u;    // odd pair: 6, even pair: 18
}

// the four registers (code pairs 4q .. 4q+3 of the lane's row) of step q as offset codes
__device__ __forceinline__ void unpack_step_off(const Raw<8>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[8] = {raw.v[0].x, raw.v[0].y, raw.v[0].z, raw.v[0].w, raw.v[1].x, raw.v[1].y, raw.v[1].z, raw.v[1].w};
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const uint32_t u = w[2 * q + j] ^ 0x80808080u;
    o[2 * j] = f16x2_sub(prmt(u, 0x64646464u, 0x4140u), 0x64806480u);
    o[2 * j + 1] = f16x2_sub(prmt(u, 0x64646464u, 0x4342u), 0x64806480u);
  }
}
__device__ __forceinline__ void unpack_step_off(const Raw<4>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[4] = {raw.v[0].x, raw.v[0].y, raw.v[0].z, raw.v[0].w};
  const uint32_t v = w[q];  // nibble c of each half goes to bits 4..7
  o[0] = and_xor(v << 4, 0x00F000F0u, 0x54805480u);
  o[1] = and_xor(v, 0x00F000F0u, 0x54805480u);
  o[2] = and_xor(v >> 4, 0x00F000F0u, 0x54805480u);
  o[3] = and_xor(v >> 8, 0x00F000F0u, 0x54805480u);
}
__device__ __forceinline__ void unpack_step_off(const Raw<2>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[2] = {raw.v[0].x, raw.v[0].y};
  const uint32_t v = w[q >> 1];
  // pairs c = 4(q&1) + j; field c of each half to bits 8..9 (odd c) or 6..7 (even c): the
  // shift that puts an odd c at bit 8 puts c - 1 at bit 6
  uint32_t s01, s23;  // fields (c0, c0+1) and (c0+2, c0+3) in place
  if ((q & 1) == 0) {
    s01 = v << 6;
    s23 = v << 2;
  } else {
    s01 = v >> 2;
    s23 = v >> 6;
  }
  o[0] = and_xor(s01, 0x00C000C0u, 0x4C804C80u);
  o[1] = and_xor(s01, 0x03000300u, 0x46004600u);
  o[2] = and_xor(s23, 0x00C000C0u, 0x4C804C80u);
  o[3] = and_xor(s23, 0x03000300u, 0x46004600u);
}

// The same registers as exact fp16 integers q (the constant subtracted per pair): one more
// instruction per pair and no extra MMAs, the better trade when a pass multiplies every code
// with several token tiles.  Fields are read where they sit (p = 0 / 4 at 4 bits, p = 0..8 at 2
// bits: the subtraction is exact whatever the constant).
__device__ __forceinline__ void unpack_step_exact(const Raw<8>& raw, int q, uint32_t (&o)[4]) { unpack_step_off(raw, q, o); }
__device__ __forceinline__ void unpack_step_exact(const Raw<4>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[4] = {raw.v[0].x, raw.v[0].y, raw.v[0].z, raw.v[0].w};
  const uint32_t lo = w[q], hi = lo >> 8;
  o[0] = f16x2_sub(and_xor(lo, 0x000F000Fu, 0x64086408u), 0x64086408u);  // 1032 + q
  o[1] = f16x2_sub(and_xor(lo, 0x00F000F0u, 0x54805480u), 0x54805480u);  // 72 + q
  o[2] = f16x2_sub(and_xor(hi, 0x000F000Fu, 0x64086408u), 0x64086408u);
  o[3] = f16x2_sub(and_xor(hi, 0x00F000F0u, 0x54805480u), 0x54805480u);
}
__device__ __forceinline__ void unpack_step_exact(const Raw<2>& raw, int q, uint32_t (&o)[4]) {
  const uint32_t w[2] = {raw.v[0].x, raw.v[0].y};
  const uint32_t lo = w[q >> 1], hi = lo >> 10;
  // 2^(10-p) + 2 as fp16 for p = 0, 2, 4, 6, 8: 1026, 258, 66, 18, 6
  const uint32_t mag[5] = {0x64026402u, 0x5C085C08u, 0x54205420u, 0x4C804C80u, 0x46004600u};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = 4 * (q & 1) + j;  // pair (c, c+8) of the 16-code word
    const int pi = c < 5 ? c : c - 5;
    o[j] = f16x2_sub(and_xor(c < 5 ? lo : hi, 0x00030003u << (2 * pi), mag[pi]), mag[pi]);
  }
}

// is the fp32 value outside what fp16 can hold (it would be saturated)?
__device__ __forceinline__ bool beyond_f16(float v) { return fabsf(v) > 65504.0f; }
// do both bf16 halves fit fp16?  (exponent field above that of 65504 = 2^15 * 1.999: bf16 exponent >= 143)
__device__ __forceinline__ bool bf16x2_beyond_f16(uint32_t v) {
  return ((v >> 7) & 0xffu) >= 143u || ((v >> 23) & 0xffu) >= 143u;
}
// two bf16 values -> two fp16 values (exact inside the fp16 range, saturating outside)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2_sat(uint32_t v) {
  const float lo = fminf(fmaxf(__uint_as_float(v << 16), -65504.0f), 65504.0f);
  const float hi = fminf(fmaxf(__uint_as_float(v & 0xffff0000u), -65504.0f), 65504.0f);
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ __half f32_to_f16_sat(float v) {
  return __float2half_rn(fminf(fmaxf(v, -65504.0f), 65504.0f));
}

// position of input k (natural order) in the activation layout described at the top
template <int BITS>
__device__ __forceinline__ int act_pos(int k) {
  const int kk = k & 127, t = kk >> 5, i = kk & 31;
  int j = i;
  if (BITS != 8) {
    constexpr int B = BITS == 4 ? 8 : 16;  // codes per unpacked word
    const int o = i & (B - 1);
    j = (i & ~(B - 1)) + (o < B / 2 ? 2 * o : 2 * (o - B / 2) + 1);
  }
  return (k & ~127) + (((j >> 3) * 4 + t) << 3) + (j & 7);
}

__device__ __forceinline__ float load_scale_ro(const void* scales, bool f16, size_t idx) {
  return f16 ? __half2float(__ldg(reinterpret_cast<const __half*>(scales) + idx))
             : __ldg(reinterpret_cast<const float*>(scales) + idx);
}

}  // namespace emoe
