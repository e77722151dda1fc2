// Grouped expert FFN on packed weights with tensor-core multiply-adds, for bf16 activations
// and small-to-moderate token counts per expert (the decode regime).  Paper Sections 1/2.1
// (each activated expert is an independent FFN) on the Section 3.2 storage (b-bit codes plus a
// scale channel, decompressed as q * s) — formed here in registers.
//
// The work is bound by streaming the packed weights from HBM, so the kernel is built around
// that stream: every lane pulls the codes of two output channels straight from global memory
// into registers (128-bit loads at 8 and 4 bits, 64-bit at 2 bits, so that the four lanes of a
// quad always cover exactly one 128-input scale group), turns them into bf16 *integers* with
// one bitwidth-specialised unpack, and feeds them as the A operand of mma.m16n8k16; the
// expert's tokens are the (small) N dimension, staged in shared memory.  The codes are exact
// in bf16, products accumulate in fp32, and each 128-input group's partial sum is multiplied
// by its fp32/fp16 scale before it joins the running total, so the result equals q * s * x
// with no rounding of the dequantised weight.
//
// k-order trick: an MMA does not care in which order the reduction index is enumerated as
// long as A and B agree.  The unpack yields code pairs (c, c+4) of an 8-code word at 4 bits
// and (c, c+8) of a 16-code word at 2 bits, so the activations are stored in that interleaved
// order once (scatter_x_kernel for x, the first phase's epilogue for the hidden vector) and
// B fragments become plain 128-bit shared-memory loads.
#include "common.cuh"

namespace emoe {
namespace {

constexpr int MMA_WARPS = 4;
constexpr int MMA_THREADS = MMA_WARPS * 32;
constexpr int MMA_MT = 2;          // 16-row tiles per warp
constexpr int MMA_KCH = 512;       // inputs per staged activation chunk (4 segments of 128)
constexpr int MMA_XPAD = 8;        // bf16 elements of row padding in shared memory
constexpr int MMA_XSTRIDE = MMA_KCH + MMA_XPAD;

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
  asm volatile(
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

// position of element `o` (natural order) inside its interleaved block
template <int BITS>
__device__ __forceinline__ int interleaved_pos(int k) {
  if (BITS == 8) return k;
  constexpr int B = BITS == 4 ? 8 : 16;  // block length
  const int o = k & (B - 1);
  return (k & ~(B - 1)) + (o < B / 2 ? 2 * o : 2 * (o - B / 2) + 1);
}

__device__ __forceinline__ float load_scale(const void* scales, bool f16, size_t idx) {
  return f16 ? __half2float(__ldg(reinterpret_cast<const __half*>(scales) + idx))
             : __ldg(reinterpret_cast<const float*>(scales) + idx);
}

// ---- the kernel body for one bitwidth -----------------------------------------------------------
template <int BITS, int NT>
__device__ __forceinline__ void ffn_mma_body(int phase, const LayerDims& L, const ExpertDev& ex,
                                             const __nv_bfloat16* __restrict__ in, int begin, int cnt,
                                             __nv_bfloat16* __restrict__ hidden, float* __restrict__ o_part,
                                             int ksplit, int n_pairs, __nv_bfloat16* xsm) {
  constexpr int LANE_BYTES = 32 * BITS / 8;  // bytes of one row a lane owns per 128-input segment
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const int K = phase == 0 ? L.d_model : L.d_ff;
  const int G = L.group > 0 ? L.group : K;
  const int ngroups = K / G;
  const bool swiglu_in = phase == 0 && L.act == EMOE_ACT_SWIGLU;
  const bool sf16 = L.scale_f16 != 0;
  const size_t row_bytes = static_cast<size_t>(K) * BITS / 8;

  // which matrix and which 16 rows each m-tile of this warp covers
  const int rows_per_warp = swiglu_in ? 16 : 16 * MMA_MT;
  const int row0 = (blockIdx.x * MMA_WARPS + warp) * rows_per_warp;
  const uint8_t* wbase[MMA_MT][2];
  const void* sbase[MMA_MT];
  size_t srow[MMA_MT][2];
#pragma unroll
  for (int mt = 0; mt < MMA_MT; ++mt) {
    const int mat = phase == 0 ? (swiglu_in ? mt : 0) : (L.act == EMOE_ACT_SWIGLU ? 2 : 1);
    const int r = swiglu_in ? row0 : row0 + 16 * mt;
    sbase[mt] = ex.scales[mat];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int rr = min(r + g + 8 * h, N - 1);
      wbase[mt][h] = ex.packed[mat] + static_cast<size_t>(rr) * row_bytes + t * LANE_BYTES;
      srow[mt][h] = static_cast<size_t>(rr) * ngroups;
    }
  }

  const int chunks_total = (K + MMA_KCH - 1) / MMA_KCH;
  const int cpz = (chunks_total + ksplit - 1) / ksplit;
  const int kc_begin = blockIdx.y * cpz;
  const int kc_end = min(chunks_total, kc_begin + cpz);

  for (int p0 = 0; p0 < cnt; p0 += NT * 8) {
    const int ntok = min(NT * 8, cnt - p0);
    float tot[MMA_MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MMA_MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) tot[mt][nt][i] = 0.0f;

    for (int kc = kc_begin; kc < kc_end; ++kc) {
      const int k0 = kc * MMA_KCH;
      const int klen = min(MMA_KCH, K - k0);
      // stage the activation chunk [NT*8 tokens][klen] (rows past the expert's tokens are zero)
      __syncthreads();
      for (int idx = tid; idx < NT * 8 * (MMA_KCH / 8); idx += MMA_THREADS) {
        const int r = idx / (MMA_KCH / 8), v = idx % (MMA_KCH / 8);
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (r < ntok && v * 8 < klen)
          val = *reinterpret_cast<const uint4*>(in + static_cast<size_t>(begin + p0 + r) * K + k0 + v * 8);
        *reinterpret_cast<uint4*>(xsm + r * MMA_XSTRIDE + v * 8) = val;
      }
      __syncthreads();

      const int nseg = klen / 128;
      for (int sg = 0; sg < nseg; ++sg) {
        const int kseg = k0 + sg * 128;
        const size_t boff = static_cast<size_t>(kseg) * BITS / 8;
        Raw<BITS> raw[MMA_MT][2];
#pragma unroll
        for (int mt = 0; mt < MMA_MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) raw[mt][h] = load_raw<BITS>(wbase[mt][h] + boff);
        const int grp = kseg / G;
        float sc[MMA_MT][2];
#pragma unroll
        for (int mt = 0; mt < MMA_MT; ++mt)
#pragma unroll
          for (int h = 0; h < 2; ++h) sc[mt][h] = load_scale(sbase[mt], sf16, srow[mt][h] + grp);

        // B fragments of this segment: the lane's 32 interleaved activations of token (nt*8 + g)
        uint4 bq[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (nt * 8 < ntok) {
            const uint4* src = reinterpret_cast<const uint4*>(xsm + (nt * 8 + g) * MMA_XSTRIDE + sg * 128 + t * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q) bq[nt][q] = src[q];
          }
        }
#pragma unroll
        for (int mt = 0; mt < MMA_MT; ++mt) {
          uint32_t P0[16], P1[16];
          unpack(raw[mt][0], P0);
          unpack(raw[mt][1], P1);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            if (nt * 8 < ntok) {
              float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                mma_bf16(acc, P0[4 * q], P1[4 * q], P0[4 * q + 1], P1[4 * q + 1], bq[nt][q].x, bq[nt][q].y);
                mma_bf16(acc, P0[4 * q + 2], P1[4 * q + 2], P0[4 * q + 3], P1[4 * q + 3], bq[nt][q].z, bq[nt][q].w);
              }
              tot[mt][nt][0] = fmaf(sc[mt][0], acc[0], tot[mt][nt][0]);
              tot[mt][nt][1] = fmaf(sc[mt][0], acc[1], tot[mt][nt][1]);
              tot[mt][nt][2] = fmaf(sc[mt][1], acc[2], tot[mt][nt][2]);
              tot[mt][nt][3] = fmaf(sc[mt][1], acc[3], tot[mt][nt][3]);
            }
          }
        }
      }
    }

    // epilogue: lane holds rows (g, g+8) x tokens (2t, 2t+1) of every tile
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tok = nt * 8 + 2 * t + (i & 1);
        if (tok >= ntok) continue;
        const size_t slot = static_cast<size_t>(begin + p0 + tok);
        if (swiglu_in) {
          const int n = row0 + g + 8 * (i >> 1);
          if (n < N) {
            const float a = tot[0][nt][i], b = tot[1][nt][i];
            const float h = a / (1.0f + expf(-a)) * b;
            hidden[slot * N + interleaved_pos<BITS>(n)] = __float2bfloat16_rn(h);
          }
        } else {
#pragma unroll
          for (int mt = 0; mt < MMA_MT; ++mt) {
            const int n = row0 + 16 * mt + g + 8 * (i >> 1);
            if (n >= N) continue;
            if (phase == 0)
              hidden[slot * N + interleaved_pos<BITS>(n)] = __float2bfloat16_rn(fmaxf(tot[mt][nt][i], 0.0f));
            else
              o_part[(static_cast<size_t>(blockIdx.y) * n_pairs + slot) * N + n] = tot[mt][nt][i];
          }
        }
      }
    }
  }
}

template <int NT>
__global__ void __launch_bounds__(MMA_THREADS)
    ffn_mma_kernel(int phase, LayerDims L, const ExpertDev* __restrict__ experts, const __nv_bfloat16* __restrict__ in,
                   const int32_t* __restrict__ off, __nv_bfloat16* __restrict__ hidden, float* __restrict__ o_part,
                   int ksplit, int n_pairs) {
  __shared__ __align__(16) __nv_bfloat16 xsm[NT * 8 * MMA_XSTRIDE];
  const int e = blockIdx.z;
  const int begin = off[e];
  const int cnt = off[e + 1] - begin;
  if (cnt <= 0) return;  // only activated experts are touched
  const ExpertDev ex = experts[e];
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const int rows_per_cta = (phase == 0 && L.act == EMOE_ACT_SWIGLU) ? 16 * MMA_WARPS : 16 * MMA_MT * MMA_WARPS;
  if (static_cast<int>(blockIdx.x) * rows_per_cta >= N) return;
  switch (ex.bits) {
    case 2: ffn_mma_body<2, NT>(phase, L, ex, in, begin, cnt, hidden, o_part, ksplit, n_pairs, xsm); break;
    case 4: ffn_mma_body<4, NT>(phase, L, ex, in, begin, cnt, hidden, o_part, ksplit, n_pairs, xsm); break;
    case 8: ffn_mma_body<8, NT>(phase, L, ex, in, begin, cnt, hidden, o_part, ksplit, n_pairs, xsm); break;
    default: break;
  }
}

// x rows -> expert-sorted order, in the k-interleave of the owning expert's bitwidth
__global__ void __launch_bounds__(128)
    scatter_x_kernel(const ExpertDev* __restrict__ experts, const __nv_bfloat16* __restrict__ x,
                     const int32_t* __restrict__ ids, const int32_t* __restrict__ perm, int top_k, int d, int n_pairs,
                     __nv_bfloat16* __restrict__ xs) {
  const int slot = blockIdx.x;
  const int pair = perm[slot];
  if (pair < 0 || pair >= n_pairs) return;
  const int bits = experts[ids[pair]].bits;
  const uint4* src = reinterpret_cast<const uint4*>(x + static_cast<size_t>(pair / top_k) * d);
  uint4* dst = reinterpret_cast<uint4*>(xs + static_cast<size_t>(slot) * d);
  for (int b = threadIdx.x; b < d / 16; b += blockDim.x) {  // 16 elements = two 128-bit vectors
    const uint4 a = src[2 * b], c = src[2 * b + 1];
    uint4 oa, oc;
    if (bits == 8) {
      oa = a;
      oc = c;
    } else if (bits == 4) {  // [0,4,1,5,2,6,3,7] inside each 8
      oa = make_uint4(prmt(a.x, a.z, 0x5410u), prmt(a.x, a.z, 0x7632u), prmt(a.y, a.w, 0x5410u), prmt(a.y, a.w, 0x7632u));
      oc = make_uint4(prmt(c.x, c.z, 0x5410u), prmt(c.x, c.z, 0x7632u), prmt(c.y, c.w, 0x5410u), prmt(c.y, c.w, 0x7632u));
    } else {  // [0,8,1,9,...,7,15] inside each 16
      oa = make_uint4(prmt(a.x, c.x, 0x5410u), prmt(a.x, c.x, 0x7632u), prmt(a.y, c.y, 0x5410u), prmt(a.y, c.y, 0x7632u));
      oc = make_uint4(prmt(a.z, c.z, 0x5410u), prmt(a.z, c.z, 0x7632u), prmt(a.w, c.w, 0x5410u), prmt(a.w, c.w, 0x7632u));
    }
    dst[2 * b] = oa;
    dst[2 * b + 1] = oc;
  }
}

int pick_nt(int T) { return T <= 8 ? 1 : (T <= 16 ? 2 : 4); }

}  // namespace

bool ffn_mma_supported(const LayerDims& L) {
  if (!L.act_bf16) return false;
  if (L.d_model % 128 != 0 || L.d_ff % 128 != 0) return false;
  if (L.group != 0 && L.group % 128 != 0) return false;
  return true;
}

int ffn_mma_ksplit(const LayerDims& L, int T) {
  const int row_blocks = (L.d_model + 16 * MMA_MT * MMA_WARPS - 1) / (16 * MMA_MT * MMA_WARPS);
  const long long active = T * static_cast<long long>(L.top_k) < L.E ? T * static_cast<long long>(L.top_k) : L.E;
  const long long ctas = row_blocks * active;
  const int chunks = (L.d_ff + MMA_KCH - 1) / MMA_KCH;
  long long z = (4 * 148 + ctas - 1) / ctas;
  if (z > chunks) z = chunks;
  if (z > 16) z = 16;
  if (z < 1) z = 1;
  return static_cast<int>(z);
}

cudaError_t launch_scatter_x(const LayerDims& L, const ExpertDev* experts, const void* x, const int32_t* ids,
                             const int32_t* perm, __nv_bfloat16* xs, int n_pairs, cudaStream_t st) {
  scatter_x_kernel<<<n_pairs, 128, 0, st>>>(experts, reinterpret_cast<const __nv_bfloat16*>(x), ids, perm, L.top_k,
                                            L.d_model, n_pairs, xs);
  return cudaGetLastError();
}

cudaError_t launch_ffn_mma(int phase, const LayerDims& L, const ExpertDev* experts, const __nv_bfloat16* in,
                           const int32_t* off, __nv_bfloat16* hidden, float* o_part, int ksplit, int n_pairs, int T,
                           cudaStream_t st) {
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const int rows_per_cta = (phase == 0 && L.act == EMOE_ACT_SWIGLU) ? 16 * MMA_WARPS : 16 * MMA_MT * MMA_WARPS;
  const dim3 grid((N + rows_per_cta - 1) / rows_per_cta, phase == 0 ? 1 : ksplit, L.E);
  const int z = phase == 0 ? 1 : ksplit;
  switch (pick_nt(T)) {
    case 1: ffn_mma_kernel<1><<<grid, MMA_THREADS, 0, st>>>(phase, L, experts, in, off, hidden, o_part, z, n_pairs); break;
    case 2: ffn_mma_kernel<2><<<grid, MMA_THREADS, 0, st>>>(phase, L, experts, in, off, hidden, o_part, z, n_pairs); break;
    default: ffn_mma_kernel<4><<<grid, MMA_THREADS, 0, st>>>(phase, L, experts, in, off, hidden, o_part, z, n_pairs); break;
  }
  return cudaGetLastError();
}

}  // namespace emoe
