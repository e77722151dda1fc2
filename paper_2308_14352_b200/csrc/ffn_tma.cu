// Grouped expert FFN on packed weights: TMA-staged weight stream + tensor-core multiply-adds,
// for bf16 activations in the decode regime.  Paper Sections 1/2.1 (each activated expert is an
// independent FFN) on the Section 3.2 storage (b-bit codes + scale channel, w~ = q * s formed
// in registers).
//
// Same shape of arithmetic as ffn_mma.cu (codes as exact small integers in the A operand of
// mma.m16n8k16, tokens as the N dimension, fp32 accumulation per 128-input segment, then
// total += scale * segment), with two differences.  The operands are fp16: the codes are read
// as offset codes c + q with one logic instruction per pair and the constant is taken out
// again per segment (ffn_tile.cuh), and the activations (bf16 values) travel as fp16, exact
// inside the fp16 range and saturated outside.  And the bytes travel differently: the kernel is
// bound by streaming packed weights from HBM, so the bytes in flight must not depend on registers:
//   * the kernel is persistent and runs BOTH projections of a layer: a CTA pulls work items
//     (activated expert, block of output rows[, split-K slice]) from a device-side counter, the
//     first projection's items before the second's, most expensive bitwidth first, and its
//     producer warp runs ahead across item boundaries, so the weight stream never drains
//     between tiles; an item of the second projection waits until the consumers of the first
//     have counted the expert's hidden vectors complete (release / acquire on a counter in
//     the expert's plan record);
//   * the producer keeps a ring of STAGES shared-memory stages full.  One stage holds two
//     64-row x 128-byte boxes of packed codes, fetched by two TMA tensor copies (128-byte
//     swizzle, so that the consumers' 128-bit reads are conflict free), the matching slice of
//     the expert's activations, fetched by one bulk copy per token row, and a small record
//     that tells the consumers which item and which inputs the stage belongs to;
//   * the producer's lanes also start small asynchronous copies (cp.async) of the stage's
//     scales (128 rows x up to 4 segments, 16 bytes per row) that complete on the same
//     mbarrier, so that no warp ever waits on a global load of a scale;
//   * four consumer warps wait on the stage's mbarrier, read their 16-row tiles from shared
//     memory, unpack step by step, issue the MMAs, and hand the stage back through a second
//     mbarrier.
// 128 bytes of a row are 128 / 256 / 512 inputs at 8 / 4 / 2 bits, so a stage covers 1 / 2 / 4
// scale segments.  Every wait is bounded: a wait that runs out sets a bit in the context's
// check word and the CTA winds down without touching the stage.
#include <cuda.h>

#include "common.cuh"
#include "ffn_tile.cuh"
#include "pipe.cuh"

namespace emoe {
namespace {

// Consumer warps of a CTA: four, each with two 16-row tiles of a stage's 128 rows; or (SPLIT) eight,
// one tile each, in CTAs that are fewer per SM but bring more consumer warps to it in all: the
// consumers are bound by the latency of their own instruction stream, which more warps hide.
__host__ __device__ constexpr int consumer_warps(bool split) { return split ? 8 : 4; }
__host__ __device__ constexpr int tma_threads(bool split) { return (consumer_warps(split) + 1) * 32; }  // + the producer warp
#ifndef EMOE_TMA_SPLIT_NT1
#define EMOE_TMA_SPLIT_NT1 0  // 1: 8-token tiles take the eight-warp variant (as measured: slower, see consumer_warps)
#endif
#ifndef EMOE_TMA_SPLIT_STAGES
#define EMOE_TMA_SPLIT_STAGES 4
#endif
#ifndef EMOE_TMA_SPLIT_CTAS
#define EMOE_TMA_SPLIT_CTAS 2
#endif
constexpr int TMA_SCALE_BYTES = 128 * 16;                   // raw scales of a stage: 16 bytes per row
constexpr int TMA_BOX_ROWS = 64;
constexpr int TMA_BOX_BYTES = TMA_BOX_ROWS * 128;  // 8 KB
constexpr int TMA_XROW_MAX = 512 * 2 + 64;         // bytes per token row of a stage (row stride = 64 mod 128)
#ifndef EMOE_TMA_STAGES_NT1
#define EMOE_TMA_STAGES_NT1 2
#endif
#ifndef EMOE_TMA_UNROLL_SEGS
#define EMOE_TMA_UNROLL_SEGS 0
#endif
#ifndef EMOE_TMA_L2PROMO
#define EMOE_TMA_L2PROMO CU_TENSOR_MAP_L2_PROMOTION_L2_256B
#endif
#ifndef EMOE_TMA_CTAS_NT1
#define EMOE_TMA_CTAS_NT1 3
#endif

// MMA row g of a 16-row tile -> row of the shared-memory box, chosen per bitwidth so that the
// lanes of one shared-memory transaction fall into different 16-byte columns after the swizzle.
template <int BITS>
__device__ __forceinline__ int box_row_of(int g) {
  if (BITS == 8) return g;
  if (BITS == 4) return ((g & 1) << 2) | (g >> 1);
  return ((g & 3) << 1) | (g >> 2);
}

// the lane's raw codes of one row for segment `sg` of the stage: `row` points at the row's 128
// bytes inside a swizzled box, `swz` is the row's swizzle term (row index mod 8)
template <int BITS>
__device__ __forceinline__ Raw<BITS> lds_raw(const unsigned char* row, int swz, int sg, int t);
template <>
__device__ __forceinline__ Raw<8> lds_raw<8>(const unsigned char* row, int swz, int sg, int t) {
  (void)sg;
  Raw<8> r;
  r.v[0] = *reinterpret_cast<const uint4*>(row + (((2 * t) ^ swz) << 4));
  r.v[1] = *reinterpret_cast<const uint4*>(row + (((2 * t + 1) ^ swz) << 4));
  return r;
}
template <>
__device__ __forceinline__ Raw<4> lds_raw<4>(const unsigned char* row, int swz, int sg, int t) {
  Raw<4> r;
  r.v[0] = *reinterpret_cast<const uint4*>(row + (((4 * sg + t) ^ swz) << 4));
  return r;
}
template <>
__device__ __forceinline__ Raw<2> lds_raw<2>(const unsigned char* row, int swz, int sg, int t) {
  Raw<2> r;
  r.v[0] = *reinterpret_cast<const uint2*>(row + (((2 * sg + (t >> 1)) ^ swz) << 4) + ((t & 1) << 3));
  return r;
}

// a stage = two weight boxes + the activation tile, padded so that every stage (and with it
// every swizzled box) starts on a 1024-byte boundary
__host__ __device__ constexpr int stage_bytes_for(int nt) {
  return 2 * TMA_BOX_BYTES + (nt * 8 * TMA_XROW_MAX + TMA_SCALE_BYTES + 1023) / 1024 * 1024;
}
__host__ __device__ constexpr int scale_tile_offset(int nt) { return 2 * TMA_BOX_BYTES + nt * 8 * TMA_XROW_MAX; }

// The scales a stage needs from row n (groups of inputs k0 .. k0 + 128*segs) sit in one short
// byte window of the scale channel; it is copied from the 4-byte boundary at or below its start.
// group index of input k (groups of G inputs, G a multiple of 128 or the whole row);
// gshift = log2(G) when G is a power of two, else -1
__device__ __forceinline__ int group_of(int k, int gshift, int G, int ngroups) {
  return ngroups == 1 ? 0 : (gshift >= 0 ? (k >> gshift) : k / G);
}

struct TmaArgs {
  int phase_begin, phase_end;  // projections this launch runs: [0,1), [1,2) or both, [0,2)
  LayerDims L;
  const ExpertDev* experts;
  const CUtensorMap* tmaps;  // [E][3]
  const __half* xs;          // input of the first projection (tokens in expert order, fp16)
  const int32_t* off;
  int* plan;  // header {activated experts, item counters} + one PlanRec per activated expert
  __half* hidden;         // output of the first projection, input of the second (bf16 values as fp16)
  float* o_part;
  int ksplit;         // split-K slices of the second projection
  int row_blocks[2];  // row blocks of an expert per projection
  int ngroups[2];     // scale groups per row, per projection
  int gshift;         // log2(group size) if it is a power of two, else -1
  int n_pairs;
  int* check_word;
  // floor(2^32 / d) + 1 for the divisors of the item index, per projection: n / d = umulhi(n, magic) for the
  // small n and d met here (n * d < 2^32), instead of an integer division in front of every item's first copy
  uint32_t mg_units[2], mg_ksplit[2], mg_rb[2];
};

__host__ __device__ inline uint32_t div_magic(uint32_t d) { return d <= 1 ? 0u : static_cast<uint32_t>((1ull << 32) / d) + 1u; }
__device__ __forceinline__ int fast_div(int n, int d, uint32_t magic) { return d <= 1 ? n : static_cast<int>(__umulhi(static_cast<uint32_t>(n), magic)); }

// what differs between the two projections
struct PhaseDims {
  int K, N, rows_per_item, row_blocks, ksplit, mat_first;
  bool swiglu_in;
  uint32_t mg_units, mg_ksplit, mg_rb;
};
__device__ __forceinline__ PhaseDims phase_dims(const TmaArgs& a, int phase) {
  PhaseDims d;
  d.K = phase == 0 ? a.L.d_model : a.L.d_ff;
  d.N = phase == 0 ? a.L.d_ff : a.L.d_model;
  d.swiglu_in = phase == 0 && a.L.act == EMOE_ACT_SWIGLU;
  d.rows_per_item = d.swiglu_in ? TMA_BOX_ROWS : 2 * TMA_BOX_ROWS;
  d.row_blocks = a.row_blocks[phase];
  d.ksplit = phase == 0 ? 1 : a.ksplit;
  d.mat_first = phase == 0 ? 0 : (a.L.act == EMOE_ACT_SWIGLU ? 2 : 1);
  d.mg_units = a.mg_units[phase];
  d.mg_ksplit = a.mg_ksplit[phase];
  d.mg_rb = a.mg_rb[phase];
  return d;
}

// what a stage holds, written by the producer before it arms the stage's barrier
struct StageMeta {
  int e, rb, z, begin, p0, ntok, k0, bits;
  int flags;  // 1 = first stage of an item pass, 2 = last, 4 = no more work, 8 = stage carries no inputs,
              // 16 = last stage of a first-projection item whose completion the second projection waits for
  int phase;
  int ai;  // index of the expert's plan record
  int pad;
};
constexpr int META_FIRST = 1, META_LAST = 2, META_STOP = 4, META_EMPTY = 8, META_DONE = 16;

// How long the second projection of an expert waits for its hidden vectors (polls of ~0.1 us).
constexpr unsigned DEP_WAIT_LIMIT = 1u << 20;

template <int BITS, int NT, bool SPLIT>
__device__ __forceinline__ void consume_stage(const TmaArgs& a, int phase, int rb, int k0, int ntok,
                                              const unsigned char* st, int warp_full, int lane, uint32_t bar_empty,
                                              float (&tot)[2][NT][4]) {
  // SPLIT: warps 2p and 2p+1 share the 32 rows (or the w1 / w3 tiles) that warp p owns otherwise
  const int warp = SPLIT ? warp_full >> 1 : warp_full;
  const int mt_own = warp_full & 1;
  constexpr int KSPAN = 1024 / BITS;  // inputs per stage (128 bytes of a row)
  constexpr int SEGS = KSPAN / 128;   // scale segments per stage
  // one token tile: offset codes (fewest instructions per code); more: exact codes (no MMAs for
  // the constants, which would have to be repeated per token tile)
  constexpr bool OFFSET_CODES = NT == 1 && BITS != 8;
  const LayerDims& L = a.L;
  const int K = phase == 0 ? L.d_model : L.d_ff;
  const bool swiglu_in = phase == 0 && L.act == EMOE_ACT_SWIGLU;
  const int g = lane >> 2, t = lane & 3;
  const int gp = box_row_of<BITS>(g);
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const int ngroups = a.ngroups[phase];
  const int ssz = L.scale_f16 ? 2 : 4;
  const int nseg = min(SEGS, (K - k0) / 128);
  const int g0 = group_of(k0, a.gshift, L.group, ngroups);
  // Everything that does not depend on the segment, once per stage.  The lane's four rows (2
  // tiles x rows gp, gp+8) sit at fixed distances from the first one, in the boxes (128 bytes
  // per row) and in the scale tile (16 bytes per row): tile 1 is the other box (gated
  // projection) or 16 rows further down, rows gp+8 are 8 rows further down.  A row's scale
  // window starts at the 4-byte boundary at or below its first scale of the stage; the rows of a
  // lane are an even number of rows apart, so the distance to that boundary is the same for all.
  const int swz = gp & 7;  // swizzle term of all four rows (they differ by multiples of 8)
  const int box_first = swiglu_in ? 0 : (warp >> 1);
  const int r_first = (swiglu_in ? 16 * warp : 32 * (warp & 1)) + gp;
  const int nrow = (swiglu_in ? rb * TMA_BOX_ROWS + 16 * warp : rb * 2 * TMA_BOX_ROWS + 32 * warp) + gp;
  const int dmt = swiglu_in ? TMA_BOX_BYTES : 16 * 128;
  const unsigned char* row_base = st + box_first * TMA_BOX_BYTES + r_first * 128;
  const unsigned char* sc_base = st + scale_tile_offset(NT) + (box_first * TMA_BOX_ROWS + r_first) * 16 +
                                 (((min(nrow, N - 1) * ngroups + g0) * ssz) & 3);
  const unsigned char* xlane = st + 2 * TMA_BOX_BYTES + g * TMA_XROW_MAX + t * 16;
#if EMOE_TMA_UNROLL_SEGS
#pragma unroll
#else
#pragma unroll 1
#endif
  for (int sg = 0; sg < SEGS; ++sg) {
    if (sg < nseg) {
      // B fragments: piece q of lane t sits at (q*4 + t) * 16 bytes of the segment
      uint4 bq[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        if (nt * 8 < ntok) {
          const unsigned char* src = xlane + nt * 8 * TMA_XROW_MAX + sg * 256;
#pragma unroll
          for (int q = 0; q < 4; ++q) bq[nt][q] = *reinterpret_cast<const uint4*>(src + q * 64);
        }
      }
      // - sum_k c_k x_k of the segment (see ffn_tile.cuh): the same for every output channel, so
      // one pair of MMAs per step, with the constants as A operand, serves both 16-row tiles
      float osum[NT][2];  // per token (2t, 2t+1)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float da[4] = {0.0f, 0.0f, 0.0f, 0.0f}, db[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (OFFSET_CODES && nt * 8 < ntok) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            mma_f16(da, offset_const<BITS>(0), offset_const<BITS>(0), offset_const<BITS>(1), offset_const<BITS>(1),
                    bq[nt][q].x, bq[nt][q].y);
            mma_f16(db, offset_const<BITS>(2), offset_const<BITS>(2), offset_const<BITS>(3), offset_const<BITS>(3),
                    bq[nt][q].z, bq[nt][q].w);
          }
        }
        osum[nt][0] = -(da[0] + db[0]);
        osum[nt][1] = -(da[1] + db[1]);
      }
      const int sdelta = (group_of(k0 + sg * 128, a.gshift, L.group, ngroups) - g0) * ssz;
      // one 16-row tile at a time, one k16-pair step at a time: the codes of a step live in 8
      // registers and go straight into the MMAs.  The k-steps alternate between two partial
      // accumulators so that consecutive MMAs do not depend on each other; the first starts from
      // the constant's share.
#pragma unroll
      for (int mi = 0; mi < (SPLIT ? 1 : 2); ++mi) {
        const int mt = SPLIT ? mt_own : mi;  // which tile; its totals live in tot[mi]
        const Raw<BITS> raw0 = lds_raw<BITS>(row_base + mt * dmt, swz, sg, t);
        const Raw<BITS> raw1 = lds_raw<BITS>(row_base + mt * dmt + 8 * 128, swz, sg, t);
        const unsigned char* sc = sc_base + mt * (dmt >> 3) + sdelta;
        float s0, s1;
        if (ssz == 2) {
          s0 = __half2float(*reinterpret_cast<const __half*>(sc));
          s1 = __half2float(*reinterpret_cast<const __half*>(sc + 8 * 16));
        } else {
          s0 = *reinterpret_cast<const float*>(sc);
          s1 = *reinterpret_cast<const float*>(sc + 8 * 16);
        }
        float pa[NT][4], pb[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          pa[nt][0] = pa[nt][2] = osum[nt][0];
          pa[nt][1] = pa[nt][3] = osum[nt][1];
#pragma unroll
          for (int i = 0; i < 4; ++i) pb[nt][i] = 0.0f;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t c0[4], c1[4];
          if (OFFSET_CODES) {
            unpack_step_off(raw0, q, c0);
            unpack_step_off(raw1, q, c1);
          } else {
            unpack_step_exact(raw0, q, c0);
            unpack_step_exact(raw1, q, c1);
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            if (nt * 8 < ntok) {
              mma_f16(pa[nt], c0[0], c1[0], c0[1], c1[1], bq[nt][q].x, bq[nt][q].y);
              mma_f16(pb[nt], c0[2], c1[2], c0[3], c1[3], bq[nt][q].z, bq[nt][q].w);
            }
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          tot[mi][nt][0] = fmaf(s0, pa[nt][0] + pb[nt][0], tot[mi][nt][0]);
          tot[mi][nt][1] = fmaf(s0, pa[nt][1] + pb[nt][1], tot[mi][nt][1]);
          tot[mi][nt][2] = fmaf(s1, pa[nt][2] + pb[nt][2], tot[mi][nt][2]);
          tot[mi][nt][3] = fmaf(s1, pa[nt][3] + pb[nt][3], tot[mi][nt][3]);
        }
      }
    }
  }
  // shared memory of the stage is no longer needed
  __syncwarp();
  if (lane == 0) mbar_arrive(bar_empty);
}

// This warp's share of an expert's hidden vectors is written: make it visible to the bulk copies
// of other SMs (release), then count it.
__device__ __forceinline__ void count_item_done(PlanRec* recs, int ai, int lane) {
  // the hidden values live in global memory: the fence restricted to that space costs some 40 cycles where the
  // unrestricted one (which also settles the shared-memory side) was measured at 800 to 1300
  asm volatile("fence.proxy.async.global;" ::: "memory");
  __syncwarp();
  if (lane == 0)  // release: the hidden values this warp stored are visible before the count is
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(&recs[ai].done), "r"(1) : "memory");
}

// the hidden vector is rounded to bf16 (the layer's activation type), then carried as fp16;
// the same without the report: a saturated value is recognised afterwards by its bit pattern (+-65504 is
// not a bf16 number, so a hidden value can only be there by saturation), for the positions that are stored
__device__ __forceinline__ __half hidden_half(float h) { return f32_to_f16_sat(__bfloat162float(__float2bfloat16_rn(h))); }
__device__ __forceinline__ bool half_saturated(__half v) { return (__half_as_ushort(v) & 0x7fffu) == 0x7bffu; }

// results of one item pass: lane holds rows (gp, gp+8) x tokens (2t, 2t+1) of every tile.
// SPLIT: a warp holds one tile (tot[0]); in a gated first projection the warp with the w3 tile
// hands its totals to the warp with the w1 tile of the same rows through shared memory (xch, one
// slot per warp pair, guarded by a full / free pair of barriers with bounded waits).
template <int BITS, int NT, bool SPLIT>
__device__ __forceinline__ bool store_item(const TmaArgs& a, const StageMeta& m, int warp_full, int lane,
                                           float (&tot)[2][NT][4], float* xch, uint32_t bar_x, int& n_exchanged,
                                           volatile int* abort_flag) {
  const LayerDims& L = a.L;
  const int N = m.phase == 0 ? L.d_ff : L.d_model;
  const bool swiglu_in = m.phase == 0 && L.act == EMOE_ACT_SWIGLU;
  const int warp = SPLIT ? warp_full >> 1 : warp_full;
  const int mt_own = warp_full & 1;
  const int g = lane >> 2, t = lane & 3;
  const int gp = box_row_of<BITS>(g);
  if (SPLIT && swiglu_in) {
    float* slot = xch + warp * (NT * 4 * 32);
    const uint32_t full = bar_x + 8 * (2 * warp), free_ = bar_x + 8 * (2 * warp + 1);
    const uint32_t par = n_exchanged & 1;
    ++n_exchanged;
    if (mt_own == 1) {  // the w3 tile: hand over, nothing to store
      if (!mbar_wait(free_, par ^ 1, a.check_word, abort_flag)) return false;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) slot[(nt * 4 + i) * 32 + lane] = tot[0][nt][i];
      __syncwarp();
      if (lane == 0) mbar_arrive(full);
      return true;
    }
    if (!mbar_wait(full, par, a.check_word, abort_flag)) return false;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) tot[1][nt][i] = slot[(nt * 4 + i) * 32 + lane];
    __syncwarp();
    if (lane == 0) mbar_arrive(free_);
  }
  // Values first, for all positions at once (independent instruction streams), then the stores under
  // their predicates: a position-by-position loop with early exits ran as one long dependent chain.
  bool beyond = false;
  if (swiglu_in) {
    __half hv[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float av = tot[0][nt][i], bv = tot[1][nt][i];
        hv[nt][i] = hidden_half(av / (1.0f + expf(-av)) * bv);
      }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tok = nt * 8 + 2 * t + (i & 1);
        const int n = m.rb * TMA_BOX_ROWS + 16 * warp + gp + 8 * (i >> 1);
        if (tok < m.ntok && n < N) {
          a.hidden[static_cast<size_t>(m.begin + m.p0 + tok) * N + act_pos<BITS>(n)] = hv[nt][i];
          beyond |= half_saturated(hv[nt][i]);
        }
      }
  } else if (m.phase == 0) {
    __half hv[2][NT][4];
#pragma unroll
    for (int mi = 0; mi < (SPLIT ? 1 : 2); ++mi)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) hv[mi][nt][i] = hidden_half(fmaxf(tot[mi][nt][i], 0.0f));
#pragma unroll
    for (int mi = 0; mi < (SPLIT ? 1 : 2); ++mi)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int mt = SPLIT ? mt_own : mi;
          const int tok = nt * 8 + 2 * t + (i & 1);
          const int n = m.rb * 2 * TMA_BOX_ROWS + 32 * warp + 16 * mt + gp + 8 * (i >> 1);
          if (tok < m.ntok && n < N) {
            a.hidden[static_cast<size_t>(m.begin + m.p0 + tok) * N + act_pos<BITS>(n)] = hv[mi][nt][i];
            beyond |= half_saturated(hv[mi][nt][i]);
          }
        }
  } else {
    float* plane = a.o_part + static_cast<size_t>(m.z) * a.n_pairs * N;
#pragma unroll
    for (int mi = 0; mi < (SPLIT ? 1 : 2); ++mi)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int mt = SPLIT ? mt_own : mi;
          const int tok = nt * 8 + 2 * t + (i & 1);
          const int n = m.rb * 2 * TMA_BOX_ROWS + 32 * warp + 16 * mt + gp + 8 * (i >> 1);
          if (tok < m.ntok && n < N) plane[static_cast<size_t>(m.begin + m.p0 + tok) * N + n] = tot[mi][nt][i];
        }
  }
  if (beyond) atomicOr(a.check_word, CHECK_F16_RANGE);  // saturated above: reported, not silent
  return true;
}

// ring depth and CTAs per SM by token-tile count: more, smaller CTAs when registers allow, so
// that every scheduler has several consumer warps to switch between
template <int NT, bool SPLIT>
__host__ __device__ constexpr int stages_for() { return SPLIT ? EMOE_TMA_SPLIT_STAGES : (NT == 1 ? EMOE_TMA_STAGES_NT1 : 3); }
template <int NT, bool SPLIT>
__host__ __device__ constexpr int ctas_per_sm_for() { return SPLIT ? EMOE_TMA_SPLIT_CTAS : (NT == 1 ? EMOE_TMA_CTAS_NT1 : (NT == 2 ? 2 : 1)); }

template <int NT, bool SPLIT>
__host__ __device__ constexpr int smem_bytes_for() {
  return stages_for<NT, SPLIT>() * stage_bytes_for(NT) + 1024;  // + slack to align the base to 1024
}

template <int NT, bool SPLIT>
__global__ void __launch_bounds__(tma_threads(SPLIT), ctas_per_sm_for<NT, SPLIT>()) ffn_tma_kernel(const __grid_constant__ TmaArgs a) {
  constexpr int TMA_CONSUMER_WARPS = consumer_warps(SPLIT);
  constexpr int STAGES = stages_for<NT, SPLIT>();
  constexpr int STAGE_BYTES = stage_bytes_for(NT);
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 8];  // full, empty; SPLIT: (full, free) per warp pair of the w3 -> w1 hand-over
  __shared__ __align__(16) StageMeta meta[STAGES];
  __shared__ float xch[SPLIT ? 4 * NT * 4 * 32 : 1];
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    abort_word = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(bars + s), 33);  // full: lane 0's arrival (+ bulk-copy bytes) and every lane's scale copies
      mbar_init(smem_u32(bars + STAGES + s), TMA_CONSUMER_WARPS);  // empty: one arrival per consumer warp
    }
    for (int i = 0; i < 8; ++i) mbar_init(smem_u32(bars + 2 * STAGES + i), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Token rows of a stage that no copy fills keep whatever shared memory held.  That is
  // harmless: a column of the MMA result depends only on its own column of B, and columns past
  // the expert's token count are never stored.
  __syncthreads();
  // Everything above overlaps the tail of the kernel in front.  A launch that starts with the
  // first projection needs that kernel's results (the plan) at once; a launch of the second
  // projection alone finds plan, weights and scales older than the kernel in front, so its
  // producer starts fetching them and waits only before the first copy of a hidden vector (see
  // `waited` below).
  if (warp == TMA_CONSUMER_WARPS) {
    // The tensor maps are older than every kernel of the chain: pull them towards L2 now, so that
    // the first copy of an expert's matrix does not wait for its descriptor to come from HBM.
    const int n_maps = 3 * a.L.E;
    const int i = (static_cast<int>(blockIdx.x) * 32 + lane) % ((n_maps + 31) / 32 * 32);
    if (i < n_maps) asm volatile("prefetch.global.L2 [%0];" ::"l"(a.tmaps + i));
  }
  if (a.phase_begin == 0) pdl_wait();
  pdl_trigger();

  const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + STAGES);
  const LayerDims& L = a.L;
  PlanRec* recs = reinterpret_cast<PlanRec*>(reinterpret_cast<char*>(a.plan) + PLAN_HEADER_BYTES);
  // both projections in this launch: an item of the second projection waits until the expert's
  // hidden vectors are complete (PlanRec::done, raised by the consumers of the first projection)
  const bool fused = a.phase_begin == 0 && a.phase_end == 2;

  if (warp == TMA_CONSUMER_WARPS) {
    // ---------------- producer warp ----------------
    // the record the CTA's first item most likely needs, requested together with the header
    const int ai_guess = min(static_cast<int>(blockIdx.x) / (a.phase_begin == 0 ? a.row_blocks[0] : a.row_blocks[1] * a.ksplit),
                             L.E - 1);
    const PlanRec rec_guess = recs[ai_guess];
    const int n_active = *reinterpret_cast<volatile const int*>(a.plan);
    // items: the first projection's (expert, row block), then the second's (expert, row block,
    // split-K slice), each list expert-major in plan order
    const int n_items0 = a.phase_begin == 0 ? n_active * a.row_blocks[0] : 0;
    const int n_items1 = a.phase_end == 2 ? n_active * a.row_blocks[1] * a.ksplit : 0;
    const int n_items = n_items0 + n_items1;
    const int ssz = L.scale_f16 ? 2 : 4;
    int it = 0;
    bool ok = true;
    bool waited = a.phase_begin == 0;  // false: copies of activation rows are parked until pdl_wait()
    int n_parked = 0;
    int park_stage[STAGES], park_row[STAGES], park_k0[STAGES], park_klen[STAGES], park_ntok[STAGES];
    // A CTA's first item is its own index; the counter hands out the items after those.
    int item_cur = blockIdx.x, item_next = 0;
    while (ok) {
      const int item = item_cur;
      if (item >= n_items || *abort_flag) break;
      const int phase = item < n_items0 ? 0 : 1;
      const int li = item - (phase == 0 ? 0 : n_items0);
      const PhaseDims pd = phase_dims(a, phase);
      const int K = pd.K;
      const bool swiglu_in = pd.swiglu_in;
      const int mat_first = pd.mat_first;
      const int ngroups_k = a.ngroups[phase];
      const int ai = fast_div(li, pd.ksplit * pd.row_blocks, pd.mg_units);
      const PlanRec rec = (it == 0 && ai == ai_guess) ? rec_guess : recs[ai];
      const __half* in = phase == 0 ? a.xs : a.hidden;
      const int lz = fast_div(li, pd.ksplit, pd.mg_ksplit);  // (expert, row block) index
      const int z = li - lz * pd.ksplit;
      const int rb = lz - fast_div(lz, pd.row_blocks, pd.mg_rb) * pd.row_blocks;
      const int e = rec.e;
      const int begin = rec.begin;
      const int cnt = rec.cnt;
      const CUtensorMap* maps = a.tmaps + static_cast<size_t>(e) * 3;
      const int bits = rec.bits;
      const int kshift = bits == 8 ? 7 : (bits == 4 ? 8 : 9);  // log2 of the inputs per stage
      const int kspan = 1 << kshift;
      const int steps_total = (K + kspan - 1) >> kshift;
      const int spz = fast_div(steps_total + pd.ksplit - 1, pd.ksplit, pd.mg_ksplit);
      const int step_begin = z * spz;
      const int nsteps = max(0, min(steps_total, step_begin + spz) - step_begin);
      const int npass = (cnt + NT * 8 - 1) / (NT * 8);
      const int row0 = rb * pd.rows_per_item;
      bool need_dep = fused && phase == 1;
      // scale rows of the item this lane copies (rows l, l+32, l+64, l+96 of a stage, box-major): start
      // of each row's scale channel as a byte offset from its 4-byte-aligned matrix base
      const char* srow_base[4];
      int srow_off[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int row = lane + 32 * r;  // neighbouring lanes take neighbouring rows: their 4-byte copies spread over the banks
        const int n = min(swiglu_in ? row0 + (row & 63) : row0 + row, pd.N - 1);
        // constant indices only: a record indexed by a variable would live in local memory
        const void* sc_first = mat_first == 0 ? rec.scales[0] : (mat_first == 1 ? rec.scales[1] : rec.scales[2]);
        srow_base[r] = static_cast<const char*>(swiglu_in ? ((row >> 6) ? rec.scales[1] : rec.scales[0]) : sc_first);
        srow_off[r] = n * ngroups_k * ssz;
      }
      for (int pass = 0; pass < npass && ok; ++pass) {
        const int p0 = pass * NT * 8;
        const int ntok = min(NT * 8, cnt - p0);
        const int nst = max(nsteps, 1);  // an empty split-K slice still has to store its zeros
        for (int s = 0; s < nst; ++s, ++it) {
          const int stage = it % STAGES;
          const uint32_t par = (it / STAGES) & 1;
          if (!mbar_wait(bar_empty + 8 * stage, par ^ 1, a.check_word, abort_flag)) {
            ok = false;
            break;
          }
          unsigned char* st = smem + stage * STAGE_BYTES;
          const uint32_t full = bar_full + 8 * stage;
          const int k0 = (step_begin + s) * kspan;
          const int klen = nsteps > 0 ? min(kspan, K - k0) : 0;
          // Lanes 30 and 31 start the two weight boxes at once; lane 0 writes the record and announces
          // the bytes.  The order among them is free: the stage cannot complete before all 33
          // arrivals are in, and the byte count may run ahead of its announcement.
          if (klen > 0 && lane >= 30) {
            const int c0 = k0 * bits / 8;
            const int bx = lane - 30;
            if (swiglu_in) tma_load_2d(smem_u32(st + bx * TMA_BOX_BYTES), maps + bx, c0, row0, full);
            else tma_load_2d(smem_u32(st + bx * TMA_BOX_BYTES), maps + mat_first, c0, row0 + bx * TMA_BOX_ROWS, full);
          }
          if (lane == 0) {
            const int flags = (s == 0 ? META_FIRST : 0) | (s == nst - 1 ? META_LAST : 0) | (klen == 0 ? META_EMPTY : 0) |
                              (fused && phase == 0 && s == nst - 1 && pass == npass - 1 ? META_DONE : 0);
            // the record as three 16-byte stores (field order of StageMeta)
            uint4* mq = reinterpret_cast<uint4*>(&meta[stage]);
            mq[0] = make_uint4(e, rb, z, begin);
            mq[1] = make_uint4(p0, ntok, k0, bits);
            mq[2] = make_uint4(flags, phase, ai, 0);
            if (klen > 0) mbar_expect_tx(full, 2 * TMA_BOX_BYTES + ntok * klen * 2);
            else mbar_arrive(full);
          }
          __syncwarp();
          if (klen > 0) {
            // scales: lane l copies the windows of rows l, l+32, l+64, l+96 of the stage (box-major)
            const int nseg = klen / 128;
            const int g0 = group_of(k0, a.gshift, L.group, ngroups_k),
                      g1 = group_of(k0 + (nseg - 1) * 128, a.gshift, L.group, ngroups_k);
            const uint32_t sdst = smem_u32(st + scale_tile_offset(NT));
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              const int b0 = (srow_off[r] + g0 * ssz) & ~3;
              const int b1 = srow_off[r] + (g1 + 1) * ssz;
#pragma unroll 1
              for (int w = 0; b0 + 4 * w < b1; ++w)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sdst + (lane + 32 * r) * 16 + 4 * w),
                             "l"(srow_base[r] + b0 + 4 * w)
                             : "memory");
            }
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(full) : "memory");
            if (need_dep) {
              // The codes and scales of the stage are on their way; the hidden vectors may still be
              // in the making on other SMs.  Every lane acquires the counter itself, so that its
              // own copies below are ordered behind the writers' stores.
              need_dep = false;
              // every consumer warp that stores hidden values counts once per item (SPLIT, gated layer: the
              // warps with the w1 tiles only)
              const int expect = a.row_blocks[0] * ((SPLIT && L.act == EMOE_ACT_SWIGLU) ? 4 : TMA_CONSUMER_WARPS);
              const int* done = &recs[ai].done;
              bool ready = false;
              for (unsigned i = 0; i < DEP_WAIT_LIMIT; ++i) {
                int v;
                asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(done) : "memory");
                ready = __all_sync(0xffffffffu, v >= expect);
                if (ready || *abort_flag) break;
                __nanosleep(100);
              }
              if (!ready) {
                if (lane == 0) {
                  *abort_flag = 1;
                  atomicOr(a.check_word, CHECK_WAIT_TIMEOUT);
                }
                ok = false;
                break;
              }
              asm volatile("fence.proxy.async.global;" ::: "memory");  // generic-proxy stores (global memory) -> bulk-copy reads
            }
            if (waited) {
              for (int r = lane; r < ntok; r += 32)
                bulk_load(smem_u32(st + 2 * TMA_BOX_BYTES + r * TMA_XROW_MAX),
                          in + static_cast<size_t>(begin + p0 + r) * K + k0, klen * 2, full);
            } else {
              park_stage[n_parked] = stage;
              park_row[n_parked] = begin + p0;
              park_k0[n_parked] = k0;
              park_klen[n_parked] = klen;
              park_ntok[n_parked] = ntok;
              ++n_parked;
            }
          } else {
            mbar_arrive(full);  // with lane 0's arrival above: 33 in all
          }
          if (!waited && n_parked == STAGES) {  // the ring is full: nothing more can be fetched early
            pdl_wait();
            waited = true;
            for (int i = 0; i < n_parked; ++i)
              for (int r = lane; r < park_ntok[i]; r += 32)
                bulk_load(smem_u32(smem + park_stage[i] * STAGE_BYTES + 2 * TMA_BOX_BYTES + r * TMA_XROW_MAX),
                          a.hidden + static_cast<size_t>(park_row[i] + r) * K + park_k0[i], park_klen[i] * 2,
                          bar_full + 8 * park_stage[i]);
            n_parked = 0;
          }
        }
      }
      // the ring still holds several stages of work for the consumers: fetching the next item
      // only now costs them nothing and no CTA sits on items it is not yet working on
      if (lane == 0) item_next = gridDim.x + atomicAdd(a.plan + 1 + a.phase_begin, 1);
      item_cur = __shfl_sync(0xffffffffu, item_next, 0);
      if (item_cur < n_items) {
        // pull the next item's scale rows towards L2 while its codes are still far away
        const int phn = item_cur < n_items0 ? 0 : 1;
        const int lin = item_cur - (phn == 0 ? 0 : n_items0);
        const PhaseDims pn = phase_dims(a, phn);
        const PlanRec rn = recs[fast_div(lin, pn.ksplit * pn.row_blocks, pn.mg_units)];
        const int lzn = fast_div(lin, pn.ksplit, pn.mg_ksplit);
        const int rbn = lzn - fast_div(lzn, pn.row_blocks, pn.mg_rb) * pn.row_blocks;
        const int ngroups = a.ngroups[phn];
        const int rows = min(pn.rows_per_item, pn.N - rbn * pn.rows_per_item);
        const int lines = (rows * ngroups * ssz + 127) / 128;
        const size_t offs = static_cast<size_t>(rbn) * pn.rows_per_item * ngroups * ssz;
        const int nm = pn.swiglu_in ? 2 : 1;
        for (int i = lane; i < nm * lines; i += 32) {
          const int second = i >= lines ? 1 : 0;  // nm is 1 or 2: no division needed
          const char* base = static_cast<const char*>(pn.swiglu_in ? (second ? rn.scales[1] : rn.scales[0]) : (pn.mat_first == 0 ? rn.scales[0] : (pn.mat_first == 1 ? rn.scales[1] : rn.scales[2]))) + offs;
          asm volatile("prefetch.global.L2 [%0];" ::"l"(base + static_cast<size_t>(i - second * lines) * 128));
        }
      }
    }
    if (!waited) {  // fewer stages than the ring holds: release the parked copies now
      pdl_wait();
      waited = true;
      for (int i = 0; i < n_parked; ++i)
        for (int r = lane; r < park_ntok[i]; r += 32)
          bulk_load(smem_u32(smem + park_stage[i] * STAGE_BYTES + 2 * TMA_BOX_BYTES + r * TMA_XROW_MAX),
                    a.hidden + static_cast<size_t>(park_row[i] + r) * L.d_ff + park_k0[i], park_klen[i] * 2,
                    bar_full + 8 * park_stage[i]);
      n_parked = 0;
    }
    if (ok && !*abort_flag) {  // tell the consumers that nothing else comes
      const int stage = it % STAGES;
      const uint32_t par = (it / STAGES) & 1;
      if (mbar_wait(bar_empty + 8 * stage, par ^ 1, a.check_word, abort_flag)) {
        if (lane == 0) {
          meta[stage].flags = META_STOP;
          mbar_arrive(bar_full + 8 * stage);  // lane 0 arrives twice: once for itself, once in place of a copy
        }
        __syncwarp();
        mbar_arrive(bar_full + 8 * stage);
      }
    }
  } else {
    // ---------------- consumer warps ----------------
    float tot[2][NT][4];
    int n_exchanged = 0;
    const uint32_t bar_x = smem_u32(bars + 2 * STAGES);
    // A finished first-projection item is counted one stage late: by then its stores have long
    // been acknowledged and the fence in front of the count costs nothing.  It is never held back
    // across a wait, because the stage waited for may be the one that waits for this count.
    int pending_ai = -1;
    for (int it = 0;; ++it) {
      const int stage = it % STAGES;
      const uint32_t par = (it / STAGES) & 1;
      if (pending_ai >= 0 && !__shfl_sync(0xffffffffu, mbar_try_wait(bar_full + 8 * stage, par) ? 1 : 0, 0)) {
        count_item_done(recs, pending_ai, lane);
        pending_ai = -1;
      }
      if (!mbar_wait(bar_full + 8 * stage, par, a.check_word, abort_flag)) break;
      const StageMeta m = meta[stage];
      if (m.flags & META_STOP) break;
      if (m.flags & META_FIRST) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) tot[mt][nt][i] = 0.0f;
      }
      const unsigned char* st = smem + stage * STAGE_BYTES;
      if (!(m.flags & META_EMPTY)) {
        switch (m.bits) {
          case 2: consume_stage<2, NT, SPLIT>(a, m.phase, m.rb, m.k0, m.ntok, st, warp, lane, bar_empty + 8 * stage, tot); break;
          case 4: consume_stage<4, NT, SPLIT>(a, m.phase, m.rb, m.k0, m.ntok, st, warp, lane, bar_empty + 8 * stage, tot); break;
          default: consume_stage<8, NT, SPLIT>(a, m.phase, m.rb, m.k0, m.ntok, st, warp, lane, bar_empty + 8 * stage, tot); break;
        }
      } else {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * stage);
      }
      if (m.flags & META_LAST) {
        bool ok;
        switch (m.bits) {
          case 2: ok = store_item<2, NT, SPLIT>(a, m, warp, lane, tot, xch, bar_x, n_exchanged, abort_flag); break;
          case 4: ok = store_item<4, NT, SPLIT>(a, m, warp, lane, tot, xch, bar_x, n_exchanged, abort_flag); break;
          default: ok = store_item<8, NT, SPLIT>(a, m, warp, lane, tot, xch, bar_x, n_exchanged, abort_flag); break;
        }
        if (!ok) break;
      }
      if (pending_ai >= 0) {
        count_item_done(recs, pending_ai, lane);
        pending_ai = -1;
      }
      // the warps that stored hidden values count the item (SPLIT, gated layer: not the w3 warps)
      if ((m.flags & META_LAST) && (m.flags & META_DONE) && !(SPLIT && a.L.act == EMOE_ACT_SWIGLU && (warp & 1))) pending_ai = m.ai;
    }
    if (pending_ai >= 0) count_item_done(recs, pending_ai, lane);
  }
  if (*abort_flag) {
    // a wait ran out: give copies that may still be in flight time to land before the CTA's
    // shared memory is released
#pragma unroll 1
    for (int i = 0; i < 2000; ++i) __nanosleep(100);
  }
}

template <int NT, bool SPLIT>
cudaError_t launch_nt(const TmaArgs& a, int max_items, cudaStream_t st) {
  constexpr int SMEM = smem_bytes_for<NT, SPLIT>();
  constexpr int TMA_THREADS = tma_threads(SPLIT);
  static int ctas_per_device[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!ctas_per_device[dev]) {
    e = cudaFuncSetAttribute(ffn_tma_kernel<NT, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return e;
    int per_sm = 0, sms = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ffn_tma_kernel<NT, SPLIT>, TMA_THREADS, SMEM);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    ctas_per_device[dev] = (per_sm > 0 ? per_sm : 1) * sms;
  }
  const int grid = max_items < ctas_per_device[dev] ? max_items : ctas_per_device[dev];
  return launch_chain(ffn_tma_kernel<NT, SPLIT>, dim3(grid), dim3(TMA_THREADS), SMEM, st, a);
}

}  // namespace

bool ffn_tma_supported(const LayerDims& L) {
  // tensor maps use 128-byte x 64-row boxes: every packed row must hold at least 128 bytes at
  // the narrowest width (2 bits)
  return ffn_mma_supported(L) && L.d_model >= 512 && L.d_ff >= 512;
}

int ffn_tma_ksplit(const LayerDims& L, int T) {
  const int row_blocks = (L.d_model + 2 * TMA_BOX_ROWS - 1) / (2 * TMA_BOX_ROWS);
  const long long pairs = static_cast<long long>(T) * L.top_k;
  const long long active = pairs < L.E ? pairs : L.E;
  const long long ctas = row_blocks * active;
  const int steps_min = (L.d_ff + 511) / 512;  // stages at the widest span (2 bits)
  // enough slices that the second projection's items outnumber the resident CTAs (3 per SM)
  // about four times: short items at the end of the launch keep its tail short (as measured: the
  // same on the Switch-base-like layer at 64 tokens as twice as many CTAs' worth, 3 % faster on
  // the Mixtral-like layer at 4 tokens; fewer slices were slower on both)
  long long z = (12 * 148 + ctas - 1) / ctas;
  // A handful of tokens leaves most SMs without an item: the slices are then cut as fine as the
  // 8-bit stages allow (narrower experts get empty slices, which only store zeros), so that the
  // second projection of the one or two activated experts is a short step on many SMs instead
  // of a chain of stages on a few (single token, Switch-base-like layer: 8 % off the launch).
  const int steps_max = (L.d_ff + 127) / 128;
  const int cap = ctas * 4 <= 148 ? steps_max : steps_min;
  if (z > cap) z = cap;
  if (z > 16) z = 16;
  if (z < 1) z = 1;
  return static_cast<int>(z);
}

cudaError_t launch_ffn_tma(int phase_begin, int phase_end, const LayerDims& L, const ExpertDev* experts,
                           const void* tmaps, const __nv_bfloat16* xs, const int32_t* off, int* plan,
                           __nv_bfloat16* hidden, float* o_part, int ksplit, int n_pairs, int T, int token_tiles,
                           int* check_word, cudaStream_t st) {
  if (phase_begin < 0 || phase_end > 2 || phase_begin >= phase_end) return cudaErrorInvalidValue;
  const int rows_first = L.act == EMOE_ACT_SWIGLU ? TMA_BOX_ROWS : 2 * TMA_BOX_ROWS;
  TmaArgs a;
  a.phase_begin = phase_begin;
  a.phase_end = phase_end;
  a.L = L;
  a.experts = experts;
  a.tmaps = static_cast<const CUtensorMap*>(tmaps);
  a.xs = reinterpret_cast<const __half*>(xs);
  a.off = off;
  a.plan = plan;
  a.hidden = reinterpret_cast<__half*>(hidden);
  a.o_part = o_part;
  a.ksplit = ksplit;
  a.row_blocks[0] = (L.d_ff + rows_first - 1) / rows_first;
  a.row_blocks[1] = (L.d_model + 2 * TMA_BOX_ROWS - 1) / (2 * TMA_BOX_ROWS);
  a.ngroups[0] = L.group > 0 ? L.d_model / L.group : 1;
  a.ngroups[1] = L.group > 0 ? L.d_ff / L.group : 1;
  a.gshift = -1;
  for (int b = 7; b < 31; ++b)
    if (L.group == (1 << b)) a.gshift = b;
  a.n_pairs = n_pairs;
  a.check_word = check_word;
  for (int p = 0; p < 2; ++p) {
    const int ks = p == 0 ? 1 : ksplit;
    a.mg_units[p] = div_magic(static_cast<uint32_t>(ks * a.row_blocks[p]));
    a.mg_ksplit[p] = div_magic(static_cast<uint32_t>(ks));
    a.mg_rb[p] = div_magic(static_cast<uint32_t>(a.row_blocks[p]));
  }
  const long long active_max = n_pairs < L.E ? n_pairs : L.E;
  long long per_expert = 0;
  if (phase_begin == 0) per_expert += a.row_blocks[0];
  if (phase_end == 2) per_expert += static_cast<long long>(a.row_blocks[1]) * ksplit;
  const long long items = active_max * per_expert;
  const int max_items = items > (1 << 30) ? (1 << 30) : static_cast<int>(items);
  const int nt = token_tiles > 0 ? token_tiles : ffn_token_tiles(L, T);
  if (nt == 1) return launch_nt<1, EMOE_TMA_SPLIT_NT1 != 0>(a, max_items, st);
  if (nt == 2) return launch_nt<2, false>(a, max_items, st);
  return launch_nt<4, false>(a, max_items, st);
}

// Host-side tensor-map encoder (driver entry point looked up once; no link against libcuda).
// dtype: 0 = bytes, 1 = fp16.  2-D row-major image [outer][inner], box [box_outer][box_inner],
// 128-byte swizzle (box_inner * element size must be 128 bytes or less).
int encode_tmap_2d(void* out_map, int dtype, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride_bytes,
                   uint32_t box_inner, uint32_t box_outer, bool swizzle128) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p) return -1;
    fn = reinterpret_cast<EncodeFn>(p);
  }
  if (row_stride_bytes % 16 != 0 || (reinterpret_cast<uintptr_t>(base) & 15) != 0) return -2;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {row_stride_bytes};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(static_cast<CUtensorMap*>(out_map), dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8,
                        2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, EMOE_TMA_L2PROMO,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -3;
}

// One tensor map per scale channel whose rows are a multiple of 16 bytes: a [N][row_bytes] byte image,
// boxes of 128 rows x 32 bytes, no swizzle (the int8 streaming kernel's scale windows).
int encode_scale_tmap(void* out_map, const void* scales, int N, int row_bytes) {
  if (row_bytes < 32 || row_bytes % 16 != 0 || N < 128) return -2;
  return encode_tmap_2d(out_map, 0, scales, static_cast<uint64_t>(row_bytes), static_cast<uint64_t>(N),
                        static_cast<uint64_t>(row_bytes), 32, 128, false);
}

// One tensor map per packed matrix: a [N][row_bytes] byte image, 64-row x 128-byte boxes, 128-byte swizzle.
int encode_weight_tmap(void* out_map, const void* packed, int N, int K, int bits) {
  const uint64_t row_bytes = static_cast<uint64_t>(K) * bits / 8;
  if (row_bytes < 128 || N < TMA_BOX_ROWS) return -2;
  return encode_tmap_2d(out_map, 0, packed, row_bytes, static_cast<uint64_t>(N), row_bytes, 128, TMA_BOX_ROWS);
}

}  // namespace emoe
