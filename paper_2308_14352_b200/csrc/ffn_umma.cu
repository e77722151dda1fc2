// Grouped expert GEMM on packed weights with tcgen05 tensor-core MMAs, for experts that hold
// many tokens (prefill, large decode batches).  Paper Sections 1/2.1 (each activated expert is
// an independent FFN) on the Section 3.2 storage (b-bit codes + scale channel, w~ = q * s).
//
// Shape of one work unit: 128 output channels (UMMA M, "swap-AB": the weight rows are the M side)
// x a group of up to three 128-token tiles of one expert (one accumulator of 128 tensor-memory
// columns per token tile, neighbouring tiles issued as one N = 256 MMA) x all inputs.  The
// dequantised A operand, the expensive part, is shared by the whole group, and it never touches
// shared memory: the dequantisation warps write it into TENSOR MEMORY (tcgen05.st, 32 columns per
// 64-input stage, a ring of four stages behind the accumulators) and the MMA takes it from there
// (the [a_tmem] operand form).  Shared memory then carries only the packed boxes and the
// activation tiles: with A in shared memory too, the operand reads of the MMAs, the stores of the
// dequantisation and the TMA writes together asked for more than the 128 bytes per cycle an SM
// has, and the tensor pipe ran at a third of its rate.
//   warp 0    TMA producer: packed code boxes (128 rows x 128 bytes, the decode kernel's tensor
//             maps) into a 2-deep raw ring, and the tokens' activations (one box of 128 tokens x
//             64 inputs per token tile, fp16, K-major, 128-byte swizzle) into a 4-deep ring;
//   warps 2-9 two threads per output channel: read the channel's packed bytes from the raw ring,
//             dequantise to fp16 (code -> exact fp16 integer by mantissa insertion, then one
//             multiply by the group scale: |error| <= 2^-12 relative, the only approximation of
//             this path), and store their 32 values as 16 columns of the channel's tensor-memory
//             lane; later the epilogue: tensor memory -> registers -> activation -> global memory;
//   warp 1    one thread issues tcgen05.mma (M128 N256/N128 K16, fp16 x fp16 -> fp32 in TMEM) per
//             16 inputs and commits each stage back to the producers.
// SwiGLU's first projection runs a unit twice, first against w1, then against w3 (all 384
// accumulator columns for one matrix at a time keep the group at three token tiles): the first
// pass parks its raw sums in a per-CTA scratch block in global memory (written and read back by
// the same thread, L2-resident), the second pass's epilogue forms silu(a) * b.
// Activations travel as fp16 (exact for bf16 values inside the fp16 range, saturated outside);
// the hidden vector is rounded to bf16 first, as the definition asks, then stored as fp16.
// The reduction index is enumerated in the order the unpack emits code pairs; the activation
// buffers are written in that same order (scatter_x16_kernel, first-projection epilogue).
// Every wait is bounded (see pipe.cuh); tensor memory is always released before exit.
#include <cuda.h>

#include "common.cuh"
#include "ffn_tile.cuh"
#include "pipe.cuh"
#include "umma.cuh"

namespace emoe {
namespace {

constexpr int UM_TOK = 128;                // tokens per tile (UMMA N)
constexpr int UM_ROWS = 128;               // output channels per tile (UMMA M)
constexpr int UM_BK = 64;                  // inputs per operand stage: one 128-byte row of fp16
constexpr int UM_STAGES = 4;               // operand stages: A in tensor memory (32 columns each), B in shared memory
constexpr int UM_RAW_STAGES = 2;
constexpr int UM_TILE_BYTES = 128 * 128;   // a [128 tokens][64] fp16 operand tile, or a [128 rows][128 B] packed tile
constexpr int UM_GROUP = 3;                // token tiles that share one dequantised A stage
constexpr int UM_B_STAGE_BYTES = UM_GROUP * UM_TILE_BYTES;
constexpr int UM_SMEM_BYTES = UM_RAW_STAGES * UM_TILE_BYTES + UM_STAGES * UM_B_STAGE_BYTES + 1024;  // 225 KB + alignment slack
constexpr int UM_ACC_COLS = UM_GROUP * UM_TOK;  // accumulators: tensor-memory columns 0 .. 383
constexpr int UM_A_COLS = UM_BK / 2;             // one A stage: 64 fp16 inputs = 32 columns; stages at 384, 416, 448, 480
constexpr int UM_MAX_CTAS = 160;                 // grid limit (one CTA per SM): sizes the scratch of the gated first projection
#ifndef EMOE_UM_UNPACK_WARPS
#define EMOE_UM_UNPACK_WARPS 8
#endif
constexpr int UM_UNPACK_WARPS = EMOE_UM_UNPACK_WARPS;  // two (or four) threads per output channel
static_assert(UM_UNPACK_WARPS == 8 || UM_UNPACK_WARPS == 16, "a thread stores its 32 or 16 values as one block of 16 or 8 tensor-memory columns");
constexpr int UM_PARTS = UM_UNPACK_WARPS / 4;            // each dequantises its share of a stage and reads its share of the columns
constexpr int UM_THREADS = (2 + UM_UNPACK_WARPS) * 32;
constexpr int UM_TMEM_COLS = 512;

// position of input k in the activation buffers of this path: the unpack emits the code pairs
// (c, c+4) of an 8-code word at 4 bits and (c, c+8) of a 16-code word at 2 bits
template <int BITS>
__device__ __forceinline__ int pair_pos(int k) {
  if (BITS == 8) return k;
  constexpr int B = BITS == 4 ? 8 : 16;
  const int o = k & (B - 1);
  return (k & ~(B - 1)) + (o < B / 2 ? 2 * o : 2 * (o - B / 2) + 1);
}
__device__ __forceinline__ int pair_pos_rt(int bits, int k) {
  return bits == 8 ? k : (bits == 4 ? pair_pos<4>(k) : pair_pos<2>(k));
}

__device__ __forceinline__ uint32_t h2_fma(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}
__device__ __forceinline__ uint32_t h2_add(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("add.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t h2_mul(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// ---- dequantise one 16-byte chunk of a packed row to fp16 (q * s), 8 values per output chunk ----
// 8 bits: 16 codes -> 2 chunks.  byte ^ 0x80 = q + 128 goes into the mantissa of 1024.
__device__ __forceinline__ void dequant_chunk8(const uint4& raw, uint32_t s2, uint4 (&out)[2]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  uint32_t o[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t u = w[i] ^ 0x80808080u;
    o[2 * i] = h2_mul(h2_add(prmt(u, 0x64646464u, 0x5140u), 0xE480E480u), s2);      // -(1024 + 128)
    o[2 * i + 1] = h2_mul(h2_add(prmt(u, 0x64646464u, 0x5342u), 0xE480E480u), s2);
  }
  out[0] = make_uint4(o[0], o[1], o[2], o[3]);
  out[1] = make_uint4(o[4], o[5], o[6], o[7]);
}
// 4 bits: one 8-code word -> one chunk, pair order (c, c+4).
__device__ __forceinline__ uint4 dequant_word4(uint32_t w, uint32_t s2) {
  const uint32_t hi = w >> 8;
  const uint32_t t0 = h2_add(and_xor(w, 0x000F000Fu, 0x64086408u), 0xE408E408u);               // v - 1032
  const uint32_t t1 = h2_fma(and_xor(w, 0x00F000F0u, 0x64806480u), 0x2C002C00u, 0xD480D480u);  // v/16 - 72
  const uint32_t t2 = h2_add(and_xor(hi, 0x000F000Fu, 0x64086408u), 0xE408E408u);
  const uint32_t t3 = h2_fma(and_xor(hi, 0x00F000F0u, 0x64806480u), 0x2C002C00u, 0xD480D480u);
  return make_uint4(h2_mul(t0, s2), h2_mul(t1, s2), h2_mul(t2, s2), h2_mul(t3, s2));
}
// 2 bits: one 16-code word -> two chunks, pair order (c, c+8).
__device__ __forceinline__ void dequant_word2(uint32_t w, uint32_t s2, uint4 (&out)[2]) {
  // field at mantissa bit p of 1024: v = 1024 + (q + 2) * 2^p;  q = v * 2^-p - (1024 * 2^-p + 2)
  const uint32_t msk[5] = {0x00030003u, 0x000C000Cu, 0x00300030u, 0x00C000C0u, 0x03000300u};
  const uint32_t mag[5] = {0x64026402u, 0x64086408u, 0x64206420u, 0x64806480u, 0x66006600u};
  const uint32_t mul[5] = {0x3C003C00u, 0x34003400u, 0x2C002C00u, 0x24002400u, 0x1C001C00u};
  const uint32_t add[5] = {0xE402E402u, 0xDC08DC08u, 0xD420D420u, 0xCC80CC80u, 0xC600C600u};
  uint32_t o[8];
  const uint32_t hi = w >> 10;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const int p = c < 5 ? c : c - 5;
    o[c] = h2_mul(h2_fma(and_xor(c < 5 ? w : hi, msk[p], mag[p]), mul[p], add[p]), s2);
  }
  out[0] = make_uint4(o[0], o[1], o[2], o[3]);
  out[1] = make_uint4(o[4], o[5], o[6], o[7]);
}
__device__ __forceinline__ uint32_t pick_word(const uint4& v, int i) {
  return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}
// Output chunks 2*pp and 2*pp+1 (16 inputs) of operand stage j of a packed row.
__device__ __forceinline__ void dequant_pair(int bits, const unsigned char* rrow, int rin, int j, int pp, uint32_t s2,
                                             uint4 (&out)[2]) {
  if (bits == 8) {
    dequant_chunk8(*reinterpret_cast<const uint4*>(rrow + (((4 * j + pp) ^ (rin & 7)) << 4)), s2, out);
  } else if (bits == 4) {
    const uint4 raw = *reinterpret_cast<const uint4*>(rrow + (((2 * j + (pp >> 1)) ^ (rin & 7)) << 4));
    out[0] = dequant_word4(pick_word(raw, 2 * (pp & 1)), s2);
    out[1] = dequant_word4(pick_word(raw, 2 * (pp & 1) + 1), s2);
  } else {
    const uint4 raw = *reinterpret_cast<const uint4*>(rrow + ((j ^ (rin & 7)) << 4));
    dequant_word2(pick_word(raw, pp), s2, out);
  }
}

__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const uint32_t (&r)[16]) { tmem_st16(taddr, r); }
__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const uint32_t (&r)[8]) { tmem_st8(taddr, r); }

struct UmmaArgs {
  int phase;
  LayerDims L;
  const CUtensorMap* wmaps;  // [E][3] packed-weight tensor maps (boxes of 64 rows x 128 bytes)
  const int* plan;           // header + PlanRec per activated expert
  __half* hidden16;          // first projection's output (fp16, pair order)
  float* o;                  // second projection's output [n_pairs][d_model]
  int zsplit;                // second projection: slices of the inputs per unit (1 or 2), slice z into plane z of o
  size_t plane_stride;       // floats between the planes of o
  float* scratch;            // gated first projection: [gridDim.x][384 token columns][128 channels] raw sums of the w1 pass
  int* check_word;
};

// the tiles of this CTA: linear index = blockIdx.x, += gridDim.x over
// (activated expert, group of `group` token tiles, row block) with the row block running fastest
struct TileWalk {
  const PlanRec* recs;
  int n_active, row_blocks, lin, a, base, group, zs;
  PlanRec rec;
  int tiles_of_a;
  __device__ __forceinline__ void init(const int* plan, int rb, int token_tiles_per_group, int zsplit) {
    zs = zsplit;
    n_active = *reinterpret_cast<const volatile int*>(plan);
    recs = reinterpret_cast<const PlanRec*>(reinterpret_cast<const char*>(plan) + PLAN_HEADER_BYTES);
    row_blocks = rb;
    // Grouping token tiles shares the dequantisation but makes fewer, longer work units: take the
    // largest group (up to the limit) that still leaves every CTA of the grid a unit.  Every
    // thread that walks the tiles computes the same answer from the plan.
    group = 1;
    for (int g = token_tiles_per_group; g > 1; --g) {
      long long units = 0;
      for (int i = 0; i < n_active; ++i) units += (recs[i].cnt + g * UM_TOK - 1) / (g * UM_TOK);
      if (units * rb * zs >= static_cast<long long>(gridDim.x)) {
        group = g;
        break;
      }
    }
    lin = blockIdx.x;
    a = -1;
    base = 0;
    tiles_of_a = 0;
  }
  // advances to the CTA's next tile (tt = index of its token group); false when there is none
  __device__ __forceinline__ bool next(int& tt, int& rb, int& z) {
    while (a < 0 || lin >= base + tiles_of_a) {
      base += tiles_of_a;
      ++a;
      if (a >= n_active) return false;
      rec = recs[a];
      tiles_of_a = row_blocks * zs * ((rec.cnt + group * UM_TOK - 1) / (group * UM_TOK));
    }
    const int local = lin - base;
    tt = local / (row_blocks * zs);
    const int rz = local - tt * row_blocks * zs;  // the slices of a row block lie next to each other
    rb = rz / zs;
    z = rz - rb * zs;
    lin += gridDim.x;
    return true;
  }
};

__global__ void __launch_bounds__(UM_THREADS, 1)
    ffn_umma_kernel(const UmmaArgs a, const __grid_constant__ CUtensorMap tmap_b) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * UM_RAW_STAGES + 3 * UM_STAGES + 2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* raw_ring = smem;
  unsigned char* b_ring = smem + UM_RAW_STAGES * UM_TILE_BYTES;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  const uint32_t bar_raw_full = smem_u32(bars);
  const uint32_t bar_raw_empty = smem_u32(bars + UM_RAW_STAGES);
  const uint32_t bar_b_full = smem_u32(bars + 2 * UM_RAW_STAGES);
  const uint32_t bar_a_full = smem_u32(bars + 2 * UM_RAW_STAGES + UM_STAGES);
  const uint32_t bar_ab_empty = smem_u32(bars + 2 * UM_RAW_STAGES + 2 * UM_STAGES);
  const uint32_t bar_acc_full = smem_u32(bars + 2 * UM_RAW_STAGES + 3 * UM_STAGES);
  const uint32_t bar_acc_empty = bar_acc_full + 8;

  if (threadIdx.x == 0) {
    abort_word = 0;
    for (int s = 0; s < UM_RAW_STAGES; ++s) {
      mbar_init(bar_raw_full + 8 * s, 1);
      mbar_init(bar_raw_empty + 8 * s, UM_UNPACK_WARPS);
    }
    for (int s = 0; s < UM_STAGES; ++s) {
      mbar_init(bar_b_full + 8 * s, 1);
      mbar_init(bar_a_full + 8 * s, UM_UNPACK_WARPS);
      mbar_init(bar_ab_empty + 8 * s, 1);
    }
    mbar_init(bar_acc_full, 1);
    mbar_init(bar_acc_empty, UM_UNPACK_WARPS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), UM_TMEM_COLS);  // three accumulators + four A stages
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  pdl_wait();  // barrier set-up and the tensor-memory allocation overlap the kernel in front
  pdl_trigger();

  const LayerDims& L = a.L;
  const int N = a.phase == 0 ? L.d_ff : L.d_model;
  const int K = a.phase == 0 ? L.d_model : L.d_ff;
  const bool gated = a.phase == 0 && L.act == EMOE_ACT_SWIGLU;
  const int npass = gated ? 2 : 1;  // a gated unit runs against w1, then against w3
  const int mat_first = a.phase == 0 ? 0 : (L.act == EMOE_ACT_SWIGLU ? 2 : 1);
  const int row_blocks = (N + UM_ROWS - 1) / UM_ROWS;
  const int kb_total = K / UM_BK;

  TileWalk walk;
  const int zs = a.phase == 0 ? 1 : a.zsplit;
  const int kb_len = kb_total / zs;  // steps of a unit
  walk.init(a.plan, row_blocks, UM_GROUP, zs);
  const int group = walk.group;
  int tt, rb, z;

  if (warp == 0) {
    // ---------------- TMA producer (one lane) ----------------
    if (lane == 0) {
      int raw_it = 0, ab_it = 0;
      bool ok = true;
      while (ok && walk.next(tt, rb, z)) {
        const PlanRec rec = walk.rec;
        const CUtensorMap* maps = a.wmaps + static_cast<size_t>(rec.e) * 3;
        const int kbs = (1024 / rec.bits) / UM_BK;  // operand stages per packed box (128 bytes of a row)
        const int row0 = rb * UM_ROWS;
        const int tok0 = rec.begin + tt * group * UM_TOK;
        const int ntt = min(group, (rec.cnt - tt * group * UM_TOK + UM_TOK - 1) / UM_TOK);  // token tiles of this group
        for (int pass = 0; pass < npass && ok; ++pass) {
          const CUtensorMap* mp = maps + (gated ? pass : mat_first);
          const int kb_end = (z + 1) * kb_len;
          for (int kb = z * kb_len; kb < kb_end && ok;) {
            const int rs = raw_it % UM_RAW_STAGES;
            if (!mbar_wait(bar_raw_empty + 8 * rs, ((raw_it / UM_RAW_STAGES) & 1) ^ 1, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            const uint32_t rfull = bar_raw_full + 8 * rs;
            mbar_expect_tx(rfull, UM_TILE_BYTES);
            const int c0 = (kb / kbs) * 128;
            const uint32_t dst = smem_u32(raw_ring + rs * UM_TILE_BYTES);
            tma_load_2d(dst, mp, c0, row0, rfull);
            tma_load_2d(dst + UM_TILE_BYTES / 2, mp, c0, row0 + 64, rfull);
            ++raw_it;
            for (int j = 0; j < kbs && kb < kb_end; ++j, ++kb) {
              const int s = ab_it % UM_STAGES;
              if (!mbar_wait(bar_ab_empty + 8 * s, ((ab_it / UM_STAGES) & 1) ^ 1, a.check_word, abort_flag)) {
                ok = false;
                break;
              }
              const uint32_t bfull = bar_b_full + 8 * s;
              mbar_expect_tx(bfull, ntt * UM_TILE_BYTES);
              for (int t = 0; t < ntt; ++t)
                tma_load_2d(smem_u32(b_ring + s * UM_B_STAGE_BYTES + t * UM_TILE_BYTES), &tmap_b, kb * UM_BK, tok0 + t * UM_TOK,
                            bfull);
              ++ab_it;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (one lane) ----------------
    if (lane == 0) {
      // kind::f16, fp16 x fp16 -> fp32, A from tensor memory, B K-major from shared memory, M = 128, N = 128
      const uint32_t idesc = (1u << 4) | ((UM_TOK >> 3) << 17) | ((UM_ROWS >> 4) << 24);
      // two neighbouring token tiles as one N = 256 MMA
      const uint32_t idesc2 = (1u << 4) | (((2 * UM_TOK) >> 3) << 17) | ((UM_ROWS >> 4) << 24);
      int ab_it = 0, unit_it = 0;
      bool ok = true;
      while (ok && walk.next(tt, rb, z)) {
        const int ntt = min(group, (walk.rec.cnt - tt * group * UM_TOK + UM_TOK - 1) / UM_TOK);
        for (int pass = 0; pass < npass && ok; ++pass, ++unit_it) {
          if (!mbar_wait(bar_acc_empty, ((unit_it & 1) ^ 1), a.check_word, abort_flag)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const int kb0 = z * kb_len;
          for (int kb = kb0; kb < kb0 + kb_len; ++kb, ++ab_it) {
            const int s = ab_it % UM_STAGES;
            const uint32_t par = (ab_it / UM_STAGES) & 1;
            if (!mbar_wait(bar_a_full + 8 * s, par, a.check_word, abort_flag) ||
                !mbar_wait(bar_b_full + 8 * s, par, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t a_t = tmem_base + UM_ACC_COLS + s * UM_A_COLS;
            const uint32_t bs = smem_u32(b_ring + s * UM_B_STAGE_BYTES);
            // accumulator of token tile j: columns j * 128; the B tiles of a group lie back to back, so
            // tiles j and j+1 form one 256-token operand
            for (int j = 0; j < ntt; j += 2) {
              const bool two = j + 1 < ntt;
              const uint64_t db = umma_desc(bs + j * UM_TILE_BYTES);
              const uint32_t acc_col = tmem_base + j * UM_TOK;
              const uint32_t id = two ? idesc2 : idesc;
#pragma unroll
              for (int k4 = 0; k4 < UM_BK / 16; ++k4)  // 16 inputs: 8 columns of A, 32 bytes (2 descriptor units) of B
                umma_f16_ts(acc_col, a_t + 8 * k4, db + 2 * k4, id, (kb > kb0 || k4 > 0) ? 1u : 0u);
            }
            umma_commit(bar_ab_empty + 8 * s);  // the stage may be refilled once these MMAs have read it
          }
          if (ok) umma_commit(bar_acc_full);
        }
      }
    }
  } else {
    // ---------------- dequantise (two threads per output channel), then epilogue ----------------
    const int quarter = warp & 3;          // TMEM lanes this warp may access: 32 * quarter ...
    const int part = (warp - 2) >> 2;      // which half of a stage's inputs (and of the token columns) is this warp's
    const int r = 32 * quarter + lane;     // channel of the tile = row of the operand = TMEM lane
    const int box = r >> 6, rin = r & 63;
    const int G = L.group > 0 ? L.group : K;
    const int ngroups = K / G;
    const bool sf16 = L.scale_f16 != 0;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16);
    // scratch block of this CTA, token-column major: [384 columns][128 channels], so that the 32 lanes of a warp
    // (32 neighbouring channels) touch 128 contiguous bytes per column
    float* park = a.scratch + static_cast<size_t>(blockIdx.x) * UM_ROWS * UM_ACC_COLS + r;
    int raw_it = 0, ab_it = 0, unit_it = 0;
    bool ok = true;
    while (ok && walk.next(tt, rb, z)) {
      const PlanRec rec = walk.rec;
      const int bits = rec.bits;
      const int kbs = (1024 / bits) / UM_BK;
      const int n = min(rb * UM_ROWS + r, N - 1);
      const size_t srow = static_cast<size_t>(n) * ngroups;
      for (int pass = 0; pass < npass && ok; ++pass, ++unit_it) {
        const void* sp = rec.scales[gated ? pass : mat_first];
        // scales of this step, the next one and the one after: a load has two steps to come back from L2
        const int spg = G / UM_BK;  // steps per scale group (G is a multiple of 128, or the whole row)
        const int kb_first = z * kb_len;
        float sv = load_scale_ro(sp, sf16, srow + min(kb_first / spg, ngroups - 1)),
              sv_n1 = load_scale_ro(sp, sf16, srow + min((kb_first + 1) / spg, ngroups - 1)), sv_n2;
        // group of the step two ahead, kept by counting (a division by the group size per step was a
        // third of the step's instructions)
        int g2 = (kb_first + 2) / spg, c2 = (kb_first + 2) % spg;
        bool tiny_scale = false;  // q * s below the smallest normal fp16 number would lose bits in the fp16 operand
        const int kb_end = (z + 1) * kb_len;
        for (int kb = z * kb_len; kb < kb_end && ok;) {
          const int rs = raw_it % UM_RAW_STAGES;
          if (!mbar_wait(bar_raw_full + 8 * rs, (raw_it / UM_RAW_STAGES) & 1, a.check_word, abort_flag)) {
            ok = false;
            break;
          }
          const unsigned char* rrow = raw_ring + rs * UM_TILE_BYTES + box * (UM_TILE_BYTES / 2) + rin * 128;
          for (int j = 0; j < kbs && kb < kb_end; ++j, ++kb, ++ab_it) {
            const int s = ab_it % UM_STAGES;
            if (!mbar_wait(bar_ab_empty + 8 * s, ((ab_it / UM_STAGES) & 1) ^ 1, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            tc_fence_after();  // the MMAs that read this stage's columns are complete
            sv_n2 = load_scale_ro(sp, sf16, srow + min(g2, ngroups - 1));
            if (++c2 == spg) {
              c2 = 0;
              ++g2;
            }
            tiny_scale |= sv != 0.0f && fabsf(sv) < 6.104e-5f;
            const __half sh = __float2half_rn(sv);
            const uint32_t s2 = static_cast<uint32_t>(__half_as_ushort(sh)) * 0x00010001u;
            constexpr int QN = 4 / UM_PARTS;  // 16-input pieces of the stage per thread
            uint32_t v[8 * QN];               // this thread's inputs of the stage, two per register
#pragma unroll
            for (int q = 0; q < QN; ++q) {
              uint4 o[2];
              dequant_pair(bits, rrow, rin, j, QN * part + q, s2, o);
              v[8 * q + 0] = o[0].x, v[8 * q + 1] = o[0].y, v[8 * q + 2] = o[0].z, v[8 * q + 3] = o[0].w;
              v[8 * q + 4] = o[1].x, v[8 * q + 5] = o[1].y, v[8 * q + 6] = o[1].z, v[8 * q + 7] = o[1].w;
            }
            tmem_st_cols(lane_base + UM_ACC_COLS + s * UM_A_COLS + 8 * QN * part, v);
            tmem_st_wait();
            sv = sv_n1;
            sv_n1 = sv_n2;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_a_full + 8 * s);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_raw_empty + 8 * rs);
          ++raw_it;
        }
        if (!ok) break;
        if (tiny_scale) atomicOr(a.check_word, CHECK_F16_RANGE);
        // ---- epilogue: this warp's 32 channels x its half of the token columns ----
        if (!mbar_wait(bar_acc_full, unit_it & 1, a.check_word, abort_flag)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const int nrow = rb * UM_ROWS + r;
        const int tok_first = tt * group * UM_TOK;
        const int ntt = min(group, (rec.cnt - tok_first + UM_TOK - 1) / UM_TOK);
        const int hpos = a.phase == 0 ? pair_pos_rt(bits, min(nrow, N - 1)) : 0;
#pragma unroll 1
        for (int jc = 0; jc < ntt * (UM_TOK / UM_PARTS / 32); ++jc) {
          // token tile j of the group, 32 columns from cc on (this warp's share of the tile's columns)
          const int j = jc / (UM_TOK / UM_PARTS / 32);
          const int cc = (UM_TOK / UM_PARTS) * part + 32 * (jc % (UM_TOK / UM_PARTS / 32));
          const int tokens = min(UM_TOK, rec.cnt - tok_first - j * UM_TOK);
          const size_t slot0 = static_cast<size_t>(rec.begin) + static_cast<size_t>(tok_first) + static_cast<size_t>(j) * UM_TOK;
          uint32_t va[32];
          tmem_ld32(lane_base + j * UM_TOK + cc, va);
          tmem_ld_wait();
          float* pk = park + static_cast<size_t>(j * UM_TOK + cc) * UM_ROWS;
          if (gated && pass == 0) {
            // the w1 sums wait in the scratch block for the w3 pass of the same unit
#pragma unroll
            for (int c = 0; c < 32; ++c) pk[c * UM_ROWS] = __uint_as_float(va[c]);
            continue;
          }
          // one compact unrolled loop per case (the conditions are uniform; a single loop with all cases
          // inside was several times the code, fetched anew at every unit's end)
          if (nrow >= N) continue;
          const int live = min(32, tokens - cc);  // token columns of this chunk that exist
          if (a.phase != 0) {
            float* dst = a.o + z * a.plane_stride + (slot0 + cc) * N + nrow;
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (c < live) dst[static_cast<size_t>(c) * N] = __uint_as_float(va[c]);
          } else {
            __half* dst = a.hidden16 + (slot0 + cc) * N + hpos;
            bool beyond = false;
            if (gated) {
              float av[32];
#pragma unroll
              for (int c = 0; c < 32; ++c) av[c] = pk[c * UM_ROWS];  // all loads first: one round trip to L2, not 32
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                // the hidden vector is a bf16 tensor
                const float h = __bfloat162float(__float2bfloat16_rn(av[c] / (1.0f + expf(-av[c])) * __uint_as_float(va[c])));
                beyond |= beyond_f16(h);
                if (c < live) dst[static_cast<size_t>(c) * N] = __float2half_rn(fminf(fmaxf(h, -65504.0f), 65504.0f));
              }
            } else {
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const float h = __bfloat162float(__float2bfloat16_rn(fmaxf(__uint_as_float(va[c]), 0.0f)));
                beyond |= beyond_f16(h);
                if (c < live) dst[static_cast<size_t>(c) * N] = __float2half_rn(fminf(h, 65504.0f));
              }
            }
            if (beyond) atomicOr(a.check_word, CHECK_F16_RANGE);  // saturated above: reported, not silent
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acc_empty);
      }
    }
  }

  // wind-down: everybody meets, then the allocating warp releases tensor memory
  if (*abort_flag)
    for (int i = 0; i < 2000; ++i) __nanosleep(100);  // let copies in flight land
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, UM_TMEM_COLS);
  }
}

// x rows -> expert order, fp16, pair order of the owning expert's bitwidth (saturating)
__global__ void __launch_bounds__(128)
    scatter_x16_kernel(const ExpertDev* __restrict__ experts, const __nv_bfloat16* __restrict__ x,
                       const int32_t* __restrict__ ids, const int32_t* __restrict__ perm, const int32_t* __restrict__ off,
                       int E, int* __restrict__ plan, int top_k, int d, int n_pairs, int cnt_lo, int cnt_hi,
                       __half* __restrict__ xs, int* __restrict__ check_word) {
  pdl_wait();
  pdl_trigger();
  if (plan && blockIdx.x == 0 && threadIdx.x < 32) {
    // work plan: activated experts, widest codes first
    const int lane = threadIdx.x;
    PlanRec* recs = reinterpret_cast<PlanRec*>(reinterpret_cast<char*>(plan) + PLAN_HEADER_BYTES);
    int base = 0;
    for (int b = 8; b >= 2; b >>= 1) {
      for (int e0 = 0; e0 < E; e0 += 32) {
        const int e = e0 + lane;
        const int cnt = e < E ? off[e + 1] - off[e] : 0;
        const bool act = cnt >= cnt_lo && cnt <= cnt_hi && experts[e].bits == b;
        const unsigned m = __ballot_sync(0xffffffffu, act);
        if (act) {
          PlanRec& r = recs[base + __popc(m & ((1u << lane) - 1u))];
          r.e = e;
          r.begin = off[e];
          r.cnt = cnt;
          r.bits = b;
          r.scales[0] = experts[e].scales[0];
          r.scales[1] = experts[e].scales[1];
          r.scales[2] = experts[e].scales[2];
          r.done = 0;
        }
        base += __popc(m);
      }
    }
    if (lane == 0) {
      plan[0] = base;
      plan[1] = 0;
      plan[2] = 0;
    }
  }
  const int slot = blockIdx.x;
  const int pair = perm[slot];
  if (pair < 0 || pair >= n_pairs) return;
  const int e_slot = ids[pair];
  if (e_slot < 0 || e_slot >= E) return;  // a slot the permutation did not write (stale entry behind a dropped pair)
  const int cnt_slot = off[e_slot + 1] - off[e_slot];
  if (cnt_slot < cnt_lo || cnt_slot > cnt_hi) return;  // this expert's rows belong to another kernel family
  const int bits = experts[e_slot].bits;
  const __nv_bfloat16* src = x + static_cast<size_t>(pair / top_k) * d;
  __half* dst = xs + static_cast<size_t>(slot) * d;
  bool beyond = false;
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    const float xv = __bfloat162float(src[k]);
    beyond |= beyond_f16(xv);
    dst[pair_pos_rt(bits, k)] = __float2half_rn(fminf(fmaxf(xv, -65504.0f), 65504.0f));
  }
  if (beyond) atomicOr(check_word, CHECK_F16_RANGE);  // saturated: reported, not silent
}

}  // namespace

bool ffn_umma_supported(const LayerDims& L) {
  // the same tensor maps as the TMA path; K in whole 128-byte packed rows at every width
  return ffn_tma_supported(L) && L.d_model % 512 == 0 && L.d_ff % 512 == 0;
}

cudaError_t launch_scatter_x16(const LayerDims& L, const ExpertDev* experts, const void* x, const int32_t* ids,
                               const int32_t* perm, const int32_t* off, int* plan, void* xs16, int n_pairs,
                               int cnt_lo, int cnt_hi, int* check_word, cudaStream_t st) {
  return launch_chain(scatter_x16_kernel, dim3(n_pairs), dim3(128), 0, st, experts, reinterpret_cast<const __nv_bfloat16*>(x), ids,
                      perm, off, L.E, plan, L.top_k, L.d_model, n_pairs, cnt_lo, cnt_hi, reinterpret_cast<__half*>(xs16), check_word);
}

size_t ffn_umma_scratch_bytes(const LayerDims& L) {
  return L.act == EMOE_ACT_SWIGLU ? static_cast<size_t>(UM_MAX_CTAS) * UM_ROWS * UM_ACC_COLS * sizeof(float) : 0;
}

// Slices of the second projection's inputs per unit: two when whole units alone would leave the last round of
// CTAs mostly idle (the estimate assumes uniform routing; the kernel is right for any routing).
int ffn_umma_zsplit(const LayerDims& L, int T, int sms) {
  const long long per_expert = (static_cast<long long>(T) * L.top_k + L.E - 1) / L.E;
  const long long units = static_cast<long long>(L.E) * ((per_expert + UM_GROUP * UM_TOK - 1) / (UM_GROUP * UM_TOK)) *
                          ((L.d_model + UM_ROWS - 1) / UM_ROWS);
  if (sms <= 0 || units < sms) return 1;
  const bool halves_ok = (L.d_ff / UM_BK / 2) % 8 == 0;  // a slice starts on a packed box at every width
  // share of the CTA rounds that does work, with whole units and with halves
  const double whole = static_cast<double>(units) / (((units + sms - 1) / sms) * sms);
  const double halves = static_cast<double>(2 * units) / (((2 * units + sms - 1) / sms) * sms);
  return (halves_ok && halves > whole + 0.03) ? 2 : 1;
}

cudaError_t launch_ffn_umma(int phase, const LayerDims& L, const void* wmaps, const int* plan, const void* in16,
                            void* hidden16, float* o, float* scratch, int n_pairs, int zsplit, int* check_word,
                            cudaStream_t st) {
  if (phase == 0 && L.act == EMOE_ACT_SWIGLU && !scratch) return cudaErrorInvalidValue;
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const int K = phase == 0 ? L.d_model : L.d_ff;
  CUtensorMap tmap_b;
  if (encode_tmap_2d(&tmap_b, /*fp16*/ 1, in16, static_cast<uint64_t>(K), static_cast<uint64_t>(n_pairs),
                     static_cast<uint64_t>(K) * 2, UM_BK, UM_TOK) != 0)
    return cudaErrorInvalidValue;
  static int sms_of_device[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!sms_of_device[dev]) {
    e = cudaFuncSetAttribute(ffn_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, UM_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms_of_device[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  const long long row_blocks = (N + UM_ROWS - 1) / UM_ROWS;
  // upper bound of the tile count: every pair alone in a token tile
  long long tiles = row_blocks * (static_cast<long long>(n_pairs < L.E ? n_pairs : L.E) + n_pairs / UM_TOK) * (phase == 1 ? zsplit : 1);
  const int cap = sms_of_device[dev] < UM_MAX_CTAS ? sms_of_device[dev] : UM_MAX_CTAS;
  const int grid = static_cast<int>(tiles < cap ? tiles : cap);
  UmmaArgs a;
  a.phase = phase;
  a.L = L;
  a.wmaps = static_cast<const CUtensorMap*>(wmaps);
  a.plan = plan;
  a.hidden16 = reinterpret_cast<__half*>(hidden16);
  a.o = o;
  a.scratch = scratch;
  a.zsplit = zsplit < 1 ? 1 : zsplit;
  a.plane_stride = static_cast<size_t>(n_pairs) * L.d_model;
  a.check_word = check_word;
  return launch_chain(ffn_umma_kernel, dim3(grid), dim3(UM_THREADS), UM_SMEM_BYTES, st, a, tmap_b);
}

}  // namespace emoe
