// Grouped expert FFN on packed weights for the decode regime (a few tokens per expert): the
// packed codes go to the 5th-generation tensor cores as 8-bit integer operands.
// Paper Sections 1/2.1 (each activated expert is an independent FFN) on the Section 3.2 storage
// (b-bit codes q + scale channel, w~ = q * s): nothing is decompressed in memory; the codes are
// multiplied as integers and the scale of a group of inputs is applied to the group's integer
// sum, which gives q * s * x summed exactly as the definition does.
//
// The kernel is bound by streaming packed weights from HBM, so everything is arranged to keep
// the per-code work of the SM's ordinary cores as small as possible:
//   * 8-bit codes: none.  A TMA box of 128 rows x 128 bytes (128-byte swizzle) IS a K-major
//     int8 operand tile; tcgen05.mma reads it from shared memory as it arrived.
//   * 4-bit codes: a word of eight nibbles becomes two words of int8 (the nibble in the high
//     half of its byte = 16 q, signed): 3 instructions per 8 codes.  2-bit codes: a word of
//     sixteen fields becomes four words (field in the top two bits of its byte = 64 q): 7 per
//     16.  The unpacked bytes go straight to tensor memory (tcgen05.st) and are the A operand
//     from there, so they never cost shared-memory bandwidth.  The factors 16 and 64 are
//     divided out with the scale (a power of two: exact).
//   * the activations are two-limb block-scaled integers (act_q.cuh): the tokens' hi and lo
//     limbs are 2 x NT columns of the B operand, fetched by TMA; one MMA pass yields
//     sum q*hi and sum q*lo as exact int32 per 128-input segment.
//   * per segment, the epilogue warps read the 2 x NT int32 columns from tensor memory and do
//     total[t] += (s[n][g] * sx[t][g]) * float(128 * hi + lo) in fp32.
// Shape of the work: persistent CTAs, one per SM, pull items (activated expert, block of 128
// output rows[, split-K slice]) of the first projection, then of the second, from a device
// counter; an item of the second projection waits (bounded) until the expert's hidden vectors
// are complete.  Warp roles: 4 epilogue warps (one thread per output row = tensor-memory lane),
// 2 x 4 unpack warps (alternating A tiles, one thread per row), one TMA producer warp, one
// MMA-issuing warp.  Rings: shared-memory stages (codes + activation tile + scales), two A
// tiles and a ring of accumulators in tensor memory, each with full/empty mbarriers.  Every
// wait is bounded: a wait that runs out sets CHECK_WAIT_TIMEOUT and the CTA winds down.
#include <cuda.h>

#include "act_q.cuh"
#include "common.cuh"
#include "pipe.cuh"
#include "umma.cuh"

namespace emoe {
namespace {

constexpr int I8_ROWS = 128;                         // output rows of an item = UMMA M
constexpr int I8_BOX_ROWS = 64;                      // rows of one weight box (the tensor maps' box)
constexpr int I8_BOX_BYTES = I8_BOX_ROWS * 128;      // 8 KB
constexpr int I8_MAT_BYTES = 2 * I8_BOX_BYTES;       // 128 rows x 128 bytes of one matrix
constexpr int I8_WARP_UNPACK0 = 4;                   // warps 0-3 epilogue, 4-7 and 8-11 unpack
constexpr int I8_WARP_PRODUCER = 12;
constexpr int I8_WARP_MMA = 13;
constexpr int I8_THREADS = 14 * 32;
constexpr int I8_MAX_STAGES = 8;
constexpr int I8_TMEM_COLS = 512;
constexpr int I8_A_COLS = 128;                       // an unpacked A tile: 128 rows x 512 bytes = 128 columns
constexpr int I8_D_COL0 = 2 * I8_A_COLS;             // accumulators behind the two A tiles
constexpr int I8_D_COLS = I8_TMEM_COLS - I8_D_COL0;  // 256 columns of accumulators
constexpr int I8_MAX_DBUF = 16;
constexpr int I8_SCALE_BYTES = I8_ROWS * 16;         // raw scales of a stage: a 16-byte window per row
constexpr int I8_SX_BYTES = 4 * 32 * 4;              // activation block scales of a stage: [4 segments][32 tokens]
constexpr int I8_SMEM_LIMIT = 227 * 1024;

// a shared-memory stage: weight boxes of 1 or 2 matrices | activation tiles of up to 4 segments
// (2*NT rows x 128 bytes each) | weight-scale windows | activation block scales
struct StageLayout {
  int b_off, sc_off, sx_off, bytes;
};
__host__ __device__ inline StageLayout stage_layout(int nt, int nmat) {
  StageLayout s;
  s.b_off = nmat * I8_MAT_BYTES;
  s.sc_off = s.b_off + 4 * (2 * nt) * 128;
  s.sx_off = s.sc_off + nmat * I8_SCALE_BYTES;
  s.bytes = (s.sx_off + I8_SX_BYTES + 1023) / 1024 * 1024;
  return s;
}

struct I8Args {
  int phase_begin, phase_end;  // projections this launch runs: [0,1), [1,2) or both, [0,2)
  LayerDims L;
  const CUtensorMap* wmaps;  // [E][3] packed-weight maps: byte image [N][K*bits/8], boxes 64 rows x 128 bytes
  int* plan;                 // header {activated experts, item counters} + one PlanRec per activated expert
  const float* xsc;          // block scales of the first projection's input [P][d/128]
  int8_t* hq;                // hidden vectors as limbs [P][2][f] (written by the first projection)
  float* hsc;                // their block scales [P][f/128]
  float* o_part;             // [ksplit][P][d]
  int ksplit;
  int row_blocks[2];
  int ngroups[2];
  int gshift;  // log2(group size) if it is a power of two, else -1
  int n_pairs;
  int stages;
  unsigned wait_limit;      // polls before a pipeline wait gives up
  unsigned dep_wait_limit;  // polls (~0.1 us each) before the wait for an expert's hidden vectors gives up
  int dep_extra;            // test hook: completions expected beyond the real count (0 in production)
  int* check_word;
};

struct PhaseDims {
  int K, N, row_blocks, ksplit, mat_first, nmat;
};
template <bool DUAL>
__device__ __forceinline__ PhaseDims phase_dims(const I8Args& a, int phase) {
  PhaseDims d;
  d.K = phase == 0 ? a.L.d_model : a.L.d_ff;
  d.N = phase == 0 ? a.L.d_ff : a.L.d_model;
  d.row_blocks = a.row_blocks[phase];
  d.ksplit = phase == 0 ? 1 : a.ksplit;
  d.mat_first = phase == 0 ? 0 : (DUAL ? 2 : 1);
  d.nmat = (DUAL && phase == 0) ? 2 : 1;
  return d;
}

// what a stage holds, written by the producer before it arms the stage's barrier
struct StageMeta {
  int e, rb, z, begin;
  int p0, ntok, k0, bits;
  int flags, phase, ai, nseg;
};
constexpr int META_FIRST = 1, META_LAST = 2, META_STOP = 4, META_EMPTY = 8, META_DONE = 16;

__device__ __forceinline__ int group_of(int k, int gshift, int G, int ngroups) {
  return ngroups == 1 ? 0 : (gshift >= 0 ? (k >> gshift) : k / G);
}

__device__ __forceinline__ bool wait_lim(uint32_t bar, uint32_t parity, unsigned limit, int* check_word,
                                         volatile int* abort_flag) {
  for (unsigned i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (i > 64) __nanosleep(40);
  }
  *abort_flag = 1;
  atomicOr(check_word, CHECK_WAIT_TIMEOUT);
  return false;
}

// the same for a whole warp: every lane polls, the answer is made uniform (the warp-wide
// instructions that follow a wait need all lanes on the same path, also when a wait runs out)
__device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity, unsigned limit, int* check_word,
                                          volatile int* abort_flag) {
  return __all_sync(0xffffffffu, wait_lim(bar, parity, limit, check_word, abort_flag) ? 1 : 0) != 0;
}

// ---- unpack: one 16-byte chunk of a packed row -> int8 words (code * 16 or code * 64) --------
__device__ __forceinline__ void unpack4(const uint4& v, uint32_t (&o)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[2 * i] = (w[i] << 4) & 0xF0F0F0F0u;  // nibbles 0 2 4 6 of the word
    o[2 * i + 1] = w[i] & 0xF0F0F0F0u;     // nibbles 1 3 5 7
  }
}
__device__ __forceinline__ void unpack2(const uint4& v, uint32_t (&o)[16]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[4 * i] = (w[i] << 6) & 0xC0C0C0C0u;      // fields 0 4 8 12 of the word
    o[4 * i + 1] = (w[i] << 4) & 0xC0C0C0C0u;  // fields 1 5 9 13
    o[4 * i + 2] = (w[i] << 2) & 0xC0C0C0C0u;  // fields 2 6 10 14
    o[4 * i + 3] = w[i] & 0xC0C0C0C0u;         // fields 3 7 11 15
  }
}

// a ring position and the parity of its current round
struct Ring {
  int i;
  uint32_t ph;
  __device__ __forceinline__ void next(int n) {
    if (++i == n) {
      i = 0;
      ph ^= 1u;
    }
  }
};

template <int NT, bool DUAL>
__global__ void __launch_bounds__(I8_THREADS, 1)
    ffn_i8_kernel(const __grid_constant__ I8Args a, const __grid_constant__ CUtensorMap tmap_x,
                  const __grid_constant__ CUtensorMap tmap_h) {
  constexpr int NMAT_MAX = DUAL ? 2 : 1;
  constexpr int NCOL = 2 * NT;                  // accumulator columns of one segment: hi and lo limb of NT tokens
  constexpr int NDBUF = I8_D_COLS / NCOL;       // accumulators in the ring
  constexpr int B_SEG_BYTES = NCOL * 128;       // activation tile of one segment
  static_assert(NDBUF <= I8_MAX_DBUF && NDBUF >= 4, "accumulator ring");
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * I8_MAX_STAGES + 4 + 2 * I8_MAX_DBUF + 1];
  __shared__ __align__(16) StageMeta meta[I8_MAX_STAGES];
  __shared__ __align__(16) uint32_t s_max[2][32][4];  // [item parity][token][epilogue warp]: largest |h| of the warp's rows
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const StageLayout SL = stage_layout(NT, NMAT_MAX);
  const int STAGES = a.stages;

  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * I8_MAX_STAGES;
  const uint32_t bar_afull = bar_empty + 8 * I8_MAX_STAGES, bar_aempty = bar_afull + 16;
  const uint32_t bar_dfull = bar_aempty + 16, bar_dempty = bar_dfull + 8 * I8_MAX_DBUF;
  const uint32_t bar_xchg = bar_dempty + 8 * I8_MAX_DBUF;

  if (threadIdx.x == 0) {
    abort_word = 0;
    for (int s = 0; s < I8_MAX_STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 33);  // the producer's lane 0 (+ TMA bytes) and every lane's small copies
      mbar_init(bar_empty + 8 * s, 5);  // the MMAs that read the stage (one commit) + the four epilogue warps
    }
    for (int w = 0; w < 2; ++w) {
      mbar_init(bar_afull + 8 * w, 4);   // the four warps of the unpack group
      mbar_init(bar_aempty + 8 * w, 1);  // commit of the MMAs that read the tile
    }
    for (int d = 0; d < I8_MAX_DBUF; ++d) {
      mbar_init(bar_dfull + 8 * d, 1);   // commit of the segment's MMAs
      mbar_init(bar_dempty + 8 * d, 4);  // the four epilogue warps have read it
    }
    mbar_init(bar_xchg, 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == I8_WARP_MMA) tmem_alloc(smem_u32(&tmem_base_slot), I8_TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  // everything above overlaps the tail of the kernel in front; the plan, the activations and (for
  // a launch of the second projection alone) the hidden vectors come from kernels of the chain
  pdl_wait();
  pdl_trigger();

  const LayerDims& L = a.L;
  PlanRec* recs = reinterpret_cast<PlanRec*>(reinterpret_cast<char*>(a.plan) + PLAN_HEADER_BYTES);
  const bool fused = a.phase_begin == 0 && a.phase_end == 2;
  const int ssz = L.scale_f16 ? 2 : 4;

  if (warp == I8_WARP_PRODUCER) {
    // ---------------- producer warp ----------------
    const int n_active = *reinterpret_cast<volatile const int*>(a.plan);
    const int n_items0 = a.phase_begin == 0 ? n_active * a.row_blocks[0] : 0;
    const int n_items1 = a.phase_end == 2 ? n_active * a.row_blocks[1] * a.ksplit : 0;
    const int n_items = n_items0 + n_items1;
    Ring ring{0, 0};
    bool ok = true;
    int item = blockIdx.x;  // a CTA's first item is its own index; the counter hands out the rest
    while (ok) {
      if (item >= n_items || __any_sync(0xffffffffu, *abort_flag != 0)) break;
      const int phase = item < n_items0 ? 0 : 1;
      const int li = item - (phase == 0 ? 0 : n_items0);
      const PhaseDims pd = phase_dims<DUAL>(a, phase);
      const int K = pd.K;
      const int ngroups_k = a.ngroups[phase];
      const int ai = li / (pd.ksplit * pd.row_blocks);
      const PlanRec rec = recs[ai];
      const int z = li % pd.ksplit;
      const int rb = (li / pd.ksplit) % pd.row_blocks;
      const CUtensorMap* maps = a.wmaps + static_cast<size_t>(rec.e) * 3;
      const CUtensorMap* bmap = phase == 0 ? &tmap_x : &tmap_h;
      const float* act_scale = phase == 0 ? a.xsc : a.hsc;
      const int nblk = K / 128;  // activation blocks per row
      const int bits = rec.bits;
      const int kspan = 1024 / bits;
      const int steps_total = (K + kspan - 1) / kspan;
      const int spz = (steps_total + pd.ksplit - 1) / pd.ksplit;
      const int step_begin = z * spz;
      const int nsteps = max(0, min(steps_total, step_begin + spz) - step_begin);
      const int npass = (rec.cnt + NT - 1) / NT;
      const int row0 = rb * I8_ROWS;
      bool need_dep = fused && phase == 1;
      // scale rows this lane copies (rows 4l .. 4l+3 of every matrix of the stage): byte offset of
      // the row's scale channel from its 4-byte-aligned base
      int srow_off[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) srow_off[r] = min(row0 + 4 * lane + r, pd.N - 1) * ngroups_k * ssz;
      for (int pass = 0; pass < npass && ok; ++pass) {
        const int p0 = pass * NT;
        const int ntok = min(NT, rec.cnt - p0);
        const int nst = max(nsteps, 1);  // an empty split-K slice still has to store its zeros
        for (int s = 0; s < nst; ++s) {
          if (!wait_warp(bar_empty + 8 * ring.i, ring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
            ok = false;
            break;
          }
          unsigned char* st = smem + ring.i * SL.bytes;
          const uint32_t full = bar_full + 8 * ring.i;
          const int k0 = (step_begin + s) * kspan;
          const int klen = nsteps > 0 ? min(kspan, K - k0) : 0;
          const int nseg = klen / 128;
          if (lane == 0) {
            const int flags = (s == 0 ? META_FIRST : 0) | (s == nst - 1 ? META_LAST : 0) | (klen == 0 ? META_EMPTY : 0) |
                              (fused && phase == 0 && s == nst - 1 && pass == npass - 1 ? META_DONE : 0);
            uint4* mq = reinterpret_cast<uint4*>(&meta[ring.i]);
            mq[0] = make_uint4(rec.e, rb, z, rec.begin);
            mq[1] = make_uint4(p0, ntok, k0, bits);
            mq[2] = make_uint4(flags, phase, ai, nseg);
            if (klen > 0) {
              mbar_expect_tx(full, pd.nmat * I8_MAT_BYTES + nseg * B_SEG_BYTES);
              const int c0 = k0 * bits / 8;
              for (int m = 0; m < pd.nmat; ++m) {
                const CUtensorMap* mp = maps + pd.mat_first + m;
                tma_load_2d(smem_u32(st + m * I8_MAT_BYTES), mp, c0, row0, full);
                tma_load_2d(smem_u32(st + m * I8_MAT_BYTES + I8_BOX_BYTES), mp, c0, row0 + I8_BOX_ROWS, full);
              }
            } else {
              mbar_arrive(full);
            }
          }
          __syncwarp();
          if (klen > 0) {
            // weight scales: lane l copies the windows of rows 4l .. 4l+3 of every matrix
            const int g0 = group_of(k0, a.gshift, L.group, ngroups_k),
                      g1 = group_of(k0 + (nseg - 1) * 128, a.gshift, L.group, ngroups_k);
            const uint32_t sdst = smem_u32(st + SL.sc_off);
            for (int m = 0; m < pd.nmat; ++m) {
              const char* sbase = static_cast<const char*>(rec.scales[pd.mat_first + m]);
#pragma unroll
              for (int r = 0; r < 4; ++r) {
                const int b0 = (srow_off[r] + g0 * ssz) & ~3;
                const int b1 = srow_off[r] + (g1 + 1) * ssz;
#pragma unroll 1
                for (int w = 0; b0 + 4 * w < b1; ++w)
                  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sdst + (m * I8_ROWS + 4 * lane + r) * 16 + 4 * w),
                               "l"(sbase + b0 + 4 * w)
                               : "memory");
              }
            }
            if (need_dep) {
              // codes and scales of the stage are on their way; the hidden vectors may still be in the
              // making on other SMs.  Every lane acquires the counter itself, so that its own copies
              // below are ordered behind the writers' stores.
              need_dep = false;
              const int expect = a.row_blocks[0] * 4 + a.dep_extra;
              const int* done = &recs[ai].done;
              bool ready = false;
              for (unsigned i = 0; i < a.dep_wait_limit; ++i) {
                int v;
                asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(done) : "memory");
                ready = __all_sync(0xffffffffu, v >= expect);
                if (ready || __any_sync(0xffffffffu, *abort_flag != 0)) break;
                __nanosleep(100);
              }
              if (!ready) {
                if (lane == 0) {
                  *abort_flag = 1;
                  atomicOr(a.check_word, CHECK_WAIT_TIMEOUT);
                }
                ok = false;
                // the stage's barrier stays incomplete: nobody consumes it, the copies already issued
                // land in the CTA's own shared memory during the wind-down pause
                break;
              }
              asm volatile("fence.proxy.async;" ::: "memory");  // generic-proxy stores -> TMA reads
            }
            // activation block scales of the tile's tokens
            if (lane < ntok) {
              const float* src = act_scale + static_cast<size_t>(rec.begin + p0 + lane) * nblk + k0 / 128;
              const uint32_t xdst = smem_u32(st + SL.sx_off) + lane * 4;
              for (int sg = 0; sg < nseg; ++sg)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(xdst + sg * 128), "l"(src + sg) : "memory");
            }
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(full) : "memory");
            if (lane == 0) {
              // the tokens' limb rows: rows 2*slot (hi) and 2*slot+1 (lo) of the activation image
              for (int sg = 0; sg < nseg; ++sg)
                tma_load_2d(smem_u32(st + SL.b_off + sg * B_SEG_BYTES), bmap, k0 + sg * 128, 2 * (rec.begin + p0), full);
            }
          } else {
            mbar_arrive(full);  // with lane 0's arrival above: 33 in all
          }
          ring.next(STAGES);
        }
      }
      // the ring still holds several stages of work: fetching the next item only now costs nothing
      // and no CTA sits on items it is not yet working on
      int item_next = 0;
      if (lane == 0) item_next = gridDim.x + atomicAdd(a.plan + 1 + a.phase_begin, 1);
      item = __shfl_sync(0xffffffffu, item_next, 0);
    }
    if (ok && !__any_sync(0xffffffffu, *abort_flag != 0)) {  // tell the others that nothing else comes
      if (wait_warp(bar_empty + 8 * ring.i, ring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
        if (lane == 0) {
          meta[ring.i].flags = META_STOP;
          mbar_arrive(bar_full + 8 * ring.i);  // lane 0 arrives twice: once for itself, once in place of a copy
        }
        __syncwarp();
        mbar_arrive(bar_full + 8 * ring.i);
      }
    }
  } else if (warp == I8_WARP_MMA) {
    // ---------------- MMA issuer (one lane) ----------------
    if (lane == 0) {
      // kind::i8: s8 x s8 -> s32, both operands K-major, M = 128, N = 2 * NT
      const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((static_cast<uint32_t>(NCOL) >> 3) << 17) |
                             ((static_cast<uint32_t>(I8_ROWS) >> 4) << 24);
      Ring ring{0, 0}, dring{0, 0};
      uint32_t q = 0;  // A tiles that went through tensor memory so far
      bool ok = true;
      while (ok) {
        if (!wait_lim(bar_full + 8 * ring.i, ring.ph, a.wait_limit, a.check_word, abort_flag)) break;
        tc_fence_after();
        const StageMeta m = meta[ring.i];
        if (m.flags & META_STOP) break;
        if (m.flags & META_EMPTY) {
          mbar_arrive(bar_empty + 8 * ring.i);
          ring.next(STAGES);
          continue;
        }
        const uint32_t st = smem_u32(smem + ring.i * SL.bytes);
        const int nmat = (DUAL && m.phase == 0) ? 2 : 1;
        for (int mt = 0; mt < nmat && ok; ++mt) {
          const uint32_t abuf = q & 1u;
          if (m.bits != 8) {
            if (!wait_lim(bar_afull + 8 * abuf, (q >> 1) & 1u, a.wait_limit, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            tc_fence_after();
          }
          const uint64_t adesc = umma_desc(st + mt * I8_MAT_BYTES);
          for (int sg = 0; sg < m.nseg; ++sg) {
            if (!wait_lim(bar_dempty + 8 * dring.i, dring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + I8_D_COL0 + dring.i * NCOL;
            const uint64_t bdesc = umma_desc(st + SL.b_off + sg * B_SEG_BYTES);
#pragma unroll
            for (int j = 0; j < 4; ++j) {  // 32 inputs per MMA
              if (m.bits == 8)
                umma_i8_ss(d_tmem, adesc + 2 * j, bdesc + 2 * j, idesc, j > 0 ? 1u : 0u);
              else
                umma_i8_ts(d_tmem, tmem_base + abuf * I8_A_COLS + sg * 32 + j * 8, bdesc + 2 * j, idesc, j > 0 ? 1u : 0u);
            }
            umma_commit(bar_dfull + 8 * dring.i);
            dring.next(NDBUF);
          }
          if (!ok) break;
          if (m.bits != 8) {
            umma_commit(bar_aempty + 8 * abuf);
            ++q;
          }
        }
        if (!ok) break;
        umma_commit(bar_empty + 8 * ring.i);  // the stage's shared memory may be refilled once these MMAs have read it
        ring.next(STAGES);
      }
    }
  } else if (warp >= I8_WARP_UNPACK0) {
    // ---------------- unpack warps: packed codes -> int8 rows in tensor memory ----------------
    const uint32_t wg = static_cast<uint32_t>(warp - I8_WARP_UNPACK0) >> 2;  // 0 or 1: which A tile is ours
    const int r = 32 * (warp & 3) + lane;                                    // row of the item = tensor-memory lane
    const uint32_t a_tmem = tmem_base + (static_cast<uint32_t>(32 * (warp & 3)) << 16) + wg * I8_A_COLS;
    const int row_off = (r >> 6) * I8_BOX_BYTES + (r & 63) * 128;
    const int swz = r & 7;
    Ring ring{0, 0};
    uint32_t q = 0, uses = 0;
    bool ok = true;
    while (ok) {
      if (!wait_warp(bar_full + 8 * ring.i, ring.ph, a.wait_limit, a.check_word, abort_flag)) break;
      const int flags = meta[ring.i].flags;
      if (flags & META_STOP) break;
      const int bits = meta[ring.i].bits, nseg = meta[ring.i].nseg, phase = meta[ring.i].phase;
      if (!(flags & META_EMPTY) && bits != 8) {
        const int nmat = (DUAL && phase == 0) ? 2 : 1;
        for (int mt = 0; mt < nmat; ++mt, ++q) {
          if ((q & 1u) != wg) continue;
          if (!wait_warp(bar_aempty + 8 * wg, (uses & 1u) ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const unsigned char* row = smem + ring.i * SL.bytes + mt * I8_MAT_BYTES + row_off;
          if (bits == 4) {
            // a 16-byte chunk = 32 codes = 8 columns; 4 chunks per 128-input segment
#pragma unroll 2
            for (int c = 0; c < 4 * nseg; ++c) {
              uint32_t o[8];
              unpack4(*reinterpret_cast<const uint4*>(row + ((c ^ swz) << 4)), o);
              tmem_st8(a_tmem + 8 * c, o);
            }
          } else {
            // a 16-byte chunk = 64 codes = 16 columns; 2 chunks per segment
#pragma unroll 2
            for (int c = 0; c < 2 * nseg; ++c) {
              uint32_t o[16];
              unpack2(*reinterpret_cast<const uint4*>(row + ((c ^ swz) << 4)), o);
              tmem_st16(a_tmem + 16 * c, o);
            }
          }
          tmem_st_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_afull + 8 * wg);
          ++uses;
        }
      }
      ring.next(STAGES);
    }
  } else {
    // ---------------- epilogue warps: one thread per output row ----------------
    const int r = 32 * warp + lane;
    const uint32_t d_tmem0 = tmem_base + (static_cast<uint32_t>(32 * warp) << 16) + I8_D_COL0;
    float tot[NMAT_MAX][NT];
    Ring ring{0, 0}, dring{0, 0};
    uint32_t exchanges = 0;  // first-projection items finished so far (each uses the exchange barrier once)
    bool ok = true;
    while (ok) {
      if (!wait_warp(bar_full + 8 * ring.i, ring.ph, a.wait_limit, a.check_word, abort_flag)) break;
      const StageMeta m = meta[ring.i];
      if (m.flags & META_STOP) break;
      if (m.flags & META_FIRST) {
#pragma unroll
        for (int mt = 0; mt < NMAT_MAX; ++mt)
#pragma unroll
          for (int t = 0; t < NT; ++t) tot[mt][t] = 0.0f;
      }
      const int N = m.phase == 0 ? L.d_ff : L.d_model;
      const int n = m.rb * I8_ROWS + r;
      if (!(m.flags & META_EMPTY)) {
        const unsigned char* st = smem + ring.i * SL.bytes;
        const int nmat = (DUAL && m.phase == 0) ? 2 : 1;
        const int ngroups = a.ngroups[m.phase];
        const int g0 = group_of(m.k0, a.gshift, L.group, ngroups);
        // the row's scale window starts at the 4-byte boundary at or below its first scale of the stage
        const unsigned char* sc_row = st + SL.sc_off + r * 16 + (((min(n, N - 1) * ngroups + g0) * ssz) & 3);
        const float unit = m.bits == 8 ? 1.0f : (m.bits == 4 ? 0.0625f : 0.015625f);  // codes arrive as 16 q / 64 q
#pragma unroll
        for (int mt = 0; mt < NMAT_MAX; ++mt) {
          if (mt >= nmat || !ok) break;
#pragma unroll 1
          for (int sg = 0; sg < m.nseg; ++sg) {
            if (!wait_warp(bar_dfull + 8 * dring.i, dring.ph, a.wait_limit, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const unsigned char* sc = sc_row + mt * I8_SCALE_BYTES + (group_of(m.k0 + sg * 128, a.gshift, L.group, ngroups) - g0) * ssz;
            const float sw = unit * (ssz == 2 ? __half2float(*reinterpret_cast<const __half*>(sc))
                                              : *reinterpret_cast<const float*>(sc));
            const float* sx = reinterpret_cast<const float*>(st + SL.sx_off) + sg * 32;
            const uint32_t d_tmem = d_tmem0 + dring.i * NCOL;
#pragma unroll
            for (int half = 0; half < (NT + 15) / 16; ++half) {
              constexpr int TT = NT < 16 ? NT : 16;  // tokens per read
              uint32_t acc[2 * TT];
              if constexpr (TT == 8) tmem_ld16(d_tmem, acc);
              else tmem_ld32(d_tmem + half * 32, acc);
              tmem_ld_wait();
              if (half == (NT + 15) / 16 - 1) {  // the accumulator may be overwritten
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_dempty + 8 * dring.i);
              }
#pragma unroll
              for (int t = 0; t < TT; ++t) {
                if (half * 16 + t < m.ntok) {
                  const int v = static_cast<int>(acc[2 * t]) * 128 + static_cast<int>(acc[2 * t + 1]);
                  tot[mt][half * 16 + t] = fmaf(static_cast<float>(v), sw * sx[half * 16 + t], tot[mt][half * 16 + t]);
                }
              }
            }
            dring.next(NDBUF);
          }
        }
        if (!ok) break;
      }
      // the stage's scales are no longer needed
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * ring.i);
      if (m.flags & META_LAST) {
        if (m.phase == 0) {
          // hidden values of this row: activation, rounded to bf16 (the hidden vector is a bf16
          // tensor), then to limbs under the block scale of the item's 128 rows
          float h[NT];
          const uint32_t par = exchanges & 1u;
          ++exchanges;
#pragma unroll
          for (int t = 0; t < NT; ++t) {
            float v;
            if (DUAL) {
              const float av = tot[0][t], bv = tot[NMAT_MAX - 1][t];
              v = av / (1.0f + expf(-av)) * bv;
            } else {
              v = fmaxf(tot[0][t], 0.0f);
            }
            h[t] = (t < m.ntok && n < N) ? __bfloat162float(__float2bfloat16_rn(v)) : 0.0f;
            const uint32_t mx = redux_max_u32(__float_as_uint(h[t]) & 0x7fffffffu);
            if (lane == 0) s_max[par][t][warp] = mx;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_xchg);
          if (!wait_warp(bar_xchg, par, a.wait_limit, a.check_word, abort_flag)) break;
          const int col = m.rb * I8_ROWS + act_q_pos_rt(m.bits, r);
#pragma unroll
          for (int t = 0; t < NT; ++t) {
            if (t < m.ntok) {
              const uint4 mw = *reinterpret_cast<const uint4*>(&s_max[par][t][0]);
              const int E = act_q_block_exp(max(max(mw.x, mw.y), max(mw.z, mw.w)));
              const size_t slot = static_cast<size_t>(m.begin + m.p0 + t);
              if (n < N) {
                const int v = act_q_int(h[t], act_q_inv_scale(E));
                a.hq[(2 * slot) * N + col] = static_cast<int8_t>(v >> 7);
                a.hq[(2 * slot + 1) * N + col] = static_cast<int8_t>(v & 127);
              }
              if (r == t) a.hsc[slot * (N / 128) + m.rb] = act_q_scale(E);
            }
          }
          if (m.flags & META_DONE) {
            // this warp's share of the expert's hidden vectors is written: make it visible to the
            // copies of other SMs (release), then count it
            asm volatile("fence.proxy.async;" ::: "memory");
            __syncwarp();
            if (lane == 0)
              asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(&recs[m.ai].done), "r"(1) : "memory");
          }
        } else if (n < N) {
#pragma unroll
          for (int t = 0; t < NT; ++t)
            if (t < m.ntok)
              a.o_part[(static_cast<size_t>(m.z) * a.n_pairs + (m.begin + m.p0 + t)) * N + n] = tot[0][t];
        }
      }
      ring.next(STAGES);
    }
  }

  // wind-down: after a wait that ran out, give copies and MMAs in flight time to land before the
  // CTA's shared and tensor memory are released
  if (*abort_flag) {
#pragma unroll 1
    for (int i = 0; i < 2000; ++i) __nanosleep(100);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == I8_WARP_MMA) {
    tc_fence_after();
    tmem_dealloc(tmem_base, I8_TMEM_COLS);
  }
}

int stages_for(int nt, int nmat) {
  const StageLayout sl = stage_layout(nt, nmat);
  int s = (I8_SMEM_LIMIT - 1024 /*alignment slack*/ - 3072 /*static*/) / sl.bytes;
  return s > I8_MAX_STAGES ? I8_MAX_STAGES : s;
}

template <int NT, bool DUAL>
cudaError_t launch_variant(const I8Args& a_in, const CUtensorMap& tx, const CUtensorMap& th, long long items, cudaStream_t st) {
  static int sms_of_device[64] = {};
  I8Args a = a_in;
  a.stages = stages_for(NT, DUAL ? 2 : 1);
  if (a.stages < 3) return cudaErrorInvalidValue;
  const int smem = a.stages * stage_layout(NT, DUAL ? 2 : 1).bytes + 1024;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!sms_of_device[dev]) {
    e = cudaFuncSetAttribute(ffn_i8_kernel<NT, DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    sms_of_device[dev] = sms;
  }
  // one CTA per SM: more than half of an SM's shared memory per CTA keeps a second one out (a CTA
  // that holds an item but waits for tensor memory would stall the experts that depend on it)
  if (smem <= 116 * 1024) return cudaErrorInvalidValue;
  const int grid = static_cast<int>(items < sms_of_device[dev] ? items : sms_of_device[dev]);
  return launch_chain(ffn_i8_kernel<NT, DUAL>, dim3(grid), dim3(I8_THREADS), smem, st, a, tx, th);
}

}  // namespace

bool ffn_i8_supported(const LayerDims& L) {
  // bf16 activations, inputs in whole 128-blocks, scale groups of whole blocks; the tensor maps use
  // 128-byte x 64-row boxes: every packed row must hold at least 128 bytes at the narrowest width
  return ffn_mma_supported(L) && L.d_model >= 512 && L.d_ff >= 512;
}

// tokens per tile (columns of the B operand / 2): the epilogue's work per segment grows with the
// tile, an expert with more tokens than the tile takes another pass over its weights (from L2)
int ffn_i8_token_tile(const LayerDims& L, int T) {
  const double mean = static_cast<double>(T) * L.top_k / L.E;
  return mean <= 6.0 ? 8 : (mean <= 12.0 ? 16 : 32);
}

int ffn_i8_ksplit(const LayerDims& L, int T) {
  const int row_blocks = (L.d_model + I8_ROWS - 1) / I8_ROWS;
  const long long pairs = static_cast<long long>(T) * L.top_k;
  const long long active = pairs < L.E ? pairs : L.E;
  const long long units = row_blocks * active;
  // enough slices that the second projection's items outnumber the CTAs (one per SM) about three
  // times: short items at the end of the launch keep its tail short
  long long z = (3 * 148 + units - 1) / units;
  const int steps_min = (L.d_ff + 511) / 512;  // stages at the widest span (2 bits)
  const int steps_max = (L.d_ff + 127) / 128;
  const int cap = units * 2 <= 148 ? steps_max : steps_min;
  if (z > cap) z = cap;
  if (z > 16) z = 16;
  if (z < 1) z = 1;
  return static_cast<int>(z);
}

cudaError_t launch_ffn_i8(int phase_begin, int phase_end, const LayerDims& L, const void* wmaps, const void* xq,
                          const float* xsc, int* plan, void* hq, float* hsc, float* o_part, int ksplit, int n_pairs,
                          int T, int token_tile, unsigned wait_limit, int dep_extra, int* check_word, cudaStream_t st) {
  if (phase_begin < 0 || phase_end > 2 || phase_begin >= phase_end) return cudaErrorInvalidValue;
  const int nt = token_tile > 0 ? token_tile : ffn_i8_token_tile(L, T);
  I8Args a;
  a.phase_begin = phase_begin;
  a.phase_end = phase_end;
  a.L = L;
  a.wmaps = static_cast<const CUtensorMap*>(wmaps);
  a.plan = plan;
  a.xsc = xsc;
  a.hq = static_cast<int8_t*>(hq);
  a.hsc = hsc;
  a.o_part = o_part;
  a.ksplit = ksplit;
  a.row_blocks[0] = (L.d_ff + I8_ROWS - 1) / I8_ROWS;
  a.row_blocks[1] = (L.d_model + I8_ROWS - 1) / I8_ROWS;
  a.ngroups[0] = L.group > 0 ? L.d_model / L.group : 1;
  a.ngroups[1] = L.group > 0 ? L.d_ff / L.group : 1;
  a.gshift = -1;
  for (int b = 7; b < 31; ++b)
    if (L.group == (1 << b)) a.gshift = b;
  a.n_pairs = n_pairs;
  a.stages = 0;
  a.wait_limit = wait_limit ? wait_limit : PIPE_WAIT_LIMIT;
  a.dep_wait_limit = wait_limit ? wait_limit : (1u << 20);
  a.dep_extra = dep_extra;
  a.check_word = check_word;
  // activation images: [2 * n_pairs rows][K bytes], boxes of 2*nt rows x 128 bytes, 128-byte swizzle
  CUtensorMap tx, th;
  if (encode_tmap_2d(&tx, 0, xq, static_cast<uint64_t>(L.d_model), 2ull * n_pairs, static_cast<uint64_t>(L.d_model), 128, 2 * nt) != 0)
    return cudaErrorInvalidValue;
  if (encode_tmap_2d(&th, 0, hq, static_cast<uint64_t>(L.d_ff), 2ull * n_pairs, static_cast<uint64_t>(L.d_ff), 128, 2 * nt) != 0)
    return cudaErrorInvalidValue;
  const long long active_max = n_pairs < L.E ? n_pairs : L.E;
  long long per_expert = 0;
  if (phase_begin == 0) per_expert += a.row_blocks[0];
  if (phase_end == 2) per_expert += static_cast<long long>(a.row_blocks[1]) * ksplit;
  const long long items = active_max * per_expert;
  const bool dual = L.act == EMOE_ACT_SWIGLU;
  if (nt == 8) return dual ? launch_variant<8, true>(a, tx, th, items, st) : launch_variant<8, false>(a, tx, th, items, st);
  if (nt == 16) return dual ? launch_variant<16, true>(a, tx, th, items, st) : launch_variant<16, false>(a, tx, th, items, st);
  if (nt == 32) return dual ? launch_variant<32, true>(a, tx, th, items, st) : launch_variant<32, false>(a, tx, th, items, st);
  return cudaErrorInvalidValue;
}

}  // namespace emoe
