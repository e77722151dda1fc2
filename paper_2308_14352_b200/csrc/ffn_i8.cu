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
// are complete.
// Warp roles and rings (every ring has full/empty mbarriers, every wait is bounded: a wait that
// runs out sets CHECK_WAIT_TIMEOUT and the CTA winds down):
//   producer warp     walks the items; per stage: a record of what the stage holds into the deeper
//                     SIDE ring, then the weight boxes by TMA into the STAGE ring (shared memory,
//                     128 bytes of every row of 1 or 2 matrices per stage);
//   feeder warp       follows the records: the tokens' limb rows (TMA, into the stage) and their
//                     block scales (into the side ring); it is the one that waits for an expert's
//                     hidden vectors, so the weights never wait for them.  (Every step of these
//                     chains is a shared-memory or copy-engine operation of a hundred cycles and
//                     more under load: one warp doing all of it could not fill a stage in time.)
//   unpack warps      2 x 4 warps, one thread per row: a 4- or 2-bit stage, one 128-input segment
//                     at a time, into the A ring (8 segments of 32 columns in tensor memory);
//   MMA warps         one thread each: four K=32 MMAs per segment into the accumulator ring (groups
//                     of up to four segments of one matrix), commits release A segments, stages
//                     and publish accumulator groups.  Issuing an MMA costs the thread some fifty
//                     cycles and a 2-bit stream needs one every sixty, so two threads take the
//                     accumulator groups in turn (each feeds one group of epilogue warps);
//                     In the general scale mode (SCALE_STAGE) it also copies, with cp.async, the few
//                     bytes of weight scales every row needs for the stage into the SCALE ring: under
//                     load a global load takes a microsecond, so the scales travel as far ahead as
//                     the weights do;
//   epilogue warps    2 x 4 warps, one thread per output row (= tensor-memory lane) in each group of
//                     four: accumulator groups -> registers -> scaled fp32 totals.  The two groups
//                     of warps take the accumulator groups in turn (their per-group work is a chain
//                     of dependent steps: waits, a tensor-memory load, a few multiply-adds, so two
//                     such chains per scheduler run twice as fast as one); at the end of an item the
//                     second hands its partial totals to the first through shared memory.  They
//                     work from the side and scale rings only, so a stage's shared memory is free
//                     again as soon as its MMAs have read it, however far the epilogue lags.
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
constexpr int I8_WARP_UNPACK0 = 8;                   // warps 0-3 and 4-7 epilogue, 8-11 and 12-15 unpack
constexpr int I8_WARP_PRODUCER = 16;
constexpr int I8_WARP_MMA = 17;
constexpr int I8_WARP_MMA1 = 18;                     // the second MMA-issuing warp
constexpr int I8_WARP_FEEDER = 19;                   // the activation feeder
constexpr int I8_THREADS = 20 * 32;
constexpr int I8_MAX_STAGES = 8;
constexpr int I8_SIDE = 16;                          // entries of the side ring
// Weight scales travel ahead of their use in one of three ways, chosen per projection on the host:
//   SCALE_BLOCK   a row's whole scale channel is at most 32 bytes: the 128 rows of an item are one
//                 contiguous block, fetched by one bulk copy per matrix and item pass;
//   SCALE_WINDOW  longer rows whose length is a multiple of 16 bytes: 32-byte windows of the 128 rows
//                 (16 fp16 scales = 2048 inputs), one TMA box per matrix whenever the inputs move
//                 into the next window;
//   SCALE_STAGE   anything else (odd row lengths, unaligned channels, group sizes that are not a
//                 power of two): a warp copies each stage's few bytes per row with cp.async.
// The first two cost one instruction per matrix and thousands of inputs; the third is the slow,
// general path.
constexpr int SCALE_BLOCK = 0, SCALE_WINDOW = 1, SCALE_STAGE = 2;
constexpr int I8_CHUNKS = 4;                         // entries of the scale ring in the first two modes
constexpr int I8_CHUNK_ROW = 32;                     // bytes per row of an entry
constexpr int I8_CHUNK_BYTES = I8_ROWS * I8_CHUNK_ROW;  // one matrix of one entry: 4 KB
constexpr int I8_SCALE_RING = 8;                     // entries of the ring in the third mode
constexpr int I8_SCALE_TILE = I8_ROWS * 16;          // one matrix of one stage: a 16-byte window per row
constexpr int I8_TMEM_COLS = 512;
constexpr int I8_A_SLOTS = 8;                        // A ring: unpacked 128-input segments, 32 columns each
constexpr int I8_A_SLOT_COLS = 32;
constexpr int I8_D_COL0 = I8_A_SLOTS * I8_A_SLOT_COLS;  // accumulators behind the A ring
constexpr int I8_D_COLS = I8_TMEM_COLS - I8_D_COL0;     // 256 columns of accumulators
constexpr int I8_MAX_GROUPS = 4;
constexpr int I8_SMEM_LIMIT = 227 * 1024;
constexpr int I8_STATIC_SMEM = 12 * 1024;            // barriers, side ring, exchange buffer (upper bound)

// a shared-memory stage: weight boxes of 1 or 2 matrices | limb tiles of up to 4 segments
// (2*NT rows x 128 bytes each)
__host__ __device__ constexpr int stage_b_off(int nmat) { return nmat * I8_MAT_BYTES; }
__host__ __device__ constexpr int stage_bytes(int nt, int nmat) { return nmat * I8_MAT_BYTES + 4 * (2 * nt) * 128; }

struct I8Args {
  int phase_begin, phase_end;  // projections this launch runs: [0,1), [1,2) or both, [0,2)
  LayerDims L;
  const CUtensorMap* wmaps;  // [E][3] packed-weight maps: byte image [N][K*bits/8], boxes 64 rows x 128 bytes
  const CUtensorMap* smaps;  // [E][3] scale-channel maps: byte image [N][row bytes], boxes 128 rows x 32 bytes (SCALE_WINDOW)
  int scale_mode[2];         // per projection: SCALE_BLOCK / SCALE_WINDOW / SCALE_STAGE
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
  long long* prof;          // per-CTA timers of a profiling build, else null
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

// what a stage holds, written by the producer before it publishes the stage
struct StageMeta {
  int e, rb, z, begin;
  int p0, ntok, k0, bits;
  int flags, phase, ai, nseg;
  const void* scales[2];  // scale channels of the stage's matrices
  int chunk, win0, pitch;  // scale-ring entry of the stage, first byte of a row it holds, bytes per row in it
  uint32_t sc_rel;         // byte distance of the scale of segment 0..3 from that of segment 0, 8 bits each
  uint32_t sc_addr;        // shared-memory address of row 0's scale of segment 0 (block and window modes)
  int pad[3];
};
constexpr int META_FIRST = 1, META_LAST = 2, META_STOP = 4, META_EMPTY = 8, META_DONE = 16;
constexpr int META_NEW_CHUNK = 32;  // the stage is the first to use its scale-ring entry
constexpr int META_END_CHUNK = 64;  // ... the last
constexpr int META_DEP = 128;       // the stage's activations are hidden vectors that may still be in the making

// an entry of the side ring: the record of a stage and the block scales of its tokens' limbs
struct SideEntry {
  StageMeta m;
  float sx[4][32];  // [segment][token]
};

__device__ __forceinline__ int group_of(int k, int gshift, int G, int ngroups) {
  return ngroups == 1 ? 0 : (gshift >= 0 ? (k >> gshift) : k / G);
}

__device__ __forceinline__ bool wait_lim(uint32_t bar, uint32_t parity, unsigned limit, int* check_word,
                                         volatile int* abort_flag) {
  // Most of a CTA's warps wait at any time.  A warp that polls in a tight loop takes issue slots
  // and shared-memory cycles from the few that work (measured: a third of all issue slots), so a
  // wait that is not over at once backs off: sleeps of 32, 64, ... up to 1024 ns between polls.
  if (mbar_try_wait(bar, parity)) return true;
  unsigned ns = 32;
  for (unsigned i = 0; i < limit; ++i) {
    __nanosleep(ns);
    if (ns < 1024) ns += ns;
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 3u) == 3u && *abort_flag) return false;
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

// Optional per-CTA timers (build with -DEMOE_I8_PROFILE; the buffer is set by
// emoe_debug_set_profile_buffer): cycles each role spends in its waits, read with clock64.
#ifdef EMOE_I8_PROFILE
#define PROF_DECL long long prof_t0 = 0, prof_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}
#define PROF_BEGIN prof_t0 = clock64()
#define PROF_END(i) prof_acc[i] += clock64() - prof_t0
#define PROF_STORE(base, n)                                                     \
  if (a.prof && lane == 0)                                                      \
    for (int pi = 0; pi < (n); ++pi) a.prof[blockIdx.x * 32 + (base) + pi] = prof_acc[pi]
#define PROF_LAP(i)                    \
  {                                    \
    const long long now__ = clock64(); \
    prof_acc[i] += now__ - prof_t0;    \
    prof_t0 = now__;                   \
  }
#else
#define PROF_DECL
#define PROF_BEGIN
#define PROF_END(i)
#define PROF_STORE(base, n)
#define PROF_LAP(i)
#endif

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
  constexpr int NCOL = 2 * NT;                 // accumulator columns of one segment: hi and lo limb of NT tokens
  constexpr int GSEGS = NT == 32 ? 2 : 4;      // segments of one accumulator group
  constexpr int GCOLS = GSEGS * NCOL;          // 64 / 128 / 128 columns
  constexpr int NGRP = I8_D_COLS / GCOLS;      // groups in the ring: 4 / 2 / 2
  constexpr int B_SEG_BYTES = NCOL * 128;      // limb tile of one segment
  constexpr int STAGE_BYTES = stage_bytes(NT, NMAT_MAX);
  constexpr int B_OFF = stage_b_off(NMAT_MAX);
  static_assert(NGRP >= 2 && NGRP <= I8_MAX_GROUPS, "accumulator ring");
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * I8_MAX_STAGES + 2 * I8_SIDE + 2 * I8_A_SLOTS + 2 * I8_MAX_GROUPS + 1 + 2 * I8_SCALE_RING +
                                        2 * I8_CHUNKS + 2 + I8_SIDE];
  __shared__ __align__(16) SideEntry side[I8_SIDE];
  __shared__ __align__(16) uint32_t s_max[2][32][4];  // [item parity][token][epilogue warp]: largest |h| of the warp's rows
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int STAGES = a.stages;

  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * I8_MAX_STAGES;
  const uint32_t bar_sfull = bar_empty + 8 * I8_MAX_STAGES, bar_sempty = bar_sfull + 8 * I8_SIDE;
  const uint32_t bar_afull = bar_sempty + 8 * I8_SIDE, bar_aempty = bar_afull + 8 * I8_A_SLOTS;
  const uint32_t bar_dfull = bar_aempty + 8 * I8_A_SLOTS, bar_dempty = bar_dfull + 8 * I8_MAX_GROUPS;
  const uint32_t bar_xchg = bar_dempty + 8 * I8_MAX_GROUPS;
  const uint32_t bar_wfull = bar_xchg + 8, bar_wempty = bar_wfull + 8 * I8_SCALE_RING;
  const uint32_t bar_cfull = bar_wempty + 8 * I8_SCALE_RING, bar_cempty = bar_cfull + 8 * I8_CHUNKS;
  const uint32_t bar_xfull = bar_cempty + 8 * I8_CHUNKS, bar_xempty = bar_xfull + 8;
  const uint32_t bar_mready = bar_xempty + 8;
  // the scale ring sits behind the stages in dynamic shared memory (entries of either kind)
  unsigned char* scale_ring = smem + STAGES * STAGE_BYTES;
  constexpr int SCALE_ENTRY = NMAT_MAX * I8_SCALE_TILE;
  constexpr int CHUNK_ENTRY = NMAT_MAX * I8_CHUNK_BYTES;
  // behind it: the partial totals the second group of epilogue warps hands to the first, [matrix][token][row]
  float* xbuf = reinterpret_cast<float*>(scale_ring + I8_SCALE_RING * SCALE_ENTRY);

  if (threadIdx.x == 0) {
    abort_word = 0;
    for (int s = 0; s < I8_MAX_STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);   // the producer's lane 0 (+ the bytes of its TMA copies)
      mbar_init(bar_empty + 8 * s, 10);  // the two MMA warps (a commit each, or a plain arrival) + the eight unpack warps
    }
    for (int s = 0; s < I8_SIDE; ++s) {
      mbar_init(bar_sfull + 8 * s, 32);   // every lane of the feeder warp, after its small copies
      mbar_init(bar_mready + 8 * s, 1);   // the producer: the record is written
      mbar_init(bar_sempty + 8 * s, 8);  // the eight epilogue warps
    }
    for (int s = 0; s < I8_A_SLOTS; ++s) {
      mbar_init(bar_afull + 8 * s, 4);   // the four warps of the unpack group that owns the slot
      mbar_init(bar_aempty + 8 * s, 1);  // commit of the MMAs that read the segment
    }
    for (int d = 0; d < I8_MAX_GROUPS; ++d) {
      mbar_init(bar_dfull + 8 * d, 1);   // commit of the group's MMAs
      mbar_init(bar_dempty + 8 * d, 4);  // the four epilogue warps that own the group have read it
    }
    mbar_init(bar_xchg, 4);
    for (int w = 0; w < I8_SCALE_RING; ++w) {
      mbar_init(bar_wfull + 8 * w, 32);   // every lane of the scale warp, after its copies
      mbar_init(bar_wempty + 8 * w, 8);   // the eight epilogue warps
    }
    for (int c = 0; c < I8_CHUNKS; ++c) {
      mbar_init(bar_cfull + 8 * c, 1);    // the producer's lane 0 (+ the bytes of its copies)
      mbar_init(bar_cempty + 8 * c, 8);   // the eight epilogue warps
    }
    mbar_init(bar_xfull, 4);   // the second group of epilogue warps has written its partial totals
    mbar_init(bar_xempty, 4);  // the first has read them
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

  if (warp == I8_WARP_PRODUCER) {
    // ---------------- producer warp ----------------
    const int n_active = *reinterpret_cast<volatile const int*>(a.plan);
    const int n_items0 = a.phase_begin == 0 ? n_active * a.row_blocks[0] : 0;
    const int n_items1 = a.phase_end == 2 ? n_active * a.row_blocks[1] * a.ksplit : 0;
    const int n_items = n_items0 + n_items1;
    Ring ring{0, 0}, sring{0, 0}, cring{0, 0};
    bool ok = true;
    const int ssz = L.scale_f16 ? 2 : 4;
    PROF_DECL;
#ifdef EMOE_I8_PROFILE
    const long long prof_start = clock64();
#endif
    int item = blockIdx.x;  // a CTA's first item is its own index; the counter hands out the rest
    while (ok) {
      if (item >= n_items || __any_sync(0xffffffffu, *abort_flag != 0)) break;
      const int phase = item < n_items0 ? 0 : 1;
      const int li = item - (phase == 0 ? 0 : n_items0);
      const PhaseDims pd = phase_dims<DUAL>(a, phase);
      const int K = pd.K;
      const int ai = li / (pd.ksplit * pd.row_blocks);
      const PlanRec rec = recs[ai];
      const int z = li % pd.ksplit;
      const int rb = (li / pd.ksplit) % pd.row_blocks;
      const CUtensorMap* maps = a.wmaps + static_cast<size_t>(rec.e) * 3;
      const int bits = rec.bits;
      const int kspan = 1024 / bits;
      const int steps_total = (K + kspan - 1) / kspan;
      const int spz = (steps_total + pd.ksplit - 1) / pd.ksplit;
      const int step_begin = z * spz;
      const int nsteps = max(0, min(steps_total, step_begin + spz) - step_begin);
      const int npass = (rec.cnt + NT - 1) / NT;
      const int row0 = rb * I8_ROWS;
      // scale channels of the item's matrices (picked with constant indices: the record stays in registers)
      const void* const sc_m0 = phase == 0 ? rec.scales[0] : (DUAL ? rec.scales[2] : rec.scales[1]);
      const void* const sc_m1 = (DUAL && phase == 0) ? rec.scales[1] : sc_m0;
      bool need_dep = fused && phase == 1;
      const int smode = a.scale_mode[phase];
      const int ngroups_k = a.ngroups[phase];
      const int row_bytes = ngroups_k * ssz;  // a row's scale channel
      for (int pass = 0; pass < npass && ok; ++pass) {
        const int p0 = pass * NT;
        const int ntok = min(NT, rec.cnt - p0);
        const int nst = max(nsteps, 1);  // an empty split-K slice still has to store its zeros
        int cur_win = -1, cur_chunk = 0;
        for (int s = 0; s < nst; ++s) {
          PROF_BEGIN;
          if (!wait_warp(bar_empty + 8 * ring.i, ring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag) ||
              !wait_warp(bar_sempty + 8 * sring.i, sring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
            ok = false;
            break;
          }
          PROF_END(0);
          unsigned char* st = smem + ring.i * STAGE_BYTES;
          const uint32_t full = bar_full + 8 * ring.i;
          SideEntry* se = &side[sring.i];
          const int k0 = (step_begin + s) * kspan;
          const int klen = nsteps > 0 ? min(kspan, K - k0) : 0;
          const int nseg = klen / 128;
          // the scale-ring entry of the stage: the item's block, or the 32-byte window its inputs fall into
          int cflags = 0, stage_win0 = 0;
          if (klen > 0 && smode != SCALE_STAGE) {
            const int win = smode == SCALE_BLOCK ? 0 : (group_of(k0, a.gshift, L.group, ngroups_k) * ssz) / I8_CHUNK_ROW;
            stage_win0 = win * I8_CHUNK_ROW;
            if (win != cur_win) {
              if (!wait_warp(bar_cempty + 8 * cring.i, cring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
                ok = false;
                break;
              }
              if (lane == 0) {
                const uint32_t cfull = bar_cfull + 8 * cring.i;
                unsigned char* cdst = scale_ring + cring.i * CHUNK_ENTRY;
                if (smode == SCALE_BLOCK) {
                  mbar_expect_tx(cfull, pd.nmat * I8_ROWS * row_bytes);
                  for (int m = 0; m < pd.nmat; ++m)
                    bulk_load(smem_u32(cdst + m * I8_CHUNK_BYTES),
                              static_cast<const char*>(m == 0 ? sc_m0 : sc_m1) + static_cast<size_t>(row0) * row_bytes,
                              I8_ROWS * row_bytes, cfull);
                } else {
                  mbar_expect_tx(cfull, pd.nmat * I8_CHUNK_BYTES);
                  for (int m = 0; m < pd.nmat; ++m)
                    tma_load_2d(smem_u32(cdst + m * I8_CHUNK_BYTES), a.smaps + static_cast<size_t>(rec.e) * 3 + pd.mat_first + m,
                                win * I8_CHUNK_ROW, row0, cfull);
                }
              }
              cur_win = win;
              cur_chunk = cring.i;
              cring.next(I8_CHUNKS);
              cflags |= META_NEW_CHUNK;
            }
            const int k0n = k0 + kspan;
            const bool last = s == nst - 1 || k0n >= K ||
                              (smode == SCALE_WINDOW && (group_of(k0n, a.gshift, L.group, ngroups_k) * ssz) / I8_CHUNK_ROW != win);
            if (last) {
              cflags |= META_END_CHUNK;
              cur_win = -1;
            }
          }
          if (lane == 0) {
            const int flags = (s == 0 ? META_FIRST : 0) | (s == nst - 1 ? META_LAST : 0) | (klen == 0 ? META_EMPTY : 0) |
                              (fused && phase == 0 && s == nst - 1 && pass == npass - 1 ? META_DONE : 0) | cflags |
                              (need_dep && klen > 0 ? META_DEP : 0);
            uint4* mq = reinterpret_cast<uint4*>(&se->m);
            mq[0] = make_uint4(rec.e, rb, z, rec.begin);
            mq[1] = make_uint4(p0, ntok, k0, bits);
            mq[2] = make_uint4(flags, phase, ai, nseg);
            se->m.scales[0] = sc_m0;
            se->m.scales[1] = sc_m1;
            se->m.chunk = cur_chunk;
            se->m.win0 = stage_win0;
            se->m.pitch = smode == SCALE_BLOCK ? row_bytes : I8_CHUNK_ROW;
            {
              const int g0 = group_of(k0, a.gshift, L.group, ngroups_k);
              uint32_t rel = 0;
              for (int sg = 0; sg < 4; ++sg)
                rel |= static_cast<uint32_t>((group_of(k0 + min(sg, max(nseg, 1) - 1) * 128, a.gshift, L.group, ngroups_k) - g0) * ssz)
                       << (8 * sg);
              se->m.sc_rel = rel;
              se->m.sc_addr = smem_u32(scale_ring) + cur_chunk * CHUNK_ENTRY + g0 * ssz - stage_win0;
            }
            // all bytes the stage will receive (the feeder's limb rows included), then the record is published
            if (klen > 0) mbar_expect_tx(full, pd.nmat * I8_MAT_BYTES + nseg * B_SEG_BYTES);
            else mbar_arrive(full);
            mbar_arrive(bar_mready + 8 * sring.i);
          }
          if (klen > 0) need_dep = false;
          __syncwarp();
          // the weight boxes: lane l fetches box l (matrix l / 2, upper or lower 64 rows), one instruction for all
          if (klen > 0 && lane < 2 * pd.nmat) {
            const int mtx = lane >> 1, half = lane & 1;
            tma_load_2d(smem_u32(st + mtx * I8_MAT_BYTES + half * I8_BOX_BYTES), maps + pd.mat_first + mtx, k0 * bits / 8,
                        row0 + half * I8_BOX_ROWS, full);
          }
          ring.next(STAGES);
          sring.next(I8_SIDE);
        }
      }
      // the ring still holds several stages of work: fetching the next item only now costs nothing
      // and no CTA sits on items it is not yet working on
      int item_next = 0;
      if (lane == 0) item_next = gridDim.x + atomicAdd(a.plan + 1 + a.phase_begin, 1);
      item = __shfl_sync(0xffffffffu, item_next, 0);
    }
#ifdef EMOE_I8_PROFILE
    prof_acc[2] = clock64() - prof_start;
#endif
    PROF_STORE(0, 3);
    if (ok && !__any_sync(0xffffffffu, *abort_flag != 0)) {  // tell the others that nothing else comes
      if (wait_warp(bar_empty + 8 * ring.i, ring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag) &&
          wait_warp(bar_sempty + 8 * sring.i, sring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
        if (lane == 0) {
          side[sring.i].m.flags = META_STOP;
          mbar_arrive(bar_full + 8 * ring.i);
          mbar_arrive(bar_mready + 8 * sring.i);
        }
      }
    }
  } else if (warp == I8_WARP_FEEDER) {
    // ---------------- feeder warp: the tokens' limb rows and block scales of every stage ----------------
    Ring ring{0, 0}, sring{0, 0}, wring{0, 0};
    while (true) {
      if (!wait_warp(bar_mready + 8 * sring.i, sring.ph, a.wait_limit, a.check_word, abort_flag)) break;
      SideEntry* se = &side[sring.i];
      const uint4 m0 = *reinterpret_cast<const uint4*>(&se->m.e);       // e, rb, z, begin
      const uint4 m1 = *reinterpret_cast<const uint4*>(&se->m.p0);      // p0, ntok, k0, bits
      const uint4 m2 = *reinterpret_cast<const uint4*>(&se->m.flags);   // flags, phase, ai, nseg
      const int flags = static_cast<int>(m2.x), phase = static_cast<int>(m2.y), ai = static_cast<int>(m2.z),
                nseg = static_cast<int>(m2.w);
      const uint32_t sfull = bar_sfull + 8 * sring.i;
      if (flags & META_STOP) {
        mbar_arrive(sfull);
        break;
      }
      if (!(flags & META_EMPTY)) {
        const int begin = static_cast<int>(m0.w), p0 = static_cast<int>(m1.x), ntok = static_cast<int>(m1.y),
                  k0 = static_cast<int>(m1.z);
        if (flags & META_DEP) {
          // The hidden vectors may still be in the making on other SMs.  Every lane acquires the
          // counter itself, so that its own copies below are ordered behind the writers' stores.
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
            // the stage's barriers stay incomplete: nobody consumes it; the weight copies already
            // issued land in the CTA's own shared memory during the wind-down pause
            if (lane == 0) {
              *abort_flag = 1;
              atomicOr(a.check_word, CHECK_WAIT_TIMEOUT);
            }
            break;
          }
          asm volatile("fence.proxy.async;" ::: "memory");  // generic-proxy stores -> TMA reads
        }
        const int K = phase == 0 ? L.d_model : L.d_ff;
        if (a.scale_mode[phase] == SCALE_STAGE) {
          // General scale mode: lane l copies the windows of rows 4l .. 4l+3 of every matrix of the stage.
          // The scales a stage needs from a row (groups of inputs k0 .. k0 + 128 * segments) are a few
          // neighbouring bytes of the row's scale channel; they are copied in 4-byte words from the
          // 4-byte boundary at or below the first one, into a 16-byte window per row.
          if (!wait_warp(bar_wempty + 8 * wring.i, wring.ph ^ 1u, a.wait_limit, a.check_word, abort_flag)) break;
          const int ssz = L.scale_f16 ? 2 : 4;
          const int N = phase == 0 ? L.d_ff : L.d_model;
          const int ngroups = a.ngroups[phase];
          const int nmat = (DUAL && phase == 0) ? 2 : 1;
          const int rb = static_cast<int>(m0.y);
          const int g0 = group_of(k0, a.gshift, L.group, ngroups), g1 = group_of(k0 + (nseg - 1) * 128, a.gshift, L.group, ngroups);
          const uint32_t sdst = smem_u32(scale_ring + wring.i * SCALE_ENTRY);
          const char* const sb0 = static_cast<const char*>(se->m.scales[0]);
          const char* const sb1 = static_cast<const char*>(se->m.scales[1]);
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const int row = 4 * lane + r;
            const int off = min(rb * I8_ROWS + row, N - 1) * ngroups * ssz;
            const int b0 = (off + g0 * ssz) & ~3;
            const int b1 = off + (g1 + 1) * ssz;
            for (int mt = 0; mt < nmat; ++mt) {
              const char* sbase = mt == 0 ? sb0 : sb1;
#pragma unroll 1
              for (int w = 0; b0 + 4 * w < b1; ++w)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sdst + (mt * I8_ROWS + row) * 16 + 4 * w),
                             "l"(sbase + b0 + 4 * w)
                             : "memory");
            }
          }
          asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar_wfull + 8 * wring.i) : "memory");
          wring.next(I8_SCALE_RING);
        }
        // block scales of the tile's tokens
        if (lane < ntok) {
          const float* src = (phase == 0 ? a.xsc : a.hsc) + static_cast<size_t>(begin + p0 + lane) * (K / 128) + k0 / 128;
          const uint32_t xdst = smem_u32(&se->sx[0][lane]);
          for (int sg = 0; sg < nseg; ++sg)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(xdst + sg * 128), "l"(src + sg) : "memory");
        }
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(sfull) : "memory");
        // the tokens' limb rows: rows 2*slot (hi) and 2*slot+1 (lo) of the activation image; lane l fetches segment l
        if (lane < nseg)
          tma_load_2d(smem_u32(smem + ring.i * STAGE_BYTES + B_OFF + lane * B_SEG_BYTES), phase == 0 ? &tmap_x : &tmap_h,
                      k0 + lane * 128, 2 * (begin + p0), bar_full + 8 * ring.i);
      } else {
        mbar_arrive(sfull);
      }
      ring.next(STAGES);
      sring.next(I8_SIDE);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");  // nothing of this warp is in flight when the CTA ends
  } else if (warp == I8_WARP_MMA || warp == I8_WARP_MMA1) {
    // ---------------- MMA issuers (one lane of each of the two warps) ----------------
    if (lane == 0) {
      const uint32_t mi = warp == I8_WARP_MMA ? 0u : 1u;  // even or odd accumulator groups
      // kind::i8: s8 x s8 -> s32, both operands K-major, M = 128, N = 2 * NT
      const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((static_cast<uint32_t>(NCOL) >> 3) << 17) |
                             ((static_cast<uint32_t>(I8_ROWS) >> 4) << 24);
      Ring ring{0, 0}, sring{0, 0};
      uint32_t qs = 0;  // segments that went through the A ring so far
      uint32_t gq = 0;  // accumulator groups so far: group gq lives in slot gq % NGRP, even ones belong to the
                        // first group of epilogue warps, odd ones to the second
      bool ok = true;
      PROF_DECL;
      while (ok) {
        PROF_BEGIN;
        if (!wait_lim(bar_full + 8 * ring.i, ring.ph, a.wait_limit, a.check_word, abort_flag)) break;
        PROF_END(0);
        tc_fence_after();
        const StageMeta m = side[sring.i].m;
        if (m.flags & META_STOP) break;
        if (m.flags & META_EMPTY) {
          mbar_arrive(bar_empty + 8 * ring.i);
          ring.next(STAGES);
          sring.next(I8_SIDE);
          continue;
        }
        const uint32_t st = smem_u32(smem + ring.i * STAGE_BYTES);
        const int nmat = (DUAL && m.phase == 0) ? 2 : 1;
        bool issued = false;
        for (int mt = 0; mt < nmat && ok; ++mt) {
          const uint64_t adesc = umma_desc(st + mt * I8_MAT_BYTES);
          for (int sg0 = 0; sg0 < m.nseg && ok; sg0 += GSEGS) {
            if ((gq & 1u) != mi) {  // the other warp's group: only keep the counters in step
              if (m.bits != 8) qs += min(m.nseg, sg0 + GSEGS) - sg0;
              ++gq;
              continue;
            }
            issued = true;
            const uint32_t gslot = gq % NGRP;
            PROF_BEGIN;
            if (!wait_lim(bar_dempty + 8 * gslot, ((gq / NGRP) & 1u) ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            PROF_END(2);
            tc_fence_after();
            const int sg1 = min(m.nseg, sg0 + GSEGS);
            for (int sg = sg0; sg < sg1; ++sg) {
              const uint32_t d_tmem = tmem_base + I8_D_COL0 + gslot * GCOLS + (sg - sg0) * NCOL;
              const uint64_t bdesc = umma_desc(st + B_OFF + sg * B_SEG_BYTES);
              if (m.bits == 8) {
                PROF_BEGIN;
#pragma unroll
                for (int j = 0; j < 4; ++j)  // 32 inputs per MMA
                  umma_i8_ss(d_tmem, adesc + 2 * j, bdesc + 2 * j, idesc, j > 0 ? 1u : 0u);
                PROF_END(3);
              } else {
                const uint32_t slot = qs & (I8_A_SLOTS - 1);
                PROF_BEGIN;
                if (!wait_lim(bar_afull + 8 * slot, (qs / I8_A_SLOTS) & 1u, a.wait_limit, a.check_word, abort_flag)) {
                  ok = false;
                  break;
                }
                PROF_END(1);
                tc_fence_after();
                const uint32_t a_tmem = tmem_base + slot * I8_A_SLOT_COLS;
                PROF_BEGIN;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  umma_i8_ts(d_tmem, a_tmem + 8 * j, bdesc + 2 * j, idesc, j > 0 ? 1u : 0u);
                PROF_END(3);
                PROF_BEGIN;
                umma_commit(bar_aempty + 8 * slot);
                PROF_END(4);
                ++qs;
              }
            }
            if (!ok) break;
            PROF_BEGIN;
            umma_commit(bar_dfull + 8 * gslot);
            PROF_END(4);
            ++gq;
          }
        }
        if (!ok) break;
        // the stage's shared memory may be refilled once the MMAs of both warps have read it
        if (issued) umma_commit(bar_empty + 8 * ring.i);
        else mbar_arrive(bar_empty + 8 * ring.i);
        ring.next(STAGES);
        sring.next(I8_SIDE);
      }
#ifdef EMOE_I8_PROFILE
      if (a.prof && mi == 0) {
        for (int pi = 0; pi < 3; ++pi) a.prof[blockIdx.x * 32 + 3 + pi] = prof_acc[pi];
        a.prof[blockIdx.x * 32 + 28] = prof_acc[3];
        a.prof[blockIdx.x * 32 + 29] = prof_acc[4];
      }
#endif
    }
  } else if (warp >= I8_WARP_UNPACK0) {
    // ---------------- unpack warps: packed codes -> int8 rows in tensor memory ----------------
    // segment number qs of the kernel goes to slot qs % 8 of the A ring; even segments are this
    // group's if wg = 0, odd ones if wg = 1
    const uint32_t wg = static_cast<uint32_t>(warp - I8_WARP_UNPACK0) >> 2;
    const int r = 32 * (warp & 3) + lane;  // row of the item = tensor-memory lane
    const uint32_t a_tmem0 = tmem_base + (static_cast<uint32_t>(32 * (warp & 3)) << 16);
    const int row_off = (r >> 6) * I8_BOX_BYTES + (r & 63) * 128;
    const int swz = r & 7;
    Ring ring{0, 0}, sring{0, 0};
    uint32_t qs = 0;
    bool ok = true;
    PROF_DECL;
    while (ok) {
      PROF_BEGIN;
      if (!wait_warp(bar_full + 8 * ring.i, ring.ph, a.wait_limit, a.check_word, abort_flag)) break;
      PROF_END(0);
      const int flags = side[sring.i].m.flags;
      if (flags & META_STOP) break;
      const int bits = side[sring.i].m.bits, nseg = side[sring.i].m.nseg, phase = side[sring.i].m.phase;
      if (!(flags & META_EMPTY) && bits != 8) {
        const int nmat = (DUAL && phase == 0) ? 2 : 1;
        for (int mt = 0; mt < nmat && ok; ++mt) {
          const unsigned char* row = smem + ring.i * STAGE_BYTES + mt * I8_MAT_BYTES + row_off;
          for (int sg = 0; sg < nseg; ++sg, ++qs) {
            if ((qs & 1u) != wg) continue;
            const uint32_t slot = qs & (I8_A_SLOTS - 1);
            PROF_BEGIN;
            if (!wait_warp(bar_aempty + 8 * slot, ((qs / I8_A_SLOTS) & 1u) ^ 1u, a.wait_limit, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            PROF_END(1);
            PROF_BEGIN;
            tc_fence_after();
            const uint32_t a_tmem = a_tmem0 + slot * I8_A_SLOT_COLS;
            if (bits == 4) {
              // a 16-byte chunk = 32 codes = 8 columns; 4 chunks per segment
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                uint32_t o[8];
                unpack4(*reinterpret_cast<const uint4*>(row + (((4 * sg + c) ^ swz) << 4)), o);
                tmem_st8(a_tmem + 8 * c, o);
              }
            } else {
              // a 16-byte chunk = 64 codes = 16 columns; 2 chunks per segment
#pragma unroll
              for (int c = 0; c < 2; ++c) {
                uint32_t o[16];
                unpack2(*reinterpret_cast<const uint4*>(row + (((2 * sg + c) ^ swz) << 4)), o);
                tmem_st16(a_tmem + 16 * c, o);
              }
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_afull + 8 * slot);
            PROF_END(2);
          }
        }
      }
      // this warp is through with the stage (its codes and its record), whatever the width
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * ring.i);
      ring.next(STAGES);
      sring.next(I8_SIDE);
    }
    if (warp == I8_WARP_UNPACK0) { PROF_STORE(6, 3); }
  } else {
    // ---------------- epilogue warps: one thread per output row in each group of four warps ----------------
    const uint32_t ew = static_cast<uint32_t>(warp) >> 2;  // which of the two groups
    const int wq = warp & 3;                               // the warp's quarter of the tensor-memory lanes
    const int r = 32 * wq + lane;
    const uint32_t d_tmem0 = tmem_base + (static_cast<uint32_t>(32 * wq) << 16) + I8_D_COL0;
    float tot[NMAT_MAX][NT];  // this group's share of the row's totals
    Ring sring{0, 0}, wring{0, 0}, cring{0, 0};
    uint32_t gq = 0;         // accumulator groups so far (as the MMA warp counts them)
    uint32_t items = 0;      // items finished so far
    uint32_t exchanges = 0;  // first-projection items finished so far (each uses the exchange barrier once)
    bool ok = true;
    PROF_DECL;
    while (ok) {
      PROF_BEGIN;
      if (!wait_warp(bar_sfull + 8 * sring.i, sring.ph, a.wait_limit, a.check_word, abort_flag)) break;
      PROF_END(0);
      const SideEntry& se = side[sring.i];
      // Under load a shared-memory load takes a hundred cycles and more and every instruction of
      // this chain waits for the one before, so the record is read in one batch, nothing branches
      // on a loaded value where a batch of loads can be issued instead, and what does not depend
      // on the row (offsets, addresses) was worked out once by the producer.
      const uint4 q1 = *reinterpret_cast<const uint4*>(&se.m.p0);     // p0, ntok, k0, bits
      const uint4 q2 = *reinterpret_cast<const uint4*>(&se.m.flags);  // flags, phase, ai, nseg
      const uint4 q4 = *reinterpret_cast<const uint4*>(&se.m.chunk);  // chunk, win0, pitch, sc_rel
      const uint32_t sc_addr0 = se.m.sc_addr;
      const int flags = static_cast<int>(q2.x), phase = static_cast<int>(q2.y), nseg = static_cast<int>(q2.w);
      const int ntok = static_cast<int>(q1.y);
      if (flags & META_STOP) break;
      PROF_BEGIN;
      if (flags & META_FIRST) {
#pragma unroll
        for (int mt = 0; mt < NMAT_MAX; ++mt)
#pragma unroll
          for (int t = 0; t < NT; ++t) tot[mt][t] = 0.0f;
      }
      if (!(flags & META_EMPTY)) {
        const int nmat = (DUAL && phase == 0) ? 2 : 1;
        const int ssz = L.scale_f16 ? 2 : 4;
        const bool per_stage = a.scale_mode[phase] == SCALE_STAGE;
        uint32_t sc_row;  // shared-memory address of this row's scale of segment 0, first matrix
        int mat_stride;
        if (per_stage) {
          if (!wait_warp(bar_wfull + 8 * wring.i, wring.ph, a.wait_limit, a.check_word, abort_flag)) break;
          // the row's window starts at the 4-byte boundary at or below its first scale of the stage
          const int N = phase == 0 ? L.d_ff : L.d_model;
          const int ngroups = a.ngroups[phase];
          const int g0 = group_of(static_cast<int>(q1.z), a.gshift, L.group, ngroups);
          const int n = se.m.rb * I8_ROWS + r;
          sc_row = smem_u32(scale_ring) + wring.i * SCALE_ENTRY + r * 16 + (((min(n, N - 1) * ngroups + g0) * ssz) & 3);
          mat_stride = I8_SCALE_TILE;
        } else {
          PROF_LAP(6);
          if (flags & META_NEW_CHUNK) {
            if (!wait_warp(bar_cfull + 8 * cring.i, cring.ph, a.wait_limit, a.check_word, abort_flag)) break;
            cring.next(I8_CHUNKS);
          }
          PROF_LAP(7);
          sc_row = sc_addr0 + r * static_cast<int>(q4.z);
          mat_stride = I8_CHUNK_BYTES;
        }
        uint32_t sraw[NMAT_MAX][4];  // the stage's scales of this row as stored (fp16 or fp32 bits)
#pragma unroll
        for (int sg = 0; sg < 4; ++sg) {
          const uint32_t off = (q4.w >> (8 * sg)) & 0xffu;
#pragma unroll
          for (int mt = 0; mt < NMAT_MAX; ++mt) {
            const uint32_t ad = sc_row + (mt < nmat ? mt : 0) * mat_stride + off;
            if (ssz == 2) asm volatile("ld.shared.u16 %0, [%1];" : "=r"(sraw[mt][sg]) : "r"(ad));
            else asm volatile("ld.shared.u32 %0, [%1];" : "=r"(sraw[mt][sg]) : "r"(ad));
          }
        }
        __syncwarp();
        if (per_stage) {
          if (lane == 0) mbar_arrive(bar_wempty + 8 * wring.i);
          wring.next(I8_SCALE_RING);
        } else if (flags & META_END_CHUNK) {
          if (lane == 0) mbar_arrive(bar_cempty + 8 * static_cast<int>(q4.x));
        }
        PROF_LAP(3);
        const uint32_t sx_addr = smem_u32(&se.sx[0][0]);
#pragma unroll
        for (int mt = 0; mt < NMAT_MAX; ++mt) {
          if (mt >= nmat || !ok) break;
#pragma unroll
          for (int g = 0; g < 4 / GSEGS; ++g) {
            if (g * GSEGS >= nseg) break;
            const uint32_t gslot = gq % NGRP, gpar = (gq / NGRP) & 1u;
            const bool mine = (gq & 1u) == ew;
            ++gq;
            if (!mine) continue;
            PROF_BEGIN;
            if (!wait_warp(bar_dfull + 8 * gslot, gpar, a.wait_limit, a.check_word, abort_flag)) {
              ok = false;
              break;
            }
            PROF_LAP(1);
            tc_fence_after();
            const uint32_t d_tmem = d_tmem0 + gslot * GCOLS;
            // the group in chunks of 32 columns (2 segments at NT = 8, 1 at 16, half a segment at 32)
            constexpr int NCHUNK = GCOLS / 32;
            constexpr int TOK_PER_CHUNK = NT < 16 ? NT : 16;  // tokens of one segment inside a chunk
            constexpr int PIECES = 32 / (2 * TOK_PER_CHUNK);  // segments (or half segments) inside a chunk
            const int ncols = min(GSEGS, nseg - g * GSEGS) * NCOL;
#pragma unroll
            for (int c = 0; c < NCHUNK; ++c) {
              if (c * 32 >= ncols) break;
              uint32_t acc[32];
              tmem_ld32(d_tmem + c * 32, acc);
              // the tokens' block scales of the chunk's pieces, requested under the tensor-memory load
              float sxv[PIECES][TOK_PER_CHUNK];
#pragma unroll
              for (int u = 0; u < PIECES; ++u) {
                const int col0 = c * 32 + u * 2 * TOK_PER_CHUNK;
                const int sg = min(g * GSEGS + col0 / NCOL, 3), t0 = (col0 % NCOL) / 2;
#pragma unroll
                for (int t = 0; t < TOK_PER_CHUNK; t += 4)
                  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                               : "=f"(sxv[u][t]), "=f"(sxv[u][t + 1]), "=f"(sxv[u][t + 2]), "=f"(sxv[u][t + 3])
                               : "r"(sx_addr + (sg * 32 + t0 + t) * 4));
              }
              tmem_ld_wait();
              const bool more = (c + 1) * 32 < ncols;
              if (!more) {  // the last chunk is in registers: the accumulators may be overwritten
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_dempty + 8 * gslot);
              }
              PROF_LAP(4);
#pragma unroll
              for (int u = 0; u < PIECES; ++u) {
                const int col0 = c * 32 + u * 2 * TOK_PER_CHUNK;  // first column of this piece in the group
                const int sg = g * GSEGS + col0 / NCOL;            // its segment in the stage
                const int t0 = (col0 % NCOL) / 2;                  // its first token
                // (the factor 16 or 64 of the unpacked codes is taken out once, at the end of the item)
                const uint32_t raw = sraw[mt][sg < 4 ? sg : 3];
                const float sv = ssz == 2 ? __half2float(__ushort_as_half(static_cast<unsigned short>(raw))) : __uint_as_float(raw);
                const float s = sv;
                // tokens in pairs: a pair past the expert's tokens is skipped, inside a pair nothing branches;
                // a segment past the stage's last is skipped too (its token scales are whatever the entry held)
#pragma unroll
                for (int t = 0; t < TOK_PER_CHUNK; t += 2) {
                  if (sg < nseg && t0 + t < ntok) {
#pragma unroll
                    for (int tt = t; tt < t + 2; ++tt) {
                      const int v = static_cast<int>(acc[u * 2 * TOK_PER_CHUNK + 2 * tt]) * 128 +
                                    static_cast<int>(acc[u * 2 * TOK_PER_CHUNK + 2 * tt + 1]);
                      tot[mt][t0 + tt] = fmaf(static_cast<float>(v), s * sxv[u][tt], tot[mt][t0 + tt]);
                    }
                  }
                }
              }
            }
            PROF_LAP(5);
          }
        }
        if (!ok) break;
      }
      if (!(flags & META_LAST)) {
        // the side entry is no longer needed
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_sempty + 8 * sring.i);
      } else {
        // end of an item: the whole record is needed once more, then the entry is released
        const StageMeta m = se.m;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_sempty + 8 * sring.i);
        const int N = m.phase == 0 ? L.d_ff : L.d_model;
        const int n = m.rb * I8_ROWS + r;
        // 4- and 2-bit codes were multiplied as 16 q and 64 q: taken out here, once per item
        const float unit = m.bits == 8 ? 1.0f : (m.bits == 4 ? 0.0625f : 0.015625f);
        PROF_BEGIN;
        // the two groups of warps put their shares of the totals together: the second writes, the first adds
        const uint32_t ipar = items & 1u;
        ++items;
        if (ew == 1) {
          if (!wait_warp(bar_xempty, ipar ^ 1u, a.wait_limit, a.check_word, abort_flag)) break;
#pragma unroll
          for (int mt = 0; mt < NMAT_MAX; ++mt)
#pragma unroll
            for (int t = 0; t < NT; ++t)
              if (t < m.ntok) xbuf[(mt * NT + t) * I8_ROWS + r] = tot[mt][t];  // (scaled by the reader)
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_xfull);
          sring.next(I8_SIDE);
          continue;
        }
        if (!wait_warp(bar_xfull, ipar, a.wait_limit, a.check_word, abort_flag)) break;
#pragma unroll
        for (int mt = 0; mt < NMAT_MAX; ++mt)
#pragma unroll
          for (int t = 0; t < NT; ++t)
            if (t < m.ntok) tot[mt][t] = unit * (tot[mt][t] + xbuf[(mt * NT + t) * I8_ROWS + r]);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_xempty);
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
            if (lane == 0) s_max[par][t][wq] = mx;
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
        PROF_END(2);
      }
      sring.next(I8_SIDE);
    }
    if (warp == 0) { PROF_STORE(9, 8); }
    if (warp == 4) { PROF_STORE(20, 8); }
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
  static_assert(I8_CHUNKS * I8_CHUNK_BYTES == I8_SCALE_RING * I8_SCALE_TILE, "both kinds of scale ring take the same room");
  int s = (I8_SMEM_LIMIT - 1024 /*alignment slack*/ - I8_STATIC_SMEM - I8_SCALE_RING * nmat * I8_SCALE_TILE - nmat * nt * I8_ROWS * 4) /
          stage_bytes(nt, nmat);
  return s > I8_MAX_STAGES ? I8_MAX_STAGES : s;
}

template <int NT, bool DUAL>
cudaError_t launch_variant(const I8Args& a_in, const CUtensorMap& tx, const CUtensorMap& th, long long items, cudaStream_t st) {
  static int sms_of_device[64] = {};
  I8Args a = a_in;
  a.stages = stages_for(NT, DUAL ? 2 : 1);
  if (a.stages < 3) return cudaErrorInvalidValue;
  const int smem = a.stages * stage_bytes(NT, DUAL ? 2 : 1) + I8_SCALE_RING * (DUAL ? 2 : 1) * I8_SCALE_TILE +
                   (DUAL ? 2 : 1) * NT * I8_ROWS * 4 + 1024;
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

long long* g_i8_profile = nullptr;

bool ffn_i8_supported(const LayerDims& L) {
  // bf16 activations, inputs in whole 128-blocks, scale groups of whole blocks; the tensor maps use
  // 128-byte x 64-row boxes: every packed row must hold at least 128 bytes at the narrowest width
  return ffn_mma_supported(L) && L.d_model >= 512 && L.d_ff >= 512;
}

// tokens per tile (columns of the B operand / 2): the epilogue's work per segment grows with the
// tile, an expert with more tokens than the tile takes another pass over its weights (from L2)
int ffn_i8_token_tile(const LayerDims& L, int T) {
  const double mean = static_cast<double>(T) * L.top_k / L.E;
  // a gated layer's stage carries two weight boxes: with 32-token tiles fewer than three stages fit
  const int widest = L.act == EMOE_ACT_SWIGLU ? 16 : 32;
  return mean <= 6.0 ? 8 : (mean <= 12.0 ? 16 : widest);
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

cudaError_t launch_ffn_i8(int phase_begin, int phase_end, const LayerDims& L, const void* wmaps, const void* smaps, const void* xq,
                          const float* xsc, int* plan, void* hq, float* hsc, float* o_part, int ksplit, int n_pairs,
                          int T, int token_tile, unsigned wait_limit, int dep_extra, int* check_word, cudaStream_t st) {
  if (phase_begin < 0 || phase_end > 2 || phase_begin >= phase_end) return cudaErrorInvalidValue;
  const int nt = token_tile > 0 ? token_tile : ffn_i8_token_tile(L, T);
  I8Args a;
  a.phase_begin = phase_begin;
  a.phase_end = phase_end;
  a.L = L;
  a.wmaps = static_cast<const CUtensorMap*>(wmaps);
  a.smaps = static_cast<const CUtensorMap*>(smaps);
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
  // how the weight scales travel (smaps is null when a scale channel of the table is not 16-byte aligned)
  for (int p = 0; p < 2; ++p) {
    const int row_bytes = a.ngroups[p] * (L.scale_f16 ? 2 : 4);
    const bool pow2_groups = a.ngroups[p] == 1 || a.gshift >= 0;
    a.scale_mode[p] = !smaps || !pow2_groups ? SCALE_STAGE
                      : row_bytes <= I8_CHUNK_ROW ? SCALE_BLOCK
                      : row_bytes % 16 == 0 ? SCALE_WINDOW
                                            : SCALE_STAGE;
  }
  // both kinds of ring entry share one region of shared memory: one projection on the general path
  // puts the other there too
  if (a.scale_mode[0] == SCALE_STAGE || a.scale_mode[1] == SCALE_STAGE) a.scale_mode[0] = a.scale_mode[1] = SCALE_STAGE;
  a.n_pairs = n_pairs;
  a.stages = 0;
  a.wait_limit = wait_limit ? wait_limit : (1u << 20);  // polls of up to a microsecond each
  a.dep_wait_limit = wait_limit ? wait_limit : (1u << 20);
  a.dep_extra = dep_extra;
  a.check_word = check_word;
  a.prof = g_i8_profile;
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
