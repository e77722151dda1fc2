// Device pieces shared by the kernels that prepare the expert stage: the work plan of the
// persistent expert kernels and the copy of one activation row into expert order, in the layout
// and number format the expert kernel of the call wants.
#pragma once
#include "act_q.cuh"
#include "common.cuh"
#include "ffn_tile.cuh"

namespace emoe {

// Work plan of the persistent expert kernels, written by one warp: activated experts whose token
// count lies in [cnt_lo, cnt_hi], widest codes (most bytes) first; the item counters restart from
// zero.  off: exclusive offsets of the experts' slots (global or shared memory).
__device__ __forceinline__ void build_plan(int* plan, const ExpertDev* __restrict__ experts, const int32_t* off, int E,
                                           int cnt_lo, int cnt_hi, int lane) {
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

// Per-expert counts -> exclusive offsets, by one warp: s_off[e + 1] holds the count of expert e on
// entry (s_off[0] = 0) and the offset of expert e + 1 on exit; the counts go to counts_out.
__device__ __forceinline__ void counts_to_offsets(int* s_off, int32_t* __restrict__ counts_out, int E, int lane) {
  int carry = 0;
  for (int e0 = 0; e0 < E; e0 += 32) {
    const int e = e0 + lane;
    const int c = e < E ? s_off[e + 1] : 0;
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (e < E) {
      counts_out[e] = c;
      s_off[e + 1] = carry + incl;
    }
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
}

// One activation row into the layout of the owning expert's bitwidth (optionally as fp16).
__device__ __forceinline__ void scatter_row(const __nv_bfloat16* __restrict__ src_row, __nv_bfloat16* __restrict__ dst_row,
                                            int d, int bits, int to_f16, int* __restrict__ check_word) {
  bool beyond = false;
  // one thread moves 16 consecutive inputs: half b of lane t's 32-block of a 128-input segment
  for (int u = threadIdx.x; u < d / 16; u += blockDim.x) {
    const int seg = (u >> 3) * 128, t = (u >> 1) & 3, b = u & 1;
    const uint4* src = reinterpret_cast<const uint4*>(src_row + seg + t * 32 + b * 16);
    uint4 a = src[0], c = src[1];
    if (to_f16) {  // the streaming kernel multiplies in fp16: same layout, 16-bit values converted in place
      beyond |= bf16x2_beyond_f16(a.x) | bf16x2_beyond_f16(a.y) | bf16x2_beyond_f16(a.z) | bf16x2_beyond_f16(a.w) |
                bf16x2_beyond_f16(c.x) | bf16x2_beyond_f16(c.y) | bf16x2_beyond_f16(c.z) | bf16x2_beyond_f16(c.w);
      a = make_uint4(bf16x2_to_f16x2_sat(a.x), bf16x2_to_f16x2_sat(a.y), bf16x2_to_f16x2_sat(a.z), bf16x2_to_f16x2_sat(a.w));
      c = make_uint4(bf16x2_to_f16x2_sat(c.x), bf16x2_to_f16x2_sat(c.y), bf16x2_to_f16x2_sat(c.z), bf16x2_to_f16x2_sat(c.w));
    }
    uint4 oa, oc;
    if (bits == 8) {
      oa = a;
      oc = c;
    } else if (bits == 4) {  // pair order (c, c+4) inside each 8
      oa = make_uint4(prmt(a.x, a.z, 0x5410u), prmt(a.x, a.z, 0x7632u), prmt(a.y, a.w, 0x5410u), prmt(a.y, a.w, 0x7632u));
      oc = make_uint4(prmt(c.x, c.z, 0x5410u), prmt(c.x, c.z, 0x7632u), prmt(c.y, c.w, 0x5410u), prmt(c.y, c.w, 0x7632u));
    } else {  // pair order (c, c+8) inside each 16
      oa = make_uint4(prmt(a.x, c.x, 0x5410u), prmt(a.x, c.x, 0x7632u), prmt(a.y, c.y, 0x5410u), prmt(a.y, c.y, 0x7632u));
      oc = make_uint4(prmt(a.z, c.z, 0x5410u), prmt(a.z, c.z, 0x7632u), prmt(a.w, c.w, 0x5410u), prmt(a.w, c.w, 0x7632u));
    }
    // pieces q = 2b and 2b+1 of lane t, stored piece-major
    *reinterpret_cast<uint4*>(dst_row + seg + (((2 * b) * 4 + t) << 3)) = oa;
    *reinterpret_cast<uint4*>(dst_row + seg + (((2 * b + 1) * 4 + t) << 3)) = oc;
  }
  // a value the fp16 operand cannot hold was saturated: the result is no longer the definition's
  if (beyond && check_word) atomicOr(check_word, CHECK_F16_RANGE);
}

// One activation row into slot `slot` of the activation buffer, in the format the expert kernel
// wants: fmt 0 = bf16 and 1 = fp16 in the k-interleaved layout (ffn_tile.cuh), 2 = two-limb
// block-scaled integers with their block scales (act_q.cuh; the slot's two limb rows take the
// same 2 * d bytes as a 16-bit row).
__device__ __forceinline__ void scatter_any(const __nv_bfloat16* __restrict__ src_row, __nv_bfloat16* __restrict__ xs,
                                            float* __restrict__ xsc, int slot, int d, int bits, int fmt,
                                            int* __restrict__ check_word) {
  if (fmt == 2) {
    int8_t* q = reinterpret_cast<int8_t*>(xs) + static_cast<size_t>(slot) * 2 * d;
    act_q_row(src_row, q, q + d, xsc + static_cast<size_t>(slot) * (d / 128), d, bits);
  } else {
    scatter_row(src_row, xs + static_cast<size_t>(slot) * d, d, bits, fmt, check_word);
  }
}

}  // namespace emoe
