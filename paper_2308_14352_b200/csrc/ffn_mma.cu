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
#include <cmath>

#include "common.cuh"
#include "ffn_tile.cuh"
#include "scatter.cuh"

namespace emoe {
namespace {

constexpr int MMA_WARPS = 4;
constexpr int MMA_THREADS = MMA_WARPS * 32;
constexpr int MMA_MT = 2;          // 16-row tiles per warp
constexpr int MMA_KCH = 512;       // inputs per staged activation chunk (4 segments of 128)
constexpr int MMA_XPAD = 32;       // bf16 elements of row padding in shared memory
constexpr int MMA_XSTRIDE = MMA_KCH + MMA_XPAD;

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
          for (int h = 0; h < 2; ++h) sc[mt][h] = load_scale_ro(sbase[mt], sf16, srow[mt][h] + grp);

        // B fragments of this segment: the lane's 32 interleaved activations of token (nt*8 + g)
        uint4 bq[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (nt * 8 < ntok) {
            const uint4* src = reinterpret_cast<const uint4*>(xsm + (nt * 8 + g) * MMA_XSTRIDE + sg * 128 + t * 8);
#pragma unroll
            for (int q = 0; q < 4; ++q) bq[nt][q] = src[q * 4];  // piece q of lane t sits at (q*4 + t) * 16 bytes
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
            hidden[slot * N + act_pos<BITS>(n)] = __float2bfloat16_rn(h);
          }
        } else {
#pragma unroll
          for (int mt = 0; mt < MMA_MT; ++mt) {
            const int n = row0 + 16 * mt + g + 8 * (i >> 1);
            if (n >= N) continue;
            if (phase == 0)
              hidden[slot * N + act_pos<BITS>(n)] = __float2bfloat16_rn(fmaxf(tot[mt][nt][i], 0.0f));
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
  pdl_wait();
  pdl_trigger();
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

// x rows -> expert-sorted order, in the activation layout of the owning expert's bitwidth
__global__ void __launch_bounds__(128)
    scatter_x_kernel(const ExpertDev* __restrict__ experts, const __nv_bfloat16* __restrict__ x,
                     const int32_t* __restrict__ ids, const int32_t* __restrict__ perm, const int32_t* __restrict__ off,
                     int E, int* __restrict__ plan, int top_k, int d, int n_pairs, int fmt, int cnt_lo, int cnt_hi,
                     __nv_bfloat16* __restrict__ xs, float* __restrict__ xsc, int* __restrict__ check_word) {
  pdl_wait();
  pdl_trigger();
  if (plan && blockIdx.x == 0 && threadIdx.x < 32) build_plan(plan, experts, off, E, cnt_lo, cnt_hi, threadIdx.x);
  const int slot = blockIdx.x;
  const int pair = perm[slot];
  if (pair < 0 || pair >= n_pairs) return;
  const int e_slot = ids[pair];
  if (e_slot < 0 || e_slot >= E) return;  // a slot the permutation did not write (stale entry behind a dropped pair)
  const int cnt_slot = off[e_slot + 1] - off[e_slot];
  if (cnt_slot < cnt_lo || cnt_slot > cnt_hi) return;  // this expert's rows belong to another kernel family
  scatter_any(x + static_cast<size_t>(pair / top_k) * d, xs, xsc, slot, d, experts[e_slot].bits, fmt, check_word);
}

// Permutation and scatter in one launch for small batches (at most PS_MAX_PAIRS pairs): one CTA
// per pair.  Every CTA reads all expert ids and works out its own pair's slot (pairs with a lower
// expert id come first, then pairs of the same expert with a lower index: the stable counting
// sort of the definition), writes perm / slot_of_pair for it and copies its row; CTA 0 also
// writes counts, offsets and the work plan.  No CTA waits for another.
constexpr int PS_MAX_PAIRS = 1024;
__global__ void __launch_bounds__(128)
    permute_scatter_kernel(const ExpertDev* __restrict__ experts, const __nv_bfloat16* __restrict__ x,
                           const int32_t* __restrict__ ids, int E, int top_k, int d, int n_pairs, int fmt,
                           int32_t* __restrict__ counts, int32_t* __restrict__ off, int32_t* __restrict__ perm,
                           int32_t* __restrict__ slot_of_pair, int* __restrict__ plan, int* __restrict__ check_word,
                           __nv_bfloat16* __restrict__ xs, float* __restrict__ xsc) {
  __shared__ int s_ids[PS_MAX_PAIRS];
  __shared__ int s_off[EMOE_MAX_EXPERTS + 1];
  __shared__ int s_red[2][4];
  pdl_wait();
  pdl_trigger();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int q = tid; q < n_pairs; q += blockDim.x) s_ids[q] = ids[q];
  __syncthreads();
  const int p = blockIdx.x;
  const int e = s_ids[p];
  const bool valid = e >= 0 && e < E;
  // pairs in front of this one in expert order
  int before = 0, same = 0;
  for (int q = tid; q < n_pairs; q += blockDim.x) {
    const int eq = s_ids[q];
    before += (eq >= 0 && eq < e) || (eq == e && q < p);
    same += eq == e;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    before += __shfl_xor_sync(0xffffffffu, before, o);
    same += __shfl_xor_sync(0xffffffffu, same, o);
  }
  if (lane == 0) {
    s_red[0][warp] = before;
    s_red[1][warp] = same;
  }
  __syncthreads();
  const int slot = s_red[0][0] + s_red[0][1] + s_red[0][2] + s_red[0][3];
  if (p == 0) {
    // counts, offsets, plan (this CTA only); invalid ids are reported and own no slot
    for (int ee = tid; ee <= E; ee += blockDim.x) s_off[ee] = 0;
    __syncthreads();
    bool bad = false;
    for (int q = tid; q < n_pairs; q += blockDim.x) {
      const int eq = s_ids[q];
      if (eq >= 0 && eq < E) atomicAdd(&s_off[eq + 1], 1);
      else bad = true;
    }
    if (bad) atomicOr(check_word, CHECK_BAD_EXPERT_ID);
    __syncthreads();
    if (warp == 0) counts_to_offsets(s_off, counts, E, lane);
    __syncthreads();
    for (int ee = tid; ee <= E; ee += blockDim.x) off[ee] = s_off[ee];
    if (warp == 0) build_plan(plan, experts, s_off, E, 1, 0x7fffffff, lane);
  }
  if (!valid) {
    if (tid == 0) slot_of_pair[p] = -1;
    return;
  }
  if (tid == 0) {
    perm[slot] = p;
    slot_of_pair[p] = slot;
  }
  scatter_any(x + static_cast<size_t>(p / top_k) * d, xs, xsc, slot, d, experts[e].bits, fmt, check_word);
}


}  // namespace

// 8-token tiles a CTA handles per pass over its weights.  A pass with one tile is the cheapest
// per byte by far (measured on the streaming kernel: 1 : 1.6 for one against two tiles), and an
// expert with more tokens simply takes another pass over its own weights (from L2), so one tile
// wins as long as the mean tokens per expert under uniform routing stay below about 12 (expected
// passes below 1.6); beyond that two tiles.  Four tiles only on request.
int ffn_token_tiles(const LayerDims& L, int T) {
  const double mean = static_cast<double>(T) * L.top_k / L.E;
  return mean <= 12.0 ? 1 : 2;
}

// Enough tokens per expert (mean of 16 under uniform routing) that the experts with many tokens
// are a dense contraction: those go to the tcgen05 grouped GEMM.
bool ffn_many_tokens(const LayerDims& L, int T) { return static_cast<double>(T) * L.top_k / L.E >= 16.0; }

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
                             const int32_t* perm, const int32_t* off, int* plan, __nv_bfloat16* xs, float* xsc, int n_pairs,
                             int fmt, int cnt_lo, int cnt_hi, int* check_word, cudaStream_t st) {
  return launch_chain(scatter_x_kernel, dim3(n_pairs), dim3(128), 0, st, experts, reinterpret_cast<const __nv_bfloat16*>(x), ids,
                      perm, off, L.E, plan, L.top_k, L.d_model, n_pairs, fmt, cnt_lo, cnt_hi, xs, xsc, check_word);
}

bool permute_scatter_supported(const LayerDims& L, int n_pairs) { return n_pairs <= PS_MAX_PAIRS && L.E <= EMOE_MAX_EXPERTS; }

cudaError_t launch_permute_scatter(const LayerDims& L, const ExpertDev* experts, const void* x, const int32_t* ids,
                                   int32_t* counts, int32_t* off, int32_t* perm, int32_t* slot_of_pair, int* plan,
                                   __nv_bfloat16* xs, float* xsc, int n_pairs, int fmt, int* check_word, cudaStream_t st) {
  return launch_chain(permute_scatter_kernel, dim3(n_pairs), dim3(128), 0, st, experts, reinterpret_cast<const __nv_bfloat16*>(x),
                      ids, L.E, L.top_k, L.d_model, n_pairs, fmt, counts, off, perm, slot_of_pair, plan, check_word,
                      xs, xsc);
}

cudaError_t launch_ffn_mma(int phase, const LayerDims& L, const ExpertDev* experts, const __nv_bfloat16* in,
                           const int32_t* off, __nv_bfloat16* hidden, float* o_part, int ksplit, int n_pairs, int T,
                           cudaStream_t st) {
  const int N = phase == 0 ? L.d_ff : L.d_model;
  const int rows_per_cta = (phase == 0 && L.act == EMOE_ACT_SWIGLU) ? 16 * MMA_WARPS : 16 * MMA_MT * MMA_WARPS;
  const dim3 grid((N + rows_per_cta - 1) / rows_per_cta, phase == 0 ? 1 : ksplit, L.E);
  const int z = phase == 0 ? 1 : ksplit;
  switch (ffn_token_tiles(L, T)) {
    case 1: return launch_chain(ffn_mma_kernel<1>, grid, dim3(MMA_THREADS), 0, st, phase, L, experts, in, off, hidden, o_part, z, n_pairs);
    case 2: return launch_chain(ffn_mma_kernel<2>, grid, dim3(MMA_THREADS), 0, st, phase, L, experts, in, off, hidden, o_part, z, n_pairs);
    default: return launch_chain(ffn_mma_kernel<4>, grid, dim3(MMA_THREADS), 0, st, phase, L, experts, in, off, hidden, o_part, z, n_pairs);
  }
}

}  // namespace emoe
