// Internal declarations shared by the .cu files of libemoe (not part of the ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/emoe.h"

namespace emoe {

// Device copy of one layer's expert table (one entry per expert).
struct ExpertDev {
  int32_t bits;
  int32_t pad;
  const uint8_t* packed[3];
  const void* scales[3];
};

// Bits of the device-side check word.
enum : int {
  CHECK_BAD_EXPERT_ID = 1,
  CHECK_WAIT_TIMEOUT = 2,  // a bounded wait inside a kernel ran out
  CHECK_F16_RANGE = 4,     // a kernel that carries activations as fp16 met a value outside the fp16 range
};

// Work plan of the persistent expert kernels, built on the device after the permutation:
// a 16-byte header {activated experts, item counter of the first projection, of the second, 0}
// followed by one record per activated expert, widest codes first.  `done` counts the finished
// pieces of the expert's first projection (zeroed with the plan): the fused expert kernel starts
// an expert's second projection once the count is complete.
struct PlanRec {
  int32_t e, begin, cnt, bits;
  const void* scales[3];
  int32_t done;
  int32_t pad;
};
constexpr size_t PLAN_HEADER_BYTES = 16;
inline size_t plan_bytes(int E) { return PLAN_HEADER_BYTES + sizeof(PlanRec) * static_cast<size_t>(E); }

struct LayerDims {
  int d_model, d_ff, E, top_k, act, gate_mode, group, scale_f16, act_bf16;
};

// ---- programmatic dependent launch ---------------------------------------------------------
// The kernels of a forward call form a chain on one stream.  When enabled (per host thread,
// set by the forward call from its context), every launch carries the "programmatic stream
// serialization" attribute: the next kernel of the chain may start its prologue (barrier set-up,
// tensor-memory allocation, fetching weights that no kernel of the chain writes) while the
// current one drains.  Device side, every kernel executes pdl_wait() before it touches anything
// an earlier kernel of the chain wrote or read, and pdl_trigger() right after, which lets the
// kernel behind it start.  Without the attribute both are no-ops.
extern thread_local bool g_pdl_enabled;

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chain(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  if (g_pdl_enabled) {
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// expert cache of a context (cache.cu)
struct ExpertCache;
void cache_destroy(ExpertCache* c);

// ---- launchers (each enqueues on `st` and returns the launch error) ---------------------
cudaError_t launch_pack(const float* W, int N, int K, int bits, int group, int scale_f16, int full_range, uint8_t* packed,
                        void* scales, cudaStream_t st);
cudaError_t launch_requant(const uint8_t* in_packed, const void* in_scales, int N, int K, int bits_in, int bits_out,
                           int group, int scale_f16, int full_range, uint8_t* packed, void* scales, cudaStream_t st);

cudaError_t launch_router_topk(const void* x, int x_bf16, int T, int d, const float* Wr, const float* bias,
                               int bias_stride, int E, int top_k, int renorm, int32_t* ids, float* gates,
                               float* logits, cudaStream_t st);

cudaError_t launch_permute(const int32_t* ids, int n_pairs, int E, int32_t* counts, int32_t* off, int32_t* perm,
                           int32_t* slot_of_pair, int* check_word, cudaStream_t st);

// Generic CUDA-core grouped GEMV.
//   phase 0: hidden[slot][f] = act(x[token(slot)] . W~first)      (x gathered through perm)
//   phase 1: o[slot][d]      = hidden[slot] . W~last
// hidden is fp32 (act_bf16 = 0) or bf16 (act_bf16 = 1).
cudaError_t launch_ffn_gemv(int phase, const LayerDims& L, const ExpertDev* experts, const void* x,
                            const int32_t* perm, const int32_t* off, void* hidden, float* o, int n_pairs,
                            cudaStream_t st);

// Tensor-core (mma.sync bf16) grouped kernel for bf16 activations.
// xs: x rows scattered into expert order with the per-bitwidth k-interleave, [n_pairs][d_model] bf16.
// hidden: same interleave, [n_pairs][d_ff] bf16.  o_part: [ksplit][n_pairs][d_model] fp32.
bool ffn_mma_supported(const LayerDims& L);
int ffn_mma_ksplit(const LayerDims& L, int T);
int ffn_token_tiles(const LayerDims& L, int T);
bool ffn_many_tokens(const LayerDims& L, int T);
// plan (nullable): plan_bytes(E) bytes, the work plan for the persistent TMA kernels, filled by block 0.
// fmt: 0 = bf16, 1 = fp16 (saturating; same layout: the TMA-staged kernel's input), 2 = two-limb
// block-scaled integers (act_q.cuh: the int8 tensor-core kernel's input; xsc receives the block scales).
// cnt_lo .. cnt_hi: only experts with that many tokens are listed in the plan and have their rows
// written (1 .. INT_MAX: all activated experts); lets two kernel families share one forward call.
cudaError_t launch_scatter_x(const LayerDims& L, const ExpertDev* experts, const void* x, const int32_t* ids,
                             const int32_t* perm, const int32_t* off, int* plan, __nv_bfloat16* xs, float* xsc, int n_pairs,
                             int fmt, int cnt_lo, int cnt_hi, int* check_word, cudaStream_t st);
// Permutation + scatter + plan in one launch (one CTA per pair) for batches of at most 1024 pairs.
bool permute_scatter_supported(const LayerDims& L, int n_pairs);
bool decode_layer_supported(const LayerDims& L, int T);
int decode_layer_resident_ctas(int device);
cudaError_t launch_decode_layer(const LayerDims& L, const ExpertDev* experts, const void* x, int T, const float* Wr,
                                const float* bias, int bias_stride, const int32_t* ids_in, const float* gates_in,
                                int32_t* ids, float* gates, int32_t* counts, int32_t* off, int32_t* perm,
                                int32_t* slot_of_pair, void* hidden, float* y, float* zpart, size_t zpart_floats,
                                int resident_ctas, int sms, unsigned* sync, unsigned wait_limit, int extra_arrivals,
                                int* check_word, cudaStream_t st);
bool route_permute_scatter_supported(const LayerDims& L, int T, int resident_ctas);
int route_permute_scatter_resident_ctas(int device);
cudaError_t launch_route_permute_scatter(const LayerDims& L, const ExpertDev* experts, const void* x, int T, const float* Wr,
                                         const float* bias, int bias_stride, int32_t* ids, float* gates, int32_t* counts,
                                         int32_t* off, int32_t* perm, int32_t* slot_of_pair, int* plan, __nv_bfloat16* xs,
                                         float* xsc, int fmt, unsigned* sync, unsigned wait_limit, int extra_arrivals,
                                         int* check_word, cudaStream_t st);
cudaError_t launch_permute_scatter(const LayerDims& L, const ExpertDev* experts, const void* x, const int32_t* ids,
                                   int32_t* counts, int32_t* off, int32_t* perm, int32_t* slot_of_pair, int* plan,
                                   __nv_bfloat16* xs, float* xsc, int n_pairs, int fmt, int* check_word, cudaStream_t st);
cudaError_t launch_ffn_mma(int phase, const LayerDims& L, const ExpertDev* experts, const __nv_bfloat16* in,
                           const int32_t* off, __nv_bfloat16* hidden, float* o_part, int ksplit, int n_pairs,
                           int T, cudaStream_t st);

// TMA-staged variant of the tensor-core kernel (needs one tensor map per packed matrix, built
// on the host by encode_weight_tmap and kept next to the expert table: tmaps[e*3 + m], 128 bytes each).
bool ffn_tma_supported(const LayerDims& L);
int ffn_tma_ksplit(const LayerDims& L, int T);
int encode_weight_tmap(void* out_map, const void* packed, int N, int K, int bits);
// Phases [phase_begin, phase_end) of the FFN in one launch: (0,1) first projection, (1,2) second,
// (0,2) both, the second projection of an expert starting as soon as its hidden vectors are complete.
// token_tiles: 8-token tiles per pass (1, 2 or 4), 0 = by the routing statistics of (L, T).
cudaError_t launch_ffn_tma(int phase_begin, int phase_end, const LayerDims& L, const ExpertDev* experts,
                           const void* tmaps, const __nv_bfloat16* xs, const int32_t* off, int* plan,
                           __nv_bfloat16* hidden, float* o_part, int ksplit, int n_pairs, int T, int token_tiles,
                           int* check_word, cudaStream_t st);

// The weight-streaming kernel on 8-bit integer tensor-core operands (tcgen05 kind::i8, accumulators
// and unpacked codes in tensor memory).  xq / hq: activations as two-limb block-scaled integers
// [n_pairs][2][K] with block scales xsc / hsc [n_pairs][K/128] (act_q.cuh).  token_tile: tokens
// per pass (8, 16 or 32), 0 = by the routing statistics of (L, T).  wait_limit: polls before a
// wait inside the kernel gives up (0 = default); dep_extra: test hook, 0 in production.
extern long long* g_i8_profile;  // device buffer [CTAs][16] for the timers of a profiling build (null otherwise)
bool ffn_i8_supported(const LayerDims& L);
int ffn_i8_ksplit(const LayerDims& L, int T);
int ffn_i8_token_tile(const LayerDims& L, int T);
// smaps: [E][3] tensor maps of the scale channels (encode_scale_tmap), or null when a channel is not 16-byte aligned.
int encode_scale_tmap(void* out_map, const void* scales, int N, int row_bytes);
cudaError_t launch_ffn_i8(int phase_begin, int phase_end, const LayerDims& L, const void* wmaps, const void* smaps, const void* xq,
                          const float* xsc, int* plan, void* hq, float* hsc, float* o_part, int ksplit, int n_pairs,
                          int T, int token_tile, unsigned wait_limit, int dep_extra, int* check_word, cudaStream_t st);

// swizzle128: the 128-byte swizzle (operand tiles) or none (plain rows)
int encode_tmap_2d(void* out_map, int dtype, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride_bytes,
                   uint32_t box_inner, uint32_t box_outer, bool swizzle128 = true);

// tcgen05 grouped GEMM for experts with many tokens (fp16 operands, fp32 accumulation in tensor
// memory).  xs16 / hidden16: activations in expert order, fp16, pair order; o: [n_pairs][d_model].
bool ffn_umma_supported(const LayerDims& L);
cudaError_t launch_scatter_x16(const LayerDims& L, const ExpertDev* experts, const void* x, const int32_t* ids,
                               const int32_t* perm, const int32_t* off, int* plan, void* xs16, int n_pairs,
                               int cnt_lo, int cnt_hi, int* check_word, cudaStream_t st);
size_t ffn_umma_scratch_bytes(const LayerDims& L);  // scratch of the gated first projection (0 for other layers)
cudaError_t launch_ffn_umma(int phase, const LayerDims& L, const void* wmaps, const int* plan, const void* in16,
                            void* hidden16, float* o, float* scratch, int n_pairs, int zsplit, int* check_word,
                            cudaStream_t st);
int ffn_umma_zsplit(const LayerDims& L, int T, int sms);  // 1 or 2 slices of the second projection's inputs per unit

// y[t] = sum_j gates[t][j] * sum_z o_part[z][slot_of_pair[t*k+j]]
// o_part holds ksplit partial results, each [n_pairs_stride][d].
cudaError_t launch_combine(const float* o_part, int ksplit, size_t n_pairs_stride, const float* gates,
                           const int32_t* slot_of_pair, int T, int top_k, int d, float* y, cudaStream_t st);

}  // namespace emoe
