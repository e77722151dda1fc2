// emoe_moe_forward_routed_static: the routed layer forward for callers that must not
// allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need a layer
// forward: code running inside a framework that owns the whole device heap and forbids
// outside allocations, plug-ins loaded into a process whose memory pool is fixed at start-up,
// or latency-critical loops where an allocation (which may synchronise the device) is not
// acceptable.  emoe_create allocates, so those callers cannot have a context.  This entry
// point needs none: its intermediate buffers live in a fixed array that is part of the
// library image on every GPU that loads it.
//
// The array below is that scratch.  In host code its name is only a handle of the host-side
// shadow of the symbol, never a device address; the device address is obtained once per
// device with cudaGetSymbolAddress and that pointer is what the kernels receive.
#include <climits>
#include <cstring>

#include "common.cuh"

using namespace emoe;

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = size_t(8) << 20;  // 8 MiB, held by every GPU that loads the library
constexpr int STATIC_MAX_PAIRS = 64;                       // T * top_k
constexpr int MAX_DEVICES = 64;

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

char* g_scratch_addr[MAX_DEVICES] = {};  // device address of g_static_scratch, per device

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

struct StaticLayout {
  size_t check, table, counts, off, perm, slot_of_pair, xs, hidden, o_part, total;
  int ksplit;
};

bool dims_from_desc(const emoe_layer_desc* d, LayerDims* L) {
  if (!d || d->d_model <= 0 || d->d_ff <= 0) return false;
  if (d->n_experts < 1 || d->n_experts > EMOE_MAX_EXPERTS) return false;
  if (d->top_k < 1 || d->top_k > d->n_experts || d->top_k > EMOE_MAX_TOP_K) return false;
  if (d->act != EMOE_ACT_RELU && d->act != EMOE_ACT_SWIGLU) return false;
  if (d->gate_mode != EMOE_GATE_SOFTMAX && d->gate_mode != EMOE_GATE_SOFTMAX_RENORM) return false;
  if (d->scale_dtype != EMOE_DTYPE_F32 && d->scale_dtype != EMOE_DTYPE_F16) return false;
  if (d->act_dtype != EMOE_DTYPE_F32 && d->act_dtype != EMOE_DTYPE_BF16) return false;
  if (d->group < 0 || (d->group > 0 && (d->d_model % d->group != 0 || d->d_ff % d->group != 0))) return false;
  L->d_model = d->d_model;
  L->d_ff = d->d_ff;
  L->E = d->n_experts;
  L->top_k = d->top_k;
  L->act = d->act;
  L->gate_mode = d->gate_mode;
  L->group = d->group;
  L->scale_f16 = d->scale_dtype == EMOE_DTYPE_F16;
  L->act_bf16 = d->act_dtype == EMOE_DTYPE_BF16;
  return true;
}

StaticLayout layout_for(const LayerDims& L, int T) {
  StaticLayout w{};
  const size_t P = static_cast<size_t>(T) * L.top_k;
  w.ksplit = ffn_mma_supported(L) ? ffn_mma_ksplit(L, T) : 1;
  size_t o = 0;
  w.check = o;        o += align_up(sizeof(int));
  w.table = o;        o += align_up(sizeof(ExpertDev) * L.E);
  w.counts = o;       o += align_up(static_cast<size_t>(L.E) * 4);
  w.off = o;          o += align_up(static_cast<size_t>(L.E + 1) * 4);
  w.perm = o;         o += align_up(P * 4);
  w.slot_of_pair = o; o += align_up(P * 4);
  w.xs = o;           o += align_up(L.act_bf16 ? P * L.d_model * 2 : 0);
  w.hidden = o;       o += align_up(P * L.d_ff * (L.act_bf16 ? 2 : 4));
  // fewer split-K partials if the usual number would not fit the fixed array
  while (w.ksplit > 1 && o + align_up(static_cast<size_t>(w.ksplit) * P * L.d_model * 4) > STATIC_SCRATCH_BYTES) --w.ksplit;
  w.o_part = o;       o += align_up(static_cast<size_t>(w.ksplit) * P * L.d_model * 4);
  w.total = o;
  return w;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// The expert table reaches the scratch array as kernel parameters, 64 entries (3.5 KB) per
// launch: parameters are copied when the launch is enqueued (or captured), so no copy node ever
// keeps the address of a host buffer that has gone out of scope, and no pageable copy stalls
// the calling thread behind earlier work on the stream.
constexpr int TABLE_CHUNK = 64;
struct TableChunk {
  ExpertDev e[TABLE_CHUNK];
};
__global__ void write_table_kernel(const __grid_constant__ TableChunk c, ExpertDev* dst, int n, int* check_word) {
  const int i = threadIdx.x;
  if (i < n) dst[i] = c.e[i];
  if (check_word && i == 0) *check_word = 0;  // the array keeps the previous call's contents
}

}  // namespace

extern "C" int emoe_moe_forward_routed_static(int device, const emoe_layer_desc* desc, const void* x, int T,
                                              const int32_t* ids, const float* gates,
                                              const emoe_expert* host_experts, float* y, void* stream) {
  LayerDims L;
  if (!dims_from_desc(desc, &L) || !x || !ids || !gates || !host_experts || !y || T <= 0) return EMOE_ERR_INVALID_ARG;
  if (device < 0 || device >= MAX_DEVICES) return EMOE_ERR_INVALID_ARG;
  if (L.d_model % 32 != 0 || L.d_ff % 32 != 0) return EMOE_ERR_UNSUPPORTED;
  if (!aligned(x, 16) || !aligned(y, 16)) return EMOE_ERR_ALIGNMENT;
  const int nmat = L.act == EMOE_ACT_RELU ? 2 : 3;
  for (int e = 0; e < L.E; ++e) {
    const int b = host_experts[e].bits;
    if (b != 2 && b != 4 && b != 8) return EMOE_ERR_UNSUPPORTED;
    const int wpv = 128 / b;
    if (L.d_model % wpv != 0 || L.d_ff % wpv != 0 || (L.group > 0 && L.group % wpv != 0)) return EMOE_ERR_UNSUPPORTED;
    for (int m = 0; m < nmat; ++m) {
      if (!host_experts[e].packed[m] || !host_experts[e].scales[m]) return EMOE_ERR_INVALID_ARG;
      if (!aligned(host_experts[e].packed[m], 16)) return EMOE_ERR_ALIGNMENT;
      if (!aligned(host_experts[e].scales[m], 4)) return EMOE_ERR_ALIGNMENT;
    }
  }
  // the fixed array bounds the problem size: refuse anything that does not fit
  if (static_cast<long long>(T) * L.top_k > STATIC_MAX_PAIRS) return EMOE_ERR_WORKSPACE;
  const StaticLayout w = layout_for(L, T);
  if (w.total > STATIC_SCRATCH_BYTES) return EMOE_ERR_WORKSPACE;

  if (cudaSetDevice(device) != cudaSuccess) return EMOE_ERR_CUDA;
  if (!g_scratch_addr[device]) {
    // set-up, once per device, with that device current: the symbol's device address
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return EMOE_ERR_CUDA;
    g_scratch_addr[device] = static_cast<char*>(p);
  }
  char* ws = g_scratch_addr[device];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int P = T * L.top_k;

  ExpertDev* table = reinterpret_cast<ExpertDev*>(ws + w.table);
  int* check = reinterpret_cast<int*>(ws + w.check);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + w.counts);
  int32_t* off = reinterpret_cast<int32_t*>(ws + w.off);
  int32_t* perm = reinterpret_cast<int32_t*>(ws + w.perm);
  int32_t* slot_of_pair = reinterpret_cast<int32_t*>(ws + w.slot_of_pair);
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(ws + w.xs);
  void* hidden = ws + w.hidden;
  float* o_part = reinterpret_cast<float*>(ws + w.o_part);

#define EMOE_TRY(call) \
  do {                 \
    if ((call) != cudaSuccess) return EMOE_ERR_CUDA; \
  } while (0)
  // the expert table travels as launch parameters; the first chunk's kernel also clears the check
  // word (the array keeps whatever the previous call left)
  for (int e0 = 0; e0 < L.E; e0 += TABLE_CHUNK) {
    TableChunk chunk;
    const int n = L.E - e0 < TABLE_CHUNK ? L.E - e0 : TABLE_CHUNK;
    for (int i = 0; i < n; ++i) {
      chunk.e[i].bits = host_experts[e0 + i].bits;
      chunk.e[i].pad = 0;
      for (int m = 0; m < 3; ++m) {
        chunk.e[i].packed[m] = static_cast<const uint8_t*>(host_experts[e0 + i].packed[m]);
        chunk.e[i].scales[m] = host_experts[e0 + i].scales[m];
      }
    }
    for (int i = n; i < TABLE_CHUNK; ++i) chunk.e[i] = ExpertDev{};
    write_table_kernel<<<1, TABLE_CHUNK, 0, st>>>(chunk, table + e0, n, e0 == 0 ? check : nullptr);
    EMOE_TRY(cudaGetLastError());
  }
  EMOE_TRY(launch_permute(ids, P, L.E, counts, off, perm, slot_of_pair, check, st));
  if (ffn_mma_supported(L)) {
    EMOE_TRY(launch_scatter_x(L, table, x, ids, perm, off, nullptr, xs, nullptr, P, 0, 1, INT_MAX, check, st));
    EMOE_TRY(launch_ffn_mma(0, L, table, xs, off, reinterpret_cast<__nv_bfloat16*>(hidden), o_part, 1, P, T, st));
    EMOE_TRY(launch_ffn_mma(1, L, table, reinterpret_cast<const __nv_bfloat16*>(hidden), off,
                            reinterpret_cast<__nv_bfloat16*>(hidden), o_part, w.ksplit, P, T, st));
    EMOE_TRY(launch_combine(o_part, w.ksplit, static_cast<size_t>(P), gates, slot_of_pair, T, L.top_k, L.d_model, y, st));
  } else {
    EMOE_TRY(launch_ffn_gemv(0, L, table, x, perm, off, hidden, o_part, P, st));
    EMOE_TRY(launch_ffn_gemv(1, L, table, x, perm, off, hidden, o_part, P, st));
    EMOE_TRY(launch_combine(o_part, 1, static_cast<size_t>(P), gates, slot_of_pair, T, L.top_k, L.d_model, y, st));
  }
#undef EMOE_TRY
  return EMOE_OK;
}

extern "C" int emoe_static_device_status(int device, void* stream) {
  if (device < 0 || device >= MAX_DEVICES) return EMOE_ERR_INVALID_ARG;
  if (cudaSetDevice(device) != cudaSuccess) return EMOE_ERR_CUDA;
  if (!g_scratch_addr[device]) return EMOE_OK;  // no call has run on this device yet
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  // the check word is the first thing in the scratch array (StaticLayout::check == 0)
  if (cudaMemcpyAsync(&word, g_scratch_addr[device], sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return EMOE_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return EMOE_ERR_CUDA;
  if (word & CHECK_WAIT_TIMEOUT) return EMOE_ERR_TIMEOUT;
  return word ? EMOE_ERR_DEVICE_CHECK : EMOE_OK;
}
