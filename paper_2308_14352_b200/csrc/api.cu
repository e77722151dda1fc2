// C ABI of libemoe: context, argument checks, and the orchestration of one layer forward
// (router -> Top-K -> permutation -> expert FFNs on packed weights -> combine).  All
// arithmetic is in the kernels of the sibling files; nothing here touches tensor data on the
// host.
#include <climits>
#include <cstring>
#include <new>
#include <unordered_map>
#include <vector>

#include "common.cuh"

using namespace emoe;

namespace emoe {
thread_local bool g_pdl_enabled = false;
}

namespace {

constexpr int MAX_TABLES = 128;  // distinct expert tables a context can keep on the device
constexpr size_t TMAP_BYTES = 128;  // sizeof(CUtensorMap)
// one table block: the expert entries followed by one tensor map per (expert, matrix)
constexpr size_t TABLE_MAPS_OFFSET = (sizeof(ExpertDev) * EMOE_MAX_EXPERTS + 127) / 128 * 128;
// ... followed by one tensor map per (expert, scale channel) for the int8 streaming kernel's scale windows
constexpr size_t TABLE_SMAPS_OFFSET = TABLE_MAPS_OFFSET + TMAP_BYTES * 3 * EMOE_MAX_EXPERTS;
constexpr size_t TABLE_BLOCK_BYTES = TABLE_SMAPS_OFFSET + TMAP_BYTES * 3 * EMOE_MAX_EXPERTS;

struct TableEntry {
  std::vector<emoe_expert> host;
  int d_model = 0, d_ff = 0, act = 0;
  bool has_tmaps = false;
  bool scales16 = false;  // every scale channel is 16-byte aligned (bulk copies of scales are possible)
};

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

struct WorkspaceLayout {
  size_t ids, gates, counts, off, perm, slot_of_pair, plan, xs, hidden, xsc, hsc, o_part, um_scratch, um_scratch_bytes, total;
  int ksplit;
};

bool make_dims(const emoe_layer_desc* d, LayerDims* L) {
  if (!d) return false;
  if (d->d_model <= 0 || d->d_ff <= 0) return false;
  if (d->n_experts < 1 || d->n_experts > EMOE_MAX_EXPERTS) return false;
  if (d->top_k < 1 || d->top_k > d->n_experts || d->top_k > EMOE_MAX_TOP_K) return false;
  if (d->act != EMOE_ACT_RELU && d->act != EMOE_ACT_SWIGLU) return false;
  if (d->gate_mode != EMOE_GATE_SOFTMAX && d->gate_mode != EMOE_GATE_SOFTMAX_RENORM) return false;
  if (d->scale_dtype != EMOE_DTYPE_F32 && d->scale_dtype != EMOE_DTYPE_F16) return false;
  if (d->act_dtype != EMOE_DTYPE_F32 && d->act_dtype != EMOE_DTYPE_BF16) return false;
  if (d->group < 0) return false;
  if (d->group > 0 && (d->d_model % d->group != 0 || d->d_ff % d->group != 0)) return false;
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

WorkspaceLayout make_layout(const LayerDims& L, int T) {
  WorkspaceLayout w{};
  const size_t P = static_cast<size_t>(T) * L.top_k;
  w.ksplit = 1;
  if (ffn_mma_supported(L)) w.ksplit = ffn_mma_ksplit(L, T);
  if (ffn_tma_supported(L) && ffn_tma_ksplit(L, T) > w.ksplit) w.ksplit = ffn_tma_ksplit(L, T);
  if (ffn_i8_supported(L) && ffn_i8_ksplit(L, T) > w.ksplit) w.ksplit = ffn_i8_ksplit(L, T);
  size_t o = 0;
  w.ids = o;          o += align_up(P * 4);
  w.gates = o;        o += align_up(P * 4);
  w.counts = o;       o += align_up(static_cast<size_t>(L.E) * 4);
  w.off = o;          o += align_up(static_cast<size_t>(L.E + 1) * 4);
  w.perm = o;         o += align_up(P * 4);
  w.slot_of_pair = o; o += align_up(P * 4);
  w.plan = o;         o += 2 * align_up(plan_bytes(L.E));  // two plans: one per kernel family of a forward call
  w.xs = o;           o += align_up(L.act_bf16 ? P * L.d_model * 2 : 0);
  w.hidden = o;       o += align_up(P * L.d_ff * (L.act_bf16 ? 2 : 4));
  // block scales of the integer activations (int8 tensor-core kernel): one fp32 per 128 inputs
  w.xsc = o;          o += align_up(ffn_i8_supported(L) ? P * (L.d_model / 128) * 4 : 0);
  w.hsc = o;          o += align_up(ffn_i8_supported(L) ? P * (L.d_ff / 128) * 4 : 0);
  w.o_part = o;       o += align_up(static_cast<size_t>(w.ksplit) * P * L.d_model * 4);
  // scratch of the tcgen05 kernel's gated first projection: only calls with at least one full token tile of
  // pairs can take that kernel's many-token shapes
  w.um_scratch = o;
  w.um_scratch_bytes = (ffn_umma_supported(L) && P >= 128) ? ffn_umma_scratch_bytes(L) : 0;
  o += align_up(w.um_scratch_bytes);
  w.total = o;
  return w;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

struct emoe_ctx {
  int device = 0;
  char* workspace = nullptr;
  size_t workspace_bytes = 0;
  int* check_word = nullptr;        // device
  int* check_host = nullptr;        // pinned
  char* tables_dev = nullptr;  // MAX_TABLES blocks of TABLE_BLOCK_BYTES
  char* tables_pin = nullptr;  // pinned mirror, never rewritten once filled
  std::vector<TableEntry> tables;
  int last_cuda = 0;
  int ffn_path = 0;
  bool pdl = true;  // programmatic dependent launch along the kernel chain of a forward call
  bool fuse_projections = true;  // weight-streaming kernel: both projections in one launch
  bool fuse_routing = false;     // router + Top-K + permutation + scatter + plan in one launch (small batches)
  bool timing = false;
  unsigned wait_limit = 0;  // polls before a wait inside the int8 streaming kernel gives up (0 = its default)
  int dep_extra = 0;        // test hook: extra completions the second projection waits for
  int fuse_layer = 2;       // small layer, a handful of tokens: the whole layer in one launch (0 never, 1 whenever it can, 2 where it was measured faster)
  int resident_layer_ctas = -1;  // CTAs of the one-launch layer kernel the device holds at once (-1: not asked yet)
  int sms = 0;
  const int32_t* last_counts = nullptr;  // device: per-expert pair counts of the last forward call
  int last_counts_n = 0;
  // tensor maps by what they describe: a matrix that comes back (a cache slot, a resident expert in a
  // new table) is not encoded again
  struct MapKey {
    const void* ptr;
    int a, b, c;
    bool operator==(const MapKey& o) const { return ptr == o.ptr && a == o.a && b == o.b && c == o.c; }
  };
  struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
      size_t h = reinterpret_cast<size_t>(k.ptr) * 0x9E3779B97F4A7C15ull;
      h ^= (static_cast<size_t>(k.a) << 40) ^ (static_cast<size_t>(k.b) << 16) ^ static_cast<size_t>(k.c);
      return h;
    }
  };
  struct MapBytes {
    char b[128];
    int rc;
  };
  std::unordered_map<MapKey, MapBytes, MapKeyHash> map_cache;
  int resident_route_ctas = -1;  // CTAs of the one-launch routing kernel the device holds at once (-1 = not asked yet)
  int kernels_last = 0;  // kernels the last forward call enqueued
  ExpertCache* cache = nullptr;  // expert cache (cache.cu), optional
  std::vector<cudaEvent_t> table_events;  // per table block: its upload has left the pinned mirror
  std::vector<uint64_t> table_used;       // per table block: last use (for recycling)
  uint64_t table_clock = 0;
  std::vector<cudaEvent_t> events;  // triples (start, mid, end) per timed forward call
  size_t events_used = 0;
  std::vector<char> events_one_launch;  // per triple: both projections ran as one launch (no second interval)
};

namespace {

int cuda_fail(emoe_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda = static_cast<int>(e);
  return EMOE_ERR_CUDA;
}

#define EMOE_CUDA(ctx, call)                          \
  do {                                                \
    cudaError_t e__ = (call);                         \
    if (e__ != cudaSuccess) return cuda_fail(ctx, e__); \
  } while (0)

// a kernel launch of a forward call: counted, so that callers can report how many kernels ran
#define EMOE_LAUNCH(ctx, call) \
  do {                         \
    EMOE_CUDA(ctx, call);      \
    ++(ctx)->kernels_last;     \
  } while (0)

// encode_weight_tmap / encode_scale_tmap through the context's cache (kind 0: packed weights with
// a = N, b = K, c = bits; kind 1: scale channel with a = N, b = row bytes)
int cached_tmap(emoe_ctx* ctx, int kind, void* out, const void* ptr, int a, int b, int c) {
  const emoe_ctx::MapKey key{ptr, a, b, kind == 0 ? c : -1};
  auto it = ctx->map_cache.find(key);
  if (it == ctx->map_cache.end()) {
    if (ctx->map_cache.size() > 16384) ctx->map_cache.clear();
    emoe_ctx::MapBytes mb;
    std::memset(mb.b, 0, sizeof(mb.b));
    mb.rc = kind == 0 ? encode_weight_tmap(mb.b, ptr, a, b, c) : encode_scale_tmap(mb.b, ptr, a, b);
    it = ctx->map_cache.emplace(key, mb).first;
  }
  std::memcpy(out, it->second.b, 128);
  return it->second.rc;
}

// Device copy of a host expert table (entries + tensor maps); uploaded on `st` the first time
// its content is seen.  *tmaps is null when the shape has no TMA path.
int get_table(emoe_ctx* ctx, const LayerDims& L, const emoe_expert* host, cudaStream_t st, const ExpertDev** out,
              const void** tmaps, const void** smaps) {
  const int E = L.E;
  for (size_t i = 0; i < ctx->tables.size(); ++i) {
    const TableEntry& te = ctx->tables[i];
    if (static_cast<int>(te.host.size()) != E || te.d_model != L.d_model || te.d_ff != L.d_ff || te.act != L.act) continue;
    bool same = true;
    for (int e = 0; e < E && same; ++e) {
      same = te.host[e].bits == host[e].bits;
      for (int m = 0; m < 3 && same; ++m)
        same = te.host[e].packed[m] == host[e].packed[m] && te.host[e].scales[m] == host[e].scales[m];
    }
    if (same) {
      ctx->table_used[i] = ++ctx->table_clock;
      *out = reinterpret_cast<const ExpertDev*>(ctx->tables_dev + i * TABLE_BLOCK_BYTES);
      *tmaps = te.has_tmaps ? ctx->tables_dev + i * TABLE_BLOCK_BYTES + TABLE_MAPS_OFFSET : nullptr;
      *smaps = te.has_tmaps && te.scales16 ? ctx->tables_dev + i * TABLE_BLOCK_BYTES + TABLE_SMAPS_OFFSET : nullptr;
      return EMOE_OK;
    }
  }
  // A new table: the next unused block, or (tables that change from call to call, e.g. pointers
  // into an expert cache) the block that was used longest ago, once its upload has left the
  // pinned mirror.  Kernels that read the old device copy were enqueued earlier on the stream.
  size_t slot = ctx->tables.size();
  const bool recycle = slot >= MAX_TABLES;
  if (recycle) {
    slot = 0;
    for (size_t i = 1; i < ctx->tables.size(); ++i)
      if (ctx->table_used[i] < ctx->table_used[slot]) slot = i;
    EMOE_CUDA(ctx, cudaEventSynchronize(ctx->table_events[slot]));
  }
  char* pin_block = ctx->tables_pin + slot * TABLE_BLOCK_BYTES;
  ExpertDev* pin = reinterpret_cast<ExpertDev*>(pin_block);
  const int nmat = L.act == EMOE_ACT_RELU ? 2 : 3;
  bool maps_ok = ffn_tma_supported(L);
  bool scales16 = true;
  const int ssz = L.scale_f16 ? 2 : 4;
  for (int e = 0; e < E; ++e) {
    pin[e].bits = host[e].bits;
    pin[e].pad = 0;
    for (int m = 0; m < 3; ++m) {
      pin[e].packed[m] = static_cast<const uint8_t*>(host[e].packed[m]);
      pin[e].scales[m] = host[e].scales[m];
    }
    for (int m = 0; m < nmat && maps_ok; ++m) {
      const bool first = m < nmat - 1;
      const int N = first ? L.d_ff : L.d_model, K = first ? L.d_model : L.d_ff;
      maps_ok = cached_tmap(ctx, 0, pin_block + TABLE_MAPS_OFFSET + TMAP_BYTES * (3 * e + m), host[e].packed[m], N, K,
                            host[e].bits) == 0;
      // the scale channel's map, where its rows allow one (long rows in multiples of 16 bytes)
      const int row_bytes = (L.group > 0 ? K / L.group : 1) * ssz;
      char* smap = pin_block + TABLE_SMAPS_OFFSET + TMAP_BYTES * (3 * e + m);
      if (!aligned(host[e].scales[m], 16)) scales16 = false;
      else if (cached_tmap(ctx, 1, smap, host[e].scales[m], N, row_bytes, 0) != 0) std::memset(smap, 0, TMAP_BYTES);
    }
  }
  char* dev = ctx->tables_dev + slot * TABLE_BLOCK_BYTES;
  if (maps_ok) {  // entries + weight maps in one copy, the scale maps (behind the unused weight maps) in another
    EMOE_CUDA(ctx, cudaMemcpyAsync(dev, pin_block, TABLE_MAPS_OFFSET + TMAP_BYTES * 3 * E, cudaMemcpyHostToDevice, st));
    if (scales16)
      EMOE_CUDA(ctx, cudaMemcpyAsync(dev + TABLE_SMAPS_OFFSET, pin_block + TABLE_SMAPS_OFFSET, TMAP_BYTES * 3 * E,
                                     cudaMemcpyHostToDevice, st));
  } else {
    EMOE_CUDA(ctx, cudaMemcpyAsync(dev, pin_block, sizeof(ExpertDev) * E, cudaMemcpyHostToDevice, st));
  }
  TableEntry te;
  te.host.assign(host, host + E);
  te.d_model = L.d_model;
  te.d_ff = L.d_ff;
  te.act = L.act;
  te.has_tmaps = maps_ok;
  te.scales16 = scales16;
  if (recycle) {
    ctx->tables[slot] = std::move(te);
  } else {
    ctx->tables.push_back(std::move(te));
    cudaEvent_t ev;
    EMOE_CUDA(ctx, cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    ctx->table_events.push_back(ev);
    ctx->table_used.push_back(0);
  }
  EMOE_CUDA(ctx, cudaEventRecord(ctx->table_events[slot], st));
  ctx->table_used[slot] = ++ctx->table_clock;
  *out = reinterpret_cast<const ExpertDev*>(dev);
  *tmaps = maps_ok ? dev + TABLE_MAPS_OFFSET : nullptr;
  *smaps = maps_ok && scales16 ? dev + TABLE_SMAPS_OFFSET : nullptr;
  return EMOE_OK;
}

int check_experts(const LayerDims& L, const emoe_expert* host) {
  const int nmat = L.act == EMOE_ACT_RELU ? 2 : 3;
  for (int e = 0; e < L.E; ++e) {
    const int b = host[e].bits;
    if (b != 2 && b != 4 && b != 8) return EMOE_ERR_UNSUPPORTED;
    const int wpv = 128 / b;  // weights per 128-bit load
    if (L.d_model % wpv != 0 || L.d_ff % wpv != 0) return EMOE_ERR_UNSUPPORTED;
    if (L.group > 0 && L.group % wpv != 0) return EMOE_ERR_UNSUPPORTED;
    for (int m = 0; m < nmat; ++m) {
      if (!host[e].packed[m] || !host[e].scales[m]) return EMOE_ERR_INVALID_ARG;
      if (!aligned(host[e].packed[m], 16)) return EMOE_ERR_ALIGNMENT;
      if (!aligned(host[e].scales[m], 4)) return EMOE_ERR_ALIGNMENT;
    }
  }
  return EMOE_OK;
}

int forward_impl(emoe_ctx* ctx, const emoe_layer_desc* desc, const void* x, int T, const float* router_W,
                 const float* router_bias, int bias_token_stride, const int32_t* ids_in, const float* gates_in,
                 const emoe_expert* host_experts, float* y, int32_t* out_ids, float* out_gates, int32_t* out_perm,
                 cudaStream_t st) {
  LayerDims L;
  if (!ctx || !make_dims(desc, &L)) return EMOE_ERR_INVALID_ARG;
  if (!x || !y || !host_experts || T <= 0) return EMOE_ERR_INVALID_ARG;
  const bool routed = ids_in != nullptr;
  if (routed ? gates_in == nullptr : router_W == nullptr) return EMOE_ERR_INVALID_ARG;
  if (!routed && router_bias && bias_token_stride != 0 && bias_token_stride != L.E) return EMOE_ERR_INVALID_ARG;
  if (L.d_model % 32 != 0 || L.d_ff % 32 != 0) return EMOE_ERR_UNSUPPORTED;
  if (static_cast<long long>(T) * L.top_k > 0x7fffffffLL / 4) return EMOE_ERR_UNSUPPORTED;
  if (!aligned(x, 16) || !aligned(y, 16)) return EMOE_ERR_ALIGNMENT;
  int rc = check_experts(L, host_experts);
  if (rc != EMOE_OK) return rc;
  const WorkspaceLayout w = make_layout(L, T);
  if (w.total > ctx->workspace_bytes) return EMOE_ERR_WORKSPACE;
  EMOE_CUDA(ctx, cudaSetDevice(ctx->device));
  struct PdlScope {
    explicit PdlScope(bool on) { g_pdl_enabled = on; }
    ~PdlScope() { g_pdl_enabled = false; }
  } pdl_scope(ctx->pdl && !ctx->timing);

  ctx->kernels_last = 0;
  const ExpertDev* table = nullptr;
  const void* tmaps = nullptr;
  const void* smaps = nullptr;
  rc = get_table(ctx, L, host_experts, st, &table, &tmaps, &smaps);
  if (rc != EMOE_OK) return rc;

  char* ws = ctx->workspace;
  const int P = T * L.top_k;
  int32_t* ids = reinterpret_cast<int32_t*>(ws + w.ids);
  float* gates = reinterpret_cast<float*>(ws + w.gates);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + w.counts);
  int32_t* off = reinterpret_cast<int32_t*>(ws + w.off);
  int32_t* perm = reinterpret_cast<int32_t*>(ws + w.perm);
  int32_t* slot_of_pair = reinterpret_cast<int32_t*>(ws + w.slot_of_pair);
  int* plan = reinterpret_cast<int*>(ws + w.plan);
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(ws + w.xs);
  void* hidden = ws + w.hidden;
  float* xsc = reinterpret_cast<float*>(ws + w.xsc);
  float* hsc = reinterpret_cast<float*>(ws + w.hsc);
  float* o_part = reinterpret_cast<float*>(ws + w.o_part);
  float* um_scratch = w.um_scratch_bytes ? reinterpret_cast<float*>(ws + w.um_scratch) : nullptr;

  ctx->last_counts = counts;
  ctx->last_counts_n = L.E;
  const int32_t* ids_use = routed ? ids_in : ids;
  const float* gates_use = routed ? gates_in : gates;
  const bool can_tma = ffn_tma_supported(L) && tmaps != nullptr;
  const bool can_i8 = ffn_i8_supported(L) && tmaps != nullptr;
  // (a gated layer needs the kernel's scratch block, which calls below one token tile of pairs do not carry)
  const bool can_umma = ffn_umma_supported(L) && tmaps != nullptr && (L.act != EMOE_ACT_SWIGLU || um_scratch != nullptr);
  // many tokens per expert: the tcgen05 grouped GEMM; otherwise the weight-streaming kernels
  const bool many_tokens = ffn_many_tokens(L, T);
  // skewed loads: experts with few tokens stream through the TMA kernel, the others take the
  // tcgen05 grouped GEMM, in the same forward call
  // ... unless the experts hold hundreds of tokens each on average: then next to nobody is left for the streaming
  // family, whose launch, cleared split-K plane and second plan would only cost
  const bool dense_tokens = static_cast<double>(T) * L.top_k / L.E >= 256.0;
  const bool use_hybrid = can_umma && can_tma && (ctx->ffn_path == 5 || (ctx->ffn_path == 0 && many_tokens && !dense_tokens));
  const bool use_umma = !use_hybrid && can_umma && (ctx->ffn_path == 4 || (ctx->ffn_path == 0 && many_tokens));
  // the weight-streaming kernels: the fp16 mma.sync one by default (the faster of the two as measured), the
  // one on int8 tcgen05 operands on request
  const bool use_i8 = !use_hybrid && !use_umma && can_i8 && ctx->ffn_path == 6;
  const bool use_tma = !use_hybrid && !use_umma && !use_i8 && can_tma && (ctx->ffn_path == 0 || ctx->ffn_path == 3);
  const bool use_mma = ffn_mma_supported(L) && ctx->ffn_path != 1;
  if (ctx->ffn_path == 2 && !use_mma) return EMOE_ERR_UNSUPPORTED;
  if (ctx->ffn_path == 3 && !use_tma) return EMOE_ERR_UNSUPPORTED;
  if (ctx->ffn_path == 4 && !use_umma) return EMOE_ERR_UNSUPPORTED;
  if (ctx->ffn_path == 5 && !use_hybrid) return EMOE_ERR_UNSUPPORTED;
  if (ctx->ffn_path == 6 && !use_i8) return EMOE_ERR_UNSUPPORTED;
  // small batches on the streaming kernels: permutation, scatter and plan in one launch
  const bool one_launch_permute = (use_tma || use_i8) && ctx->fuse_projections && permute_scatter_supported(L, P);
  // ... and, when the router runs here too, router and Top-K in that same launch
  if (ctx->resident_route_ctas < 0) ctx->resident_route_ctas = route_permute_scatter_resident_ctas(ctx->device);
  const bool one_launch_route =
      ctx->fuse_routing && one_launch_permute && !routed && route_permute_scatter_supported(L, T, ctx->resident_route_ctas);
  // a handful of tokens on a small layer: router, both projections and the gate-weighted sum in one launch
  bool one_launch_layer = false;
  // as measured on a Switch-base-sized layer: 1.8 x faster than the chain of launches for one pair, 1.5 x for two to four, 1.25 x
  // for eight, slower for sixteen (the projections then take several passes of dependent loads per warp)
  const bool layer_wanted = ctx->fuse_layer == 1 || (ctx->fuse_layer == 2 && P <= 8);
  if (layer_wanted && ctx->ffn_path == 0 && decode_layer_supported(L, T)) {
    if (ctx->resident_layer_ctas < 0) {
      ctx->resident_layer_ctas = decode_layer_resident_ctas(ctx->device);
      EMOE_CUDA(ctx, cudaDeviceGetAttribute(&ctx->sms, cudaDevAttrMultiProcessorCount, ctx->device));
    }
    one_launch_layer = ctx->sms >= T && ctx->resident_layer_ctas >= ctx->sms;  // at least one CTA per SM, one per token
  }
  if (!routed && !one_launch_route && !one_launch_layer)
    EMOE_LAUNCH(ctx, launch_router_topk(x, L.act_bf16, T, L.d_model, router_W, router_bias, bias_token_stride, L.E,
                                      L.top_k, L.gate_mode == EMOE_GATE_SOFTMAX_RENORM, ids, gates, nullptr, st));
  unsigned* route_sync = reinterpret_cast<unsigned*>(ctx->check_word + 1);
  const unsigned route_wait = ctx->wait_limit ? ctx->wait_limit : (1u << 22);
  if (!one_launch_permute && !one_launch_layer)
    EMOE_LAUNCH(ctx, launch_permute(ids_use, P, L.E, counts, off, perm, slot_of_pair, ctx->check_word, st));
  int ksplit = 1;
  cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
  if (ctx->timing) {
    while (ctx->events.size() < ctx->events_used + 3) {
      cudaEvent_t e;
      EMOE_CUDA(ctx, cudaEventCreate(&e));
      ctx->events.push_back(e);
    }
    for (int i = 0; i < 3; ++i) ev[i] = ctx->events[ctx->events_used + i];
    if (ctx->events_one_launch.size() < ctx->events_used / 3 + 1) ctx->events_one_launch.resize(ctx->events_used / 3 + 1);
    ctx->events_one_launch[ctx->events_used / 3] = 0;
    ctx->events_used += 3;
  }
  if (one_launch_layer) {
    if (ev[0]) EMOE_CUDA(ctx, cudaEventRecord(ev[0], st));
    EMOE_LAUNCH(ctx, launch_decode_layer(L, table, x, T, routed ? nullptr : router_W, router_bias, bias_token_stride, ids_in, gates_in,
                                         ids, gates, counts, off, perm, slot_of_pair, hidden, y, o_part,
                                         static_cast<size_t>(w.ksplit) * P * L.d_model, ctx->resident_layer_ctas, ctx->sms,
                                         reinterpret_cast<unsigned*>(ctx->check_word + 4), route_wait, ctx->dep_extra,
                                         ctx->check_word, st));
    if (ev[1]) {  // one interval for the whole layer
      EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
      ctx->events_one_launch[ctx->events_used / 3 - 1] = 1;
    }
    if (out_ids) EMOE_CUDA(ctx, cudaMemcpyAsync(out_ids, ids_use, sizeof(int32_t) * P, cudaMemcpyDeviceToDevice, st));
    if (out_gates) EMOE_CUDA(ctx, cudaMemcpyAsync(out_gates, gates_use, sizeof(float) * P, cudaMemcpyDeviceToDevice, st));
    if (out_perm) EMOE_CUDA(ctx, cudaMemcpyAsync(out_perm, perm, sizeof(int32_t) * P, cudaMemcpyDeviceToDevice, st));
    return EMOE_OK;
  }
  if (use_hybrid) {
    // experts with up to HYBRID_STREAM_TOKENS tokens: passes of 8-token tiles through the streaming
    // kernel; the others: 128-token tiles on tcgen05.  Each family has its own plan and writes only
    // its own slots of xs / hidden / o_part.
#ifndef EMOE_HYBRID_TOKENS
#define EMOE_HYBRID_TOKENS 32
#endif
#ifndef EMOE_HYBRID_TILES
#define EMOE_HYBRID_TILES 1  // 8-token tiles per pass of the streaming family
#endif
    constexpr int HYBRID_STREAM_TOKENS = EMOE_HYBRID_TOKENS;
    int* plan_heavy = reinterpret_cast<int*>(reinterpret_cast<char*>(plan) + align_up(plan_bytes(L.E)));
    __nv_bfloat16* hid = reinterpret_cast<__nv_bfloat16*>(hidden);
    // many tokens in the call: the streaming family's tail matters little, every further split-K plane costs a
    // cleared and a re-read [P][d] fp32 array
    ksplit = ffn_tma_ksplit(L, T) < 2 ? ffn_tma_ksplit(L, T) : 2;
    EMOE_LAUNCH(ctx, launch_scatter_x(L, table, x, ids_use, perm, off, plan, xs, nullptr, P, 1, 1, HYBRID_STREAM_TOKENS, ctx->check_word, st));
    EMOE_LAUNCH(ctx, launch_scatter_x16(L, table, x, ids_use, perm, off, plan_heavy, xs, P, HYBRID_STREAM_TOKENS + 1, INT_MAX, ctx->check_word, st));
    if (ev[0]) EMOE_CUDA(ctx, cudaEventRecord(ev[0], st));
    // the tcgen05 kernel writes plane 0 only: the other split-K planes of its slots must read as zero
    if (ksplit > 1)
      EMOE_CUDA(ctx, cudaMemsetAsync(o_part + static_cast<size_t>(P) * L.d_model, 0,
                                     static_cast<size_t>(ksplit - 1) * P * L.d_model * sizeof(float), st));
    if (ctx->fuse_projections) {
      EMOE_LAUNCH(ctx, launch_ffn_tma(0, 2, L, table, tmaps, xs, off, plan, hid, o_part, ksplit, P, T, EMOE_HYBRID_TILES, ctx->check_word, st));
    } else {
      EMOE_LAUNCH(ctx, launch_ffn_tma(0, 1, L, table, tmaps, xs, off, plan, hid, o_part, ksplit, P, T, EMOE_HYBRID_TILES, ctx->check_word, st));
      EMOE_LAUNCH(ctx, launch_ffn_tma(1, 2, L, table, tmaps, xs, off, plan, hid, o_part, ksplit, P, T, EMOE_HYBRID_TILES, ctx->check_word, st));
    }
    EMOE_LAUNCH(ctx, launch_ffn_umma(0, L, tmaps, plan_heavy, xs, hidden, o_part, um_scratch, P, 1, ctx->check_word, st));
    EMOE_LAUNCH(ctx, launch_ffn_umma(1, L, tmaps, plan_heavy, hidden, hidden, o_part, um_scratch, P, 1, ctx->check_word, st));
    if (ev[1]) {  // one interval for the whole expert stage
      EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
      ctx->events_one_launch[ctx->events_used / 3 - 1] = 1;
      ev[2] = nullptr;
    }
  } else if (use_umma) {
    {  // the second projection's units may be halves of the inputs, summed by the combine step like any split-K
      int sms = 0;
      EMOE_CUDA(ctx, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device));
      ksplit = ffn_umma_zsplit(L, T, sms);
      if (ksplit > w.ksplit) ksplit = w.ksplit;  // the workspace holds w.ksplit planes
    }
    EMOE_LAUNCH(ctx, launch_scatter_x16(L, table, x, ids_use, perm, off, plan, xs, P, 1, INT_MAX, ctx->check_word, st));
    if (ev[0]) EMOE_CUDA(ctx, cudaEventRecord(ev[0], st));
    EMOE_LAUNCH(ctx, launch_ffn_umma(0, L, tmaps, plan, xs, hidden, o_part, um_scratch, P, 1, ctx->check_word, st));
    if (ev[1]) EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
    EMOE_LAUNCH(ctx, launch_ffn_umma(1, L, tmaps, plan, hidden, hidden, o_part, um_scratch, P, ksplit, ctx->check_word, st));
  } else if (use_i8) {
    ksplit = ffn_i8_ksplit(L, T);
    if (one_launch_route)
      EMOE_LAUNCH(ctx, launch_route_permute_scatter(L, table, x, T, router_W, router_bias, bias_token_stride, ids, gates, counts,
                                                    off, perm, slot_of_pair, plan, xs, xsc, 2, route_sync, route_wait,
                                                    ctx->dep_extra, ctx->check_word, st));
    else if (one_launch_permute)
      EMOE_LAUNCH(ctx, launch_permute_scatter(L, table, x, ids_use, counts, off, perm, slot_of_pair, plan, xs, xsc, P, 2,
                                              ctx->check_word, st));
    else
      EMOE_LAUNCH(ctx, launch_scatter_x(L, table, x, ids_use, perm, off, plan, xs, xsc, P, 2, 1, INT_MAX, ctx->check_word, st));
    if (ev[0]) EMOE_CUDA(ctx, cudaEventRecord(ev[0], st));
    if (ctx->fuse_projections) {
      // one launch: an expert's second projection starts when its hidden vectors are complete
      EMOE_LAUNCH(ctx, launch_ffn_i8(0, 2, L, tmaps, smaps, xs, xsc, plan, hidden, hsc, o_part, ksplit, P, T, 0, ctx->wait_limit,
                                     ctx->dep_extra, ctx->check_word, st));
      if (ev[1]) {  // one interval only: the end event of the triple stays unused
        EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
        ctx->events_one_launch[ctx->events_used / 3 - 1] = 1;
        ev[2] = nullptr;
      }
    } else {
      EMOE_LAUNCH(ctx, launch_ffn_i8(0, 1, L, tmaps, smaps, xs, xsc, plan, hidden, hsc, o_part, ksplit, P, T, 0, ctx->wait_limit, 0,
                                     ctx->check_word, st));
      if (ev[1]) EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
      EMOE_LAUNCH(ctx, launch_ffn_i8(1, 2, L, tmaps, smaps, xs, xsc, plan, hidden, hsc, o_part, ksplit, P, T, 0, ctx->wait_limit, 0,
                                     ctx->check_word, st));
    }
  } else if (use_tma) {
    ksplit = ffn_tma_ksplit(L, T);
    if (one_launch_route)
      EMOE_LAUNCH(ctx, launch_route_permute_scatter(L, table, x, T, router_W, router_bias, bias_token_stride, ids, gates, counts,
                                                    off, perm, slot_of_pair, plan, xs, nullptr, 1, route_sync, route_wait,
                                                    ctx->dep_extra, ctx->check_word, st));
    else if (one_launch_permute)
      EMOE_LAUNCH(ctx, launch_permute_scatter(L, table, x, ids_use, counts, off, perm, slot_of_pair, plan, xs, nullptr, P, 1,
                                              ctx->check_word, st));
    else
      EMOE_LAUNCH(ctx, launch_scatter_x(L, table, x, ids_use, perm, off, plan, xs, nullptr, P, 1, 1, INT_MAX, ctx->check_word, st));
    if (ev[0]) EMOE_CUDA(ctx, cudaEventRecord(ev[0], st));
    __nv_bfloat16* hid = reinterpret_cast<__nv_bfloat16*>(hidden);
    if (ctx->fuse_projections) {
      // one launch: an expert's second projection starts when its hidden vectors are complete
      EMOE_LAUNCH(ctx, launch_ffn_tma(0, 2, L, table, tmaps, xs, off, plan, hid, o_part, ksplit, P, T, 0, ctx->check_word, st));
      if (ev[1]) {  // one interval only: the end event of the triple stays unused
        EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
        ctx->events_one_launch[ctx->events_used / 3 - 1] = 1;
        ev[2] = nullptr;
      }
    } else {
      EMOE_LAUNCH(ctx, launch_ffn_tma(0, 1, L, table, tmaps, xs, off, plan, hid, o_part, ksplit, P, T, 0, ctx->check_word, st));
      if (ev[1]) EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
      EMOE_LAUNCH(ctx, launch_ffn_tma(1, 2, L, table, tmaps, xs, off, plan, hid, o_part, ksplit, P, T, 0, ctx->check_word, st));
    }
  } else if (use_mma) {
    ksplit = ffn_mma_ksplit(L, T);
    EMOE_LAUNCH(ctx, launch_scatter_x(L, table, x, ids_use, perm, off, nullptr, xs, nullptr, P, 0, 1, INT_MAX, ctx->check_word, st));
    if (ev[0]) EMOE_CUDA(ctx, cudaEventRecord(ev[0], st));
    EMOE_LAUNCH(ctx, launch_ffn_mma(0, L, table, xs, off, reinterpret_cast<__nv_bfloat16*>(hidden), o_part, 1, P, T, st));
    if (ev[1]) EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
    EMOE_LAUNCH(ctx, launch_ffn_mma(1, L, table, reinterpret_cast<const __nv_bfloat16*>(hidden), off,
                                  reinterpret_cast<__nv_bfloat16*>(hidden), o_part, ksplit, P, T, st));
  } else {
    if (ev[0]) EMOE_CUDA(ctx, cudaEventRecord(ev[0], st));
    EMOE_LAUNCH(ctx, launch_ffn_gemv(0, L, table, x, perm, off, hidden, o_part, P, st));
    if (ev[1]) EMOE_CUDA(ctx, cudaEventRecord(ev[1], st));
    EMOE_LAUNCH(ctx, launch_ffn_gemv(1, L, table, x, perm, off, hidden, o_part, P, st));
  }
  if (ev[2]) EMOE_CUDA(ctx, cudaEventRecord(ev[2], st));
  EMOE_LAUNCH(ctx, launch_combine(o_part, ksplit, static_cast<size_t>(P), gates_use, slot_of_pair, T, L.top_k, L.d_model,
                                y, st));
  if (out_ids) EMOE_CUDA(ctx, cudaMemcpyAsync(out_ids, ids_use, sizeof(int32_t) * P, cudaMemcpyDeviceToDevice, st));
  if (out_gates) EMOE_CUDA(ctx, cudaMemcpyAsync(out_gates, gates_use, sizeof(float) * P, cudaMemcpyDeviceToDevice, st));
  if (out_perm) EMOE_CUDA(ctx, cudaMemcpyAsync(out_perm, perm, sizeof(int32_t) * P, cudaMemcpyDeviceToDevice, st));
  return EMOE_OK;
}

}  // namespace

namespace emoe {
ExpertCache*& ctx_cache(emoe_ctx* ctx) { return ctx->cache; }
int ctx_device(const emoe_ctx* ctx) { return ctx->device; }
int ctx_cuda_fail(emoe_ctx* ctx, cudaError_t e) { return cuda_fail(ctx, e); }
}  // namespace emoe

extern "C" {

emoe_ctx* emoe_create(int device, size_t workspace_bytes, int* status) {
  int dummy;
  if (!status) status = &dummy;
  *status = EMOE_OK;
  emoe_ctx* ctx = new (std::nothrow) emoe_ctx();
  if (!ctx) {
    *status = EMOE_ERR_INVALID_ARG;
    return nullptr;
  }
  ctx->device = device;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess && workspace_bytes > 0) e = cudaMalloc(&ctx->workspace, workspace_bytes);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->check_word, 8 * sizeof(int));  // + the grid counters of the routing kernel (2) and of the one-launch layer (3)
  if (e == cudaSuccess) e = cudaMemset(ctx->check_word, 0, 8 * sizeof(int));
  if (e == cudaSuccess) e = cudaMallocHost(&ctx->check_host, sizeof(int));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->tables_dev, TABLE_BLOCK_BYTES * MAX_TABLES);
  if (e == cudaSuccess) e = cudaMallocHost(&ctx->tables_pin, TABLE_BLOCK_BYTES * MAX_TABLES);
  if (e != cudaSuccess) {
    *status = EMOE_ERR_CUDA;
    ctx->last_cuda = static_cast<int>(e);
    emoe_destroy(ctx);
    return nullptr;
  }
  ctx->workspace_bytes = workspace_bytes;
  return ctx;
}

int emoe_destroy(emoe_ctx* ctx) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  if (ctx->workspace) cudaFree(ctx->workspace);
  if (ctx->check_word) cudaFree(ctx->check_word);
  if (ctx->check_host) cudaFreeHost(ctx->check_host);
  if (ctx->tables_dev) cudaFree(ctx->tables_dev);
  if (ctx->tables_pin) cudaFreeHost(ctx->tables_pin);
  for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
  for (cudaEvent_t e : ctx->table_events) cudaEventDestroy(e);
  cache_destroy(ctx->cache);
  delete ctx;
  return EMOE_OK;
}

size_t emoe_workspace_bytes(const emoe_layer_desc* desc, int T) {
  LayerDims L;
  if (!make_dims(desc, &L) || T <= 0) return 0;
  // enough for every call of up to T tokens: a call with very few tokens splits the second
  // projection finer and may need more partial-sum rows per token than a larger one
  size_t need = make_layout(L, T).total;
  for (int t = 1; t < T && t <= 256; ++t) {
    const size_t n = make_layout(L, t).total;
    if (n > need) need = n;
  }
  return need;
}

int emoe_last_cuda_error(const emoe_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

int emoe_device_status(emoe_ctx* ctx, void* stream) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  EMOE_CUDA(ctx, cudaSetDevice(ctx->device));
  EMOE_CUDA(ctx, cudaMemcpyAsync(ctx->check_host, ctx->check_word, sizeof(int), cudaMemcpyDeviceToHost, st));
  EMOE_CUDA(ctx, cudaMemsetAsync(ctx->check_word, 0, 8 * sizeof(int), st));  // also the grid counters a timed-out wait left behind
  EMOE_CUDA(ctx, cudaStreamSynchronize(st));
  if (*ctx->check_host & CHECK_WAIT_TIMEOUT) return EMOE_ERR_TIMEOUT;
  if (*ctx->check_host & CHECK_BAD_EXPERT_ID) return EMOE_ERR_DEVICE_CHECK;
  if (*ctx->check_host & CHECK_F16_RANGE) return EMOE_ERR_RANGE;
  return *ctx->check_host ? EMOE_ERR_DEVICE_CHECK : EMOE_OK;
}

const char* emoe_status_string(int status) {
  switch (status) {
    case EMOE_OK: return "ok";
    case EMOE_ERR_INVALID_ARG: return "invalid argument";
    case EMOE_ERR_UNSUPPORTED: return "unsupported bitwidth, enum value or shape";
    case EMOE_ERR_ALIGNMENT: return "pointer or row size not sufficiently aligned";
    case EMOE_ERR_WORKSPACE: return "context workspace (or expert-table cache) too small";
    case EMOE_ERR_CUDA: return "CUDA call failed (see emoe_last_cuda_error)";
    case EMOE_ERR_DEVICE_CHECK: return "a kernel found inconsistent data";
    case EMOE_ERR_CACHE_FULL: return "every slot of the expert cache is in use";
    case EMOE_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case EMOE_ERR_RANGE: return "a value left the fp16 range of the selected kernel's operands";
    default: return "unknown status";
  }
}

size_t emoe_packed_bytes(int N, int K, int bits) {
  if (N <= 0 || K <= 0 || (bits != 2 && bits != 4 && bits != 8)) return 0;
  if ((static_cast<long long>(K) * bits) % 8 != 0) return 0;
  return static_cast<size_t>(N) * (static_cast<size_t>(K) * bits / 8);
}

size_t emoe_scales_bytes(int N, int K, int group, int scale_dtype) {
  if (N <= 0 || K <= 0 || group < 0) return 0;
  if (scale_dtype != EMOE_DTYPE_F32 && scale_dtype != EMOE_DTYPE_F16) return 0;
  const int G = group > 0 ? group : K;
  if (K % G != 0) return 0;
  return static_cast<size_t>(N) * (K / G) * (scale_dtype == EMOE_DTYPE_F16 ? 2 : 4);
}

int emoe_pack_expert(emoe_ctx* ctx, const float* W, int N, int K, int bits, int group, int scale_dtype,
                     void* out_packed, void* out_scales, void* stream) {
  return emoe_pack_expert_mode(ctx, W, N, K, bits, group, scale_dtype, EMOE_RANGE_SYMMETRIC, out_packed, out_scales, stream);
}

int emoe_pack_expert_mode(emoe_ctx* ctx, const float* W, int N, int K, int bits, int group, int scale_dtype,
                          int range_mode, void* out_packed, void* out_scales, void* stream) {
  if (range_mode != EMOE_RANGE_SYMMETRIC && range_mode != EMOE_RANGE_FULL) return EMOE_ERR_UNSUPPORTED;
  if (!ctx || !W || !out_packed || !out_scales || N <= 0 || K <= 0 || group < 0) return EMOE_ERR_INVALID_ARG;
  if (bits != 2 && bits != 4 && bits != 8) return EMOE_ERR_UNSUPPORTED;
  if (scale_dtype != EMOE_DTYPE_F32 && scale_dtype != EMOE_DTYPE_F16) return EMOE_ERR_UNSUPPORTED;
  const int G = group > 0 ? group : K;
  if (K % G != 0) return EMOE_ERR_INVALID_ARG;
  if (G % 4 != 0) return EMOE_ERR_UNSUPPORTED;
  if (!aligned(W, 16) || !aligned(out_packed, 16) || !aligned(out_scales, 4)) return EMOE_ERR_ALIGNMENT;
  EMOE_CUDA(ctx, cudaSetDevice(ctx->device));
  EMOE_CUDA(ctx, launch_pack(W, N, K, bits, group, scale_dtype == EMOE_DTYPE_F16, range_mode == EMOE_RANGE_FULL, static_cast<uint8_t*>(out_packed),
                             out_scales, static_cast<cudaStream_t>(stream)));
  return EMOE_OK;
}

int emoe_requantize_expert(emoe_ctx* ctx, const void* in_packed, const void* in_scales, int N, int K, int bits_in,
                           int bits_out, int group, int scale_dtype, void* out_packed, void* out_scales,
                           void* stream) {
  return emoe_requantize_expert_mode(ctx, in_packed, in_scales, N, K, bits_in, bits_out, group, scale_dtype,
                                     EMOE_RANGE_SYMMETRIC, out_packed, out_scales, stream);
}

int emoe_requantize_expert_mode(emoe_ctx* ctx, const void* in_packed, const void* in_scales, int N, int K, int bits_in,
                                int bits_out, int group, int scale_dtype, int range_mode, void* out_packed,
                                void* out_scales, void* stream) {
  if (range_mode != EMOE_RANGE_SYMMETRIC && range_mode != EMOE_RANGE_FULL) return EMOE_ERR_UNSUPPORTED;
  if (!ctx || !in_packed || !in_scales || !out_packed || !out_scales || N <= 0 || K <= 0 || group < 0)
    return EMOE_ERR_INVALID_ARG;
  if (bits_in != 2 && bits_in != 4 && bits_in != 8) return EMOE_ERR_UNSUPPORTED;
  if (bits_out != 2 && bits_out != 4 && bits_out != 8) return EMOE_ERR_UNSUPPORTED;
  if (scale_dtype != EMOE_DTYPE_F32 && scale_dtype != EMOE_DTYPE_F16) return EMOE_ERR_UNSUPPORTED;
  const int G = group > 0 ? group : K;
  if (K % G != 0) return EMOE_ERR_INVALID_ARG;
  if (G % 4 != 0) return EMOE_ERR_UNSUPPORTED;
  if (in_packed == out_packed || in_scales == out_scales) return EMOE_ERR_INVALID_ARG;  // not in place
  if (!aligned(in_packed, 16) || !aligned(out_packed, 16) || !aligned(in_scales, 4) || !aligned(out_scales, 4))
    return EMOE_ERR_ALIGNMENT;
  EMOE_CUDA(ctx, cudaSetDevice(ctx->device));
  EMOE_CUDA(ctx, launch_requant(static_cast<const uint8_t*>(in_packed), in_scales, N, K, bits_in, bits_out, group,
                                scale_dtype == EMOE_DTYPE_F16, range_mode == EMOE_RANGE_FULL, static_cast<uint8_t*>(out_packed), out_scales,
                                static_cast<cudaStream_t>(stream)));
  return EMOE_OK;
}

int emoe_router_topk(emoe_ctx* ctx, const void* x, int act_dtype, int T, int d, const float* router_W,
                     const float* router_bias, int bias_token_stride, int E, int top_k, int gate_mode,
                     int32_t* out_ids, float* out_gates, float* out_logits, void* stream) {
  if (!ctx || !x || !router_W || !out_ids || !out_gates || T <= 0 || d <= 0) return EMOE_ERR_INVALID_ARG;
  if (E < 1 || E > EMOE_MAX_EXPERTS || top_k < 1 || top_k > E || top_k > EMOE_MAX_TOP_K) return EMOE_ERR_INVALID_ARG;
  if (act_dtype != EMOE_DTYPE_F32 && act_dtype != EMOE_DTYPE_BF16) return EMOE_ERR_UNSUPPORTED;
  if (gate_mode != EMOE_GATE_SOFTMAX && gate_mode != EMOE_GATE_SOFTMAX_RENORM) return EMOE_ERR_UNSUPPORTED;
  if (router_bias && bias_token_stride != 0 && bias_token_stride != E) return EMOE_ERR_INVALID_ARG;
  EMOE_CUDA(ctx, cudaSetDevice(ctx->device));
  EMOE_CUDA(ctx, launch_router_topk(x, act_dtype == EMOE_DTYPE_BF16, T, d, router_W, router_bias, bias_token_stride, E,
                                    top_k, gate_mode == EMOE_GATE_SOFTMAX_RENORM, out_ids, out_gates, out_logits,
                                    static_cast<cudaStream_t>(stream)));
  return EMOE_OK;
}

int emoe_permute(emoe_ctx* ctx, const int32_t* ids, int n_pairs, int E, int32_t* out_counts, int32_t* out_off,
                 int32_t* out_perm, int32_t* out_slot_of_pair, void* stream) {
  if (!ctx || !ids || !out_counts || !out_off || !out_perm || n_pairs <= 0) return EMOE_ERR_INVALID_ARG;
  if (E < 1 || E > EMOE_MAX_EXPERTS) return EMOE_ERR_INVALID_ARG;
  EMOE_CUDA(ctx, cudaSetDevice(ctx->device));
  EMOE_CUDA(ctx, launch_permute(ids, n_pairs, E, out_counts, out_off, out_perm, out_slot_of_pair, ctx->check_word,
                                static_cast<cudaStream_t>(stream)));
  return EMOE_OK;
}

int emoe_moe_forward(emoe_ctx* ctx, const emoe_layer_desc* desc, const void* x, int T, const float* router_W,
                     const float* router_bias, int bias_token_stride, const emoe_expert* host_experts, float* y,
                     int32_t* out_ids, float* out_gates, int32_t* out_perm, void* stream) {
  if (!router_W) return EMOE_ERR_INVALID_ARG;
  return forward_impl(ctx, desc, x, T, router_W, router_bias, bias_token_stride, nullptr, nullptr, host_experts, y,
                      out_ids, out_gates, out_perm, static_cast<cudaStream_t>(stream));
}

int emoe_moe_forward_routed(emoe_ctx* ctx, const emoe_layer_desc* desc, const void* x, int T, const int32_t* ids,
                            const float* gates, const emoe_expert* host_experts, float* y, int32_t* out_perm,
                            void* stream) {
  if (!ids || !gates) return EMOE_ERR_INVALID_ARG;
  return forward_impl(ctx, desc, x, T, nullptr, nullptr, 0, ids, gates, host_experts, y, nullptr, nullptr, out_perm,
                      static_cast<cudaStream_t>(stream));
}

int emoe_set_timing(emoe_ctx* ctx, int enabled) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  ctx->timing = enabled != 0;
  ctx->events_used = 0;
  return EMOE_OK;
}

int emoe_read_timing(emoe_ctx* ctx, float* out_first_ms, float* out_second_ms, int* out_calls) {
  if (!ctx || !out_first_ms || !out_second_ms || !out_calls) return EMOE_ERR_INVALID_ARG;
  float a = 0.f, b = 0.f;
  const size_t n = ctx->events_used / 3;
  for (size_t i = 0; i < n; ++i) {
    float ms = 0.f;
    const bool one = ctx->events_one_launch[i] != 0;
    EMOE_CUDA(ctx, cudaEventSynchronize(ctx->events[3 * i + (one ? 1 : 2)]));
    EMOE_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->events[3 * i], ctx->events[3 * i + 1]));
    a += ms;
    if (!one) {
      EMOE_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->events[3 * i + 1], ctx->events[3 * i + 2]));
      b += ms;
    }
  }
  *out_first_ms = a;
  *out_second_ms = b;
  *out_calls = static_cast<int>(n);
  ctx->events_used = 0;
  return EMOE_OK;
}

int emoe_set_dependent_launch(emoe_ctx* ctx, int enabled) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  ctx->pdl = enabled != 0;
  return EMOE_OK;
}

int emoe_last_expert_counts(emoe_ctx* ctx, int32_t* out_counts, int n_experts, void* stream) {
  if (!ctx || !out_counts || !ctx->last_counts || n_experts != ctx->last_counts_n) return EMOE_ERR_INVALID_ARG;
  EMOE_CUDA(ctx, cudaSetDevice(ctx->device));
  EMOE_CUDA(ctx, cudaMemcpyAsync(out_counts, ctx->last_counts, sizeof(int32_t) * n_experts, cudaMemcpyDeviceToHost,
                                 static_cast<cudaStream_t>(stream)));
  EMOE_CUDA(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  return EMOE_OK;
}

int emoe_kernels_last_forward(const emoe_ctx* ctx) { return ctx ? ctx->kernels_last : 0; }

int emoe_set_fused_projections(emoe_ctx* ctx, int enabled) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  ctx->fuse_projections = enabled != 0;
  return EMOE_OK;
}

int emoe_set_fused_routing(emoe_ctx* ctx, int enabled) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  ctx->fuse_routing = enabled != 0;
  return EMOE_OK;
}

int emoe_set_fused_layer(emoe_ctx* ctx, int enabled) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  if (enabled < 0 || enabled > 2) return EMOE_ERR_INVALID_ARG;
  ctx->fuse_layer = enabled;
  return EMOE_OK;
}

int emoe_set_wait_limit(emoe_ctx* ctx, unsigned polls) {
  if (!ctx) return EMOE_ERR_INVALID_ARG;
  ctx->wait_limit = polls;
  return EMOE_OK;
}

int emoe_debug_expect_extra_completions(emoe_ctx* ctx, int extra) {
  if (!ctx || extra < 0) return EMOE_ERR_INVALID_ARG;
  ctx->dep_extra = extra;
  return EMOE_OK;
}

#ifdef EMOE_I8_PROFILE
int emoe_debug_set_profile_buffer(void* dev_buffer) {
  g_i8_profile = static_cast<long long*>(dev_buffer);
  return EMOE_OK;
}
#endif

int emoe_set_ffn_path(emoe_ctx* ctx, int path) {
  if (!ctx || path < 0 || path > 6) return EMOE_ERR_INVALID_ARG;
  ctx->ffn_path = path;
  return EMOE_OK;
}

}  // extern "C"
