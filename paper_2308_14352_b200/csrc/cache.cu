// Expert cache in HBM with predict-then-prefetch staging from pinned host memory: the B200
// analogue of the paper's storage hierarchy (Section 3.3: experts live in slow storage, a buffer
// of fixed size in fast memory holds some of them, experts predicted from the previous layers'
// activations are preloaded while the current layer computes, and an eviction policy built on
// activation frequency and layer distance decides who leaves).  Here slow storage is pinned host
// memory, fast memory is a fixed set of equally sized HBM slots, loading is cudaMemcpyAsync on a
// copy stream, and ordering between the copy stream and the compute stream is carried by two CUDA
// events per slot (contents ready / last reader done), so no call ever blocks the host.
//
// The bookkeeping (which expert sits in which slot, who is evicted, the counters) is plain host
// code in CachePolicy and has no CUDA in it: the same object backs the device cache and the
// host-only test hooks (emoe_policy_*), so its decisions can be checked without a GPU.
#include <algorithm>
#include <cstring>
#include <new>
#include <unordered_map>
#include <vector>

#include "common.cuh"

namespace emoe {

struct CacheExpert {
  int64_t id;
  int layer, bits;
  const void* host[6];  // packed[0..2], scales[0..2] in pinned host memory (null = matrix not present)
  size_t bytes[6];
  size_t offset[6];  // placement inside a slot
  int slot;
  int64_t freq;        // activations so far (acquire calls)
  bool by_prefetch;    // brought in by a prefetch and not used since
};

struct CacheSlot {
  int expert;  // index into experts, -1 = free
  int pins;    // acquired and not yet released
  int64_t last_touch;
  int64_t loaded_at;  // clock value when the present content was placed
};

class CachePolicy {
 public:
  CachePolicy(int n_slots, int n_layers, int policy) : n_layers_(n_layers), policy_(policy), clock_(0) {
    slots_.assign(static_cast<size_t>(n_slots), CacheSlot{-1, 0, 0, 0});
    std::memset(&stats_, 0, sizeof(stats_));
  }
  int add(const CacheExpert& e) {
    if (index_.count(e.id)) return -1;
    index_[e.id] = static_cast<int>(experts_.size());
    experts_.push_back(e);
    return static_cast<int>(experts_.size()) - 1;
  }
  int find(int64_t id) const {
    auto it = index_.find(id);
    return it == index_.end() ? -1 : it->second;
  }
  CacheExpert& expert(int i) { return experts_[static_cast<size_t>(i)]; }
  const CacheSlot& slot(int s) const { return slots_[static_cast<size_t>(s)]; }
  int n_slots() const { return static_cast<int>(slots_.size()); }
  emoe_cache_stats& stats() { return stats_; }

  // Eviction order (Section 3.3, "Cache eviction policy"): the expert with the highest score
  // L = -f / D leaves first, f its activation frequency, D the distance of its layer from the
  // current one.  The paper takes f from an offline profile; here it is the running activation
  // count plus one, so that an expert that was preloaded but not used yet (count 0) is still
  // ranked by its layer distance instead of being the first to go.  EMOE_EVICT_FORWARD takes D as
  // the number of layers until the expert's layer runs again, (i - I) mod S, which is what the
  // text asks for (layers about to run are kept);
  // EMOE_EVICT_PRINTED takes the printed (S - i + I) mod S.  D = 0 (the current layer) is
  // protected: such an expert goes only when nothing else can.  For comparison (the paper's
  // evaluation sets its rule against the textbook ones): EMOE_EVICT_LRU, least recently touched
  // first; EMOE_EVICT_FIFO, loaded earliest first; EMOE_EVICT_LFU, fewest activations first (ties:
  // loaded earliest).  Remaining ties: lowest slot.
  bool better_victim(int sa, int sb, int current_layer) const {  // is slot sa a better victim than sb?
    const CacheExpert& a = experts_[static_cast<size_t>(slots_[static_cast<size_t>(sa)].expert)];
    const CacheExpert& b = experts_[static_cast<size_t>(slots_[static_cast<size_t>(sb)].expert)];
    if (policy_ == EMOE_EVICT_LRU) {
      const int64_t ta = slots_[static_cast<size_t>(sa)].last_touch, tb = slots_[static_cast<size_t>(sb)].last_touch;
      return ta != tb ? ta < tb : sa < sb;
    }
    if (policy_ == EMOE_EVICT_FIFO || policy_ == EMOE_EVICT_LFU) {
      if (policy_ == EMOE_EVICT_LFU && a.freq != b.freq) return a.freq < b.freq;
      const int64_t la = slots_[static_cast<size_t>(sa)].loaded_at, lb = slots_[static_cast<size_t>(sb)].loaded_at;
      return la != lb ? la < lb : sa < sb;
    }
    const int da = distance(a.layer, current_layer), db = distance(b.layer, current_layer);
    if ((da == 0) != (db == 0)) return db == 0;  // the unprotected one
    if (da == 0) return a.freq != b.freq ? a.freq < b.freq : sa < sb;
    // -fa/da > -fb/db  <=>  fa * db < fb * da   (exact in integers), f = count + 1
    const int64_t lhs = (a.freq + 1) * db, rhs = (b.freq + 1) * da;
    return lhs != rhs ? lhs < rhs : sa < sb;
  }
  int distance(int layer, int current_layer) const {
    const int S = n_layers_ > 0 ? n_layers_ : 1;
    const int d = policy_ == EMOE_EVICT_PRINTED ? (S - layer + current_layer) % S : (layer - current_layer) % S;
    return d < 0 ? d + S : d;
  }
  // A slot for expert `ei`: a free one, else the best victim among unpinned slots.  Returns -1
  // when every slot is pinned.  *evicted = expert index that left, or -1.
  int place(int ei, int current_layer, int* evicted) {
    *evicted = -1;
    int best = -1;
    for (int s = 0; s < n_slots(); ++s)
      if (slots_[static_cast<size_t>(s)].expert < 0) {
        best = s;
        break;
      }
    if (best < 0) {
      for (int s = 0; s < n_slots(); ++s) {
        if (slots_[static_cast<size_t>(s)].pins > 0) continue;
        if (best < 0 || better_victim(s, best, current_layer)) best = s;
      }
      if (best < 0) return -1;
      *evicted = slots_[static_cast<size_t>(best)].expert;
      experts_[static_cast<size_t>(*evicted)].slot = -1;
      ++stats_.evictions;
    }
    slots_[static_cast<size_t>(best)].expert = ei;
    slots_[static_cast<size_t>(best)].last_touch = ++clock_;
    slots_[static_cast<size_t>(best)].loaded_at = clock_;
    experts_[static_cast<size_t>(ei)].slot = best;
    for (int m = 0; m < 6; ++m) stats_.bytes_copied += static_cast<int64_t>(experts_[static_cast<size_t>(ei)].bytes[m]);
    return best;
  }
  // prefetch request for one expert: slot to load into, or -1 (already resident / no slot)
  int prefetch(int ei, int current_layer, int* evicted) {
    *evicted = -1;
    CacheExpert& e = experts_[static_cast<size_t>(ei)];
    if (e.slot >= 0) {
      ++stats_.prefetch_redundant;
      return -1;
    }
    const int s = place(ei, current_layer, evicted);
    if (s < 0) {
      ++stats_.prefetch_refused;
      return -1;
    }
    e.by_prefetch = true;
    ++stats_.prefetched;
    return s;
  }
  // the expert is about to be used: *load = 1 if it has to be loaded now into the returned slot
  int acquire(int ei, int current_layer, int* load, int* evicted) {
    *load = 0;
    *evicted = -1;
    CacheExpert& e = experts_[static_cast<size_t>(ei)];
    int s = e.slot;
    if (s >= 0) {
      ++stats_.hits;
      if (e.by_prefetch) ++stats_.prefetch_hits;
    } else {
      s = place(ei, current_layer, evicted);
      if (s < 0) return -1;
      ++stats_.misses;
      *load = 1;
    }
    e.by_prefetch = false;
    ++e.freq;
    ++slots_[static_cast<size_t>(s)].pins;
    slots_[static_cast<size_t>(s)].last_touch = ++clock_;
    return s;
  }
  int release(int ei) {
    const int s = experts_[static_cast<size_t>(ei)].slot;
    if (s < 0 || slots_[static_cast<size_t>(s)].pins <= 0) return -1;
    --slots_[static_cast<size_t>(s)].pins;
    return s;
  }

 private:
  int n_layers_, policy_;
  int64_t clock_;
  std::vector<CacheExpert> experts_;
  std::unordered_map<int64_t, int> index_;
  std::vector<CacheSlot> slots_;
  emoe_cache_stats stats_;
};

// the device side of the cache: slots and their events
struct ExpertCache {
  CachePolicy policy;
  int device;
  size_t slot_bytes;
  char* base;  // n_slots * slot_bytes of HBM
  std::vector<cudaEvent_t> ready;  // contents of the slot are complete (recorded on the copy stream)
  std::vector<cudaEvent_t> idle;   // last reader of the slot is done (recorded on the compute stream)
  std::vector<char> idle_valid;
  // exposed-copy accounting: event pairs around the waits of acquire calls, summed on request
  bool timing = false;
  std::vector<cudaEvent_t> timed;  // pairs (before, after), timing enabled
  size_t timed_used = 0;
  double exposed_ns = 0.0;
  long long timed_acquires = 0;
  ExpertCache(int n_slots, int n_layers, int pol) : policy(n_slots, n_layers, pol), device(0), slot_bytes(0), base(nullptr) {}
};

void cache_destroy(ExpertCache* c) {
  if (!c) return;
  for (cudaEvent_t e : c->ready) cudaEventDestroy(e);
  for (cudaEvent_t e : c->idle) cudaEventDestroy(e);
  for (cudaEvent_t e : c->timed) cudaEventDestroy(e);
  if (c->base) cudaFree(c->base);
  delete c;
}

namespace {

constexpr size_t SLOT_ALIGN = 256;

int fill_expert(CacheExpert* e, int64_t id, int layer, int bits, const void* const* host_packed, const void* const* host_scales,
                const size_t* bytes) {
  if (bits != 2 && bits != 4 && bits != 8) return EMOE_ERR_UNSUPPORTED;
  if (layer < 0 || !host_packed || !host_scales || !bytes) return EMOE_ERR_INVALID_ARG;
  e->id = id;
  e->layer = layer;
  e->bits = bits;
  e->slot = -1;
  e->freq = 0;
  e->by_prefetch = false;
  size_t off = 0;
  for (int m = 0; m < 6; ++m) {
    e->host[m] = m < 3 ? host_packed[m] : host_scales[m - 3];
    e->bytes[m] = bytes[m];
    if ((e->host[m] == nullptr) != (bytes[m] == 0)) return EMOE_ERR_INVALID_ARG;
    e->offset[m] = off;
    off += (bytes[m] + SLOT_ALIGN - 1) / SLOT_ALIGN * SLOT_ALIGN;
  }
  return EMOE_OK;
}

// enqueue the copies of an expert into its slot on the copy stream, behind the slot's last reader
cudaError_t load_into_slot(ExpertCache* c, const CacheExpert& e, int s, cudaStream_t copy) {
  cudaError_t err = cudaSuccess;
  if (c->idle_valid[static_cast<size_t>(s)]) err = cudaStreamWaitEvent(copy, c->idle[static_cast<size_t>(s)], 0);
  char* dst = c->base + static_cast<size_t>(s) * c->slot_bytes;
  for (int m = 0; m < 6 && err == cudaSuccess; ++m)
    if (e.bytes[m]) err = cudaMemcpyAsync(dst + e.offset[m], e.host[m], e.bytes[m], cudaMemcpyHostToDevice, copy);
  if (err == cudaSuccess) err = cudaEventRecord(c->ready[static_cast<size_t>(s)], copy);
  return err;
}

void expert_pointers(const ExpertCache* c, const CacheExpert& e, emoe_expert* out) {
  const char* dst = c->base + static_cast<size_t>(e.slot) * c->slot_bytes;
  out->bits = e.bits;
  out->reserved = 0;
  for (int m = 0; m < 3; ++m) {
    out->packed[m] = e.bytes[m] ? dst + e.offset[m] : nullptr;
    out->scales[m] = e.bytes[m + 3] ? dst + e.offset[m + 3] : nullptr;
  }
}

}  // namespace

// ---- accessors into the context (api.cu) ----------------------------------------------------
ExpertCache*& ctx_cache(emoe_ctx* ctx);
int ctx_device(const emoe_ctx* ctx);
int ctx_cuda_fail(emoe_ctx* ctx, cudaError_t e);

}  // namespace emoe

using namespace emoe;

extern "C" {

int emoe_cache_create(emoe_ctx* ctx, int n_slots, size_t slot_bytes, int n_layers, int policy) {
  if (!ctx || n_slots <= 0 || slot_bytes == 0 || n_layers <= 0) return EMOE_ERR_INVALID_ARG;
  if (policy < EMOE_EVICT_FORWARD || policy > EMOE_EVICT_FIFO) return EMOE_ERR_UNSUPPORTED;
  if (ctx_cache(ctx)) return EMOE_ERR_INVALID_ARG;  // one cache per context
  ExpertCache* c = new (std::nothrow) ExpertCache(n_slots, n_layers, policy);
  if (!c) return EMOE_ERR_INVALID_ARG;
  c->device = ctx_device(ctx);
  c->slot_bytes = (slot_bytes + SLOT_ALIGN - 1) / SLOT_ALIGN * SLOT_ALIGN;
  cudaError_t e = cudaSetDevice(c->device);
  if (e == cudaSuccess) e = cudaMalloc(&c->base, static_cast<size_t>(n_slots) * c->slot_bytes);
  for (int s = 0; s < n_slots && e == cudaSuccess; ++s) {
    cudaEvent_t ev;
    e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e == cudaSuccess) c->ready.push_back(ev);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e == cudaSuccess) c->idle.push_back(ev);
  }
  c->idle_valid.assign(static_cast<size_t>(n_slots), 0);
  if (e != cudaSuccess) {
    cache_destroy(c);
    return ctx_cuda_fail(ctx, e);
  }
  ctx_cache(ctx) = c;
  return EMOE_OK;
}

int emoe_register_expert(emoe_ctx* ctx, int64_t id, int layer, int bits, const void* const* host_pinned_packed,
                         const void* const* host_pinned_scales, const size_t* bytes) {
  if (!ctx || !ctx_cache(ctx)) return EMOE_ERR_INVALID_ARG;
  ExpertCache* c = ctx_cache(ctx);
  CacheExpert e;
  const int rc = fill_expert(&e, id, layer, bits, host_pinned_packed, host_pinned_scales, bytes);
  if (rc != EMOE_OK) return rc;
  if (e.offset[5] + e.bytes[5] > c->slot_bytes) return EMOE_ERR_INVALID_ARG;  // does not fit a slot
  for (int m = 0; m < 3; ++m)
    if (e.bytes[m] && (reinterpret_cast<uintptr_t>(e.host[m]) & 15)) return EMOE_ERR_ALIGNMENT;
  return c->policy.add(e) < 0 ? EMOE_ERR_INVALID_ARG : EMOE_OK;
}

int emoe_prefetch_experts(emoe_ctx* ctx, const int64_t* ids, int n, int current_layer, void* copy_stream) {
  if (!ctx || !ctx_cache(ctx) || (n > 0 && !ids) || n < 0) return EMOE_ERR_INVALID_ARG;
  ExpertCache* c = ctx_cache(ctx);
  cudaError_t err = cudaSetDevice(c->device);
  if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
  for (int i = 0; i < n; ++i) {
    const int ei = c->policy.find(ids[i]);
    if (ei < 0) return EMOE_ERR_INVALID_ARG;
    int evicted;
    const int s = c->policy.prefetch(ei, current_layer, &evicted);
    if (s < 0) continue;  // resident already, or every slot is in use: a prefetch never waits
    err = load_into_slot(c, c->policy.expert(ei), s, static_cast<cudaStream_t>(copy_stream));
    if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
  }
  return EMOE_OK;
}

int emoe_cache_acquire(emoe_ctx* ctx, const int64_t* ids, int n, int current_layer, void* compute_stream, void* copy_stream,
                       emoe_expert* out_experts) {
  if (!ctx || !ctx_cache(ctx) || n <= 0 || !ids || !out_experts) return EMOE_ERR_INVALID_ARG;
  ExpertCache* c = ctx_cache(ctx);
  cudaError_t err = cudaSetDevice(c->device);
  if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
  for (int i = 0; i < n; ++i)  // nothing is touched unless every id is known
    if (c->policy.find(ids[i]) < 0) return EMOE_ERR_INVALID_ARG;
  int rc = EMOE_OK, done = 0;
  cudaEvent_t t_after = nullptr;
  if (c->timing) {
    while (c->timed.size() < c->timed_used + 2) {
      cudaEvent_t ev;
      err = cudaEventCreate(&ev);
      if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
      c->timed.push_back(ev);
    }
    err = cudaEventRecord(c->timed[c->timed_used], static_cast<cudaStream_t>(compute_stream));
    if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
    t_after = c->timed[c->timed_used + 1];
    c->timed_used += 2;
  }
  for (; done < n && rc == EMOE_OK; ++done) {
    const int ei = c->policy.find(ids[done]);
    int load, evicted;
    const int s = c->policy.acquire(ei, current_layer, &load, &evicted);
    if (s < 0) {
      rc = EMOE_ERR_CACHE_FULL;
      break;
    }
    if (load) {
      err = load_into_slot(c, c->policy.expert(ei), s, static_cast<cudaStream_t>(copy_stream));
      if (err != cudaSuccess) rc = ctx_cuda_fail(ctx, err);
    }
    // the compute stream goes on when the slot's contents are complete (no host wait)
    if (rc == EMOE_OK) {
      err = cudaStreamWaitEvent(static_cast<cudaStream_t>(compute_stream), c->ready[static_cast<size_t>(s)], 0);
      if (err != cudaSuccess) rc = ctx_cuda_fail(ctx, err);
    }
    if (rc == EMOE_OK) expert_pointers(c, c->policy.expert(ei), &out_experts[done]);
  }
  if (t_after) {  // recorded even after a failure, so that every pair of the record is complete
    err = cudaEventRecord(t_after, static_cast<cudaStream_t>(compute_stream));
    if (err != cudaSuccess && rc == EMOE_OK) rc = ctx_cuda_fail(ctx, err);
  }
  if (rc != EMOE_OK) {
    // all or nothing: the experts acquired so far by this call are let go again, so that a failed
    // call leaves no slot protected (their activation counts keep the increment)
    for (int i = 0; i < done; ++i) c->policy.release(c->policy.find(ids[i]));
  }
  return rc;
}

int emoe_cache_release(emoe_ctx* ctx, const int64_t* ids, int n, void* compute_stream) {
  if (!ctx || !ctx_cache(ctx) || n <= 0 || !ids) return EMOE_ERR_INVALID_ARG;
  ExpertCache* c = ctx_cache(ctx);
  cudaError_t err = cudaSetDevice(c->device);
  if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
  for (int i = 0; i < n; ++i)
    if (c->policy.find(ids[i]) < 0) return EMOE_ERR_INVALID_ARG;
  int rc = EMOE_OK;
  for (int i = 0; i < n; ++i) {  // an id that is not held does not keep the others from being released
    const int s = c->policy.release(c->policy.find(ids[i]));
    if (s < 0) {
      rc = EMOE_ERR_INVALID_ARG;
      continue;
    }
    err = cudaEventRecord(c->idle[static_cast<size_t>(s)], static_cast<cudaStream_t>(compute_stream));
    if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
    c->idle_valid[static_cast<size_t>(s)] = 1;
  }
  return rc;
}

int emoe_cache_slot_of(emoe_ctx* ctx, int64_t id) {
  if (!ctx || !ctx_cache(ctx)) return -1;
  ExpertCache* c = ctx_cache(ctx);
  const int ei = c->policy.find(id);
  return ei < 0 ? -1 : c->policy.expert(ei).slot;
}

int emoe_cache_get_stats(emoe_ctx* ctx, emoe_cache_stats* out) {
  if (!ctx || !ctx_cache(ctx) || !out) return EMOE_ERR_INVALID_ARG;
  ExpertCache* c = ctx_cache(ctx);
  for (size_t i = 0; i + 1 < c->timed_used; i += 2) {
    cudaError_t err = cudaEventSynchronize(c->timed[i + 1]);
    float ms = 0.0f;
    if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, c->timed[i], c->timed[i + 1]);
    if (err != cudaSuccess) return ctx_cuda_fail(ctx, err);
    c->exposed_ns += static_cast<double>(ms) * 1e6;
    ++c->timed_acquires;
  }
  c->timed_used = 0;
  *out = c->policy.stats();
  out->exposed_copy_ns = static_cast<int64_t>(c->exposed_ns + 0.5);
  out->timed_acquires = c->timed_acquires;
  return EMOE_OK;
}

int emoe_cache_set_timing(emoe_ctx* ctx, int enabled) {
  if (!ctx || !ctx_cache(ctx)) return EMOE_ERR_INVALID_ARG;
  ctx_cache(ctx)->timing = enabled != 0;
  return EMOE_OK;
}

// ---- the same bookkeeping without a device (for checks that run on the host alone) ------------
struct emoe_policy {
  CachePolicy p;
  emoe_policy(int n_slots, int n_layers, int policy) : p(n_slots, n_layers, policy) {}
};

emoe_policy* emoe_policy_create(int n_slots, int n_layers, int policy) {
  if (n_slots <= 0 || n_layers <= 0) return nullptr;
  if (policy < EMOE_EVICT_FORWARD || policy > EMOE_EVICT_FIFO) return nullptr;
  return new (std::nothrow) emoe_policy(n_slots, n_layers, policy);
}
void emoe_policy_destroy(emoe_policy* p) { delete p; }
int emoe_policy_register(emoe_policy* p, int64_t id, int layer, int64_t bytes) {
  if (!p || layer < 0 || bytes < 0) return EMOE_ERR_INVALID_ARG;
  CacheExpert e;
  std::memset(&e, 0, sizeof(e));
  e.id = id;
  e.layer = layer;
  e.bits = 8;
  e.slot = -1;
  e.bytes[0] = static_cast<size_t>(bytes);
  return p->p.add(e) < 0 ? EMOE_ERR_INVALID_ARG : EMOE_OK;
}
// returns the slot the expert is loaded into, -1 if nothing is loaded; *evicted_id = id that left or -1
int emoe_policy_prefetch(emoe_policy* p, int64_t id, int current_layer, int64_t* evicted_id) {
  if (!p || !evicted_id) return -2;
  const int ei = p->p.find(id);
  if (ei < 0) return -2;
  int ev;
  const int s = p->p.prefetch(ei, current_layer, &ev);
  *evicted_id = ev >= 0 ? p->p.expert(ev).id : -1;
  return s;
}
// returns the slot; *loaded = 1 on a miss; -1 = every slot pinned
int emoe_policy_acquire(emoe_policy* p, int64_t id, int current_layer, int* loaded, int64_t* evicted_id) {
  if (!p || !loaded || !evicted_id) return -2;
  const int ei = p->p.find(id);
  if (ei < 0) return -2;
  int ev;
  const int s = p->p.acquire(ei, current_layer, loaded, &ev);
  *evicted_id = ev >= 0 ? p->p.expert(ev).id : -1;
  return s;
}
int emoe_policy_release(emoe_policy* p, int64_t id) {
  if (!p) return -2;
  const int ei = p->p.find(id);
  return ei < 0 ? -2 : p->p.release(ei);
}
int emoe_policy_get_stats(emoe_policy* p, emoe_cache_stats* out) {
  if (!p || !out) return EMOE_ERR_INVALID_ARG;
  *out = p->p.stats();
  return EMOE_OK;
}

// Ranks the experts of the next layer by a first-order prior (Section 3.3, "Estimating expert
// activation a priori", reduced to one previous layer): score[e] = mean over the previous layer's
// picks p of prior[p][e]; out_order lists the experts by descending score, ties by lower index.
int emoe_rank_experts(const float* prior, int n_experts, const int32_t* prev_ids, int n_prev, int32_t* out_order) {
  if (!prior || !prev_ids || !out_order || n_experts <= 0 || n_prev <= 0) return EMOE_ERR_INVALID_ARG;
  std::vector<double> score(static_cast<size_t>(n_experts), 0.0);
  for (int j = 0; j < n_prev; ++j) {
    if (prev_ids[j] < 0 || prev_ids[j] >= n_experts) return EMOE_ERR_INVALID_ARG;
    for (int e = 0; e < n_experts; ++e) score[static_cast<size_t>(e)] += static_cast<double>(prior[static_cast<size_t>(prev_ids[j]) * n_experts + e]);
  }
  for (int e = 0; e < n_experts; ++e) out_order[e] = e;
  std::stable_sort(out_order, out_order + n_experts,
                   [&](int32_t a, int32_t b) { return score[static_cast<size_t>(a)] > score[static_cast<size_t>(b)]; });
  return EMOE_OK;
}

int emoe_build_profile2(const int32_t* trace, int n_tokens, int n_layers, int top_k, int n_experts, float* out_prior2) {
  if (!trace || !out_prior2 || n_tokens <= 0 || n_layers <= 0 || top_k <= 0 || n_experts <= 0) return EMOE_ERR_INVALID_ARG;
  if (n_experts > EMOE_MAX_EXPERTS || top_k > n_experts) return EMOE_ERR_INVALID_ARG;
  const size_t E = static_cast<size_t>(n_experts);
  const size_t per_layer = E * E * E;
  std::vector<double> cnt(per_layer);
  std::vector<long long> seen(E * E);
  for (int n = 0; n < n_layers; ++n) {
    float* out = out_prior2 + static_cast<size_t>(n) * per_layer;
    if (n < 2) {  // no two previous layers
      std::fill(out, out + per_layer, 0.0f);
      continue;
    }
    std::fill(cnt.begin(), cnt.end(), 0.0);
    std::fill(seen.begin(), seen.end(), 0LL);
    for (int t = 0; t < n_tokens; ++t) {
      const int32_t* row = trace + (static_cast<size_t>(t) * n_layers) * top_k;
      const int32_t* l2 = row + static_cast<size_t>(n - 2) * top_k;
      const int32_t* l1 = row + static_cast<size_t>(n - 1) * top_k;
      const int32_t* l0 = row + static_cast<size_t>(n) * top_k;
      for (int i = 0; i < top_k; ++i)
        for (int j = 0; j < top_k; ++j) {
          const int a = l2[i], b = l1[j];
          if (a < 0 || a >= n_experts || b < 0 || b >= n_experts) return EMOE_ERR_INVALID_ARG;
          ++seen[a * E + b];
          for (int k = 0; k < top_k; ++k) {
            const int e = l0[k];
            if (e < 0 || e >= n_experts) return EMOE_ERR_INVALID_ARG;
            cnt[(a * E + b) * E + e] += 1.0;
          }
        }
    }
    for (size_t ab = 0; ab < E * E; ++ab)
      for (size_t e = 0; e < E; ++e)
        out[ab * E + e] = seen[ab] ? static_cast<float>(cnt[ab * E + e] / static_cast<double>(seen[ab]))
                                   : static_cast<float>(1.0 / static_cast<double>(E));
  }
  return EMOE_OK;
}

int emoe_rank_experts2(const float* prior2_layer, int n_experts, const int32_t* prev2_ids, int n_prev2,
                       const int32_t* prev1_ids, int n_prev1, int32_t* out_order) {
  if (!prior2_layer || !prev2_ids || !prev1_ids || !out_order || n_experts <= 0 || n_prev2 <= 0 || n_prev1 <= 0)
    return EMOE_ERR_INVALID_ARG;
  const size_t E = static_cast<size_t>(n_experts);
  std::vector<double> score(E, 0.0);
  for (int i = 0; i < n_prev2; ++i) {
    if (prev2_ids[i] < 0 || prev2_ids[i] >= n_experts) return EMOE_ERR_INVALID_ARG;
    for (int j = 0; j < n_prev1; ++j) {
      if (prev1_ids[j] < 0 || prev1_ids[j] >= n_experts) return EMOE_ERR_INVALID_ARG;
      const float* row = prior2_layer + (static_cast<size_t>(prev2_ids[i]) * E + static_cast<size_t>(prev1_ids[j])) * E;
      for (size_t e = 0; e < E; ++e) score[e] += static_cast<double>(row[e]);
    }
  }
  for (int e = 0; e < n_experts; ++e) out_order[e] = e;
  std::stable_sort(out_order, out_order + n_experts,
                   [&](int32_t a, int32_t b) { return score[static_cast<size_t>(a)] > score[static_cast<size_t>(b)]; });
  return EMOE_OK;
}

}  // extern "C"
