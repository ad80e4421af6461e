// C-ABI layer of libswarm: argument validation, workspace carving and kernel sequencing.
// No device memory is allocated here; every scratch byte comes from the caller's workspace.  (swarm_create
// allocates one 64-byte word of pinned host memory, the completion word of swarm_step_host.)
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstdlib>
#include <cstring>
#include <new>

#include "swarm_internal.cuh"

// Stage ranges for timeline tools (Nsight Systems and the like): compiled in with -DSWARM_NVTX, absent otherwise.
// A range covers the enqueueing of a stage on the host; the tools attach the kernels launched inside it.
#ifdef SWARM_NVTX
#include <nvtx3/nvToolsExt.h>
struct StageRange {
  explicit StageRange(const char* name) { nvtxRangePushA(name); }
  ~StageRange() { nvtxRangePop(); }
};
#define SWARM_RANGE(name) StageRange swarm_range_(name)
#else
#define SWARM_RANGE(name) do { } while (0)
#endif

using namespace swarm;

struct swarm_ctx {
  swarm_shape shape;
  Geometry geo;
  WorkspaceLayout lay;
  uint8_t* ws;
  int64_t ws_bytes;
  int user_splits;            // 0 = chosen from the shape
  int select_sms;             // SMs the scorer leaves to the selection CTAs; < 0 = chosen from the shape
  bool index_prefetch;        // swarm_set_index_prefetch
  cudaStream_t tail_stream;   // swarm_set_tail_stream: where swarm_step enqueues cluster resolution (null: inside the step)
  cudaEvent_t ev_selected;    // recorded on the step's stream behind the selection; the tail stream waits for it
  cudaEvent_t ev_resolved;    // recorded on the tail stream behind the resolution; swarm_tail_join waits for it
  bool tail_pending;          // a resolution has been enqueued on the tail stream since the last join
  cudaError_t last_err;
  cudaGraphExec_t host_graph;  // swarm_step_host: the recorded step, valid for the arguments in host_key
  unsigned char host_key[256];
  bool host_graph_ok;
  bool host_graph_signals;    // the recorded step ends by raising *done_h
  bool has_cache;
  swarm_cache cache;
  int32_t* submit_order;      // optional outputs of the resolution (swarm_set_submit_order)
  int32_t* submit_info;
  unsigned* done_h;           // one word of pinned host memory the publish kernel raises when a host step is complete,
  unsigned* done_d;           // and the address the device writes it through (both null if the allocation failed)
};

namespace {

inline int64_t align256(int64_t x) { return (x + 255) & ~int64_t(255); }

int32_t check_shape(const swarm_shape* s) {
  if (s == nullptr) return SWARM_ERR_INVALID_ARG;
  if (s->batch < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->top_k < 1 || s->max_pages_per_req < 1 ||
      s->max_clusters_total < 1 || s->n_pool_pages < 1 || s->n_queues < 1 || s->n_queues > 32 ||
      s->n_q_heads % s->n_kv_heads != 0 || (s->flags & ~(SWARM_ORDER_BY_ID | SWARM_UNIT_LOAD)) != 0u ||
      s->local_window_pages < 0 || s->local_window_pages > s->top_k || s->reserved != 0)
    return SWARM_ERR_INVALID_ARG;
  if (s->head_dim != kHeadDim || (s->page_size != 16 && s->page_size != 32)) return SWARM_ERR_UNSUPPORTED;
  // launch-grid and index-width limits
  const int64_t bh = (int64_t)s->batch * s->n_q_heads;
  if (bh * s->top_k >= (int64_t(1) << 31) || bh * kMaxSplits >= (int64_t(1) << 31) || s->batch > 65535 ||
      (int64_t)s->n_kv_heads * (s->n_q_heads / s->n_kv_heads) > 65535 ||
      (int64_t)s->page_size * s->max_pages_per_req >= (int64_t(1) << 31))
    return SWARM_ERR_UNSUPPORTED;
  return SWARM_OK;
}

WorkspaceLayout make_layout(const swarm_shape& s) {
  WorkspaceLayout l;
  const int64_t bh = (int64_t)s.batch * s.n_q_heads;
  int64_t off = 0;
  l.n_guard = 0;
  auto place = [&](int64_t bytes) -> int64_t {               // a guard, then the region
    l.guard[l.n_guard++] = off;
    const int64_t at = off + kGuardBytes;
    off = align256(at + bytes);
    return at;
  };
  l.status = place(256 + 1024);
  l.scores = place(bh * s.max_pages_per_req * 4);
  l.n_tok = place(bh * 4);
  l.q_stage = place(bh * kHeadDim * 2);
  l.flags_alt = align256((int64_t)s.max_clusters_total + 16);          // two arrays: alternate steps of the overlapped
  l.flags = place(2 * l.flags_alt);                                    // tail mark alternate ones
  l.part_acc = place(bh * kMaxSplits * kHeadDim * 4);
  l.part_ml = place(bh * kMaxSplits * 2 * 4);
  l.items = place((int64_t)s.max_clusters_total * 16);
  l.selmap = place(bh * selmap_pitch_bytes(s.max_pages_per_req));
  l.tickets = place(bh * 4);
  l.ctl = place(64 * 4);
  l.ready = place((int64_t)s.batch * head_pairs(s.n_kv_heads) * 4);
  l.sel_ready = place((int64_t)s.batch * s.n_kv_heads * 4);
  l.selmap_ll = place(bh * selmap_pitch_bytes(s.max_pages_per_req) * 2);
  l.scores_ll = place(bh <= kLlScoreLists ? bh * s.max_pages_per_req * 8 : 0);
  l.guard[l.n_guard++] = off;
  l.total = off + kGuardBytes;
  return l;
}

int pick_splits(const swarm_ctx* ctx, bool paged, bool fused = false) {
  // One CTA fits per SM (the shared-memory rings).  Two regimes, both measured:
  //  - one wave: as many splits as keep every CTA resident at once (inside the fused step one SM is left for
  //    the resolution CTA); right when a group's pages do not give many CTAs enough to do;
  //  - several waves: about 2.6 CTAs per SM in total.  The hardware then hands the next CTA to whichever SM
  //    frees up, which evens out both the groups' unequal page unions and a group count that does not divide
  //    the SMs (at 128 groups: 0.62 -> 0.67 of the memory rate; at 32 groups with long unions: 0.73 -> 0.91).
  // For gathered buffers: one wave, at least 4 pages per split.
  if (ctx->user_splits > 0) return ctx->user_splits;
  const Geometry& g = ctx->geo;
  const int64_t groups = attention_groups(g, paged);
  const int sms = sm_count();
  int64_t n = std::max<int64_t>(1, (sms - (fused ? 1 : 0)) / groups);
  if (paged) {
    // 16-token units a group probably streams: the heads of a group share roughly half of their pages
    const double est_units = 0.55 * std::min(g.g, 8) * g.k * (g.S / 16);
    int64_t waves = std::max<int64_t>(1, std::llround(2.6 * sms / (double)groups));
    if (waves == 1 && groups > sms) waves = 2;
    if (waves > n && est_units / (double)waves >= 64.0) {
      n = waves;
      // Short ranges (under ~1 MB of K/V) spend a third of a CTA's life on fixed costs: then fewer, longer CTAs
      // in exactly two waves (pick_more completes the second) beat 2.6 uneven ones (16 requests x 32K tokens:
      // attention 55.4 -> 54.3 us).
      const int64_t two_waves = 2 * (int64_t)(sms - (fused ? 1 : 0)) / groups;
      if (est_units / (double)n < 128.0 && two_waves >= 1 && two_waves < n) n = two_waves;
    }
  } else {
    n = std::min<int64_t>(n, std::max(1, g.k / 4));
  }
  n = std::min<int64_t>(n, kMaxSplits);
  // The CTA that merges a head reads the splits' partials sixteen at a time: a few splits past a multiple of 16
  // cost it another trip to L2 (128K tokens, 8 groups: 16 splits 29.9 us per step, 18 splits 30.2).
  if (n > 16 && (n % 16) * 4 <= n) n -= n % 16;
  return (int)std::max<int64_t>(n, 1);
}

// Several waves of CTAs: the last `more` groups get one range more, so that the grid is a whole number of waves
// (one CTA per SM at a time).  0 when the grid is one wave, when the caller fixed the split count, or when it would
// take more than half of the groups.
int pick_more(const swarm_ctx* ctx, bool paged, int n_splits, bool fused = false) {
  if (ctx->user_splits > 0 || !paged || n_splits + 1 > kMaxSplits) return 0;
  const int64_t groups = attention_groups(ctx->geo, paged);
  const int64_t sms = sm_count() - (fused ? 1 : 0), ctas = groups * n_splits;
  if (ctas <= sms) return 0;
  const int64_t more = (sms - ctas % sms) % sms;
  // (a partial last wave leaves SMs idle at the end: 64 ragged requests, 1024 -> 1036 CTAs = 7 waves: attention
  // 179.6 -> 174.6 us; where it would take more than half of the groups the ranges are long and it gains nothing)
  return 2 * more <= groups ? (int)more : 0;
}

// The hand-off counters of a step (see StepTickets).  The scorer's tickets exist only when the streaming scorer
// runs; `with_attention`: the selection also announces its heads to an attention kernel launched by the same call.
// `bitmaps_by_word`: the page bitmaps go to the attention kernel as self-validating words instead of behind a
// ticket per KV head -- for attention grids of one wave, where the step is a chain of latencies and the hand-off
// is on it (128K tokens: 29.15 -> 28.64 us per step, 32K tokens: 18.1 -> 17.1); with several waves the CTAs
// that wait would all be polling while the scorer and the selection still need the memory system (4 x 512K
// tokens: 224.5 -> 226.5 us).
StepTickets step_tickets(const swarm_ctx* ctx, const Geometry& g, bool with_attention, bool bitmaps_by_word = false) {
  StepTickets t;
  t.ctl = reinterpret_cast<unsigned*>(ctx->ws + ctx->lay.ctl);
  t.ready = score_raises_tickets(g) ? reinterpret_cast<unsigned*>(ctx->ws + ctx->lay.ready) : nullptr;
  t.sel_ready = (with_attention && t.ready != nullptr) ? reinterpret_cast<unsigned*>(ctx->ws + ctx->lay.sel_ready) : nullptr;
  // (few lists: the instances of the selection kernel that carry the code for it, see launch_topk)
  const bool few = (long long)g.B * g.Hq <= kLlScoreLists && g.Pmax <= 16384;
  t.selmap_ll = (t.sel_ready != nullptr && bitmaps_by_word && few) ? reinterpret_cast<uint2*>(ctx->ws + ctx->lay.selmap_ll) : nullptr;
  // ... and with an even row length (16-byte loads of two pairs) so do the scores
  t.scores_ll = (t.selmap_ll != nullptr && g.Pmax % 2 == 0) ? reinterpret_cast<uint2*>(ctx->ws + ctx->lay.scores_ll) : nullptr;
  return t;
}

// SMs the scorer leaves free so that the selection CTAs are resident while it runs (they wait for its
// tickets); inside a step with an overlapped tail one more for the resolution CTA of the previous step.
int reserved_sms(const swarm_ctx* ctx, const Geometry& g, bool tail) {
  if (!score_raises_tickets(g)) return 0;
  int n = ctx->select_sms;
  if (n < 0) {
    // Selection CTAs of up to 256 threads fit on an SM beside a scorer CTA (registers and shared memory were
    // sized for it): nothing to reserve.  Larger ones need an SM of their own: one per list, at most a
    // quarter of the device (measured at 64 requests of up to 16384 pages: 37 reserved SMs beat both 0 and 54).
    const int threads = topk_threads(g.Pmax);
    const long long lists = (long long)g.B * g.Hq;
    const int per_sm = std::max(1, 1024 / threads);
    n = threads <= 256 ? 0 : (int)std::min<long long>((lists + per_sm - 1) / per_sm, sm_count() / 4);
  }
  n += tail ? 1 : 0;
  return std::min(n, sm_count() - 8);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool bad(const void* p) { return p == nullptr || !aligned16(p); }

int32_t fail(swarm_ctx* ctx, cudaError_t e) {
  ctx->last_err = e;
  return SWARM_ERR_CUDA;
}

#define SWARM_TRY(expr)                              \
  do {                                               \
    cudaError_t e_ = (expr);                         \
    if (e_ != cudaSuccess) return fail(ctx, e_);     \
  } while (0)

int32_t need_ws(const swarm_ctx* ctx) {
  if (ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  if (ctx->ws == nullptr) return SWARM_ERR_WORKSPACE_TOO_SMALL;
  return SWARM_OK;
}

template <class T>
T* ws_ptr(const swarm_ctx* ctx, int64_t off) { return reinterpret_cast<T*>(ctx->ws + off); }

bool select_inputs_ok(const swarm_inputs* in) {
  return in && !bad(in->q) && !bad(in->ksum) && !bad(in->page_base) && !bad(in->ctx_len);
}
bool resolve_inputs_ok(const swarm_inputs* in) {
  return in && !bad(in->page_base) && !bad(in->page2cluster) && !bad(in->cluster_base) &&
         !bad(in->cluster_replica_mask) && !bad(in->cluster_size);
}
bool pool_inputs_ok(const swarm_inputs* in) {
  return in && !bad(in->kv_pool) && !bad(in->page_base) && !bad(in->ctx_len);
}

// The device's address of a pinned host buffer (unified addressing), or null when the device cannot store to it
// directly (pageable memory, no mapping, misaligned) or when the pointer itself is null.
template <class T>
T* device_view(T* host, size_t align) {
  if (host == nullptr || (reinterpret_cast<uintptr_t>(host) & (align - 1)) != 0) return nullptr;
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return nullptr;
  return static_cast<T*>(attr.devicePointer);
}

// Arguments of the cluster-resolution body; sel == nullptr when the flags were set by the selection kernel.
ResolveArgs step_resolve_args(swarm_ctx* ctx, const swarm_inputs* in, const int32_t* sel, const int32_t* n_sel,
                              int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq, int32_t* queue_load) {
  return make_resolve_args(ctx->geo, sel, n_sel, in->page_base, in->page2cluster, in->cluster_base,
                           in->cluster_replica_mask, in->cluster_size, ws_ptr<uint8_t>(ctx, ctx->lay.flags),
                           ws_ptr<unsigned>(ctx, ctx->lay.status + 64), ws_ptr<uint4>(ctx, ctx->lay.items), uniq, queue_of,
                           n_uniq, queue_load, ws_ptr<uint32_t>(ctx, ctx->lay.status),
                           ctx->has_cache ? &ctx->cache : nullptr, ctx->submit_order, ctx->submit_info);
}

}  // namespace

extern "C" {

int32_t swarm_version(void) { return 100; }

int64_t swarm_workspace_bytes(const swarm_shape* shape) {
  const int32_t rc = check_shape(shape);
  if (rc != SWARM_OK) return -(int64_t)rc;
  return make_layout(*shape).total;
}

int32_t swarm_create(const swarm_shape* shape, swarm_ctx** out_ctx) {
  if (out_ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  const int32_t rc = check_shape(shape);
  if (rc != SWARM_OK) return rc;
  swarm_ctx* ctx = new (std::nothrow) swarm_ctx();
  if (ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  ctx->shape = *shape;
  Geometry& g = ctx->geo;
  g.B = shape->batch; g.Hq = shape->n_q_heads; g.Hkv = shape->n_kv_heads; g.g = g.Hq / g.Hkv;
  g.S = shape->page_size; g.k = shape->top_k; g.D = shape->n_queues; g.Pmax = shape->max_pages_per_req;
  g.Cmax = shape->max_clusters_total; g.flags = shape->flags; g.n_pool_pages = shape->n_pool_pages;
  g.W = shape->local_window_pages;
  g.scorer = SWARM_SCORER_AUTO;
  ctx->lay = make_layout(*shape);
  ctx->ws = nullptr;
  ctx->ws_bytes = 0;
  ctx->user_splits = 0;
  ctx->select_sms = -1;
  ctx->index_prefetch = false;
  ctx->tail_stream = nullptr;
  ctx->ev_selected = nullptr;
  ctx->ev_resolved = nullptr;
  ctx->tail_pending = false;
  ctx->last_err = cudaSuccess;
  ctx->host_graph = nullptr;
  ctx->host_graph_ok = true;
  ctx->host_graph_signals = false;
  ctx->has_cache = false;
  ctx->submit_order = nullptr;
  ctx->submit_info = nullptr;
  std::memset(ctx->host_key, 0, sizeof ctx->host_key);
  ctx->done_h = nullptr;
  ctx->done_d = nullptr;
  void* flag = nullptr;
  if (cudaHostAlloc(&flag, 64, cudaHostAllocMapped) == cudaSuccess) {
    void* flag_d = nullptr;
    if (cudaHostGetDevicePointer(&flag_d, flag, 0) == cudaSuccess) {
      ctx->done_h = static_cast<unsigned*>(flag);
      ctx->done_d = static_cast<unsigned*>(flag_d);
      *ctx->done_h = 0u;
    } else {
      cudaFreeHost(flag);
    }
  }
  cudaGetLastError();                                     // without the word, host steps wait on the stream
  cudaError_t e = configure_score();
  if (e == cudaSuccess) e = configure_topk();
  if (e == cudaSuccess) e = configure_resolve();
  if (e == cudaSuccess) e = configure_attention();
  if (e == cudaSuccess) e = configure_medoid();
  if (e != cudaSuccess) {
    if (ctx->done_h != nullptr) cudaFreeHost(ctx->done_h);
    delete ctx;
    return SWARM_ERR_CUDA;
  }
  *out_ctx = ctx;
  return SWARM_OK;
}

int32_t swarm_destroy(swarm_ctx* ctx) {
  if (ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  if (ctx->host_graph != nullptr) cudaGraphExecDestroy(ctx->host_graph);
  if (ctx->done_h != nullptr) cudaFreeHost(ctx->done_h);
  if (ctx->ev_selected != nullptr) cudaEventDestroy(ctx->ev_selected);
  if (ctx->ev_resolved != nullptr) cudaEventDestroy(ctx->ev_resolved);
  delete ctx;
  return SWARM_OK;
}

int32_t swarm_set_workspace(swarm_ctx* ctx, void* device_mem, int64_t bytes, void* stream) {
  if (ctx == nullptr || device_mem == nullptr || (reinterpret_cast<uintptr_t>(device_mem) & 255u))
    return SWARM_ERR_INVALID_ARG;
  if (bytes < ctx->lay.total) return SWARM_ERR_WORKSPACE_TOO_SMALL;
  ctx->ws = static_cast<uint8_t*>(device_mem);
  ctx->ws_bytes = bytes;
  // regions that must hold zeros between calls: status word, ticket counters, dedup flags
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SWARM_TRY(cudaMemsetAsync(ctx->ws + ctx->lay.status, 0, 256, st));
  SWARM_TRY(cudaMemsetAsync(ctx->ws + ctx->lay.flags, 0, 2 * ctx->lay.flags_alt, st));
  SWARM_TRY(cudaMemsetAsync(ctx->ws + ctx->lay.tickets, 0, ctx->lay.total - ctx->lay.tickets, st));   // and the hand-off counters
  for (int i = 0; i < ctx->lay.n_guard; ++i)               // canaries last: the spans above run over some of them
    SWARM_TRY(cudaMemsetAsync(ctx->ws + ctx->lay.guard[i], kCanaryByte, kGuardBytes, st));
  return SWARM_OK;
}

int32_t swarm_check_workspace(swarm_ctx* ctx, void* stream, uint32_t* damaged) {
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (damaged == nullptr) return SWARM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static_assert(sizeof(ctx->lay.guard) / sizeof(ctx->lay.guard[0]) <= 32, "one bit per guard");
  unsigned char host[20 * kGuardBytes];
  for (int i = 0; i < ctx->lay.n_guard; ++i)
    SWARM_TRY(cudaMemcpyAsync(host + i * kGuardBytes, ctx->ws + ctx->lay.guard[i], kGuardBytes, cudaMemcpyDeviceToHost, st));
  SWARM_TRY(cudaStreamSynchronize(st));
  uint32_t bits = 0u;
  for (int i = 0; i < ctx->lay.n_guard; ++i)
    for (int j = 0; j < kGuardBytes; ++j)
      if (host[i * kGuardBytes + j] != (unsigned char)kCanaryByte) { bits |= 1u << i; break; }
  *damaged = bits;
  return SWARM_OK;
}

int32_t swarm_set_attn_splits(swarm_ctx* ctx, int32_t n_splits) {
  if (ctx == nullptr || n_splits < 0 || n_splits > kMaxSplits) return SWARM_ERR_INVALID_ARG;
  ctx->user_splits = n_splits;
  return SWARM_OK;
}

int32_t swarm_set_tail_stream(swarm_ctx* ctx, void* tail_stream) {
  if (ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  if (tail_stream != nullptr && ctx->ev_selected == nullptr) {
    SWARM_TRY(cudaEventCreateWithFlags(&ctx->ev_selected, cudaEventDisableTiming));
    SWARM_TRY(cudaEventCreateWithFlags(&ctx->ev_resolved, cudaEventDisableTiming));
  }
  ctx->tail_stream = static_cast<cudaStream_t>(tail_stream);
  ctx->tail_pending = false;
  if (ctx->host_graph != nullptr) { cudaGraphExecDestroy(ctx->host_graph); ctx->host_graph = nullptr; }
  return SWARM_OK;
}

int32_t swarm_tail_join(swarm_ctx* ctx, void* stream) {
  if (ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  if (ctx->tail_stream == nullptr || !ctx->tail_pending) return SWARM_OK;
  SWARM_TRY(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), ctx->ev_resolved, 0));
  ctx->tail_pending = false;
  return SWARM_OK;
}

int32_t swarm_set_select_sms(swarm_ctx* ctx, int32_t n_sms) {
  if (ctx == nullptr || n_sms < -1 || n_sms > 1024) return SWARM_ERR_INVALID_ARG;
  ctx->select_sms = n_sms;
  if (ctx->host_graph != nullptr) { cudaGraphExecDestroy(ctx->host_graph); ctx->host_graph = nullptr; }
  return SWARM_OK;
}

int32_t swarm_set_scorer(swarm_ctx* ctx, int32_t kind) {
  if (ctx == nullptr || kind < SWARM_SCORER_AUTO || kind > SWARM_SCORER_FP32) return SWARM_ERR_INVALID_ARG;
  if (kind == SWARM_SCORER_TENSOR && !score_streams(ctx->geo)) return SWARM_ERR_UNSUPPORTED;
  ctx->geo.scorer = kind;
  if (ctx->host_graph != nullptr) { cudaGraphExecDestroy(ctx->host_graph); ctx->host_graph = nullptr; }
  return SWARM_OK;
}

int32_t swarm_set_index_prefetch(swarm_ctx* ctx, int32_t on) {
  if (ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  ctx->index_prefetch = on != 0;
  if (ctx->host_graph != nullptr) { cudaGraphExecDestroy(ctx->host_graph); ctx->host_graph = nullptr; }
  return SWARM_OK;
}

int32_t swarm_set_cache(swarm_ctx* ctx, const swarm_cache* cache) {
  if (ctx == nullptr) return SWARM_ERR_INVALID_ARG;
  if (cache != nullptr && (cache->resident == nullptr || cache->freq == nullptr || !(cache->t_base >= 0.f) ||
                           !(cache->t_transfer >= 0.f)))
    return SWARM_ERR_INVALID_ARG;
  ctx->has_cache = cache != nullptr;
  if (cache != nullptr) ctx->cache = *cache;
  if (ctx->host_graph != nullptr) { cudaGraphExecDestroy(ctx->host_graph); ctx->host_graph = nullptr; }
  return SWARM_OK;
}

int32_t swarm_set_submit_order(swarm_ctx* ctx, int32_t* submit_order, int32_t* submit_info) {
  if (ctx == nullptr || (submit_order == nullptr && submit_info != nullptr) || !aligned16(submit_order) ||
      !aligned16(submit_info))
    return SWARM_ERR_INVALID_ARG;
  ctx->submit_order = submit_order;
  ctx->submit_info = submit_info;
  if (ctx->host_graph != nullptr) { cudaGraphExecDestroy(ctx->host_graph); ctx->host_graph = nullptr; }
  return SWARM_OK;
}

int64_t swarm_build_clusters_workspace_bytes(int32_t n_entries) {
  if (n_entries < 1 || n_entries > 32768) return -(int64_t)SWARM_ERR_UNSUPPORTED;
  return build_clusters_workspace_bytes(n_entries);
}

int32_t swarm_build_clusters(const float* dist, int32_t n_entries, float tau, void* workspace, int64_t workspace_bytes,
                             int32_t* density, int32_t* cluster_ptr, int32_t* cluster_members, int64_t members_cap,
                             int32_t* medoid, int32_t* n_clusters, int32_t* dev_status, void* stream) {
  if (n_entries < 1 || !(tau >= 0.f) || bad(dist) || bad(workspace) || bad(density) || bad(cluster_ptr) ||
      bad(cluster_members) || bad(medoid) || bad(n_clusters) || bad(dev_status) || members_cap < n_entries ||
      members_cap > 0x7FFFFFFFLL)                            // cluster_ptr holds 32-bit offsets
    return SWARM_ERR_INVALID_ARG;
  if (n_entries > 32768) return SWARM_ERR_UNSUPPORTED;
  if (workspace_bytes < build_clusters_workspace_bytes(n_entries)) return SWARM_ERR_WORKSPACE_TOO_SMALL;
  const cudaError_t e = launch_build_clusters(dist, n_entries, tau, workspace, density, cluster_ptr, cluster_members,
                                              members_cap, medoid, n_clusters, dev_status,
                                              static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SWARM_OK : SWARM_ERR_CUDA;
}

int64_t swarm_cache_admit_workspace_bytes(int32_t n_clusters) {
  if (n_clusters < 1 || n_clusters > 65536) return -(int64_t)SWARM_ERR_UNSUPPORTED;
  return cache_admit_workspace_bytes(n_clusters);
}

int32_t swarm_cache_admit(const float* score, const uint16_t* cluster_size, int32_t n_clusters, int64_t capacity_pages,
                          void* workspace, int64_t workspace_bytes, uint8_t* resident, int32_t* info, void* stream) {
  if (n_clusters < 1 || capacity_pages < 0 || bad(score) || bad(cluster_size) || bad(workspace) || bad(resident) ||
      !aligned16(info))
    return SWARM_ERR_INVALID_ARG;
  if (n_clusters > 65536) return SWARM_ERR_UNSUPPORTED;
  if (workspace_bytes < cache_admit_workspace_bytes(n_clusters)) return SWARM_ERR_WORKSPACE_TOO_SMALL;
  const cudaError_t e = launch_cache_admit(score, cluster_size, n_clusters, capacity_pages, workspace, resident, info,
                                           static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? SWARM_OK : SWARM_ERR_CUDA;
}

int32_t swarm_last_cuda_error(const swarm_ctx* ctx) { return ctx ? (int32_t)ctx->last_err : 0; }

int32_t swarm_device_status(swarm_ctx* ctx, void* stream, uint32_t* bits) {
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (bits == nullptr) return SWARM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* dev = ws_ptr<uint32_t>(ctx, ctx->lay.status);
  SWARM_TRY(cudaMemcpyAsync(bits, dev, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
  SWARM_TRY(cudaMemsetAsync(dev, 0, sizeof(uint32_t), st));
  SWARM_TRY(cudaStreamSynchronize(st));
  return SWARM_OK;
}

int32_t swarm_build_summaries(swarm_ctx* ctx, const swarm_inputs* in, void* ksum_out, void* stream) {
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (!pool_inputs_ok(in) || bad(ksum_out)) return SWARM_ERR_INVALID_ARG;
  SWARM_TRY(launch_build_summaries(ctx->geo, static_cast<const uint16_t*>(in->kv_pool), in->page_base, in->ctx_len,
                                   static_cast<uint16_t*>(ksum_out), ws_ptr<uint32_t>(ctx, ctx->lay.status),
                                   static_cast<cudaStream_t>(stream)));
  return SWARM_OK;
}

int32_t swarm_select(swarm_ctx* ctx, const swarm_inputs* in, float* scores, int32_t* sel, int32_t* n_sel,
                     void* stream) {
  SWARM_RANGE("swarm_select");
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (!select_inputs_ok(in) || bad(sel) || bad(n_sel) || (scores && !aligned16(scores))) return SWARM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* sc = scores ? scores : ws_ptr<float>(ctx, ctx->lay.scores);
  TopkLinks links;
  links.tk = step_tickets(ctx, ctx->geo, false);
  links.req_base = in->page_base;
  SWARM_TRY(launch_page_score(ctx->geo, static_cast<const uint16_t*>(in->q), static_cast<const uint16_t*>(in->ksum),
                              in->page_base, in->ctx_len, sc, ws_ptr<uint32_t>(ctx, ctx->lay.status), st, links.tk.ready,
                              reserved_sms(ctx, ctx->geo, false)));
  SWARM_TRY(launch_topk(ctx->geo, sc, in->ctx_len, sel, n_sel, ws_ptr<uint32_t>(ctx, ctx->lay.status), st, true, links,
                        ws_ptr<uint8_t>(ctx, ctx->lay.selmap)));
  return SWARM_OK;
}

int32_t swarm_resolve_clusters(swarm_ctx* ctx, const swarm_inputs* in, const int32_t* sel, const int32_t* n_sel,
                               int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq, int32_t* queue_load,
                               void* stream) {
  SWARM_RANGE("swarm_resolve_clusters");
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (!resolve_inputs_ok(in) || bad(sel) || bad(n_sel) || bad(uniq) || bad(queue_of) || bad(n_uniq) ||
      bad(queue_load))
    return SWARM_ERR_INVALID_ARG;
  SWARM_TRY(launch_resolve(step_resolve_args(ctx, in, sel, n_sel, uniq, queue_of, n_uniq, queue_load), static_cast<cudaStream_t>(stream), false));
  return SWARM_OK;
}

int32_t swarm_gather(swarm_ctx* ctx, const swarm_inputs* in, const int32_t* sel, const int32_t* n_sel, void* k_out,
                     void* v_out, int32_t* n_tok, void* stream) {
  SWARM_RANGE("swarm_gather");
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (!pool_inputs_ok(in) || bad(sel) || bad(n_sel) || bad(k_out) || bad(v_out) || (n_tok && !aligned16(n_tok)))
    return SWARM_ERR_INVALID_ARG;
  SWARM_TRY(launch_gather(ctx->geo, static_cast<const uint16_t*>(in->kv_pool), sel, n_sel, in->page_base,
                          in->ctx_len, static_cast<uint16_t*>(k_out), static_cast<uint16_t*>(v_out), n_tok,
                          ws_ptr<uint32_t>(ctx, ctx->lay.status), static_cast<cudaStream_t>(stream)));
  return SWARM_OK;
}

int32_t swarm_sparse_attn(swarm_ctx* ctx, const void* q, const void* k_g, const void* v_g, const int32_t* n_tok,
                          float* out, float* lse, void* stream) {
  SWARM_RANGE("swarm_sparse_attn");
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (bad(q) || bad(k_g) || bad(v_g) || bad(n_tok) || bad(out) || bad(lse)) return SWARM_ERR_INVALID_ARG;
  AttnArgs a{};
  a.q = static_cast<const uint16_t*>(q);
  a.k_g = static_cast<const uint16_t*>(k_g);
  a.v_g = static_cast<const uint16_t*>(v_g);
  a.n_tok = n_tok;
  a.part_acc = ws_ptr<float>(ctx, ctx->lay.part_acc);
  a.part_ml = ws_ptr<float>(ctx, ctx->lay.part_ml);
  a.tickets = ws_ptr<unsigned>(ctx, ctx->lay.tickets);
  a.out = out;
  a.lse = lse;
  a.n_splits = pick_splits(ctx, false);
  SWARM_TRY(launch_attention(ctx->geo, a, ws_ptr<uint32_t>(ctx, ctx->lay.status), static_cast<cudaStream_t>(stream),
                             /*overlap=*/true));
  return SWARM_OK;
}

namespace {
AttnArgs paged_args(const swarm_ctx* ctx, const swarm_inputs* in, float* out, float* lse) {
  AttnArgs a{};
  a.q = static_cast<const uint16_t*>(in->q);
  a.kv_pool = static_cast<const uint16_t*>(in->kv_pool);
  a.selmap = ws_ptr<uint8_t>(ctx, ctx->lay.selmap);
  a.selmap_pitch = selmap_pitch_bytes(ctx->geo.Pmax);
  a.page_base = in->page_base;
  a.ctx_len = in->ctx_len;
  a.part_acc = ws_ptr<float>(ctx, ctx->lay.part_acc);
  a.part_ml = ws_ptr<float>(ctx, ctx->lay.part_ml);
  a.tickets = ws_ptr<unsigned>(ctx, ctx->lay.tickets);
  a.out = out;
  a.lse = lse;
  a.n_splits = pick_splits(ctx, true);
  a.n_more = pick_more(ctx, true, a.n_splits);
  return a;
}
}  // namespace

int32_t swarm_sparse_attn_paged(swarm_ctx* ctx, const swarm_inputs* in, const int32_t* sel, const int32_t* n_sel,
                                float* out, float* lse, void* stream) {
  SWARM_RANGE("swarm_sparse_attn_paged");
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (!pool_inputs_ok(in) || bad(in->q) || bad(out) || bad(lse) || ((sel == nullptr) != (n_sel == nullptr)) ||
      (sel && (bad(sel) || bad(n_sel))))
    return SWARM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (sel != nullptr)   // otherwise: the page bitmaps of this ctx's last swarm_select / swarm_step are reused
    SWARM_TRY(launch_selmap_from_sel(ctx->geo, sel, n_sel, ws_ptr<uint8_t>(ctx, ctx->lay.selmap), st));
  SWARM_TRY(launch_attention(ctx->geo, paged_args(ctx, in, out, lse), ws_ptr<uint32_t>(ctx, ctx->lay.status), st,
                             /*overlap=*/true));
  return SWARM_OK;
}

namespace {
int32_t step_impl(swarm_ctx* ctx, const swarm_inputs* in, const swarm_outputs* o, void* stream, const HostMirror* host,
                  int parts);
constexpr int kStepBegin = 1, kStepEnd = 2;
}

int32_t swarm_step(swarm_ctx* ctx, const swarm_inputs* in, const swarm_outputs* o, void* stream) {
  return step_impl(ctx, in, o, stream, nullptr, kStepBegin | kStepEnd);
}

int32_t swarm_step_begin(swarm_ctx* ctx, const swarm_inputs* in, const swarm_outputs* o, void* stream) {
  return step_impl(ctx, in, o, stream, nullptr, kStepBegin);
}

int32_t swarm_step_end(swarm_ctx* ctx, const swarm_inputs* in, const swarm_outputs* o, void* stream) {
  return step_impl(ctx, in, o, stream, nullptr, kStepEnd);
}

int32_t swarm_cluster_flags(swarm_ctx* ctx, void** flags, int64_t* n_bytes) {
  if (flags == nullptr || n_bytes == nullptr) return SWARM_ERR_INVALID_ARG;
  const int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  *flags = ws_ptr<uint8_t>(ctx, ctx->lay.flags);
  *n_bytes = ctx->geo.Cmax;
  return SWARM_OK;
}

namespace {
// The fused step, or one of its two halves (the selection with its cluster marks; attention + cluster resolution).
// `host` (swarm_step_host only) makes the last kernel store the small results into host memory too.
int32_t step_impl(swarm_ctx* ctx, const swarm_inputs* in, const swarm_outputs* o, void* stream, const HostMirror* host,
                  int parts) {
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (!select_inputs_ok(in) || !resolve_inputs_ok(in) || !pool_inputs_ok(in) || o == nullptr || bad(o->sel) ||
      bad(o->n_sel) || bad(o->uniq) || bad(o->queue_of) || bad(o->n_uniq) || bad(o->queue_load) || bad(o->out) ||
      bad(o->lse) || (o->scores && !aligned16(o->scores)) || (o->n_tok && !aligned16(o->n_tok)) ||
      ((o->k_out == nullptr) != (o->v_out == nullptr)) || (o->n_tok && !o->k_out) || (o->k_out && (!aligned16(o->k_out) || !aligned16(o->v_out))))
    return SWARM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* status = ws_ptr<uint32_t>(ctx, ctx->lay.status);
  const uint16_t* q = static_cast<const uint16_t*>(in->q);
  const uint16_t* pool = static_cast<const uint16_t*>(in->kv_pool);
  float* sc = o->scores ? o->scores : ws_ptr<float>(ctx, ctx->lay.scores);

  // Overlapped tail only for a whole step (the halves exchange the flag array between them).
  const bool whole = parts == (kStepBegin | kStepEnd);
  const bool tail = ctx->tail_stream != nullptr && whole && host == nullptr;   // (a host step waits for everything anyway)
  // the attention CTAs wait per KV head for the selection -- unless a gather sits between the two kernels,
  // which waits for all of the selection anyway
  const bool attn_tickets = whole && o->k_out == nullptr;
  TopkLinks links;
  const bool one_wave = (long long)attention_groups(ctx->geo, true) * pick_splits(ctx, true, !tail) + (tail ? 0 : 1) <= sm_count();
  links.tk = step_tickets(ctx, ctx->geo, attn_tickets, one_wave);
  links.req_base = in->page_base;
  links.flags_alt = tail ? ctx->lay.flags_alt : 0;
  if (parts & kStepBegin) {
    SWARM_RANGE("swarm: score + select");
    SWARM_TRY(launch_page_score(ctx->geo, q, static_cast<const uint16_t*>(in->ksum), in->page_base, in->ctx_len, sc,
                                status, st, links.tk.ready, reserved_sms(ctx, ctx->geo, tail), links.tk.scores_ll, links.tk.ctl,
                                ctx->index_prefetch));
    // the selection kernel also marks the selected pages' clusters and writes the per-head page bitmaps
    SWARM_TRY(launch_topk(ctx->geo, sc, in->ctx_len, o->sel, o->n_sel, status, st, true, links,
                          ws_ptr<uint8_t>(ctx, ctx->lay.selmap), in->page_base, in->page2cluster, in->cluster_base,
                          ws_ptr<uint8_t>(ctx, ctx->lay.flags), in->cluster_replica_mask, in->cluster_size));
  }
  if (!(parts & kStepEnd)) return SWARM_OK;

  SWARM_RANGE("swarm: resolve + gather + attention");
  if (o->k_out != nullptr)
    SWARM_TRY(launch_gather(ctx->geo, pool, o->sel, o->n_sel, in->page_base, in->ctx_len,
                            static_cast<uint16_t*>(o->k_out), static_cast<uint16_t*>(o->v_out), o->n_tok, status, st));
  AttnArgs a = paged_args(ctx, in, o->out, o->lse);
  ResolveArgs rs = step_resolve_args(ctx, in, nullptr, o->n_sel, o->uniq, o->queue_of, o->n_uniq, o->queue_load);
  if (host != nullptr) {
    a.host = *host;
    rs.host = *host;
  }
  if (attn_tickets) a.tk = links.tk;
  if (tail) {
    // Cluster resolution as a kernel of its own on the tail stream, forked behind the selection: nothing on the
    // step's stream waits for it, so its serial pass runs beside this step's attention and the next step's
    // scoring and selection.  (On the step's own stream it would not: a kernel launched behind another, even
    // one that never waits for it, was measured to complete only after it.)
    rs.tail_ctl = links.tk.ctl;
    rs.flags_alt = ctx->lay.flags_alt;
    SWARM_TRY(cudaEventRecord(ctx->ev_selected, st));
    SWARM_TRY(cudaStreamWaitEvent(ctx->tail_stream, ctx->ev_selected, 0));
    SWARM_TRY(launch_resolve(rs, ctx->tail_stream, /*overlap=*/false));
    SWARM_TRY(cudaEventRecord(ctx->ev_resolved, ctx->tail_stream));
    ctx->tail_pending = true;
    a.n_splits = pick_splits(ctx, true, /*fused=*/false);
    a.n_more = pick_more(ctx, true, a.n_splits, /*fused=*/false);
    // With the index prefetch the SMs the attention CTAs leave are worth something to the next step's scorer
    // (its CTAs fetch their first blocks there): they are released as soon as the CTAs have read all their pages.
    // (Without it the early release was measured 1.5 us slower: the scorer's CTAs only sat there.)
    a.release_early = ctx->index_prefetch && attn_tickets;
    SWARM_TRY(launch_attention(ctx->geo, a, status, st, /*overlap=*/true, nullptr));
    return SWARM_OK;
  }
  // Otherwise one launch runs them side by side: the attention CTAs plus one CTA for the resolution (whose
  // serial pass is the longest item of the step).
  a.n_splits = pick_splits(ctx, true, /*fused=*/true);
  a.n_more = pick_more(ctx, true, a.n_splits, /*fused=*/true);
  SWARM_TRY(launch_attention(ctx->geo, a, status, st, /*overlap=*/true, &rs));
  return SWARM_OK;
}

// Everything swarm_step_host enqueues for one step: q in, the step, the results out.  *signals is set when the
// last operation raises ctx->done_h on completion.
int32_t enqueue_host_step(swarm_ctx* ctx, const swarm_inputs* in, const swarm_outputs* o, const void* q_host,
                          float* out_host, float* lse_host, int32_t* n_uniq_host, int32_t* queue_load_host,
                          cudaStream_t st, bool* signals) {
  *signals = false;
  const int64_t bh = (int64_t)ctx->geo.B * ctx->geo.Hq;
  uint16_t* q_dev = ws_ptr<uint16_t>(ctx, ctx->lay.q_stage);
  // q: read over the bus by a kernel when the device can address the buffer, else one copy operation
  const void* q_view = device_view<const void>(q_host, 16);
  if (q_view != nullptr) SWARM_TRY(launch_fetch(q_view, q_dev, bh * kHeadDim * 2, st));
  else SWARM_TRY(cudaMemcpyAsync(q_dev, q_host, bh * kHeadDim * 2, cudaMemcpyHostToDevice, st));
  swarm_inputs local = *in;
  local.q = q_dev;
  // Results: when every destination is pinned host memory the device can address (and 16-byte aligned for
  // out), the step's last kernel stores them there as it produces them and raises the completion word (or,
  // without that word, one small kernel stores them after the step); otherwise one copy operation per buffer.
  float* out_d = device_view<float>(out_host, 16);
  float* lse_d = device_view<float>(lse_host, 4);
  int32_t* n_uniq_d = device_view<int32_t>(n_uniq_host, 4);
  int32_t* queue_load_d = device_view<int32_t>(queue_load_host, 4);
  const bool direct = (out_host == nullptr || out_d) && (lse_host == nullptr || lse_d) &&
                      (n_uniq_host == nullptr || n_uniq_d) && (queue_load_host == nullptr || queue_load_d);
  if (direct && ctx->done_d != nullptr) {
    const HostMirror host{out_d, lse_d, n_uniq_d, queue_load_d, ws_ptr<unsigned>(ctx, ctx->lay.status + 96), ctx->done_d,
                          (unsigned)bh + 1u};                // one arrival per head, one for the resolution
    const int32_t rc = step_impl(ctx, &local, o, st, &host, kStepBegin | kStepEnd);
    *signals = rc == SWARM_OK;
    return rc;
  }
  const int32_t rc = swarm_step(ctx, &local, o, st);
  if (rc != SWARM_OK) return rc;
  if (direct) {
    SWARM_TRY(launch_publish(ctx->geo, o->out, o->lse, o->n_uniq, o->queue_load, out_d, lse_d, n_uniq_d, queue_load_d, st));
    return SWARM_OK;
  }
  if (out_host) SWARM_TRY(cudaMemcpyAsync(out_host, o->out, bh * kHeadDim * 4, cudaMemcpyDeviceToHost, st));
  if (lse_host) SWARM_TRY(cudaMemcpyAsync(lse_host, o->lse, bh * 4, cudaMemcpyDeviceToHost, st));
  if (n_uniq_host) SWARM_TRY(cudaMemcpyAsync(n_uniq_host, o->n_uniq, 4, cudaMemcpyDeviceToHost, st));
  if (queue_load_host)
    SWARM_TRY(cudaMemcpyAsync(queue_load_host, o->queue_load, ctx->geo.D * 4, cudaMemcpyDeviceToHost, st));
  return SWARM_OK;
}

// Waits for the word the publish kernel raises; gives up after ~50 ms (a failed launch never raises it) and lets
// the caller fall back to the stream, which also reports the error.
bool wait_done_word(swarm_ctx* ctx) {
  volatile unsigned* done = ctx->done_h;
  const auto t0 = std::chrono::steady_clock::now();
  for (;;) {
    for (int i = 0; i < 2048; ++i)
      if (*done != 0u) {
        std::atomic_thread_fence(std::memory_order_acquire);
        return true;
      }
    if (std::chrono::steady_clock::now() - t0 > std::chrono::milliseconds(50)) return false;
  }
}

// The arguments a captured host step depends on; a replay is valid only while none of them changes.
struct HostStepKey {
  swarm_inputs in;
  swarm_outputs out;
  const void* q_host;
  void *out_host, *lse_host, *n_uniq_host, *queue_load_host;
  void* stream;
  int user_splits;
};
}  // namespace

static_assert(sizeof(HostStepKey) <= 256, "host_key too small");

int32_t swarm_build_medoid_index(swarm_ctx* ctx, const swarm_inputs* in, const int32_t* medoid_page,
                                 void* medoid_ksum_out, int32_t* cluster_ctx_len_out, void* stream) {
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (in == nullptr || bad(in->ksum) || bad(in->page_base) || bad(in->cluster_base) || bad(medoid_page) ||
      bad(medoid_ksum_out) || bad(cluster_ctx_len_out))
    return SWARM_ERR_INVALID_ARG;
  SWARM_TRY(launch_cluster_len(ctx->geo, in->cluster_base, cluster_ctx_len_out, static_cast<cudaStream_t>(stream)));
  SWARM_TRY(launch_medoid_rows(ctx->geo, static_cast<const uint16_t*>(in->ksum), in->page_base, in->cluster_base,
                               medoid_page, static_cast<uint16_t*>(medoid_ksum_out),
                               ws_ptr<uint32_t>(ctx, ctx->lay.status), static_cast<cudaStream_t>(stream)));
  return SWARM_OK;
}

int32_t swarm_step_medoid(swarm_ctx* ctx, const swarm_inputs* in, const swarm_medoid_index* idx,
                          const swarm_outputs* o, void* stream) {
  SWARM_RANGE("swarm_step_medoid");
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (in == nullptr || bad(in->q) || !resolve_inputs_ok(in) || !pool_inputs_ok(in) || idx == nullptr ||
      bad(idx->medoid_ksum) || bad(idx->cluster_page_ptr) || bad(idx->cluster_pages) || bad(idx->cluster_ctx_len) ||
      o == nullptr || bad(o->sel) ||
      bad(o->n_sel) || bad(o->uniq) || bad(o->queue_of) || bad(o->n_uniq) || bad(o->queue_load) || bad(o->out) ||
      bad(o->lse) || (o->scores && !aligned16(o->scores)) || o->k_out != nullptr || o->v_out != nullptr ||
      o->n_tok != nullptr || idx->top_k_clusters < 1 || idx->n_member_entries < 0 || idx->max_clusters_per_req < 1 ||
      idx->max_clusters_per_req > ctx->geo.Pmax ||
      (idx->entry_replica_mask != nullptr && (!aligned16(idx->entry_replica_mask) || ctx->geo.Cmax < ctx->geo.n_pool_pages)))
    return SWARM_ERR_INVALID_ARG;
  if (selmap_pitch_bytes(ctx->geo.Pmax) > kMaxExpandRowBytes ||
      (int64_t)ctx->geo.B * ctx->geo.Hq * idx->top_k_clusters >= (int64_t(1) << 31))
    return SWARM_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* status = ws_ptr<uint32_t>(ctx, ctx->lay.status);
  float* sc = o->scores ? o->scores : ws_ptr<float>(ctx, ctx->lay.scores);
  const int32_t* len_c = idx->cluster_ctx_len;             // clusters of each request x page size

  // the page kernels, run over the index: one "page" per cluster, requests laid out like cluster_base
  Geometry gc = ctx->geo;
  gc.Pmax = idx->max_clusters_per_req;
  gc.k = idx->top_k_clusters;
  gc.W = 0;
  gc.n_pool_pages = ctx->geo.Cmax;
  TopkLinks links;
  links.tk = step_tickets(ctx, gc, false);
  links.req_base = in->cluster_base;
  SWARM_TRY(launch_page_score(gc, static_cast<const uint16_t*>(in->q), static_cast<const uint16_t*>(idx->medoid_ksum),
                              in->cluster_base, len_c, sc, status, st, links.tk.ready, reserved_sms(ctx, gc, false)));
  SWARM_TRY(launch_topk(gc, sc, len_c, o->sel, o->n_sel, status, st, true, links));
  // selected clusters -> page bitmaps per head (for attention) and cluster flags (for the resolve kernel)
  SWARM_TRY(launch_expand_clusters(ctx->geo, idx->top_k_clusters, o->sel, o->n_sel, in->cluster_base,
                                   idx->cluster_page_ptr, idx->cluster_pages, in->ctx_len,
                                   ws_ptr<uint8_t>(ctx, ctx->lay.selmap), ws_ptr<uint8_t>(ctx, ctx->lay.flags), status, st,
                                   true, idx->entry_replica_mask != nullptr ? in->page_base : nullptr,
                                   idx->n_member_entries, in->page_base, in->page2cluster));
  AttnArgs a = paged_args(ctx, in, o->out, o->lse);
  a.n_splits = pick_splits(ctx, true, /*fused=*/true);
  a.n_more = pick_more(ctx, true, a.n_splits, /*fused=*/true);
  ResolveArgs rs = step_resolve_args(ctx, in, nullptr, o->n_sel, o->uniq, o->queue_of, o->n_uniq, o->queue_load);
  if (idx->entry_replica_mask != nullptr) {
    // entry-level scheduling: the units are the pool pages, every one of weight 1, each with its own replica set
    rs.cluster_base = in->page_base;
    rs.replica_mask = idx->entry_replica_mask;
    rs.cluster_size = nullptr;
    rs.geo.flags |= SWARM_UNIT_LOAD;
    rs.has_cache = false;
  }
  SWARM_TRY(launch_attention(ctx->geo, a, status, st, /*overlap=*/true, &rs));
  return SWARM_OK;
}

int32_t swarm_step_host(swarm_ctx* ctx, const swarm_inputs* in, const swarm_outputs* o, const void* q_host,
                        float* out_host, float* lse_host, int32_t* n_uniq_host, int32_t* queue_load_host,
                        void* stream) {
  SWARM_RANGE("swarm_step_host");
  int32_t rc = need_ws(ctx);
  if (rc != SWARM_OK) return rc;
  if (in == nullptr || o == nullptr || q_host == nullptr) return SWARM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // A step is seven small operations; issued one by one their launch cost exceeds their run time.  The
  // first call with a given set of pointers records them into a CUDA graph, later calls replay it.
  HostStepKey key;
  std::memset(&key, 0, sizeof key);
  key.in = *in;
  key.in.q = nullptr;                                     // ignored by this entry point
  key.out = *o;
  key.q_host = q_host;
  key.out_host = out_host; key.lse_host = lse_host; key.n_uniq_host = n_uniq_host; key.queue_load_host = queue_load_host;
  key.stream = stream;
  key.user_splits = ctx->user_splits;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  const bool can_capture = ctx->host_graph_ok && st != nullptr &&
                           cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
  if (can_capture) {
    if (ctx->host_graph == nullptr || std::memcmp(&key, ctx->host_key, sizeof key) != 0) {
      if (ctx->host_graph != nullptr) { cudaGraphExecDestroy(ctx->host_graph); ctx->host_graph = nullptr; }
      cudaGraph_t graph = nullptr;
      if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        rc = enqueue_host_step(ctx, in, o, q_host, out_host, lse_host, n_uniq_host, queue_load_host, st,
                               &ctx->host_graph_signals);
        const cudaError_t e = cudaStreamEndCapture(st, &graph);
        if (rc == SWARM_OK && e == cudaSuccess && graph != nullptr &&
            cudaGraphInstantiate(&ctx->host_graph, graph, 0) == cudaSuccess) {
          std::memcpy(ctx->host_key, &key, sizeof key);
        } else {
          ctx->host_graph = nullptr;
          ctx->host_graph_ok = false;                     // e.g. pageable host memory: use plain launches from now on
          cudaGetLastError();
        }
        if (graph != nullptr) cudaGraphDestroy(graph);
        if (rc != SWARM_OK) return rc;
      } else {
        ctx->host_graph_ok = false;
        cudaGetLastError();
      }
    }
    if (ctx->host_graph != nullptr) {
      // The results land in host memory through the publish kernel, which raises a word there when all of them
      // are visible: waiting on that word returns a few microseconds before the stream reports completion.
      if (ctx->host_graph_signals) *static_cast<volatile unsigned*>(ctx->done_h) = 0u;
      SWARM_TRY(cudaGraphLaunch(ctx->host_graph, st));
      if (ctx->host_graph_signals && wait_done_word(ctx)) return SWARM_OK;
      SWARM_TRY(cudaStreamSynchronize(st));
      return SWARM_OK;
    }
  }
  bool signals = false;
  if (ctx->done_h != nullptr) *static_cast<volatile unsigned*>(ctx->done_h) = 0u;
  rc = enqueue_host_step(ctx, in, o, q_host, out_host, lse_host, n_uniq_host, queue_load_host, st, &signals);
  if (rc != SWARM_OK) return rc;
  if (signals && cap == cudaStreamCaptureStatusNone && wait_done_word(ctx)) return SWARM_OK;
  SWARM_TRY(cudaStreamSynchronize(st));
  return SWARM_OK;
}

}  // extern "C"
