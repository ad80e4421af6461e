// Internal declarations shared by the kernels and the C-ABI layer of libswarm (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "swarm.h"

namespace swarm {

constexpr int kHeadDim = 128;

// Where each scratch region sits inside the caller-provided workspace (byte offsets, 256-aligned).
struct WorkspaceLayout {
  int64_t status;        // uint32 status word; +64: ticket counter of the resolve kernel; +96: of the publish kernel (all start at 0);
                         // +256: 1 KiB of time stamps in development builds
  int64_t scores;        // f32 [B][Hq][Pmax]          (used when the caller passes no scores buffer)
  int64_t n_tok;         // i32 [B][Hq]                (used when the caller passes no n_tok buffer)
  int64_t q_stage;       // bf16 [B][Hq][d]            (swarm_step_host)
  int64_t flags;         // u8  2 x [max_clusters_total] cluster dedup flags (zero between calls); the second array
  int64_t flags_alt;     //     starts flags_alt bytes after the first and is used by the overlapped tail only
  int64_t part_acc;      // f32 [B*Hq][max_splits][d]  split-K partial outputs
  int64_t part_ml;       // f32 [B*Hq][max_splits][2]  split-K partial (max, sum)
  int64_t items;         // uint4 [max_clusters_total]  (replica mask, weight, output slot, -) of the serial pass
  int64_t selmap;        // u8  [B*Hq][pitch]           per-head bitmap of the selected pages
  int64_t tickets;       // u32 [B*Hq]                 arrival counters of the split merge (zero between calls)
  int64_t ctl;           // u32 [64]                   control words of the step's hand-offs, see StepTickets (zero at set-up)
  int64_t ready;         // u32 [B][head pairs]        score units complete (scorer -> selection; zero between steps)
  int64_t sel_ready;     // u32 [B][Hkv]               heads selected (selection -> attention; zero between steps)
  int64_t selmap_ll;     // uint2 [B*Hq][pitch/4]      the page bitmaps as self-validating {word, epoch} pairs (zero at set-up)
  int64_t scores_ll;     // uint2 [B*Hq][Pmax]         the scores as {score, epoch} pairs (zero at set-up); only for shapes of
                         //                            at most kLlScoreLists lists, else empty
  int64_t total;
  // 256 canary bytes sit in front of every region and behind the last one (kCanaryByte, written by
  // swarm_set_workspace; swarm_check_workspace reports the ones that no longer hold it)
  int64_t guard[20];
  int n_guard;
};
constexpr int kGuardBytes = 256;
constexpr int kCanaryByte = 0xA5;

// Hand-offs between the kernels of a step.  The kernels are chained by programmatic dependent launch, so a
// kernel is resident before its predecessor has finished; instead of waiting for the whole predecessor it
// waits (bounded) for the counter of exactly the data it reads:
//   ready[b][hp]      the scorer adds 1 for every (16-page tile, KV head) of request b and KV-head pair hp whose
//                     scores are stored; the selection of a head starts when its pair has all of them
//   sel_ready[b][kv]  a selection CTA adds 1 when its head's page bitmap is stored; the attention CTAs of (b, kv)
//                     start when all g heads have arrived.  For attention grids of one wave the bitmaps travel
//                     as self-validating words instead (selmap_ll, see ll_word_store) and this ticket is unused
// Every wait is on a kernel launched earlier in the same stream whose CTAs are all resident (that is the
// condition for the dependent launch), so no waiter can hold a resource the producer needs.  The counters are
// set back to zero by the last CTA that needs them (ctl words count those).  A null pointer switches a
// hand-off off: the consumer then waits for its whole predecessor (griddepcontrol.wait).
struct StepTickets {
  unsigned* ready;
  unsigned* sel_ready;
  unsigned* ctl;   // [0] selection CTAs finished; [1] attention CTAs past their wait; [2] steps whose cluster marks
                   // are complete; [3] steps whose cluster resolution has finished ([2], [3]: overlapped tail only);
                   // [4] steps whose attention kernel has finished: the epoch of the self-validating bitmaps
  uint2* selmap_ll;  // with sel_ready: the bitmaps travel as {word, epoch + 1} pairs instead (see ll_word_store)
  uint2* scores_ll;  // with selmap_ll: so do the scores, [B*Hq][Pmax] pairs; the selection then waits for no ticket
};
constexpr int kLlScoreLists = 128;                          // shapes with more lists keep the scorer's tickets
constexpr int kCtlTopkDone = 0, kCtlAttnPast = 1, kCtlMarked = 2, kCtlResolved = 3, kCtlEpoch = 4;
constexpr unsigned kTicketWaitLimit = 1u << 22;            // polls, ~100 ns apart
__host__ __device__ inline int head_pairs(int Hkv) { return (Hkv + 1) / 2; }

// Bounded wait until the counter *p has reached `target` (acquire; the difference is taken modulo 2^32, so
// counters that only ever grow may wrap); false when the limit ran out.
__device__ __forceinline__ bool wait_at_least(const unsigned* p, unsigned target) {
  for (unsigned polls = 0; polls < kTicketWaitLimit; ++polls) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    if ((int)(v - target) >= 0) return true;
    __nanosleep(64);
  }
  return false;
}
// Release / acquire-release updates of a counter at GPU scope.  Called by one thread after a warp- or CTA-wide
// barrier: the barrier orders the other threads' stores before this thread's release, which is cumulative over
// them.  (A plain __threadfence() is the sequentially consistent fence, which costs far more.)
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_relaxed_add(unsigned* p, unsigned v) {   // no result: nothing waits for it
  asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned atom_acq_rel_add(unsigned* p, unsigned v) {
  unsigned prev;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(prev) : "l"(p), "r"(v) : "memory");
  return prev;
}
__device__ __forceinline__ void st_release(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ bool wait_zero(const unsigned* p) {
  for (unsigned polls = 0; polls < kTicketWaitLimit; ++polls) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    if (v == 0u) return true;
    __nanosleep(64);
  }
  return false;
}

constexpr int kMaxSplits = 64;

// Self-validating words.  Where a CTA that is already waiting is handed a few hundred bytes, a release / acquire
// pair costs two more trips to L2 than the data: the release waits for the stores to be acknowledged, the
// consumer polls the flag and only then fetches what it covers.  Instead every 32-bit word travels with its own
// evidence in one 8-byte store (single-copy atomic): {word, flag}, the flag being the count of finished steps + 1
// (never the 0 of fresh memory, never a value an earlier step wrote).  The consumer reads the pair with a volatile
// load until the flag matches; no ordering between words is needed.  (Not ld.global.cg: on this part a repeated
// .cg load of a line was served the first, stale answer about a million times in a row.)
__device__ __forceinline__ void ll_word_store(uint2* p, uint32_t word, uint32_t flag) {
  asm volatile("st.global.cg.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(word), "r"(flag) : "memory");
}
__device__ __forceinline__ uint2 ll_word_load(const uint2* p) {
  uint2 v;
  asm volatile("ld.volatile.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  return v;
}
constexpr unsigned kLlWaitLimit = 1u << 20;                // re-reads, each a trip to L2 (~0.7 us)
// 0 that the compiler cannot tell from a value depending on x: added to an operand, it makes that instruction
// wait for the load that produced x.
__device__ __forceinline__ unsigned zero_after(unsigned x) {
  unsigned z;
  asm volatile("and.b32 %0, %1, 0;" : "=r"(z) : "r"(x));
  return z;
}

// Row pitch of the per-head selection bitmap: one bit per page, rounded up to 16 bytes.
__host__ __device__ inline int selmap_pitch_bytes(int Pmax) { return ((Pmax + 7) / 8 + 15) & ~15; }

struct Geometry {   // plain copy of the shape in kernel-friendly form
  int B, Hq, Hkv, g, S, k, D, Pmax, Cmax;
  int W;                // local window in pages: the last W pages of a request are always selected
  unsigned flags;
  long long n_pool_pages;
  int scorer;           // SWARM_SCORER_*: which kernel scores the pages
};

// ---- one-time per-device kernel attribute set-up (dynamic shared-memory limits) ---------------
cudaError_t configure_score();
int sm_count();         // SMs of the device current at configure_score() (148 on B200)
cudaError_t configure_topk();
int topk_threads(int Pmax);   // threads of the selection CTA launched for lists of up to Pmax pages
cudaError_t configure_resolve();
cudaError_t configure_attention();
cudaError_t configure_medoid();

// ---- kernel launchers (each returns cudaGetLastError() after the launch) ----------------------
cudaError_t launch_build_summaries(const Geometry& geo, const uint16_t* kv_pool, const int64_t* page_base,
                                   const int32_t* ctx_len, uint16_t* ksum, uint32_t* status, cudaStream_t st);
bool score_streams(const Geometry& geo);          // the shape allows the streaming tensor-core scorer
bool score_raises_tickets(const Geometry& geo);   // ... and it is the one that will run: it counts its progress on `ready`
// `ready` (StepTickets::ready, may be null) is raised by the streaming scorer only; `reserve_sms` SMs are left
// free for the selection CTAs that wait on it.  `scores_ll` with `ctl` (StepTickets, may be null): the streaming
// scorer also stores every score as a {score, epoch + 1} pair there.  `index_early`: the streaming scorer's CTAs ask
// for their first blocks of `ksum` -- located through ctx_len and page_base -- before they wait for what precedes
// the kernel in the stream (the caller vouches that it writes none of the three).
cudaError_t launch_page_score(const Geometry& geo, const uint16_t* q, const uint16_t* ksum,
                              const int64_t* page_base, const int32_t* ctx_len, float* scores, uint32_t* status,
                              cudaStream_t st, unsigned* ready = nullptr, int reserve_sms = 0, uint2* scores_ll = nullptr,
                              const unsigned* ctl = nullptr, bool index_early = false);
// `overlap`: launch with programmatic dependent launch after the previous kernel of the stream.
// `selmap` (optional): per (request, head) bitmap of the selected pages, rows of selmap_pitch_bytes(Pmax).
// `flags` with the three tables (optional): also mark the selected pages' clusters (see launch_resolve).
// `links`: how the kernel is tied to its neighbours (all zero: it waits for the whole previous kernel and
// announces nothing).  tk.ready needs req_base (what the scorer was given as page_base).
struct TopkLinks {
  StepTickets tk{nullptr, nullptr, nullptr, nullptr, nullptr};
  const int64_t* req_base = nullptr;
  long long flags_alt = 0;      // bytes between the two cluster-flag arrays of the overlapped tail, else 0
};
cudaError_t launch_topk(const Geometry& geo, const float* scores, const int32_t* ctx_len, int32_t* sel,
                        int32_t* n_sel, uint32_t* status, cudaStream_t st, bool overlap, const TopkLinks& links,
                        uint8_t* selmap = nullptr, const int64_t* page_base = nullptr,
                        const int32_t* page2cluster = nullptr, const int64_t* cluster_base = nullptr,
                        uint8_t* flags = nullptr, const uint32_t* replica_mask = nullptr,
                        const uint16_t* cluster_size = nullptr);
// Everything the cluster-resolution body needs (see resolve_body.cuh).  sel == nullptr: the flags are already
// set (by the selection or the expansion kernel) and a single CTA runs the tail.
// Host-step extension of the fused attention + resolution kernel: the step's small results are also stored
// into host memory the device can address, and the last of `arrivals` finishing parts (one per query head,
// one for the resolution CTA) raises *done_h after a system-wide fence.  All null / zero when unused.
struct HostMirror {
  float* out_h;
  float* lse_h;
  int32_t* n_uniq_h;
  int32_t* queue_load_h;
  unsigned* ticket;        // arrival counter in the workspace; zero between launches
  unsigned* done_h;
  unsigned arrivals;
};

struct ResolveArgs {
  Geometry geo;
  swarm_cache cache;
  bool has_cache;
  const int32_t* sel;
  const int32_t* n_sel;
  const int64_t* page_base;
  const int32_t* page2cluster;
  const int64_t* cluster_base;
  const uint32_t* replica_mask;
  const uint16_t* cluster_size;
  uint8_t* flags;
  unsigned* ticket;
  uint4* items;
  int32_t* uniq;
  uint8_t* queue_of;
  int32_t* n_uniq;
  int32_t* queue_load;
  uint32_t* status;
  int items_cap;
  int32_t* submit_order;   // optional: submission order (indices into uniq), see resolve_body.cuh
  int32_t* submit_info;    // optional: [0] batches, [1] clusters submitted
  HostMirror host{};
  // Overlapped tail (the kernel runs beside the NEXT step's scoring and selection): the control words of
  // StepTickets, and the distance between the two flag arrays that alternate steps mark.  Null / 0 otherwise.
  unsigned* tail_ctl = nullptr;
  long long flags_alt = 0;
};
ResolveArgs make_resolve_args(const Geometry& geo, const int32_t* sel, const int32_t* n_sel, const int64_t* page_base,
                              const int32_t* page2cluster, const int64_t* cluster_base, const uint32_t* replica_mask,
                              const uint16_t* cluster_size, uint8_t* flags_ws, unsigned* ticket, uint4* items,
                              int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq, int32_t* queue_load, uint32_t* status,
                              const swarm_cache* cache = nullptr, int32_t* submit_order = nullptr,
                              int32_t* submit_info = nullptr);
cudaError_t launch_resolve(const ResolveArgs& r, cudaStream_t st, bool overlap);
cudaError_t launch_gather(const Geometry& geo, const uint16_t* kv_pool, const int32_t* sel, const int32_t* n_sel,
                          const int64_t* page_base, const int32_t* ctx_len, uint16_t* k_out, uint16_t* v_out,
                          int32_t* n_tok, uint32_t* status, cudaStream_t st);
// The step's small results written by a kernel into device-addressable host memory (any *_h may be null).
cudaError_t launch_publish(const Geometry& geo, const float* out, const float* lse, const int32_t* n_uniq,
                           const int32_t* queue_load, float* out_h, float* lse_h, int32_t* n_uniq_h,
                           int32_t* queue_load_h, cudaStream_t st);
// `bytes` (a multiple of 16) from device-addressable host memory into device memory, by a kernel.
cudaError_t launch_fetch(const void* src_h, void* dst, long long bytes, cudaStream_t st);
// Attention over contiguous gathered buffers (pool == nullptr) or straight from the pool (k_g == nullptr).
struct AttnArgs {
  const uint16_t* q;
  const uint16_t* k_g;
  const uint16_t* v_g;
  const int32_t* n_tok;
  const uint16_t* kv_pool;
  const uint8_t* selmap;   // paged mode: per (request, head) bitmap of selected pages, rows of selmap_pitch bytes
                           // (with tk.selmap_ll: the same words as {word, epoch} pairs there instead)
  int selmap_pitch;
  const int64_t* page_base;
  const int32_t* ctx_len;
  float* part_acc;
  float* part_ml;
  unsigned* tickets;   // [B*Hq] arrival counters of the split merge; zero between launches
  float* out;
  float* lse;
  int n_splits;
  int n_more;          // the last n_more groups are cut into n_splits + 1 ranges (a grid of whole waves), the others into n_splits
  bool release_early = false;   // inside a step: the CTAs let the next kernel's CTAs become resident once they have read all their pages
  HostMirror host{};
  StepTickets tk{nullptr, nullptr, nullptr, nullptr, nullptr};   // paged mode inside a step: wait per KV head for the selection (sel_ready, ctl)
};
// `fused_resolve` (paged mode only): one extra CTA of the grid runs cluster resolution with these arguments.
cudaError_t launch_attention(const Geometry& geo, const AttnArgs& a, uint32_t* status, cudaStream_t st,
                             bool overlap = false, const ResolveArgs* fused_resolve = nullptr);
// (request, head group) units the attention grid is split over: one per KV head (and per 8 heads of the
// group) in paged mode, one per query head for gathered buffers.
int attention_groups(const Geometry& geo, bool paged);
cudaError_t launch_selmap_from_sel(const Geometry& geo, const int32_t* sel, const int32_t* n_sel, uint8_t* selmap,
                                   cudaStream_t st);

// Medoid index (cluster-granular selection): see medoid.cu.
constexpr int kMaxExpandRowBytes = 160 * 1024;            // longest per-head page bitmap the expansion assembles in shared memory
cudaError_t launch_medoid_rows(const Geometry& geo, const uint16_t* ksum, const int64_t* page_base,
                               const int64_t* cluster_base, const int32_t* medoid_page, uint16_t* medoid_ksum,
                               uint32_t* status, cudaStream_t st);
cudaError_t launch_cluster_len(const Geometry& geo, const int64_t* cluster_base, int32_t* len, cudaStream_t st);
cudaError_t launch_expand_clusters(const Geometry& geo, int k_c, const int32_t* sel_c, const int32_t* n_sel_c,
                                   const int64_t* cluster_base, const int64_t* cluster_page_ptr,
                                   const int32_t* cluster_pages, const int32_t* ctx_len, uint8_t* selmap, uint8_t* flags,
                                   uint32_t* status, cudaStream_t st, bool overlap, const int64_t* entry_base,
                                   long long n_member_entries, const int64_t* page_base, const int32_t* page2cluster);

// Algorithm 1 (offline co-activation clustering): see cluster.cu.
long long build_clusters_workspace_bytes(int n);
cudaError_t launch_build_clusters(const float* dist, int n, float tau, void* workspace, int32_t* rho, int32_t* ptr,
                                  int32_t* members, long long members_cap, int32_t* medoid, int32_t* n_clusters,
                                  int32_t* dev_status, cudaStream_t st);

// Admission of clusters to the fast tier by Eq. 6 score (cluster.cu).
long long cache_admit_workspace_bytes(int n);
cudaError_t launch_cache_admit(const float* score, const uint16_t* size, int n, long long capacity, void* workspace,
                               uint8_t* resident, int32_t* info, cudaStream_t st);

// ---- device helpers ---------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// One part of a host step is complete.  Called by one thread of the CTA after a CTA-wide barrier that every
// thread reached past its stores: the barrier orders those before this thread's system-wide fence, which is
// cumulative over them.
__device__ __forceinline__ void host_arrive(const HostMirror& h) {
  __threadfence_system();
  const unsigned arrived = atomicAdd(h.ticket, 1u);
  if (arrived == h.arrivals - 1u) {
    *h.ticket = 0u;                                         // ready for the next launch
    __threadfence_system();
    *reinterpret_cast<volatile unsigned*>(h.done_h) = 1u;
  }
}

__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ int pages_of(int ctx_len, int S) { return (ctx_len + S - 1) / S; }

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// start while its predecessor in the stream is still running; it must call pdl_wait() before it
// touches anything the predecessor writes.  Both are no-ops for ordinary launches.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

// Launches `kernel` so that it may overlap the tail of the previous kernel in `st` (see pdl_wait).
template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool overlap,
                       Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Development-only time stamps (compiled in with -DSWARM_TRACE): thread 0 of one CTA records %globaltimer (ns)
// at up to 16 numbered points of a kernel into the workspace's trace block (1 KiB behind the status block:
// 16 slots per source file, SWARM_TRACE_FILE selects the group), where a developer reads them back from the
// workspace tensor.  Absent from normal builds.
#ifdef SWARM_TRACE
__device__ __forceinline__ unsigned long long trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
#ifndef SWARM_TRACE_FILE
#define SWARM_TRACE_FILE 0
#endif
#if SWARM_TRACE_FILE == 0 && defined(SWARM_TRACE_CTA_F0)
#define SWARM_TRACE_CTA SWARM_TRACE_CTA_F0
#elif SWARM_TRACE_FILE == 1 && defined(SWARM_TRACE_CTA_F1)
#define SWARM_TRACE_CTA SWARM_TRACE_CTA_F1
#elif SWARM_TRACE_FILE == 2 && defined(SWARM_TRACE_CTA_F2)
#define SWARM_TRACE_CTA SWARM_TRACE_CTA_F2
#endif
#ifndef SWARM_TRACE_CTA
#define SWARM_TRACE_CTA 0
#endif
#define SWARM_STAMP_RAW(status, i, any_cta)                                                          \
  do {                                                                                               \
    if (threadIdx.x == 0 && ((any_cta) || (blockIdx.x == (SWARM_TRACE_CTA) && blockIdx.y == 0 && blockIdx.z == 0)))  \
      reinterpret_cast<unsigned long long*>(status)[32 + 16 * (SWARM_TRACE_FILE) + (i)] = trace_now(); \
  } while (0)
#endif
#if defined(SWARM_TRACE) && SWARM_TRACE == 1      // phases inside one kernel
#define SWARM_STAMP(status, i) SWARM_STAMP_RAW(status, i, false)
#define SWARM_STAMP_ANY_CTA(status, i) SWARM_STAMP_RAW(status, i, true)
#else
#define SWARM_STAMP(status, i) do { } while (0)
#define SWARM_STAMP_ANY_CTA(status, i) do { } while (0)
#endif
#if defined(SWARM_TRACE) && SWARM_TRACE == 2      // entry of the first CTA / exit of the last CTA of kernel k
#define SWARM_KERNEL_BEGIN(status, k) SWARM_STAMP_RAW(status, 2 * (k), false)
#define SWARM_KERNEL_END(status, k) SWARM_STAMP_RAW(status, 2 * (k) + 1, true)
#else
#define SWARM_KERNEL_BEGIN(status, k) do { } while (0)
#define SWARM_KERNEL_END(status, k) do { } while (0)
#endif

}  // namespace swarm
