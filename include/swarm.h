/* swarm.h -- C ABI of the B200 (sm_100a) KVCache retrieval hot path.
 *
 * One decode step of one layer, for a batch of requests whose KV cache lives in a paged
 * pool in device memory:
 *   (1) score every page of every request against the query (page upper bound over per-page
 *       min/max key summaries),
 *   (2) keep the top_k pages per query head,
 *   (3) map the selected pages to co-activation clusters, merge duplicates and route every
 *       cluster to the least loaded of the queues that hold a replica of it,
 *   (4) gather the selected pages' K/V and run single-row attention over them.
 *
 * Conventions that hold for every entry point unless stated otherwise:
 *   - Every data pointer is a DEVICE pointer owned by the caller, 16-byte aligned.  The library
 *     allocates no device memory, frees nothing of the caller's and never synchronises the host
 *     (exceptions are named below: swarm_device_status and swarm_step_host).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work is
 *     enqueued on it and the call returns at once.  A ctx must be used from one stream at a time.
 *   - Return value: SWARM_OK or an error code from host-side validation / launch.  Nothing is
 *     enqueued when an error is returned.
 *   - Faults seen on the device (table entry out of range, cluster without replica) never trap:
 *     they set bits in a status word (swarm_device_status), the offending item is skipped or gets
 *     a sentinel, and the kernel finishes.
 *   - bf16 tensors are raw 16-bit words.  Layouts are row-major with the last index fastest.
 *   - head_dim is 128; page_size is 16 or 32 tokens; 1 <= n_queues <= 32; n_q_heads is a multiple
 *     of n_kv_heads and query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - Inputs must be finite (no NaN / Inf).
 */
#ifndef SWARM_H_
#define SWARM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes (host side) ---------------------------------------------------------- */
#define SWARM_OK 0
#define SWARM_ERR_INVALID_ARG 1         /* null / misaligned pointer, dimension out of range        */
#define SWARM_ERR_UNSUPPORTED 2         /* valid but not implemented (head_dim != 128, ...)        */
#define SWARM_ERR_WORKSPACE_TOO_SMALL 3 /* swarm_set_workspace not called or too few bytes         */
#define SWARM_ERR_CUDA 4                /* a CUDA call failed; see swarm_last_cuda_error           */
#define SWARM_ERR_STATIC_SCRATCH_TOO_SMALL 5 /* problem exceeds the built-in scratch of swarm_sparse_attn_static */

/* ---- bits of the device status word ---------------------------------------------------- */
#define SWARM_DEV_BAD_PAGE 1u           /* a selected page id lies outside its request             */
#define SWARM_DEV_BAD_CLUSTER 2u        /* page2cluster entry outside the request's cluster range  */
#define SWARM_DEV_BAD_REPLICA 4u        /* replica mask is 0 or names a queue >= n_queues          */
#define SWARM_DEV_BAD_LENGTH 8u         /* ctx_len < 1 or more pages than the request owns         */
#define SWARM_DEV_TIMEOUT 16u           /* a bounded wait expired (a copy, or a hand-off between kernels) */

/* ---- flags in swarm_shape.flags --------------------------------------------------------- */
#define SWARM_ORDER_BY_ID 1u            /* schedule clusters by id only (default: by number of
                                           replicas ascending, then id; Sec. 5.1)                  */
#define SWARM_UNIT_LOAD 2u              /* a cluster adds 1 to its queue (default: its page count) */

typedef struct swarm_ctx swarm_ctx;

/* Problem shape; fixed for the lifetime of a ctx. */
typedef struct swarm_shape {
  int32_t batch;              /* B  requests                                                     */
  int32_t n_q_heads;          /* Hq                                                              */
  int32_t n_kv_heads;         /* Hkv                                                             */
  int32_t head_dim;           /* d  (128)                                                        */
  int32_t page_size;          /* S  tokens per page (16 or 32)                                   */
  int32_t top_k;              /* k  pages kept per query head                                    */
  int32_t n_queues;           /* D  simulated SSD queues                                         */
  int32_t max_pages_per_req;  /* Pmax: upper bound on ceil(ctx_len[b] / S); row pitch of scores  */
  int32_t max_clusters_total; /* upper bound on cluster_base[B]; capacity of uniq / queue_of     */
  uint32_t flags;
  int64_t n_pool_pages;       /* pages in the pool (page_base[B] <= n_pool_pages)                */
  int32_t local_window_pages; /* W: the last W pages of every request are always selected and    */
                              /* take W of the k places (local window of Sec. 4.2, Tier 1 (2));  */
                              /* 0 <= W <= top_k; 0 = plain top-k                                */
  int32_t reserved;           /* must be 0                                                       */
} swarm_shape;

/* Read-only device-resident inputs of a step. */
typedef struct swarm_inputs {
  const void* q;                        /* bf16 [B][Hq][d]                                       */
  const void* ksum;                     /* bf16 [n_pool_pages][Hkv][2][d]      0 = min, 1 = max  */
  const void* kv_pool;                  /* bf16 [n_pool_pages][Hkv][2][S][d]   0 = K,   1 = V    */
  const int64_t* page_base;             /* [B+1] request b owns pool pages [base[b], base[b+1])  */
  const int32_t* ctx_len;               /* [B] tokens; 1 <= len <= S * (base[b+1] - base[b])     */
  const int32_t* page2cluster;          /* [n_pool_pages] cluster id local to the page's request */
  const int64_t* cluster_base;          /* [B+1] global cluster id = cluster_base[b] + local id  */
  const uint32_t* cluster_replica_mask; /* [n_clusters] bit j set <=> a replica sits on queue j  */
  const uint16_t* cluster_size;         /* [n_clusters] pages in the cluster                     */
} swarm_inputs;

/* Device-resident outputs of a step.  Pointers marked "optional" may be NULL. */
typedef struct swarm_outputs {
  float* scores;       /* optional, f32 [B][Hq][Pmax]; entries p >= pages of the request untouched */
  int32_t* sel;        /* [B][Hq][k] selected page ids (request-local), ascending, -1 padded       */
  int32_t* n_sel;      /* [B][Hq]    min(k, pages of the request)                                  */
  int32_t* uniq;       /* [max_clusters_total] global ids of the clusters to fetch, ascending      */
  uint8_t* queue_of;   /* [max_clusters_total] queue serving uniq[i]; 0xFF if it has no replica    */
  int32_t* n_uniq;     /* [1]                                                                      */
  int32_t* queue_load; /* [D] load routed to each queue this step                                  */
  void* k_out;         /* optional, bf16 [B][Hq][k*S][d] gathered keys, zero beyond n_tok rows     */
  void* v_out;         /* optional, bf16 [B][Hq][k*S][d] gathered values (given iff k_out is)      */
  int32_t* n_tok;      /* optional, [B][Hq] valid gathered tokens (only together with k_out)       */
  float* out;          /* f32 [B][Hq][d] attention output                                          */
  float* lse;          /* f32 [B][Hq] natural-log sum of exp of the scaled logits                  */
} swarm_outputs;

/* Optional DRAM-tier cache state (Sec. 4.2 "hot clusters", Sec. 5.2 "cache replacement").  Device pointers,
 * indexed by global cluster id.  See swarm_set_cache. */
typedef struct swarm_cache {
  const uint8_t* resident; /* [n_clusters] 1 = the cluster is held in the fast tier: activated but not fetched */
  int32_t* freq;           /* [n_clusters] activation frequency f_i, updated in place every step               */
  float* score;            /* [n_clusters] cost-effectiveness score of Eq. 6, rewritten every step; may be NULL */
  int32_t* n_hit;          /* [1] activated clusters found resident this step; may be NULL                     */
  float t_base;            /* T_base: addressing latency per fetch                                             */
  float t_transfer;        /* T_transfer: transfer cost per entry (page)                                       */
} swarm_cache;

/* Medoid index for cluster-granular selection (Sec. 4.2, Tier 1 (1): the medoid of each cluster is its index
 * entry and is scored against the query to decide whether the cluster is retrieved).  Device pointers.
 * Clusters carry their global id (cluster_base[b] + local id), as in the other cluster tables. */
typedef struct swarm_medoid_index {
  const void* medoid_ksum;          /* bf16 [max_clusters_total][Hkv][2][d]: key summary (min, max) of each cluster's */
                                    /* medoid page, written by swarm_build_medoid_index                               */
  const int64_t* cluster_page_ptr;  /* [n_clusters + 1] start of each cluster's members in cluster_pages               */
  const int32_t* cluster_pages;     /* member pages of the clusters, ids local to the request                          */
  const uint32_t* entry_replica_mask; /* NULL: the selected clusters are scheduled as units (cluster tables of the     */
                                    /* inputs).  Otherwise entry-level scheduling, the paper's exact model (Sec. 5.1    */
                                    /* with the placement of Eq. 7): [n_pool_pages] queues holding a copy of each page; */
                                    /* see swarm_step_medoid                                                            */
  const int32_t* cluster_ctx_len;   /* [B] clusters of request b x page_size (the index seen as a context of its own), */
                                    /* written by swarm_build_medoid_index                                              */
  int64_t n_member_entries;         /* length of cluster_pages: offsets in cluster_page_ptr beyond it set               */
                                    /* SWARM_DEV_BAD_CLUSTER and the cluster is skipped                                 */
  int32_t top_k_clusters;           /* k_c clusters kept per query head                                                */
  int32_t max_clusters_per_req;     /* upper bound on the clusters of one request (<= max_pages_per_req); row pitch    */
                                    /* of the cluster scores                                                           */
} swarm_medoid_index;

/* Lifetime.  swarm_create validates the shape and allocates only host memory.
 * The CUDA device current at creation must stay current for every later call with this ctx. */
int32_t swarm_create(const swarm_shape* shape, swarm_ctx** out_ctx);
int32_t swarm_destroy(swarm_ctx* ctx);

/* Scratch memory.  The caller allocates swarm_workspace_bytes(shape) bytes of device memory
 * (256-byte aligned) and hands them over; they must stay valid while the ctx is used.  The caller
 * need not initialise them: swarm_set_workspace enqueues the clearing it needs on `stream`.
 * swarm_workspace_bytes returns < 0 (minus an error code) for an invalid shape. */
int64_t swarm_workspace_bytes(const swarm_shape* shape);
int32_t swarm_set_workspace(swarm_ctx* ctx, void* device_mem, int64_t bytes, void* stream);

/* Debugging aid: the workspace regions are separated by 256 canary bytes each (one in front of every region,
 * one behind the last), written by swarm_set_workspace.  Copies them back and sets bit i of *damaged for every
 * canary i (in workspace order) that no longer holds its pattern, i.e. some kernel wrote outside its region.
 * SYNCHRONISES `stream`.  Stands in for a memory checker where none can be run. */
int32_t swarm_check_workspace(swarm_ctx* ctx, void* stream, uint32_t* damaged);

/* Attaches (or, with NULL, detaches) cache state to the ctx; the struct is copied.  While attached,
 * swarm_resolve_clusters and swarm_step compute the full Eq. 8: the clusters to fetch are the activated
 * ones minus the resident ones (only those appear in uniq / queue_of / queue_load), and the bookkeeping of
 * Sec. 5.2 runs in the same kernel: freq += 1 for every activated cluster, freq -= 1 for every resident
 * cluster that was not activated, score = freq * (t_base + size * t_transfer) / size for every cluster. */
int32_t swarm_set_cache(swarm_ctx* ctx, const swarm_cache* cache);

/* Attaches (or, with NULL, detaches) the optional output of the batched submission (Sec. 5.1: the head of
 * every SSD bucket is taken into one submission batch, then the next heads, and so on).  While attached,
 * swarm_resolve_clusters, swarm_step and swarm_step_medoid also write
 *   submit_order[j]  int32 [max_clusters_total]: index into uniq of the j-th submitted cluster.  Bucket q
 *                    holds the clusters assigned to queue q in assignment order (replica count ascending, then
 *                    position in uniq; position alone under SWARM_ORDER_BY_ID); batch r is the r-th cluster of
 *                    every bucket that has one, in queue order; batches follow one another.
 *   submit_info[0]   number of batches (the largest bucket), submit_info[1] clusters submitted (those with a
 *                    bad replica mask are left out).  submit_info may be NULL.
 * Device pointers, 16-byte aligned; the caller keeps them valid while attached. */
int32_t swarm_set_submit_order(swarm_ctx* ctx, int32_t* submit_order, int32_t* submit_info);

/* Number of key-range splits used by the attention kernels (>= 1; 0 restores the default chosen
 * from the shape).  Results do not depend on it beyond floating-point rounding. */
int32_t swarm_set_attn_splits(swarm_ctx* ctx, int32_t n_splits);

/* Overlapped tail of swarm_step (off by default).  Cluster resolution ends in a serial pass (the greedy queue
 * assignment of Sec. 5.1) whose result feeds the I/O side, not the next layer's computation.  With a tail
 * stream attached (another cudaStream_t of the same device; NULL detaches), swarm_step enqueues the
 * resolution there, ordered behind the step's selection, and `stream` itself carries only scoring, selection
 * and attention: the next swarm_step on `stream` starts as soon as this step's attention has finished, while
 * the resolution of this step may still run.  uniq / queue_of / n_uniq / queue_load (and the cache state and
 * submission order, when attached) are then complete once the TAIL stream has run the resolution:
 *   swarm_tail_join(ctx, s)   makes stream s wait for the last resolution enqueued by this ctx (no host
 *                             synchronisation).  Required before s reads those outputs, and before a stream
 *                             capture that recorded steps of this ctx is ended (a capture must join the
 *                             streams it forked).
 * sel, n_sel, out, lse, scores are complete in `stream` order as always.  The resolutions of consecutive steps
 * never overlap each other (they follow one another on the tail stream), and the step keeps two sets of dedup
 * flags so that the next step's selection may mark clusters while this step's resolution still reads its own.
 * swarm_step_begin / swarm_step_end / swarm_step_host are not affected.  Attach or detach while no step of the
 * ctx is in flight. */
int32_t swarm_set_tail_stream(swarm_ctx* ctx, void* tail_stream);
int32_t swarm_tail_join(swarm_ctx* ctx, void* stream);

/* SMs the scoring kernel leaves free for the selection kernel, whose CTAs are resident beside it and start on
 * a head as soon as its scores are complete (-1 restores the default chosen from the shape).  Tuning only:
 * results do not depend on it. */
int32_t swarm_set_select_sms(swarm_ctx* ctx, int32_t n_sms);

/* Which kernel scores the pages (stage 1).  The result is the same sum either way, within fp32 rounding.
 *   SWARM_SCORER_AUTO    the streaming tensor-core kernel whenever the shape allows it (batch <= 512 and fewer
 *                        than 2^31 pool pages), else the fp32-pipe kernel
 *   SWARM_SCORER_TENSOR  the streaming tensor-core kernel; SWARM_ERR_UNSUPPORTED if the shape does not allow it
 *   SWARM_SCORER_FP32    the fp32-pipe kernel (16-byte row loads, sign-split weights in registers) */
#define SWARM_SCORER_AUTO 0
#define SWARM_SCORER_TENSOR 1
#define SWARM_SCORER_FP32 2
int32_t swarm_set_scorer(swarm_ctx* ctx, int32_t kind);

/* Index prefetch (off by default).  The page index (inputs->ksum, located through ctx_len and page_base) does not
 * depend on the queries (Sec. 4.2, Tier 1: it is built when pages are written).  With `on` != 0 the scoring kernel
 * of swarm_step / swarm_step_begin asks for its first blocks of it as soon as its CTAs are resident, before it
 * waits for the work that precedes the step in the stream -- in a chain of steps: while the previous step's
 * attention kernel merges its partial results -- and the attention kernel of a step lets the next kernel's CTAs
 * become resident as soon as its own have read all their pages.  Everything that reads q (scoring itself,
 * selection, attention) still starts after the preceding work has completed.
 * The caller vouches that the operation enqueued directly before the step in its stream writes none of ksum,
 * ctx_len and page_base (an index update for newly written pages goes at least one operation earlier, or the
 * switch stays off).  Results do not depend on it. */
int32_t swarm_set_index_prefetch(swarm_ctx* ctx, int32_t on);

/* Index build (not part of a decode step): per page and KV head, element-wise min and max of
 * the valid tokens' keys -- the compact index the scorer reads instead of the keys themselves
 * (the role the in-memory cluster index plays in Sec. 4.2, Tier 1).
 * Reads inputs->kv_pool, page_base, ctx_len; writes ksum_out bf16 [n_pool_pages][Hkv][2][d] for
 * the pages that exist; padding tokens of a partial last page are ignored. */
int32_t swarm_build_summaries(swarm_ctx* ctx, const swarm_inputs* inputs, void* ksum_out, void* stream);

/* Stages 1-2: activation scoring and top-k selection (Sec. 2.3: relevance scores of the cached
 * entries against the query, only the highest-scoring entries are activated).
 *   score[b][h][p] = sum_i max(q[b][h][i] * kmin[p][i], q[b][h][i] * kmax[p][i])   in fp32
 *   sel[b][h][:]   = the min(k, P_b) pages of largest score, ties to the lower page id,
 *                    written in ascending page id; remaining slots -1.
 * Reads inputs->q, ksum, page_base, ctx_len.  `scores` may be NULL (kept in the workspace). */
int32_t swarm_select(swarm_ctx* ctx, const swarm_inputs* inputs, float* scores, int32_t* sel, int32_t* n_sel,
                     void* stream);

/* Stage 3: global merge of the activated clusters (Eq. 8, without the already-resident term) and
 * load-balanced bucket scheduling (Sec. 5.1).  Every selected page is mapped through page2cluster;
 * the union over all heads and requests is deduplicated; clusters are visited by (number of
 * replicas ascending, global id ascending) -- by id only under SWARM_ORDER_BY_ID -- and each goes
 * to the replica queue with the smallest load so far (lowest queue id on a tie), adding its
 * cluster_size (or 1 under SWARM_UNIT_LOAD) to that queue.
 * Reads inputs->page_base, page2cluster, cluster_base, cluster_replica_mask, cluster_size. */
int32_t swarm_resolve_clusters(swarm_ctx* ctx, const swarm_inputs* inputs, const int32_t* sel,
                               const int32_t* n_sel, int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq,
                               int32_t* queue_load, void* stream);

/* Stage 4a: copy the selected pages' K and V blocks, in `sel` order, into contiguous per-head
 * buffers (the transfer the paper performs across storage tiers, Sec. 6; here within HBM).
 * Rows beyond the valid tokens are zero.  n_tok may be NULL.
 * `sel` as swarm_select writes it: ascending page ids.  What matters is that a partial last page of a request,
 * if selected, is the LAST entry of its head (swarm_sparse_attn masks only the end of the buffer); a selection
 * that places it elsewhere sets SWARM_DEV_BAD_PAGE and that page is skipped (its slot is zero-filled). */
int32_t swarm_gather(swarm_ctx* ctx, const swarm_inputs* inputs, const int32_t* sel, const int32_t* n_sel,
                     void* k_out, void* v_out, int32_t* n_tok, void* stream);

/* Stage 4b: Eq. 1 for one query row per head over its own gathered tokens,
 *   out[b][h] = softmax_t(q . K_t / sqrt(d)) V_t  over t < n_tok[b][h],  lse = log sum exp,
 * computed as split-K partials (fp32) merged by their log-sum-exp.  k_g / v_g are
 * bf16 [B][Hq][k*S][d].  n_tok[b][h] must be in [1, k*S]: a value outside [0, k*S] sets SWARM_DEV_BAD_LENGTH
 * and is clamped to that range. */
int32_t swarm_sparse_attn(swarm_ctx* ctx, const void* q, const void* k_g, const void* v_g, const int32_t* n_tok,
                          float* out, float* lse, void* stream);

/* Stage 4 without the copy: the same attention, reading the selected pages straight from the pool
 * (what swarm_step runs).  Reads inputs->q, kv_pool, page_base, ctx_len.  Tokens beyond ctx_len in a
 * partial last page are masked.  n_sel[b][h] must be >= 1.
 * sel and n_sel may both be NULL: the selection made by the last swarm_select or swarm_step on this
 * ctx is attended (its per-head page bitmaps are kept in the workspace), without rebuilding them. */
int32_t swarm_sparse_attn_paged(swarm_ctx* ctx, const swarm_inputs* inputs, const int32_t* sel,
                                const int32_t* n_sel, float* out, float* lse, void* stream);

/* swarm_sparse_attn for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this entry point; it exists for integration reasons only.)
 *
 * Some hosts of this library may not call cudaMalloc or hand over a workspace: code running inside
 * another framework's memory-pool callback or under a fixed, fully pre-reserved memory budget, and
 * plugins loaded into a process whose allocator they do not own.  For them this variant computes
 * exactly what swarm_sparse_attn computes, takes no ctx and no workspace, and allocates nothing on
 * the host or the device: the split-K partial results live in a fixed array compiled into the
 * library (static __device__ storage, SWARM_STATIC_SCRATCH_BYTES bytes, resident on every GPU
 * that loads the library until the process exits).
 *
 *   q, k_g, v_g, n_tok, out, lse   as for swarm_sparse_attn (device pointers, 16-byte aligned);
 *                                  k_g / v_g are bf16 [batch][n_q_heads][top_k * page_size][128]
 *   batch, n_q_heads, top_k, page_size   the shape (page_size 16 or 32)
 *
 * Limit: batch * n_q_heads <= SWARM_STATIC_MAX_HEADS; larger problems are rejected with
 * SWARM_ERR_STATIC_SCRATCH_TOO_SMALL and nothing is enqueued.  The number of key-range splits is
 * chosen so that the partials fit the array.
 * Set-up: the first call on each device looks up the array's device address (with that device
 * current).  Make that first call outside any CUDA stream capture.
 * Sharing: every call on a device uses the same array, and the array keeps what the last call
 * wrote.  The partial results need no clearing (each call overwrites every slot it later reads).
 * The per-head arrival counters must be zero when a call starts: they are zero when the library is
 * loaded and the kernel sets each one back to zero after using it, so nothing has to be cleared
 * between calls.  Two calls whose kernels overlap on the GPU (different streams, or graph
 * branches) race on the array; serialise them.
 * Device-side faults: the kernel reports them like the other entry points (n_tok outside [0, top_k * page_size]
 * sets SWARM_DEV_BAD_LENGTH and is clamped; a bounded wait that runs out sets SWARM_DEV_TIMEOUT and leaves
 * out / lse of that head undefined), in a status word inside the same array.
 * swarm_sparse_attn_static_status copies that word to *bits and clears it; it SYNCHRONISES `stream` and, like
 * the entry point itself, allocates nothing. */
#define SWARM_STATIC_MAX_HEADS 2048
#define SWARM_STATIC_SCRATCH_BYTES (256 + 4096 * (128 + 2) * 4 + SWARM_STATIC_MAX_HEADS * 4)
int32_t swarm_sparse_attn_static(const void* q, const void* k_g, const void* v_g, const int32_t* n_tok,
                                 int32_t batch, int32_t n_q_heads, int32_t top_k, int32_t page_size, float* out,
                                 float* lse, void* stream);
int32_t swarm_sparse_attn_static_status(void* stream, uint32_t* bits);

/* The fused step: stages 1-4 enqueued back to back with no host round trip.  Attention reads the
 * selected pages straight from the pool; the gathered copies are written only when k_out / v_out
 * are given.  Three launches on `stream`: scoring, selection, and one kernel in which cluster resolution
 * runs as one extra CTA beside the attention CTAs (with swarm_set_tail_stream the resolution is a kernel of its own on the
 * tail stream).  The kernels are chained by programmatic dependent launch and hand their data over head by
 * head: the selection of a KV-head pair starts when that pair's scores are stored, the attention of a KV head
 * when its heads are selected.  Integer outputs equal those of the
 * four separate calls exactly; out / lse agree within rounding.  The call can be captured into a
 * CUDA graph by the caller (stream capture). */
int32_t swarm_step(swarm_ctx* ctx, const swarm_inputs* inputs, const swarm_outputs* outputs, void* stream);

/* The fused step in two halves, for a step whose query heads are spread over several ctxs (one per GPU, each
 * holding the K/V and summaries of its own KV heads and all the cluster tables): stages 1-2 are independent
 * per head, stage 3 needs the union of the activated clusters over ALL heads (Eq. 8), stage 4 is per head again.
 *   swarm_step_begin     scoring and selection (the first two launches of swarm_step): sel / n_sel (and scores)
 *                        are written, and the dedup flag of every cluster that holds a selected page is set
 *   swarm_cluster_flags  the flag array in the workspace: *flags = device pointer to max_clusters_total bytes
 *                        (0 or 1, indexed by global cluster id), *n_bytes = max_clusters_total.  Between the two
 *                        halves the caller combines the arrays of all ctxs element-wise by maximum (an all-reduce
 *                        over the GPUs, on the same stream) so that every one holds the union
 *   swarm_step_end       attention over this ctx's heads and cluster resolution of the union (the third launch);
 *                        consumes the flags (they are zero again afterwards).  With identical tables every ctx
 *                        computes the same uniq / queue_of / n_uniq / queue_load
 * begin followed by end on one ctx with nothing in between is swarm_step.  Same arguments and errors as
 * swarm_step; both halves must be given the same inputs and outputs. */
int32_t swarm_step_begin(swarm_ctx* ctx, const swarm_inputs* inputs, const swarm_outputs* outputs, void* stream);
int32_t swarm_step_end(swarm_ctx* ctx, const swarm_inputs* inputs, const swarm_outputs* outputs, void* stream);
int32_t swarm_cluster_flags(swarm_ctx* ctx, void** flags, int64_t* n_bytes);

/* Index build for swarm_step_medoid (not part of a decode step): copies, for every cluster, the key summary of
 * its medoid page medoid_page[cluster] (page id local to the request) into row `cluster` of medoid_ksum_out
 * (bf16 [max_clusters_total][Hkv][2][d]), and writes cluster_ctx_len_out [B] (int32).  Reads inputs->ksum,
 * page_base, cluster_base.  Which member is the medoid is decided offline (Algorithm 1) and is an input here. */
int32_t swarm_build_medoid_index(swarm_ctx* ctx, const swarm_inputs* inputs, const int32_t* medoid_page,
                                 void* medoid_ksum_out, int32_t* cluster_ctx_len_out, void* stream);

/* The decode step with the paper's own selector (Sec. 4.2 Tier 1 (1), Sec. 4.1): clusters, not pages, are
 * scored and retrieved.
 *   score[b][h][c] = the page upper bound of swarm_select evaluated on the medoid page of cluster c
 *   sel[b][h][:]   = the min(k_c, C_b) clusters of largest score (ties to the lower id), ascending, ids local
 *                    to the request, -1 padded; n_sel their number           (outputs->sel is [B][Hq][k_c])
 *   uniq, queue_of, n_uniq, queue_load: as in swarm_step for the union of the selected clusters
 *   out, lse: Eq. 1 of every head over ALL pages of its selected clusters (clusters are the retrieval unit)
 * outputs->scores (optional) is [B][Hq][max_clusters_per_req]; k_out, v_out and n_tok must be NULL.
 * Entry-level scheduling (index->entry_replica_mask given): the I/O set of Eq. 8 is the union of the member
 * PAGES of all selected clusters; each page is one unit of weight 1 with replica set entry_replica_mask[pool
 * page] (a page stored with several clusters has several copies).  uniq then holds pool page ids
 * (page_base[b] + page), queue_of / queue_load / the submission order refer to pages, the cluster tables of the
 * inputs and the cache state are not used by the scheduling, and the ctx must have been created with
 * max_clusters_total >= n_pool_pages (SWARM_ERR_INVALID_ARG otherwise; uniq and queue_of sized accordingly).
 * A member page outside the request sets SWARM_DEV_BAD_PAGE and is skipped.  The local window of the shape
 * (Sec. 4.2, Tier 1 (2)) applies: the last local_window_pages pages of every request join every head's set of
 * attended pages and are scheduled like the members of the selected clusters (through page2cluster, or as
 * pages under entry-level scheduling); the window does not take places from the top_k_clusters clusters.  Page bitmaps longer than 160 KiB per head (1.3 M pages) are SWARM_ERR_UNSUPPORTED. */
int32_t swarm_step_medoid(swarm_ctx* ctx, const swarm_inputs* inputs, const swarm_medoid_index* index,
                          const swarm_outputs* outputs, void* stream);

/* Which clusters the fast tier holds (no ctx; Sec. 4.2 Tier 1 (3): the fast tier is filled with the clusters of
 * highest Eq. 6 score under a fixed capacity; Sec. 5.2: the cached set follows the updated scores).  Clusters are taken in
 * descending score (the Eq. 6 values swarm_set_cache maintains; ties to the lower id) while their sizes
 * (cluster_size, pages) still fit into capacity_pages; the first cluster that does not fit ends the admission.
 * Writes resident[c] = 1 or 0 for every cluster -- the table swarm_set_cache reads -- and, if info is not NULL,
 * info[0] = clusters admitted, info[1] = pages used.  Device pointers, 16-byte aligned; n_clusters <= 65536;
 * workspace: swarm_cache_admit_workspace_bytes(n_clusters) bytes (< 0: minus an error code). */
int64_t swarm_cache_admit_workspace_bytes(int32_t n_clusters);
int32_t swarm_cache_admit(const float* score, const uint16_t* cluster_size, int32_t n_clusters, int64_t capacity_pages,
                          void* workspace, int64_t workspace_bytes, uint8_t* resident, int32_t* info, void* stream);

/* Offline index build (no ctx; not part of a decode step): Algorithm 1, co-activation clustering of n entries
 * from their distance matrix dist (fp32 [n][n] row-major, d = 1 - co-activation probability) and the cluster
 * radius tau.  All pointers are device pointers, 16-byte aligned.
 *   density[i]  = #{ j != i : dist[i][j] <= tau }                                   (Step 3, Eq. 4)
 *   medoids     entries by (density descending, index ascending); an entry already covered is skipped
 *   expansion   C = {m}; the candidates { e != m : dist[m][e] <= tau } are visited once by (dist[m][e] ascending,
 *               index ascending); a candidate joins when the average of its distances to the current members is
 *               <= tau (Step 4, Eq. 5): fp32 sum in joining order over dist[member][candidate], compared against
 *               tau * |C|.  Covered entries stay candidates, so an entry may join several clusters (replicas).
 *   stop        when every entry is covered.
 * Outputs: clusters in creation order as cluster_ptr [n + 1] (only n_clusters + 1 entries are written) and
 * cluster_members (joining order, medoid first), medoid [n] (n_clusters written), n_clusters [1],
 * dev_status [1] = 0, or 1 if cluster_members (members_cap entries, at least n, below 2^31) was too small -- the output is
 * then incomplete.  n <= 32768.  workspace: swarm_build_clusters_workspace_bytes(n) bytes (< 0: minus an error code). */
int64_t swarm_build_clusters_workspace_bytes(int32_t n_entries);
int32_t swarm_build_clusters(const float* dist, int32_t n_entries, float tau, void* workspace, int64_t workspace_bytes,
                             int32_t* density, int32_t* cluster_ptr, int32_t* cluster_members, int64_t members_cap,
                             int32_t* medoid, int32_t* n_clusters, int32_t* dev_status, void* stream);

/* End-to-end convenience for callers holding the per-step data in HOST memory (pinned memory
 * recommended): copies q_host (bf16 [B][Hq][d]) into the ctx's staging area, runs swarm_step with
 * `inputs` (whose q field is ignored) and `outputs`, copies out, lse, n_uniq, queue_load back into
 * the given host buffers and WAITS for completion.  Any *_host pointer may be NULL to skip it.
 * Result buffers that are pinned and addressable by the device (unified addressing; out_host 16-byte aligned)
 * are written by the step's last kernel itself, which stores each result there as it produces it; otherwise by
 * one copy operation each.  q_host, likewise, is read over the bus by a kernel when the device can address it
 * (16-byte aligned), else copied.  When the results are stored by the kernel the call returns as soon as they
 * are visible in host memory (the last part of the kernel to finish raises a word of pinned memory owned by the
 * ctx after a system-wide fence), which is a few microseconds before the stream itself reports completion;
 * later work on the stream is ordered as usual.  Device-side outputs that have no host buffer (sel, uniq,
 * queue_of, the submission order) are complete when the stream is.
 * With pinned host buffers and a non-default stream the first call with a given set of pointers
 * records these operations into a CUDA graph (owned by the ctx) and later calls replay it; the
 * tensor shapes and the device tables must then stay where they are, their contents may change. */
int32_t swarm_step_host(swarm_ctx* ctx, const swarm_inputs* inputs, const swarm_outputs* outputs,
                        const void* q_host, float* out_host, float* lse_host, int32_t* n_uniq_host,
                        int32_t* queue_load_host, void* stream);

/* Reads and clears the device status word.  SYNCHRONISES `stream`. */
int32_t swarm_device_status(swarm_ctx* ctx, void* stream, uint32_t* bits);

/* Last cudaError_t recorded by this ctx (0 = none). */
int32_t swarm_last_cuda_error(const swarm_ctx* ctx);

/* Library version: major * 10000 + minor * 100 + patch. */
int32_t swarm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SWARM_H_ */
