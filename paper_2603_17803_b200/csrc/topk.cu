// Stage 2: per-head top-k page selection (Sec. 2.3: only the entries with the highest scores are
// activated).  One CTA per (request, query head).
//
// Scores become order-preserving 32-bit keys (-0 folded onto +0 so the two compare equal).  A
// most-significant-digit radix select finds the exact key T of the k-th best page and how many
// pages tie with it.  The digits are taken relative to the list's own [min, max] key range, 12
// bits at a time: page scores of one head sit in a narrow band (often a single binade), and digits
// cut from the raw bit pattern would throw them all into a handful of histogram bins.  With range-
// relative digits the shared-memory atomics spread over all 4096 bins and two levels usually finish.
// The result is then written in page-id order: every page with key > T, plus the first
// (k - #greater) pages with key == T, placed by a block-wide scan of per-thread counts.  That order
// gives "ties go to the lower page id" and the ascending-id output at once.
//
// topk_regs keeps ITEMS consecutive pages per thread in registers (lists of up to 16384 pages; in the
// largest instance a list of at most half that length is handled with half the pages per thread);
// topk_generic walks lists of any length in shared or global memory with the same algorithm.
#define SWARM_TRACE_FILE 1
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kBins = 4096;
constexpr int kDigitBits = 12;
constexpr int kRankMax = 64;                               // finish by direct ranking at or below this many candidates

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Optional by-products of the selection, written while the selected pages are still in registers.
//   selmap  one bit per page and query head (bit p%8 of byte p/8 of row [b][h], rows of `selmap_pitch`
//           bytes): lets the attention kernel form, per KV head, the union of its query heads' pages.
//   flags   cluster dedup flags (see resolve.cu): flag[cluster_base[b] + page2cluster[...]] = 1.
struct TopkExtras {
  uint8_t* selmap;
  int selmap_pitch;
  const int64_t* page_base;
  const int32_t* page2cluster;
  const int64_t* cluster_base;
  uint8_t* flags;
  uint32_t* status;
  // tables the next kernels read through dependent loads; pulled into L2 while this kernel waits for the scores
  const uint32_t* replica_mask;
  const uint16_t* cluster_size;
  long long n_pool_pages;
  // hand-offs (see StepTickets): wait for the scorer's tickets instead of the whole scorer; announce each head
  const int64_t* req_base;        // [B+1] pages (or, for the medoid index, clusters) each request owns
  StepTickets tk;
  long long flags_alt;            // > 0: two flag arrays this many bytes apart, used by alternate steps (overlapped tail)
  uint32_t ll_flag;               // with tk.selmap_ll: the flag this step's bitmap words carry (set by the kernel)
};

// What a selection CTA does before it reads its head's scores.  With tickets: one thread waits (bounded) until
// the scorer has stored every tile of the head's KV pair; a request whose length the scorer refuses never gets
// tickets and is not waited for.  Without: the whole previous kernel.  Returns false when the head has no
// usable scores (refused length, or the wait ran out): the CTA then writes an empty selection.
__device__ __forceinline__ bool scores_ready(const Geometry& geo, const TopkExtras& x, int b, int kvh, int len_b, bool* s_flag) {
  // (Overlapped tail: the flag array this step marks was last read by the resolution of the step before the
  // previous one, which has finished by now in any schedule that keeps up; make sure of it.)
  if (threadIdx.x == 0 && x.flags_alt > 0) {
    const unsigned marked = x.tk.ctl[kCtlMarked];
    if (marked >= 1u && !wait_at_least(x.tk.ctl + kCtlResolved, marked - 1u)) atomicOr(x.status, SWARM_DEV_TIMEOUT);
  }
  if (x.tk.ready == nullptr) {
    pdl_wait();
    if (threadIdx.x == 0 && x.tk.ctl != nullptr) red_relaxed_add(x.tk.ctl + kCtlTopkDone, 1u);
    return true;
  }
  if (threadIdx.x == 0) {
    const int P = pages_of(len_b, geo.S);
    bool ok = len_b >= 1 && P <= geo.Pmax && (long long)P <= x.req_base[b + 1] - x.req_base[b];
    if (ok && x.tk.scores_ll == nullptr) {                 // (self-validating scores are waited for one by one, by their readers)
      const int hp = kvh / 2;
      const unsigned target = (unsigned)((P + 15) / 16) * (unsigned)min(2, geo.Hkv - 2 * hp);
      ok = wait_at_least(x.tk.ready + (long long)b * head_pairs(geo.Hkv) + hp, target);
      if (!ok) atomicOr(x.status, SWARM_DEV_TIMEOUT);
    }
    // this CTA is past its wait (no result comes back: an atomic with one held the CTA's next barrier); the count
    // also says that the CTA has read the step's epoch, which it is made to wait for
    red_relaxed_add(x.tk.ctl + kCtlTopkDone, 1u + zero_after(x.ll_flag));
    *s_flag = ok;
  }
  __syncthreads();
  return *s_flag;
}

// An empty selection for head bh (no usable scores).
__device__ __forceinline__ void write_empty_selection(const Geometry& geo, const TopkExtras& x, int bh, int32_t* out,
                                                      int32_t* n_sel, int threads) {
  for (int j = threadIdx.x; j < geo.k; j += threads) out[j] = -1;
  if (threadIdx.x == 0) n_sel[bh] = 0;
  if (x.tk.selmap_ll != nullptr) {
    uint2* row = x.tk.selmap_ll + (long long)bh * (x.selmap_pitch / 4);
    for (int w = threadIdx.x; w < x.selmap_pitch / 4; w += threads) ll_word_store(row + w, 0u, x.ll_flag);
  }
  if (x.selmap != nullptr) {
    uint8_t* row = x.selmap + (long long)bh * x.selmap_pitch;
    for (int o = threadIdx.x * 4; o + 4 <= x.selmap_pitch; o += threads * 4) *reinterpret_cast<uint32_t*>(row + o) = 0u;
  }
}

// The head's page bitmap is stored: announce it to the attention CTAs of its KV head (a barrier, then one
// release that is cumulative over the CTA's stores so far).
__device__ __forceinline__ void selection_announce(const Geometry& geo, const TopkExtras& x, int b, int kvh) {
  if (x.tk.sel_ready == nullptr || x.tk.selmap_ll != nullptr) return;   // (self-validating bitmaps announce themselves)
  __syncthreads();
  if (threadIdx.x == 0) red_release_add(x.tk.sel_ready + (long long)b * geo.Hkv + kvh, 1u);
}

// What a selection CTA does last.  The last CTA of the grid (its scores arrive last, so it tends to finish last)
// tidies up: once every CTA is past its wait for the scorer nobody reads the scorer's tickets any more, and they
// go back to zero.
__device__ __forceinline__ void selection_done(const Geometry& geo, const TopkExtras& x) {
  if (x.tk.ctl == nullptr) return;
  if (threadIdx.x == 0 && blockIdx.x == gridDim.x - 1) {
    if (!wait_at_least(x.tk.ctl + kCtlTopkDone, gridDim.x)) atomicOr(x.status, SWARM_DEV_TIMEOUT);
    if (x.tk.ready != nullptr)
      for (int i = 0; i < geo.B * head_pairs(geo.Hkv); ++i) x.tk.ready[i] = 0u;
    if (x.flags_alt > 0) x.tk.ctl[kCtlMarked] += 1u;        // one more step has its cluster marks (complete when this kernel is)
    // last of all: whoever reads 0 here (the attention kernel, before it lets the next step start) also sees
    // the cleared tickets
    st_release(x.tk.ctl + kCtlTopkDone, 0u);
  }
}

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Spread over the whole grid: one 128-byte line per thread and step, at most ~8 MiB in total.
__device__ __forceinline__ void prefetch_tables(const Geometry& geo, const TopkExtras& x) {
  if (x.flags == nullptr) return;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x, nthreads = (long long)gridDim.x * blockDim.x;
  const long long cap = 8LL << 20;
  const long long p2c_bytes = min(x.n_pool_pages * 4, cap), mask_bytes = min((long long)geo.Cmax * 4, cap),
                  size_bytes = min((long long)geo.Cmax * 2, cap);
  for (long long o = tid * 128; o < p2c_bytes; o += nthreads * 128)
    prefetch_l2(reinterpret_cast<const char*>(x.page2cluster) + o);
  if (x.replica_mask != nullptr)
    for (long long o = tid * 128; o < mask_bytes; o += nthreads * 128)
      prefetch_l2(reinterpret_cast<const char*>(x.replica_mask) + o);
  if (x.cluster_size != nullptr)
    for (long long o = tid * 128; o < size_bytes; o += nthreads * 128)
      prefetch_l2(reinterpret_cast<const char*>(x.cluster_size) + o);
}

// Bases of request b in the page and cluster tables.  They are inputs, not results of the previous kernel, so
// they are read before the wait on it.
struct RequestBases {
  long long pb, cb, cn;
};
__device__ __forceinline__ RequestBases load_bases(const TopkExtras& x, int b) {
  RequestBases r{0, 0, 0};
  if (x.flags != nullptr) {
    r.pb = x.page_base[b];
    r.cb = x.cluster_base[b];
    r.cn = x.cluster_base[b + 1];
  }
  return r;
}
__device__ __forceinline__ void mark_cluster(const Geometry& geo, const TopkExtras& x, const RequestBases& rb, int p) {
  const int c = x.page2cluster[rb.pb + p];
  if (c < 0 || c >= rb.cn - rb.cb || rb.cb + c >= geo.Cmax) atomicOr(x.status, SWARM_DEV_BAD_CLUSTER);
  else x.flags[rb.cb + c] = 1;
}

// Shared state of one radix-select run.
struct SelectState {
  int hist[kBins];
  int warp_tot[32];
  uint32_t red_min[32], red_max[32];
  uint32_t cand[kRankMax]; // candidate keys of the chosen bin, when few enough to finish by direct ranking
  int n_cand;          // number of keys in the chosen bin (set by narrow), then the fill counter of cand[]
  uint32_t base;       // keys below `base` are out; candidates satisfy key - base < 2^bits
  int bits;            // undecided low bits of the candidates
  int remaining;       // rank still to find among the candidates (counted from the top)
};

// Where digit `bin` is counted.  Thread t owns the PER consecutive digits below (kBins - 1 - t*PER); its
// j-th digit lives at word j*THREADS + t, so the threads of a warp touch consecutive words when they read
// or clear their digits (no bank conflicts).
template <int THREADS>
__device__ __forceinline__ int hist_slot(uint32_t bin) {
  constexpr int PER = kBins / THREADS;
  const uint32_t idx = (uint32_t)(kBins - 1) - bin;         // rank of the digit from the top
  return (int)((idx % PER) * THREADS + idx / PER);
}

// Sum of the totals of the warps before `warp` (THREADS / 32 <= 32 totals in shared memory): every warp reduces
// the masked totals with shuffles instead of each thread adding them up one by one.
template <int THREADS>
__device__ __forceinline__ int totals_before(const int* warp_tot, int warp, int lane) {
  int v = (lane < THREADS / 32 && lane < warp) ? warp_tot[lane] : 0;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// After the histogram of the current level is complete: locate the bin holding rank `remaining`
// from the top, narrow (base, bits, remaining), clear the histogram.  All threads call it.
template <int THREADS>
__device__ __forceinline__ void narrow(SelectState& st, int tid, int shift) {
  constexpr int PER = kBins / THREADS;                      // bins per thread, highest bins first
  const int lane = tid & 31, warp = tid >> 5;
  int c[PER], sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    c[j] = st.hist[j * THREADS + tid];
    sum += c[j];
  }
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) st.warp_tot[warp] = incl;
  const uint32_t base = st.base;
  const int remaining = st.remaining;
  __syncthreads();
  int above = incl - sum + totals_before<THREADS>(st.warp_tot, warp, lane);
#pragma unroll
  for (int j = 0; j < PER; ++j) st.hist[j * THREADS + tid] = 0;
  if (above < remaining && remaining <= above + sum) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (above < remaining && remaining <= above + c[j]) {
        st.base = base + ((uint32_t)(kBins - 1 - (tid * PER + j)) << shift);
        st.bits = shift;
        st.remaining = remaining - above;
        st.n_cand = c[j];
        above = remaining;                                   // stop
      } else {
        above += c[j];
      }
    }
  }
  __syncthreads();
}

template <int THREADS>
__device__ __forceinline__ void block_minmax(SelectState& st, int tid, uint32_t lo, uint32_t hi) {
  const int lane = tid & 31, warp = tid >> 5;
  lo = __reduce_min_sync(0xFFFFFFFFu, lo);
  hi = __reduce_max_sync(0xFFFFFFFFu, hi);
  if (lane == 0) { st.red_min[warp] = lo; st.red_max[warp] = hi; }
  __syncthreads();
  if (warp == 0) {
    lo = lane < THREADS / 32 ? st.red_min[lane] : 0xFFFFFFFFu;
    hi = lane < THREADS / 32 ? st.red_max[lane] : 0u;
    lo = __reduce_min_sync(0xFFFFFFFFu, lo);
    hi = __reduce_max_sync(0xFFFFFFFFu, hi);
    if (lane == 0) {
      st.base = lo;
      st.bits = 32 - __clz(hi - lo);                        // 0 when every key is equal
    }
  }
  __syncthreads();
}

// The chosen bin holds few keys (already gathered in st.cand[0 .. n)): rank them directly.  The key whose
// rank interval contains `remaining` is the k-th best key; ties share the interval, so every thread that
// finds it writes the same values.
template <int THREADS>
__device__ __forceinline__ void finish_by_ranking(SelectState& st, int tid, int n) {
  const int remaining = st.remaining;
  const int lane = tid & 31, warp = tid >> 5;
  __syncthreads();
  // one warp per candidate: the lanes hold all (at most 64) candidates, two ballots count those above and equal
  const bool v0 = lane < n, v1 = lane + 32 < n;
  const uint32_t o0 = v0 ? st.cand[lane] : 0u, o1 = v1 ? st.cand[lane + 32] : 0u;
  for (int i = warp; i < n; i += THREADS / 32) {
    const uint32_t mine = st.cand[i];
    const int gt = __popc(__ballot_sync(0xFFFFFFFFu, v0 && o0 > mine)) + __popc(__ballot_sync(0xFFFFFFFFu, v1 && o1 > mine));
    const int eq = __popc(__ballot_sync(0xFFFFFFFFu, v0 && o0 == mine)) + __popc(__ballot_sync(0xFFFFFFFFu, v1 && o1 == mine));
    if (lane == 0 && gt < remaining && remaining <= gt + eq) {
      st.base = mine;
      st.bits = 0;
      st.remaining = remaining - gt;
    }
  }
  __syncthreads();
}

// ---- register-resident variant -------------------------------------------------------------------
// The selection of one list with ITEMS consecutive pages per thread (the kernel was launched for lists of up to
// THREADS * MAX_ITEMS pages; rows of the page bitmap are that long).
template <int THREADS, int ITEMS, int MAX_ITEMS, bool kEarly>
__device__ __forceinline__ bool topk_regs_body(SelectState& st, const Geometry& geo, const TopkExtras& x,
                                               const RequestBases& rb, const float* __restrict__ s,
                                               int32_t* __restrict__ out, int32_t* __restrict__ n_sel,
                                               uint32_t* __restrict__ status, int bh, int b, int kvh, int len_b, bool* s_flag,
                                               int P, int Pw, int k_eff, int k_sel) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // thread t owns pages [t*ITEMS, (t+1)*ITEMS); keys of pages that do not exist are never used
  uint32_t key[ITEMS];
  const int p0 = tid * ITEMS;
  // The clusters of this thread's pages: an input table, read while the scores are still being written, so that
  // marking the selected pages' clusters later costs no memory round trip.
  // (Only with few lists: all heads of a request read the same entries, and with thousands of lists that is
  // hundreds of megabytes of cache traffic for the one page in 30-60 that ends up selected.)
  int cl[kEarly ? ITEMS : 1];
  if (kEarly && x.flags != nullptr) {
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) cl[j] = p0 + j < P ? x.page2cluster[rb.pb + p0 + j] : -1;
  }
  if (!scores_ready(geo, x, b, kvh, len_b, s_flag)) return false;   // the scores come from the previous kernel
  SWARM_STAMP(status, 1);
  const bool full = p0 + ITEMS <= Pw;                       // all of this thread's pages exist and are scored: no per-page checks
  if (kEarly && x.tk.scores_ll != nullptr) {             // (few lists only, like kEarly: see launch_topk)
    // {score, epoch} pairs that the scorer may still be writing: all of this thread's pairs are asked for together
    // (two per 16-byte load: the row length is even) and asked for again until every existing page's carries this
    // step's flag (bounded)
    const uint2* pairs = x.tk.scores_ll + (long long)bh * geo.Pmax + p0;
    unsigned bad = 0u, polls = 0u;
    do {
      bad = 0u;
#pragma unroll
      for (int j = 0; j < ITEMS; j += 2) {
        key[j] = key[j + 1] = 0u;
        if (p0 + j < P) {
          uint4 v;
          asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(pairs + j) : "memory");
          key[j] = score_key(__uint_as_float(v.x));
          bad |= v.y ^ x.ll_flag;
          if (p0 + j + 1 < P) {
            key[j + 1] = score_key(__uint_as_float(v.z));
            bad |= v.w ^ x.ll_flag;
          }
        }
      }
    } while (bad != 0u && ++polls < kLlWaitLimit);
    if (bad != 0u) atomicOr(x.status, SWARM_DEV_TIMEOUT);
  } else if (p0 + ITEMS <= P && (geo.Pmax & 3) == 0) {
#pragma unroll
    for (int j = 0; j < ITEMS; j += 4) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(s + p0 + j));   // written by a kernel that may still run: not through L1
      key[j] = score_key(v.x); key[j + 1] = score_key(v.y); key[j + 2] = score_key(v.z); key[j + 3] = score_key(v.w);
    }
  } else {
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) key[j] = p0 + j < P ? score_key(__ldcg(s + p0 + j)) : 0u;
  }
  if (tid == 0) st.remaining = k_sel;
  SWARM_STAMP(status, 2);

  uint32_t T = 0u;
  int need_eq = P;                                          // k_sel == Pw keeps everything
  if (k_sel == 0) {
    T = 0xFFFFFFFFu;                                        // nothing but the window
    need_eq = 0;
  } else if (k_sel < Pw) {
    uint32_t lo = 0xFFFFFFFFu, hi = 0u;
    if (full) {
#pragma unroll
      for (int j = 0; j < ITEMS; ++j) { lo = min(lo, key[j]); hi = max(hi, key[j]); }
    } else {
#pragma unroll
      for (int j = 0; j < ITEMS; ++j)
        if (p0 + j < Pw) { lo = min(lo, key[j]); hi = max(hi, key[j]); }
    }
    block_minmax<THREADS>(st, tid, lo, hi);
    SWARM_STAMP(status, 3);
    for (int level = 0; level < 4 && st.bits > 0; ++level) {
      const uint32_t base = st.base;
      const int bits = st.bits;
      const int shift = max(bits - kDigitBits, 0);
      const uint32_t width_m1 = bits >= 32 ? 0xFFFFFFFFu : ((1u << bits) - 1u);
      if (full) {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
          const uint32_t rel = key[j] - base;
          if (rel <= width_m1) atomicAdd(&st.hist[hist_slot<THREADS>(rel >> shift)], 1);
        }
      } else {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
          const uint32_t rel = key[j] - base;
          if (p0 + j < Pw && rel <= width_m1) atomicAdd(&st.hist[hist_slot<THREADS>(rel >> shift)], 1);
        }
      }
      __syncthreads();
      SWARM_STAMP(status, 4 + 2 * level);
      narrow<THREADS>(st, tid, shift);
      SWARM_STAMP(status, 5 + 2 * level);
      const int n_cand = st.n_cand;
      if (st.bits > 0 && n_cand <= kRankMax) {
        // few keys left: gather them and rank directly instead of running more digit levels
        const uint32_t cbase = st.base;
        const uint32_t cwidth_m1 = (1u << st.bits) - 1u;
        __syncthreads();                                    // everyone has read n_cand before it becomes the fill counter
        if (tid == 0) st.n_cand = 0;
        __syncthreads();
#pragma unroll
        for (int j = 0; j < ITEMS; ++j)
          if ((full || p0 + j < Pw) && key[j] - cbase <= cwidth_m1) st.cand[atomicAdd(&st.n_cand, 1)] = key[j];
        finish_by_ranking<THREADS>(st, tid, n_cand);
      }
    }
    T = st.base;
    need_eq = st.remaining;
  }
  SWARM_STAMP(status, 12);

  // ordered output: packed (greater, equal) counts per thread, one block-wide exclusive scan.  A thread keeps
  // its pages above the threshold (window pages rank above every score) and at it as two bit masks: about one
  // page in P / k is selected, so everything after the scan walks the set bits instead of all ITEMS pages.
  unsigned gt_mask = 0u, eq_mask = 0u;
  if (full) {
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      gt_mask |= (unsigned)(key[j] > T) << j;
      eq_mask |= (unsigned)(key[j] == T) << j;
    }
  } else {
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      if (p0 + j < P) {
        const bool win = p0 + j >= Pw;
        gt_mask |= (unsigned)(win || key[j] > T) << j;
        eq_mask |= (unsigned)(!win && key[j] == T) << j;
      }
    }
  }
  const int cnt = __popc(gt_mask) | (__popc(eq_mask) << 16);
  int incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();                                          // warp_tot may still be read by narrow()
  if (lane == 31) st.warp_tot[warp] = incl;
  __syncthreads();
  const int before = incl - cnt + totals_before<THREADS>(st.warp_tot, warp, lane);
  const int gt_before = before & 0xFFFF, eq_before = before >> 16;
  // The page bitmap goes out first and the head is announced to the attention CTAs right behind it: a release
  // waits for every store issued before it to be acknowledged, so the selection list, the cluster marks and the
  // rest (which the attention does not read) are stored after the announcement, not before.
  unsigned picked = 0u;                                     // bit j: page p0 + j is selected
  for (unsigned todo = gt_mask | eq_mask; todo != 0u; todo &= todo - 1u) {
    const unsigned bit = todo & (0u - todo);
    if ((gt_mask & bit) || eq_before + __popc(eq_mask & (bit - 1u)) < need_eq) picked |= bit;
  }
  if (kEarly && x.tk.selmap_ll != nullptr) {              // (few lists only, like kEarly: see launch_topk)
    // as {word, epoch} pairs: neighbouring lanes put their bytes together, the first of each group stores
    uint2* row = x.tk.selmap_ll + (long long)bh * (x.selmap_pitch / 4);
    unsigned word = picked;
    if (ITEMS == 8) {
      word |= __shfl_down_sync(0xFFFFFFFFu, word, 1) << 8;
      word |= __shfl_down_sync(0xFFFFFFFFu, word, 2) << 16;
    } else {
      word |= __shfl_down_sync(0xFFFFFFFFu, word, 1) << 16;
    }
    constexpr int kLanesPerWord = 32 / ITEMS;
    const int w = tid / kLanesPerWord;
    if (tid % kLanesPerWord == 0 && w < x.selmap_pitch / 4) ll_word_store(row + w, word, x.ll_flag);
    if (ITEMS < MAX_ITEMS)                                 // the part of the bitmap row these threads do not reach
      for (int w2 = THREADS * ITEMS / 32 + tid; w2 < x.selmap_pitch / 4; w2 += THREADS) ll_word_store(row + w2, 0u, x.ll_flag);
  }
  {                                                        // the plain bitmap (behind the pairs, if any: later calls read it)
    if (x.selmap != nullptr && p0 < x.selmap_pitch * 8) {
      uint8_t* row = x.selmap + (long long)bh * x.selmap_pitch + p0 / 8;
      if (ITEMS == 8) *row = (uint8_t)picked;
      else *reinterpret_cast<uint16_t*>(row) = (uint16_t)picked;
    }
    if (ITEMS < MAX_ITEMS && x.selmap != nullptr) {        // the part of the bitmap row these threads do not reach
      uint8_t* row = x.selmap + (long long)bh * x.selmap_pitch;
      for (int o = THREADS * ITEMS / 8 + tid * 4; o + 4 <= x.selmap_pitch; o += THREADS * 4)
        *reinterpret_cast<uint32_t*>(row + o) = 0u;
    }
  }
  selection_announce(geo, x, b, kvh);
  for (unsigned todo = picked; todo != 0u; todo &= todo - 1u) {
    const unsigned bit = todo & (0u - todo), below = bit - 1u;
    const int eq_b = eq_before + __popc(eq_mask & below);
    out[gt_before + __popc(gt_mask & below) + min(eq_b, need_eq)] = p0 + (__ffs(bit) - 1);
  }
  if (kEarly && x.flags != nullptr) {
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      if ((picked >> j) & 1u) {
        const int c = cl[kEarly ? j : 0];
        if (c < 0 || c >= rb.cn - rb.cb || rb.cb + c >= geo.Cmax) atomicOr(x.status, SWARM_DEV_BAD_CLUSTER);
        else x.flags[rb.cb + c] = 1;
      }
    }
  } else if (x.flags != nullptr) {
    // four selected pages at a time: all the table reads first, then the flag stores -- a byte store may alias
    // anything, so interleaving them would make every read wait for the store before it
    for (unsigned todo = picked; todo != 0u;) {
      int c[4];
      bool have[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        have[i] = todo != 0u;
        const int j = __ffs(todo) - 1;
        todo &= todo - 1u;                                  // 0 stays 0
        c[i] = have[i] ? x.page2cluster[rb.pb + p0 + j] : 0;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (have[i]) {
          if (c[i] < 0 || c[i] >= rb.cn - rb.cb || rb.cb + c[i] >= geo.Cmax) atomicOr(x.status, SWARM_DEV_BAD_CLUSTER);
          else x.flags[rb.cb + c[i]] = 1;
        }
      }
    }
  }
  for (int j = k_eff + tid; j < geo.k; j += THREADS) out[j] = -1;
  if (tid == 0) n_sel[bh] = k_eff;
  SWARM_STAMP(status, 13);
  return true;
}

template <int THREADS, int ITEMS, bool kEarly>
__global__ void __launch_bounds__(THREADS)
topk_regs_kernel(Geometry geo, const float* __restrict__ scores, const int32_t* __restrict__ ctx_len,
                 int32_t* __restrict__ sel, int32_t* __restrict__ n_sel, uint32_t* __restrict__ status, TopkExtras x) {
  __shared__ SelectState st;
  __shared__ bool s_flag;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.x, b = bh / geo.Hq, kvh = (bh - b * geo.Hq) / geo.g;
  pdl_launch_dependents();
  SWARM_STAMP(status, 0);
  SWARM_KERNEL_BEGIN(status, 1);
  for (int i = tid; i < kBins; i += THREADS) st.hist[i] = 0;
  prefetch_tables(geo, x);
  const RequestBases rb = load_bases(x, b);
  const int len_b = ctx_len[b];
  const float* s = scores + (long long)bh * geo.Pmax;
  int32_t* out = sel + (long long)bh * geo.k;
  if (x.flags_alt > 0) x.flags += (x.tk.ctl[kCtlMarked] & 1u) * x.flags_alt;   // stable: the previous step's selection has finished
  // the step's epoch (stable too: the previous step's attention kernel, which raises it, has finished)
  x.ll_flag = x.tk.selmap_ll != nullptr ? *reinterpret_cast<const volatile unsigned*>(x.tk.ctl + kCtlEpoch) + 1u : 0u;
  const int P = max(0, min(pages_of(len_b, geo.S), geo.Pmax));   // invalid lengths are reported by the scorer
  const int k_eff = min(geo.k, P);
  const int Pw = P - min(geo.W, P);                         // pages [Pw, P) are the local window: always kept
  const int k_sel = k_eff - (P - Pw);                       // places left for the scored pages [0, Pw)
  // A list half as long as the kernel's capacity is handled with half the pages per thread: the work of every
  // phase is per page held, and the lists of one launch differ in length (ragged batches).
  bool ok;
  if (ITEMS == 16 && P <= THREADS * 8)
    ok = topk_regs_body<THREADS, 8, ITEMS, kEarly>(st, geo, x, rb, s, out, n_sel, status, bh, b, kvh, len_b, &s_flag, P, Pw, k_eff, k_sel);
  else
    ok = topk_regs_body<THREADS, ITEMS, ITEMS, kEarly>(st, geo, x, rb, s, out, n_sel, status, bh, b, kvh, len_b, &s_flag, P, Pw, k_eff, k_sel);
  if (!ok) {
    write_empty_selection(geo, x, bh, out, n_sel, THREADS);
    selection_announce(geo, x, b, kvh);
  }
  selection_done(geo, x);
  SWARM_KERNEL_END(status, 1);
}

// ---- generic variant: any list length, keys in shared memory when they fit, else re-read ----------
constexpr int kGenericThreads = 1024;

template <bool kKeysInSmem>
__global__ void __launch_bounds__(kGenericThreads)
topk_generic_kernel(Geometry geo, const float* __restrict__ scores, const int32_t* __restrict__ ctx_len,
                    int32_t* __restrict__ sel, int32_t* __restrict__ n_sel, uint32_t* __restrict__ status, TopkExtras x) {
  extern __shared__ uint32_t skeys[];
  __shared__ SelectState st;
  __shared__ int warp_gt[32], warp_eq[32];
  __shared__ bool s_flag;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.x, b = bh / geo.Hq, kvh = (bh - b * geo.Hq) / geo.g;
  pdl_launch_dependents();
  for (int i = tid; i < kBins; i += kGenericThreads) st.hist[i] = 0;
  prefetch_tables(geo, x);
  const RequestBases rb = load_bases(x, b);
  const int len_b = ctx_len[b];
  const float* s = scores + (long long)bh * geo.Pmax;
  int32_t* out = sel + (long long)bh * geo.k;
  if (x.flags_alt > 0) x.flags += (x.tk.ctl[kCtlMarked] & 1u) * x.flags_alt;
  x.ll_flag = x.tk.selmap_ll != nullptr ? *reinterpret_cast<const volatile unsigned*>(x.tk.ctl + kCtlEpoch) + 1u : 0u;
  if (!scores_ready(geo, x, b, kvh, len_b, &s_flag)) {
    write_empty_selection(geo, x, bh, out, n_sel, kGenericThreads);
    selection_announce(geo, x, b, kvh);
    selection_done(geo, x);
    return;
  }
  const int P = max(0, min(pages_of(len_b, geo.S), geo.Pmax));
  const int k_eff = min(geo.k, P);
  const int Pw = P - min(geo.W, P);                         // see topk_regs_kernel
  const int k_sel = k_eff - (P - Pw);
  auto key_at = [&](int i) -> uint32_t { return kKeysInSmem ? skeys[i] : score_key(__ldcg(s + i)); };

  uint32_t lo = 0xFFFFFFFFu, hi = 0u;
  for (int i = tid; i < P; i += kGenericThreads) {
    const uint32_t key = score_key(__ldcg(s + i));
    if (kKeysInSmem) skeys[i] = key;
    if (i < Pw) {
      lo = min(lo, key);
      hi = max(hi, key);
    }
  }
  if (tid == 0) st.remaining = k_sel;
  uint32_t T = 0u;
  int need_eq = P;
  if (k_sel == 0) {
    T = 0xFFFFFFFFu;
    need_eq = 0;
    __syncthreads();
  } else if (k_sel < Pw) {
    block_minmax<kGenericThreads>(st, tid, lo, hi);
    for (int level = 0; level < 4 && st.bits > 0; ++level) {
      const uint32_t base = st.base;
      const int bits = st.bits;
      const int shift = max(bits - kDigitBits, 0);
      const uint32_t width_m1 = bits >= 32 ? 0xFFFFFFFFu : ((1u << bits) - 1u);
      for (int i = tid; i < Pw; i += kGenericThreads) {
        const uint32_t rel = key_at(i) - base;
        if (rel <= width_m1) atomicAdd(&st.hist[hist_slot<kGenericThreads>(rel >> shift)], 1);
      }
      __syncthreads();
      narrow<kGenericThreads>(st, tid, shift);
    }
    T = st.base;
    need_eq = st.remaining;
  } else {
    __syncthreads();
  }

  // ordered ballot/popc compaction; warp w owns the contiguous span [w*seg, (w+1)*seg)
  const int seg = (((P + 31) / 32 + 31) & ~31);
  const int w_lo = min(P, warp * seg), w_hi = min(P, w_lo + seg);
  int cnt_gt = 0, cnt_eq = 0;
  for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < w_hi ? key_at(i) : 0u;
    cnt_gt += __popc(__ballot_sync(0xFFFFFFFFu, i < w_hi && (key > T || i >= Pw)));
    cnt_eq += __popc(__ballot_sync(0xFFFFFFFFu, i < w_hi && key == T && i < Pw));
  }
  if (lane == 0) { warp_gt[warp] = cnt_gt; warp_eq[warp] = cnt_eq; }
  __syncthreads();
  int gt_before = 0, eq_before = 0;
  for (int w2 = 0; w2 < warp; ++w2) { gt_before += warp_gt[w2]; eq_before += warp_eq[w2]; }
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < w_hi ? key_at(i) : 0u;
    const bool gt = i < w_hi && (key > T || i >= Pw), eq = i < w_hi && key == T && i < Pw;
    const unsigned bg = __ballot_sync(0xFFFFFFFFu, gt), be = __ballot_sync(0xFFFFFFFFu, eq);
    const int my_gt = gt_before + __popc(bg & lt_mask);
    const int my_eq = eq_before + __popc(be & lt_mask);
    const bool take = gt || (eq && my_eq < need_eq);
    if (take) {
      out[my_gt + min(my_eq, need_eq)] = i;
      if (x.flags != nullptr) mark_cluster(geo, x, rb, i);
    }
    const unsigned word = __ballot_sync(0xFFFFFFFFu, take);
    if (lane == 0 && i0 / 8 + 4 <= x.selmap_pitch) {
      if (x.tk.selmap_ll != nullptr) ll_word_store(x.tk.selmap_ll + (long long)bh * (x.selmap_pitch / 4) + i0 / 32, word, x.ll_flag);
      if (x.selmap != nullptr) *reinterpret_cast<uint32_t*>(x.selmap + (long long)bh * x.selmap_pitch + i0 / 8) = word;
    }
    gt_before += __popc(bg);
    eq_before += __popc(be);
  }
  if (x.tk.selmap_ll != nullptr) {                          // words past the last page of the request
    for (int w = (P + 31) / 32 + tid; w < x.selmap_pitch / 4; w += kGenericThreads)
      ll_word_store(x.tk.selmap_ll + (long long)bh * (x.selmap_pitch / 4) + w, 0u, x.ll_flag);
  }
  if (x.selmap != nullptr) {
    const int first = ((P + 31) / 32) * 4;
    for (int o = first + tid * 4; o + 4 <= x.selmap_pitch; o += kGenericThreads * 4)
      *reinterpret_cast<uint32_t*>(x.selmap + (long long)bh * x.selmap_pitch + o) = 0u;
  }
  for (int j = k_eff + tid; j < geo.k; j += kGenericThreads) out[j] = -1;
  if (tid == 0) n_sel[bh] = k_eff;
  selection_announce(geo, x, b, kvh);
  selection_done(geo, x);
}

constexpr size_t kSmemKeyBytes = 160 * 1024;

}  // namespace

int topk_threads(int Pmax) { return Pmax <= 1024 ? 128 : Pmax <= 2048 ? 256 : Pmax <= 4096 ? 512 : 1024; }

cudaError_t configure_topk() {
  return cudaFuncSetAttribute(topk_generic_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)kSmemKeyBytes);
}

cudaError_t launch_topk(const Geometry& geo, const float* scores, const int32_t* ctx_len, int32_t* sel,
                        int32_t* n_sel, uint32_t* status, cudaStream_t st, bool overlap, const TopkLinks& links,
                        uint8_t* selmap, const int64_t* page_base, const int32_t* page2cluster,
                        const int64_t* cluster_base, uint8_t* flags, const uint32_t* replica_mask,
                        const uint16_t* cluster_size) {
  TopkExtras x;
  x.selmap = selmap;
  x.selmap_pitch = selmap_pitch_bytes(geo.Pmax);
  x.page_base = page_base;
  x.page2cluster = page2cluster;
  x.cluster_base = cluster_base;
  x.flags = flags;
  x.status = status;
  x.replica_mask = replica_mask;
  x.cluster_size = cluster_size;
  x.n_pool_pages = geo.n_pool_pages;
  x.req_base = links.req_base;
  x.tk = links.tk;
  x.flags_alt = flags != nullptr ? links.flags_alt : 0;
  if (x.req_base == nullptr) x.tk.ready = nullptr;         // the validity test of a request needs its page count
  if (x.tk.ready == nullptr) x.tk.selmap_ll = x.tk.scores_ll = nullptr;     // (the epoch is counted with the scorer's tickets)
  x.ll_flag = 0u;
  // few lists: every thread reads the page -> cluster entries of all its pages up front (kEarly)
  const bool early = flags != nullptr && (long long)geo.B * geo.Hq <= 128;
  // Only the few-lists instances of the register-resident kernel carry the code for self-validating words (the
  // others keep the register count that lets a 256-thread CTA sit beside a scorer CTA); callers ask for them only
  // where these instances run (step_tickets).
  if ((x.tk.selmap_ll != nullptr || x.tk.scores_ll != nullptr) && (!early || geo.Pmax > 16384)) return cudaErrorInvalidValue;
  const dim3 grid(geo.B * geo.Hq);
#define SWARM_TOPK_REGS(THREADS, ITEMS)                                                                           \
  return early ? launch_pdl(topk_regs_kernel<THREADS, ITEMS, true>, grid, dim3(THREADS), 0, st, overlap, geo, scores, \
                            ctx_len, sel, n_sel, status, x)                                                         \
               : launch_pdl(topk_regs_kernel<THREADS, ITEMS, false>, grid, dim3(THREADS), 0, st, overlap, geo, scores, \
                            ctx_len, sel, n_sel, status, x)
  if (geo.Pmax <= 1024) SWARM_TOPK_REGS(128, 8);
  if (geo.Pmax <= 2048) SWARM_TOPK_REGS(256, 8);
  if (geo.Pmax <= 4096) SWARM_TOPK_REGS(512, 8);
  if (geo.Pmax <= 8192) SWARM_TOPK_REGS(1024, 8);
  if (geo.Pmax <= 16384) SWARM_TOPK_REGS(1024, 16);
#undef SWARM_TOPK_REGS
  const size_t key_bytes = (size_t)geo.Pmax * sizeof(uint32_t);
  if (key_bytes <= kSmemKeyBytes)
    return launch_pdl(topk_generic_kernel<true>, grid, dim3(kGenericThreads), key_bytes, st, overlap, geo, scores,
                      ctx_len, sel, n_sel, status, x);
  return launch_pdl(topk_generic_kernel<false>, grid, dim3(kGenericThreads), 0, st, overlap, geo, scores, ctx_len,
                    sel, n_sel, status, x);
}

}  // namespace swarm
