// Stage 3: cluster resolution, global merge and load-balanced bucket scheduling (Eq. 8; Sec. 5.1), written as
// a device function that two kernels run: resolve_kernel (swarm_resolve_clusters) and, inside the fused step,
// block 0 of the attention kernel (beside the attention CTAs; as a kernel of its own on a second stream it
// lost about 2 us whenever the attention kernel started).
//
//   mark     (all CTAs; inside the fused step the selection kernel has done it and this phase is skipped)
//            every selected (request, page) -> global cluster id; flag[id] = 1.
//            Idempotent byte stores: concurrent writers store the same value, so the dedup needs no
//            atomics.  Four independent slots per thread keep the dependent loads overlapped.
//   tail     (the CTA that finishes marking last, found with one ticket counter)
//     compact  ordered compaction of the flags -> uniq[] ascending by id: each lane takes 4 flags
//              with one load (the replica masks and sizes of those clusters are requested in the same
//              round trip), a warp scan places them; the flags are cleared on the way so the next call
//              starts from zeros.  The clusters that need the serial pass are packed, with their output
//              slots, into per-warp segments of an item list (shared memory when it fits).
//              With cache state attached (swarm_set_cache) the same pass drops the activated clusters
//              that are resident (Eq. 8) and updates the activation frequencies and Eq. 6 scores.
//     route    single-replica clusters go to their queue (integer histogram, order-free).  Clusters
//              with R >= 2 replicas are visited by (R ascending, id ascending) by one warp: lane j
//              keeps (load[j] << 5 | j); one redux.min over the lanes named by the replica mask
//              picks the least-loaded replica with ties to the lowest queue id, and only the lane
//              whose value equals the minimum adds the cluster's weight.
//              Under SWARM_ORDER_BY_ID the same warp visits every cluster in id order instead.
//     submit   (optional output) the batched submission order of Sec. 5.1, see the end of the body.
#pragma once
#include "swarm_internal.cuh"

namespace swarm {
namespace resolve_detail {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kSlotsPerThread = 4;
constexpr size_t kItemStageBytes = 96 * 1024;            // shared-memory stage of the serial pass's operands
constexpr size_t kResolveSmemBytes = kItemStageBytes + kItemStageBytes / 2;   // + key and rank of the submission order

__device__ __forceinline__ int nonzero_bytes(uint32_t w) {
  // number of non-zero bytes in w (flags are 0 or 1, but any non-zero byte counts)
  const uint32_t t = (w | (w >> 1) | (w >> 2) | (w >> 3) | (w >> 4) | (w >> 5) | (w >> 6) | (w >> 7)) & 0x01010101u;
  return __popc(t);
}

// `cta` of `n_ctas` CTAs of kThreads threads run the body; dynamic shared memory holds at least
// items_cap * 16 bytes.
template <bool kCached>
__device__ __forceinline__ void resolve_body(const ResolveArgs& r, int cta, int n_ctas) {
  const Geometry& geo = r.geo;
  const swarm_cache& cache = r.cache;
  const int32_t* __restrict__ sel = r.sel;
  const int32_t* __restrict__ n_sel = r.n_sel;
  const int64_t* __restrict__ page_base = r.page_base;
  const int32_t* __restrict__ page2cluster = r.page2cluster;
  const int64_t* __restrict__ cluster_base = r.cluster_base;
  const uint32_t* __restrict__ replica_mask = r.replica_mask;
  const uint16_t* __restrict__ cluster_size = r.cluster_size;
  uint8_t* __restrict__ flags = r.flags;                 // (the overlapped tail picks one of two arrays below)
  unsigned* __restrict__ ticket = r.ticket;
  uint4* __restrict__ items = r.items;
  int32_t* __restrict__ uniq = r.uniq;
  uint8_t* __restrict__ queue_of = r.queue_of;
  int32_t* __restrict__ n_uniq = r.n_uniq;
  int32_t* __restrict__ queue_load = r.queue_load;
  uint32_t* __restrict__ status = r.status;
  const int items_cap = r.items_cap;
  (void)n_sel;
  extern __shared__ uint4 s_items[];                     // (mask, weight << 5, output slot, -) of the serial pass, when they fit
  __shared__ int2 s_seg[kWarps];                         // (start, length) of each warp's segment of the item list
  __shared__ int warp_cnt[kWarps];
  __shared__ int s_load[32];
  __shared__ unsigned s_classes;
  __shared__ unsigned s_item_m[32], s_item_w[32];
  __shared__ bool s_last;
  __shared__ int s_hits;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_hits = 0;
  pdl_launch_dependents();                               // the next kernel in the stream may be scheduled while this one runs
  const long long c_all = cluster_base[geo.B];           // an input table: not written by the previous kernel
  pdl_wait();                                            // the flags / the selection come from the previous kernel
  const int C = (int)min((long long)geo.Cmax, c_all);
  unsigned err = (c_all > geo.Cmax) ? SWARM_DEV_BAD_CLUSTER : 0u;
  // Overlapped tail: nothing after this kernel in the step waits for it, so it runs beside the next step's
  // scoring and selection.  That selection marks the other one of two flag arrays (the selection kernel counts
  // the steps it has marked; step n uses array (n - 1) & 1), and this kernel first lets the resolution of the
  // step before finish, which shares its outputs and scratch.
  unsigned step_no = 0u;
  if (r.tail_ctl != nullptr) {
    step_no = *reinterpret_cast<volatile unsigned*>(r.tail_ctl + kCtlMarked);
    flags += ((step_no - 1u) & 1u) * r.flags_alt;
    if (tid == 0 && !wait_at_least(r.tail_ctl + kCtlResolved, step_no - 1u)) err |= SWARM_DEV_TIMEOUT;
    __syncthreads();
  }

  SWARM_STAMP(status, 0);
  SWARM_KERNEL_BEGIN(status, 3);
  // ---- mark (skipped when the selection kernel already set the flags: sel == nullptr) -------------
  if (sel != nullptr) {
    const long long slots = (long long)geo.B * geo.Hq * geo.k;
    const long long base = (long long)cta * (kThreads * kSlotsPerThread) + tid;
    int p[kSlotsPerThread], bh[kSlotsPerThread];
    bool live[kSlotsPerThread];
#pragma unroll
    for (int u = 0; u < kSlotsPerThread; ++u) {
      const long long idx = base + (long long)u * kThreads;
      live[u] = idx < slots;
      bh[u] = live[u] ? (int)(idx / geo.k) : 0;
      p[u] = live[u] ? sel[idx] : -1;
    }
#pragma unroll
    for (int u = 0; u < kSlotsPerThread; ++u) {
      const long long idx = base + (long long)u * kThreads;
      live[u] = live[u] && (int)(idx - (long long)bh[u] * geo.k) < n_sel[bh[u]];
    }
    long long cid[kSlotsPerThread];
#pragma unroll
    for (int u = 0; u < kSlotsPerThread; ++u) {
      cid[u] = -1;
      if (!live[u]) continue;
      const int b = bh[u] / geo.Hq;
      const long long pb = page_base[b];
      if (p[u] < 0 || p[u] >= page_base[b + 1] - pb) { err |= SWARM_DEV_BAD_PAGE; continue; }
      const int c = page2cluster[pb + p[u]];
      const long long cb = cluster_base[b];
      if (c < 0 || c >= cluster_base[b + 1] - cb || cb + c >= C) { err |= SWARM_DEV_BAD_CLUSTER; continue; }
      cid[u] = cb + c;
    }
#pragma unroll
    for (int u = 0; u < kSlotsPerThread; ++u)
      if (cid[u] >= 0) flags[cid[u]] = 1;
  }
  if (err) atomicOr(status, err);
  err = 0u;

  // ---- which CTA is last? -------------------------------------------------------------------------
  if (n_ctas > 1) {
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(ticket, 1u) == (unsigned)n_ctas - 1u);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
  } else {
    __syncthreads();   // one CTA: its own marks are visible to all of its threads after the barrier
  }
  SWARM_STAMP_ANY_CTA(status, 1);

  // ---- compact (flags are read past L1: other CTAs wrote them) -------------------------------------
  // Every lane takes 4 flags (one word) at a time, so that up to 1024 clusters keep all 256 threads busy in a
  // single pass; warp w owns a contiguous range of words, which keeps the ids in ascending order.
  if (tid < 32) s_load[tid] = 0;
  if (tid == 0) s_classes = 0u;
  const int n_vec = (C + 3) / 4;                         // the flag array is padded to 16 bytes
  const int vec_per_warp = (n_vec + kWarps - 1) / kWarps;
  const int v_lo = min(n_vec, warp * vec_per_warp), v_hi = min(n_vec, v_lo + vec_per_warp);
  uint32_t* f1 = reinterpret_cast<uint32_t*>(flags);
  const unsigned valid_bits = geo.D == 32 ? 0xFFFFFFFFu : ((1u << geo.D) - 1u);
  const bool by_id = (geo.flags & SWARM_ORDER_BY_ID) != 0;
  const bool unit = (geo.flags & SWARM_UNIT_LOAD) != 0;

  // One word of flags with the replica masks and sizes of its 4 clusters, all requested in the same memory
  // round trip; a row that would cross the end of the tables is read entry by entry.
  struct Row {
    uint32_t f;
    uint4 mk;
    uint2 sz;
    uint32_t res;                                          // with cache state: the 4 clusters' resident bytes ...
    int4 fr;                                               // ... and their frequency counters
  };
  // vector loads of the cache state need its arrays aligned like the library's own tables
  const bool cache_vec = kCached && (reinterpret_cast<uintptr_t>(cache.resident) & 3u) == 0 &&
                         (reinterpret_cast<uintptr_t>(cache.freq) & 15u) == 0;
  const bool need_sz = !unit || (kCached && cache.score != nullptr);   // unit loads need no size table, Eq. 6 does
  auto load_row = [&](int v, bool with_flags) -> Row {
    Row r;
    r.f = 0u;
    r.mk = make_uint4(0u, 0u, 0u, 0u);
    r.sz = make_uint2(0u, 0u);
    r.res = 0u;
    r.fr = make_int4(0, 0, 0, 0);
    if (v < v_hi) {
      if (with_flags) r.f = __ldcg(f1 + v);
      if (v * 4 + 4 <= C) {
        r.mk = ldg_nc_v4(reinterpret_cast<const uint4*>(replica_mask + v * 4));
        if (need_sz) r.sz = __ldg(reinterpret_cast<const uint2*>(cluster_size + v * 4));
        if (kCached && cache_vec) {
          r.res = *reinterpret_cast<const uint32_t*>(cache.resident + v * 4);
          r.fr = *reinterpret_cast<const int4*>(cache.freq + v * 4);
        }
      }
      if (v * 4 + 4 > C || (kCached && !cache_vec)) {
        uint32_t* mk = &r.mk.x;
        uint32_t* sz = &r.sz.x;
        int* fr = &r.fr.x;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (v * 4 + j < C) {
            if (v * 4 + 4 > C) {
              mk[j] = replica_mask[v * 4 + j];
              if (need_sz) sz[j >> 1] |= (uint32_t)cluster_size[v * 4 + j] << (16 * (j & 1));
            }
            if (kCached) {
              r.res |= (cache.resident[v * 4 + j] != 0 ? 1u : 0u) << (8 * j);
              fr[j] = cache.freq[v * 4 + j];
            }
          }
        }
      }
    }
    return r;
  };

  // pass 1: count.  With one word per lane (up to 1024 clusters) the row stays in registers for pass 2.
  const bool one_vec = v_hi - v_lo <= 32;
  Row keep = load_row(v_lo + lane, true);
  int cnt = 0;
  if (one_vec) {
    cnt = nonzero_bytes(keep.f);
    if (kCached) {                                         // activated but resident: not fetched (Eq. 8)
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (((keep.f >> (8 * j)) & 0xFFu) && ((keep.res >> (8 * j)) & 0xFFu)) --cnt;
    }
  } else {
    for (int v0 = v_lo; v0 < v_hi; v0 += 128) {            // four independent loads in flight per lane
      uint32_t f[4], res[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + 32 * u + lane;
        f[u] = v < v_hi ? __ldcg(f1 + v) : 0u;
        res[u] = 0u;
        if (kCached && v < v_hi) {                         // the resident bytes travel with the flags
          if (cache_vec && v * 4 + 4 <= C) {
            res[u] = *reinterpret_cast<const uint32_t*>(cache.resident + v * 4);
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (v * 4 + j < C) res[u] |= (cache.resident[v * 4 + j] != 0 ? 1u : 0u) << (8 * j);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        cnt += nonzero_bytes(f[u]);
        if (kCached) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (((f[u] >> (8 * j)) & 0xFFu) && ((res[u] >> (8 * j)) & 0xFFu)) --cnt;
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
  if (lane == 0) warp_cnt[warp] = cnt;
  __syncthreads();
  int before = 0, n = 0;
  for (int w2 = 0; w2 < kWarps; ++w2) {
    if (w2 < warp) before += warp_cnt[w2];
    n += warp_cnt[w2];
  }
  // pass 2: place the ids, clear the flags, validate each cluster's replica mask and route the single-replica
  // ones.  The clusters that need the serial pass are packed, in id order, into this warp's segment of the
  // item list, which starts at the warp's first output position (a segment cannot outgrow the warp's ids).
  const bool staged = n <= items_cap;
  // submission order (optional): (replica class, queue) keys, kept in shared memory next to the items so that
  // the ordering pass at the end does not have to read the results back from global memory
  uint32_t* order_key = reinterpret_cast<uint32_t*>(s_items + items_cap);
  const bool order_keys_early = r.submit_order != nullptr && staged;
  const int seg_base = before;
  int seg_len = 0;
  unsigned classes = 0u;
  Row cur = keep;
  for (int v0 = v_lo; v0 < v_hi; v0 += 32) {
    const int v = v0 + lane;
    const Row nxt = load_row(v + 32, true);                // the next row travels while this one is processed
    const uint32_t f = cur.f;
    if (f) __stcg(f1 + v, 0u);                             // leave zeros for the next call
    unsigned fetch_bits = 0u, serial_bits = 0u;            // bit j: cluster v*4+j is fetched / needs the serial pass
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bool on = ((f >> (8 * j)) & 0xFFu) != 0u;
      bool fetch = on;
      if (kCached) {
        // cache bookkeeping of Sec. 5.2 for every cluster, activated or not
        const int c = v * 4 + j;
        if (v < v_hi && c < C) {
          const bool res = ((cur.res >> (8 * j)) & 0xFFu) != 0u;
          int fr = (&cur.fr.x)[j];
          if (on) ++fr; else if (res) --fr;
          if (on || res) cache.freq[c] = fr;
          if (cache.score != nullptr) {
            const float size_f = (float)(((&cur.sz.x)[j >> 1] >> (16 * (j & 1))) & 0xFFFFu);
            cache.score[c] = (float)fr * (cache.t_base + size_f * cache.t_transfer) / size_f;
          }
          if (on && res) { fetch = false; atomicAdd(&s_hits, 1); }
        }
      }
      const unsigned m = (&cur.mk.x)[j];
      const bool valid = m != 0u && !(m & ~valid_bits);
      fetch_bits |= (fetch ? 1u : 0u) << j;
      serial_bits |= (fetch && valid && (by_id || __popc(m) > 1) ? 1u : 0u) << j;
    }
    // one scan for both output positions: ids in the low half, serial items in the high half
    const int mine = __popc(fetch_bits) | (__popc(serial_bits) << 16);
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += t;
    }
    int pos = before + ((incl - mine) & 0xFFFF);
    int spos = seg_base + seg_len + ((incl - mine) >> 16);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if ((fetch_bits >> j) & 1u) {
        const int c = v * 4 + j, i = pos++;
        uniq[i] = c;
        const unsigned m = (&cur.mk.x)[j];
        const unsigned size = ((&cur.sz.x)[j >> 1] >> (16 * (j & 1))) & 0xFFFFu;
        const unsigned wgt = unit ? 1u : size;
        if ((serial_bits >> j) & 1u) {
          classes |= 1u << (__popc(m) - 1);
          const uint4 item = make_uint4(m, wgt << 5, (unsigned)i, 0u);   // what the serial pass needs
          if (staged) s_items[spos] = item;                // the serial pass then never waits on global memory
          else items[spos] = item;
          ++spos;
        } else if (m == 0u || (m & ~valid_bits)) {
          err |= SWARM_DEV_BAD_REPLICA;
          queue_of[i] = 0xFF;
          if (order_keys_early) order_key[i] = 0xFFFFFFFFu;
        } else {
          const int qd = __ffs(m) - 1;                     // a single replica: nothing to decide
          queue_of[i] = (uint8_t)qd;
          atomicAdd(&s_load[qd], (int)wgt);
          if (order_keys_early) order_key[i] = 32u + (unsigned)qd;
        }
      }
    }
    const int tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
    before += tot & 0xFFFF;
    seg_len += tot >> 16;
    cur = nxt;
  }
  if (lane == 0) s_seg[warp] = make_int2(seg_base, seg_len);
  if (staged)                                              // in shared memory the serial pass walks one flat list:
    for (int k = seg_base + seg_len + lane; k < before; k += 32)   // blank the rest of this warp's slots
      s_items[k] = make_uint4(0u, 0u, 0u, 0u);
  SWARM_STAMP_ANY_CTA(status, 2);
  if (classes) atomicOr(&s_classes, classes);
  if (err) atomicOr(status, err);
  __syncthreads();
  SWARM_STAMP_ANY_CTA(status, 3);

  // ---- the ordered greedy, one warp ------------------------------------------------------------------
  // It walks the warps' segments in order, which is id order (from shared memory: all of them as one list,
  // the unused slots blank).  32 clusters at a time are staged in shared
  // memory so that the serial loop is a plain counted loop whose operands are fetched one step ahead of
  // the dependent chain select -> redux.min -> compare -> add.
  if (warp == 0) {
    unsigned L = ((unsigned)s_load[lane] << 5) | (unsigned)lane;     // (load, queue id) in one comparable word
    const unsigned todo = by_id ? 1u : (s_classes & ~1u);
    // Common case: everything the serial pass has to visit is of one replica class (or the order is by id) and
    // sits in shared memory.  The warps' segments then hold exactly the visit order, densely, and the pass is a
    // flat loop over each segment: no per-batch staging, the next item fetched while the current one is decided;
    // lane r of every group of 32 keeps the queue of the group's r-th cluster.
    const bool flat = staged && __popc(todo) <= 1;
    if (flat && todo != 0u) {
      for (int w2 = 0; w2 < kWarps; ++w2) {
        const int base = s_seg[w2].x, len = s_seg[w2].y;
        for (int g0 = 0; g0 < len; g0 += 32) {
          const int cnt_g = min(32, len - g0);
          unsigned my_q = 0u;
          uint4 it = s_items[base + g0];
          for (int rr = 0; rr < cnt_g; ++rr) {
            const uint4 nx = s_items[min(base + g0 + rr + 1, items_cap - 1)];
            const unsigned key = ((it.x >> lane) & 1u) ? L : 0xFFFFFFFFu;
            const unsigned best = __reduce_min_sync(0xFFFFFFFFu, key);
            if (L == best) L += it.y;
            if (lane == rr) my_q = best & 31u;
            it = nx;
          }
          if (lane < cnt_g) s_items[base + g0 + lane].w = my_q;
        }
      }
    }
    for (int R = by_id ? 0 : 2; R <= (by_id ? 0 : geo.D) && !flat; ++R) {
      if (!by_id && !((todo >> (R - 1)) & 1u)) continue;
      for (int w2 = 0; w2 < (staged ? 1 : kWarps); ++w2) {
        const int base = staged ? 0 : s_seg[w2].x, len = staged ? n : s_seg[w2].y;
        // (mask, weight, output slot) of 32 clusters per step, fetched two steps ahead of their use
        auto item_at = [&](int k) -> uint4 {
          return k >= len ? make_uint4(0u, 0u, 0u, 0u) : (staged ? s_items[base + k] : items[base + k]);
        };
        uint4 pre0 = item_at(lane);
        uint4 pre1 = item_at(32 + lane);
        for (int k0 = 0; k0 < len; k0 += 32) {
          const unsigned m = pre0.x, wgt = pre0.y, slot = pre0.z;
          pre0 = pre1;
          pre1 = item_at(k0 + 64 + lane);
          const bool mine = m != 0u && (by_id || __popc(m) == R);
          const unsigned pending = __ballot_sync(0xFFFFFFFFu, mine);
          const int cnt_p = __popc(pending);
          if (cnt_p == 0) continue;
          const int rank = __popc(pending & ((1u << lane) - 1u));
          if (mine) { s_item_m[rank] = m; s_item_w[rank] = wgt; }
          __syncwarp();
          unsigned my_q = 0u;
          unsigned mm = s_item_m[0], ww = s_item_w[0];
          for (int r = 0; r < cnt_p; ++r) {
            const unsigned mm_next = s_item_m[min(r + 1, 31)], ww_next = s_item_w[min(r + 1, 31)];
            const unsigned key = ((mm >> lane) & 1u) ? L : 0xFFFFFFFFu;
            const unsigned best = __reduce_min_sync(0xFFFFFFFFu, key);   // ~55 cycles per cluster end to end;
            if (L == best) L += ww;                                      // shuffle-, ballot- and register-based
            if (rank == r) my_q = best & 31u;                            // variants measured slower on sm_100
            mm = mm_next;
            ww = ww_next;
          }
          // From shared memory the choice goes back into the item and is written out after the pass: a global
          // store issued while the attention kernel starts or retires was measured to hold this warp for 2 us.
          if (mine) {
            if (staged) s_items[base + k0 + lane].w = my_q;
            else queue_of[slot] = (uint8_t)my_q;
          }
          __syncwarp();
        }
      }
    }
    SWARM_STAMP_ANY_CTA(status, 4);
    SWARM_KERNEL_END(status, 3);
    if (staged) {
      __syncwarp();
      for (int k = lane; k < n; k += 32) {
        const uint4 item = s_items[k];
        if (item.x != 0u) {
          queue_of[item.z] = (uint8_t)item.w;
          if (order_keys_early) order_key[item.z] = (by_id ? 0u : (unsigned)__popc(item.x) * 32u) + item.w;
        }
      }
    }
    if (lane < geo.D) queue_load[lane] = (int)(L >> 5);
    if (lane < geo.D && r.host.queue_load_h != nullptr) r.host.queue_load_h[lane] = (int)(L >> 5);
    if (lane == 0 && r.host.n_uniq_h != nullptr) *r.host.n_uniq_h = n;
    if (lane == 0) {
      *n_uniq = n;
      if (kCached && cache.n_hit != nullptr) *cache.n_hit = s_hits;
      if (n_ctas > 1) *ticket = 0u;                               // ready for the next call
    }
  }

  // ---- batched submission order (Sec. 5.1, last paragraph; only when the caller attached the output) ------
  // Bucket q holds its clusters in assignment order: (replica count ascending, position in uniq ascending), or
  // position alone under SWARM_ORDER_BY_ID.  Batch r takes the r-th cluster of every bucket that has one, in
  // queue order.  Three steps: every thread forms the (class, queue) key of its clusters; one warp walks the
  // keys in position order and ranks each cluster inside its (class, queue) group; every thread then turns
  // (class, queue, rank) into the cluster's place in the submission order with the bucket sizes alone.
  if (r.submit_order != nullptr) {
    __shared__ int s_group[33 * 32];                       // clusters per (class, queue); then the start of each group in its bucket
    __shared__ int s_bucket[32];                           // clusters per queue
    uint32_t* key_of = staged ? reinterpret_cast<uint32_t*>(s_items + items_cap) : reinterpret_cast<uint32_t*>(items);
    uint32_t* rank_of = key_of + (staged ? items_cap : n);
    for (int i = tid; i < 33 * 32; i += kThreads) s_group[i] = 0;
    __syncthreads();                                       // also: every queue_of entry is written
    if (!order_keys_early) {
      // from global memory: four clusters per thread and turn, so that the two dependent reads of each
      // (its id, then that id's replica mask) overlap with the others'
      for (int i0 = tid; i0 < n; i0 += 4 * kThreads) {
        unsigned q[4], m[4];
        int id[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kThreads;
          q[u] = i < n ? __ldcg(queue_of + i) : 0xFFu;
          id[u] = (i < n && !by_id) ? __ldcg(uniq + i) : -1;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) m[u] = id[u] >= 0 ? replica_mask[id[u]] : 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kThreads;
          // clusters with a bad replica mask are not submitted
          if (i < n) key_of[i] = q[u] >= 32u ? 0xFFFFFFFFu : ((unsigned)__popc(m[u]) * 32u + q[u]);
        }
      }
    }
    __syncthreads();
    // The walk is one warp's; its keys come from shared memory.  When the keys live in global memory (more
    // clusters than the item stage holds, which then is free) they are brought in by all threads, a stage at a time.
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(s_items);
    const int walk_cap = staged ? max(n, 1) : (int)(kResolveSmemBytes / 4);
    for (int c0 = 0; c0 < n; c0 += walk_cap) {
      const int m_keys = min(walk_cap, n - c0);
      if (!staged) {
        for (int i = tid; i < m_keys; i += kThreads) s_keys[i] = key_of[c0 + i];
        __syncthreads();
      }
      if (warp == 0) {
        const unsigned lt = (1u << lane) - 1u;
        for (int i0 = c0; i0 < c0 + m_keys; i0 += 32) {
          const int i = i0 + lane;
          const uint32_t key = i >= c0 + m_keys ? 0xFFFFFFFFu : (staged ? key_of[i] : s_keys[i - c0]);
          const unsigned same = __match_any_sync(0xFFFFFFFFu, key);
          if (key != 0xFFFFFFFFu) {
            rank_of[i] = (uint32_t)(s_group[key] + __popc(same & lt));
          }
          __syncwarp();
          if (key != 0xFFFFFFFFu && (same & lt) == 0u) s_group[key] += __popc(same);   // the group's first lane
          __syncwarp();
        }
      }
      __syncthreads();
    }
    if (tid < 32) {                                        // bucket sizes; group counts -> group starts
      int run = 0;
      for (int c = 0; c <= 32; ++c) {
        const int t = s_group[c * 32 + tid];
        s_group[c * 32 + tid] = run;
        run += t;
      }
      s_bucket[tid] = run;
    }
    __syncthreads();
    int submitted = 0, rounds = 0;
    for (int q = 0; q < geo.D; ++q) {
      submitted += s_bucket[q];
      rounds = max(rounds, s_bucket[q]);
    }
    for (int i0 = tid; i0 < n; i0 += 4 * kThreads) {       // four per turn: the reads of key and rank overlap
      uint32_t key4[4], rank4[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kThreads;
        key4[u] = i < n ? key_of[i] : 0xFFFFFFFFu;
        rank4[u] = i < n ? rank_of[i] : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t key = key4[u];
        if (key == 0xFFFFFFFFu) continue;
        const int q = (int)(key & 31u);
        const int depth = s_group[key] + (int)rank4[u];    // position inside bucket q
        int pos = 0;
        for (int q2 = 0; q2 < geo.D; ++q2) pos += min(s_bucket[q2], depth) + ((q2 < q && s_bucket[q2] > depth) ? 1 : 0);
        r.submit_order[pos] = i0 + u * kThreads;
      }
    }
    if (tid == 0 && r.submit_info != nullptr) {
      r.submit_info[0] = rounds;
      r.submit_info[1] = submitted;
    }
  }
  if (r.host.done_h != nullptr) {                          // host step: the resolution's results are in host memory
    __syncthreads();
    if (tid == 0) host_arrive(r.host);
  }
  if (r.tail_ctl != nullptr) {                             // overlapped tail: this step's resolution has finished
    __syncthreads();
    if (tid == 0) st_release(r.tail_ctl + kCtlResolved, step_no);
  }
}

}  // namespace resolve_detail
}  // namespace swarm
