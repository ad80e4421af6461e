// Stage 3: cluster resolution, global merge and load-balanced bucket scheduling (Eq. 8 without the
// already-resident term; Sec. 5.1).  One CTA: the stage is a few thousand integer operations with a
// serial tail, and it runs beside the attention kernels, off the critical path.
//
//   mark     every selected (request, page) -> global cluster id; flag[id] = 1.  Idempotent byte
//            stores: concurrent writers store the same value, so no atomics are needed.
//   compact  ordered ballot/popc compaction of the flags -> uniq[] ascending by id.
//   route    single-replica clusters go to their queue (integer histogram, order-free).  Clusters
//            with R >= 2 replicas are visited by (R ascending, id ascending) by one warp: lane j
//            owns load[j]; one redux.min over (load << 5 | lane) restricted to the replica mask
//            picks the least-loaded replica with ties to the lowest queue id.
//            Under SWARM_ORDER_BY_ID the same warp visits every cluster in id order instead.
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kResolveThreads = 1024;
constexpr int kResolveWarps = kResolveThreads / 32;
constexpr int kSmemFlagBytes = 192 * 1024;

template <bool kSmemFlags>
__global__ void __launch_bounds__(kResolveThreads)
resolve_kernel(Geometry geo, const int32_t* __restrict__ sel, const int32_t* __restrict__ n_sel,
               const int64_t* __restrict__ page_base, const int32_t* __restrict__ page2cluster,
               const int64_t* __restrict__ cluster_base, const uint32_t* __restrict__ replica_mask,
               const uint16_t* __restrict__ cluster_size, uint8_t* __restrict__ flags_ws,
               int32_t* __restrict__ uniq, uint8_t* __restrict__ queue_of, int32_t* __restrict__ n_uniq,
               int32_t* __restrict__ queue_load, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t sflags[];
  __shared__ int warp_cnt[kResolveWarps];
  __shared__ int s_load[32];
  __shared__ unsigned s_classes;
  __shared__ int s_total;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint8_t* flags = kSmemFlags ? sflags : flags_ws;
  const long long c_all = cluster_base[geo.B];
  const int C = (int)min((long long)geo.Cmax, c_all);
  unsigned err = (c_all > geo.Cmax) ? SWARM_DEV_BAD_CLUSTER : 0u;

  // clear (the flag array is padded to a multiple of 16 bytes)
  {
    uint4* f4 = reinterpret_cast<uint4*>(flags);
    for (int i = tid; i < (C + 15) / 16; i += kResolveThreads) f4[i] = make_uint4(0, 0, 0, 0);
  }
  if (tid < 32) s_load[tid] = 0;
  if (tid == 0) s_classes = 0u;
  __syncthreads();

  // mark
  const long long slots = (long long)geo.B * geo.Hq * geo.k;
  for (long long idx = tid; idx < slots; idx += kResolveThreads) {
    const int bh = (int)(idx / geo.k), j = (int)(idx % geo.k);
    if (j >= n_sel[bh]) continue;
    const int b = bh / geo.Hq;
    const int p = sel[idx];
    const long long pb = page_base[b];
    if (p < 0 || p >= page_base[b + 1] - pb) { err |= SWARM_DEV_BAD_PAGE; continue; }
    const int c = page2cluster[pb + p];
    const long long cb = cluster_base[b];
    if (c < 0 || c >= cluster_base[b + 1] - cb || cb + c >= C) { err |= SWARM_DEV_BAD_CLUSTER; continue; }
    flags[cb + c] = 1;
  }
  __syncthreads();

  // compact: warp w owns the contiguous span [w*seg, (w+1)*seg)
  const int seg = (((C + kResolveWarps - 1) / kResolveWarps) + 31) & ~31;
  const int lo = min(C, warp * seg), hi = min(C, lo + seg);
  int cnt = 0;
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    cnt += __popc(__ballot_sync(0xFFFFFFFFu, i < hi && flags[i]));
  }
  if (lane == 0) warp_cnt[warp] = cnt;
  __syncthreads();
  int before = 0;
  for (int w2 = 0; w2 < warp; ++w2) before += warp_cnt[w2];
  if (tid == kResolveThreads - 1) s_total = before + cnt;
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    const bool f = i < hi && flags[i];
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, f);
    if (f) uniq[before + __popc(bal & lt_mask)] = i;
    before += __popc(bal);
  }
  __syncthreads();   // uniq[] (global) written by this CTA is visible to it after the barrier
  const int n = s_total;
  const unsigned valid_bits = geo.D == 32 ? 0xFFFFFFFFu : ((1u << geo.D) - 1u);
  const bool by_id = (geo.flags & SWARM_ORDER_BY_ID) != 0;
  const bool unit = (geo.flags & SWARM_UNIT_LOAD) != 0;

  // validate masks, route single-replica clusters, record which replica counts occur
  unsigned classes = 0u;
  for (int i = tid; i < n; i += kResolveThreads) {
    const int c = uniq[i];
    const unsigned m = replica_mask[c];
    if (m == 0u || (m & ~valid_bits)) { err |= SWARM_DEV_BAD_REPLICA; queue_of[i] = 0xFF; continue; }
    const int R = __popc(m);
    if (R == 1 && !by_id) {
      const int qd = __ffs(m) - 1;
      queue_of[i] = (uint8_t)qd;
      atomicAdd(&s_load[qd], unit ? 1 : (int)cluster_size[c]);
    } else {
      classes |= 1u << (R - 1);
    }
  }
  if (classes) atomicOr(&s_classes, classes);
  if (err) atomicOr(status, err);
  __syncthreads();

  if (warp == 0) {
    unsigned load = (unsigned)s_load[lane];
    const unsigned todo = by_id ? 1u : (s_classes & ~1u);   // one sweep by id, or one sweep per replica count
    for (int R = by_id ? 0 : 2; R <= (by_id ? 0 : geo.D); ++R) {
      if (!by_id && !((todo >> (R - 1)) & 1u)) continue;
      for (int i0 = 0; i0 < n; i0 += 32) {
        const int i = i0 + lane;
        unsigned m = 0u, wgt = 0u;
        if (i < n) {
          const int c = uniq[i];
          m = replica_mask[c];
          if (m == 0u || (m & ~valid_bits)) m = 0u;
          wgt = unit ? 1u : (unsigned)cluster_size[c];
        }
        const bool mine = m != 0u && (by_id || __popc(m) == R);
        unsigned pending = __ballot_sync(0xFFFFFFFFu, mine);
        int my_q = 0;
        while (pending) {
          const int src = __ffs(pending) - 1;
          pending &= pending - 1;
          const unsigned mm = __shfl_sync(0xFFFFFFFFu, m, src);
          const unsigned ww = __shfl_sync(0xFFFFFFFFu, wgt, src);
          const unsigned key = ((mm >> lane) & 1u) ? ((load << 5) | (unsigned)lane) : 0xFFFFFFFFu;
          const int qd = (int)(__reduce_min_sync(0xFFFFFFFFu, key) & 31u);
          if (lane == qd) load += ww;
          if (lane == src) my_q = qd;
        }
        if (mine) queue_of[i] = (uint8_t)my_q;
      }
    }
    if (lane < geo.D) queue_load[lane] = (int)load;
    if (lane == 0) *n_uniq = n;
  }
}

}  // namespace

cudaError_t configure_resolve() {
  return cudaFuncSetAttribute(resolve_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemFlagBytes);
}

cudaError_t launch_resolve(const Geometry& geo, const int32_t* sel, const int32_t* n_sel, const int64_t* page_base,
                           const int32_t* page2cluster, const int64_t* cluster_base, const uint32_t* replica_mask,
                           const uint16_t* cluster_size, uint8_t* flags_ws, int32_t* uniq, uint8_t* queue_of,
                           int32_t* n_uniq, int32_t* queue_load, uint32_t* status, cudaStream_t st) {
  const size_t flag_bytes = ((size_t)geo.Cmax + 15) & ~(size_t)15;
  if (flag_bytes <= (size_t)kSmemFlagBytes)
    resolve_kernel<true><<<1, kResolveThreads, flag_bytes, st>>>(geo, sel, n_sel, page_base, page2cluster,
                                                                 cluster_base, replica_mask, cluster_size, flags_ws,
                                                                 uniq, queue_of, n_uniq, queue_load, status);
  else
    resolve_kernel<false><<<1, kResolveThreads, 0, st>>>(geo, sel, n_sel, page_base, page2cluster, cluster_base,
                                                         replica_mask, cluster_size, flags_ws, uniq, queue_of,
                                                         n_uniq, queue_load, status);
  return cudaGetLastError();
}

}  // namespace swarm
