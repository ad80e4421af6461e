// Stage 3 as a kernel of its own (swarm_resolve_clusters); the algorithm is in resolve_body.cuh.
#define SWARM_TRACE_FILE 3
#include "resolve_body.cuh"

namespace swarm {
namespace {

using namespace resolve_detail;

template <bool kCached>
__global__ void __launch_bounds__(kThreads) resolve_kernel(ResolveArgs r) {
  resolve_body<kCached>(r, (int)blockIdx.x, (int)gridDim.x);
}

}  // namespace

cudaError_t configure_resolve() {
  // static + dynamic shared memory exceed the 48 KiB that needs no opt-in
  cudaError_t e = cudaFuncSetAttribute(resolve_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kResolveSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(resolve_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kResolveSmemBytes);
  return e;
}

ResolveArgs make_resolve_args(const Geometry& geo, const int32_t* sel, const int32_t* n_sel, const int64_t* page_base,
                              const int32_t* page2cluster, const int64_t* cluster_base, const uint32_t* replica_mask,
                              const uint16_t* cluster_size, uint8_t* flags_ws, unsigned* ticket, uint4* items,
                              int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq, int32_t* queue_load, uint32_t* status,
                              const swarm_cache* cache, int32_t* submit_order, int32_t* submit_info) {
  ResolveArgs r{};
  r.submit_order = submit_order;
  r.submit_info = submit_info;
  r.geo = geo;
  r.has_cache = cache != nullptr;
  if (cache != nullptr) r.cache = *cache;
  r.sel = sel; r.n_sel = n_sel; r.page_base = page_base; r.page2cluster = page2cluster; r.cluster_base = cluster_base;
  r.replica_mask = replica_mask; r.cluster_size = cluster_size; r.flags = flags_ws; r.ticket = ticket; r.items = items;
  r.uniq = uniq; r.queue_of = queue_of; r.n_uniq = n_uniq; r.queue_load = queue_load; r.status = status;
  r.items_cap = (int)(kItemStageBytes / sizeof(uint4));
  return r;
}

cudaError_t launch_resolve(const ResolveArgs& r, cudaStream_t st, bool overlap) {
  const long long slots = (long long)r.geo.B * r.geo.Hq * r.geo.k;
  const unsigned grid =
      r.sel == nullptr ? 1u : (unsigned)((slots + kThreads * kSlotsPerThread - 1) / (kThreads * kSlotsPerThread));
  // The dynamic shared memory stages the serial pass's operands.
  if (r.has_cache)
    return launch_pdl(resolve_kernel<true>, dim3(grid), dim3(kThreads), kResolveSmemBytes, st, overlap, r);
  return launch_pdl(resolve_kernel<false>, dim3(grid), dim3(kThreads), kResolveSmemBytes, st, overlap, r);
}

}  // namespace swarm
