// Cluster-granular selection through the medoid index (Sec. 4.2, Tier 1 (1)): every cluster is represented
// by its medoid, the medoid is scored against the query, the best clusters are retrieved whole (Sec. 4.1:
// clusters are the retrieval unit) and all of their pages are attended.
//
// The scoring and the top-k are the page kernels run over a context whose "pages" are the clusters: the
// index holds the key summary of each cluster's medoid page, one row per cluster, requests back to back
// exactly like cluster_base.  What this file adds is the glue around them:
//   medoid_rows_kernel     index build: copy the summary rows of the medoid pages into the index
//   cluster_len_kernel     pseudo context lengths (clusters of the request x page size) for the page kernels
//   expand_clusters_kernel selected clusters -> per-head bitmap of their member pages plus the local window (what
//                          the attention kernel reads) and the cluster flags (what the resolve kernel reads)
#include "swarm_internal.cuh"

namespace swarm {
namespace {

// One CTA per cluster: 2 * d bf16 per KV head = 512 bytes per head, 16-byte vectors.
__global__ void __launch_bounds__(128)
medoid_rows_kernel(Geometry geo, const uint16_t* __restrict__ ksum, const int64_t* __restrict__ page_base,
                   const int64_t* __restrict__ cluster_base, const int32_t* __restrict__ medoid_page,
                   uint16_t* __restrict__ medoid_ksum, uint32_t* __restrict__ status) {
  const long long c = blockIdx.x;
  if (c >= cluster_base[geo.B]) return;
  int b = 0;                                              // request of cluster c (binary search over cluster_base)
  {
    int lo = 0, hi = geo.B;
    while (hi - lo > 1) {
      const int mid = (lo + hi) / 2;
      if (cluster_base[mid] <= c) lo = mid; else hi = mid;
    }
    b = lo;
  }
  const long long pb = page_base[b];
  const int p = medoid_page[c];
  const int vec_per_row = geo.Hkv * 2 * kHeadDim / 8;
  uint4* dst = reinterpret_cast<uint4*>(medoid_ksum + c * geo.Hkv * 2 * kHeadDim);
  if (p < 0 || p >= page_base[b + 1] - pb) {
    if (threadIdx.x == 0) atomicOr(status, SWARM_DEV_BAD_PAGE);
    for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) dst[i] = make_uint4(0, 0, 0, 0);
    return;
  }
  const uint16_t* src = ksum + (pb + p) * geo.Hkv * 2 * kHeadDim;
  for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) dst[i] = ldg_nc_v4(src + (long long)i * 8);
}

__global__ void cluster_len_kernel(int B, int S, const int64_t* __restrict__ cluster_base, int32_t* __restrict__ len) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) len[b] = (int32_t)min((long long)(cluster_base[b + 1] - cluster_base[b]) * S, 0x7FFFFFFFLL);
}

// One CTA per (request, query head).  The head's bitmap row is assembled in shared memory (bit p % 8 of byte
// p / 8, the layout the selection kernel writes) and stored whole, so rows need no clearing between steps.
__global__ void __launch_bounds__(256)
expand_clusters_kernel(Geometry geo, int k_c, int pitch, const int32_t* __restrict__ sel_c,
                       const int32_t* __restrict__ n_sel_c, const int64_t* __restrict__ cluster_base,
                       const int64_t* __restrict__ cluster_page_ptr, const int32_t* __restrict__ cluster_pages,
                       const int32_t* __restrict__ ctx_len, uint8_t* __restrict__ selmap, uint8_t* __restrict__ flags,
                       uint32_t* __restrict__ status, const int64_t* __restrict__ entry_base, long long n_member_entries,
                       const int64_t* __restrict__ page_base, const int32_t* __restrict__ page2cluster) {
  extern __shared__ uint32_t s_row[];
  const int bh = blockIdx.x, b = bh / geo.Hq;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = pages_of(ctx_len[b], geo.S);               // inputs: read before the wait
  const long long cb = cluster_base[b], cn = cluster_base[b + 1];
  for (int i = tid; i < pitch / 4; i += blockDim.x) s_row[i] = 0u;
  pdl_wait();                                               // the cluster selection comes from the previous kernel
  __syncthreads();
  const int n = min(n_sel_c[bh], k_c);
  unsigned err = 0u;
  for (int j = warp; j < n; j += blockDim.x / 32) {         // one warp per selected cluster
    const int c = sel_c[(long long)bh * k_c + j];
    if (c < 0 || c >= cn - cb || cb + c >= geo.Cmax) { err |= SWARM_DEV_BAD_CLUSTER; continue; }
    const long long e0 = cluster_page_ptr[cb + c], e1 = cluster_page_ptr[cb + c + 1];
    if (e0 < 0 || e1 < e0 || e1 > n_member_entries) { err |= SWARM_DEV_BAD_CLUSTER; continue; }   // corrupt member offsets
    // what gets scheduled: the cluster as a whole, or (entry level) each of its pages on its own
    if (lane == 0 && entry_base == nullptr) flags[cb + c] = 1;
    for (long long e = e0 + lane; e < e1; e += 32) {
      const int p = cluster_pages[e];
      if (p < 0 || p >= P || p >= pitch * 8) {
        err |= SWARM_DEV_BAD_PAGE;
      } else {
        atomicOr(&s_row[p >> 5], 1u << (p & 31));
        if (entry_base != nullptr) {
          const long long unit = entry_base[b] + p;
          if (unit < geo.Cmax) flags[unit] = 1;
          else err |= SWARM_DEV_BAD_CLUSTER;
        }
      }
    }
  }
  // the local window (Sec. 4.2, Tier 1 (2)): the last W pages of the request join every head's set and are
  // scheduled like the members of the selected clusters
  for (int p = max(0, P - geo.W) + tid; p < P && p < pitch * 8; p += blockDim.x) {
    atomicOr(&s_row[p >> 5], 1u << (p & 31));
    if (entry_base != nullptr) {
      const long long unit = entry_base[b] + p;
      if (unit < geo.Cmax) flags[unit] = 1;
      else err |= SWARM_DEV_BAD_CLUSTER;
    } else {
      const int c = page2cluster[page_base[b] + p];
      if (c < 0 || c >= cn - cb || cb + c >= geo.Cmax) err |= SWARM_DEV_BAD_CLUSTER;
      else flags[cb + c] = 1;
    }
  }
  if (err) atomicOr(status, err);
  __syncthreads();
  uint32_t* row = reinterpret_cast<uint32_t*>(selmap + (long long)bh * pitch);
  for (int i = tid; i < pitch / 4; i += blockDim.x) row[i] = s_row[i];
}

}  // namespace

cudaError_t configure_medoid() {
  return cudaFuncSetAttribute(expand_clusters_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxExpandRowBytes);
}

cudaError_t launch_medoid_rows(const Geometry& geo, const uint16_t* ksum, const int64_t* page_base,
                               const int64_t* cluster_base, const int32_t* medoid_page, uint16_t* medoid_ksum,
                               uint32_t* status, cudaStream_t st) {
  medoid_rows_kernel<<<dim3((unsigned)geo.Cmax), dim3(128), 0, st>>>(geo, ksum, page_base, cluster_base, medoid_page,
                                                                    medoid_ksum, status);
  return cudaGetLastError();
}

cudaError_t launch_cluster_len(const Geometry& geo, const int64_t* cluster_base, int32_t* len, cudaStream_t st) {
  cluster_len_kernel<<<dim3((geo.B + 127) / 128), dim3(128), 0, st>>>(geo.B, geo.S, cluster_base, len);
  return cudaGetLastError();
}

cudaError_t launch_expand_clusters(const Geometry& geo, int k_c, const int32_t* sel_c, const int32_t* n_sel_c,
                                   const int64_t* cluster_base, const int64_t* cluster_page_ptr,
                                   const int32_t* cluster_pages, const int32_t* ctx_len, uint8_t* selmap, uint8_t* flags,
                                   uint32_t* status, cudaStream_t st, bool overlap, const int64_t* entry_base,
                                   long long n_member_entries, const int64_t* page_base, const int32_t* page2cluster) {
  const int pitch = selmap_pitch_bytes(geo.Pmax);
  return launch_pdl(expand_clusters_kernel, dim3((unsigned)(geo.B * geo.Hq)), dim3(256), (size_t)pitch, st, overlap, geo,
                    k_c, pitch, sel_c, n_sel_c, cluster_base, cluster_page_ptr, cluster_pages, ctx_len, selmap, flags,
                    status, entry_base, n_member_entries, page_base, page2cluster);
}

}  // namespace swarm
