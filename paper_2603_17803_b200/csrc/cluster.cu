// Algorithm 1: offline co-activation clustering on a given distance matrix (Sec. 4.1, Steps 3 and 4).
//
//   density_kernel   rho[i] = #{ j != i : D[i][j] <= tau }  -- one warp per row, 16-byte loads; the only part
//                    that touches the whole n x n matrix, bound by HBM bandwidth (4 n^2 bytes read once)
//   queue_kernel     medoid queue: entries by (rho descending, index ascending), each entry's place found by
//                    counting the entries that precede it (n^2 integer compares on data held in shared memory)
//   expand_kernel    one CTA walks the queue.  For an uncovered medoid m: the candidates { e != m : D[m][e] <= tau }
//                    are compacted in index order, placed by (distance, index) rank, and then joined greedily.
//                    Between two joins neither the running sums nor the bound tau * |C| change, so the next
//                    candidate to join is the first one in queue order whose sum passes: a block-wide minimum
//                    finds it, and the number of dependent steps is the cluster size, not the candidate count.
//                    A candidate's sum is a plain fp32 accumulation in joining order over D[member][candidate],
//                    so every decision is the one a sequential fp32 walk takes.
// Covered entries remain candidates of later medoids: an entry can sit in several clusters (the paper's replicas).
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kExpandThreads = 1024;

__global__ void __launch_bounds__(256)
density_kernel(const float* __restrict__ dist, int n, float tau, int32_t* __restrict__ rho) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
  if (row >= n) return;
  const float* r = dist + (long long)row * n;
  int cnt = 0;
  if ((n & 3) == 0) {                                     // rows are 16-byte aligned
    for (int j = lane * 4; j < n; j += 128) {
      const uint4 v = ldg_nc_v4(r + j);
      cnt += (__uint_as_float(v.x) <= tau && j != row) + (__uint_as_float(v.y) <= tau && j + 1 != row) +
             (__uint_as_float(v.z) <= tau && j + 2 != row) + (__uint_as_float(v.w) <= tau && j + 3 != row);
    }
  } else {
    for (int j = lane; j < n; j += 32) cnt += (__ldg(r + j) <= tau && j != row);
  }
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
  if (lane == 0) rho[row] = cnt;
}

// queue[place] = i with place = #{ j : rho[j] > rho[i] or (rho[j] == rho[i] and j < i) }
__global__ void __launch_bounds__(256)
queue_kernel(const int32_t* __restrict__ rho, int n, int32_t* __restrict__ queue) {
  __shared__ int s_rho[2048];
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int mine = i < n ? rho[i] : 0;
  int place = 0;
  for (int base = 0; base < n; base += 2048) {
    __syncthreads();
    for (int t = threadIdx.x; t < 2048 && base + t < n; t += blockDim.x) s_rho[t] = rho[base + t];
    __syncthreads();
    const int lim = min(2048, n - base);
    for (int t = 0; t < lim; ++t) {
      const int other = s_rho[t];
      place += (other > mine) || (other == mine && base + t < i);
    }
  }
  if (i < n) queue[place] = i;
}

struct ExpandArgs {
  const float* dist;
  int n;
  float tau;
  const int32_t* queue;
  // scratch, n entries each
  int32_t* cand_raw;     // candidates in index order
  int32_t* cand;         // candidates in (distance, index) order
  float* sum;            // running sum of the candidate's distances to the members
  uint8_t* covered;
  // outputs
  int32_t* ptr;
  int32_t* members;
  long long members_cap;
  int32_t* medoid;
  int32_t* n_clusters;
  int32_t* dev_status;   // 0 ok, 1 members_cap too small
};

__global__ void __launch_bounds__(kExpandThreads) expand_kernel(ExpandArgs a) {
  __shared__ int s_warp[32];
  __shared__ int s_total, s_next, s_newly;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = a.n;
  pdl_wait();                                             // the queue comes from the previous kernel
  for (int i = tid; i < n; i += kExpandThreads) a.covered[i] = 0;
  if (tid == 0) a.ptr[0] = 0;
  __syncthreads();
  int n_cov = 0, n_clu = 0;
  long long fill = 0;
  bool overflow = false;
  for (int qi = 0; qi < n && n_cov < n && !overflow; ++qi) {
    const int m = a.queue[qi];
    if (a.covered[m]) continue;                           // uniform: every thread reads the same byte
    const float* row_m = a.dist + (long long)m * n;

    // ---- candidates in index order (ordered compaction, chunks of kExpandThreads entries) ----
    int n_cand = 0;
    for (int base = 0; base < n; base += kExpandThreads) {
      const int e = base + tid;
      const bool is_cand = e < n && e != m && row_m[e] <= a.tau;
      const unsigned bal = __ballot_sync(0xFFFFFFFFu, is_cand);
      if (lane == 0) s_warp[warp] = __popc(bal);
      __syncthreads();
      int before = 0, total = 0;
      for (int w = 0; w < kExpandThreads / 32; ++w) {
        const int c = s_warp[w];
        if (w < warp) before += c;
        total += c;
      }
      if (is_cand) a.cand_raw[n_cand + before + __popc(bal & ((1u << lane) - 1u))] = e;
      n_cand += total;
      __syncthreads();
    }
    // ---- place them by (distance to the medoid, index); the sum starts as that distance ----
    for (int i = tid; i < n_cand; i += kExpandThreads) {
      const int e = a.cand_raw[i];
      const float de = row_m[e];
      int place = 0;
      for (int j = 0; j < n_cand; ++j) {
        const int o = a.cand_raw[j];
        const float d_o = row_m[o];
        place += (d_o < de) || (d_o == de && o < e);
      }
      a.cand[place] = e;
      a.sum[place] = de;
    }
    __syncthreads();

    // ---- greedy joins ----
    if (fill + 1 > a.members_cap) { overflow = true; break; }
    if (tid == 0) a.members[fill] = m;
    int size = 1, from = 0;                               // members so far; candidates before `from` are decided
    while (from < n_cand) {
      const float bound = a.tau * (float)size;
      int first = n_cand;                                 // first undecided candidate whose average passes
      for (int i = from + tid; i < n_cand; i += kExpandThreads)
        if (a.sum[i] <= bound) { first = i; break; }
      first = __reduce_min_sync(0xFFFFFFFFu, first);
      if (lane == 0) s_warp[warp] = first;
      __syncthreads();
      if (warp == 0) {
        int v = s_warp[lane];
        v = __reduce_min_sync(0xFFFFFFFFu, v);
        if (lane == 0) s_next = v;
      }
      __syncthreads();
      const int at = s_next;
      if (at >= n_cand) break;
      if (fill + size + 1 > a.members_cap) { overflow = true; break; }
      const int e = a.cand[at];
      if (tid == 0) a.members[fill + size] = e;
      ++size;
      const float* row_e = a.dist + (long long)e * n;
      for (int i = at + 1 + tid; i < n_cand; i += kExpandThreads) a.sum[i] = a.sum[i] + row_e[a.cand[i]];
      from = at + 1;
      __syncthreads();
    }
    if (overflow) break;
    // ---- the cluster is final: cover its members ----
    __syncthreads();
    if (tid == 0) s_newly = 0;
    __syncthreads();
    int newly = 0;
    for (int i = tid; i < size; i += kExpandThreads) {
      const int e = a.members[fill + i];
      if (!a.covered[e]) { a.covered[e] = 1; ++newly; }   // members of one cluster are distinct
    }
    if (newly) atomicAdd(&s_newly, newly);
    __syncthreads();
    n_cov += s_newly;
    fill += size;
    if (tid == 0) {
      a.medoid[n_clu] = m;
      a.ptr[n_clu + 1] = (int32_t)fill;
    }
    ++n_clu;
    __syncthreads();
  }
  if (tid == 0) {
    *a.n_clusters = n_clu;
    *a.dev_status = overflow ? 1 : 0;
  }
}

}  // namespace

// ---- admission to the fast tier (Sec. 4.2, Tier 1 (3)): clusters in descending Eq. 6 score while they fit -------
namespace {

// order[place] = c with place = #{ j : score[j] > score[c] or (score[j] == score[c] and j < c) }
__global__ void __launch_bounds__(256)
score_order_kernel(const float* __restrict__ score, int n, int32_t* __restrict__ order) {
  __shared__ float s_sc[2048];
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const float mine = i < n ? score[i] : 0.f;
  int place = 0;
  for (int base = 0; base < n; base += 2048) {
    __syncthreads();
    for (int t = threadIdx.x; t < 2048 && base + t < n; t += blockDim.x) s_sc[t] = score[base + t];
    __syncthreads();
    const int lim = min(2048, n - base);
    for (int t = 0; t < lim; ++t) {
      const float other = s_sc[t];
      place += (other > mine) || (other == mine && base + t < i);
    }
  }
  if (i < n) order[place] = i;
}

// One CTA walks the order: running page count by a block scan per chunk; a cluster is admitted while the count
// stays within the capacity, and the first one that does not fit ends the admission (everything after it is out).
__global__ void __launch_bounds__(1024)
admit_kernel(const int32_t* __restrict__ order, const uint16_t* __restrict__ size, int n, long long capacity,
             uint8_t* __restrict__ resident, int32_t* __restrict__ info) {
  __shared__ long long s_warp[32];
  __shared__ long long s_used_final;
  __shared__ int s_first_out;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  long long used = 0;                                      // pages of the clusters before the current chunk
  int admitted = 0;
  bool closed = false;
  for (int base = 0; base < n; base += 1024) {
    const int r = base + tid;
    const int c = r < n ? order[r] : -1;
    const long long mine = c >= 0 ? (long long)size[c] : 0;
    long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += t;
    }
    if (tid == 0) s_first_out = 1 << 30;
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    long long before = used;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    const bool fits = !closed && c >= 0 && before + incl <= capacity;
    if (c >= 0 && !fits) atomicMin(&s_first_out, r);
    __syncthreads();
    const int first_out = s_first_out;                     // rank of the first cluster that does not fit (if any)
    const bool in = c >= 0 && !closed && r < first_out;
    if (c >= 0) resident[c] = in ? 1 : 0;
    if (!closed) {
      if (first_out < (1 << 30)) {
        if (r == first_out) s_used_final = before + incl - mine;   // pages used when the admission ended
        admitted += first_out - base;
      } else {
        for (int w = 0; w < 32; ++w) used += s_warp[w];
        admitted += min(1024, n - base);
      }
    }
    __syncthreads();
    if (!closed && first_out < (1 << 30)) {
      used = s_used_final;
      closed = true;
    }
  }
  if (tid == 0 && info != nullptr) {
    info[0] = admitted;
    info[1] = (int32_t)min(used, 0x7FFFFFFFLL);
  }
}

}  // namespace

long long cache_admit_workspace_bytes(int n) { return ((long long)n * 4 + 255) / 256 * 256; }

cudaError_t launch_cache_admit(const float* score, const uint16_t* size, int n, long long capacity, void* workspace,
                               uint8_t* resident, int32_t* info, cudaStream_t st) {
  int32_t* order = static_cast<int32_t*>(workspace);
  score_order_kernel<<<dim3((n + 255) / 256), dim3(256), 0, st>>>(score, n, order);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_pdl(admit_kernel, dim3(1), dim3(1024), 0, st, true, order, size, n, capacity, resident, info);
}

long long build_clusters_workspace_bytes(int n) {
  // queue, cand_raw, cand (int32), sum (float), covered (bytes), each padded to 256 bytes
  const long long words = ((long long)n * 4 + 255) / 256 * 256;
  return 4 * words + ((long long)n + 255) / 256 * 256;
}

cudaError_t launch_build_clusters(const float* dist, int n, float tau, void* workspace, int32_t* rho, int32_t* ptr,
                                  int32_t* members, long long members_cap, int32_t* medoid, int32_t* n_clusters,
                                  int32_t* dev_status, cudaStream_t st) {
  const long long words = ((long long)n * 4 + 255) / 256 * 256;
  char* ws = static_cast<char*>(workspace);
  ExpandArgs a;
  a.dist = dist; a.n = n; a.tau = tau;
  int32_t* queue = reinterpret_cast<int32_t*>(ws);
  a.queue = queue;
  a.cand_raw = reinterpret_cast<int32_t*>(ws + words);
  a.cand = reinterpret_cast<int32_t*>(ws + 2 * words);
  a.sum = reinterpret_cast<float*>(ws + 3 * words);
  a.covered = reinterpret_cast<uint8_t*>(ws + 4 * words);
  a.ptr = ptr; a.members = members; a.members_cap = members_cap; a.medoid = medoid; a.n_clusters = n_clusters;
  a.dev_status = dev_status;
  density_kernel<<<dim3((n + 7) / 8), dim3(256), 0, st>>>(dist, n, tau, rho);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  queue_kernel<<<dim3((n + 255) / 256), dim3(256), 0, st>>>(rho, n, queue);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_pdl(expand_kernel, dim3(1), dim3(kExpandThreads), 0, st, true, a);
}

}  // namespace swarm
