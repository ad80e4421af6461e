// Stage 2: per-head top-k page selection (Sec. 2.3: only the entries with the highest scores are
// activated).  One CTA per (request, query head).
//
// Scores become order-preserving 32-bit keys (-0 folded onto +0 so the two compare equal).  A
// most-significant-digit radix select (4 passes of 8 bits, warp-aggregated shared-memory
// histograms) finds the exact key T of the k-th best page and how many pages tie with it.  The
// result is then written by an ordered ballot/popc compaction in page-id order: every page with
// key > T, plus the first (k - #greater) pages with key == T.  That order gives "ties go to the
// lower page id" and the ascending-id output at once.
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kTopkThreads = 1024;
constexpr int kTopkWarps = kTopkThreads / 32;

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <bool kKeysInSmem>
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(Geometry geo, const float* __restrict__ scores, const int32_t* __restrict__ ctx_len,
            int32_t* __restrict__ sel, int32_t* __restrict__ n_sel) {
  extern __shared__ uint32_t skeys[];
  __shared__ int hist[257];
  __shared__ int warp_gt[kTopkWarps], warp_eq[kTopkWarps];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.x, b = bh / geo.Hq;
  const int P = max(0, min(pages_of(ctx_len[b], geo.S), geo.Pmax));   // invalid lengths are reported by the scorer
  const int k_eff = min(geo.k, P);
  const float* s = scores + (long long)bh * geo.Pmax;
  int32_t* out = sel + (long long)bh * geo.k;

  auto key_at = [&](int i) -> uint32_t { return kKeysInSmem ? skeys[i] : score_key(s[i]); };

  if (kKeysInSmem)
    for (int i = tid; i < P; i += kTopkThreads) skeys[i] = score_key(s[i]);
  if (tid == 0) { s_prefix = 0u; s_remaining = k_eff; }
  __syncthreads();

  if (k_eff > 0 && k_eff < P) {
    const int P_round = (P + 31) & ~31;
    uint32_t mask = 0u;
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < 257; i += kTopkThreads) hist[i] = 0;
      __syncthreads();
      const uint32_t prefix = s_prefix;
      for (int i = tid; i < P_round; i += kTopkThreads) {
        int digit = 256;                                   // bin 256 collects non-candidates
        if (i < P) {
          const uint32_t key = key_at(i);
          if ((key & mask) == prefix) digit = (key >> shift) & 255;
        }
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, digit);
        if (lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
      }
      __syncthreads();
      if (warp == 0) {
        // lane L owns bins [255-8L-7, 255-8L]; find the bin where the count from the top reaches `remaining`
        int local[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { local[j] = hist[255 - 8 * lane - j]; sum += local[j]; }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
          if (lane >= o) incl += t;
        }
        const int remaining = s_remaining;
        int above = incl - sum;                            // pages in bins above this lane's bins
        if (above < remaining && remaining <= incl) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (above < remaining && remaining <= above + local[j]) {
              s_prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
              s_remaining = remaining - above;
              above = remaining;                           // stop
            } else {
              above += local[j];
            }
          }
        }
      }
      mask |= 255u << shift;
      __syncthreads();
    }
  }

  // Ordered compaction.  k_eff == P keeps everything (T = 0, every key > T or == T with room).
  const bool take_all = (k_eff == P);
  const uint32_t T = take_all ? 0u : s_prefix;
  const int need_eq = take_all ? P : s_remaining;
  const int seg = (((P + kTopkWarps - 1) / kTopkWarps) + 31) & ~31;   // per-warp contiguous span
  const int lo = min(P, warp * seg), hi = min(P, lo + seg);
  int cnt_gt = 0, cnt_eq = 0;
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < hi ? key_at(i) : 0u;
    const bool gt = i < hi && key > T, eq = i < hi && key == T;
    cnt_gt += __popc(__ballot_sync(0xFFFFFFFFu, gt));
    cnt_eq += __popc(__ballot_sync(0xFFFFFFFFu, eq));
  }
  if (lane == 0) { warp_gt[warp] = cnt_gt; warp_eq[warp] = cnt_eq; }
  __syncthreads();
  int gt_before = 0, eq_before = 0;
  for (int w2 = 0; w2 < warp; ++w2) { gt_before += warp_gt[w2]; eq_before += warp_eq[w2]; }
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < hi ? key_at(i) : 0u;
    const bool gt = i < hi && key > T, eq = i < hi && key == T;
    const unsigned bg = __ballot_sync(0xFFFFFFFFu, gt), be = __ballot_sync(0xFFFFFFFFu, eq);
    const int my_gt = gt_before + __popc(bg & lt_mask);
    const int my_eq = eq_before + __popc(be & lt_mask);
    if (gt || (eq && my_eq < need_eq)) out[my_gt + min(my_eq, need_eq)] = i;
    gt_before += __popc(bg);
    eq_before += __popc(be);
  }
  for (int j = k_eff + tid; j < geo.k; j += kTopkThreads) out[j] = -1;
  if (tid == 0) n_sel[bh] = k_eff;
}

}  // namespace

cudaError_t configure_topk() {
  return cudaFuncSetAttribute(topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

cudaError_t launch_topk(const Geometry& geo, const float* scores, const int32_t* ctx_len, int32_t* sel,
                        int32_t* n_sel, cudaStream_t st) {
  const size_t key_bytes = (size_t)geo.Pmax * sizeof(uint32_t);
  const int n_lists = geo.B * geo.Hq;
  if (key_bytes <= 200 * 1024) {
    topk_kernel<true><<<n_lists, kTopkThreads, key_bytes, st>>>(geo, scores, ctx_len, sel, n_sel);
  } else {
    topk_kernel<false><<<n_lists, kTopkThreads, 0, st>>>(geo, scores, ctx_len, sel, n_sel);
  }
  return cudaGetLastError();
}

}  // namespace swarm
