// Stage 1: activation scoring (Sec. 2.3: relevance score of every cached entry against the query).
//
//   score[b][h][p] = sum_i max(q[i]*kmin[p][i], q[i]*kmax[p][i])
//                  = sum_i max(q[i],0)*kmax[p][i] + min(q[i],0)*kmin[p][i]        (kmin <= kmax)
//
// One summary row (page, kv head) is 512 contiguous bytes: 128 bf16 minima then 128 bf16 maxima.
// A warp reads a row with one 16-byte load per lane (lanes 0-15 hold minima, 16-31 maxima), so the
// sign-split form needs one FMA per element and query head, with the weights (min(q,0) on the low
// lanes, max(q,0) on the high lanes) held in registers for all G heads of the KV group.  R rows are
// in flight per warp; their R*G partial sums are summed across lanes with a transposing butterfly
// (31 shuffles for 32 sums) that leaves sum v in lane v, so the scores leave as coalesced stores.
// HBM-bound: 512 B per row against (8 unpack + 8*G FMA) warp instructions.
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kScoreWarps = 8;

template <int NV>
__device__ __forceinline__ float transpose_reduce(float (&v)[NV], int lane) {
  // After the call, lane L holds the total of value (L >> (5 - log2 NV)).
  int offset = 16;
#pragma unroll
  for (int n = NV; n > 1; n >>= 1) {
    const bool upper = (lane & offset) != 0;
#pragma unroll
    for (int j = 0; j < n / 2; ++j) {
      const float keep = upper ? v[j + n / 2] : v[j];
      const float send = upper ? v[j] : v[j + n / 2];
      v[j] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, offset);
    }
    offset >>= 1;
  }
  float r = v[0];
  for (; offset >= 1; offset >>= 1) r += __shfl_xor_sync(0xFFFFFFFFu, r, offset);
  return r;
}

template <int G, int R>
__global__ void __launch_bounds__(kScoreWarps * 32)
page_score_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ ksum,
                  const int64_t* __restrict__ page_base, const int32_t* __restrict__ ctx_len,
                  float* __restrict__ scores, uint32_t* __restrict__ status, int iters) {
  constexpr int NV = G * R;
  static_assert(NV <= 32 && (NV & (NV - 1)) == 0, "R*G must be a power of two <= 32");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tiles = geo.g / G;
  const int kvh = blockIdx.y / tiles, tile = blockIdx.y % tiles;
  const int b = blockIdx.z;
  const int len = ctx_len[b];
  const long long base = page_base[b];
  const int P = pages_of(len, geo.S);
  if (len < 1 || P > page_base[b + 1] - base || P > geo.Pmax) {
    if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) atomicOr(status, SWARM_DEV_BAD_LENGTH);
    return;
  }
  const int pages_per_cta = kScoreWarps * R * iters;
  const int p_cta = blockIdx.x * pages_per_cta;
  if (p_cta >= P) return;

  // Weights of this lane's 8 coordinates for each of the G heads.
  const int h0 = kvh * geo.g + tile * G;
  float w[G][8];
#pragma unroll
  for (int hh = 0; hh < G; ++hh) {
    const uint4 qq = *reinterpret_cast<const uint4*>(q + ((long long)(b * geo.Hq + h0 + hh) * kHeadDim + (lane & 15) * 8));
    const uint32_t words[4] = {qq.x, qq.y, qq.z, qq.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float lo = bf16_lo(words[e]), hi = bf16_hi(words[e]);
      w[hh][2 * e] = lane < 16 ? fminf(lo, 0.f) : fmaxf(lo, 0.f);
      w[hh][2 * e + 1] = lane < 16 ? fminf(hi, 0.f) : fmaxf(hi, 0.f);
    }
  }

  const long long row_stride = (long long)geo.Hkv * 2 * kHeadDim;   // elements between consecutive pages
  const uint16_t* rows = ksum + ((base * geo.Hkv + kvh) * 2) * (long long)kHeadDim + lane * 8;

  auto load_rows = [&](int p0, uint4 (&dst)[R]) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int p = p0 + r;
      dst[r] = p < P ? ldg_nc_v4(rows + p * row_stride) : make_uint4(0, 0, 0, 0);
    }
  };

  uint4 cur[R], nxt[R];
  int p0 = p_cta + warp * R;
  load_rows(p0, cur);
  for (int it = 0; it < iters; ++it) {
    const int p_next = p0 + kScoreWarps * R;
    if (it + 1 < iters) load_rows(p_next, nxt);
    float v[NV];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const uint32_t words[4] = {cur[r].x, cur[r].y, cur[r].z, cur[r].w};
      float x[8];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        x[2 * e] = bf16_lo(words[e]);
        x[2 * e + 1] = bf16_hi(words[e]);
      }
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) s = fmaf(w[hh][e], x[e], s);
        v[hh * R + r] = s;
      }
    }
    const float total = transpose_reduce<NV>(v, lane);
    constexpr int kShift = NV == 32 ? 0 : NV == 16 ? 1 : NV == 8 ? 2 : NV == 4 ? 3 : NV == 2 ? 4 : 5;
    const int idx = lane >> kShift;
    const int hh = idx / R, r = idx % R;
    if ((lane & ((1 << kShift) - 1)) == 0 && p0 + r < P)
      scores[((long long)(b * geo.Hq + h0 + hh)) * geo.Pmax + p0 + r] = total;
    if (it + 1 < iters) {
#pragma unroll
      for (int r2 = 0; r2 < R; ++r2) cur[r2] = nxt[r2];
    }
    p0 = p_next;
  }
}

template <int G, int R>
cudaError_t launch_one(const Geometry& geo, const uint16_t* q, const uint16_t* ksum, const int64_t* page_base,
                       const int32_t* ctx_len, float* scores, uint32_t* status, cudaStream_t st) {
  // Pages per CTA: enough CTAs to fill the 148 SMs several times over, yet >= 2 batches per warp
  // when the context is long so the next batch's loads overlap the current batch's arithmetic.
  const long long rows_total = (long long)geo.B * geo.Hkv * geo.Pmax;
  int iters = 1;
  while (iters < 8 && rows_total / (kScoreWarps * R * iters * 2) >= 148LL * 8) iters *= 2;
  const int pages_per_cta = kScoreWarps * R * iters;
  dim3 grid((geo.Pmax + pages_per_cta - 1) / pages_per_cta, geo.Hkv * (geo.g / G), geo.B);
  page_score_kernel<G, R><<<grid, kScoreWarps * 32, 0, st>>>(geo, q, ksum, page_base, ctx_len, scores, status, iters);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_page_score(const Geometry& geo, const uint16_t* q, const uint16_t* ksum,
                              const int64_t* page_base, const int32_t* ctx_len, float* scores, uint32_t* status,
                              cudaStream_t st) {
  // Heads of a KV group are processed G at a time, G the largest of 8/4/2/1 dividing the group size.
  if (geo.g % 8 == 0) return launch_one<8, 4>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 4 == 0) return launch_one<4, 8>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 2 == 0) return launch_one<2, 8>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  return launch_one<1, 8>(geo, q, ksum, page_base, ctx_len, scores, status, st);
}

}  // namespace swarm
