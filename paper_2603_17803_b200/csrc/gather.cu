// Stage 4a: gather of the selected pages (the cross-tier transfer of Sec. 6, here a copy inside
// HBM), and the index build that produces the per-page min/max key summaries.
//
// Both are pure streaming kernels: 16-byte loads and stores, one contiguous K (or V) block of
// S*256 bytes per (page, kv head), no reuse -- bound by HBM bandwidth.
#include "swarm_internal.cuh"

namespace swarm {
namespace {

// One CTA per (b, h, slot j): copies the K block and the V block of page sel[b][h][j] for head
// kv(h) into rows [j*S, (j+1)*S) of the head's gathered buffers.  Rows of padding tokens and whole
// unused slots are written as zeros.
__global__ void __launch_bounds__(256)
gather_kernel(Geometry geo, const uint16_t* __restrict__ kv_pool, const int32_t* __restrict__ sel,
              const int32_t* __restrict__ n_sel, const int64_t* __restrict__ page_base,
              const int32_t* __restrict__ ctx_len, uint16_t* __restrict__ k_out, uint16_t* __restrict__ v_out,
              int32_t* __restrict__ n_tok, uint32_t* __restrict__ status) {
  const int j = blockIdx.x % geo.k, bh = blockIdx.x / geo.k, b = bh / geo.Hq, h = bh % geo.Hq;
  const int S = geo.S;
  const int len = ctx_len[b];
  const int P = pages_of(len, S);
  const int tail = len - S * (P - 1);                       // valid tokens of the last page
  const int ns = n_sel[bh];
  const long long blk = (long long)S * kHeadDim;            // elements per K (or V) block
  int p = j < ns ? sel[(long long)bh * geo.k + j] : -1;
  if (j < ns && (p < 0 || p >= P)) {
    if (threadIdx.x == 0) atomicOr(status, SWARM_DEV_BAD_PAGE);
    p = -1;
  }
  // The attention over gathered buffers masks only the end of the last slot: a partial page anywhere else would
  // put its padding rows among the valid tokens.  The library's own selections are ascending, so this can only
  // happen with a selection the caller wrote.
  if (p == P - 1 && tail != S && j != ns - 1) {
    if (threadIdx.x == 0) atomicOr(status, SWARM_DEV_BAD_PAGE);
    p = -1;
  }
  const int valid = p < 0 ? 0 : (p == P - 1 ? tail : S);
  const uint4 zero = make_uint4(0, 0, 0, 0);
  const uint16_t* src = kv_pool + (((page_base[b] + max(p, 0)) * geo.Hkv + h / geo.g) * 2) * blk;
  uint4* kd = reinterpret_cast<uint4*>(k_out + ((long long)bh * geo.k + j) * blk);
  uint4* vd = reinterpret_cast<uint4*>(v_out + ((long long)bh * geo.k + j) * blk);
  const int vec_per_block = S * kHeadDim / 8;               // 16-byte vectors per block (16 per token)
  for (int i = threadIdx.x; i < vec_per_block; i += blockDim.x) {
    const bool ok = (i >> 4) < valid;
    kd[i] = ok ? ldg_nc_v4(src + (long long)i * 8) : zero;
    vd[i] = ok ? ldg_nc_v4(src + blk + (long long)i * 8) : zero;
  }
  if (n_tok != nullptr && j == 0 && threadIdx.x == 0) {
    // sel is ascending, so a partial page can only be the last selected one
    int rows = 0;
    if (ns > 0) {
      const int last = sel[(long long)bh * geo.k + ns - 1];
      rows = ns * S - (last == P - 1 ? S - tail : 0);
    }
    n_tok[bh] = rows;
  }
}

// One warp per (pool page, kv head): lanes 0-15 scan the even tokens, lanes 16-31 the odd tokens,
// each over 8 coordinates; the halves are merged with one shuffle and lanes 0-15 write the 256-byte
// minima row, lanes 16-31 the maxima row.
__global__ void __launch_bounds__(256)
summaries_kernel(Geometry geo, const uint16_t* __restrict__ kv_pool, const int64_t* __restrict__ page_base,
                 const int32_t* __restrict__ ctx_len, uint16_t* __restrict__ ksum, uint32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.z, kvh = blockIdx.y;
  const int S = geo.S;
  const int len = ctx_len[b];
  const int P = pages_of(len, S);
  const long long base = page_base[b];
  if (len < 1 || P > page_base[b + 1] - base) {
    if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) atomicOr(status, SWARM_DEV_BAD_LENGTH);
    return;
  }
  const int p = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (p >= P) return;
  const int valid = p == P - 1 ? len - S * (P - 1) : S;
  const uint16_t* K = kv_pool + (((base + p) * geo.Hkv + kvh) * 2) * (long long)S * kHeadDim;
  const int c = lane & 15, half = lane >> 4;
  float lo[8], hi[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) { lo[e] = INFINITY; hi[e] = -INFINITY; }
  for (int t = half; t < valid; t += 2) {
    const uint4 v = ldg_nc_v4(K + (long long)t * kHeadDim + c * 8);
    const uint32_t words[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = bf16_lo(words[e]), d2 = bf16_hi(words[e]);
      lo[2 * e] = fminf(lo[2 * e], a);         hi[2 * e] = fmaxf(hi[2 * e], a);
      lo[2 * e + 1] = fminf(lo[2 * e + 1], d2); hi[2 * e + 1] = fmaxf(hi[2 * e + 1], d2);
    }
  }
  uint32_t packed[4];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    lo[e] = fminf(lo[e], __shfl_xor_sync(0xFFFFFFFFu, lo[e], 16));
    hi[e] = fmaxf(hi[e], __shfl_xor_sync(0xFFFFFFFFu, hi[e], 16));
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float a = half ? hi[2 * e] : lo[2 * e], d2 = half ? hi[2 * e + 1] : lo[2 * e + 1];
    packed[e] = (__float_as_uint(a) >> 16) | (__float_as_uint(d2) & 0xFFFF0000u);   // values are bf16 already
  }
  uint4* dst = reinterpret_cast<uint4*>(ksum + (((base + p) * geo.Hkv + kvh) * 2 + half) * (long long)kHeadDim + c * 8);
  *dst = make_uint4(packed[0], packed[1], packed[2], packed[3]);
}

}  // namespace

cudaError_t launch_gather(const Geometry& geo, const uint16_t* kv_pool, const int32_t* sel, const int32_t* n_sel,
                          const int64_t* page_base, const int32_t* ctx_len, uint16_t* k_out, uint16_t* v_out,
                          int32_t* n_tok, uint32_t* status, cudaStream_t st) {
  const unsigned grid = (unsigned)geo.k * geo.B * geo.Hq;   // validated to fit at ctx creation
  gather_kernel<<<grid, 256, 0, st>>>(geo, kv_pool, sel, n_sel, page_base, ctx_len, k_out, v_out, n_tok, status);
  return cudaGetLastError();
}

cudaError_t launch_build_summaries(const Geometry& geo, const uint16_t* kv_pool, const int64_t* page_base,
                                   const int32_t* ctx_len, uint16_t* ksum, uint32_t* status, cudaStream_t st) {
  dim3 grid((geo.Pmax + 7) / 8, geo.Hkv, geo.B);
  summaries_kernel<<<grid, 256, 0, st>>>(geo, kv_pool, page_base, ctx_len, ksum, status);
  return cudaGetLastError();
}

// Per-step data moved by kernels between the device and host memory the device can address (pinned, unified
// addressing) instead of by copy operations: a copy node between kernels costs several microseconds of
// engine hand-over, a load or store over the bus does not.
//   fetch_kernel    the step's queries, host -> workspace (volatile loads: the host rewrites the buffer between calls)
//   publish_kernel  the step's small results, device -> host; 16-byte vectors for out, words for the rest (used
//                   when the step's last kernel cannot store them itself, see HostMirror)
namespace {
__global__ void __launch_bounds__(256)
fetch_kernel(const uint4* src_h, uint4* __restrict__ dst, int n16) {
  pdl_launch_dependents();                                  // the scorer sets itself up meanwhile
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x) {
    uint4 v;
    asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(src_h + i));
    dst[i] = v;
  }
}

__global__ void __launch_bounds__(256)
publish_kernel(const float* __restrict__ out, const float* __restrict__ lse, const int32_t* __restrict__ n_uniq,
               const int32_t* __restrict__ queue_load, float* out_h, float* lse_h, int32_t* n_uniq_h,
               int32_t* queue_load_h, int n_out4, int n_lse, int n_queues) {
  pdl_wait();                                               // the results come from the previous kernel
  const int t = blockIdx.x * blockDim.x + threadIdx.x, stride = gridDim.x * blockDim.x;
  if (out_h != nullptr)
    for (int i = t; i < n_out4; i += stride)
      reinterpret_cast<float4*>(out_h)[i] = __ldcg(reinterpret_cast<const float4*>(out) + i);
  if (lse_h != nullptr)
    for (int i = t; i < n_lse; i += stride) lse_h[i] = __ldcg(lse + i);
  if (queue_load_h != nullptr)
    for (int i = t; i < n_queues; i += stride) queue_load_h[i] = __ldcg(queue_load + i);
  if (n_uniq_h != nullptr && t == 0) *n_uniq_h = __ldcg(n_uniq);
}
}  // namespace

cudaError_t launch_fetch(const void* src_h, void* dst, long long bytes, cudaStream_t st) {
  const int n16 = (int)(bytes / 16);
  const int grid = max(1, min(32, (n16 + 255) / 256));
  fetch_kernel<<<dim3(grid), dim3(256), 0, st>>>(static_cast<const uint4*>(src_h), static_cast<uint4*>(dst), n16);
  return cudaGetLastError();
}

cudaError_t launch_publish(const Geometry& geo, const float* out, const float* lse, const int32_t* n_uniq,
                           const int32_t* queue_load, float* out_h, float* lse_h, int32_t* n_uniq_h,
                           int32_t* queue_load_h, cudaStream_t st) {
  const int n_out4 = geo.B * geo.Hq * kHeadDim / 4;
  const int grid = max(1, min(32, (n_out4 + 255) / 256));
  return launch_pdl(publish_kernel, dim3(grid), dim3(256), 0, st, true, out, lse, n_uniq, queue_load, out_h, lse_h,
                    n_uniq_h, queue_load_h, n_out4, geo.B * geo.Hq, geo.D);
}

}  // namespace swarm
