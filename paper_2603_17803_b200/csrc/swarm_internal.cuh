// Internal declarations shared by the kernels and the C-ABI layer of libswarm (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "swarm.h"

namespace swarm {

constexpr int kHeadDim = 128;

// Where each scratch region sits inside the caller-provided workspace (byte offsets, 256-aligned).
struct WorkspaceLayout {
  int64_t status;        // uint32 status word
  int64_t scores;        // f32 [B][Hq][Pmax]          (used when the caller passes no scores buffer)
  int64_t n_tok;         // i32 [B][Hq]                (used when the caller passes no n_tok buffer)
  int64_t q_stage;       // bf16 [B][Hq][d]            (swarm_step_host)
  int64_t flags;         // u8  [max_clusters_total]   (cluster dedup when it does not fit in smem)
  int64_t part_acc;      // f32 [B*Hq][max_splits][d]  split-K partial outputs
  int64_t part_ml;       // f32 [B*Hq][max_splits][2]  split-K partial (max, sum)
  int64_t total;
};

constexpr int kMaxSplits = 64;

struct Geometry {   // plain copy of the shape in kernel-friendly form
  int B, Hq, Hkv, g, S, k, D, Pmax, Cmax;
  unsigned flags;
  long long n_pool_pages;
};

// ---- one-time per-device kernel attribute set-up (dynamic shared-memory limits) ---------------
cudaError_t configure_topk();
cudaError_t configure_resolve();

// ---- kernel launchers (each returns cudaGetLastError() after the launch) ----------------------
cudaError_t launch_build_summaries(const Geometry& geo, const uint16_t* kv_pool, const int64_t* page_base,
                                   const int32_t* ctx_len, uint16_t* ksum, uint32_t* status, cudaStream_t st);
cudaError_t launch_page_score(const Geometry& geo, const uint16_t* q, const uint16_t* ksum,
                              const int64_t* page_base, const int32_t* ctx_len, float* scores, uint32_t* status,
                              cudaStream_t st);
cudaError_t launch_topk(const Geometry& geo, const float* scores, const int32_t* ctx_len, int32_t* sel,
                        int32_t* n_sel, cudaStream_t st);
cudaError_t launch_resolve(const Geometry& geo, const int32_t* sel, const int32_t* n_sel, const int64_t* page_base,
                           const int32_t* page2cluster, const int64_t* cluster_base, const uint32_t* replica_mask,
                           const uint16_t* cluster_size, uint8_t* flags_ws, int32_t* uniq, uint8_t* queue_of,
                           int32_t* n_uniq, int32_t* queue_load, uint32_t* status, cudaStream_t st);
cudaError_t launch_gather(const Geometry& geo, const uint16_t* kv_pool, const int32_t* sel, const int32_t* n_sel,
                          const int64_t* page_base, const int32_t* ctx_len, uint16_t* k_out, uint16_t* v_out,
                          int32_t* n_tok, uint32_t* status, cudaStream_t st);
// Attention over contiguous gathered buffers (pool == nullptr) or straight from the pool (k_g == nullptr).
struct AttnArgs {
  const uint16_t* q;
  const uint16_t* k_g;
  const uint16_t* v_g;
  const int32_t* n_tok;
  const uint16_t* kv_pool;
  const int32_t* sel;
  const int32_t* n_sel;
  const int64_t* page_base;
  const int32_t* ctx_len;
  float* part_acc;
  float* part_ml;
  float* out;
  float* lse;
  int n_splits;
};
cudaError_t launch_attention(const Geometry& geo, const AttnArgs& a, uint32_t* status, cudaStream_t st);

// ---- device helpers ---------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ int pages_of(int ctx_len, int S) { return (ctx_len + S - 1) / S; }

}  // namespace swarm
