// Shared device/host helpers of the MoIN CUDA library (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <limits.h>
#include <stdint.h>

#include "../../include/moin.h"

namespace moin {

// ----------------------------------------------------------------------------------------
// Device status block (one per process; its device address is passed to kernels).
// ----------------------------------------------------------------------------------------
struct DeviceStatus {
  int timeout_flag;
  int timeout_site;
  int invalid_expert_ids;
  int reserved[5];
};

// Plan buffer layout (int32 words).  Header first, then the arrays.
constexpr int kPlanHeaderWords = 16;
enum PlanHeader { PH_NSEG = 0, PH_NTILES = 1, PH_NLORA = 2, PH_MAXSEG = 3, PH_T = 4, PH_E = 5 };
constexpr int kPlanChunk = 256;   // tokens per histogram chunk
constexpr int kTileRows = 128;    // rows per GEMM tile

struct PlanView {   // pointers into the plan buffer
  int* header;
  int* perm;         // [T]   token indices ordered by (expert, token)
  int* seg_expert;   // [Smax]
  int* seg_start;    // [Smax + 1]
  int4* seg_tab;     // [Smax + 1] packed (expert, start, length, 0): one 16-byte load per segment
  int* tile_row0;    // [T + 1]
  int* tile_rows;    // [T]
  int* tile_expert;  // [T]
  int* rank;         // [T]   scratch
  int* key;          // [T]   scratch
  int* keybase;      // [E+1] scratch
  int* hist;         // [n_chunks * (E+1)] scratch
  int T, E, Smax, n_chunks;
};

__host__ __device__ inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline PlanView plan_view(void* buffer, int T, int E, size_t* total_words = nullptr) {
  PlanView v;
  v.T = T; v.E = E;
  v.Smax = T < E ? T : E;
  v.n_chunks = (T + kPlanChunk - 1) / kPlanChunk;
  int* base = reinterpret_cast<int*>(buffer);
  size_t off = 0;
  auto take = [&](size_t n) { size_t o = off; off += align_up(n, 4); return base ? base + o : nullptr; };
  v.header = take(kPlanHeaderWords);
  v.perm = take(T);
  v.seg_expert = take(v.Smax + 1);
  v.seg_start = take(v.Smax + 2);
  v.seg_tab = reinterpret_cast<int4*>(take(4 * (size_t)(v.Smax + 1)));
  v.tile_row0 = take(T + 1);
  v.tile_rows = take(T + 1);
  v.tile_expert = take(T + 1);
  v.rank = take(T);
  v.key = take(T);
  v.keybase = take(E + 2);
  v.hist = take((size_t)v.n_chunks * (size_t)(E + 1));
  if (total_words) *total_words = off;
  return v;
}
inline size_t plan_bytes(int T, int E) {
  size_t words = 0;
  plan_view(nullptr, T, E, &words);
  return words * sizeof(int);
}

// ----------------------------------------------------------------------------------------
// Small device utilities
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Streaming 16-byte load that does not allocate in L1 (adapter weights are read once).
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint4 ldg_cached(const void* p) {
  return __ldg(reinterpret_cast<const uint4*>(p));
}

// mma.sync m16n8k16, bf16 x bf16 -> fp32 (warp-level tensor-core path for the skinny LoRA products)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Function between the two low-rank matrices (MOIN_ACT_*).
__device__ __forceinline__ float lora_act(float v, int act) {
  switch (act) {
    case MOIN_ACT_RELU: return fmaxf(v, 0.f);
    case MOIN_ACT_SILU: return v / (1.f + __expf(-v));
    case MOIN_ACT_GELU: return 0.5f * v * (1.f + erff(v * 0.70710678118654752f));
    default: return v;
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Launchers implemented in the .cu files (host side).
int plan_launches(int T, int E);   // kernels launch_plan_build issues for this shape
cudaError_t launch_plan_build(const int* token_expert, const PlanView& v, DeviceStatus* status, bool want_tiles,
                              cudaStream_t stream);
// Register-fed short-segment kernels: one launch covers up to kMaxStreamJobs projections sharing a plan.
constexpr int kMaxStreamJobs = 4;
struct ShrinkJobs {
  const __nv_bfloat16* x[kMaxStreamJobs];
  const __nv_bfloat16* A[kMaxStreamJobs];
  float* h[kMaxStreamJobs];
  const int* slot_of_expert[kMaxStreamJobs];
  const int* slot_rank[kMaxStreamJobs];   // per-slot rank (nullptr: the pool's r)
  int r[kMaxStreamJobs], d_in[kMaxStreamJobs], per_seg[kMaxStreamJobs];
  int n;
};
struct ExpandJobs {
  const float* h[kMaxStreamJobs];
  const __nv_bfloat16* B[kMaxStreamJobs];
  const float* y0[kMaxStreamJobs];
  __nv_bfloat16* y[kMaxStreamJobs];
  const int* slot_of_expert[kMaxStreamJobs];
  const int* slot_rank[kMaxStreamJobs];   // per-slot rank (nullptr: the pool's r)
  int act[kMaxStreamJobs];                // MOIN_ACT_* applied to h
  int r[kMaxStreamJobs], d_out[kMaxStreamJobs], rows_per_item[kMaxStreamJobs], per_seg[kMaxStreamJobs];
  int n;
};
cudaError_t launch_lora_shrink_stream(const PlanView& pv, ShrinkJobs jobs, int n_sms, cudaStream_t stream);
cudaError_t launch_lora_expand_stream(const PlanView& pv, ExpandJobs jobs, float scale, int n_sms,
                                      cudaStream_t stream);
cudaError_t launch_gemm_warp(const __nv_bfloat16* x, const __nv_bfloat16* W, __nv_bfloat16* y, float* y0, int T,
                             int d_in, int d_out, cudaStream_t stream);
cudaError_t launch_route_top2_simple(const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                                     const int* cmap, int Q, int K, int D, int* out_expert, int* out_centroid,
                                     int* out_second, float* out_best, float* out_margin, cudaStream_t stream);
cudaError_t launch_route_finish_top2(const unsigned long long* keys, const unsigned long long* keys2,
                                     const __nv_bfloat16* q, const int* cmap, int Q, int D, int* out_expert,
                                     int* out_centroid, int* out_second, float* out_best, float* out_margin,
                                     cudaStream_t stream);
cudaError_t launch_kmeans_mean(const PlanView& pv, const __nv_bfloat16* x, __nv_bfloat16* c_new, int D, int n_sms,
                               cudaStream_t stream);
cudaError_t launch_inv_norm(const __nv_bfloat16* c, int K, int D, float* inv_norm, cudaStream_t stream);
cudaError_t launch_route_simple(const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                                const int* cmap, int Q, int K, int D, int* out_expert, int* out_centroid,
                                float* out_best, cudaStream_t stream);
bool route_cluster_supported(int Q, int K, int D);
cudaError_t launch_route_cluster(const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                                 const int* cmap, int Q, int K, int D, int* out_expert, int* out_centroid,
                                 float* out_best, cudaStream_t stream);
cudaError_t launch_route_finish(const unsigned long long* keys, const __nv_bfloat16* q, const int* cmap, int Q, int D,
                                int* out_expert, int* out_centroid, float* out_best, cudaStream_t stream);

// Host state of the entry points (api.cu): one record per device ordinal, filled on the first call made with
// that device current.  Streams, events, the status block's address and the kernels' shared-memory opt-ins all
// belong to one device, so nothing here is shared between devices.
constexpr int kMaxDevices = 64;
constexpr int kOptinSlots = 48;
struct HostState {
  DeviceStatus* status = nullptr;  // device address of the status block
  int device = -1;
  int n_sms = 0;
  int gemm_impl = 0;               // MOIN_OPT_GEMM_IMPL (process-wide option, copied in on every call)
  // fork/join inside one call: independent kernels of a call run on `side` between two events
  cudaStream_t side[kMaxStreamJobs] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t ev_fork = nullptr, ev_join[kMaxStreamJobs] = {nullptr, nullptr, nullptr, nullptr};
  size_t smem_optin[kOptinSlots] = {};   // dynamic shared memory already opted in, per kernel (see ensure_smem_optin)
};
moin_status host_state(HostState** out);      // lazily initialised for the current device
moin_status record_cuda(cudaError_t e);       // MOIN_OK or MOIN_ERR_CUDA (remembers e)

// Kernels that need more than 48 KB of dynamic shared memory opt in with cudaFuncSetAttribute; the driver keeps
// that attribute per device, so the "already done" note is kept per device too (slot = one id per kernel).
enum {
  OPTIN_TC_GEMM = 0,        // + 4 * (BN index) + EPI, 12 entries; + 12 for the short-ring instantiations
  OPTIN_ROUTE_CLUSTER = 24, OPTIN_ROUTE_SIMPLE = 25, OPTIN_ATTENTION = 29
};
template <class Fn>
inline cudaError_t ensure_smem_optin(int slot, Fn* fn, size_t bytes) {
  HostState* hs = nullptr;
  if (host_state(&hs) != MOIN_OK) return cudaErrorInvalidDevice;
  if (hs->smem_optin[slot] >= bytes) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) hs->smem_optin[slot] = bytes;
  return e;
}

// Brackets the launches issued during its lifetime with two CUDA events when profiling is enabled.
struct ProfScope {
  ProfScope(int kernel, int launches, cudaStream_t stream);
  ~ProfScope();
  int slot;
  cudaStream_t stream;
  bool nvtx;
};

}  // namespace moin
