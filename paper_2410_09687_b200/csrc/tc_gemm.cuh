// tcgen05 / TMEM / TMA GEMM family (host-side interface).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace moin {

// 2-D row-major bf16 tensor [rows, cols] -> TMA map with a [box_rows x 64] box, 128-byte swizzle, zero fill
// (columns of the box beyond `cols` read as zero).
moin_status make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);

// Shape predicates (host): can the tcgen05 kernels take this problem?
bool tc_gemm_supported(int T, int d_in, int d_out);
bool tc_router_supported(int Q, int K, int D);
bool tc_fused_supported(int r);

// y = x W^T (bf16) and optionally y0 = x W^T (fp32).
moin_status launch_tc_gemm(HostState* hs, const __nv_bfloat16* x, const __nv_bfloat16* W, __nv_bfloat16* y, float* y0,
                           int T, int d_in, int d_out, cudaStream_t stream);
// The same for up to kTcMaxStoreJobs projections that share T and d_in, in one launch that takes part in
// programmatic dependent launch (waits for the kernel before it, lets the kernel after it start beside it).
constexpr int kTcMaxStoreJobs = 3;
moin_status launch_tc_gemm_group(HostState* hs, const __nv_bfloat16* const* xs, const __nv_bfloat16* const* Ws,
                                 __nv_bfloat16* const* ys, float* const* y0s, const int* d_outs, int n_jobs, int T,
                                 int d_in, cudaStream_t stream);
// keys[i] = max over k of (orderable(<q_i,c_k> * inv_norm[k]) << 32 | (0xFFFFFFFF - k)), merged with atomicMax.
moin_status launch_tc_router(HostState* hs, const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                             int Q, int K, int D, unsigned long long* keys, cudaStream_t stream,
                             unsigned long long* keys2 = nullptr);   // keys2 != nullptr: also the runner-up
// Tile mode: hb = hi/lo bf16 parts of s * x A_e^T per row tile ([2][T][r]), then y = [x | hi | lo] [W ; B_e ; B_e]^T
// in one GEMM.
moin_status launch_tc_shrink_group(HostState* hs, const PlanView& pv, const moin_pool* const* pools,
                                   const __nv_bfloat16* const* xs, __nv_bfloat16* const* hbs, int n_jobs, float scale,
                                   cudaStream_t stream);
constexpr int kTcMaxShrinkJobs = 3;   // projections one grouped shrink launch can take
moin_status launch_tc_fused(HostState* hs, const PlanView& pv, const moin_pool* pool, const __nv_bfloat16* x,
                            const __nv_bfloat16* W, __nv_bfloat16* y, __nv_bfloat16* hb, cudaStream_t stream);

// TMA-staged segmented LoRA kernels (short segments), up to 4 projections per launch.  The shrink writes
// lora_stream_parts(d_in) partial results hpart[part][T][r] per projection; the expand sums them in index order.
// `queue` is one int of device scratch (the work counter, reset by the launcher on `stream`).
int lora_stream_parts(int d_in);
bool lora_shrink_tma_supported(int d_in);
size_t lora_stream_ring_bytes();
moin_status launch_lora_shrink_tma(HostState* hs, const PlanView& pv, const moin_pool* const* pools,
                                   const __nv_bfloat16* const* x, float* const* hpart, int n_jobs, int* queue,
                                   size_t ring_bytes, cudaStream_t stream);
moin_status launch_lora_expand_tma(HostState* hs, const PlanView& pv, const moin_pool* const* pools,
                                   const float* const* hpart, const int* parts, const float* const* y0,
                                   __nv_bfloat16* const* y, int n_jobs, float scale, int* queue, size_t ring_bytes,
                                   cudaStream_t stream);

}  // namespace moin
