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
// `cta_budget` > 0: widen the tiles until the launch has at most that many CTAs (when it runs beside other kernels).
moin_status launch_tc_gemm(HostState* hs, const __nv_bfloat16* x, const __nv_bfloat16* W, __nv_bfloat16* y, float* y0,
                           int T, int d_in, int d_out, cudaStream_t stream, int cta_budget = 0);
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

// Causal GQA attention on tcgen05 (attention_tc.cu).  q not rotated, k rotated.
bool attention_tc_supported(int n_heads, int n_kv_heads, int head_dim);
moin_status launch_attention_tc(HostState* hs, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                const int* cu, __nv_bfloat16* out, const float2* rope, int R,
                                int T, int max_seqlen, int n_heads, int n_kv_heads, float scale_log2,
                                cudaStream_t stream);

}  // namespace moin
