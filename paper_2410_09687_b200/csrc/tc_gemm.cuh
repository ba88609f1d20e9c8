// tcgen05 / TMEM / TMA GEMM family (host-side interface).
#pragma once
#include "common.cuh"

namespace moin {

// Shape predicates (host): can the tcgen05 kernels take this problem?
bool tc_gemm_supported(int T, int d_in, int d_out);
bool tc_router_supported(int Q, int K, int D);
bool tc_fused_supported(int r);

// y = x W^T (bf16) and optionally y0 = x W^T (fp32).
moin_status launch_tc_gemm(HostState* hs, const __nv_bfloat16* x, const __nv_bfloat16* W, __nv_bfloat16* y, float* y0,
                           int T, int d_in, int d_out, cudaStream_t stream);
// keys[i] = max over k of (orderable(<q_i,c_k> * inv_norm[k]) << 32 | (0xFFFFFFFF - k)), merged with atomicMax.
moin_status launch_tc_router(HostState* hs, const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                             int Q, int K, int D, unsigned long long* keys, cudaStream_t stream);
// Tile mode: hb = bf16(s * x A_e^T) per row tile, then y = [x | hb] [W ; B_e]^T in one GEMM.
moin_status launch_tc_lora_tiles(HostState* hs, const PlanView& pv, const moin_pool* pool, const __nv_bfloat16* x,
                                 const __nv_bfloat16* W, __nv_bfloat16* y, __nv_bfloat16* hb, float scale,
                                 cudaStream_t stream);

}  // namespace moin
