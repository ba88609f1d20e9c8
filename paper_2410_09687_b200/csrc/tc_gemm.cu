// placeholder until the tcgen05 kernels land: nothing is supported, callers use the warp-MMA paths
#include "tc_gemm.cuh"
namespace moin {
bool tc_gemm_supported(int, int, int) { return false; }
bool tc_router_supported(int, int, int) { return false; }
bool tc_fused_supported(int) { return false; }
moin_status launch_tc_gemm(HostState*, const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*, float*, int, int, int, cudaStream_t) { return MOIN_ERR_BAD_SHAPE; }
moin_status launch_tc_router(HostState*, const __nv_bfloat16*, const __nv_bfloat16*, const float*, int, int, int, unsigned long long*, cudaStream_t) { return MOIN_ERR_BAD_SHAPE; }
moin_status launch_tc_lora_tiles(HostState*, const PlanView&, const moin_pool*, const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*, __nv_bfloat16*, float, cudaStream_t) { return MOIN_ERR_BAD_SHAPE; }
}
