"""B200-native MoIN serving hot path: thin Python binding over the C-ABI CUDA library.

The binding only marshals arguments (torch tensors -> device pointers); every step of the
path runs in the library's CUDA kernels.  There is no CPU or PyTorch fallback: if the
library is missing or no sm_100 GPU is present, calls raise.
"""
from .binding import (MoinError, Router, Pool, Plan, DecoderModel, lib, lib_path, route, route_top2, route_static, ROUTE_STATIC_MAX_Q, plan_build, kmeans_update, AdapterCache, lora_linear, lora_linear_group, JobGroup,
                      decoder_forward, dequant_fp8, pool_set_adapter, device_status, device_status_reset, selftest_bounded_wait, set_option, profile_enable, profile_read, PLAN_AUTO, PLAN_SEGMENTS,
                      PLAN_TILES, LOGITS_ALL, LOGITS_LAST, LOGITS_NONE, OPT_GEMM_IMPL, OPT_NVTX, ACT_NONE, ACT_RELU, ACT_SILU, ACT_GELU, EXPORTED_SYMBOLS)

__all__ = ["MoinError", "Router", "Pool", "Plan", "DecoderModel", "lib", "lib_path", "route", "route_top2", "route_static", "ROUTE_STATIC_MAX_Q", "plan_build", "kmeans_update", "AdapterCache",
           "lora_linear", "lora_linear_group", "JobGroup", "decoder_forward", "dequant_fp8", "pool_set_adapter", "device_status", "device_status_reset", "selftest_bounded_wait", "set_option", "profile_enable", "profile_read", "PLAN_AUTO",
           "PLAN_SEGMENTS", "PLAN_TILES", "LOGITS_ALL", "LOGITS_LAST", "LOGITS_NONE", "OPT_GEMM_IMPL", "OPT_NVTX", "ACT_NONE", "ACT_RELU", "ACT_SILU", "ACT_GELU",
           "EXPORTED_SYMBOLS"]
