// C ABI entry points: argument validation, workspace carving, kernel launches.
#include <string.h>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"
#include "tc_gemm.cuh"

namespace moin {

__device__ DeviceStatus g_device_status;

static thread_local int t_last_cuda_error = 0;
static HostState g_states[kMaxDevices];
static int g_opt_gemm_impl = 0, g_opt_nvtx = 0;   // moin_set_option: process-wide

moin_status record_cuda(cudaError_t e) {
  if (e == cudaSuccess) return MOIN_OK;
  t_last_cuda_error = (int)e;
  return MOIN_ERR_CUDA;
}

moin_status host_state(HostState** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { record_cuda(e); return MOIN_ERR_NO_DEVICE; }
  if (dev < 0 || dev >= kMaxDevices) return MOIN_ERR_NO_DEVICE;
  HostState& g_state = g_states[dev];
  if (g_state.device != dev) {
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) { record_cuda(e); return MOIN_ERR_NO_DEVICE; }
    if (prop.major != 10) return MOIN_ERR_NO_DEVICE;  // built for sm_100a only
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_device_status);
    if (e != cudaSuccess) return record_cuda(e);
    g_state.status = reinterpret_cast<DeviceStatus*>(p);
    if (g_state.ev_fork == nullptr) {
      e = cudaEventCreateWithFlags(&g_state.ev_fork, cudaEventDisableTiming);
      for (int j = 0; j < kMaxStreamJobs && e == cudaSuccess; ++j) {
        e = cudaStreamCreateWithFlags(&g_state.side[j], cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&g_state.ev_join[j], cudaEventDisableTiming);
      }
      if (e != cudaSuccess) return record_cuda(e);
    }
    g_state.n_sms = prop.multiProcessorCount;
    g_state.device = dev;
  }
  g_state.gemm_impl = g_opt_gemm_impl;
  *out = &g_state;
  return MOIN_OK;
}

// ---- profiling (per-kernel CUDA events; off by default)
struct ProfState {
  int capacity = 0, count = 0;
  cudaEvent_t* start = nullptr;
  cudaEvent_t* stop = nullptr;
  int* kernel = nullptr;
  int* launches = nullptr;
};
static ProfState g_prof;

ProfScope::ProfScope(int kernel, int launches, cudaStream_t s) : slot(-1), stream(s), nvtx(g_opt_nvtx != 0) {
  if (nvtx) nvtxRangePushA(moin_kernel_name(kernel));
  if (g_prof.capacity > 0 && g_prof.count < g_prof.capacity) {
    slot = g_prof.count++;
    g_prof.kernel[slot] = kernel;
    g_prof.launches[slot] = launches;
    cudaEventRecord(g_prof.start[slot], stream);
  }
}
ProfScope::~ProfScope() {
  if (slot >= 0) cudaEventRecord(g_prof.stop[slot], stream);
  if (nvtx) nvtxRangePop();
}

__global__ void set_int_kernel(int* p, int v) { *p = v; }

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace moin

using namespace moin;

extern "C" {

const char* moin_status_string(moin_status s) {
  switch (s) {
    case MOIN_OK: return "MOIN_OK";
    case MOIN_ERR_INVALID_ARG: return "MOIN_ERR_INVALID_ARG";
    case MOIN_ERR_BAD_SHAPE: return "MOIN_ERR_BAD_SHAPE";
    case MOIN_ERR_MISALIGNED: return "MOIN_ERR_MISALIGNED";
    case MOIN_ERR_WORKSPACE: return "MOIN_ERR_WORKSPACE";
    case MOIN_ERR_UNSUPPORTED_RANK: return "MOIN_ERR_UNSUPPORTED_RANK";
    case MOIN_ERR_CUDA: return "MOIN_ERR_CUDA";
    case MOIN_ERR_TIMEOUT: return "MOIN_ERR_TIMEOUT";
    case MOIN_ERR_NO_DEVICE: return "MOIN_ERR_NO_DEVICE";
    default: return "MOIN_ERR_UNKNOWN";
  }
}

int32_t moin_version(void) { return 100; }
int32_t moin_last_cuda_error(void) { return t_last_cuda_error; }

moin_status moin_set_option(int32_t key, int32_t value) {
  if (key == MOIN_OPT_GEMM_IMPL && value >= 0 && value <= 2) {
    g_opt_gemm_impl = value;
    return MOIN_OK;
  }
  if (key == MOIN_OPT_NVTX && (value == 0 || value == 1)) {
    g_opt_nvtx = value;
    return MOIN_OK;
  }
  return MOIN_ERR_INVALID_ARG;
}

moin_status moin_pool_set_adapter(const moin_pool* pool, int32_t expert, int32_t slot, const void* A_src,
                                  const void* B_src, moin_stream stream) {
  if (!pool || !pool->slot_of_expert || expert < 0 || expert >= pool->E || slot < -1 || slot >= pool->n_slots)
    return MOIN_ERR_INVALID_ARG;
  if (slot >= 0 && (!A_src || !B_src || !pool->A || !pool->B)) return MOIN_ERR_INVALID_ARG;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  cudaStream_t s = (cudaStream_t)stream;
  if (slot >= 0) {
    const size_t na = (size_t)pool->r * pool->d_in * sizeof(__nv_bfloat16), nb = (size_t)pool->d_out * pool->r * sizeof(__nv_bfloat16);
    char* A = const_cast<char*>(reinterpret_cast<const char*>(pool->A)) + (size_t)slot * na;
    char* B = const_cast<char*>(reinterpret_cast<const char*>(pool->B)) + (size_t)slot * nb;
    cudaError_t e = cudaMemcpyAsync(A, A_src, na, cudaMemcpyDefault, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(B, B_src, nb, cudaMemcpyDefault, s);
    if (e != cudaSuccess) return record_cuda(e);
  }
  set_int_kernel<<<1, 1, 0, s>>>(const_cast<int*>(pool->slot_of_expert) + expert, slot);   // after the copies, in stream order
  return record_cuda(cudaGetLastError());
}

moin_status moin_device_status(moin_device_status_t* out, moin_stream stream) {
  if (!out) return MOIN_ERR_INVALID_ARG;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  cudaStream_t s = (cudaStream_t)stream;
  static_assert(sizeof(moin_device_status_t) == sizeof(DeviceStatus), "status layout");
  cudaError_t e = cudaMemcpyAsync(out, hs->status, sizeof(DeviceStatus), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  return record_cuda(e);
}

moin_status moin_device_status_reset(moin_stream stream) {
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  return record_cuda(cudaMemsetAsync(hs->status, 0, sizeof(DeviceStatus), (cudaStream_t)stream));
}

moin_status moin_profile_enable(int32_t capacity) {
  if (capacity < 0) return MOIN_ERR_INVALID_ARG;
  for (int i = 0; i < g_prof.capacity; ++i) {
    cudaEventDestroy(g_prof.start[i]);
    cudaEventDestroy(g_prof.stop[i]);
  }
  delete[] g_prof.start; delete[] g_prof.stop; delete[] g_prof.kernel; delete[] g_prof.launches;
  g_prof = ProfState();
  if (capacity == 0) return MOIN_OK;
  g_prof.start = new cudaEvent_t[capacity];
  g_prof.stop = new cudaEvent_t[capacity];
  g_prof.kernel = new int[capacity];
  g_prof.launches = new int[capacity];
  for (int i = 0; i < capacity; ++i) {
    cudaError_t e = cudaEventCreate(&g_prof.start[i]);
    if (e == cudaSuccess) e = cudaEventCreate(&g_prof.stop[i]);
    if (e != cudaSuccess) return record_cuda(e);
  }
  g_prof.capacity = capacity;
  return MOIN_OK;
}

moin_status moin_profile_read(moin_profile_record* out, int32_t capacity, int32_t* n) {
  if (!n || capacity < 0 || (capacity > 0 && !out)) return MOIN_ERR_INVALID_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return record_cuda(e);
  *n = g_prof.count;
  for (int i = 0; i < g_prof.count && i < capacity; ++i) {
    out[i].kernel = g_prof.kernel[i];
    out[i].launches = g_prof.launches[i];
    out[i].ms = 0.f;
    cudaEventElapsedTime(&out[i].ms, g_prof.start[i], g_prof.stop[i]);
  }
  g_prof.count = 0;
  return MOIN_OK;
}

const char* moin_kernel_name(int32_t k) {
  static const char* names[MOIN_K_COUNT] = {"route_simple", "route_tc", "route_finish", "plan", "gemm_warp", "gemm_tc",
                                            "lora_shrink_stream", "lora_expand_stream", "lora_shrink_tc",
                                            "lora_fused_tc", "decoder_glue", "attention", "route_cluster", "kmeans_update"};
  return (k >= 0 && k < MOIN_K_COUNT) ? names[k] : "unknown";
}

/* ------------------------------------------------------------------ router */

moin_status moin_router_prepare(const void* centroids, int32_t K, int32_t D, float* inv_norm, moin_stream stream) {
  if (!centroids || !inv_norm || K < 1) return MOIN_ERR_INVALID_ARG;
  if (D < 8 || D > 8192 || (D % 8) != 0) return MOIN_ERR_BAD_SHAPE;
  if (!aligned16(centroids)) return MOIN_ERR_MISALIGNED;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  ProfScope prof(MOIN_K_GLUE, 1, (cudaStream_t)stream);
  return record_cuda(launch_inv_norm((const __nv_bfloat16*)centroids, K, D, inv_norm, (cudaStream_t)stream));
}

size_t moin_route_workspace_bytes(int32_t Q, int32_t K, int32_t D) {
  (void)K; (void)D;
  return align_up((size_t)(Q > 0 ? Q : 0) * sizeof(unsigned long long), 256) + 256;
}

// Kernel choice shared by moin_route and moin_route_static, so that both compute the same values for the same
// shapes and options: 0 = cluster kernel (decode-sized batch: one launch, no scratch), 1 = tensor-core GEMM with
// one 64-bit key of scratch per query, 2 = CUDA-core kernel (no scratch).
static moin_status route_choice(const HostState* hs, int Q, int K, int D, int* choice) {
  const bool tc_ok = tc_router_supported(Q, K, D);
  bool use_tc = tc_ok && (long long)Q * K >= (1ll << 16);
  if (hs->gemm_impl == 1) use_tc = false;
  if (hs->gemm_impl == 2) {
    if (!tc_ok) return MOIN_ERR_BAD_SHAPE;
    use_tc = true;
  }
  if (hs->gemm_impl == 0 && route_cluster_supported(Q, K, D)) *choice = 0;
  else *choice = use_tc ? 1 : 2;
  return MOIN_OK;
}

static moin_status route_launch(HostState* hs, int choice, const moin_router* router, const void* queries, int Q,
                                int32_t* out_expert, int32_t* out_centroid, float* out_best_sim,
                                unsigned long long* keys, cudaStream_t s) {
  const int K = router->K, D = router->D;
  if (choice == 0) {
    ProfScope prof(MOIN_K_ROUTE_CLUSTER, 1, s);
    return record_cuda(launch_route_cluster((const __nv_bfloat16*)queries, (const __nv_bfloat16*)router->centroids,
                                            router->inv_norm, router->centroid_to_expert, Q, K, D, out_expert,
                                            out_centroid, out_best_sim, s));
  }
  if (choice == 1) {
    // the merge across column tiles is a max, so the keys must start from zero
    cudaError_t e = cudaMemsetAsync(keys, 0, (size_t)Q * sizeof(unsigned long long), s);
    if (e != cudaSuccess) return record_cuda(e);
    moin_status st;
    {
      ProfScope prof(MOIN_K_ROUTE_TC, 1, s);
      st = launch_tc_router(hs, (const __nv_bfloat16*)queries, (const __nv_bfloat16*)router->centroids,
                            router->inv_norm, Q, K, D, keys, s);
    }
    if (st) return st;
    ProfScope prof(MOIN_K_ROUTE_FINISH, 1, s);
    return record_cuda(launch_route_finish(keys, (const __nv_bfloat16*)queries, router->centroid_to_expert, Q, D,
                                           out_expert, out_centroid, out_best_sim, s));
  }
  ProfScope prof(MOIN_K_ROUTE_SIMPLE, 1, s);
  return record_cuda(launch_route_simple((const __nv_bfloat16*)queries, (const __nv_bfloat16*)router->centroids,
                                         router->inv_norm, router->centroid_to_expert, Q, K, D, out_expert,
                                         out_centroid, out_best_sim, s));
}

static moin_status route_check(const moin_router* router, const void* queries, int32_t Q, const int32_t* out_expert) {
  if (!router || Q < 0) return MOIN_ERR_INVALID_ARG;
  if (Q == 0) return MOIN_OK;
  if (!queries || !out_expert || !router->centroids || !router->inv_norm || router->K < 1) return MOIN_ERR_INVALID_ARG;
  const int D = router->D;
  if (D < 8 || D > 8192 || (D % 8) != 0) return MOIN_ERR_BAD_SHAPE;
  if (!aligned16(queries) || !aligned16(router->centroids)) return MOIN_ERR_MISALIGNED;
  return MOIN_OK;
}

moin_status moin_route(const moin_router* router, const void* queries, int32_t Q, int32_t* out_expert,
                       int32_t* out_centroid, float* out_best_sim, void* workspace, size_t workspace_bytes,
                       moin_stream stream) {
  moin_status st = route_check(router, queries, Q, out_expert);
  if (st || Q == 0) return st;
  HostState* hs;
  if ((st = host_state(&hs))) return st;
  int choice;
  if ((st = route_choice(hs, Q, router->K, router->D, &choice))) return st;
  if (choice == 1 && (!workspace || workspace_bytes < moin_route_workspace_bytes(Q, router->K, router->D) ||
                      !aligned16(workspace)))
    return MOIN_ERR_WORKSPACE;
  return route_launch(hs, choice, router, queries, Q, out_expert, out_centroid, out_best_sim,
                      reinterpret_cast<unsigned long long*>(workspace), (cudaStream_t)stream);
}

size_t moin_route_top2_workspace_bytes(int32_t Q, int32_t K, int32_t D) {
  (void)K; (void)D;
  return 2 * align_up((size_t)(Q > 0 ? Q : 0) * sizeof(unsigned long long), 256) + 256;
}

moin_status moin_route_top2(const moin_router* router, const void* queries, int32_t Q, int32_t* out_expert,
                            int32_t* out_centroid, int32_t* out_second, float* out_best_sim, float* out_margin,
                            void* workspace, size_t workspace_bytes, moin_stream stream) {
  if (!router || Q < 0) return MOIN_ERR_INVALID_ARG;
  if (Q == 0) return MOIN_OK;
  if (!queries || !router->centroids || !router->inv_norm || router->K < 1) return MOIN_ERR_INVALID_ARG;
  const int K = router->K, D = router->D;
  if (D < 8 || D > 8192 || (D % 8) != 0) return MOIN_ERR_BAD_SHAPE;
  if (!aligned16(queries) || !aligned16(router->centroids)) return MOIN_ERR_MISALIGNED;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  cudaStream_t s = (cudaStream_t)stream;
  const bool tc_ok = tc_router_supported(Q, K, D);
  bool use_tc = tc_ok && (long long)Q * K >= (1ll << 16);
  if (hs->gemm_impl == 1) use_tc = false;
  if (hs->gemm_impl == 2) {
    if (!tc_ok) return MOIN_ERR_BAD_SHAPE;
    use_tc = true;
  }
  if (!use_tc) {
    ProfScope prof(MOIN_K_ROUTE_SIMPLE, 1, s);
    return record_cuda(launch_route_top2_simple((const __nv_bfloat16*)queries, (const __nv_bfloat16*)router->centroids,
                                                router->inv_norm, router->centroid_to_expert, Q, K, D, out_expert,
                                                out_centroid, out_second, out_best_sim, out_margin, s));
  }
  if (!workspace || workspace_bytes < moin_route_top2_workspace_bytes(Q, K, D) || !aligned16(workspace))
    return MOIN_ERR_WORKSPACE;
  const size_t half = align_up((size_t)Q * sizeof(unsigned long long), 256);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(workspace);
  unsigned long long* keys2 = reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(workspace) + half);
  cudaError_t e = cudaMemsetAsync(workspace, 0, 2 * half, s);
  if (e != cudaSuccess) return record_cuda(e);
  {
    ProfScope prof(MOIN_K_ROUTE_TC, 1, s);
    st = launch_tc_router(hs, (const __nv_bfloat16*)queries, (const __nv_bfloat16*)router->centroids, router->inv_norm,
                          Q, K, D, keys, s, keys2);
  }
  if (st) return st;
  ProfScope prof(MOIN_K_ROUTE_FINISH, 1, s);
  return record_cuda(launch_route_finish_top2(keys, keys2, (const __nv_bfloat16*)queries, router->centroid_to_expert, Q, D,
                                              out_expert, out_centroid, out_second, out_best_sim, out_margin, s));
}

/* Scratch of moin_route_static: one 64-bit (similarity, index) key per query.  In host code the name
 * `g_route_static_keys` is only a handle for the runtime, not a device address; the address handed to
 * kernels comes from cudaGetSymbolAddress, looked up once per device. */
static __device__ __align__(256) unsigned long long g_route_static_keys[MOIN_ROUTE_STATIC_MAX_Q];
static unsigned long long* g_route_static_ptr[kMaxDevices] = {nullptr};

moin_status moin_route_static(const moin_router* router, const void* queries, int32_t Q, int32_t* out_expert,
                              int32_t* out_centroid, float* out_best_sim, moin_stream stream) {
  moin_status st = route_check(router, queries, Q, out_expert);
  if (st || Q == 0) return st;
  if (Q > MOIN_ROUTE_STATIC_MAX_Q) return MOIN_ERR_WORKSPACE;   // beyond the built-in scratch
  HostState* hs;
  if ((st = host_state(&hs))) return st;
  int choice;
  if ((st = route_choice(hs, Q, router->K, router->D, &choice))) return st;
  unsigned long long* keys = nullptr;
  if (choice == 1) {   // only the tensor-core kernel needs scratch
    if (g_route_static_ptr[hs->device] == nullptr) {   // set-up: once per device, that device is current here
      void* p = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&p, g_route_static_keys);
      if (e != cudaSuccess) return record_cuda(e);
      g_route_static_ptr[hs->device] = reinterpret_cast<unsigned long long*>(p);
    }
    keys = g_route_static_ptr[hs->device];   // still holds the previous call's keys: route_launch clears Q of them
  }
  return route_launch(hs, choice, router, queries, Q, out_expert, out_centroid, out_best_sim, keys,
                      (cudaStream_t)stream);
}

/* ------------------------------------------------------------------ K-means update */

moin_status moin_kmeans_update(const moin_plan* plan, const void* x, const void* centroids_old, void* centroids_new,
                               float* inv_norm_new, int32_t D, moin_stream stream) {
  if (!plan || plan->T < 0 || plan->E < 1 || !centroids_old || !centroids_new) return MOIN_ERR_INVALID_ARG;
  if (D < 8 || D > 8192 || (D % 8) != 0) return MOIN_ERR_BAD_SHAPE;
  if (plan->T > 0 && (!x || !plan->buffer)) return MOIN_ERR_INVALID_ARG;
  if (!aligned16(centroids_old) || !aligned16(centroids_new) || (x && !aligned16(x))) return MOIN_ERR_MISALIGNED;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  cudaStream_t s = (cudaStream_t)stream;
  const int K = plan->E;
  if (centroids_new != centroids_old) {   // clusters without members keep their centroid
    cudaError_t e = cudaMemcpyAsync(centroids_new, centroids_old, (size_t)K * (size_t)D * sizeof(__nv_bfloat16),
                                    cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return record_cuda(e);
  }
  if (plan->T > 0) {
    PlanView pv = plan_view(plan->buffer, plan->T, plan->E);
    ProfScope prof(MOIN_K_KMEANS_UPDATE, 1, s);
    st = record_cuda(launch_kmeans_mean(pv, (const __nv_bfloat16*)x, (__nv_bfloat16*)centroids_new, D, hs->n_sms, s));
    if (st) return st;
  }
  if (inv_norm_new) {
    ProfScope prof(MOIN_K_GLUE, 1, s);
    return record_cuda(launch_inv_norm((const __nv_bfloat16*)centroids_new, K, D, inv_norm_new, s));
  }
  return MOIN_OK;
}

/* ------------------------------------------------------------------ plan */

size_t moin_plan_bytes(int32_t T, int32_t E) {
  if (T < 0 || E < 0) return 0;
  return align_up(plan_bytes(T, E), 256);
}

moin_status moin_plan_build(const int32_t* token_expert, moin_plan* plan, moin_stream stream) {
  if (!plan || plan->T < 0 || plan->E < 1) return MOIN_ERR_INVALID_ARG;
  if (plan->mode < MOIN_PLAN_AUTO || plan->mode > MOIN_PLAN_TILES) return MOIN_ERR_INVALID_ARG;
  if (plan->T == 0) return MOIN_OK;
  if (!token_expert || !plan->buffer) return MOIN_ERR_INVALID_ARG;
  if (!aligned16(plan->buffer)) return MOIN_ERR_MISALIGNED;
  if (plan->buffer_bytes < plan_bytes(plan->T, plan->E)) return MOIN_ERR_WORKSPACE;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  cudaStream_t s = (cudaStream_t)stream;
  PlanView v = plan_view(plan->buffer, plan->T, plan->E);
  {
    ProfScope prof(MOIN_K_PLAN, plan_launches(plan->T, plan->E), s);
    // the tile list serves the long-run kernels and the AUTO decision; a SEGMENTS plan leaves it empty
    st = record_cuda(launch_plan_build(token_expert, v, hs->status, plan->mode != MOIN_PLAN_SEGMENTS, s));
  }
  if (st) return st;
  if (plan->mode == MOIN_PLAN_AUTO) {
    int header[kPlanHeaderWords];
    cudaError_t e = cudaMemcpyAsync(header, v.header, sizeof(header), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return record_cuda(e);
    plan->n_segments = header[PH_NSEG];
    plan->n_tiles = header[PH_NTILES];
    plan->n_lora_tokens = header[PH_NLORA];
    plan->max_segment = header[PH_MAXSEG];
    // Long runs (few, well-filled 128-row tiles) -> fold the adapter into the tensor-core GEMM.
    const int full_tiles = (plan->T + kTileRows - 1) / kTileRows;
    plan->mode = (plan->T >= 2 * kTileRows && plan->n_tiles <= full_tiles + full_tiles / 2) ? MOIN_PLAN_TILES
                                                                                         : MOIN_PLAN_SEGMENTS;
  }
  return MOIN_OK;
}

moin_status moin_plan_read(const moin_plan* plan, int32_t* n_segments, int32_t* n_tiles, int32_t* perm,
                           int32_t* seg_expert, int32_t* seg_start, int32_t* tile_row0, int32_t* tile_rows,
                           int32_t* tile_expert, moin_stream stream) {
  if (!plan || !plan->buffer || plan->T < 1) return MOIN_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  PlanView v = plan_view(plan->buffer, plan->T, plan->E);
  int header[kPlanHeaderWords];
  cudaError_t e = cudaMemcpyAsync(header, v.header, sizeof(header), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return record_cuda(e);
  const int S = header[PH_NSEG], NT = header[PH_NTILES];
  if (n_segments) *n_segments = S;
  if (n_tiles) *n_tiles = NT;
  auto copy = [&](int32_t* dst, const int* src, size_t n) {
    if (dst && n && e == cudaSuccess) e = cudaMemcpyAsync(dst, src, n * sizeof(int), cudaMemcpyDeviceToHost, s);
  };
  copy(perm, v.perm, (size_t)plan->T);
  copy(seg_expert, v.seg_expert, (size_t)S);
  copy(seg_start, v.seg_start, (size_t)S + 1);
  copy(tile_row0, v.tile_row0, (size_t)NT);
  copy(tile_rows, v.tile_rows, (size_t)NT);
  copy(tile_expert, v.tile_expert, (size_t)NT);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  return record_cuda(e);
}

/* ------------------------------------------------------------------ routed LoRA linear layer */

size_t moin_lora_linear_workspace_bytes(int32_t T, int32_t d_in, int32_t d_out, int32_t r) {
  if (T <= 0) return 256;
  const size_t Tp = align_up((size_t)T, kTileRows) + kTileRows;
  (void)d_in;
  size_t seg = align_up((size_t)T * (size_t)(r > 0 ? r : 8) * sizeof(float), 256) +
               align_up((size_t)T * (size_t)d_out * sizeof(float), 256);
  size_t tiles = align_up(2 * Tp * (size_t)(r > 64 ? r : 64) * sizeof(__nv_bfloat16), 256);   // hi and lo parts of s * (x A^T)
  return (seg > tiles ? seg : tiles) + 256;
}

// Checks one projection job; fills T / d_in / d_out / r.  `lora` = the job carries an adapter pool.
static moin_status check_job(const moin_plan* plan, const void* x, const void* W, const moin_pool* pool, const void* y,
                             bool lora, int base_T, int base_d_in, int base_d_out, int* T, int* d_in, int* d_out,
                             int* r) {
  *T = lora ? plan->T : base_T;
  *d_in = lora ? pool->d_in : base_d_in;
  *d_out = lora ? pool->d_out : base_d_out;
  *r = 0;
  if (*T < 0) return MOIN_ERR_INVALID_ARG;
  if (*T == 0) return MOIN_OK;
  if (!x || !W || !y || x == y) return MOIN_ERR_INVALID_ARG;
  if (*d_in < 64 || (*d_in % 64) != 0 || *d_out < 8 || (*d_out % 8) != 0) return MOIN_ERR_BAD_SHAPE;
  if (!aligned16(x) || !aligned16(W) || !aligned16(y)) return MOIN_ERR_MISALIGNED;
  if (lora) {
    *r = pool->r;
    if (*r < 8 || *r > 128 || (*r % 8) != 0) return MOIN_ERR_UNSUPPORTED_RANK;
    if (!pool->A || !pool->B || !pool->slot_of_expert || !plan->buffer) return MOIN_ERR_INVALID_ARG;
    if (pool->E != plan->E) return MOIN_ERR_INVALID_ARG;
    if (pool->activation < MOIN_ACT_NONE || pool->activation > MOIN_ACT_GELU) return MOIN_ERR_INVALID_ARG;
    if (!aligned16(pool->A) || !aligned16(pool->B)) return MOIN_ERR_MISALIGNED;
    if (plan->mode != MOIN_PLAN_SEGMENTS && plan->mode != MOIN_PLAN_TILES) return MOIN_ERR_INVALID_ARG;
  }
  return MOIN_OK;
}

static moin_status pick_gemm(const HostState* hs, int T, int d_in, int d_out, bool* use_tc) {
  const bool tc_ok = tc_gemm_supported(T, d_in, d_out);
  *use_tc = tc_ok && T >= 64 && d_out >= 64;
  if (hs->gemm_impl == 1) *use_tc = false;
  if (hs->gemm_impl == 2) {
    if (!tc_ok) return MOIN_ERR_BAD_SHAPE;
    *use_tc = true;
  }
  return MOIN_OK;
}

size_t moin_lora_linear_group_workspace_bytes(int32_t T, const moin_lora_job* jobs, int32_t n_jobs) {
  size_t total = 0;   // the per-projection sizes are multiples of 256 and carry their own slack
  for (int j = 0; jobs && j < n_jobs; ++j)
    if (jobs[j].pool)
      total += align_up(moin_lora_linear_workspace_bytes(T, jobs[j].pool->d_in, jobs[j].pool->d_out, jobs[j].pool->r), 256);
  return total;
}

moin_status moin_lora_linear_group(const moin_plan* plan, const moin_lora_job* jobs, int32_t n_jobs, float scale,
                                   void* workspace, size_t workspace_bytes, moin_stream stream) {
  if (!plan || !jobs || n_jobs < 1 || n_jobs > MOIN_MAX_GROUP) return MOIN_ERR_INVALID_ARG;
  int T = 0, d_in[kMaxStreamJobs], d_out[kMaxStreamJobs], r[kMaxStreamJobs];
  for (int j = 0; j < n_jobs; ++j) {
    if (!jobs[j].pool) return MOIN_ERR_INVALID_ARG;
    moin_status st = check_job(plan, jobs[j].x, jobs[j].W, jobs[j].pool, jobs[j].y, true, 0, 0, 0, &T, &d_in[j],
                               &d_out[j], &r[j]);
    if (st) return st;
  }
  if (T == 0) return MOIN_OK;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  if (!workspace || !aligned16(workspace) || workspace_bytes < moin_lora_linear_group_workspace_bytes(T, jobs, n_jobs))
    return MOIN_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  PlanView pv = plan_view(plan->buffer, plan->T, plan->E);
  char* ws = reinterpret_cast<char*>(workspace);
  char* ws_job[kMaxStreamJobs];
  bool use_tc[kMaxStreamJobs];
  for (int j = 0; j < n_jobs; ++j) {
    ws_job[j] = ws;
    ws += align_up(moin_lora_linear_workspace_bytes(T, d_in[j], d_out[j], r[j]), 256);
    if ((st = pick_gemm(hs, T, d_in[j], d_out[j], &use_tc[j]))) return st;
  }

  if (plan->mode == MOIN_PLAN_TILES) {
    // Long runs: every projection is one grouped-shrink + one fused GEMM launch on the tensor cores.
    bool all_tc = true;
    for (int j = 0; j < n_jobs; ++j) all_tc = all_tc && use_tc[j] && tc_fused_supported(r[j]);
    if (all_tc) {
      // shrinks first: projections with the same d_in and rank share one launch (up to kTcMaxShrinkJobs)
      for (int j0 = 0; j0 < n_jobs;) {
        const moin_pool* gp[kTcMaxShrinkJobs];
        const __nv_bfloat16* gx[kTcMaxShrinkJobs];
        __nv_bfloat16* gh[kTcMaxShrinkJobs];
        int n = 0;
        while (j0 + n < n_jobs && n < kTcMaxShrinkJobs && d_in[j0 + n] == d_in[j0] && r[j0 + n] == r[j0] &&
               jobs[j0 + n].pool->activation == jobs[j0].pool->activation) {
          gp[n] = jobs[j0 + n].pool;
          gx[n] = (const __nv_bfloat16*)jobs[j0 + n].x;
          gh[n] = reinterpret_cast<__nv_bfloat16*>(ws_job[j0 + n]);
          ++n;
        }
        if ((st = launch_tc_shrink_group(hs, pv, gp, gx, gh, n, scale, s))) return st;
        j0 += n;
      }
      for (int j = 0; j < n_jobs; ++j) {
        st = launch_tc_fused(hs, pv, jobs[j].pool, (const __nv_bfloat16*)jobs[j].x, (const __nv_bfloat16*)jobs[j].W,
                             (__nv_bfloat16*)jobs[j].y, reinterpret_cast<__nv_bfloat16*>(ws_job[j]), s);
        if (st) return st;
      }
      return MOIN_OK;
    }
  }
  // Short segments.  Per projection: y0 = x W^T (fp32 + bf16 copy), h = x A_e^T, y = bf16(y0 + s h B_e^T).
  // The base GEMMs do not depend on the shrink, so each runs on one of the library's side streams between
  // a fork and a join event, concurrently with the shrink; the shrink and the expand each cover all the
  // projections of the group in ONE launch, so their launch and ramp-up costs are paid once per group.
  float* h[kMaxStreamJobs];
  float* y0[kMaxStreamJobs];
  for (int j = 0; j < n_jobs; ++j) {
    h[j] = reinterpret_cast<float*>(ws_job[j]);   // [T][r] shrink results
    y0[j] = reinterpret_cast<float*>(ws_job[j] + align_up((size_t)T * (size_t)r[j] * sizeof(float), 256));
  }
  cudaError_t ce = cudaEventRecord(hs->ev_fork, s);
  if (ce != cudaSuccess) return record_cuda(ce);
  moin_status st_gemm = MOIN_OK;
  for (int j = 0; j < n_jobs; ++j) {
    ce = cudaStreamWaitEvent(hs->side[j], hs->ev_fork, 0);
    if (ce != cudaSuccess) return record_cuda(ce);
    ProfScope prof(use_tc[j] ? MOIN_K_GEMM_TC : MOIN_K_GEMM_WARP, 1, hs->side[j]);
    moin_status sj;
    if (use_tc[j])   // the group's base GEMMs together get three quarters of the SMs, the shrink beside them the rest
      sj = launch_tc_gemm(hs, (const __nv_bfloat16*)jobs[j].x, (const __nv_bfloat16*)jobs[j].W, (__nv_bfloat16*)jobs[j].y,
                          y0[j], T, d_in[j], d_out[j], hs->side[j], hs->n_sms * 3 / 4 / n_jobs);
    else
      sj = record_cuda(launch_gemm_warp((const __nv_bfloat16*)jobs[j].x, (const __nv_bfloat16*)jobs[j].W,
                                        (__nv_bfloat16*)jobs[j].y, y0[j], T, d_in[j], d_out[j], hs->side[j]));
    if (sj && !st_gemm) st_gemm = sj;
  }
  moin_status st_shrink;
  {
    ProfScope prof(MOIN_K_SHRINK_STREAM, 1, s);
    ShrinkJobs sj = {};
    sj.n = n_jobs;
    for (int j = 0; j < n_jobs; ++j) {
      sj.x[j] = (const __nv_bfloat16*)jobs[j].x;
      sj.A[j] = (const __nv_bfloat16*)jobs[j].pool->A;
      sj.h[j] = h[j];
      sj.slot_of_expert[j] = jobs[j].pool->slot_of_expert;
      sj.slot_rank[j] = jobs[j].pool->slot_rank;
      sj.r[j] = r[j];
      sj.d_in[j] = d_in[j];
    }
    st_shrink = record_cuda(launch_lora_shrink_stream(pv, sj, hs->n_sms, s));
  }
  // always join, even after a failed launch, so the side streams never outlive the call's ordering
  for (int j = 0; j < n_jobs; ++j) {
    ce = cudaEventRecord(hs->ev_join[j], hs->side[j]);
    if (ce == cudaSuccess) ce = cudaStreamWaitEvent(s, hs->ev_join[j], 0);
    if (ce != cudaSuccess) return record_cuda(ce);
  }
  if (st_gemm) return st_gemm;
  if (st_shrink) return st_shrink;
  ProfScope prof(MOIN_K_EXPAND_STREAM, 1, s);
  ExpandJobs ej = {};
  ej.n = n_jobs;
  for (int j = 0; j < n_jobs; ++j) {
    ej.h[j] = h[j];
    ej.B[j] = (const __nv_bfloat16*)jobs[j].pool->B;
    ej.y0[j] = y0[j];
    ej.y[j] = (__nv_bfloat16*)jobs[j].y;
    ej.slot_of_expert[j] = jobs[j].pool->slot_of_expert;
    ej.slot_rank[j] = jobs[j].pool->slot_rank;
    ej.act[j] = jobs[j].pool->activation;
    ej.r[j] = r[j];
    ej.d_out[j] = d_out[j];
  }
  return record_cuda(launch_lora_expand_stream(pv, ej, scale, hs->n_sms, s));
}

moin_status moin_lora_linear(const moin_plan* plan, const void* x, const void* W, const moin_pool* pool,
                             float scale, int32_t base_T, int32_t base_d_in, int32_t base_d_out, void* y,
                             void* workspace, size_t workspace_bytes, moin_stream stream) {
  const bool lora = (plan != nullptr && pool != nullptr);
  if (lora) {   // one-job group
    moin_lora_job job = {x, W, pool, y};
    if (plan->T > 0 && workspace_bytes < moin_lora_linear_workspace_bytes(plan->T, pool->d_in, pool->d_out, pool->r))
      return MOIN_ERR_WORKSPACE;
    return moin_lora_linear_group(plan, &job, 1, scale, workspace, workspace_bytes, stream);
  }
  int T, d_in, d_out, r;
  moin_status st = check_job(plan, x, W, pool, y, false, base_T, base_d_in, base_d_out, &T, &d_in, &d_out, &r);
  if (st || T == 0) return st;
  HostState* hs;
  if ((st = host_state(&hs))) return st;
  bool use_tc;
  if ((st = pick_gemm(hs, T, d_in, d_out, &use_tc))) return st;
  cudaStream_t s = (cudaStream_t)stream;
  ProfScope prof(use_tc ? MOIN_K_GEMM_TC : MOIN_K_GEMM_WARP, 1, s);
  if (use_tc) return launch_tc_gemm(hs, (const __nv_bfloat16*)x, (const __nv_bfloat16*)W, (__nv_bfloat16*)y, nullptr, T, d_in, d_out, s);
  return record_cuda(launch_gemm_warp((const __nv_bfloat16*)x, (const __nv_bfloat16*)W, (__nv_bfloat16*)y, nullptr, T, d_in, d_out, s));
}

}  // extern "C"
