// Query router kernels: centroid inverse norms, the CUDA-core cosine-argmax kernel used for
// small problems and odd shapes, and the finishing pass shared with the tensor-core router.
#include "common.cuh"

namespace moin {

// inv_norm[k] = 1/|c_k| (0 for a zero row).  One warp per centroid.
__global__ void __launch_bounds__(256)
centroid_inv_norm_kernel(const __nv_bfloat16* __restrict__ c, int K, int D, float* __restrict__ inv_norm) {
  const int k = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (k >= K) return;
  const __nv_bfloat16* row = c + (size_t)k * D;
  float s = 0.f;
  for (int ch = lane; ch < D / 8; ch += 32) {
    const uint4 v = ldg_cached(row + ch * 8);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float a = bf16_lo(w[q]), b = bf16_hi(w[q]);
      s = fmaf(a, a, s);
      s = fmaf(b, b, s);
    }
  }
  s = warp_sum(s);
  if (lane == 0) inv_norm[k] = (s > 0.f) ? rsqrtf(s) : 0.f;
}

constexpr int kRouteQB = 8;  // queries per CTA

// One CTA = 8 queries (bf16 in shared memory), 4 warps striding over centroids.
// sim = <q, c_k> * inv_norm[k]; strict '>' keeps the lowest index on ties; NaN never wins.
__global__ void __launch_bounds__(128)
route_simple_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ c,
                    const float* __restrict__ inv_norm, const int* __restrict__ cmap, int Q, int K, int D,
                    int* __restrict__ out_expert, int* __restrict__ out_centroid, float* __restrict__ out_best) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* sq = reinterpret_cast<uint4*>(smem_raw);  // [8][D/8]
  __shared__ float s_best[4][kRouteQB];
  __shared__ int s_id[4][kRouteQB];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int q0 = blockIdx.x * kRouteQB;
  const int nch = D / 8;
  for (int i = tid; i < kRouteQB * nch; i += 128) {
    const int qi = i / nch, ch = i - qi * nch;
    sq[i] = (q0 + qi < Q) ? ldg_cached(q + (size_t)(q0 + qi) * D + ch * 8) : make_uint4(0, 0, 0, 0);
  }
  __syncthreads();
  float best = -INFINITY;
  int best_id = 0;
  for (int k = warp; k < K; k += 4) {
    float acc[kRouteQB];
#pragma unroll
    for (int j = 0; j < kRouteQB; ++j) acc[j] = 0.f;
    const __nv_bfloat16* crow = c + (size_t)k * D;
    for (int ch = lane; ch < nch; ch += 32) {
      const uint4 cv = ldg_cached(crow + ch * 8);
      const uint32_t cw[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
      for (int j = 0; j < kRouteQB; ++j) {
        const uint4 qv = sq[j * nch + ch];
        const uint32_t qw[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          acc[j] = fmaf(bf16_lo(cw[e]), bf16_lo(qw[e]), acc[j]);
          acc[j] = fmaf(bf16_hi(cw[e]), bf16_hi(qw[e]), acc[j]);
        }
      }
    }
    const float inv = inv_norm[k];
#pragma unroll
    for (int j = 0; j < kRouteQB; ++j) {
      const float dot = warp_sum(acc[j]);
      const float sim = (inv > 0.f) ? dot * inv : -INFINITY;
      if (lane == j && sim > best) {
        best = sim;
        best_id = k;
      }
    }
  }
  if (lane < kRouteQB) {
    s_best[warp][lane] = best;
    s_id[warp][lane] = best_id;
  }
  __syncthreads();
  if (tid < kRouteQB && q0 + tid < Q) {
    float b = -INFINITY;
    int id = INT_MAX;
    for (int w = 0; w < 4; ++w) {
      const float s = s_best[w][tid];
      const int i = s_id[w][tid];
      if (s > b || (s == b && s > -INFINITY && i < id)) {
        b = s;
        id = i;
      }
    }
    if (!(b > -INFINITY)) id = 0;  // nothing won (all similarities -inf or NaN)
    if (out_centroid) out_centroid[q0 + tid] = id;
    out_expert[q0 + tid] = cmap ? cmap[id] : id;
    if (out_best) {
      // divide by |q| so the reported value is the cosine
      float ss = 0.f;
      for (int ch = 0; ch < nch; ++ch) {
        const uint4 qv = sq[tid * nch + ch];
        const uint32_t qw[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          ss = fmaf(bf16_lo(qw[e]), bf16_lo(qw[e]), ss);
          ss = fmaf(bf16_hi(qw[e]), bf16_hi(qw[e]), ss);
        }
      }
      out_best[q0 + tid] = b * rsqrtf(ss);
    }
  }
}

// Finishing pass of the tensor-core router: unpack the per-query (similarity, index) key that
// the GEMM epilogues merged with 64-bit atomicMax, apply the centroid->expert map, and turn
// the winning value into a cosine by dividing by |q|.  One warp per query.
__device__ __forceinline__ float key_to_float(uint32_t u) {
  u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
  return __uint_as_float(u);
}
__global__ void __launch_bounds__(256)
route_finish_kernel(const unsigned long long* __restrict__ keys, const __nv_bfloat16* __restrict__ q,
                    const int* __restrict__ cmap, int Q, int D, int* __restrict__ out_expert,
                    int* __restrict__ out_centroid, float* __restrict__ out_best) {
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (i >= Q) return;
  const unsigned long long key = keys[i];
  int id = (key == 0ull) ? 0 : (int)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
  if (lane == 0) {
    if (out_centroid) out_centroid[i] = id;
    out_expert[i] = cmap ? cmap[id] : id;
  }
  if (out_best) {
    float ss = 0.f;
    for (int ch = lane; ch < D / 8; ch += 32) {
      const uint4 v = ldg_cached(q + (size_t)i * D + ch * 8);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        ss = fmaf(bf16_lo(w[e]), bf16_lo(w[e]), ss);
        ss = fmaf(bf16_hi(w[e]), bf16_hi(w[e]), ss);
      }
    }
    ss = warp_sum(ss);
    if (lane == 0) out_best[i] = (key == 0ull) ? -INFINITY : key_to_float((uint32_t)(key >> 32)) * rsqrtf(ss);
  }
}

cudaError_t launch_inv_norm(const __nv_bfloat16* c, int K, int D, float* inv_norm, cudaStream_t stream) {
  centroid_inv_norm_kernel<<<(K + 7) / 8, 256, 0, stream>>>(c, K, D, inv_norm);
  return cudaGetLastError();
}

cudaError_t launch_route_simple(const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                                const int* cmap, int Q, int K, int D, int* out_expert, int* out_centroid,
                                float* out_best, cudaStream_t stream) {
  const size_t smem = (size_t)kRouteQB * D * 2;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(route_simple_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * 8192 * 2);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  route_simple_kernel<<<(Q + kRouteQB - 1) / kRouteQB, 128, smem, stream>>>(q, c, inv_norm, cmap, Q, K, D, out_expert,
                                                                            out_centroid, out_best);
  return cudaGetLastError();
}

cudaError_t launch_route_finish(const unsigned long long* keys, const __nv_bfloat16* q, const int* cmap, int Q, int D,
                                int* out_expert, int* out_centroid, float* out_best, cudaStream_t stream) {
  route_finish_kernel<<<(Q + 7) / 8, 256, 0, stream>>>(keys, q, cmap, Q, D, out_expert, out_centroid, out_best);
  return cudaGetLastError();
}

}  // namespace moin
