// Query router kernels: centroid inverse norms, the CUDA-core cosine-argmax kernel used for
// small problems and odd shapes, and the finishing pass shared with the tensor-core router.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

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

// ----------------------------------------------------------------------------------------
// Small-batch router (decode-sized Q): one launch, no scratch memory.
//
// A cluster of kRcCluster CTAs serves kRcQ queries.  The centroids are cut into 16-row tiles,
// dealt round-robin to the cluster's warps (two warps share a tile, half of the k range each);
// a warp holds its tile's rows as the A operand of
// m16n8k16 (loaded straight from global memory, 16 bytes per lane: lane t of a row group takes
// k-elements 8t..8t+7 of every 32, and the queries, staged once in shared memory, are read with the
// same k assignment, so the contraction is unchanged) and the kRcQ queries as kRcQ/8 B operands.
// Every CTA merges its warps' per-query winners in its own shared memory with a 64-bit max on the
// (similarity, index) key; after a cluster barrier CTA 0 reads the other CTAs' keys through
// distributed shared memory and writes the result.
// ----------------------------------------------------------------------------------------
constexpr int kRcCluster = 8, kRcTileWarps = 4, kRcKSplit = 2, kRcWarps = kRcTileWarps * kRcKSplit, kRcQ = 32,
              kRcUnroll = 12;

__device__ __forceinline__ unsigned long long route_key(float sim, int k) {
  uint32_t u = __float_as_uint(sim);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)k);
}

// Warp w works on centroid tile (w % kRcTileWarps) of the CTA's current round and on the
// (w / kRcTileWarps)-th part of the k range; the parts are added in shared memory in a fixed order.
__global__ void __cluster_dims__(kRcCluster, 1, 1) __launch_bounds__(kRcWarps * 32)
route_cluster_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ c,
                     const float* __restrict__ inv_norm, const int* __restrict__ cmap, int Q, int K, int D,
                     int* __restrict__ out_expert, int* __restrict__ out_centroid, float* __restrict__ out_best) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ unsigned long long s_keys[kRcQ];
  __shared__ float s_part[kRcTileWarps][kRcQ / 8][4][32];
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int tw = warp % kRcTileWarps, kpart = warp / kRcTileWarps;
  const int rank = (int)cluster.block_rank();
  const int q0 = (blockIdx.x / kRcCluster) * kRcQ;
  const int pitch = D * 2 + 16;  // bytes; the 16-byte skew keeps the 8 rows of a fragment on distinct banks
  const int nch = D / 8;
  const int n_tiles = (K + 15) / 16, steps = D / 32;
  const int steps_part = (steps + kRcKSplit - 1) / kRcKSplit;
  const int s_lo = kpart * steps_part, s_hi = min(steps, s_lo + steps_part);

  // the first batch of centroid rows is requested before the queries are staged: one round trip for both
  int tile = rank * kRcTileWarps + tw;
  uint4 a0[kRcUnroll], a1[kRcUnroll];
  auto load_a = [&](int tl, int s0) {
    const int r0 = tl * 16 + g, r1 = r0 + 8;
    // rows past K read row K-1 (in bounds) and are masked at the end
    const __nv_bfloat16* a0p = c + (size_t)min(r0, K - 1) * D + t * 8;
    const __nv_bfloat16* a1p = c + (size_t)min(r1, K - 1) * D + t * 8;
#pragma unroll
    for (int u = 0; u < kRcUnroll; ++u) {
      const bool on = tl < n_tiles && s0 + u < s_hi;
      a0[u] = on ? ldg_cached(a0p + (s0 + u) * 32) : make_uint4(0, 0, 0, 0);
      a1[u] = on ? ldg_cached(a1p + (s0 + u) * 32) : make_uint4(0, 0, 0, 0);
    }
  };
  load_a(tile, s_lo);
  for (int i0 = 0; i0 < kRcQ * nch; i0 += kRcWarps * 32 * 8) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kRcWarps * 32 + tid;
      const int qi = i / nch, ch = i - qi * nch;
      v[u] = (i < kRcQ * nch && q0 + qi < Q) ? ldg_cached(q + (size_t)(q0 + qi) * D + ch * 8) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kRcWarps * 32 + tid;
      const int qi = i / nch, ch = i - qi * nch;
      if (i < kRcQ * nch) *reinterpret_cast<uint4*>(smem_raw + (size_t)qi * pitch + ch * 16) = v[u];
    }
  }
  if (tid < kRcQ) s_keys[tid] = 0ull;
  __syncthreads();

  for (bool first = true; tile - tw < n_tiles; tile += kRcCluster * kRcTileWarps, first = false) {   // CTA-uniform trip count
    float acc[kRcQ / 8][4];
#pragma unroll
    for (int j = 0; j < kRcQ / 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
    for (int s0 = s_lo; s0 < s_hi; s0 += kRcUnroll) {
      if (!first || s0 > s_lo) load_a(tile, s0);
#pragma unroll
      for (int u = 0; u < kRcUnroll; ++u) {
        if (s0 + u >= s_hi) break;
#pragma unroll
        for (int j = 0; j < kRcQ / 8; ++j) {
          const uint4 b = *reinterpret_cast<const uint4*>(smem_raw + (size_t)(j * 8 + g) * pitch + (s0 + u) * 64 + t * 16);
          mma_bf16_16816(acc[j], a0[u].x, a1[u].x, a0[u].y, a1[u].y, b.x, b.y);
          mma_bf16_16816(acc[j], a0[u].z, a1[u].z, a0[u].w, a1[u].w, b.z, b.w);
        }
      }
    }
    // add the k parts: part 1.. hand their sums to part 0 through shared memory
    if (kpart > 0) {
#pragma unroll
      for (int j = 0; j < kRcQ / 8; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) s_part[tw][j][e][lane] = acc[j][e];
    }
    __syncthreads();
    if (kpart == 0 && tile < n_tiles) {
#pragma unroll
      for (int j = 0; j < kRcQ / 8; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][e] += s_part[tw][j][e][lane];
      // acc[j][0..1]: centroid r0, queries j*8 + 2t, 2t+1;  acc[j][2..3]: centroid r1
      const int r0 = tile * 16 + g, r1 = r0 + 8;
      const float inv0 = (r0 < K) ? inv_norm[r0] : 0.f, inv1 = (r1 < K) ? inv_norm[r1] : 0.f;
#pragma unroll
      for (int j = 0; j < kRcQ / 8; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float sim0 = acc[j][e] * inv0, sim1 = acc[j][2 + e] * inv1;
          unsigned long long key = 0ull;   // 0 = no candidate (zero-norm or padding row, NaN or -inf similarity)
          if (inv0 > 0.f && sim0 > -INFINITY) key = route_key(sim0, r0);
          if (inv1 > 0.f && sim1 > -INFINITY) {
            const unsigned long long k1 = route_key(sim1, r1);
            key = k1 > key ? k1 : key;
          }
#pragma unroll
          for (int o = 4; o < 32; o <<= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
            key = other > key ? other : key;
          }
          if (g == 0 && key != 0ull) atomicMax(&s_keys[j * 8 + 2 * t + e], key);
        }
    }
    __syncthreads();   // s_part is free again
  }
  cluster.sync();
  if (rank == 0) {
    // one warp per query: lanes 0..kRcCluster-1 fetch the CTAs' keys, all lanes share the norm
    for (int qi = warp; qi < kRcQ; qi += kRcWarps) {
      if (q0 + qi >= Q) break;
      unsigned long long key = 0ull;
      if (lane < kRcCluster) key = *cluster.map_shared_rank(&s_keys[qi], lane);
#pragma unroll
      for (int o = 1; o < kRcCluster; o <<= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
      }
      key = __shfl_sync(0xffffffffu, key, 0);
      const int id = (key == 0ull) ? 0 : (int)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
      if (lane == 0) {
        if (out_centroid) out_centroid[q0 + qi] = id;
        out_expert[q0 + qi] = cmap ? cmap[id] : id;
      }
      if (out_best) {
        float ss = 0.f;
        for (int ch = lane; ch < nch; ch += 32) {
          const uint4 v = *reinterpret_cast<const uint4*>(smem_raw + (size_t)qi * pitch + ch * 16);
          const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            ss = fmaf(bf16_lo(w[e]), bf16_lo(w[e]), ss);
            ss = fmaf(bf16_hi(w[e]), bf16_hi(w[e]), ss);
          }
        }
        ss = warp_sum(ss);
        if (lane == 0)
          out_best[q0 + qi] = (key == 0ull) ? -INFINITY : key_to_float((uint32_t)(key >> 32)) * rsqrtf(ss);
      }
    }
  }
  cluster.sync();  // the other CTAs' shared memory stays alive until CTA 0 has read it
}

bool route_cluster_supported(int Q, int K, int D) {
  // few queries and at most two rounds of centroid tiles per cluster: beyond that the tensor-core GEMM wins
  return Q >= 1 && Q <= 1024 && K >= 1 && K <= 16 * 2 * kRcCluster * kRcTileWarps && (D % 32) == 0 &&
         (size_t)kRcQ * (D * 2 + 16) <= 200 * 1024;
}

cudaError_t launch_route_cluster(const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                                 const int* cmap, int Q, int K, int D, int* out_expert, int* out_centroid,
                                 float* out_best, cudaStream_t stream) {
  const size_t smem = (size_t)kRcQ * (D * 2 + 16);
  cudaError_t ce = ensure_smem_optin(OPTIN_ROUTE_CLUSTER, route_cluster_kernel, smem);
  if (ce != cudaSuccess) return ce;
  const int groups = (Q + kRcQ - 1) / kRcQ;
  route_cluster_kernel<<<groups * kRcCluster, kRcWarps * 32, smem, stream>>>(q, c, inv_norm, cmap, Q, K, D, out_expert,
                                                                            out_centroid, out_best);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------
// K-means update: centroid of every non-empty cluster = mean of its member rows.  One CTA per segment of
// the plan built from the assignments (segment = cluster id, start, length in `perm`, members in
// increasing point order); thread c owns the 8 columns 8c..8c+7 and adds the member rows in order
// (fp32), four rows' loads in flight at a time; the member indices are staged in shared memory 128 at a
// time.  HBM-bound: every point is read once.
// ----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
kmeans_mean_kernel(const int* __restrict__ header, const int* __restrict__ perm, const int4* __restrict__ seg_tab,
                   const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ c_new, int D) {
  __shared__ int s_rows[128];
  const int nseg = header[PH_NSEG];
  const int tid = threadIdx.x, nch = D / 8;
  for (int seg = blockIdx.x; seg < nseg; seg += gridDim.x) {
    const int4 e = __ldg(seg_tab + seg);   // (cluster, start, length, -)
    const int k = e.x, start = e.y, len = e.z;
    for (int c0 = 0; c0 < nch; c0 += 128) {
      const int ch = c0 + tid;
      const bool on = ch < nch;
      float acc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = 0.f;
      for (int j0 = 0; j0 < len; j0 += 128) {
        __syncthreads();
        if (j0 + tid < len) s_rows[tid] = perm[start + j0 + tid];
        __syncthreads();
        const int nb = min(128, len - j0);
        for (int j = 0; j < nb; j += 4) {
          uint4 v[4];
#pragma unroll
          for (int u = 0; u < 4; ++u)
            v[u] = (on && j + u < nb) ? ldg_stream(x + (size_t)s_rows[j + u] * D + ch * 8) : make_uint4(0, 0, 0, 0);
#pragma unroll
          for (int u = 0; u < 4; ++u) {   // rows added in member order; absent rows add zero
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              acc[2 * q] += bf16_lo(w[q]);
              acc[2 * q + 1] += bf16_hi(w[q]);
            }
          }
        }
      }
      if (on) {
        const float n = (float)len;
        uint4 o;
        o.x = pack_bf16(acc[0] / n, acc[1] / n);
        o.y = pack_bf16(acc[2] / n, acc[3] / n);
        o.z = pack_bf16(acc[4] / n, acc[5] / n);
        o.w = pack_bf16(acc[6] / n, acc[7] / n);
        *reinterpret_cast<uint4*>(c_new + (size_t)k * D + ch * 8) = o;
      }
    }
  }
}

cudaError_t launch_kmeans_mean(const PlanView& pv, const __nv_bfloat16* x, __nv_bfloat16* c_new, int D, int n_sms,
                               cudaStream_t stream) {
  long grid = pv.Smax < (long)n_sms * 16 ? pv.Smax : (long)n_sms * 16;
  if (grid < 1) grid = 1;
  kmeans_mean_kernel<<<(int)grid, 128, 0, stream>>>(pv.header, pv.perm, pv.seg_tab, x, c_new, D);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------
// Best and runner-up (top-2) router on the CUDA cores: one warp per query, lanes stride over the
// embedding, centroids in increasing order (strict '>' keeps the lowest index among equals for both
// places).  Small problems and odd shapes; the tensor-core path covers the rest.
// ----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
route_top2_simple_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ c,
                         const float* __restrict__ inv_norm, const int* __restrict__ cmap, int Q, int K, int D,
                         int* __restrict__ out_expert, int* __restrict__ out_centroid, int* __restrict__ out_second,
                         float* __restrict__ out_best, float* __restrict__ out_margin) {
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (i >= Q) return;
  const int nch = D / 8;
  float best = -INFINITY, second = -INFINITY, qq = 0.f;
  int best_k = 0, second_k = -1;
  for (int k = 0; k < K; ++k) {
    float acc = 0.f;
    for (int ch = lane; ch < nch; ch += 32) {
      const uint4 qv = ldg_cached(q + (size_t)i * D + ch * 8), cv = ldg_cached(c + (size_t)k * D + ch * 8);
      const uint32_t qw[4] = {qv.x, qv.y, qv.z, qv.w}, cw[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        acc = fmaf(bf16_lo(qw[e]), bf16_lo(cw[e]), acc);
        acc = fmaf(bf16_hi(qw[e]), bf16_hi(cw[e]), acc);
        if (k == 0) {
          qq = fmaf(bf16_lo(qw[e]), bf16_lo(qw[e]), qq);
          qq = fmaf(bf16_hi(qw[e]), bf16_hi(qw[e]), qq);
        }
      }
    }
    acc = warp_sum(acc);
    const float inv = inv_norm[k];
    const float sim = acc * inv;
    if (inv > 0.f && sim > best) {
      second = best; second_k = (best > -INFINITY) ? best_k : -1;
      best = sim; best_k = k;
    } else if (inv > 0.f && sim > second) {
      second = sim; second_k = k;
    }
  }
  qq = warp_sum(qq);
  if (lane == 0) {
    const float rq = rsqrtf(qq);
    const int id = (best > -INFINITY) ? best_k : 0;
    if (out_centroid) out_centroid[i] = id;
    if (out_expert) out_expert[i] = cmap ? cmap[id] : id;
    if (out_second) out_second[i] = (second > -INFINITY) ? second_k : -1;
    if (out_best) out_best[i] = (best > -INFINITY) ? best * rq : -INFINITY;
    if (out_margin) out_margin[i] = (second > -INFINITY) ? (best - second) * rq : INFINITY;
  }
}

// Finishing pass of the tensor-core top-2 router: unpack both keys, divide by |q|.  One warp per query.
__global__ void __launch_bounds__(256)
route_finish_top2_kernel(const unsigned long long* __restrict__ keys, const unsigned long long* __restrict__ keys2,
                         const __nv_bfloat16* __restrict__ q, const int* __restrict__ cmap, int Q, int D,
                         int* __restrict__ out_expert, int* __restrict__ out_centroid, int* __restrict__ out_second,
                         float* __restrict__ out_best, float* __restrict__ out_margin) {
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (i >= Q) return;
  const unsigned long long k1 = keys[i], k2 = keys2[i];
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
  if (lane == 0) {
    const float rq = rsqrtf(ss);
    const int id = (k1 == 0ull) ? 0 : (int)(0xFFFFFFFFu - (uint32_t)(k1 & 0xFFFFFFFFull));
    const float s1 = key_to_float((uint32_t)(k1 >> 32)), s2 = key_to_float((uint32_t)(k2 >> 32));
    if (out_centroid) out_centroid[i] = id;
    if (out_expert) out_expert[i] = cmap ? cmap[id] : id;
    if (out_second) out_second[i] = (k2 == 0ull) ? -1 : (int)(0xFFFFFFFFu - (uint32_t)(k2 & 0xFFFFFFFFull));
    if (out_best) out_best[i] = (k1 == 0ull) ? -INFINITY : s1 * rq;
    if (out_margin) out_margin[i] = (k1 == 0ull || k2 == 0ull) ? INFINITY : (s1 - s2) * rq;
  }
}

cudaError_t launch_route_top2_simple(const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                                     const int* cmap, int Q, int K, int D, int* out_expert, int* out_centroid,
                                     int* out_second, float* out_best, float* out_margin, cudaStream_t stream) {
  route_top2_simple_kernel<<<(Q + 7) / 8, 256, 0, stream>>>(q, c, inv_norm, cmap, Q, K, D, out_expert, out_centroid,
                                                           out_second, out_best, out_margin);
  return cudaGetLastError();
}
cudaError_t launch_route_finish_top2(const unsigned long long* keys, const unsigned long long* keys2,
                                     const __nv_bfloat16* q, const int* cmap, int Q, int D, int* out_expert,
                                     int* out_centroid, int* out_second, float* out_best, float* out_margin,
                                     cudaStream_t stream) {
  route_finish_top2_kernel<<<(Q + 7) / 8, 256, 0, stream>>>(keys, keys2, q, cmap, Q, D, out_expert, out_centroid, out_second,
                                                           out_best, out_margin);
  return cudaGetLastError();
}

cudaError_t launch_inv_norm(const __nv_bfloat16* c, int K, int D, float* inv_norm, cudaStream_t stream) {
  centroid_inv_norm_kernel<<<(K + 7) / 8, 256, 0, stream>>>(c, K, D, inv_norm);
  return cudaGetLastError();
}

cudaError_t launch_route_simple(const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                                const int* cmap, int Q, int K, int D, int* out_expert, int* out_centroid,
                                float* out_best, cudaStream_t stream) {
  const size_t smem = (size_t)kRouteQB * D * 2;
  cudaError_t ce = ensure_smem_optin(OPTIN_ROUTE_SIMPLE, route_simple_kernel, 8 * 8192 * 2);
  if (ce != cudaSuccess) return ce;
  route_simple_kernel<<<(Q + kRouteQB - 1) / kRouteQB, 128, smem, stream>>>(q, c, inv_norm, cmap, Q, K, D, out_expert,
                                                                            out_centroid, out_best);
  return cudaGetLastError();
}

// The same without the cosine output: nothing to reduce, so one thread per query (coalesced keys and ids).
__global__ void __launch_bounds__(256)
route_finish_ids_kernel(const unsigned long long* __restrict__ keys, const int* __restrict__ cmap, int Q,
                        int* __restrict__ out_expert, int* __restrict__ out_centroid) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= Q) return;
  const unsigned long long key = keys[i];
  const int id = (key == 0ull) ? 0 : (int)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
  if (out_centroid) out_centroid[i] = id;
  out_expert[i] = cmap ? cmap[id] : id;
}

cudaError_t launch_route_finish(const unsigned long long* keys, const __nv_bfloat16* q, const int* cmap, int Q, int D,
                                int* out_expert, int* out_centroid, float* out_best, cudaStream_t stream) {
  if (out_best == nullptr)
    route_finish_ids_kernel<<<(Q + 255) / 256, 256, 0, stream>>>(keys, cmap, Q, out_expert, out_centroid);
  else
    route_finish_kernel<<<(Q + 7) / 8, 256, 0, stream>>>(keys, q, cmap, Q, D, out_expert, out_centroid, out_best);
  return cudaGetLastError();
}

}  // namespace moin
