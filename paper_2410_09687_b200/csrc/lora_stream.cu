// Segmented LoRA shrink / expand for short segments (decode): every distinct adapter is
// streamed from HBM exactly once per call, straight from global memory into warp-MMA
// fragments.
//
// Both products are skinny (8 token columns per MMA), so they are HBM-bound on the adapter
// bytes; the tensor-core instruction used is the warp-level m16n8k16 one, which does the
// reduction over the long dimension without shuffles.  Operand fragments are loaded with one
// 16-byte load per thread and row: the MMA's k index is only a summation index, so the
// 8 consecutive elements a thread loads are assigned to the k slots it owns in two
// consecutive MMAs - as long as the other operand uses the same assignment the dot product
// is unchanged.  A warp-wide load then covers 8 rows x 64 contiguous bytes (full sectors).
#include "common.cuh"

namespace moin {

constexpr int kShrinkThreads = 128;      // 4 warps split the reduction dimension
constexpr int kShrinkWarps = kShrinkThreads / 32;
constexpr int kShrinkUnroll = 4;         // 32-wide k steps in flight per warp
constexpr int kExpandThreads = 128;      // 4 warps
constexpr int kExpandTilesPerBatch = 2;  // 16-row tiles whose loads are in flight together, per warp

// Work items of a launch span up to kMaxStreamJobs projections that share one batch plan: item index ->
// (job, segment, sub-block), jobs laid out one after the other, `per_seg[j]` items per segment in job j.
// Kernel parameters are only ever indexed with compile-time indices (a run-time index would force a
// local-memory copy of the parameter block): pick(arr, j) selects arr[j] with a compare chain.
template <class V>
__device__ __forceinline__ V pick(const V (&arr)[kMaxStreamJobs], int j) {
  V v = arr[0];
#pragma unroll
  for (int i = 1; i < kMaxStreamJobs; ++i)
    if (j == i) v = arr[i];
  return v;
}

struct ItemRef { int job, seg, sub; };
template <class Jobs>
__device__ __forceinline__ ItemRef decode_item(int item, int nseg, const Jobs& jobs) {
  ItemRef it = {0, 0, 0};
  int rem = item;
#pragma unroll
  for (int j = 0; j + 1 < kMaxStreamJobs; ++j) {
    if (it.job == j && j + 1 < jobs.n && rem >= nseg * jobs.per_seg[j]) {
      rem -= nseg * jobs.per_seg[j];
      it.job = j + 1;
    }
  }
  const int ps = pick(jobs.per_seg, it.job);
  it.seg = rem / ps;
  it.sub = rem - it.seg * ps;
  return it;
}

struct SegMeta { int slot, s0, n, job, sub, r_use; };   // r_use: rank of the slot's adapter (<= the stored rank)
template <class Jobs>
__device__ __forceinline__ SegMeta load_seg(const int4* __restrict__ seg_tab, const Jobs& jobs, int item, int items,
                                            int nseg) {
  SegMeta m = {-1, 0, 0, 0, 0, 0};
  if (item < items) {
    const ItemRef it = decode_item(item, nseg, jobs);
    const int4 e = __ldg(seg_tab + it.seg);   // (expert, start, length, -)
    m.slot = __ldg(pick(jobs.slot_of_expert, it.job) + e.x);
    const int* rank_tab = pick(jobs.slot_rank, it.job);
    m.r_use = (m.slot >= 0 && rank_tab) ? min(__ldg(rank_tab + m.slot), pick(jobs.r, it.job)) : pick(jobs.r, it.job);
    m.s0 = e.y;
    m.n = e.z;
    m.job = it.job;
    m.sub = it.sub;
  }
  return m;
}

// h[pos][rho] = sum_i A[slot][rho][i] * x[perm[pos]][i]      (fp32, pos = position in sorted order)
// Work item = (job, segment, group of 16 adapter rows); the CTA's warps interleave over k.
// Small CTAs (4 warps, 80 registers: six per SM, and room beside a base-GEMM CTA) and one CTA per item:
// the hardware's block scheduler hands the items out as slots free up, so a launch ends evenly whatever
// the base GEMMs on the side streams occupy, and a CTA's metadata hops (segment count, table entry,
// slot) hide behind the streams of the other CTAs on its SM.
__global__ void __launch_bounds__(kShrinkThreads, 6)
lora_shrink_stream_kernel(const int* __restrict__ header, const int* __restrict__ perm,
                          const int4* __restrict__ seg_tab, const ShrinkJobs jobs) {
  __shared__ float red[kShrinkWarps][32][4];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int nseg = header[PH_NSEG];
  int items = 0;
#pragma unroll
  for (int j = 0; j < kMaxStreamJobs; ++j)
    if (j < jobs.n) items += nseg * jobs.per_seg[j];
  int item = blockIdx.x;
  SegMeta nxt = load_seg(seg_tab, jobs, item, items, nseg);
  for (; item < items; item += gridDim.x) {
    const SegMeta cur = nxt;
    nxt = load_seg(seg_tab, jobs, item + gridDim.x, items, nseg);  // lookahead
    if (cur.slot < 0 || cur.sub * 16 >= cur.r_use) continue;  // uniform per CTA: no adapter, or rows beyond its rank
    const int r = pick(jobs.r, cur.job), d_in = pick(jobs.d_in, cur.job);
    const __nv_bfloat16* __restrict__ x = pick(jobs.x, cur.job);
    const __nv_bfloat16* __restrict__ A = pick(jobs.A, cur.job);
    float* __restrict__ h = pick(jobs.h, cur.job);
    const int steps = d_in >> 5;  // 32 k per step
    const int rho0 = cur.sub * 16 + g, rho1 = rho0 + 8;
    const bool v0 = rho0 < cur.r_use, v1 = rho1 < cur.r_use;   // rows beyond the slot's rank are not read
    const __nv_bfloat16* a_row0 = A + ((size_t)cur.slot * r + (v0 ? rho0 : 0)) * (size_t)d_in + 8 * t;
    const __nv_bfloat16* a_row1 = A + ((size_t)cur.slot * r + (v1 ? rho1 : 0)) * (size_t)d_in + 8 * t;
    for (int tc = 0; tc < cur.n; tc += 8) {
      const bool vx = (tc + g) < cur.n;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
      const __nv_bfloat16* x_row = nullptr;
      for (int base = 0; base < steps; base += kShrinkWarps * kShrinkUnroll) {
        uint4 a0[kShrinkUnroll], a1[kShrinkUnroll], xv[kShrinkUnroll];
        const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < kShrinkUnroll; ++u) {  // adapter bytes first: they come from HBM
          const int i = base + u * kShrinkWarps + warp;
          const bool vi = i < steps;
          a0[u] = (vi && v0) ? ldg_stream(a_row0 + i * 32) : z;
          a1[u] = (vi && v1) ? ldg_stream(a_row1 + i * 32) : z;
        }
        if (x_row == nullptr) x_row = x + (size_t)(vx ? perm[cur.s0 + tc + g] : 0) * (size_t)d_in + 8 * t;
#pragma unroll
        for (int u = 0; u < kShrinkUnroll; ++u) {
          const int i = base + u * kShrinkWarps + warp;
          xv[u] = (i < steps && vx) ? ldg_cached(x_row + i * 32) : z;
        }
#pragma unroll
        for (int u = 0; u < kShrinkUnroll; ++u) {
          mma_bf16_16816(c, a0[u].x, a1[u].x, a0[u].y, a1[u].y, xv[u].x, xv[u].y);
          mma_bf16_16816(c, a0[u].z, a1[u].z, a0[u].w, a1[u].w, xv[u].z, xv[u].w);
        }
      }
      // fixed-order reduction over the warps (deterministic)
      __syncthreads();
#pragma unroll
      for (int j = 0; j < 4; ++j) red[warp][lane][j] = c[j];
      __syncthreads();
      if (warp == 0) {
        float s[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float acc = red[0][lane][j];
#pragma unroll
          for (int w = 1; w < kShrinkWarps; ++w) acc += red[w][lane][j];
          s[j] = acc;
        }
        // c0:(rho0, col 2t) c1:(rho0, col 2t+1) c2:(rho1, col 2t) c3:(rho1, col 2t+1)
        const int col = 2 * t;
        if (tc + col < cur.n) {
          float* hp = h + (size_t)(cur.s0 + tc + col) * r;
          if (v0) hp[rho0] = s[0];
          if (v1) hp[rho1] = s[2];
        }
        if (tc + col + 1 < cur.n) {
          float* hp = h + (size_t)(cur.s0 + tc + col + 1) * r;
          if (v0) hp[rho0] = s[1];
          if (v1) hp[rho1] = s[3];
        }
      }
    }
  }
}

// y[perm[pos]][j] = bf16( y0[perm[pos]][j] + scale * sum_rho B[slot][j][rho] * h[pos][rho] )
// h is split into bf16 hi + lo parts (two MMAs) so the low-rank term keeps ~fp32 accuracy.
//
// The unit of work is one 16-row tile of B for one (segment, job); units are ordered (segment, job, tile)
// and every warp of the grid takes one contiguous, equally long range of them (tiles need no reduction
// across each other, so a range may start and end anywhere).  All warps therefore stream the same number
// of adapter bytes, whatever the mix of projection widths in the launch, and a warp's range is contiguous
// in memory inside a (segment, job).  A warp walks its range kExpandTilesPerBatch tiles at a time with
// the adapter rows and the base values y0 of a batch loaded together.  `jobs.per_seg[j]` = tiles of job j.
// VAR: some pool of the launch has a rank per slot or an activation; without it the kernel is the plain layer's
// (the rank is the stored rank, h is used as it is) and carries none of the variant's bookkeeping.
template <int P, bool VAR>  // P: number of 32-wide rho groups, ceil(max r / 32)
__global__ void __launch_bounds__(kExpandThreads, 4)
lora_expand_stream_kernel(const int* __restrict__ header, const int* __restrict__ perm,
                          const int4* __restrict__ seg_tab, const ExpandJobs jobs, float scale, int tps) {
  constexpr int TB = P > 2 ? 1 : kExpandTilesPerBatch;   // wide ranks: one tile's rows already fill the load registers
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const long long wid = (long long)blockIdx.x * (kExpandThreads / 32) + warp;
  const long long nw = (long long)gridDim.x * (kExpandThreads / 32);
  const int nseg = __ldg(header + PH_NSEG);
  const long long units = (long long)nseg * tps;
  long long u = units * wid / nw;
  const long long u_end = units * (wid + 1) / nw;
  while (u < u_end) {
    // ---- segment: expert, rows, adapter slots of all jobs (one hop after the table entry)
    const int seg = (int)(u / tps);
    const int4 e = __ldg(seg_tab + seg);   // (expert, start, length, -)
    const int s0 = e.y, n = e.z;
    int slots[kMaxStreamJobs];
#pragma unroll
    for (int j = 0; j < kMaxStreamJobs; ++j) slots[j] = (j < jobs.n) ? __ldg(jobs.slot_of_expert[j] + e.x) : -1;
    int ranks[kMaxStreamJobs];   // rank of the slot's adapter: columns of B and entries of h beyond it are not read
#pragma unroll
    for (int j = 0; j < kMaxStreamJobs; ++j)
      ranks[j] = (VAR && j < jobs.n && slots[j] >= 0 && jobs.slot_rank[j]) ? min(__ldg(jobs.slot_rank[j] + slots[j]), jobs.r[j])
                                                                     : (j < jobs.n ? jobs.r[j] : 0);
    const int row_first = (g < n) ? __ldg(perm + s0 + g) : -1;
    const long long seg_end = (long long)(seg + 1) * tps;
    int rem = (int)(u - (long long)seg * tps);
    int job = 0;
#pragma unroll
    for (int j = 0; j + 1 < kMaxStreamJobs; ++j) {
      if (job == j && j + 1 < jobs.n && rem >= jobs.per_seg[j]) {
        rem -= jobs.per_seg[j];
        job = j + 1;
      }
    }
    // ---- (segment, job) pieces of the range
    while (u < u_end && u < seg_end) {
      const int tiles_j = pick(jobs.per_seg, job);
      const int tile0 = rem;
      const long long left = u_end - u;
      const int tile1 = (left < (long long)(tiles_j - tile0)) ? tile0 + (int)left : tiles_j;
      const int slot = pick(slots, job);
      if (slot >= 0) {
        const int r = pick(jobs.r, job), d_out = pick(jobs.d_out, job);
        const int r_use = VAR ? pick(ranks, job) : r, act = VAR ? pick(jobs.act, job) : MOIN_ACT_NONE;
        const float* __restrict__ h = pick(jobs.h, job);
        const float* __restrict__ y0 = pick(jobs.y0, job);
        __nv_bfloat16* __restrict__ y = pick(jobs.y, job);
        const __nv_bfloat16* Bs = pick(jobs.B, job) + (size_t)slot * (size_t)d_out * (size_t)r;
        for (int tc = 0; tc < n; tc += 8) {
          // token operand (MMA "B" fragment): column g = token tc+g, k slots <- rho 32p + 8t .. +7
          const bool vx = (tc + g) < n;
          const int my_row = (tc == 0) ? row_first : (vx ? __ldg(perm + s0 + tc + g) : -1);
          uint32_t hh[P][4], hl[P][4];
#pragma unroll
          for (int p = 0; p < P; ++p) {
            const int rb = 32 * p + 8 * t;
            float v[8];
            if (vx && rb < r_use) {
              const float4 f0 = *reinterpret_cast<const float4*>(h + (size_t)(s0 + tc + g) * r + rb);
              const float4 f1 = *reinterpret_cast<const float4*>(h + (size_t)(s0 + tc + g) * r + rb + 4);
              v[0] = f0.x; v[1] = f0.y; v[2] = f0.z; v[3] = f0.w; v[4] = f1.x; v[5] = f1.y; v[6] = f1.z; v[7] = f1.w;
            } else {
#pragma unroll
              for (int q = 0; q < 8; ++q) v[q] = 0.f;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float s0v = (VAR ? lora_act(v[2 * q], act) : v[2 * q]) * scale;
              const float s1v = (VAR ? lora_act(v[2 * q + 1], act) : v[2 * q + 1]) * scale;
              const uint32_t hi = pack_bf16(s0v, s1v);
              hh[p][q] = hi;
              hl[p][q] = pack_bf16(s0v - bf16_lo(hi), s1v - bf16_hi(hi));
            }
          }
          const int row_c0 = __shfl_sync(0xffffffffu, my_row, (2 * t) * 4);
          const int row_c1 = __shfl_sync(0xffffffffu, my_row, (2 * t + 1) * 4);
          for (int tb = tile0; tb < tile1; tb += TB) {
            uint4 a0[TB][P], a1[TB][P];
            float b0[TB][4];
#pragma unroll
            for (int i = 0; i < TB; ++i) {
              const int ja = (tb + i) * 16 + g, jc = ja + 8;
              const bool va = (tb + i) < tile1 && ja < d_out, vc = (tb + i) < tile1 && jc < d_out;
#pragma unroll
              for (int p = 0; p < P; ++p) {
                const int rb = 32 * p + 8 * t;
                const uint4 z = make_uint4(0, 0, 0, 0);
                a0[i][p] = (va && rb < r_use) ? ldg_stream(Bs + (size_t)ja * r + rb) : z;
                a1[i][p] = (vc && rb < r_use) ? ldg_stream(Bs + (size_t)jc * r + rb) : z;
              }
              b0[i][0] = (va && row_c0 >= 0) ? __ldg(y0 + (size_t)row_c0 * d_out + ja) : 0.f;
              b0[i][1] = (va && row_c1 >= 0) ? __ldg(y0 + (size_t)row_c1 * d_out + ja) : 0.f;
              b0[i][2] = (vc && row_c0 >= 0) ? __ldg(y0 + (size_t)row_c0 * d_out + jc) : 0.f;
              b0[i][3] = (vc && row_c1 >= 0) ? __ldg(y0 + (size_t)row_c1 * d_out + jc) : 0.f;
            }
#pragma unroll
            for (int i = 0; i < TB; ++i) {
              const int ja = (tb + i) * 16 + g, jc = ja + 8;
              const bool va = (tb + i) < tile1 && ja < d_out, vc = (tb + i) < tile1 && jc < d_out;
              float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int p = 0; p < P; ++p) {
                mma_bf16_16816(c, a0[i][p].x, a1[i][p].x, a0[i][p].y, a1[i][p].y, hl[p][0], hl[p][1]);
                mma_bf16_16816(c, a0[i][p].z, a1[i][p].z, a0[i][p].w, a1[i][p].w, hl[p][2], hl[p][3]);
                mma_bf16_16816(c, a0[i][p].x, a1[i][p].x, a0[i][p].y, a1[i][p].y, hh[p][0], hh[p][1]);
                mma_bf16_16816(c, a0[i][p].z, a1[i][p].z, a0[i][p].w, a1[i][p].w, hh[p][2], hh[p][3]);
              }
              // c0:(ja, col 2t) c1:(ja, col 2t+1) c2:(jc, col 2t) c3:(jc, col 2t+1)
              if (row_c0 >= 0) {
                const size_t o = (size_t)row_c0 * d_out;
                if (va) y[o + ja] = __float2bfloat16_rn(b0[i][0] + c[0]);
                if (vc) y[o + jc] = __float2bfloat16_rn(b0[i][2] + c[2]);
              }
              if (row_c1 >= 0) {
                const size_t o = (size_t)row_c1 * d_out;
                if (va) y[o + ja] = __float2bfloat16_rn(b0[i][1] + c[1]);
                if (vc) y[o + jc] = __float2bfloat16_rn(b0[i][3] + c[3]);
              }
            }
          }
        }
      }
      u += tile1 - tile0;
      rem = 0;
      ++job;
    }
  }
}

static int stream_grid(long max_items, int n_sms, int ctas_per_sm) {
  long g = max_items < (long)n_sms * ctas_per_sm ? max_items : (long)n_sms * ctas_per_sm;
  return g < 1 ? 1 : (int)g;
}

cudaError_t launch_lora_shrink_stream(const PlanView& pv, ShrinkJobs jobs, int n_sms, cudaStream_t stream) {
  long items = 0;
  for (int j = 0; j < jobs.n; ++j) {
    jobs.per_seg[j] = (jobs.r[j] + 15) / 16;
    items += (long)pv.Smax * jobs.per_seg[j];
  }
  // one CTA per item (capped; CTAs stride over the items beyond the cap)
  lora_shrink_stream_kernel<<<stream_grid(items, n_sms, 1024), kShrinkThreads, 0, stream>>>(pv.header, pv.perm, pv.seg_tab,
                                                                                       jobs);
  return cudaGetLastError();
}

cudaError_t launch_lora_expand_stream(const PlanView& pv, ExpandJobs jobs, float scale, int n_sms,
                                      cudaStream_t stream) {
  int tps = 0, rmax = 0;
  for (int j = 0; j < jobs.n; ++j) {
    jobs.rows_per_item[j] = 16;
    jobs.per_seg[j] = (jobs.d_out[j] + 15) / 16;   // 16-row tiles per segment
    tps += jobs.per_seg[j];
    rmax = jobs.r[j] > rmax ? jobs.r[j] : rmax;
  }
  // one warp per 2 tiles at least; at most one CTA per resident slot (4 per SM)
  const long max_ctas = ((long)pv.Smax * tps + 2 * (kExpandThreads / 32) - 1) / (2 * (kExpandThreads / 32));
  const int grid = stream_grid(max_ctas, n_sms, 4);
  bool var = false;
  for (int j = 0; j < jobs.n; ++j) var = var || jobs.slot_rank[j] != nullptr || jobs.act[j] != MOIN_ACT_NONE;
#define MOIN_EXPAND(P)                                                                                          \
  do {                                                                                                          \
    if (var) lora_expand_stream_kernel<P, true><<<grid, kExpandThreads, 0, stream>>>(pv.header, pv.perm, pv.seg_tab, jobs, scale, tps); \
    else lora_expand_stream_kernel<P, false><<<grid, kExpandThreads, 0, stream>>>(pv.header, pv.perm, pv.seg_tab, jobs, scale, tps);    \
  } while (0)
  if (rmax <= 32) MOIN_EXPAND(1);
  else if (rmax <= 64) MOIN_EXPAND(2);
  else MOIN_EXPAND(4);
#undef MOIN_EXPAND
  return cudaGetLastError();
}

}  // namespace moin
