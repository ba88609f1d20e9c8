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

constexpr int kShrinkThreads = 256;      // 8 warps split the reduction dimension
constexpr int kShrinkWarps = kShrinkThreads / 32;
constexpr int kShrinkUnroll = 8;         // 32-wide k steps in flight per warp
constexpr int kExpandThreads = 128;      // 4 warps
constexpr int kExpandTilesPerBatch = 2;  // 16-row tiles whose loads are in flight together, per warp

struct SegMeta { int slot, s0, n; };
__device__ __forceinline__ SegMeta load_seg(const int* __restrict__ seg_expert, const int* __restrict__ seg_start,
                                            const int* __restrict__ slot_of_expert, int seg, bool valid) {
  SegMeta m = {-1, 0, 0};
  if (valid) {
    m.slot = slot_of_expert[seg_expert[seg]];
    m.s0 = seg_start[seg];
    m.n = seg_start[seg + 1] - m.s0;
  }
  return m;
}

// h[pos][rho] = sum_i A[slot][rho][i] * x[perm[pos]][i]      (fp32, pos = position in sorted order)
// Work item = (segment, group of 16 adapter rows); the CTA's 8 warps interleave over k.
__global__ void __launch_bounds__(kShrinkThreads, 2)
lora_shrink_stream_kernel(const int* __restrict__ header, const int* __restrict__ perm,
                          const int* __restrict__ seg_expert, const int* __restrict__ seg_start,
                          const int* __restrict__ slot_of_expert, const __nv_bfloat16* __restrict__ x,
                          const __nv_bfloat16* __restrict__ A, float* __restrict__ h, int r, int d_in) {
  __shared__ float red[kShrinkWarps][32][4];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int nseg = header[PH_NSEG];
  const int MG = (r + 15) >> 4;
  const int steps = d_in >> 5;  // 32 k per step
  const int items = nseg * MG;
  int item = blockIdx.x;
  SegMeta nxt = load_seg(seg_expert, seg_start, slot_of_expert, item / MG, item < items);
  for (; item < items; item += gridDim.x) {
    const SegMeta cur = nxt;
    const int mg = item % MG;
    const int ni = item + gridDim.x;
    nxt = load_seg(seg_expert, seg_start, slot_of_expert, ni / MG, ni < items);  // one item of lookahead
    if (cur.slot < 0) continue;  // uniform per CTA
    const int rho0 = mg * 16 + g, rho1 = rho0 + 8;
    const bool v0 = rho0 < r, v1 = rho1 < r;
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
// Work item = (segment, block of rows_per_item output features); each warp walks its 16-row tiles
// kExpandTilesPerBatch at a time with the adapter rows and the base values y0 loaded together.
template <int P>  // number of 32-wide rho groups: ceil(r / 32)
__global__ void __launch_bounds__(kExpandThreads, 4)
lora_expand_stream_kernel(const int* __restrict__ header, const int* __restrict__ perm,
                          const int* __restrict__ seg_expert, const int* __restrict__ seg_start,
                          const int* __restrict__ slot_of_expert, const float* __restrict__ h,
                          const __nv_bfloat16* __restrict__ B, const float* __restrict__ y0,
                          __nv_bfloat16* __restrict__ y, float scale, int r, int d_out, int rows_per_item) {
  constexpr int TB = kExpandTilesPerBatch;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int nseg = header[PH_NSEG];
  const int JB = (d_out + rows_per_item - 1) / rows_per_item;
  const int tiles_per_item = rows_per_item >> 4;
  const int items = nseg * JB;
  int item = blockIdx.x;
  SegMeta nxt = load_seg(seg_expert, seg_start, slot_of_expert, item / JB, item < items);
  for (; item < items; item += gridDim.x) {
    const SegMeta cur = nxt;
    const int jb = item % JB;
    const int ni = item + gridDim.x;
    nxt = load_seg(seg_expert, seg_start, slot_of_expert, ni / JB, ni < items);
    if (cur.slot < 0) continue;
    const __nv_bfloat16* Bs = B + (size_t)cur.slot * (size_t)d_out * (size_t)r;
    for (int tc = 0; tc < cur.n; tc += 8) {
      // token operand (MMA "B" fragment): column g = token tc+g, k slots <- rho 32p + 8t .. +7
      const bool vx = (tc + g) < cur.n;
      const int my_row = vx ? perm[cur.s0 + tc + g] : -1;
      uint32_t hh[P][4], hl[P][4];
#pragma unroll
      for (int p = 0; p < P; ++p) {
        const int rb = 32 * p + 8 * t;
        float v[8];
        if (vx && rb < r) {
          const float4 f0 = *reinterpret_cast<const float4*>(h + (size_t)(cur.s0 + tc + g) * r + rb);
          const float4 f1 = *reinterpret_cast<const float4*>(h + (size_t)(cur.s0 + tc + g) * r + rb + 4);
          v[0] = f0.x; v[1] = f0.y; v[2] = f0.z; v[3] = f0.w; v[4] = f1.x; v[5] = f1.y; v[6] = f1.z; v[7] = f1.w;
        } else {
#pragma unroll
          for (int q = 0; q < 8; ++q) v[q] = 0.f;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float s0v = v[2 * q] * scale, s1v = v[2 * q + 1] * scale;
          const uint32_t hi = pack_bf16(s0v, s1v);
          hh[p][q] = hi;
          hl[p][q] = pack_bf16(s0v - bf16_lo(hi), s1v - bf16_hi(hi));
        }
      }
      const int row_c0 = __shfl_sync(0xffffffffu, my_row, (2 * t) * 4);
      const int row_c1 = __shfl_sync(0xffffffffu, my_row, (2 * t + 1) * 4);
      for (int tb = warp * TB; tb < tiles_per_item; tb += 4 * TB) {
        uint4 a0[TB][P], a1[TB][P];
        float b0[TB][4];
#pragma unroll
        for (int i = 0; i < TB; ++i) {
          const int j0 = jb * rows_per_item + (tb + i) * 16;
          const int ja = j0 + g, jc = j0 + g + 8;
          const bool va = (tb + i) < tiles_per_item && ja < d_out, vc = (tb + i) < tiles_per_item && jc < d_out;
#pragma unroll
          for (int p = 0; p < P; ++p) {
            const int rb = 32 * p + 8 * t;
            const uint4 z = make_uint4(0, 0, 0, 0);
            a0[i][p] = (va && rb < r) ? ldg_stream(Bs + (size_t)ja * r + rb) : z;
            a1[i][p] = (vc && rb < r) ? ldg_stream(Bs + (size_t)jc * r + rb) : z;
          }
          b0[i][0] = (va && row_c0 >= 0) ? __ldg(y0 + (size_t)row_c0 * d_out + ja) : 0.f;
          b0[i][1] = (va && row_c1 >= 0) ? __ldg(y0 + (size_t)row_c1 * d_out + ja) : 0.f;
          b0[i][2] = (vc && row_c0 >= 0) ? __ldg(y0 + (size_t)row_c0 * d_out + jc) : 0.f;
          b0[i][3] = (vc && row_c1 >= 0) ? __ldg(y0 + (size_t)row_c1 * d_out + jc) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < TB; ++i) {
          const int j0 = jb * rows_per_item + (tb + i) * 16;
          const int ja = j0 + g, jc = j0 + g + 8;
          const bool va = (tb + i) < tiles_per_item && ja < d_out, vc = (tb + i) < tiles_per_item && jc < d_out;
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
}

static int stream_grid(long max_items, int n_sms, int ctas_per_sm) {
  long g = max_items < (long)n_sms * ctas_per_sm ? max_items : (long)n_sms * ctas_per_sm;
  return g < 1 ? 1 : (int)g;
}

cudaError_t launch_lora_shrink_stream(const PlanView& pv, const int* slot_of_expert, const __nv_bfloat16* x,
                                      const __nv_bfloat16* A, float* h, int r, int d_in, int n_sms,
                                      cudaStream_t stream) {
  const int MG = (r + 15) / 16;
  lora_shrink_stream_kernel<<<stream_grid((long)pv.Smax * MG, n_sms, 8), kShrinkThreads, 0, stream>>>(
      pv.header, pv.perm, pv.seg_expert, pv.seg_start, slot_of_expert, x, A, h, r, d_in);
  return cudaGetLastError();
}

cudaError_t launch_lora_expand_stream(const PlanView& pv, const int* slot_of_expert, const float* h,
                                      const __nv_bfloat16* B, const float* y0, __nv_bfloat16* y, float scale, int r,
                                      int d_out, int n_sms, cudaStream_t stream) {
  const int rows_per_item = d_out <= 512 ? 128 : 512;
  const int JB = (d_out + rows_per_item - 1) / rows_per_item;
  const int grid = stream_grid((long)pv.Smax * JB, n_sms, 16);
  if (r <= 32)
    lora_expand_stream_kernel<1><<<grid, kExpandThreads, 0, stream>>>(pv.header, pv.perm, pv.seg_expert, pv.seg_start,
                                                                      slot_of_expert, h, B, y0, y, scale, r, d_out,
                                                                      rows_per_item);
  else
    lora_expand_stream_kernel<2><<<grid, kExpandThreads, 0, stream>>>(pv.header, pv.perm, pv.seg_expert, pv.seg_start,
                                                                      slot_of_expert, h, B, y0, y, scale, r, d_out,
                                                                      rows_per_item);
  return cudaGetLastError();
}

}  // namespace moin
