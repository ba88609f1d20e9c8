// Base GEMM y = x W^T on warp-level MMA (m16n8k16 bf16 -> fp32).
//
// This is the small-shape / odd-shape path (and the cross-check for the tcgen05 kernels):
// 64 x 64 output tile per CTA, 4 warps of 32 x 32, k advanced 32 at a time through padded
// shared memory (80-byte row pitch: conflict-free 32-bit fragment reads).
#include "common.cuh"

namespace moin {

constexpr int kWBM = 64, kWBN = 64, kWBK = 32, kWPitch = 40;  // pitch in bf16 elements

// y[t][j] = bf16(acc), and y0[t][j] = acc (fp32) when y0 != nullptr.
__global__ void __launch_bounds__(128)
gemm_warp_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ W,
                 __nv_bfloat16* __restrict__ y, float* __restrict__ y0, int T, int d_in, int d_out) {
  __shared__ __align__(16) uint16_t As[kWBM * kWPitch];
  __shared__ __align__(16) uint16_t Bs[kWBN * kWPitch];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int wm = warp >> 1, wn = warp & 1;
  const int m0 = blockIdx.y * kWBM, n0 = blockIdx.x * kWBN;
  float c[2][4][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int q = 0; q < 4; ++q) c[i][j][q] = 0.f;

  for (int k0 = 0; k0 < d_in; k0 += kWBK) {
    uint4 ra[2], rb[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int id = tid + i * 128, row = id >> 2, kc = id & 3;
      const uint4 z = make_uint4(0, 0, 0, 0);
      ra[i] = (m0 + row < T) ? ldg_cached(x + (size_t)(m0 + row) * d_in + k0 + kc * 8) : z;
      rb[i] = (n0 + row < d_out) ? ldg_cached(W + (size_t)(n0 + row) * d_in + k0 + kc * 8) : z;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int id = tid + i * 128, row = id >> 2, kc = id & 3;
      *reinterpret_cast<uint4*>(&As[row * kWPitch + kc * 8]) = ra[i];
      *reinterpret_cast<uint4*>(&Bs[row * kWPitch + kc * 8]) = rb[i];
    }
    __syncthreads();
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
      uint32_t a[2][4], b[4][2];
#pragma unroll
      for (int mi = 0; mi < 2; ++mi) {
        const int row = wm * 32 + mi * 16 + g, kk = ks * 16 + 2 * t;
        a[mi][0] = *reinterpret_cast<const uint32_t*>(&As[row * kWPitch + kk]);
        a[mi][1] = *reinterpret_cast<const uint32_t*>(&As[(row + 8) * kWPitch + kk]);
        a[mi][2] = *reinterpret_cast<const uint32_t*>(&As[row * kWPitch + kk + 8]);
        a[mi][3] = *reinterpret_cast<const uint32_t*>(&As[(row + 8) * kWPitch + kk + 8]);
      }
#pragma unroll
      for (int ni = 0; ni < 4; ++ni) {
        const int nn = wn * 32 + ni * 8 + g, kk = ks * 16 + 2 * t;
        b[ni][0] = *reinterpret_cast<const uint32_t*>(&Bs[nn * kWPitch + kk]);
        b[ni][1] = *reinterpret_cast<const uint32_t*>(&Bs[nn * kWPitch + kk + 8]);
      }
#pragma unroll
      for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
          mma_bf16_16816(c[mi][ni], a[mi][0], a[mi][1], a[mi][2], a[mi][3], b[ni][0], b[ni][1]);
    }
  }
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int ni = 0; ni < 4; ++ni) {
      const int col = n0 + wn * 32 + ni * 8 + 2 * t;
      if (col >= d_out) continue;  // d_out is even, so col + 1 < d_out as well
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int row = m0 + wm * 32 + mi * 16 + g + hh * 8;
        if (row >= T) continue;
        const float v0 = c[mi][ni][hh * 2], v1 = c[mi][ni][hh * 2 + 1];
        const size_t o = (size_t)row * d_out + col;
        *reinterpret_cast<uint32_t*>(y + o) = pack_bf16(v0, v1);
        if (y0) *reinterpret_cast<float2*>(y0 + o) = make_float2(v0, v1);
      }
    }
}

cudaError_t launch_gemm_warp(const __nv_bfloat16* x, const __nv_bfloat16* W, __nv_bfloat16* y, float* y0, int T,
                             int d_in, int d_out, cudaStream_t stream) {
  dim3 grid((d_out + kWBN - 1) / kWBN, (T + kWBM - 1) / kWBM);
  gemm_warp_kernel<<<grid, 128, 0, stream>>>(x, W, y, y0, T, d_in, d_out);
  return cudaGetLastError();
}

}  // namespace moin
