// Segmented LoRA shrink / expand for short segments (decode), TMA-staged.
//
// Each distinct adapter is streamed from HBM exactly once per call.  A producer warp keeps a
// deep ring of shared-memory stages full with 128B-swizzled TMA boxes of the adapter matrices
// and 1-D bulk copies of the few token rows the stage needs, so the memory pipeline never
// drains at work-item boundaries; consumer warps read the stages with ldmatrix and run the
// skinny products on warp-level MMA (m16n8k16, 8 token columns).
//
//   shrink: item = (segment, 512-wide part of d_in).  Stage = A_e[:, 256 k] as 4 boxes of
//           [r x 64] + up to 8 token rows x 256 k.  Consumer warp w (of 4) owns adapter rows
//           16w..16w+15.  Output: partial h[part][pos][rho] (fp32); the parts are summed in a
//           fixed order by the expand, so the result is deterministic.
//   expand: item = (segment, 256 output features).  Stage = B_e[256 rows, r] as one box
//           (columns beyond r read as zero) + the base values y0[token][256 features] of up to
//           8 tokens.  Consumer warp w (of 8) owns row tiles w and w + 8; the hi and lo products
//           run in separate accumulators so the MMA chains stay short.  The token operand
//           (scale * sum of the shrink's partials) is reduced once per segment into shared memory.
// Every CTA takes a contiguous range of items so consecutive items share a segment.
// All waits (mbarriers, including the consumer-only barrier) are bounded.
#include "ptx.cuh"
#include "tc_gemm.cuh"

namespace moin {

constexpr int kSK = 256;                  // k columns per shrink stage
constexpr int kSPart = 512;               // k columns per shrink work item
constexpr int kSXPitch = kSK * 2 + 16;    // token row pitch in a shrink stage (conflict-free 32-bit reads)
constexpr int kShrinkConsumers = 4;
constexpr int kShrinkThreads = 32 * (1 + kShrinkConsumers);
constexpr int kEBoxRows = 256;            // output features per expand stage
constexpr int kEBoxBytes = kEBoxRows * 128;
constexpr int kEYPitch = kEBoxRows * 4 + 16;   // staged base-value row pitch (conflict-free 32-bit reads)
constexpr int kEStageBytes = (kEBoxBytes + 8 * kEYPitch + 1023) / 1024 * 1024;
constexpr int kExpandConsumers = 8;
constexpr int kExpandThreads = 32 * (1 + kExpandConsumers);
constexpr int kEHPitch = 66;              // token-operand cache row pitch (floats)
constexpr int kMaxStages = 12;
constexpr size_t kRingBytes = 190 * 1024;
constexpr int kBarBytes = 16 * kMaxStages + 64;   // full[], empty[], consumer barrier, abort flag

struct SegInfo { int slot, s0, n; };
__device__ __forceinline__ SegInfo seg_info(const int4* __restrict__ seg_tab, const int* __restrict__ slot_of_expert,
                                            int seg) {
  const int4 e = __ldg(seg_tab + seg);   // (expert, start, length, -)
  SegInfo m;
  m.slot = __ldg(slot_of_expert + e.x);
  m.s0 = e.y;
  m.n = e.z;
  return m;
}

struct RingSmem {
  uint32_t base, full0, empty0, cbar;
  volatile int* abort_flag;
  uint8_t* tail;   // shared memory after the barriers
};
__device__ __forceinline__ RingSmem ring_setup(uint8_t* smem_raw, int n_stages, int stage_bytes, int consumer_warps) {
  RingSmem rs;
  const uint32_t raw = smem_u32(smem_raw);
  rs.base = (raw + 1023u) & ~1023u;
  const uint32_t bars = rs.base + (uint32_t)n_stages * (uint32_t)stage_bytes;
  rs.full0 = bars;
  rs.empty0 = bars + 8 * kMaxStages;
  rs.cbar = bars + 16 * kMaxStages;
  rs.abort_flag = reinterpret_cast<volatile int*>(smem_raw + (bars - raw) + 16 * kMaxStages + 8);
  rs.tail = smem_raw + (bars - raw) + kBarBytes;
  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(rs.full0 + 8 * s, 1);
      mbar_init(rs.empty0 + 8 * s, consumer_warps);
    }
    mbar_init(rs.cbar, 32 * consumer_warps);   // consumer-only barrier (bounded, unlike bar.sync)
    *rs.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  return rs;
}
__device__ __forceinline__ void ring_teardown(const RingSmem& rs) {
  if (*rs.abort_flag) {   // a wait ran out: let copies in flight land before the shared memory is released
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kShrinkThreads, 1)
lora_shrink_tma_kernel(const __grid_constant__ CUtensorMap tmA, const int* __restrict__ header,
                       const int* __restrict__ perm, const int4* __restrict__ seg_tab,
                       const int* __restrict__ slot_of_expert, const __nv_bfloat16* __restrict__ x,
                       float* __restrict__ hpart, int r, int d_in, int T, int stage_bytes, int n_stages,
                       DeviceStatus* status) {
  extern __shared__ uint8_t smem_raw[];
  const RingSmem rs = ring_setup(smem_raw, n_stages, stage_bytes, kShrinkConsumers);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nseg = header[PH_NSEG];
  const int KP = (d_in + kSPart - 1) / kSPart;
  const long total = (long)nseg * KP;
  const int item_lo = (int)(total * blockIdx.x / gridDim.x), item_hi = (int)(total * (blockIdx.x + 1) / gridDim.x);
  const uint32_t a_bytes = (uint32_t)(kSK / 64) * (uint32_t)r * 128u;
  const uint32_t box_bytes = (uint32_t)r * 128u;
  uint32_t it = 0;
  int cur_seg = -1;
  SegInfo m = {-1, 0, 0};
  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    bool ok = true;
    int row = -1, row_seg = -1, row_tc = -1;
    for (int item = item_lo; item < item_hi && ok; ++item) {
      const int seg = item / KP, kp = item - seg * KP;
      if (seg != cur_seg) { m = seg_info(seg_tab, slot_of_expert, seg); cur_seg = seg; }
      if (m.slot < 0) continue;
      const int k_lo = kp * kSPart, k_hi = min(d_in, k_lo + kSPart);
      for (int tc = 0; tc < m.n && ok; tc += 8) {
        if (seg != row_seg || tc != row_tc) {   // token rows change only with the segment chunk
          row = (lane < 8 && tc + lane < m.n) ? __ldg(perm + m.s0 + tc + lane) : -1;
          row_seg = seg;
          row_tc = tc;
        }
        const uint32_t nvalid = (uint32_t)min(8, m.n - tc);
        for (int kc = k_lo; kc < k_hi; kc += kSK, ++it) {
          const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
          if (!(ok = mbar_wait(rs.empty0 + 8 * s, ph ^ 1u, rs.abort_flag, status, 11))) break;
          const uint32_t sa = rs.base + s * (uint32_t)stage_bytes, sx = sa + a_bytes;
          if (lane == 0) {
            mbar_expect_tx(rs.full0 + 8 * s, a_bytes + nvalid * (uint32_t)(kSK * 2));
#pragma unroll
            for (int b = 0; b < kSK / 64; ++b) tma_load_2d(sa + b * box_bytes, &tmA, rs.full0 + 8 * s, kc + 64 * b, m.slot * r);
          }
          if (row >= 0) bulk_load_1d(sx + lane * kSXPitch, x + (size_t)row * d_in + kc, kSK * 2, rs.full0 + 8 * s);
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers
    const int w = warp - 1, g = lane >> 2, t = lane & 3;
    const bool active = 16 * w < r;
    const int lm_row = 16 * w + ((lane >> 3) & 1) * 8 + (lane & 7);   // ldmatrix: row this lane addresses
    const int lm_chunk = lane >> 4;                                   //           k chunk offset (0/1)
    bool ok = true;
    for (int item = item_lo; item < item_hi && ok; ++item) {
      const int seg = item / KP, kp = item - seg * KP;
      if (seg != cur_seg) { m = seg_info(seg_tab, slot_of_expert, seg); cur_seg = seg; }
      if (m.slot < 0) continue;
      const int k_lo = kp * kSPart, k_hi = min(d_in, k_lo + kSPart);
      for (int tc = 0; tc < m.n && ok; tc += 8) {
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        for (int kc = k_lo; kc < k_hi; kc += kSK, ++it) {
          const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
          if (!(ok = mbar_wait(rs.full0 + 8 * s, ph, rs.abort_flag, status, 12))) break;
          if (active) {
            const uint32_t sa = rs.base + s * (uint32_t)stage_bytes, sx = sa + a_bytes + g * kSXPitch;
#pragma unroll
            for (int b = 0; b < kSK / 64; ++b) {
#pragma unroll
              for (int ks = 0; ks < 4; ++ks) {
                const int ch = 2 * ks + lm_chunk;
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4(sa + b * box_bytes + lm_row * 128 + ((ch ^ (lm_row & 7)) << 4), a0, a1, a2, a3);
                const uint32_t xo = sx + (uint32_t)(b * 64 + ks * 16 + 2 * t) * 2u;
                mma_bf16_16816(c, a0, a1, a2, a3, lds_u32(xo), lds_u32(xo + 16));
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(rs.empty0 + 8 * s);
        }
        if (ok && active) {
          // c0:(rho0, col 2t) c1:(rho0, col 2t+1) c2:(rho0+8, col 2t) c3:(rho0+8, col 2t+1)
          const int rho0 = 16 * w + g, rho1 = rho0 + 8, col = tc + 2 * t;
          float* hp = hpart + ((size_t)kp * T + (size_t)(m.s0 + col)) * r;
          if (col < m.n) {
            if (rho0 < r) hp[rho0] = c[0];
            if (rho1 < r) hp[rho1] = c[2];
          }
          if (col + 1 < m.n) {
            if (rho0 < r) hp[r + rho0] = c[1];
            if (rho1 < r) hp[r + rho1] = c[3];
          }
        }
      }
    }
  }
  ring_teardown(rs);
}

__global__ void __launch_bounds__(kExpandThreads, 1)
lora_expand_tma_kernel(const __grid_constant__ CUtensorMap tmB, const int* __restrict__ header,
                       const int* __restrict__ perm, const int4* __restrict__ seg_tab,
                       const int* __restrict__ slot_of_expert, const float* __restrict__ hpart, int KP,
                       const float* __restrict__ y0, __nv_bfloat16* __restrict__ y, float scale, int r, int d_out,
                       int T, int n_stages, DeviceStatus* status) {
  extern __shared__ uint8_t smem_raw[];
  const RingSmem rs = ring_setup(smem_raw, n_stages, kEStageBytes, kExpandConsumers);
  // token operand cache: scale * sum_parts h[part][token][rho] for the 8 token columns of the current segment chunk
  float* h_s = reinterpret_cast<float*>(rs.tail);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nseg = header[PH_NSEG];
  const int JB = (d_out + kEBoxRows - 1) / kEBoxRows;
  const long total = (long)nseg * JB;
  const int item_lo = (int)(total * blockIdx.x / gridDim.x), item_hi = (int)(total * (blockIdx.x + 1) / gridDim.x);
  uint32_t it = 0;
  int cur_seg = -1;
  SegInfo m = {-1, 0, 0};
  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    bool ok = true;
    int row = -1, row_seg = -1, row_tc = -1;
    for (int item = item_lo; item < item_hi && ok; ++item) {
      const int seg = item / JB, jb = item - seg * JB;
      if (seg != cur_seg) { m = seg_info(seg_tab, slot_of_expert, seg); cur_seg = seg; }
      if (m.slot < 0) continue;
      const uint32_t ycols = (uint32_t)min(kEBoxRows, d_out - jb * kEBoxRows);
      for (int tc = 0; tc < m.n; tc += 8, ++it) {
        if (seg != row_seg || tc != row_tc) {
          row = (lane < 8 && tc + lane < m.n) ? __ldg(perm + m.s0 + tc + lane) : -1;
          row_seg = seg;
          row_tc = tc;
        }
        const uint32_t nvalid = (uint32_t)min(8, m.n - tc);
        const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
        if (!(ok = mbar_wait(rs.empty0 + 8 * s, ph ^ 1u, rs.abort_flag, status, 13))) break;
        const uint32_t sb = rs.base + s * kEStageBytes;
        if (lane == 0) {
          mbar_expect_tx(rs.full0 + 8 * s, kEBoxBytes + nvalid * ycols * 4u);
          tma_load_2d(sb, &tmB, rs.full0 + 8 * s, 0, m.slot * d_out + jb * kEBoxRows);
        }
        if (row >= 0)
          bulk_load_1d(sb + kEBoxBytes + lane * kEYPitch, y0 + (size_t)row * d_out + jb * kEBoxRows, ycols * 4u,
                       rs.full0 + 8 * s);
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers (8 warps, 2 row tiles each)
    const int w = warp - 1, g = lane >> 2, t = lane & 3;
    const int ctid = threadIdx.x - 32;          // 0..255 among consumers
    const int KS = (r + 15) >> 4;
    const int lm_sub = ((lane >> 3) & 1) * 8 + (lane & 7), lm_chunk = lane >> 4;
    bool ok = true;
    uint32_t hh[4][2], hl[4][2];
    int h_seg = -1, h_tc = -1, row_c0 = -1, row_c1 = -1;
    uint32_t cph = 0;
    for (int item = item_lo; item < item_hi && ok; ++item) {
      const int seg = item / JB, jb = item - seg * JB;
      if (seg != cur_seg) { m = seg_info(seg_tab, slot_of_expert, seg); cur_seg = seg; }
      if (m.slot < 0) continue;
      for (int tc = 0; tc < m.n && ok; tc += 8, ++it) {
        if (seg != h_seg || tc != h_tc) {   // uniform over all consumer warps
          h_seg = seg;
          h_tc = tc;
          const bool vx = (tc + g) < m.n;
          const int my_row = vx ? __ldg(perm + m.s0 + tc + g) : -1;
          // cooperative, fixed-order sum of the shrink's partial results: thread -> (token, rho pair)
          mbar_arrive(rs.cbar);                              // previous readers of h_s are done
          if (!(ok = mbar_wait(rs.cbar, cph, rs.abort_flag, status, 15))) break;
          cph ^= 1u;
          {
            const int tok = ctid >> 5, rho = (ctid & 31) * 2;
            float v0 = 0.f, v1 = 0.f;
            if (tc + tok < m.n && rho < r) {
              const float* src = hpart + (size_t)(m.s0 + tc + tok) * r + rho;
              const size_t pstride = (size_t)T * r;
              int kp = 0;
              for (; kp + 4 <= KP; kp += 4) {   // four independent loads in flight, summed in order
                const float2 f0 = *reinterpret_cast<const float2*>(src + (size_t)kp * pstride);
                const float2 f1 = *reinterpret_cast<const float2*>(src + (size_t)(kp + 1) * pstride);
                const float2 f2 = *reinterpret_cast<const float2*>(src + (size_t)(kp + 2) * pstride);
                const float2 f3 = *reinterpret_cast<const float2*>(src + (size_t)(kp + 3) * pstride);
                v0 = (((v0 + f0.x) + f1.x) + f2.x) + f3.x;
                v1 = (((v1 + f0.y) + f1.y) + f2.y) + f3.y;
              }
              for (; kp < KP; ++kp) {
                const float2 f = *reinterpret_cast<const float2*>(src + (size_t)kp * pstride);
                v0 += f.x;
                v1 += f.y;
              }
            }
            *reinterpret_cast<float2*>(h_s + tok * kEHPitch + rho) = make_float2(v0 * scale, v1 * scale);
          }
          mbar_arrive(rs.cbar);
          if (!(ok = mbar_wait(rs.cbar, cph, rs.abort_flag, status, 16))) break;
          cph ^= 1u;
          // token operand: column g = token tc + g; k slots of step ks <- rho 16ks + {2t, 2t+1, 2t+8, 2t+9}
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int rho = 16 * ks + 8 * half + 2 * t;
              const float2 f = (ks < KS && rho < r) ? *reinterpret_cast<const float2*>(h_s + g * kEHPitch + rho)
                                                   : make_float2(0.f, 0.f);
              const uint32_t hi = pack_bf16(f.x, f.y);
              hh[ks][half] = hi;
              hl[ks][half] = pack_bf16(f.x - bf16_lo(hi), f.y - bf16_hi(hi));
            }
          }
          row_c0 = __shfl_sync(0xffffffffu, my_row, (2 * t) * 4);
          row_c1 = __shfl_sync(0xffffffffu, my_row, (2 * t + 1) * 4);
        }
        const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
        if (!(ok = mbar_wait(rs.full0 + 8 * s, ph, rs.abort_flag, status, 14))) break;
        const uint32_t sb = rs.base + s * kEStageBytes;
        float acc[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const int tile = w + kExpandConsumers * i;
          // base values of this row tile: staged as [token column][feature] fp32
          const uint32_t o0 = sb + kEBoxBytes + (2 * t) * kEYPitch + (tile * 16 + g) * 4, o1 = o0 + kEYPitch;
          const float b0 = __uint_as_float(lds_u32(o0)), b1 = __uint_as_float(lds_u32(o1));
          const float b2 = __uint_as_float(lds_u32(o0 + 32)), b3 = __uint_as_float(lds_u32(o1 + 32));
          float ch[4] = {0.f, 0.f, 0.f, 0.f}, cl[4] = {0.f, 0.f, 0.f, 0.f};
          const int R = tile * 16 + lm_sub;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            if (ks < KS) {
              const int chk = 2 * ks + lm_chunk;
              uint32_t a0, a1, a2, a3;
              ldmatrix_x4(sb + R * 128 + ((chk ^ (R & 7)) << 4), a0, a1, a2, a3);
              mma_bf16_16816(cl, a0, a1, a2, a3, hl[ks][0], hl[ks][1]);
              mma_bf16_16816(ch, a0, a1, a2, a3, hh[ks][0], hh[ks][1]);
            }
          }
          acc[i][0] = b0 + (cl[0] + ch[0]);
          acc[i][1] = b1 + (cl[1] + ch[1]);
          acc[i][2] = b2 + (cl[2] + ch[2]);
          acc[i][3] = b3 + (cl[3] + ch[3]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(rs.empty0 + 8 * s);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const int ja = jb * kEBoxRows + (w + kExpandConsumers * i) * 16 + g, jc = ja + 8;
          // c0:(ja, col 2t) c1:(ja, col 2t+1) c2:(jc, col 2t) c3:(jc, col 2t+1)
          if (row_c0 >= 0) {
            const size_t o = (size_t)row_c0 * d_out;
            if (ja < d_out) y[o + ja] = __float2bfloat16_rn(acc[i][0]);
            if (jc < d_out) y[o + jc] = __float2bfloat16_rn(acc[i][2]);
          }
          if (row_c1 >= 0) {
            const size_t o = (size_t)row_c1 * d_out;
            if (ja < d_out) y[o + ja] = __float2bfloat16_rn(acc[i][1]);
            if (jc < d_out) y[o + jc] = __float2bfloat16_rn(acc[i][3]);
          }
        }
      }
    }
  }
  ring_teardown(rs);
}

// ---------------------------------------------------------------------------------------------
int lora_stream_parts(int d_in) { return (d_in % kSK) == 0 ? (d_in + kSPart - 1) / kSPart : 1; }
bool lora_shrink_tma_supported(int d_in) { return (d_in % kSK) == 0; }

static int pick_stages(int stage_bytes) {
  int s = (int)(kRingBytes / (size_t)stage_bytes);
  return s > kMaxStages ? kMaxStages : (s < 2 ? 2 : s);
}
static size_t ring_smem(int stages, int stage_bytes) {
  return (size_t)stages * stage_bytes + 1024 + kBarBytes + 8 * kEHPitch * sizeof(float);
}
static int ring_grid(long max_items, int n_sms) {
  return (int)(max_items < n_sms ? (max_items < 1 ? 1 : max_items) : n_sms);
}

moin_status launch_lora_shrink_tma(HostState* hs, const PlanView& pv, const moin_pool* pool, const __nv_bfloat16* x,
                                   float* hpart, cudaStream_t stream) {
  const int r = pool->r, d_in = pool->d_in;
  CUtensorMap tmA;
  moin_status st = make_map(&tmA, pool->A, (uint64_t)pool->n_slots * r, d_in, (uint32_t)r);
  if (st) return st;
  const int stage_bytes = (int)align_up((size_t)(kSK / 64) * r * 128 + 8 * kSXPitch, 1024);
  const int stages = pick_stages(stage_bytes);
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(lora_shrink_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(kRingBytes + 16 * 1024));
    if (e != cudaSuccess) return record_cuda(e);
    configured = true;
  }
  const int grid = ring_grid((long)pv.Smax * lora_stream_parts(d_in), hs->n_sms);
  lora_shrink_tma_kernel<<<grid, kShrinkThreads, ring_smem(stages, stage_bytes), stream>>>(
      tmA, pv.header, pv.perm, pv.seg_tab, pool->slot_of_expert, x, hpart, r, d_in, pv.T, stage_bytes, stages, hs->status);
  return record_cuda(cudaGetLastError());
}

moin_status launch_lora_expand_tma(HostState* hs, const PlanView& pv, const moin_pool* pool, const float* hpart, int KP,
                                   const float* y0, __nv_bfloat16* y, float scale, cudaStream_t stream) {
  const int r = pool->r, d_out = pool->d_out;
  CUtensorMap tmB;
  moin_status st = make_map(&tmB, pool->B, (uint64_t)pool->n_slots * d_out, r, kEBoxRows);
  if (st) return st;
  const int stages = pick_stages(kEStageBytes);
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(lora_expand_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(kRingBytes + 16 * 1024));
    if (e != cudaSuccess) return record_cuda(e);
    configured = true;
  }
  const int grid = ring_grid((long)pv.Smax * ((d_out + kEBoxRows - 1) / kEBoxRows), hs->n_sms);
  lora_expand_tma_kernel<<<grid, kExpandThreads, ring_smem(stages, kEStageBytes), stream>>>(
      tmB, pv.header, pv.perm, pv.seg_tab, pool->slot_of_expert, hpart, KP, y0, y, scale, r, d_out, pv.T, stages,
      hs->status);
  return record_cuda(cudaGetLastError());
}

}  // namespace moin
