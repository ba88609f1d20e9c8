// Segmented LoRA shrink / expand for short segments (decode), TMA-staged, up to 4 projections per launch.
//
// Each distinct adapter is streamed from HBM exactly once per call.  A producer warp pulls work items
// from a global queue (an atomic counter), and keeps a ring of shared-memory stages full: 128B-swizzled
// TMA boxes of the adapter matrices plus 1-D bulk copies of the few token rows the stage needs.  Every
// stage carries a small descriptor (which projection, which tokens, first/last stage of an accumulation),
// so the consumer warps simply follow the ring: ldmatrix + warp-level MMA (m16n8k16, 8 token columns).
// The memory pipeline therefore never drains at item boundaries, and CTAs that start late (their SM was
// busy with a base-GEMM CTA) just take fewer items.
//
//   shrink: item = (projection, segment, 512-wide part of d_in).  Stage = A_e[:, 256 k] as 4 boxes of
//           [r x 64] + up to 8 token rows x 256 k.  Consumer warp w (of 4) owns adapter rows 16w..16w+15.
//           Output: partial h[part][pos][rho] (fp32); the parts are summed in index order by the expand, so
//           the result does not depend on which CTA computed which part.
//   expand: item = (projection, segment, 4 blocks of 256 output features).  Stage = B_e[256 rows, r] as one
//           box (columns beyond r read as zero) + the base values y0[token][256 features] of up to 8 tokens.
//           Consumer warp w (of 8) owns row tiles w and w + 8; hi and lo products run in separate
//           accumulators.  The token operand (scale * sum of the shrink's partials) is reduced into shared
//           memory whenever the (projection, segment) changes.
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
constexpr int kEBlocksPerItem = 4;        // expand stages per work item (same segment -> same token operand)
constexpr int kEBoxBytes = kEBoxRows * 128;
constexpr int kEYPitch = kEBoxRows * 4 + 16;   // staged base-value row pitch (conflict-free 32-bit reads)
constexpr int kEStageBytes = (kEBoxBytes + 8 * kEYPitch + 1023) / 1024 * 1024;
constexpr int kExpandConsumers = 8;
constexpr int kExpandThreads = 32 * (1 + kExpandConsumers);
constexpr int kEHPitch = 66;              // token-operand cache row pitch (floats)
constexpr int kMaxStages = 12;
constexpr int kBarBytes = 16 * kMaxStages + 64;        // full[], empty[], consumer barrier, abort flag
constexpr int kDescBytes = 32 * kMaxStages;            // one StageDesc per stage
constexpr int kTailBytes = kBarBytes + kDescBytes + 8 * kEHPitch * 4;

struct StageDesc {   // written by the producer before it arms the stage's barrier
  int job;           // projection index, -1 = no more work
  int slot;          // adapter slot
  int pos0;          // first sorted-token position of the stage's 8 token columns
  int nvalid;        // token columns in use (1..8)
  int sub;           // shrink: part of d_in; expand: block of 256 output features
  int flags;         // bit 0: first stage of an accumulation, bit 1: last stage, bit 2: token operand changed
  int seg_n;         // tokens in the segment
  int pad;
};

struct ShrinkTmaJobs {
  const __nv_bfloat16* x[kMaxStreamJobs];
  float* hpart[kMaxStreamJobs];
  const int* slot_of_expert[kMaxStreamJobs];
  int r[kMaxStreamJobs], d_in[kMaxStreamJobs], parts[kMaxStreamJobs];
  int n;
};
struct ExpandTmaJobs {
  const float* hpart[kMaxStreamJobs];
  const float* y0[kMaxStreamJobs];
  __nv_bfloat16* y[kMaxStreamJobs];
  const int* slot_of_expert[kMaxStreamJobs];
  int r[kMaxStreamJobs], d_out[kMaxStreamJobs], parts[kMaxStreamJobs], per_seg[kMaxStreamJobs];
  int n;
};

template <class V>
__device__ __forceinline__ V pick4(const V (&arr)[kMaxStreamJobs], int j) {   // compile-time indices only
  V v = arr[0];
#pragma unroll
  for (int i = 1; i < kMaxStreamJobs; ++i)
    if (j == i) v = arr[i];
  return v;
}
__device__ __forceinline__ const CUtensorMap* pick_map(const CUtensorMap* m0, const CUtensorMap* m1,
                                                       const CUtensorMap* m2, const CUtensorMap* m3, int j) {
  return j == 0 ? m0 : (j == 1 ? m1 : (j == 2 ? m2 : m3));
}

struct RingSmem {
  uint32_t base, full0, empty0, cbar;
  volatile int* abort_flag;
  StageDesc* desc;
  float* h_s;
};
__device__ __forceinline__ RingSmem ring_setup(uint8_t* smem_raw, int n_stages, int stage_bytes, int consumer_warps) {
  RingSmem rs;
  const uint32_t raw = smem_u32(smem_raw);
  rs.base = (raw + 1023u) & ~1023u;
  const uint32_t bars = rs.base + (uint32_t)n_stages * (uint32_t)stage_bytes;
  uint8_t* tail = smem_raw + (bars - raw);
  rs.full0 = bars;
  rs.empty0 = bars + 8 * kMaxStages;
  rs.cbar = bars + 16 * kMaxStages;
  rs.abort_flag = reinterpret_cast<volatile int*>(tail + 16 * kMaxStages + 8);
  rs.desc = reinterpret_cast<StageDesc*>(tail + kBarBytes);
  rs.h_s = reinterpret_cast<float*>(tail + kBarBytes + kDescBytes);
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

// item -> (job, segment, sub) with per_seg[j] items per segment in job j, jobs laid out one after the other
template <class Jobs>
__device__ __forceinline__ void decode_item(int item, int nseg, const Jobs& jobs, const int (&per_seg)[kMaxStreamJobs],
                                            int& job, int& seg, int& sub) {
  job = 0;
  int rem = item;
#pragma unroll
  for (int j = 0; j + 1 < kMaxStreamJobs; ++j) {
    if (job == j && j + 1 < jobs.n && rem >= nseg * per_seg[j]) {
      rem -= nseg * per_seg[j];
      job = j + 1;
    }
  }
  const int ps = pick4(per_seg, job);
  seg = rem / ps;
  sub = rem - seg * ps;
}

__global__ void __launch_bounds__(kShrinkThreads, 1)
lora_shrink_tma_kernel(const __grid_constant__ CUtensorMap tm0, const __grid_constant__ CUtensorMap tm1,
                       const __grid_constant__ CUtensorMap tm2, const __grid_constant__ CUtensorMap tm3,
                       const int* __restrict__ header, const int* __restrict__ perm, const int4* __restrict__ seg_tab,
                       const ShrinkTmaJobs jobs, int T, int stage_bytes, int n_stages, int* queue,
                       DeviceStatus* status) {
  extern __shared__ uint8_t smem_raw[];
  const RingSmem rs = ring_setup(smem_raw, n_stages, stage_bytes, kShrinkConsumers);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint32_t it = 0;
  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    const int nseg = header[PH_NSEG];
    int total = 0;
#pragma unroll
    for (int j = 0; j < kMaxStreamJobs; ++j)
      if (j < jobs.n) total += nseg * jobs.parts[j];
    bool ok = true;
    while (ok) {
      int item = 0;
      if (lane == 0) item = atomicAdd(queue, 1);
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item >= total) break;
      int job, seg, kp;
      decode_item(item, nseg, jobs, jobs.parts, job, seg, kp);
      const int4 e = __ldg(seg_tab + seg);   // (expert, start, length, -)
      const int slot = __ldg(pick4(jobs.slot_of_expert, job) + e.x);
      if (slot < 0) continue;
      const int r = pick4(jobs.r, job), d_in = pick4(jobs.d_in, job);
      const __nv_bfloat16* x = pick4(jobs.x, job);
      const CUtensorMap* map = pick_map(&tm0, &tm1, &tm2, &tm3, job);
      const uint32_t box_bytes = (uint32_t)r * 128u, a_bytes = (uint32_t)(kSK / 64) * box_bytes;
      const int k_lo = kp * kSPart, k_hi = min(d_in, k_lo + kSPart);
      for (int tc = 0; tc < e.z && ok; tc += 8) {
        const int row = (lane < 8 && tc + lane < e.z) ? __ldg(perm + e.y + tc + lane) : -1;
        const int nvalid = min(8, e.z - tc);
        for (int kc = k_lo; kc < k_hi; kc += kSK, ++it) {
          const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
          if (!(ok = mbar_wait(rs.empty0 + 8 * s, ph ^ 1u, rs.abort_flag, status, 11))) break;
          const uint32_t sa = rs.base + s * (uint32_t)stage_bytes, sx = sa + 4u * 64u * 128u;   // x rows after 4 full boxes
          if (lane == 0) {
            StageDesc d = {job, slot, e.y + tc, nvalid, kp, (kc == k_lo ? 1 : 0) | (kc + kSK >= k_hi ? 2 : 0), e.z, 0};
            rs.desc[s] = d;
            mbar_expect_tx(rs.full0 + 8 * s, a_bytes + (uint32_t)nvalid * (uint32_t)(kSK * 2));
#pragma unroll
            for (int b = 0; b < kSK / 64; ++b) tma_load_2d(sa + b * box_bytes, map, rs.full0 + 8 * s, kc + 64 * b, slot * r);
          }
          if (row >= 0) bulk_load_1d(sx + lane * kSXPitch, x + (size_t)row * d_in + kc, kSK * 2, rs.full0 + 8 * s);
        }
      }
    }
    if (ok) {   // end-of-work marker
      const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
      if (mbar_wait(rs.empty0 + 8 * s, ph ^ 1u, rs.abort_flag, status, 17) && lane == 0) {
        rs.desc[s].job = -1;
        mbar_arrive(rs.full0 + 8 * s);
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers
    const int w = warp - 1, g = lane >> 2, t = lane & 3;
    const int lm_row = 16 * w + ((lane >> 3) & 1) * 8 + (lane & 7);   // ldmatrix: row this lane addresses
    const int lm_chunk = lane >> 4;                                   //           k chunk offset (0/1)
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    for (;; ++it) {
      const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
      if (!mbar_wait(rs.full0 + 8 * s, ph, rs.abort_flag, status, 12)) break;
      const StageDesc d = rs.desc[s];
      if (d.job < 0) break;
      const int r = pick4(jobs.r, d.job);
      const bool active = 16 * w < r;
      if (d.flags & 1) c[0] = c[1] = c[2] = c[3] = 0.f;
      if (active) {
        const uint32_t box_bytes = (uint32_t)r * 128u;
        const uint32_t sa = rs.base + s * (uint32_t)stage_bytes, sx = sa + 4u * 64u * 128u + g * kSXPitch;
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
      if ((d.flags & 2) && active) {
        // c0:(rho0, col 2t) c1:(rho0, col 2t+1) c2:(rho0+8, col 2t) c3:(rho0+8, col 2t+1)
        const int rho0 = 16 * w + g, rho1 = rho0 + 8, col = 2 * t;
        float* hp = pick4(jobs.hpart, d.job) + ((size_t)d.sub * T + (size_t)(d.pos0 + col)) * r;
        if (col < d.nvalid) {
          if (rho0 < r) hp[rho0] = c[0];
          if (rho1 < r) hp[rho1] = c[2];
        }
        if (col + 1 < d.nvalid) {
          if (rho0 < r) hp[r + rho0] = c[1];
          if (rho1 < r) hp[r + rho1] = c[3];
        }
      }
    }
  }
  ring_teardown(rs);
}

__global__ void __launch_bounds__(kExpandThreads, 1)
lora_expand_tma_kernel(const __grid_constant__ CUtensorMap tm0, const __grid_constant__ CUtensorMap tm1,
                       const __grid_constant__ CUtensorMap tm2, const __grid_constant__ CUtensorMap tm3,
                       const int* __restrict__ header, const int* __restrict__ perm, const int4* __restrict__ seg_tab,
                       const ExpandTmaJobs jobs, float scale, int T, int n_stages, int* queue, DeviceStatus* status) {
  extern __shared__ uint8_t smem_raw[];
  const RingSmem rs = ring_setup(smem_raw, n_stages, kEStageBytes, kExpandConsumers);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint32_t it = 0;
  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    const int nseg = header[PH_NSEG];
    int total = 0;
#pragma unroll
    for (int j = 0; j < kMaxStreamJobs; ++j)
      if (j < jobs.n) total += nseg * jobs.per_seg[j];
    bool ok = true;
    while (ok) {
      int item = 0;
      if (lane == 0) item = atomicAdd(queue, 1);
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item >= total) break;
      int job, seg, grp;
      decode_item(item, nseg, jobs, jobs.per_seg, job, seg, grp);
      const int4 e = __ldg(seg_tab + seg);
      const int slot = __ldg(pick4(jobs.slot_of_expert, job) + e.x);
      if (slot < 0) continue;
      const int d_out = pick4(jobs.d_out, job);
      const float* y0 = pick4(jobs.y0, job);
      const CUtensorMap* map = pick_map(&tm0, &tm1, &tm2, &tm3, job);
      const int JB = (d_out + kEBoxRows - 1) / kEBoxRows;
      const int jb_lo = grp * kEBlocksPerItem, jb_hi = min(JB, jb_lo + kEBlocksPerItem);
      for (int tc = 0; tc < e.z && ok; tc += 8) {
        const int row = (lane < 8 && tc + lane < e.z) ? __ldg(perm + e.y + tc + lane) : -1;
        const int nvalid = min(8, e.z - tc);
        for (int jb = jb_lo; jb < jb_hi; ++jb, ++it) {
          const uint32_t ycols = (uint32_t)min(kEBoxRows, d_out - jb * kEBoxRows);
          const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
          if (!(ok = mbar_wait(rs.empty0 + 8 * s, ph ^ 1u, rs.abort_flag, status, 13))) break;
          const uint32_t sb = rs.base + s * kEStageBytes;
          if (lane == 0) {
            StageDesc d = {job, slot, e.y + tc, nvalid, jb, (jb == jb_lo ? 4 : 0), e.z, 0};
            rs.desc[s] = d;
            mbar_expect_tx(rs.full0 + 8 * s, kEBoxBytes + (uint32_t)nvalid * ycols * 4u);
            tma_load_2d(sb, map, rs.full0 + 8 * s, 0, slot * d_out + jb * kEBoxRows);
          }
          if (row >= 0)
            bulk_load_1d(sb + kEBoxBytes + lane * kEYPitch, y0 + (size_t)row * d_out + jb * kEBoxRows, ycols * 4u,
                         rs.full0 + 8 * s);
        }
      }
    }
    if (ok) {   // end-of-work marker
      const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
      if (mbar_wait(rs.empty0 + 8 * s, ph ^ 1u, rs.abort_flag, status, 18) && lane == 0) {
        rs.desc[s].job = -1;
        mbar_arrive(rs.full0 + 8 * s);
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers (8 warps, 2 row tiles each)
    const int w = warp - 1, g = lane >> 2, t = lane & 3;
    const int ctid = threadIdx.x - 32;          // 0..255 among consumers
    const int lm_sub = ((lane >> 3) & 1) * 8 + (lane & 7), lm_chunk = lane >> 4;
    uint32_t hh[4][2], hl[4][2];
    int row_c0 = -1, row_c1 = -1;
    uint32_t cph = 0;
    for (;; ++it) {
      const uint32_t s = it % n_stages, ph = (it / n_stages) & 1u;
      if (!mbar_wait(rs.full0 + 8 * s, ph, rs.abort_flag, status, 14)) break;
      const StageDesc d = rs.desc[s];
      if (d.job < 0) break;
      const int r = pick4(jobs.r, d.job), d_out = pick4(jobs.d_out, d.job);
      const int KS = (r + 15) >> 4;
      if (d.flags & 4) {   // new (projection, segment chunk): rebuild the token operand; uniform over the consumers
        const int KP = pick4(jobs.parts, d.job);
        const float* hpart = pick4(jobs.hpart, d.job);
        const int my_row = (g < d.nvalid) ? __ldg(perm + d.pos0 + g) : -1;
        // cooperative, index-ordered sum of the shrink's partial results: thread -> (token, rho pair)
        mbar_arrive(rs.cbar);                              // previous readers of h_s are done
        if (!mbar_wait(rs.cbar, cph, rs.abort_flag, status, 15)) break;
        cph ^= 1u;
        {
          const int tok = ctid >> 5, rho = (ctid & 31) * 2;
          float v0 = 0.f, v1 = 0.f;
          if (tok < d.nvalid && rho < r) {
            const float* src = hpart + (size_t)(d.pos0 + tok) * r + rho;
            const size_t pstride = (size_t)T * r;
            int kp = 0;
            for (; kp + 4 <= KP; kp += 4) {   // four independent loads in flight, summed in order
              const float2 f0 = __ldcg(reinterpret_cast<const float2*>(src + (size_t)kp * pstride));
              const float2 f1 = __ldcg(reinterpret_cast<const float2*>(src + (size_t)(kp + 1) * pstride));
              const float2 f2 = __ldcg(reinterpret_cast<const float2*>(src + (size_t)(kp + 2) * pstride));
              const float2 f3 = __ldcg(reinterpret_cast<const float2*>(src + (size_t)(kp + 3) * pstride));
              v0 = (((v0 + f0.x) + f1.x) + f2.x) + f3.x;
              v1 = (((v1 + f0.y) + f1.y) + f2.y) + f3.y;
            }
            for (; kp < KP; ++kp) {
              const float2 f = __ldcg(reinterpret_cast<const float2*>(src + (size_t)kp * pstride));
              v0 += f.x;
              v1 += f.y;
            }
          }
          *reinterpret_cast<float2*>(rs.h_s + tok * kEHPitch + rho) = make_float2(v0 * scale, v1 * scale);
        }
        mbar_arrive(rs.cbar);
        if (!mbar_wait(rs.cbar, cph, rs.abort_flag, status, 16)) break;
        cph ^= 1u;
        // token operand: column g = token g of the chunk; k slots of step ks <- rho 16ks + {2t, 2t+1, 2t+8, 2t+9}
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int rho = 16 * ks + 8 * half + 2 * t;
            const float2 f = (ks < KS && rho < r) ? *reinterpret_cast<const float2*>(rs.h_s + g * kEHPitch + rho)
                                                 : make_float2(0.f, 0.f);
            const uint32_t hi = pack_bf16(f.x, f.y);
            hh[ks][half] = hi;
            hl[ks][half] = pack_bf16(f.x - bf16_lo(hi), f.y - bf16_hi(hi));
          }
        }
        row_c0 = __shfl_sync(0xffffffffu, my_row, (2 * t) * 4);
        row_c1 = __shfl_sync(0xffffffffu, my_row, (2 * t + 1) * 4);
      }
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
      __nv_bfloat16* y = pick4(jobs.y, d.job);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int ja = d.sub * kEBoxRows + (w + kExpandConsumers * i) * 16 + g, jc = ja + 8;
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
  ring_teardown(rs);
}

// ---------------------------------------------------------------------------------------------
int lora_stream_parts(int d_in) { return (d_in % kSK) == 0 ? (d_in + kSPart - 1) / kSPart : 1; }
bool lora_shrink_tma_supported(int d_in) { return (d_in % kSK) == 0; }
size_t lora_stream_ring_bytes() { return 190 * 1024; }

static int pick_stages(size_t ring_bytes, int stage_bytes) {
  int s = (int)(ring_bytes / (size_t)stage_bytes);
  return s > kMaxStages ? kMaxStages : (s < 2 ? 2 : s);
}
static size_t ring_smem(int stages, int stage_bytes) { return (size_t)stages * stage_bytes + 1024 + kTailBytes; }

moin_status launch_lora_shrink_tma(HostState* hs, const PlanView& pv, const moin_pool* const* pools,
                                   const __nv_bfloat16* const* x, float* const* hpart, int n_jobs, int* queue,
                                   size_t ring_bytes, cudaStream_t stream) {
  CUtensorMap tm[kMaxStreamJobs];
  ShrinkTmaJobs jobs = {};
  jobs.n = n_jobs;
  long items = 0;
  for (int j = 0; j < kMaxStreamJobs; ++j) {
    const int jj = j < n_jobs ? j : 0;
    const moin_pool* p = pools[jj];
    moin_status st = make_map(&tm[j], p->A, (uint64_t)p->n_slots * p->r, p->d_in, (uint32_t)p->r);
    if (st) return st;
    if (j < n_jobs) {
      jobs.x[j] = x[j]; jobs.hpart[j] = hpart[j]; jobs.slot_of_expert[j] = p->slot_of_expert;
      jobs.r[j] = p->r; jobs.d_in[j] = p->d_in; jobs.parts[j] = lora_stream_parts(p->d_in);
      items += (long)pv.Smax * jobs.parts[j];
    }
  }
  // stage layout: 4 box slots of 64 rows (8 KB each) + 8 token rows, the same for every projection of the launch
  const int stage_bytes = (int)align_up((size_t)4 * 64 * 128 + 8 * kSXPitch, 1024);
  const int stages = pick_stages(ring_bytes, stage_bytes);
  cudaError_t e = ensure_smem_optin(OPTIN_SHRINK_TMA, lora_shrink_tma_kernel, 220 * 1024);
  if (e != cudaSuccess) return record_cuda(e);
  e = cudaMemsetAsync(queue, 0, sizeof(int), stream);
  if (e != cudaSuccess) return record_cuda(e);
  const int grid = (int)(items < hs->n_sms ? (items < 1 ? 1 : items) : hs->n_sms);
  lora_shrink_tma_kernel<<<grid, kShrinkThreads, ring_smem(stages, stage_bytes), stream>>>(
      tm[0], tm[1], tm[2], tm[3], pv.header, pv.perm, pv.seg_tab, jobs, pv.T, stage_bytes, stages, queue, hs->status);
  return record_cuda(cudaGetLastError());
}

moin_status launch_lora_expand_tma(HostState* hs, const PlanView& pv, const moin_pool* const* pools,
                                   const float* const* hpart, const int* parts, const float* const* y0,
                                   __nv_bfloat16* const* y, int n_jobs, float scale, int* queue, size_t ring_bytes,
                                   cudaStream_t stream) {
  CUtensorMap tm[kMaxStreamJobs];
  ExpandTmaJobs jobs = {};
  jobs.n = n_jobs;
  long items = 0;
  for (int j = 0; j < kMaxStreamJobs; ++j) {
    const int jj = j < n_jobs ? j : 0;
    const moin_pool* p = pools[jj];
    moin_status st = make_map(&tm[j], p->B, (uint64_t)p->n_slots * p->d_out, p->r, kEBoxRows);
    if (st) return st;
    if (j < n_jobs) {
      jobs.hpart[j] = hpart[j]; jobs.y0[j] = y0[j]; jobs.y[j] = y[j]; jobs.slot_of_expert[j] = p->slot_of_expert;
      jobs.r[j] = p->r; jobs.d_out[j] = p->d_out; jobs.parts[j] = parts[j];
      const int JB = (p->d_out + kEBoxRows - 1) / kEBoxRows;
      jobs.per_seg[j] = (JB + kEBlocksPerItem - 1) / kEBlocksPerItem;
      items += (long)pv.Smax * jobs.per_seg[j];
    }
  }
  const int stages = pick_stages(ring_bytes, kEStageBytes);
  cudaError_t e = ensure_smem_optin(OPTIN_EXPAND_TMA, lora_expand_tma_kernel, 220 * 1024);
  if (e != cudaSuccess) return record_cuda(e);
  e = cudaMemsetAsync(queue, 0, sizeof(int), stream);
  if (e != cudaSuccess) return record_cuda(e);
  const int grid = (int)(items < hs->n_sms ? (items < 1 ? 1 : items) : hs->n_sms);
  lora_expand_tma_kernel<<<grid, kExpandThreads, ring_smem(stages, kEStageBytes), stream>>>(
      tm[0], tm[1], tm[2], tm[3], pv.header, pv.perm, pv.seg_tab, jobs, scale, pv.T, stages, queue, hs->status);
  return record_cuda(cudaGetLastError());
}

}  // namespace moin
