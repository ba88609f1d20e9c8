// Causal grouped-query attention inside each request on tcgen05 / TMEM (head_dim 64).
//
// One work item = (request, kv head, block of query positions).  The g = n_heads / n_kv_heads query heads
// that share a kv head are stacked into one 128-row tile: row r holds position q0 + r / g of head kvh * g + r % g,
// so a block covers 128 / g positions and every staged K / V tile serves all g heads.  Persistent CTAs (two per
// SM) walk the items, longest first.  Warp roles:
//   warp 0      TMA producer: K and V tiles [64 keys x 64 dims] into small rings.  K is a K-major operand of the
//               form the GEMMs use; V, whose rows run along the output dimension of the second product, is read
//               as an MN-major operand (same staged bytes, the other operand layout), so no transposed copy exists
//   warp 1      MMA issuer: S = Q K^T into one of two TMEM buffers, O += P V into a third
//   warps 2-9   two threads per tile row (32 of a tile's 64 columns each): rotate and stage Q (128-byte swizzled
//               rows, written by hand), softmax, P as the bf16 A operand of the second product (swizzled rows
//               again), normalise and store O
// The softmax takes two passes over the keys: the first only finds each row's maximum, the second forms
// p = 2^(s - max) once per element, sums it in fp32 and multiplies by V - so the O accumulator in TMEM never
// needs rescaling.  S is recomputed in the second pass (the MMAs are a small part of the time; the
// exponentials are not).  Key tiles start at the request's first token (only the innermost coordinate of a TMA
// copy has an alignment rule, and that is the head's first dimension); the mask is key <= query position.
// Every mbarrier wait is bounded; on expiry the CTA raises the status flag, drains and returns.
#include <cuda.h>

#include "ptx.cuh"
#include "tc_gemm.cuh"

namespace moin {

constexpr int kAtThreads = 320;                  // producer warp, MMA warp, 8 softmax warps
constexpr int kAtKeys = 64;                      // keys per tile
constexpr int kAtTile = 128 * 64 * 2;            // Q and P tiles: 128 rows x 128 bytes
constexpr int kAtKV = kAtKeys * 64 * 2;          // K and V tiles: 64 keys x 128 bytes
constexpr int kAtKS = 4, kAtVS = 3;              // ring depths: a tile's loads take about as long as two tiles' work
constexpr int kAtSmem = kAtTile /*Q*/ + 2 * kAtTile /*P*/ + kAtKS * kAtKV + kAtVS * kAtKV + 1024 /*align*/ +
                        256 /*barriers*/ + 2048 /*row maxima and sums of the two half rows*/;
constexpr int kAtTmemCols = 256;                 // S0 [0,64)  S1 [64,128)  O [128,192)

struct AttParams {
  const __nv_bfloat16* q;      // [T, n_heads * 64], not rotated
  __nv_bfloat16* out;          // [T, n_heads * 64]
  const int* cu;               // [R + 1]
  const float2* rope;          // [max_seqlen, 32] (cos, sin)
  int R, n_heads, n_kv, g, ppt, n_qb;   // g heads per kv head, ppt = 128 / g positions per tile, n_qb query blocks
  float scale_log2;
  DeviceStatus* status;
};

// K-major operand with 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart (same as the GEMMs).
__device__ __forceinline__ uint64_t at_sdesc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// D fp32, A / B bf16 K-major, M = 128, N = 64
constexpr uint32_t kAtIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
// the same with B MN-major (V tile: one 128-byte row per key, the 64 output dims contiguous); a 16-key step of
// such a tile is two 8-key groups = 2048 bytes further on
constexpr uint32_t kAtIdescPV = kAtIdesc | (1u << 16);
constexpr uint64_t kAtVStep = 2048 >> 4;

__device__ __forceinline__ float fast_exp2(float x) {   // arguments are <= 0 here: 2^x in (0, 1]
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// byte offset of 16-byte chunk c of row r in a swizzled [rows x 128 bytes] tile
__device__ __forceinline__ uint32_t at_swz(int r, int c) {
  return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4));
}

struct AttItem { int req, kvh, q0, t0, L, a0, n_tiles; bool on; };
__device__ __forceinline__ AttItem at_item(const AttParams& p, int idx) {
  AttItem it;
  const int per_qb = p.R * p.n_kv;
  const int qb = p.n_qb - 1 - idx / per_qb;     // longest blocks first
  const int rem = idx % per_qb;
  it.req = rem / p.n_kv;
  it.kvh = rem % p.n_kv;
  it.q0 = qb * p.ppt;
  it.t0 = __ldg(p.cu + it.req);
  it.L = __ldg(p.cu + it.req + 1) - it.t0;
  it.on = it.q0 < it.L;
  it.a0 = it.t0;
  const int kv_end = min(it.L, it.q0 + p.ppt);   // keys of the request this block can see
  it.n_tiles = it.on ? (it.t0 + kv_end - it.a0 + kAtKeys - 1) / kAtKeys : 0;
  return it;
}

__global__ void __launch_bounds__(kAtThreads, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const AttParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t sQ = base, sP = base + kAtTile, sK = sP + 2 * kAtTile, sV = sK + kAtKS * kAtKV;
  const uint32_t bars = sV + kAtVS * kAtKV;
  uint8_t* bar_ptr = base_ptr + (bars - base);
  // barriers (8 bytes each)
  const uint32_t kfull = bars, kempty = bars + 32, vfull = bars + 64, vempty = bars + 96, sready = bars + 128,
                 sfree = bars + 144, pready = bars + 160, pfree = bars + 176, oready = bars + 192, ofree = bars + 200,
                 qready = bars + 208;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 216);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 224);
  volatile int* sm_fail = reinterpret_cast<volatile int*>(bar_ptr + 228);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kAtKS; ++i) { mbar_init(kfull + 8 * i, 1); mbar_init(kempty + 8 * i, 1); }
    for (int i = 0; i < kAtVS; ++i) { mbar_init(vfull + 8 * i, 1); mbar_init(vempty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(sready + 8 * i, 1); mbar_init(sfree + 8 * i, 256);
      mbar_init(pready + 8 * i, 256); mbar_init(pfree + 8 * i, 1);
    }
    mbar_init(oready, 1);
    mbar_init(ofree, 256);
    mbar_init(qready, 256);
    *abort_flag = 0;
    *sm_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kAtTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_items = p.n_qb * p.R * p.n_kv;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t kq = 0, vq = 0;
      bool ok = true;
      for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
        const AttItem it = at_item(p, idx);
        if (!it.on) continue;
        for (int pass = 0; pass < 2 && ok; ++pass) {
          for (int j = 0; j < it.n_tiles && ok; ++j) {
            const int a = it.a0 + j * kAtKeys;
            {
              const uint32_t s = kq % kAtKS, ph = (kq / kAtKS) & 1u;
              if (!(ok = mbar_wait(kempty + 8 * s, ph ^ 1u, abort_flag, p.status, 31))) break;
              mbar_expect_tx(kfull + 8 * s, kAtKV);
              tma_load_2d(sK + s * kAtKV, &tmK, kfull + 8 * s, it.kvh * 64, a);
              ++kq;
            }
            if (pass == 1) {
              const uint32_t s = vq % kAtVS, ph = (vq / kAtVS) & 1u;
              if (!(ok = mbar_wait(vempty + 8 * s, ph ^ 1u, abort_flag, p.status, 32))) break;
              mbar_expect_tx(vfull + 8 * s, kAtKV);
              tma_load_2d(sV + s * kAtKV, &tmV, vfull + 8 * s, it.kvh * 64, a);
              ++vq;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t kq = 0, vq = 0, sq = 0, pq = 0, nit = 0;
      bool ok = true;
      const uint64_t dq = at_sdesc(sQ);
      auto issue_s = [&]() -> bool {   // S[sq & 1] = Q K^T with the next K stage
        const uint32_t b = sq & 1u, bph = (sq >> 1) & 1u, s = kq % kAtKS, ph = (kq / kAtKS) & 1u;
        if (!mbar_wait(sfree + 8 * b, bph ^ 1u, abort_flag, p.status, 33)) return false;
        if (!mbar_wait(kfull + 8 * s, ph, abort_flag, p.status, 34)) return false;
        tc_fence_after();
        const uint64_t dk = at_sdesc(sK + s * kAtKV);
#pragma unroll
        for (int k = 0; k < 4; ++k) tc_mma_bf16(tmem + b * 64, dq + (uint64_t)(2 * k), dk + (uint64_t)(2 * k), kAtIdesc, k > 0 ? 1u : 0u);
        tc_commit(kempty + 8 * s);
        tc_commit(sready + 8 * b);
        ++sq; ++kq;
        return true;
      };
      for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
        const AttItem it = at_item(p, idx);
        if (!it.on) continue;
        if (!(ok = mbar_wait(qready, nit & 1u, abort_flag, p.status, 35))) break;
        tc_fence_after();
        // pass 1: scores only (the softmax warps take the row maxima)
        for (int j = 0; j < it.n_tiles && ok; ++j) ok = issue_s();
        if (!ok) break;
        // pass 2: scores again, then O += P V; the scores of tile j + 1 are issued before the product of tile j
        if (!(ok = mbar_wait(ofree, (nit & 1u) ^ 1u, abort_flag, p.status, 36))) break;
        ok = issue_s();
        for (int j = 0; j < it.n_tiles && ok; ++j) {
          if (j + 1 < it.n_tiles && !(ok = issue_s())) break;
          const uint32_t b = pq & 1u, bph = (pq >> 1) & 1u, s = vq % kAtVS, ph = (vq / kAtVS) & 1u;
          if (!(ok = mbar_wait(pready + 8 * b, bph, abort_flag, p.status, 37))) break;
          if (!(ok = mbar_wait(vfull + 8 * s, ph, abort_flag, p.status, 38))) break;
          tc_fence_after();
          const uint64_t dp = at_sdesc(sP + b * kAtTile), dv = at_sdesc(sV + s * kAtKV);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma_bf16(tmem + 128, dp + (uint64_t)(2 * k), dv + kAtVStep * k, kAtIdescPV, (j > 0 || k > 0) ? 1u : 0u);
          tc_commit(vempty + 8 * s);
          tc_commit(pfree + 8 * b);
          ++pq; ++vq;
        }
        if (ok) tc_commit(oready);
        ++nit;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / epilogue: two threads per tile row
    // warps 2..5 take columns 0..31 of a tile, warps 6..9 columns 32..63 (a warp may only read the TMEM lanes of its
    // quarter, warp index mod 4).  The two halves of a row meet twice per item through shared memory: for the row
    // maximum after pass 1 and for the row sum after pass 2; those two named barriers are reached by all 256
    // threads whatever happened before (a thread whose wait ran out skips the work, not the barriers), and the
    // decision to give up is taken from a flag that is only written between the item's two barriers.
    const int quarter = warp & 3, half = (warp - 2) >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int qd = p.n_heads * 64;
    float* xm = reinterpret_cast<float*>(bar_ptr + 256);      // [2][128] row maxima of the two halves
    float* xl = xm + 256;                                     // [2][128] row sums
    uint32_t sq = 0, pq = 0, nit = 0;
    bool ok = true;
    for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x) {
      const AttItem it = at_item(p, idx);
      if (!it.on) continue;
      const int pos = it.q0 + row / p.g, head = it.kvh * p.g + row % p.g;
      const bool live = pos < it.L;
      // ---- Q row: load, rotate (pairs (d, d + 32), position inside the request), lay down swizzled.  This thread
      //      takes 16-byte chunks 2 half, 2 half + 1 and their rotation partners 4 further on.
      {
        uint4 c[4];   // chunks i0c, i0c + 1, i0c + 4, i0c + 5
        const int i0c = 2 * half;
        const uint4* src = reinterpret_cast<const uint4*>(p.q + (size_t)(it.t0 + (live ? pos : 0)) * qd + head * 64);
        c[0] = live ? __ldg(src + i0c) : make_uint4(0, 0, 0, 0);
        c[1] = live ? __ldg(src + i0c + 1) : make_uint4(0, 0, 0, 0);
        c[2] = live ? __ldg(src + i0c + 4) : make_uint4(0, 0, 0, 0);
        c[3] = live ? __ldg(src + i0c + 5) : make_uint4(0, 0, 0, 0);
        if (live) {
          const float4* rt = reinterpret_cast<const float4*>(p.rope + (size_t)pos * 32);
#pragma unroll
          for (int i = 0; i < 2; ++i) {          // chunk i0c + i holds dims 8 (i0c + i) .., its partner the same + 32
            uint32_t* lo = reinterpret_cast<uint32_t*>(&c[i]);
            uint32_t* hi = reinterpret_cast<uint32_t*>(&c[i + 2]);
#pragma unroll
            for (int w = 0; w < 4; ++w) {        // word w: two consecutive dims
              const float4 cs = __ldg(rt + (8 * (i0c + i) + 2 * w) / 2);   // (cos, sin) of those two dims
              const float a0 = bf16_lo(lo[w]), a1 = bf16_hi(lo[w]), b0 = bf16_lo(hi[w]), b1 = bf16_hi(hi[w]);
              lo[w] = pack_bf16(a0 * cs.x - b0 * cs.y, a1 * cs.z - b1 * cs.w);
              hi[w] = pack_bf16(b0 * cs.x + a0 * cs.y, b1 * cs.z + a1 * cs.w);
            }
          }
        }
        uint8_t* qrow = base_ptr + (sQ - base);
        *reinterpret_cast<uint4*>(qrow + at_swz(row, i0c)) = c[0];
        *reinterpret_cast<uint4*>(qrow + at_swz(row, i0c + 1)) = c[1];
        *reinterpret_cast<uint4*>(qrow + at_swz(row, i0c + 4)) = c[2];
        *reinterpret_cast<uint4*>(qrow + at_swz(row, i0c + 5)) = c[3];
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(qready);
      }
      const int lim = it.t0 + pos;               // last visible key, batch coordinates
      // ---- pass 1: row maximum of the raw scores (the scale is positive: it commutes with the maximum)
      float m = -INFINITY;
      for (int j = 0; j < it.n_tiles && ok; ++j) {
        const uint32_t b = sq & 1u, bph = (sq >> 1) & 1u;
        if (!(ok = mbar_wait(sready + 8 * b, bph, abort_flag, p.status, 39))) break;
        tc_fence_after();
        const int key0 = it.a0 + j * kAtKeys + half * 32;
        uint32_t v[32];
        tmem_ld32(tmem + lane_addr + b * 64 + half * 32, v);
        tmem_ld_wait();
        if (key0 >= it.t0 && key0 + 31 <= lim) {   // every key of this half tile is visible to this row
#pragma unroll
          for (int c = 0; c < 32; ++c) m = fmaxf(m, __uint_as_float(v[c]));
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (key0 + c >= it.t0 && key0 + c <= lim) m = fmaxf(m, __uint_as_float(v[c]));
        }
        tc_fence_before();
        mbar_arrive(sfree + 8 * b);
        ++sq;
      }
      xm[half * 128 + row] = m;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      m = fmaxf(m, xm[(half ^ 1) * 128 + row]);
      const float mb = (m == -INFINITY) ? 0.f : m * p.scale_log2;
      // ---- pass 2: p = 2^(s - max), row sum in fp32, P tile as bf16 operand
      float l = 0.f;
      for (int j = 0; j < it.n_tiles && ok; ++j) {
        const uint32_t b = sq & 1u, bph = (sq >> 1) & 1u, pb = pq & 1u, pph = (pq >> 1) & 1u;
        if (!(ok = mbar_wait(sready + 8 * b, bph, abort_flag, p.status, 40))) break;
        if (!(ok = mbar_wait(pfree + 8 * pb, pph ^ 1u, abort_flag, p.status, 41))) break;
        tc_fence_after();
        const int key0 = it.a0 + j * kAtKeys + half * 32;
        uint8_t* prow = base_ptr + (sP - base) + pb * kAtTile;
        uint32_t v[32];
        tmem_ld32(tmem + lane_addr + b * 64 + half * 32, v);
        tmem_ld_wait();
        uint32_t w[16];
        if (key0 >= it.t0 && key0 + 31 <= lim) {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(v[c]), p.scale_log2, -mb));
            const float p1 = fast_exp2(fmaf(__uint_as_float(v[c + 1]), p.scale_log2, -mb));
            l += p0 + p1;
            w[c >> 1] = pack_bf16(p0, p1);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const int key = key0 + c;
            const float p0 = (key >= it.t0 && key <= lim) ? fast_exp2(fmaf(__uint_as_float(v[c]), p.scale_log2, -mb)) : 0.f;
            const float p1 = (key + 1 >= it.t0 && key + 1 <= lim) ? fast_exp2(fmaf(__uint_as_float(v[c + 1]), p.scale_log2, -mb)) : 0.f;
            l += p0 + p1;
            w[c >> 1] = pack_bf16(p0, p1);
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)             // chunks 4 half .. 4 half + 3 of this row
          *reinterpret_cast<uint4*>(prow + at_swz(row, 4 * half + i)) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        tc_fence_before();
        mbar_arrive(sfree + 8 * b);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(pready + 8 * pb);
        ++sq; ++pq;
      }
      xl[half * 128 + row] = l;
      if (!ok) *sm_fail = 1;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (*sm_fail) break;                       // the same for all 256 threads
      l += xl[(half ^ 1) * 128 + row];
      // ---- O / l -> out: this thread's 32 of the row's 64 dims
      if ((ok = mbar_wait(oready, nit & 1u, abort_flag, p.status, 42))) {
        tc_fence_after();
        const float inv = l > 0.f ? 1.f / l : 0.f;
        __nv_bfloat16* dst = p.out + (size_t)(it.t0 + (live ? pos : 0)) * qd + head * 64 + half * 32;
        uint32_t v[32];
        tmem_ld32(tmem + lane_addr + 128 + half * 32, v);
        tmem_ld_wait();
        if (live) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 o;
            o.x = pack_bf16(__uint_as_float(v[8 * i]) * inv, __uint_as_float(v[8 * i + 1]) * inv);
            o.y = pack_bf16(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv);
            o.z = pack_bf16(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv);
            o.w = pack_bf16(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + 8 * i) = o;
          }
        }
        tc_fence_before();
        mbar_arrive(ofree);
      }
      ++nit;
    }
  }
  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kAtTmemCols);
  }
}

bool attention_tc_supported(int n_heads, int n_kv_heads, int head_dim) {
  if (head_dim != 64 || n_kv_heads < 1 || (n_heads % n_kv_heads) != 0) return false;
  const int g = n_heads / n_kv_heads;
  return g >= 1 && g <= 128 && (128 % g) == 0;
}

// q [T, n_heads*64] (not rotated), k [T, n_kv*64] (rotated), v [T, n_kv*64] -> out [T, n_heads*64].
moin_status launch_attention_tc(HostState* hs, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                const int* cu, __nv_bfloat16* out, const float2* rope, int R,
                                int T, int max_seqlen, int n_heads, int n_kv_heads, float scale_log2,
                                cudaStream_t stream) {
  const int kvd = n_kv_heads * 64, g = n_heads / n_kv_heads;
  CUtensorMap mk, mv;
  moin_status st = make_map(&mk, k, (uint64_t)T, (uint64_t)kvd, kAtKeys);
  if (!st) st = make_map(&mv, v, (uint64_t)T, (uint64_t)kvd, kAtKeys);
  if (st) return st;
  AttParams p = {};
  p.q = q; p.out = out; p.cu = cu; p.rope = rope; p.R = R; p.n_heads = n_heads; p.n_kv = n_kv_heads; p.g = g;
  p.ppt = 128 / g; p.n_qb = (max_seqlen + p.ppt - 1) / p.ppt; p.scale_log2 = scale_log2; p.status = hs->status;
  cudaError_t e = ensure_smem_optin(OPTIN_ATTENTION, attention_tc_kernel, kAtSmem);
  if (e != cudaSuccess) return record_cuda(e);
  const long items = (long)p.n_qb * R * n_kv_heads;
  long grid = items < 2L * hs->n_sms ? items : 2L * hs->n_sms;
  if (grid < 1) grid = 1;
  attention_tc_kernel<<<(int)grid, kAtThreads, kAtSmem, stream>>>(mk, mv, p);
  return record_cuda(cudaGetLastError());
}

}  // namespace moin
