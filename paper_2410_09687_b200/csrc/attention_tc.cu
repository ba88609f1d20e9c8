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
// needs rescaling.  An item that sees at most 256 keys (four tiles: every item of a request of up to 256 tokens)
// keeps all of its scores in TMEM: S is computed once, both passes read it there, and O accumulates over the
// columns of the first score tile once that tile has been turned into P - one hand-over MMA -> softmax per item
// instead of two per tile.  Longer items stream: two score buffers, S recomputed in the second pass (the MMAs
// are a small part of the time; the exponentials are not).  Key tiles start at the request's first token (only the innermost coordinate of a TMA
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
constexpr int kAtKS = 4, kAtVS = 2;              // K: four stages (a resident item's whole key range, contiguous); V ring
constexpr int kAtCuMax = 1024;                   // request offsets kept in shared memory when there are at most this many
constexpr int kAtRopeBytes = 4096;               // (cos, sin) rows of an item's positions, when they fit (<= 16 positions)
constexpr int kAtSmem = kAtTile /*Q*/ + 2 * kAtTile /*P*/ + kAtKS * kAtKV + kAtVS * kAtKV + 1024 /*align*/ +
                        256 /*barriers*/ + 2048 /*row maxima and sums of the two half rows*/ + kAtCuMax * 4 + kAtRopeBytes;
constexpr int kAtTmemCols = 256;                 // streaming items: S0 [0,64)  S1 [64,128)  O [128,192)
constexpr int kAtResident = 4;                   // resident items: S_j [64 j, 64 j + 64), j < 4; O over S_0

struct AttParams {
  const __nv_bfloat16* q;      // [T, n_heads * 64], not rotated
  __nv_bfloat16* out;          // [T, n_heads * 64]
  const int* cu;               // [R + 1]
  const float2* rope;          // [max_seqlen, 32] (cos, sin)
  int R, n_heads, n_kv, g, ppt, n_qb;   // g heads per kv head, ppt = 128 / g positions per tile, n_qb query blocks
  int max_pos;                 // rows of the rope table
  int rope_smem, cu_smem;      // an item's rope rows / the request offsets are staged in shared memory
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
// the same with N = 64 n (n key tiles side by side in one product)
__device__ __forceinline__ uint32_t at_idesc_n(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((64 * n) >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// the same with B MN-major (V tile: one 128-byte row per key, the 64 output dims contiguous); a 16-key step of
// such a tile is two 8-key groups = 2048 bytes further on
constexpr uint32_t kAtIdescPV = kAtIdesc | (1u << 16);
constexpr uint64_t kAtVStep = 2048 >> 4;

__device__ __forceinline__ float fast_exp2(float x) {   // arguments are <= 0 here: 2^x in (0, 1]
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two-lane fp32 arithmetic (one instruction for a pair of scores) and the three-input maximum: the softmax threads
// are bound by the number of instructions they issue, not by any one pipe.
__device__ __forceinline__ uint64_t pair_f32(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpair_f32(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// byte offset of 16-byte chunk c of row r in a swizzled [rows x 128 bytes] tile
__device__ __forceinline__ uint32_t at_swz(int r, int c) {
  return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4));
}

struct AttItem { int req, kvh, q0, t0, L, a0, n_tiles; bool on; };
__device__ __forceinline__ AttItem at_item(const AttParams& p, const int* cu, int idx) {
  AttItem it;
  const int per_qb = p.R * p.n_kv;
  const int qb = p.n_qb - 1 - idx / per_qb;     // longest blocks first
  const int rem = idx % per_qb;
  it.req = rem / p.n_kv;
  it.kvh = rem % p.n_kv;
  it.q0 = qb * p.ppt;
  it.t0 = cu[it.req];
  it.L = cu[it.req + 1] - it.t0;
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
                 qready = bars + 208, sall = bars + 232, rfull = bars + 240, rempty = bars + 248;
  int* cu_s = reinterpret_cast<int*>(bar_ptr + 256 + 2048);
  const uint32_t sRope = bars + 256 + 2048 + kAtCuMax * 4;
  const int* cu = p.cu_smem ? cu_s : p.cu;
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
    mbar_init(sall, 1);
    mbar_init(rfull, 1);
    mbar_init(rempty, 256);
    *abort_flag = 0;
    *sm_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kAtTmemCols);
    tmem_relinquish();
  }
  if (p.cu_smem)
    for (int i = threadIdx.x; i <= p.R; i += kAtThreads) cu_s[i] = __ldg(p.cu + i);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_items = p.n_qb * p.R * p.n_kv;
  auto next_item = [&](int& i, AttItem& out) -> bool {   // the next item of this CTA that has any query row
    for (i += gridDim.x; i < n_items; i += gridDim.x) {
      out = at_item(p, cu, i);
      if (out.on) return true;
    }
    return false;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    // K stages and their barriers are addressed by stage, each with its own phase bit (keph: next "empty" phase to
    // wait for), because the two kinds of item use them differently: a resident item puts its tiles into stages
    // 0 .. n - 1 (one contiguous operand, one "full" barrier), a streaming item goes round the ring from kpos.
    if (lane == 0) {
      uint32_t keph = 0, kpos = 0, vq = 0, rq = 0;
      bool ok = true;
      int idx = (int)blockIdx.x - (int)gridDim.x;
      AttItem it;
      bool have = next_item(idx, it);
      auto load_rope = [&](const AttItem& n) -> bool {   // (cos, sin) rows of the item's positions, for its Q staging
        if (!p.rope_smem) return true;
        if (!mbar_wait(rempty, (rq & 1u) ^ 1u, abort_flag, p.status, 44)) return false;
        const uint32_t bytes = (uint32_t)min(p.ppt, p.max_pos - n.q0) * 256u;
        mbar_expect_tx(rfull, bytes);
        bulk_load_1d(sRope, p.rope + (size_t)n.q0 * 32, bytes, rfull);
        ++rq;
        return true;
      };
      if (have) ok = load_rope(it);
      while (have && ok) {
        AttItem nx;
        int nidx = idx;
        const bool have_nx = next_item(nidx, nx);
        auto k_free = [&](uint32_t s) -> bool {
          const bool r = mbar_wait(kempty + 8 * s, ((keph >> s) & 1u) ^ 1u, abort_flag, p.status, 31);
          keph ^= 1u << s;
          return r;
        };
        auto load_k = [&](int j) -> bool {               // streaming: next stage of the ring
          const uint32_t s = kpos;
          if (!k_free(s)) return false;
          mbar_expect_tx(kfull + 8 * s, kAtKV);
          tma_load_2d(sK + s * kAtKV, &tmK, kfull + 8 * s, it.kvh * 64, it.a0 + j * kAtKeys);
          kpos = (kpos + 1) % kAtKS;
          return true;
        };
        auto load_v = [&](int j) -> bool {
          const uint32_t s = vq % kAtVS, ph = (vq / kAtVS) & 1u;
          if (!mbar_wait(vempty + 8 * s, ph ^ 1u, abort_flag, p.status, 32)) return false;
          mbar_expect_tx(vfull + 8 * s, kAtKV);
          tma_load_2d(sV + s * kAtKV, &tmV, vfull + 8 * s, it.kvh * 64, it.a0 + j * kAtKeys);
          ++vq;
          return true;
        };
        if (it.n_tiles <= kAtResident) {   // resident item: its K tiles side by side, completion on the first barrier
          for (int j = 0; j < it.n_tiles && ok; ++j) ok = k_free((uint32_t)j);
          if (!ok) break;
          mbar_expect_tx(kfull, (uint32_t)it.n_tiles * kAtKV);
          for (int j = 0; j < it.n_tiles; ++j) tma_load_2d(sK + j * kAtKV, &tmK, kfull, it.kvh * 64, it.a0 + j * kAtKeys);
          kpos = 0;
          if (have_nx) ok = load_rope(nx);   // wanted while this item's scores are being turned into P
          for (int j = 0; j < it.n_tiles && ok; ++j) ok = load_v(j);
        } else {                           // streaming item: K for the maxima, then K and V side by side
          for (int j = 0; j < it.n_tiles && ok; ++j) ok = load_k(j);
          if (have_nx && ok) ok = load_rope(nx);
          for (int j = 0; j < it.n_tiles && ok; ++j) ok = load_k(j) && load_v(j);
        }
        it = nx;
        idx = nidx;
        have = have_nx;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t kfph = 0, kpos = 0, vq = 0, sq = 0, pq = 0, nit = 0;   // kfph: per-stage phase bits of the "full" barriers
      bool ok = true;
      const uint64_t dq = at_sdesc(sQ);
      auto issue_s = [&]() -> bool {   // S[sq & 1] = Q K^T with the next K stage of the ring
        const uint32_t b = sq & 1u, bph = (sq >> 1) & 1u, s = kpos, ph = (kfph >> s) & 1u;
        if (!mbar_wait(sfree + 8 * b, bph ^ 1u, abort_flag, p.status, 33)) return false;
        if (!mbar_wait(kfull + 8 * s, ph, abort_flag, p.status, 34)) return false;
        kfph ^= 1u << s;
        kpos = (kpos + 1) % kAtKS;
        tc_fence_after();
        const uint64_t dk = at_sdesc(sK + s * kAtKV);
#pragma unroll
        for (int k = 0; k < 4; ++k) tc_mma_bf16(tmem + b * 64, dq + (uint64_t)(2 * k), dk + (uint64_t)(2 * k), kAtIdesc, k > 0 ? 1u : 0u);
        tc_commit(kempty + 8 * s);
        tc_commit(sready + 8 * b);
        ++sq;
        return true;
      };
      for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
        const AttItem it = at_item(p, cu, idx);
        if (!it.on) continue;
        // the accumulator columns are free once the O of the item before has been read (all of its score reads
        // come earlier); then the rotated Q tile of this item
        if (!(ok = mbar_wait(ofree, (nit & 1u) ^ 1u, abort_flag, p.status, 36))) break;
        if (!(ok = mbar_wait(qready, nit & 1u, abort_flag, p.status, 35))) break;
        tc_fence_after();
        auto issue_pv = [&](uint32_t o_col, bool first) -> bool {   // O (+)= P V with the next P buffer and V stage
          const uint32_t b = pq & 1u, bph = (pq >> 1) & 1u, s = vq % kAtVS, ph = (vq / kAtVS) & 1u;
          if (!mbar_wait(pready + 8 * b, bph, abort_flag, p.status, 37)) return false;
          if (!mbar_wait(vfull + 8 * s, ph, abort_flag, p.status, 38)) return false;
          tc_fence_after();
          const uint64_t dp = at_sdesc(sP + b * kAtTile), dv = at_sdesc(sV + s * kAtKV);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma_bf16(tmem + o_col, dp + (uint64_t)(2 * k), dv + kAtVStep * k, kAtIdescPV, (!first || k > 0) ? 1u : 0u);
          tc_commit(vempty + 8 * s);
          tc_commit(pfree + 8 * b);
          ++pq; ++vq;
          return true;
        };
        if (it.n_tiles <= kAtResident) {
          // resident item: the scores against all of its keys in one product per 16 dims (the key tiles lie side
          // by side in stages 0 .. n - 1), one hand-over; then the second products as the P tiles arrive
          if (!(ok = mbar_wait(kfull, kfph & 1u, abort_flag, p.status, 34))) break;
          kfph ^= 1u;
          kpos = 0;
          tc_fence_after();
          const uint64_t dk = at_sdesc(sK);
          const uint32_t idn = at_idesc_n(it.n_tiles);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma_bf16(tmem, dq + (uint64_t)(2 * k), dk + (uint64_t)(2 * k), idn, k > 0 ? 1u : 0u);
          for (int j = 0; j < it.n_tiles; ++j) tc_commit(kempty + 8 * j);
          tc_commit(sall);
          for (int j = 0; j < it.n_tiles && ok; ++j) ok = issue_pv(0, j == 0);
        } else {
          // streaming item, pass 1: scores only (the softmax warps take the row maxima)
          for (int j = 0; j < it.n_tiles && ok; ++j) ok = issue_s();
          if (!ok) break;
          // pass 2: scores again, then O += P V; the scores of tile j + 1 are issued before the product of tile j
          ok = issue_s();
          for (int j = 0; j < it.n_tiles && ok; ++j) {
            if (j + 1 < it.n_tiles && !(ok = issue_s())) break;
            ok = issue_pv(128, j == 0);
          }
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
    uint32_t sq = 0, pq = 0, nit = 0, nres = 0;
    // Q rows: load, rotate (pairs (d, d + 32), position inside the request), lay down swizzled.  This thread takes
    // 16-byte chunks 2 half, 2 half + 1 of its row and their rotation partners 4 further on.  The loads of the
    // NEXT item's rows are issued while this item's scores are on their way and staged as soon as the Q tile is free
    // (all score MMAs of this item complete), so that the MMA warp finds the tile ready when the accumulators are.
    const int i0c = 2 * half;
    const int row_pos = row / p.g, row_head = row % p.g;   // position inside the block and head inside the group
    auto q_load = [&](const AttItem& n, uint4 (&c)[4]) {
      const int npos = n.q0 + row_pos, nhead = n.kvh * p.g + row_head;
      const bool nlive = npos < n.L;
      const uint4* src = reinterpret_cast<const uint4*>(p.q + (size_t)(n.t0 + (nlive ? npos : 0)) * qd + nhead * 64);
      c[0] = nlive ? __ldg(src + i0c) : make_uint4(0, 0, 0, 0);
      c[1] = nlive ? __ldg(src + i0c + 1) : make_uint4(0, 0, 0, 0);
      c[2] = nlive ? __ldg(src + i0c + 4) : make_uint4(0, 0, 0, 0);
      c[3] = nlive ? __ldg(src + i0c + 5) : make_uint4(0, 0, 0, 0);
    };
    uint32_t rq = 0;
    bool ok = true;
    auto q_stage = [&](const AttItem& n, uint4 (&c)[4]) {
      const int npos = n.q0 + row_pos;
      // the (cos, sin) rows of the item's positions: staged by the producer when they fit, else from the table
      if (p.rope_smem) ok = mbar_wait(rfull, rq & 1u, abort_flag, p.status, 45) && ok;
      if (npos < n.L) {
        const float4* rt = p.rope_smem ? reinterpret_cast<const float4*>(base_ptr + (sRope - base) + row_pos * 256)
                                       : reinterpret_cast<const float4*>(p.rope + (size_t)npos * 32);
#pragma unroll
        for (int i = 0; i < 2; ++i) {          // chunk i0c + i holds dims 8 (i0c + i) .., its partner the same + 32
          uint32_t* lo = reinterpret_cast<uint32_t*>(&c[i]);
          uint32_t* hi = reinterpret_cast<uint32_t*>(&c[i + 2]);
#pragma unroll
          for (int w = 0; w < 4; ++w) {        // word w: two consecutive dims
            const float4 cs = rt[(8 * (i0c + i) + 2 * w) / 2];   // (cos, sin) of those two dims
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
      if (p.rope_smem) {
        mbar_arrive(rempty);
        ++rq;
      }
    };
    int idx = (int)blockIdx.x - (int)gridDim.x;
    AttItem it;
    bool have = next_item(idx, it);
    if (have) {
      uint4 c[4];
      q_load(it, c);
      q_stage(it, c);
    }
    while (have) {
      AttItem nx;
      int nidx = idx;
      const bool have_nx = next_item(nidx, nx);
      const int pos = it.q0 + row_pos, head = it.kvh * p.g + row_head;
      const bool live = pos < it.L;
      uint4 cn[4];
      if (have_nx && it.n_tiles <= kAtResident) q_load(nx, cn);
      const bool resident = it.n_tiles <= kAtResident;
      // Scores come in half tiles of 32 keys, taken as two groups of 16.  Keys are counted from the request's first
      // token (kr); row `pos` sees kr <= pos.  A group is visible to every row of the item when it ends before the
      // item's first position, to none when it starts after the item's last one (both the same for all threads:
      // no exponentials are spent there), and is masked key by key otherwise.
      const int q_last = it.q0 + p.ppt - 1;
      auto tile_max = [&](const uint32_t (&v)[32], int kr0, float m) -> float {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int kr = kr0 + 16 * q;
          if (kr + 15 <= it.q0) {
#pragma unroll
            for (int c = 16 * q; c < 16 * q + 16; c += 2) m = max3(m, __uint_as_float(v[c]), __uint_as_float(v[c + 1]));
          } else if (kr <= q_last) {
#pragma unroll
            for (int c = 16 * q; c < 16 * q + 16; ++c)
              if (kr0 + c <= pos) m = fmaxf(m, __uint_as_float(v[c]));
          }
        }
        return m;
      };
      auto tile_p = [&](const uint32_t (&v)[32], int kr0, float mb, uint8_t* prow, float l) -> float {
        uint32_t w[16];
        const uint64_t scale2 = pair_f32(p.scale_log2, p.scale_log2), nmb2 = pair_f32(-mb, -mb);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int kr = kr0 + 16 * q;
          if (kr + 15 <= it.q0) {
            uint64_t l2 = pair_f32(l, 0.f);
#pragma unroll
            for (int c = 16 * q; c < 16 * q + 16; c += 2) {
              float x0, x1;
              unpair_f32(fma2(pair_f32(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), scale2, nmb2), x0, x1);
              const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
              l2 = add2(l2, pair_f32(p0, p1));
              w[c >> 1] = pack_bf16(p0, p1);
            }
            float la, lb;
            unpair_f32(l2, la, lb);
            l = la + lb;
          } else if (kr <= q_last) {
#pragma unroll
            for (int c = 16 * q; c < 16 * q + 16; c += 2) {
              const int k0 = kr0 + c;
              const float p0 = k0 <= pos ? fast_exp2(fmaf(__uint_as_float(v[c]), p.scale_log2, -mb)) : 0.f;
              const float p1 = k0 + 1 <= pos ? fast_exp2(fmaf(__uint_as_float(v[c + 1]), p.scale_log2, -mb)) : 0.f;
              l += p0 + p1;
              w[c >> 1] = pack_bf16(p0, p1);
            }
          } else {
#pragma unroll
            for (int c = 16 * q; c < 16 * q + 16; c += 2) w[c >> 1] = 0u;
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)               // chunks 4 half .. 4 half + 3 of this row
          *reinterpret_cast<uint4*>(prow + at_swz(row, 4 * half + i)) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        return l;
      };
      // the same for one group of 16 keys at a time (resident items: the TMEM read of the next group is in flight
      // while this one is worked on); two running maxima keep the dependent chain short
      auto group_max = [&](const uint32_t (&v)[16], int kr, float& m0, float& m1) {
        if (kr + 15 <= it.q0) {
#pragma unroll
          for (int c = 0; c < 16; c += 4) {
            m0 = max3(m0, __uint_as_float(v[c]), __uint_as_float(v[c + 1]));
            m1 = max3(m1, __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
          }
        } else if (kr <= q_last) {
#pragma unroll
          for (int c = 0; c < 16; ++c)
            if (kr + c <= pos) m0 = fmaxf(m0, __uint_as_float(v[c]));
        }
      };
      auto group_p = [&](const uint32_t (&v)[16], int kr, uint64_t scale2, uint64_t nmb2, float mb, uint32_t* w, float& l) {
        if (kr + 15 <= it.q0) {
          uint64_t l2 = pair_f32(l, 0.f);
#pragma unroll
          for (int c = 0; c < 16; c += 2) {
            float x0, x1;
            unpair_f32(fma2(pair_f32(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), scale2, nmb2), x0, x1);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            l2 = add2(l2, pair_f32(p0, p1));
            w[c >> 1] = pack_bf16(p0, p1);
          }
          float la, lb;
          unpair_f32(l2, la, lb);
          l = la + lb;
        } else if (kr <= q_last) {
#pragma unroll
          for (int c = 0; c < 16; c += 2) {
            const float p0 = kr + c <= pos ? fast_exp2(fmaf(__uint_as_float(v[c]), p.scale_log2, -mb)) : 0.f;
            const float p1 = kr + c + 1 <= pos ? fast_exp2(fmaf(__uint_as_float(v[c + 1]), p.scale_log2, -mb)) : 0.f;
            l += p0 + p1;
            w[c >> 1] = pack_bf16(p0, p1);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 8; ++c) w[c] = 0u;
        }
      };
      // group g of this thread: tile g / 2, columns half * 32 + 16 (g % 2) of it
      const uint32_t tcol = tmem + lane_addr + half * 32;
      auto g_col = [&](int g) -> uint32_t { return tcol + (uint32_t)((g >> 1) * 64 + (g & 1) * 16); };
      auto g_kr = [&](int g) -> int { return (g >> 1) * kAtKeys + half * 32 + (g & 1) * 16; };
      // ---- pass 1: row maximum of the raw scores (the scale is positive: it commutes with the maximum)
      float m = -INFINITY;
      if (resident) {
        if ((ok = ok && mbar_wait(sall, nres & 1u, abort_flag, p.status, 43))) {
          tc_fence_after();
          float m1 = -INFINITY;
          uint32_t va[16], vb[16];
          const int G = 2 * it.n_tiles;
          tmem_ld16(g_col(0), va);
          for (int g = 0; g < G; g += 2) {
            tmem_ld_wait();
            tmem_ld16(g_col(g + 1), vb);
            group_max(va, g_kr(g), m, m1);
            tmem_ld_wait();
            if (g + 2 < G) tmem_ld16(g_col(g + 2), va);
            group_max(vb, g_kr(g + 1), m, m1);
          }
          m = fmaxf(m, m1);
        }
        ++nres;
      } else {
        for (int j = 0; j < it.n_tiles && ok; ++j) {
          const uint32_t b = sq & 1u, bph = (sq >> 1) & 1u;
          if (!(ok = mbar_wait(sready + 8 * b, bph, abort_flag, p.status, 39))) break;
          tc_fence_after();
          uint32_t v[32];
          tmem_ld32(tmem + lane_addr + b * 64 + half * 32, v);
          tmem_ld_wait();
          m = tile_max(v, j * kAtKeys + half * 32, m);
          tc_fence_before();
          mbar_arrive(sfree + 8 * b);
          ++sq;
        }
      }
      xm[half * 128 + row] = m;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      m = fmaxf(m, xm[(half ^ 1) * 128 + row]);
      const float mb = (m == -INFINITY) ? 0.f : m * p.scale_log2;
      if (have_nx && resident) q_stage(nx, cn);   // every score MMA of this item is complete: the Q tile is free
      // ---- pass 2: p = 2^(s - max), row sum in fp32, P tile as bf16 operand
      float l = 0.f;
      if (resident && ok) {
        const uint64_t scale2 = pair_f32(p.scale_log2, p.scale_log2), nmb2 = pair_f32(-mb, -mb);
        uint32_t va[16], vb[16];
        tmem_ld16(g_col(0), va);
        for (int j = 0; j < it.n_tiles; ++j) {
          const uint32_t pb = pq & 1u, pph = (pq >> 1) & 1u;
          uint32_t w[16];
          tmem_ld_wait();
          tmem_ld16(g_col(2 * j + 1), vb);
          group_p(va, g_kr(2 * j), scale2, nmb2, mb, w, l);
          tmem_ld_wait();
          if (j + 1 < it.n_tiles) tmem_ld16(g_col(2 * j + 2), va);
          group_p(vb, g_kr(2 * j + 1), scale2, nmb2, mb, w + 8, l);
          if (!(ok = mbar_wait(pfree + 8 * pb, pph ^ 1u, abort_flag, p.status, 41))) break;
          uint8_t* prow = base_ptr + (sP - base) + pb * kAtTile;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<uint4*>(prow + at_swz(row, 4 * half + i)) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
          tc_fence_before();                      // this tile's scores are read: the O columns over them may be written
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          mbar_arrive(pready + 8 * pb);
          ++pq;
        }
        if (!ok) tmem_ld_wait();
      }
      for (int j = 0; j < it.n_tiles && ok && !resident; ++j) {
        const uint32_t b = sq & 1u, bph = (sq >> 1) & 1u, pb = pq & 1u, pph = (pq >> 1) & 1u;
        if (!resident && !(ok = mbar_wait(sready + 8 * b, bph, abort_flag, p.status, 40))) break;
        if (!(ok = mbar_wait(pfree + 8 * pb, pph ^ 1u, abort_flag, p.status, 41))) break;
        tc_fence_after();
        uint32_t v[32];
        tmem_ld32(tmem + lane_addr + (resident ? j : (int)b) * 64 + half * 32, v);
        tmem_ld_wait();
        l = tile_p(v, j * kAtKeys + half * 32, mb, base_ptr + (sP - base) + pb * kAtTile, l);
        tc_fence_before();                        // the scores are read: the buffer (resident: the O columns) may be written
        if (!resident) { mbar_arrive(sfree + 8 * b); ++sq; }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(pready + 8 * pb);
        ++pq;
      }
      if (have_nx && !resident) {                 // streaming item: Q was an operand up to the last score tile
        q_load(nx, cn);
        q_stage(nx, cn);
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
        tmem_ld32(tmem + lane_addr + (resident ? 0 : 128) + half * 32, v);
        tmem_ld_wait();
        tc_fence_before();                        // O is in registers: the accumulator columns may be written again
        mbar_arrive(ofree);
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
      }
      ++nit;
      it = nx;
      idx = nidx;
      have = have_nx;
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
  p.max_pos = max_seqlen;
  p.rope_smem = p.ppt * 256 <= kAtRopeBytes;
  p.cu_smem = R + 1 <= kAtCuMax;
  cudaError_t e = ensure_smem_optin(OPTIN_ATTENTION, attention_tc_kernel, kAtSmem);
  if (e != cudaSuccess) return record_cuda(e);
  const long items = (long)p.n_qb * R * n_kv_heads;
  long grid = items < 2L * hs->n_sms ? items : 2L * hs->n_sms;
  if (grid < 1) grid = 1;
  attention_tc_kernel<<<(int)grid, kAtThreads, kAtSmem, stream>>>(mk, mv, p);
  return record_cuda(cudaGetLastError());
}

}  // namespace moin
