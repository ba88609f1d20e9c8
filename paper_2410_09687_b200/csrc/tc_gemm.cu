// tcgen05 / TMEM / TMA GEMM family for sm_100a.
//
// One persistent, warp-specialised kernel computes D[128 x BN] tiles of  A[M,K] * B[N,K]^T
// (both operands K-major bf16, fp32 accumulation in tensor memory):
//   warp 0     TMA producer: 128B-swizzled [128 x 64] A boxes and [BN x 64] B boxes into a
//              multi-stage shared-memory ring, completion on mbarriers
//   warp 1     allocates TMEM, issues tcgen05.mma (one thread), commits stage release and
//              accumulator-ready barriers
//   warps 2-9  epilogue, two warps per TMEM lane quarter (half of the tile's columns each): tcgen05.ld of the
//              accumulator (TMEM lane = tile row), then one of
//              EPI_STORE   y = bf16(acc) (+ optional fp32 copy)
//              EPI_ROUTER  running (max, argmax) of acc * inv_norm[col], merged across tiles with a
//                          64-bit atomicMax on (orderable(sim) << 32 | ~col): order independent,
//                          lowest index wins ties
//              EPI_SHRINK  scale * acc for the LoRA rank columns, stored as bf16 hi + lo parts
// Two accumulator buffers in TMEM let the epilogue of tile i overlap the MMAs of tile i+1.
//
// Row tiles come either from a regular grid over M or from a batch plan (runs of tokens with
// one expert, <= 128 rows).  With a plan, EPI_STORE appends two extra K blocks per tile taken
// from hi/lo[rows, r] and B_e[d_out, r] of the tile's adapter: y = [x | hi(s h) | lo(s h)] [W ; B_e ; B_e]^T,
// so the low-rank term is added inside the accumulator (to ~fp32 accuracy) and y is written once.
// Every wait on an mbarrier is bounded; on expiry the kernel raises the status flag and returns.
#include <cuda.h>

#include "tc_gemm.cuh"
#include "ptx.cuh"

namespace moin {

constexpr int kBM = 128, kBK = 64;
constexpr int kTcThreads = 320;      // producer warp, MMA warp, eight epilogue warps
constexpr int kTcThreadsLean = 192;  // four epilogue warps and no output staging: the launch that runs beside the
                                     // adapter streams at decode size and should leave them registers and shared memory
enum { EPI_STORE = 0, EPI_ROUTER = 1, EPI_SHRINK = 2, EPI_ROUTER2 = 3 };   // ROUTER2: best and runner-up

constexpr int kMaxShrinkJobs = 3;
struct TcParams {
  int M, N, K;                 // problem: rows, output columns, reduction length
  // plan tiles (nullptr -> regular grid over M)
  const int* header;
  const int* tile_row0;
  const int* tile_rows;
  const int* tile_expert;
  const int* slot_of_expert;
  int tail_r;                  // EPI_STORE with plan: LoRA rank of the appended K block (0 = none)
  int rows_per_slot;           // rows of the B-side pool tensor per adapter slot (d_out, or r for EPI_SHRINK)
  int b_box_rows;              // rows of the B-side TMA box when it is shorter than the tile's BN (0 = BN); the
                               // rest of the stage's B region keeps stale bytes, whose columns nobody stores
  __nv_bfloat16* y;            // EPI_STORE / EPI_SHRINK output, leading dimension ldy
  __nv_bfloat16* y_lo;         // EPI_SHRINK: low part, value - bf16(value), same layout as y
  float* y0;                   // EPI_STORE: optional fp32 copy
  int tma_store;               // EPI_STORE: full 32-row groups of a tile leave through shared memory and tiled stores
  int ldy;
  float scale;                 // EPI_SHRINK
  // EPI_SHRINK over several projections that share the plan, K and the rank (n_jobs in 1..kMaxShrinkJobs):
  // tile index = row tile * n_jobs + job; job j reads x through the j-th A-side map and its pool through
  // the j-th B-side map, looks its slot up in slot_tabs[j] and writes ys[j] / ys_lo[j].  n_jobs = 0: one job
  // described by slot_of_expert / y / y_lo.
  int n_jobs;
  // ... or, when they also share x and their ranks fit one tile side by side (n_stack * stack_r <= BN): ONE pass
  // over x, the adapters' rows stacked in the B operand (job j at rows j * stack_r), N = n_stack * stack_r
  // accumulator columns, column group j stored to ys[j] / ys_lo[j].  n_stack > 1 implies n_jobs = 1.
  int n_stack, stack_r;
  const int* slot_tabs[3];
  __nv_bfloat16* ys[3];
  __nv_bfloat16* ys_lo[3];
  // per-slot adapter rank (nullable: the stored rank) and the function applied to x A^T (MOIN_ACT_*):
  const int* rank_tabs[3];     // EPI_SHRINK: table of job j (n_jobs = 0: rank_tabs[0])
  const int* slot_rank;        // EPI_STORE with plan: table of the projection's pool
  int act;                     // EPI_SHRINK
  const float* inv_norm;       // EPI_ROUTER
  unsigned long long* keys;    // EPI_ROUTER / EPI_ROUTER2: best (similarity, index) key per row
  unsigned long long* keys2;   // EPI_ROUTER2: runner-up key per row
  DeviceStatus* status;
};

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart (SBO), leading-dimension offset field 1 (unused by swizzled
// K-major layouts), descriptor version 1, base offset 0 (tiles are 1024-byte aligned).
__device__ __forceinline__ uint64_t make_sdesc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor: D fp32, A/B bf16, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t make_idesc(int bn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

__device__ __forceinline__ uint32_t orderable(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int BN> struct TcCfg {
  static constexpr int kStageBytes = (kBM + BN) * kBK * 2;
  static constexpr int kStages = (200 * 1024) / kStageBytes > 8 ? 8 : (200 * 1024) / kStageBytes;
  static constexpr int kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;   // power of two for BN in {64,128,256}
  // output staging of the store epilogue: per epilogue warp one [32 rows x 64 columns] bf16 buffer
  static constexpr int kOutBytes = 8 * 32 * 128;
  static constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 1024 /*align*/ + 1024 /*barriers*/ + kOutBytes;
};

template <int BN, int EPI>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmA3,
               const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmB3,
               const __grid_constant__ CUtensorMap tmY, const TcParams p) {
  using Cfg = TcCfg<BN>;
  constexpr int S = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  uint8_t* bar_ptr = smem_raw + (tiles_base - raw) + (size_t)S * Cfg::kStageBytes;
  const uint32_t bars = tiles_base + (uint32_t)S * Cfg::kStageBytes;
  const uint32_t full0 = bars, empty0 = bars + 8 * S, tfull0 = bars + 16 * S, tempty0 = bars + 16 * S + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 16 * S + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 16 * S + 40);
  const uint32_t out0 = bars + 1024;   // output staging (1024-byte aligned: the swizzle is a function of the address)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull0 + 8 * a, 1);
      mbar_init(tempty0 + 8 * a, blockDim.x - 64);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const bool planned = p.header != nullptr;
  const int tiles_n = (p.N + BN - 1) / BN;
  const int tiles_m = planned ? p.header[PH_NTILES] : (p.M + kBM - 1) / kBM;
  const int n_jobs = (EPI == EPI_SHRINK && p.n_jobs > 1) ? p.n_jobs : 1;   // EPI_SHRINK: tiles_n == 1
  const int total = tiles_m * tiles_n * n_jobs;
  const int nkb_main = (p.K + kBK - 1) / kBK;

  int job = 0;   // projection of the current tile (EPI_SHRINK with several jobs), set by tile_info
  int r_use = (EPI == EPI_SHRINK) ? p.N : p.tail_r;   // rank of the current tile's adapter, set by tile_info
  const bool stacked = (EPI == EPI_SHRINK) && p.n_stack > 1;
  int st_slot[kMaxShrinkJobs] = {-1, -1, -1}, st_ruse[kMaxShrinkJobs] = {0, 0, 0};   // stacked: per projection
  auto tile_info = [&](int tile, int& row0, int& rows, int& n0, int& slot) {
    int tm = tile / tiles_n;
    n0 = (tile - tm * tiles_n) * BN;
    if (EPI == EPI_SHRINK && n_jobs > 1) {   // the projections of one row tile side by side: its x tile is read once
      job = tm % n_jobs;                     // from HBM and found in L2 by the CTAs next door
      tm /= n_jobs;
    }
    slot = -1;
    if (planned) {
      row0 = p.tile_row0[tm];
      rows = p.tile_rows[tm];
      const int e = p.tile_expert[tm];
      const int* tab = p.slot_of_expert;
      if (EPI == EPI_SHRINK && p.n_jobs > 0) tab = (job == 0) ? p.slot_tabs[0] : (job == 1) ? p.slot_tabs[1] : p.slot_tabs[2];
      if (e >= 0 && tab) slot = tab[e];
      if (stacked) {
#pragma unroll
        for (int j = 0; j < kMaxShrinkJobs; ++j) {
          st_slot[j] = (j < p.n_stack && e >= 0) ? p.slot_tabs[j][e] : -1;
          st_ruse[j] = (st_slot[j] >= 0 && p.rank_tabs[j]) ? min(p.rank_tabs[j][st_slot[j]], p.stack_r) : p.stack_r;
        }
        slot = st_slot[0];
      } else if (EPI == EPI_SHRINK || EPI == EPI_STORE) {
        const int r_full = (EPI == EPI_SHRINK) ? p.N : p.tail_r;
        const int* rt = (EPI == EPI_STORE) ? p.slot_rank
                                           : (job == 0 ? p.rank_tabs[0] : job == 1 ? p.rank_tabs[1] : p.rank_tabs[2]);
        r_use = (slot >= 0 && rt) ? min(rt[slot], r_full) : r_full;
      }
    } else {
      row0 = tm * kBM;
      rows = min(kBM, p.M - row0);
    }
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
        int row0, rows, n0, slot;
        tile_info(tile, row0, rows, n0, slot);
        const bool tail = (EPI == EPI_STORE) && planned && p.tail_r > 0 && slot >= 0;
        const int nrb = (p.tail_r + kBK - 1) / kBK;   // 64-wide blocks of the rank
        const int nkb = nkb_main + (tail ? 2 * nrb : 0);   // tail: [hi(s h) | lo(s h)] x [B_e ; B_e], nrb blocks each
        const int brow = (EPI == EPI_SHRINK) ? (slot >= 0 ? slot : 0) * p.rows_per_slot : n0;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const uint32_t s = it % S, ph = (it / S) & 1u;
          if (!(ok = mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag, p.status, 1))) break;
          const uint32_t sa = tiles_base + s * Cfg::kStageBytes, sb = sa + kBM * kBK * 2;
          const uint32_t b_rows = stacked ? (uint32_t)(p.n_stack * p.stack_r)
                                          : (kb < nkb_main && p.b_box_rows > 0) ? (uint32_t)p.b_box_rows : (uint32_t)BN;
          mbar_expect_tx(full0 + 8 * s, (kBM + b_rows) * kBK * 2);
          if (stacked) {
            tma_load_2d(sa, &tmA, full0 + 8 * s, kb * kBK, row0);
#pragma unroll
            for (int j = 0; j < kMaxShrinkJobs; ++j)
              if (j < p.n_stack)   // (a projection without this adapter loads slot 0: its columns are not stored)
                tma_load_2d(sb + (uint32_t)(j * p.stack_r) * kBK * 2, j == 0 ? &tmB : j == 1 ? &tmB2 : &tmB3, full0 + 8 * s,
                            kb * kBK, (st_slot[j] >= 0 ? st_slot[j] : 0) * p.stack_r);
          } else if (kb < nkb_main) {
            const CUtensorMap* ma = &tmA;
            const CUtensorMap* mb = &tmB;
            if (EPI == EPI_SHRINK && job > 0) {
              ma = (job == 1) ? &tmA2 : &tmA3;
              mb = (job == 1) ? &tmB2 : &tmB3;
            }
            tma_load_2d(sa, ma, full0 + 8 * s, kb * kBK, row0);
            tma_load_2d(sb, mb, full0 + 8 * s, kb * kBK, brow);
          } else {
            const int j = kb - nkb_main, rb = (j >= nrb) ? j - nrb : j;   // hi blocks first, then lo blocks
            tma_load_2d(sa, j < nrb ? &tmA2 : &tmA3, full0 + 8 * s, rb * kBK, row0);
            tma_load_2d(sb, &tmB2, full0 + 8 * s, rb * kBK, slot * p.rows_per_slot + n0);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BN);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++lt) {
        int row0, rows, n0, slot;
        tile_info(tile, row0, rows, n0, slot);
        const bool tail = (EPI == EPI_STORE) && planned && p.tail_r > 0 && slot >= 0;
        const int nrb = (p.tail_r + kBK - 1) / kBK;
        const int nkb = nkb_main + (tail ? 2 * nrb : 0);
        const uint32_t acc = lt & 1u, aph = (lt >> 1) & 1u;
        if (!(ok = mbar_wait(tempty0 + 8 * acc, aph ^ 1u, abort_flag, p.status, 2))) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const uint32_t s = it % S, ph = (it / S) & 1u;
          if (!(ok = mbar_wait(full0 + 8 * s, ph, abort_flag, p.status, 3))) break;
          tc_fence_after();
          const uint32_t sa = tiles_base + s * Cfg::kStageBytes, sb = sa + kBM * kBK * 2;
          const uint64_t da = make_sdesc(sa), db = make_sdesc(sb);
          int nk16 = (min(kBK, p.K - kb * kBK) + 15) / 16;
          if (kb >= nkb_main) {
            const int j = kb - nkb_main, rb = (j >= nrb) ? j - nrb : j;
            nk16 = (min(kBK, r_use - rb * kBK) + 15) / 16;   // columns beyond the adapter's rank: no MMA (<= 0 steps)
          }
          for (int k = 0; k < nk16; ++k)
            tc_mma_bf16(tmem_d, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          tc_commit(empty0 + 8 * s);
        }
        if (ok) tc_commit(tfull0 + 8 * acc);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int q = warp & 3;             // TMEM lane quarter this warp may read
    const int trow = q * 32 + lane;     // row of the tile owned by this thread
    uint32_t lt = 0;
    uint32_t n_st = 0;                  // tiled stores issued by this warp so far
    // eight epilogue warps share a tile's columns in halves; a lean launch (kTcThreadsLean) has four, all columns each
    const int wh = (warp - 2) >> 2;
    const int c_w = (blockDim.x > kTcThreadsLean) ? BN / 2 : BN;
    const int c_lo = wh * c_w, c_hi = c_lo + c_w;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++lt) {
      int row0, rows, n0, slot;
      tile_info(tile, row0, rows, n0, slot);
      const uint32_t acc = lt & 1u, aph = (lt >> 1) & 1u;
      if (!(ok = mbar_wait(tfull0 + 8 * acc, aph, abort_flag, p.status, 4))) break;
      tc_fence_after();
      const bool row_ok = trow < rows;
      const size_t grow = (size_t)(row0 + trow);
      float best = -INFINITY;
      int best_k = 0;
      float second = -INFINITY;   // EPI_ROUTER2: runner-up of this tile's columns
      int second_k = 0;
      const int ncols = (EPI == EPI_SHRINK) ? min(BN, (p.N + 31) / 32 * 32) : BN;
      // Plain store of a warp's 32 rows when all of them belong to the tile: 64 columns at a time are laid down in
      // shared memory (128-byte swizzled rows) and leave as one tiled store of whole 128-byte lines.  Written
      // straight from registers, a warp's 16-byte pieces go to 32 different lines per instruction, and those
      // partial-line requests compete with the operand loads in L2: the main loop ran 12 % slower beside them.
      const bool staged = (EPI == EPI_STORE) && p.tma_store && (q * 32 + 32 <= rows);
      if (staged) {
#pragma unroll 1
        for (int c = (c_w >= 64 ? c_lo : 0); c < (c_w >= 64 ? c_hi : (wh == 0 ? BN : 0)); c += 64) {
          if (n0 + c >= p.N) break;
          const uint32_t buf = out0 + (uint32_t)(wh * 4 + q) * 4096u;
          if (n_st >= 1) {               // the store that last read this buffer
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
          }
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t v[32];
            tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + c + 32 * hh, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t o0 = pack_bf16(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1]));
              const uint32_t o1 = pack_bf16(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
              const uint32_t o2 = pack_bf16(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
              const uint32_t o3 = pack_bf16(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
              const uint32_t dst = buf + (uint32_t)lane * 128u + ((uint32_t)((4 * hh + j) ^ (lane & 7)) << 4);
              asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
            }
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tmY, buf, n0 + c, row0 + q * 32);
            bulk_commit();
          }
          ++n_st;
        }
      }
#pragma unroll 1
      for (int c = c_lo; c < min(ncols, c_hi) && !staged; c += 32) {
        if (n0 + c >= p.N) break;
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + c, v);
        tmem_ld_wait();
        if (EPI == EPI_ROUTER || EPI == EPI_ROUTER2) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int k = n0 + c + j;
            if (k < p.N) {
              const float inv = __ldg(p.inv_norm + k);
              const float sim = __uint_as_float(v[j]) * inv;
              if (inv > 0.f && sim > best) {
                if (EPI == EPI_ROUTER2) {
                  second = best;
                  second_k = best_k;
                }
                best = sim;
                best_k = k;
              } else if (EPI == EPI_ROUTER2 && inv > 0.f && sim > second) {
                second = sim;
                second_k = k;
              }
            }
          }
        } else if (row_ok && (EPI == EPI_STORE || stacked || slot >= 0)) {
          const float sc = (EPI == EPI_SHRINK) ? p.scale : 1.f;
          __nv_bfloat16* ybase = p.y;
          __nv_bfloat16* ylo_base = p.y_lo;
          if (EPI == EPI_SHRINK && p.n_jobs > 0) {
            ybase = (job == 0) ? p.ys[0] : (job == 1) ? p.ys[1] : p.ys[2];
            ylo_base = (job == 0) ? p.ys_lo[0] : (job == 1) ? p.ys_lo[1] : p.ys_lo[2];
          }
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            int cj = n0 + c + j;     // first of eight columns (N is a multiple of 8); stacked: of its projection
            int ru = r_use;
            bool keep = cj < p.N;
            if (stacked && keep) {
              const int jb = cj / p.stack_r;
              cj -= jb * p.stack_r;
              keep = (jb == 0 ? st_slot[0] : jb == 1 ? st_slot[1] : st_slot[2]) >= 0;
              ru = jb == 0 ? st_ruse[0] : jb == 1 ? st_ruse[1] : st_ruse[2];
              ybase = jb == 0 ? p.ys[0] : jb == 1 ? p.ys[1] : p.ys[2];
              ylo_base = jb == 0 ? p.ys_lo[0] : jb == 1 ? p.ys_lo[1] : p.ys_lo[2];
            }
            __nv_bfloat16* yrow = ybase + grow * (size_t)p.ldy + cj - j;
            if (keep) {
              float f[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[j + e]) * sc;
              if (EPI == EPI_SHRINK) {   // function between the low-rank matrices; nothing beyond the adapter's rank
#pragma unroll
                for (int e = 0; e < 8; ++e)
                  f[e] = (cj + e < ru) ? lora_act(__uint_as_float(v[j + e]), p.act) * sc : 0.f;
              }
              uint4 o;
              o.x = pack_bf16(f[0], f[1]);
              o.y = pack_bf16(f[2], f[3]);
              o.z = pack_bf16(f[4], f[5]);
              o.w = pack_bf16(f[6], f[7]);
              *reinterpret_cast<uint4*>(yrow + j) = o;
              if (EPI == EPI_SHRINK) {   // low part, so that hi + lo carries the value to ~fp32 accuracy
                uint4 l;
                l.x = pack_bf16(f[0] - bf16_lo(o.x), f[1] - bf16_hi(o.x));
                l.y = pack_bf16(f[2] - bf16_lo(o.y), f[3] - bf16_hi(o.y));
                l.z = pack_bf16(f[4] - bf16_lo(o.z), f[5] - bf16_hi(o.z));
                l.w = pack_bf16(f[6] - bf16_lo(o.w), f[7] - bf16_hi(o.w));
                *reinterpret_cast<uint4*>(ylo_base + grow * (size_t)p.ldy + cj) = l;
              }
              if (EPI == EPI_STORE && p.y0) {
                float* y0row = p.y0 + grow * (size_t)p.ldy + cj;
                *reinterpret_cast<uint4*>(y0row) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                *reinterpret_cast<uint4*>(y0row + 4) = make_uint4(v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
              }
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(tempty0 + 8 * acc);
      if (EPI == EPI_ROUTER && row_ok && best > -INFINITY) {
        const unsigned long long key = ((unsigned long long)orderable(best) << 32) |
                                       (unsigned long long)(0xFFFFFFFFu - (uint32_t)best_k);
        atomicMax(p.keys + grow, key);
      }
      if (EPI == EPI_ROUTER2 && row_ok) {
        // Two-slot merge: the max goes to keys; whatever loses a comparison there (the value it displaced, or
        // the candidate itself) is offered to keys2.  Every candidate but the overall best is a loser exactly
        // once, keys are distinct (they carry the index), and both slots are maxima: order independent.
        const float cand[2] = {best, second};
        const int cand_k[2] = {best_k, second_k};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (cand[i] > -INFINITY) {
            const unsigned long long key = ((unsigned long long)orderable(cand[i]) << 32) |
                                           (unsigned long long)(0xFFFFFFFFu - (uint32_t)cand_k[i]);
            const unsigned long long old = atomicMax(p.keys + grow, key);
            const unsigned long long loser = old < key ? old : key;
            if (loser != 0ull) atomicMax(p.keys2 + grow, loser);
          }
        }
      }
    }
  }
  // ------------------------------------------------------------------ teardown
  if (EPI == EPI_STORE && warp >= 2 && lane == 0) bulk_wait_all();   // this thread's tiled stores are complete
  if (*abort_flag) {
    // a wait ran out somewhere: give copies / MMAs still in flight time to land before the CTA's
    // shared and tensor memory are released
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

static moin_status get_encoder() {
  if (g_encode) return MOIN_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return record_cuda(e);
  if (qres != cudaDriverEntryPointSuccess || !fn) return record_cuda(cudaErrorNotSupported);
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return MOIN_OK;
}

// 2-D row-major bf16 tensor [rows, cols] -> map with a [box_rows x 64] box, 128-byte swizzle, zero fill.
moin_status make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  moin_status st = get_encoder();
  if (st) return st;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return record_cuda(cudaErrorInvalidValue);
  return MOIN_OK;
}

template <int BN, int EPI>
static moin_status launch_cfg(HostState* hs, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& a2,
                              const CUtensorMap& a3, const CUtensorMap& b2, const TcParams& p, long max_tiles,
                              cudaStream_t stream, const CUtensorMap* b3 = nullptr, const CUtensorMap* ymap = nullptr,
                              bool lean = false) {
  using Cfg = TcCfg<BN>;
  constexpr int slot = OPTIN_TC_GEMM + 4 * (BN == 256 ? 2 : BN == 128 ? 1 : 0) + EPI;
  cudaError_t e = ensure_smem_optin(slot, tc_gemm_kernel<BN, EPI>, Cfg::kSmemBytes);
  if (e != cudaSuccess) return record_cuda(e);
  long grid = max_tiles < hs->n_sms ? max_tiles : hs->n_sms;
  if (grid < 1) grid = 1;
  const int threads = lean ? kTcThreadsLean : kTcThreads;
  const size_t smem = lean ? Cfg::kSmemBytes - Cfg::kOutBytes : Cfg::kSmemBytes;   // (lean launches never stage)
  tc_gemm_kernel<BN, EPI><<<(int)grid, threads, smem, stream>>>(a, b, a2, a3, b2, b3 ? *b3 : b2, ymap ? *ymap : a, p);
  return record_cuda(cudaGetLastError());
}

// Tile width for many row tiles: the one with the least (waves of tiles over the SMs) x (time of one tile), a
// tile's time taken as proportional to BN plus a fixed part worth 64 columns.  A projection as narrow as k or v
// (N = 256) then runs as one wave of 128 x 256 tiles rather than two of 128 x 128.
static int pick_bn(long tiles_m, int N, int n_sms) {
  int best = 64;
  long best_cost = -1;
  for (int bn : {256, 128, 64}) {
    const long tiles = tiles_m * ((N + bn - 1) / bn);
    const long cost = ((tiles + n_sms - 1) / n_sms) * (bn + 64);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}
// Few row tiles (decode): a CTA's duration grows with the bytes it pulls, (128 + BN) * K * 2 (an SM receives about
// 64 bytes per clock).  This GEMM runs beside the adapter shrink and the expand waits for both, so take the widest
// tile (fewest CTAs, least re-reading of x) whose per-CTA bytes stay under a budget that keeps the GEMM the shorter
// of the two.  Measured on the decode step's kernel timeline: with 0.8e6 no GEMM outlasts its shrink (the single
// 2048 -> 2048 projection takes 128 x 64 tiles, 16 us beside a 16 us shrink); 1.1e6 left it exposed by 6 us.
static int pick_bn_small_m(int N, int K) {
  const double budget = 0.8e6;
  for (int bn : {256, 128}) {
    if ((128.0 + bn) * K * 2 <= budget && N >= bn) return bn;
  }
  return 64;
}

bool tc_gemm_supported(int T, int d_in, int d_out) { return T >= 1 && d_in >= 64 && (d_in % 8) == 0 && (d_out % 8) == 0; }
bool tc_router_supported(int Q, int K, int D) { return Q >= 1 && K >= 1 && D >= 64 && (D % 8) == 0; }
bool tc_fused_supported(int r) { return r >= 8 && r <= 128 && (r % 8) == 0; }

moin_status launch_tc_gemm(HostState* hs, const __nv_bfloat16* x, const __nv_bfloat16* W, __nv_bfloat16* y, float* y0,
                           int T, int d_in, int d_out, cudaStream_t stream, int cta_budget) {
  const long tiles_m = (T + kBM - 1) / kBM;
  int bn = (tiles_m <= 2 && y0 != nullptr) ? pick_bn_small_m(d_out, d_in) : pick_bn(tiles_m, d_out, hs->n_sms);
  // Beside the adapter streams (decode): a CTA of this kernel keeps its SM to itself (the ring takes the shared
  // memory), and while a launch still has CTAs waiting for an SM the stream kernel behind it gets none.  Widen the
  // tiles until the launch fits the share of the SMs the caller grants it.
  while (cta_budget > 0 && bn < 256 && d_out >= 2 * bn && tiles_m * ((d_out + bn - 1) / bn) > cta_budget) bn *= 2;
  CUtensorMap a, b;
  moin_status st = make_map(&a, x, T, d_in, kBM);
  if (!st) st = make_map(&b, W, d_out, d_in, bn);
  if (st) return st;
  TcParams p = {};
  p.M = T; p.N = d_out; p.K = d_in; p.y = y; p.y0 = y0; p.ldy = d_out; p.scale = 1.f; p.status = hs->status;
  CUtensorMap ym = a;
  if (y0 == nullptr) {   // (with the fp32 copy the rows are written straight from registers, both at once)
    if ((st = make_map(&ym, y, T, d_out, 32))) return st;
    p.tma_store = 1;
  }
  const long tiles = tiles_m * ((d_out + bn - 1) / bn);
  const bool lean = p.tma_store == 0;
  if (bn == 256) return launch_cfg<256, EPI_STORE>(hs, a, b, a, a, b, p, tiles, stream, nullptr, &ym, lean);
  if (bn == 128) return launch_cfg<128, EPI_STORE>(hs, a, b, a, a, b, p, tiles, stream, nullptr, &ym, lean);
  return launch_cfg<64, EPI_STORE>(hs, a, b, a, a, b, p, tiles, stream, nullptr, &ym, lean);
}

moin_status launch_tc_router(HostState* hs, const __nv_bfloat16* q, const __nv_bfloat16* c, const float* inv_norm,
                             int Q, int K, int D, unsigned long long* keys, cudaStream_t stream,
                             unsigned long long* keys2) {
  const long tiles_m = (Q + kBM - 1) / kBM;
  const int bn = pick_bn(tiles_m, K, hs->n_sms);
  CUtensorMap a, b;
  moin_status st = make_map(&a, q, Q, D, kBM);
  if (!st) st = make_map(&b, c, K, D, bn);
  if (st) return st;
  TcParams p = {};
  p.M = Q; p.N = K; p.K = D; p.inv_norm = inv_norm; p.keys = keys; p.keys2 = keys2; p.status = hs->status;
  const long tiles = tiles_m * ((K + bn - 1) / bn);
  if (keys2 != nullptr) {
    if (bn == 256) return launch_cfg<256, EPI_ROUTER2>(hs, a, b, a, a, b, p, tiles, stream);
    if (bn == 128) return launch_cfg<128, EPI_ROUTER2>(hs, a, b, a, a, b, p, tiles, stream);
    return launch_cfg<64, EPI_ROUTER2>(hs, a, b, a, a, b, p, tiles, stream);
  }
  if (bn == 256) return launch_cfg<256, EPI_ROUTER>(hs, a, b, a, a, b, p, tiles, stream);
  if (bn == 128) return launch_cfg<128, EPI_ROUTER>(hs, a, b, a, a, b, p, tiles, stream);
  return launch_cfg<64, EPI_ROUTER>(hs, a, b, a, a, b, p, tiles, stream);
}

// Long-run mode, step 1 for up to kMaxShrinkJobs projections that share the plan, d_in and the rank:
// hb_j[row, :r] = hi/lo bf16 parts of scale * x_j A_j,e^T in ONE launch (row tiles of all the projections in
// one persistent grid, so set-up, first round trip and tail are paid once).
moin_status launch_tc_shrink_group(HostState* hs, const PlanView& pv, const moin_pool* const* pools,
                                   const __nv_bfloat16* const* xs, __nv_bfloat16* const* hbs, int n_jobs, float scale,
                                   cudaStream_t stream) {
  if (n_jobs < 1 || n_jobs > kMaxShrinkJobs) return MOIN_ERR_INVALID_ARG;
  const int T = pv.T, d_in = pools[0]->d_in, r = pools[0]->r;
  CUtensorMap ax[kMaxShrinkJobs], bA[kMaxShrinkJobs];
  TcParams p = {};
  p.M = T; p.N = r; p.K = d_in; p.header = pv.header; p.tile_row0 = pv.tile_row0; p.tile_rows = pv.tile_rows;
  p.tile_expert = pv.tile_expert; p.rows_per_slot = r; p.b_box_rows = r; p.ldy = r;
  p.scale = scale; p.status = hs->status; p.n_jobs = n_jobs;
  for (int j = 0; j < n_jobs; ++j) {
    if (pools[j]->d_in != d_in || pools[j]->r != r) return MOIN_ERR_INVALID_ARG;
    moin_status st = make_map(&ax[j], xs[j], T, d_in, kBM);
    if (!st) st = make_map(&bA[j], pools[j]->A, (uint64_t)pools[j]->n_slots * r, d_in, r);   // one slot's rows, no neighbours
    if (st) return st;
    p.slot_tabs[j] = pools[j]->slot_of_expert;
    p.rank_tabs[j] = pools[j]->slot_rank;
    p.act = pools[j]->activation;
    p.ys[j] = hbs[j];
    p.ys_lo[j] = hbs[j] + (size_t)T * r;   // low parts follow the high parts in the workspace
  }
  for (int j = n_jobs; j < kMaxShrinkJobs; ++j) {   // unused maps: any valid one
    ax[j] = ax[0];
    bA[j] = bA[0];
  }
  ProfScope prof(MOIN_K_SHRINK_TC, 1, stream);
  // Projections that read the same x and whose ranks fit one tile side by side take ONE pass over x: their
  // adapters' rows are stacked in the B operand and the accumulator's column groups go to their own outputs.
  bool same_x = n_jobs > 1 && n_jobs * r <= 256;
  for (int j = 1; j < n_jobs; ++j) same_x = same_x && xs[j] == xs[0];
  if (same_x) {
    p.n_jobs = 1;
    p.n_stack = n_jobs;
    p.stack_r = r;
    p.N = n_jobs * r;
    p.b_box_rows = 0;
    const int nt = n_jobs * r;
    if (nt > 128) return launch_cfg<256, EPI_SHRINK>(hs, ax[0], bA[0], ax[1], ax[2], bA[1], p, (long)T, stream, &bA[2]);
    if (nt > 64) return launch_cfg<128, EPI_SHRINK>(hs, ax[0], bA[0], ax[1], ax[2], bA[1], p, (long)T, stream, &bA[2]);
    return launch_cfg<64, EPI_SHRINK>(hs, ax[0], bA[0], ax[1], ax[2], bA[1], p, (long)T, stream, &bA[2]);
  }
  // upper bound on row tiles without reading the plan back: every run adds at most one partial tile;
  // the grid is capped at the SM count and the kernel reads the true count
  if (r > 64) return launch_cfg<128, EPI_SHRINK>(hs, ax[0], bA[0], ax[1], ax[2], bA[1], p, (long)T * n_jobs, stream, &bA[2]);
  return launch_cfg<64, EPI_SHRINK>(hs, ax[0], bA[0], ax[1], ax[2], bA[1], p, (long)T * n_jobs, stream, &bA[2]);
}

// Long-run mode, step 2: y = [x | hi | lo] [W ; B_e ; B_e]^T with hb from step 1.
moin_status launch_tc_fused(HostState* hs, const PlanView& pv, const moin_pool* pool, const __nv_bfloat16* x,
                            const __nv_bfloat16* W, __nv_bfloat16* y, __nv_bfloat16* hb, cudaStream_t stream) {
  const int T = pv.T, d_in = pool->d_in, d_out = pool->d_out, r = pool->r;
  const long max_tiles_m = T;
  CUtensorMap ax, bW, ah, al, bB;
  __nv_bfloat16* hb_lo = hb + (size_t)T * r;
  ProfScope prof(MOIN_K_FUSED_TC, 1, stream);
  const long full_tiles_m = (T + kBM - 1) / kBM;
  const int bn = pick_bn(full_tiles_m, d_out, hs->n_sms);
  moin_status st = make_map(&ax, x, T, d_in, kBM);
  if (!st) st = make_map(&ah, hb, T, r, kBM);
  if (!st) st = make_map(&al, hb_lo, T, r, kBM);
  if (!st) st = make_map(&bW, W, d_out, d_in, bn);
  if (!st) st = make_map(&bB, pool->B, (uint64_t)pool->n_slots * d_out, r, bn);
  CUtensorMap ym;
  if (!st) st = make_map(&ym, y, T, d_out, 32);
  if (st) return st;
  TcParams p = {};
  p.M = T; p.N = d_out; p.K = d_in; p.header = pv.header; p.tile_row0 = pv.tile_row0; p.tile_rows = pv.tile_rows;
  p.tile_expert = pv.tile_expert; p.slot_of_expert = pool->slot_of_expert; p.tail_r = r; p.rows_per_slot = d_out;
  p.slot_rank = pool->slot_rank;
  p.y = y; p.ldy = d_out; p.scale = 1.f; p.status = hs->status;
  p.tma_store = 1;
  const long tiles = max_tiles_m * ((d_out + bn - 1) / bn);
  if (bn == 256) return launch_cfg<256, EPI_STORE>(hs, ax, bW, ah, al, bB, p, tiles, stream, nullptr, &ym);
  if (bn == 128) return launch_cfg<128, EPI_STORE>(hs, ax, bW, ah, al, bB, p, tiles, stream, nullptr, &ym);
  return launch_cfg<64, EPI_STORE>(hs, ax, bW, ah, al, bB, p, tiles, stream, nullptr, &ym);
}

}  // namespace moin
