// Batch plan: grouping of tokens by expert id (integer work only).
//
// Batches of up to 1024 tokens take one single-CTA launch (plan_small_kernel: a bitonic sort of
// (expert id, token) keys in shared memory).  Larger ones take a few small launches:
//   plan_rank_kernel    per 256-token chunk: sanitise ids, stable in-chunk rank, per-chunk histogram
//   plan_prefix_kernel  (batches of more than one chunk) per expert id: prefix of its counts over the chunks
//   plan_scan_kernel    one CTA: prefix over expert ids -> segment list; run tiles
//   plan_scatter_kernel per chunk: position = expert base + chunk prefix + in-chunk rank -> perm
// The result is a stable counting sort (token order is kept inside every expert segment), so
// the plan is deterministic.
#include "common.cuh"

namespace moin {

__global__ void __launch_bounds__(kPlanChunk) plan_rank_kernel(const int* __restrict__ token_expert, int T, int E,
                                                               int* __restrict__ key, int* __restrict__ rank,
                                                               int* __restrict__ hist, DeviceStatus* status) {
  __shared__ int skey[kPlanChunk];
  const int tid = threadIdx.x;
  const int t = blockIdx.x * kPlanChunk + tid;
  int k = -2;  // padding lanes never match
  if (t < T) {
    int e = token_expert[t];
    if (e >= 0 && e < E) {
      k = e;
    } else {
      k = E;  // "no adapter" bucket
      if (e != -1) atomicAdd(&status->invalid_expert_ids, 1);
    }
  }
  skey[tid] = k;
  __syncthreads();
  if (t >= T) return;
  int before = 0, after = 0;
  for (int i = 0; i < kPlanChunk; ++i) {
    int same = (skey[i] == k);
    before += same & (i < tid);
    after += same & (i > tid);
  }
  key[t] = k;
  rank[t] = before;
  if (after == 0) hist[(size_t)blockIdx.x * (size_t)(E + 1) + k] = before + 1;
}

// Block-wide scans for NT threads (a multiple of 32, at most 1024).  `smem` must hold 33 ints.
template <int NT>
__device__ __forceinline__ int block_excl_sum(int v, int* smem, int* total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();  // protect smem reuse between calls
  if (lane == 31) smem[w] = inc;
  __syncthreads();
  if (w == 0) {
    int s = (lane < NT / 32) ? smem[lane] : 0;
    int si = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, si, o);
      if (lane >= o) si += n;
    }
    smem[lane] = si - s;  // exclusive prefix of warp totals
    if (lane == 31) smem[32] = si;
  }
  __syncthreads();
  *total = smem[32];
  return smem[w] + inc - v;
}
template <int NT>
__device__ __forceinline__ int block_incl_max(int v, int* smem) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc = max(inc, n);
  }
  __syncthreads();
  if (lane == 31) smem[w] = inc;
  __syncthreads();
  if (w == 0) {
    int s = (lane < NT / 32) ? smem[lane] : INT_MIN;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s = max(s, n);
    }
    smem[lane] = s;  // inclusive max over warps 0..lane
  }
  __syncthreads();
  int prev = (w > 0) ? smem[w - 1] : INT_MIN;
  return max(inc, prev);
}

// Per expert id: exclusive prefix of its per-chunk counts over the chunks (in place) and the total.
// A CTA covers 64 expert ids (threadIdx.x, so the loads of a chunk row are coalesced) and cuts the chunks into
// kPrefixGroups consecutive ranges (threadIdx.y); a thread sums its range with its loads in flight in batches,
// the ranges' totals meet in shared memory, and a second pass over the (now cached) counts writes the prefixes.
constexpr int kPrefixIds = 64, kPrefixGroups = 4, kPrefixBatch = 16;
__global__ void __launch_bounds__(kPrefixIds * kPrefixGroups) plan_prefix_kernel(PlanView v) {
  __shared__ int s_sum[kPrefixGroups][kPrefixIds];
  const int k = blockIdx.x * kPrefixIds + threadIdx.x, g = threadIdx.y;
  const bool on = k <= v.E;
  const size_t pitch = (size_t)(v.E + 1);
  const int per = (v.n_chunks + kPrefixGroups - 1) / kPrefixGroups;
  const int c_lo = g * per, c_hi = min(v.n_chunks, c_lo + per);
  int total = 0;
  for (int c0 = c_lo; on && c0 < c_hi; c0 += kPrefixBatch) {
    int n[kPrefixBatch];
#pragma unroll
    for (int j = 0; j < kPrefixBatch; ++j) n[j] = (c0 + j < c_hi) ? __ldcg(v.hist + (size_t)(c0 + j) * pitch + k) : 0;
#pragma unroll
    for (int j = 0; j < kPrefixBatch; ++j) total += n[j];
  }
  s_sum[g][threadIdx.x] = total;
  __syncthreads();
  int run = 0;
  for (int gg = 0; gg < g; ++gg) run += s_sum[gg][threadIdx.x];
  for (int c0 = c_lo; on && c0 < c_hi; c0 += kPrefixBatch) {
    int n[kPrefixBatch];
#pragma unroll
    for (int j = 0; j < kPrefixBatch; ++j) n[j] = (c0 + j < c_hi) ? __ldcg(v.hist + (size_t)(c0 + j) * pitch + k) : 0;
#pragma unroll
    for (int j = 0; j < kPrefixBatch; ++j) {
      if (c0 + j < c_hi) v.hist[(size_t)(c0 + j) * pitch + k] = run;
      run += n[j];
    }
  }
  if (on && g == kPrefixGroups - 1) v.keybase[k] = run;
}

// Row tiles: maximal runs of equal expert id in token order, cut every kTileRows rows.  One CTA of NT
// threads; `key[t]` is the sanitised id of token t (shared or global memory).  smem: 33 ints, s_carry: 2.
// `row0` is where the tile starts are read back from to form the tile lengths: v.tile_row0 itself, or a
// shared-memory copy ([T + 1] ints) when the caller has one.
template <int NT>
__device__ __forceinline__ void plan_tiles(const PlanView& v, const int* key, int* smem, int* s_carry, int* row0) {
  const int tid = threadIdx.x;
  const int T = v.T, E = v.E;
  int carry_start = 0, carry_tiles = 0;
  for (int t0 = 0; t0 < T; t0 += NT) {
    int t = t0 + tid;
    int k = (t < T) ? key[t] : -3;
    int is_start = (t < T) && (t == 0 || key[t - 1] != k);
    int rs = block_incl_max<NT>(is_start ? t : -1, smem);
    rs = max(rs, carry_start);
    int flag = (t < T) && (((t - rs) % kTileRows) == 0);
    int tot;
    int idx = carry_tiles + block_excl_sum<NT>(flag, smem, &tot);
    if (flag) {
      v.tile_row0[idx] = t;
      if (row0 != v.tile_row0) row0[idx] = t;
      v.tile_expert[idx] = (k == E) ? -1 : k;
    }
    if (tid == NT - 1) s_carry[0] = rs;
    __syncthreads();
    carry_start = s_carry[0];
    carry_tiles += tot;
    __syncthreads();
  }
  if (tid == 0) {
    v.tile_row0[carry_tiles] = T;
    if (row0 != v.tile_row0) row0[carry_tiles] = T;
    v.header[PH_NTILES] = carry_tiles;
  }
  __syncthreads();
  for (int i = tid; i < carry_tiles; i += NT) v.tile_rows[i] = row0[i + 1] - row0[i];
}

__global__ void __launch_bounds__(1024) plan_scan_kernel(PlanView v, int do_prefix, int want_tiles) {
  constexpr int NT = 1024;
  __shared__ int smem[33];
  __shared__ int s_carry[2];
  const int tid = threadIdx.x;
  const int T = v.T, E = v.E, nc = v.n_chunks;
  const size_t pitch = (size_t)(E + 1);

  // 1. per expert id: prefix over chunks (in place) and total (done by plan_prefix_kernel for multi-chunk batches)
  for (int k = tid; do_prefix && k <= E; k += 1024) {
    int run = 0;
    for (int c = 0; c < nc; ++c) {
      int* p = v.hist + (size_t)c * pitch + k;
      int n = *p;
      *p = run;
      run += n;
    }
    v.keybase[k] = run;
  }
  __syncthreads();

  // 2. prefix over expert ids -> segment list (ascending expert id), "no adapter" bucket last
  int carry_tok = 0, carry_seg = 0, max_seg = 0;
  for (int k0 = 0; k0 < E; k0 += 1024) {
    int k = k0 + tid;
    int n = (k < E) ? v.keybase[k] : 0;
    int tot_tok, tot_seg;
    int ex_tok = block_excl_sum<NT>(n, smem, &tot_tok);
    int ex_seg = block_excl_sum<NT>(n > 0 ? 1 : 0, smem, &tot_seg);
    if (k < E) {
      v.keybase[k] = carry_tok + ex_tok;
      if (n > 0) {
        v.seg_expert[carry_seg + ex_seg] = k;
        v.seg_start[carry_seg + ex_seg] = carry_tok + ex_tok;
        v.seg_tab[carry_seg + ex_seg] = make_int4(k, carry_tok + ex_tok, n, 0);
      }
    }
    max_seg = max(max_seg, n);
    carry_tok += tot_tok;
    carry_seg += tot_seg;
  }
  max_seg = block_incl_max<NT>(max_seg, smem);
  if (tid == 1023) {
    v.seg_start[carry_seg] = carry_tok;
    v.keybase[E] = carry_tok;
    v.header[PH_NSEG] = carry_seg;
    v.header[PH_NLORA] = carry_tok;
    v.header[PH_MAXSEG] = max_seg;
    v.header[PH_T] = T;
    v.header[PH_E] = E;
  }

  // 3. row tiles (only the long-run kernels read them)
  if (want_tiles) plan_tiles<NT>(v, v.key, smem, s_carry, v.tile_row0);
  else if (tid == 0) v.header[PH_NTILES] = 0;
}

// Whole plan of a batch of at most 1024 tokens in one CTA.  The tokens are sorted by the key
// (sanitised expert id << 10 | token index) with a bitonic network in shared memory: the low bits make
// the order stable, the sorted position of a token is its place in `perm`, and the segments are the
// runs of equal id in the sorted sequence (ascending id, the "no adapter" bucket E last).
constexpr int kPlanSmallT = 1024;
constexpr int kPlanSmallE = 1 << 20;   // the id must fit above the 10 token bits of a 31-bit key
template <int NT>   // threads = sort width: the power of two at or above T, at least 128
__global__ void __launch_bounds__(NT) plan_small_kernel(const int* __restrict__ token_expert, PlanView v,
                                                        DeviceStatus* status, int want_tiles) {
  __shared__ int s_key[NT];        // sanitised id by token
  __shared__ int s_sort[NT + 1];   // sort keys, then the segment starts plus one end marker (NT segments at most)
  __shared__ int s_row0[NT + 1];   // tile starts
  __shared__ int smem[33];
  __shared__ int s_carry[2];
  const int tid = threadIdx.x;
  const int T = v.T, E = v.E;
  int k = 0x1FFFFF;  // padding sorts last
  if (tid < T) {
    int e = token_expert[tid];
    if (e >= 0 && e < E) {
      k = e;
    } else {
      k = E;  // "no adapter" bucket
      if (e != -1) atomicAdd(&status->invalid_expert_ids, 1);
    }
  }
  s_key[tid] = (tid < T) ? k : -2;
  s_sort[tid] = (k << 10) | tid;
  __syncthreads();
  for (int size = 2; size <= NT; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      const int partner = tid ^ stride;
      if (partner > tid) {
        const int a = s_sort[tid], b = s_sort[partner];
        const bool up = (tid & size) == 0;
        if ((a > b) == up) {
          s_sort[tid] = b;
          s_sort[partner] = a;
        }
      }
      __syncthreads();
    }
  }
  // sorted position p holds (id, token): perm, run starts, segment list
  const int mine = s_sort[tid];
  const int id = mine >> 10;
  if (tid < T) v.perm[tid] = mine & 1023;
  const int prev_id = (tid > 0) ? (s_sort[tid - 1] >> 10) : -1;
  const int is_start = (tid < T) && id < E && (tid == 0 || prev_id != id);
  int n_seg, n_lora;
  const int seg = block_excl_sum<NT>(is_start, smem, &n_seg);
  block_excl_sum<NT>((tid < T) && id < E, smem, &n_lora);   // tokens with an adapter sort first
  __syncthreads();                                           // every thread has read its neighbour's key
  if (is_start) s_sort[seg] = tid;                           // reuse as the segment-start list
  if (tid == 0) s_sort[n_seg] = n_lora;
  __syncthreads();
  int len = 0;
  if (is_start) {
    len = s_sort[seg + 1] - tid;
    v.seg_expert[seg] = id;
    v.seg_start[seg] = tid;
    v.seg_tab[seg] = make_int4(id, tid, len, 0);
  }
  if (tid == 0) v.seg_start[n_seg] = n_lora;
  const int max_seg = block_incl_max<NT>(len, smem);
  if (tid == NT - 1) {
    v.header[PH_NSEG] = n_seg;
    v.header[PH_NLORA] = n_lora;
    v.header[PH_MAXSEG] = max_seg;
    v.header[PH_T] = T;
    v.header[PH_E] = E;
  }
  if (want_tiles) plan_tiles<NT>(v, s_key, smem, s_carry, s_row0);
  else if (tid == 0) v.header[PH_NTILES] = 0;
}

__global__ void __launch_bounds__(kPlanChunk) plan_scatter_kernel(PlanView v) {
  const int t = blockIdx.x * kPlanChunk + threadIdx.x;
  if (t >= v.T) return;
  const int k = v.key[t];
  const int pos = v.keybase[k] + v.hist[(size_t)blockIdx.x * (size_t)(v.E + 1) + k] + v.rank[t];
  v.perm[pos] = t;
}

int plan_launches(int T, int E) {
  if (T <= kPlanSmallT && E < kPlanSmallE) return 1;
  return T > kPlanChunk ? 4 : 3;
}

cudaError_t launch_plan_build(const int* token_expert, const PlanView& v, DeviceStatus* status, bool want_tiles,
                              cudaStream_t stream) {
  if (v.T <= kPlanSmallT && v.E < kPlanSmallE) {
    if (v.T <= 128) plan_small_kernel<128><<<1, 128, 0, stream>>>(token_expert, v, status, want_tiles);
    else if (v.T <= 256) plan_small_kernel<256><<<1, 256, 0, stream>>>(token_expert, v, status, want_tiles);
    else if (v.T <= 512) plan_small_kernel<512><<<1, 512, 0, stream>>>(token_expert, v, status, want_tiles);
    else plan_small_kernel<1024><<<1, 1024, 0, stream>>>(token_expert, v, status, want_tiles);
    return cudaGetLastError();
  }
  cudaError_t e = cudaMemsetAsync(v.hist, 0, sizeof(int) * (size_t)v.n_chunks * (size_t)(v.E + 1), stream);
  if (e != cudaSuccess) return e;
  plan_rank_kernel<<<v.n_chunks, kPlanChunk, 0, stream>>>(token_expert, v.T, v.E, v.key, v.rank, v.hist, status);
  if (v.n_chunks > 1)
    plan_prefix_kernel<<<(v.E + 1 + kPrefixIds - 1) / kPrefixIds, dim3(kPrefixIds, kPrefixGroups), 0, stream>>>(v);
  plan_scan_kernel<<<1, 1024, 0, stream>>>(v, v.n_chunks > 1 ? 0 : 1, want_tiles);
  plan_scatter_kernel<<<v.n_chunks, kPlanChunk, 0, stream>>>(v);
  return cudaGetLastError();
}

}  // namespace moin
