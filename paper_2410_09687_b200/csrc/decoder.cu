// Decoder forward: glue kernels (embedding, RMSNorm, rotary embedding, causal GQA attention,
// SwiGLU) around the routed LoRA projections, and the host-side sequencing.
#include "common.cuh"
#include "tc_gemm.cuh"

namespace moin {

// token -> (position inside its request, its expert: the caller's per-token id if given, else the expert of its
// request).  One CTA per request.
__global__ void __launch_bounds__(256)
token_meta_kernel(const int* __restrict__ cu, const int* __restrict__ req_expert,
                  const int* __restrict__ token_expert_in, int R, int* __restrict__ pos,
                  int* __restrict__ token_expert, int* __restrict__ last_row) {
  const int r = blockIdx.x;
  if (r >= R) return;
  const int t0 = cu[r], t1 = cu[r + 1];
  const int e = req_expert ? req_expert[r] : -1;
  for (int t = t0 + threadIdx.x; t < t1; t += blockDim.x) {
    pos[t] = t - t0;
    token_expert[t] = token_expert_in ? token_expert_in[t] : e;
  }
  if (threadIdx.x == 0) last_row[r] = (t1 > t0) ? t1 - 1 : -1;
}

// W[j][i] = bf16(fp32(value(code[j][i]) * scale[j])): 8-bit float codes (4 exponent bits, bias 7, 3 mantissa bits,
// no infinities, 0x7F / 0xFF = NaN) -> the bf16 weight the GEMMs read.  One thread converts 16 codes.
__device__ __forceinline__ float e4m3_to_float(uint32_t c) {
  const uint32_t sign = (c & 0x80u) << 24, ex = (c >> 3) & 15u, man = c & 7u;
  if (ex == 15u && man == 7u) return __uint_as_float(0x7FC00000u);
  if (ex == 0u) return __uint_as_float(sign | __float_as_uint((float)man * 0.001953125f));   // man * 2^-9
  return __uint_as_float(sign | ((ex + 120u) << 23) | (man << 20));
}
__global__ void __launch_bounds__(256)
dequant_fp8_kernel(const uint4* __restrict__ codes, const float* __restrict__ scale, int d_in16, long n16,
                   uint4* __restrict__ out) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n16) return;
  const float sc = __ldg(scale + i / d_in16);
  const uint4 c = ldg_stream(codes + i);
  const uint32_t w[4] = {c.x, c.y, c.z, c.w};
  uint32_t o[8];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float f0 = e4m3_to_float(w[k] & 0xFFu) * sc, f1 = e4m3_to_float((w[k] >> 8) & 0xFFu) * sc;
    const float f2 = e4m3_to_float((w[k] >> 16) & 0xFFu) * sc, f3 = e4m3_to_float(w[k] >> 24) * sc;
    o[2 * k] = pack_bf16(f0, f1);
    o[2 * k + 1] = pack_bf16(f2, f3);
  }
  out[2 * i] = make_uint4(o[0], o[1], o[2], o[3]);
  out[2 * i + 1] = make_uint4(o[4], o[5], o[6], o[7]);
}

// cos/sin of pos * base^(-2i/hd), computed in double once per call.
__global__ void rope_table_kernel(float2* __restrict__ table, int n_pos, int half, double base) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pos * half) return;
  const int p = idx / half, i = idx - p * half;
  const double ang = (double)p * pow(base, -(double)i / (double)half);
  table[idx] = make_float2((float)cos(ang), (float)sin(ang));
}

__global__ void __launch_bounds__(256)
embed_kernel(const int* __restrict__ tokens, const __nv_bfloat16* __restrict__ embed, int hidden, int vocab,
             float* __restrict__ res) {
  const int t = blockIdx.x;
  int tok = tokens[t];
  tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
  const __nv_bfloat16* row = embed + (size_t)tok * hidden;
  for (int i = threadIdx.x * 8; i < hidden; i += blockDim.x * 8) {
    const uint4 v = ldg_cached(row + i);
    float4 a = make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    float4 b = make_float4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w));
    *reinterpret_cast<float4*>(res + (size_t)t * hidden + i) = a;
    *reinterpret_cast<float4*>(res + (size_t)t * hidden + i + 4) = b;
  }
}

// res[t] += add[t] (bf16, optional);  out[t] = bf16(res[t] / sqrt(mean(res[t]^2) + eps) * gain)  (optional)
// rows (nullable): gather list - CTA b normalises row rows[b] into out row b (used for last-token logits).
__global__ void __launch_bounds__(256)
add_rmsnorm_kernel(float* __restrict__ res, const __nv_bfloat16* __restrict__ add,
                   const __nv_bfloat16* __restrict__ gain, __nv_bfloat16* __restrict__ out, int hidden, float eps,
                   const int* __restrict__ rows) {
  __shared__ float s_part[8];
  const int b = blockIdx.x;
  const int t = rows ? rows[b] : b;
  if (t < 0) return;
  float* rrow = res + (size_t)t * hidden;
  float ss = 0.f;
  for (int i = threadIdx.x * 4; i < hidden; i += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(rrow + i);
    if (add) {
      const uint2 a = *reinterpret_cast<const uint2*>(add + (size_t)t * hidden + i);
      v.x += bf16_lo(a.x); v.y += bf16_hi(a.x); v.z += bf16_lo(a.y); v.w += bf16_hi(a.y);
      *reinterpret_cast<float4*>(rrow + i) = v;
    }
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  if (!out) return;
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += s_part[w];
  const float inv = rsqrtf(tot / (float)hidden + eps);
  for (int i = threadIdx.x * 4; i < hidden; i += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(rrow + i);
    const uint2 gv = *reinterpret_cast<const uint2*>(gain + i);
    uint2 o;
    o.x = pack_bf16(v.x * inv * bf16_lo(gv.x), v.y * inv * bf16_hi(gv.x));
    o.y = pack_bf16(v.z * inv * bf16_lo(gv.y), v.w * inv * bf16_hi(gv.y));
    *reinterpret_cast<uint2*>(out + (size_t)b * hidden + i) = o;
  }
}

// In-place rotary embedding on v[T][n_h * 64], pairing (i, i + 32).
__global__ void __launch_bounds__(256)
rope_kernel(__nv_bfloat16* __restrict__ v, const int* __restrict__ pos, const float2* __restrict__ table, int T,
            int n_h) {
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;  // (t, head, i)
  const long total = (long)T * n_h * 32;
  if (idx >= total) return;
  const int i = (int)(idx & 31);
  const long th = idx >> 5;
  const int t = (int)(th / n_h);
  __nv_bfloat16* p = v + th * 64;
  const float2 cs = table[pos[t] * 32 + i];
  const float a = __bfloat162float(p[i]), b = __bfloat162float(p[i + 32]);
  p[i] = __float2bfloat16_rn(a * cs.x - b * cs.y);
  p[i + 32] = __float2bfloat16_rn(b * cs.x + a * cs.y);
}

__global__ void __launch_bounds__(256)
swiglu_kernel(__nv_bfloat16* __restrict__ gate, const __nv_bfloat16* __restrict__ up, long n8) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n8) return;
  const uint4 gv = *reinterpret_cast<const uint4*>(gate + i * 8);
  const uint4 uv = *reinterpret_cast<const uint4*>(up + i * 8);
  const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, uw[4] = {uv.x, uv.y, uv.z, uv.w};
  uint32_t o[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float g0 = bf16_lo(gw[e]), g1 = bf16_hi(gw[e]);
    o[e] = pack_bf16(g0 / (1.f + __expf(-g0)) * bf16_lo(uw[e]), g1 / (1.f + __expf(-g1)) * bf16_hi(uw[e]));
  }
  *reinterpret_cast<uint4*>(gate + i * 8) = make_uint4(o[0], o[1], o[2], o[3]);
}

// Causal grouped-query attention inside each request, head_dim 64.
// Grid (query block of 64 rows, head, request); 4 warps x 16 query rows; keys and values staged 64 at a
// time, row-major [key][dim], in a two-buffer shared-memory ring filled with 16-byte asynchronous copies
// (the next tile is on its way while the current one is used); K fragments come from ldmatrix, V
// fragments from ldmatrix.trans (the transpose P V needs); online softmax in the exp2 domain.
constexpr int kAttPitch = 72;   // elements: 144-byte rows keep the 8 rows of an ldmatrix tile on distinct banks
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
  const int n = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_plain(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

__global__ void __launch_bounds__(128)
attention_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                 const __nv_bfloat16* __restrict__ v, const int* __restrict__ cu, __nv_bfloat16* __restrict__ out,
                 int n_heads, int n_kv_heads, float scale_log2, const float2* __restrict__ rope) {
  __shared__ __align__(16) uint16_t Ks[2][64 * kAttPitch];
  __shared__ __align__(16) uint16_t Vs[2][64 * kAttPitch];
  const int req = blockIdx.z, head = blockIdx.y, qb = blockIdx.x;
  const int t0 = cu[req], L = cu[req + 1] - t0;
  if (qb * 64 >= L) return;
  const int kvh = head / (n_heads / n_kv_heads);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int qd = n_heads * 64, kvd = n_kv_heads * 64;
  const int r0 = qb * 64 + warp * 16 + g, r1 = r0 + 8;  // query rows (within request) of this thread
  const int kv_end = min(L, qb * 64 + 64);
  const uint32_t ks_base = (uint32_t)__cvta_generic_to_shared(&Ks[0][0]);
  const uint32_t vs_base = (uint32_t)__cvta_generic_to_shared(&Vs[0][0]);
  constexpr uint32_t kBufBytes = 64 * kAttPitch * 2;

  auto stage = [&](int kb, int buf) {   // keys kb .. kb+63 -> buffer `buf`; rows past the request are zero-filled
#pragma unroll
    for (int i = tid; i < 64 * 8; i += 128) {
      const int key = i >> 3, ch = i & 7;
      const bool ok = kb + key < L;
      const size_t row = (size_t)(t0 + (ok ? kb + key : L - 1)) * kvd + kvh * 64 + ch * 8;
      const uint32_t off = (uint32_t)buf * kBufBytes + (uint32_t)(key * kAttPitch + ch * 8) * 2;
      cp_async_16(ks_base + off, k + row, ok);
      cp_async_16(vs_base + off, v + row, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  stage(0, 0);

  uint32_t qa[4][4];
#pragma unroll
  for (int ks = 0; ks < 4; ++ks) {
    const int d = ks * 16 + 2 * t;
    const __nv_bfloat16* p0 = q + (size_t)(t0 + r0) * qd + head * 64 + d;
    const __nv_bfloat16* p1 = q + (size_t)(t0 + r1) * qd + head * 64 + d;
    qa[ks][0] = (r0 < L) ? *reinterpret_cast<const uint32_t*>(p0) : 0u;
    qa[ks][1] = (r1 < L) ? *reinterpret_cast<const uint32_t*>(p1) : 0u;
    qa[ks][2] = (r0 < L) ? *reinterpret_cast<const uint32_t*>(p0 + 8) : 0u;
    qa[ks][3] = (r1 < L) ? *reinterpret_cast<const uint32_t*>(p1 + 8) : 0u;
  }
  if (rope != nullptr) {
    // rotary embedding of the query rows on the fly (pairing (d, d + 32): k-steps ks and ks + 2 of the same
    // thread; position = row index inside the request), rounded to bf16 as the stand-alone kernel does
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
#pragma unroll
      for (int idx = 0; idx < 4; ++idx) {
        const int row = (idx & 1) ? r1 : r0;
        if (row < L) {
          const int d0 = ks * 16 + 2 * t + ((idx & 2) ? 8 : 0);
          const float4 cc = __ldg(reinterpret_cast<const float4*>(rope + (size_t)row * 32 + d0));   // d0 is even
          const float2 c0 = make_float2(cc.x, cc.y), c1 = make_float2(cc.z, cc.w);
          const uint32_t lo = qa[ks][idx], hi = qa[ks + 2][idx];
          const float a0 = bf16_lo(lo), a1 = bf16_hi(lo), b0 = bf16_lo(hi), b1 = bf16_hi(hi);
          qa[ks][idx] = pack_bf16(a0 * c0.x - b0 * c0.y, a1 * c1.x - b1 * c1.y);
          qa[ks + 2][idx] = pack_bf16(b0 * c0.x + a0 * c0.y, b1 * c1.x + a1 * c1.y);
        }
      }
  }
  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  // ldmatrix lane roles: lane l addresses row (l & 7) of matrix (l >> 3)
  const int lm_row = lane & 7, lm_mat = lane >> 3;
  for (int kb = 0, it = 0; kb < kv_end; kb += 64, ++it) {
    const int buf = it & 1;
    __syncthreads();                       // the other buffer's readers (previous tile) are done
    if (kb + 64 < kv_end) {
      stage(kb + 64, buf ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();                       // every thread's copies of this tile have landed
    const uint32_t kbuf = ks_base + (uint32_t)buf * kBufBytes, vbuf = vs_base + (uint32_t)buf * kBufBytes;
    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int j = 0; j < 4; ++j) s[nt][j] = 0.f;
#pragma unroll
      for (int kp = 0; kp < 2; ++kp) {
        // matrices: keys nt*8.., dim chunks kp*32 + {0, 8, 16, 24}  ->  (b0, b1) of k-step 2kp and of 2kp+1
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_plain(kbuf + (uint32_t)((nt * 8 + lm_row) * kAttPitch + kp * 32 + lm_mat * 8) * 2, b0, b1, b2, b3);
        mma_bf16_16816(s[nt], qa[2 * kp][0], qa[2 * kp][1], qa[2 * kp][2], qa[2 * kp][3], b0, b1);
        mma_bf16_16816(s[nt], qa[2 * kp + 1][0], qa[2 * kp + 1][1], qa[2 * kp + 1][2], qa[2 * kp + 1][3], b2, b3);
      }
    }
    // scale, causal mask, running max
    float mx0 = m0, mx1 = m1;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int key = kb + nt * 8 + 2 * t + (j & 1);
        const int row = (j < 2) ? r0 : r1;
        const float val = (key <= row && key < L) ? s[nt][j] * scale_log2 : -INFINITY;
        s[nt][j] = val;
        if (j < 2) mx0 = fmaxf(mx0, val); else mx1 = fmaxf(mx1, val);
      }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float base0 = (mx0 == -INFINITY) ? 0.f : mx0, base1 = (mx1 == -INFINITY) ? 0.f : mx1;
    const float corr0 = exp2f(m0 - base0), corr1 = exp2f(m1 - base1);  // m = -inf -> 0
    m0 = mx0; m1 = mx1;
    l0 *= corr0; l1 *= corr1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      o[i][0] *= corr0; o[i][1] *= corr0; o[i][2] *= corr1; o[i][3] *= corr1;
    }
    uint32_t pa[4][4];  // P as A fragments: 4 k16 steps over the 64 keys
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p0 = exp2f(s[nt][0] - base0), p1 = exp2f(s[nt][1] - base0);
      const float p2 = exp2f(s[nt][2] - base1), p3 = exp2f(s[nt][3] - base1);
      l0 += p0 + p1;
      l1 += p2 + p3;
      const int ks = nt >> 1, hi = nt & 1;
      pa[ks][hi * 2 + 0] = pack_bf16(p0, p1);
      pa[ks][hi * 2 + 1] = pack_bf16(p2, p3);
    }
#pragma unroll
    for (int dp = 0; dp < 4; ++dp)
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        // matrices: keys ks*16 + {0, 8} x dims (2dp)*8.., then the same keys x dims (2dp+1)*8..; transposed on load
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(vbuf + (uint32_t)((ks * 16 + (lm_mat & 1) * 8 + lm_row) * kAttPitch + (2 * dp + (lm_mat >> 1)) * 8) * 2,
                          b0, b1, b2, b3);
        mma_bf16_16816(o[2 * dp], pa[ks][0], pa[ks][1], pa[ks][2], pa[ks][3], b0, b1);
        mma_bf16_16816(o[2 * dp + 1], pa[ks][0], pa[ks][1], pa[ks][2], pa[ks][3], b2, b3);
      }
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
#pragma unroll
  for (int dt = 0; dt < 8; ++dt) {
    const int d = head * 64 + dt * 8 + 2 * t;
    if (r0 < L) *reinterpret_cast<uint32_t*>(out + (size_t)(t0 + r0) * qd + d) = pack_bf16(o[dt][0] * i0, o[dt][1] * i0);
    if (r1 < L) *reinterpret_cast<uint32_t*>(out + (size_t)(t0 + r1) * qd + d) = pack_bf16(o[dt][2] * i1, o[dt][3] * i1);
  }
}

struct DecoderWorkspace {
  float* res; __nv_bfloat16 *xn, *q, *k, *v, *att, *o, *gate, *up, *xlast;
  __nv_bfloat16* wq[3];   // dequantised weights of the projection group in flight (quantised base only)
  int *pos, *token_expert, *last_row;
  float2* rope;
  void* plan; size_t plan_bytes;
  void* lora; size_t lora_bytes;
  size_t total;
};

static DecoderWorkspace carve(const moin_model* m, int R, int T, int max_seqlen, void* base) {
  DecoderWorkspace w;
  char* p = reinterpret_cast<char*>(base);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return base ? (void*)(p + o) : nullptr; };
  const size_t H = m->hidden, qd = (size_t)m->n_heads * m->head_dim, kvd = (size_t)m->n_kv_heads * m->head_dim;
  const size_t F = m->ffn, TT = T;
  w.res = (float*)take(TT * H * 4);
  w.xn = (__nv_bfloat16*)take(TT * (H > qd ? H : qd) * 2);
  w.q = (__nv_bfloat16*)take(TT * qd * 2);
  w.k = (__nv_bfloat16*)take(TT * kvd * 2);
  w.v = (__nv_bfloat16*)take(TT * kvd * 2);
  w.att = (__nv_bfloat16*)take(TT * qd * 2);
  w.o = (__nv_bfloat16*)take(TT * H * 2);
  w.gate = (__nv_bfloat16*)take(TT * F * 2);
  w.up = (__nv_bfloat16*)take(TT * F * 2);
  w.xlast = (__nv_bfloat16*)take((size_t)R * H * 2);
  for (int i = 0; i < 3; ++i) w.wq[i] = m->W8 ? (__nv_bfloat16*)take(F * (H > qd ? H : qd) * 2) : nullptr;
  w.pos = (int*)take(TT * 4);
  w.token_expert = (int*)take(TT * 4);
  w.last_row = (int*)take((size_t)R * 4 + 4);
  w.rope = (float2*)take((size_t)(max_seqlen > 0 ? max_seqlen : T) * 32 * sizeof(float2));
  w.plan_bytes = moin_plan_bytes(T, m->E > 0 ? m->E : 1);
  w.plan = take(w.plan_bytes);
  size_t lb = 0;
  int r = 8;
  if (m->pools) r = m->pools[0].r;
  auto one = [&](size_t din, size_t dout) { return moin_lora_linear_workspace_bytes(T, (int)din, (int)dout, r); };
  const size_t groups[5] = {one(H, qd) + 2 * one(H, kvd), one(qd, H), 2 * one(H, F), one(F, H), one(H, (size_t)m->vocab)};
  for (size_t b : groups) lb = b > lb ? b : lb;
  w.lora_bytes = lb;
  w.lora = take(lb);
  w.total = off;
  return w;
}

}  // namespace moin

using namespace moin;

extern "C" size_t moin_decoder_workspace_bytes(const moin_model* model, int32_t R, int32_t T) {
  if (!model || R < 0 || T < 0) return 0;
  return carve(model, R, T, T, nullptr).total + 256;
}

static moin_status decoder_forward_impl(const moin_model* m, const int32_t* tokens, const int32_t* cu_seqlens,
                                        const int32_t* req_expert, const int32_t* token_expert_in, int32_t R,
                                        int32_t T, int32_t max_seqlen, void* logits, int32_t logits_mode,
                                        const moin_decoder_taps* taps, void* workspace, size_t workspace_bytes,
                                        moin_stream stream) {
  if (!m || R < 0 || T < 0) return MOIN_ERR_INVALID_ARG;
  if (R == 0 || T == 0) return MOIN_OK;
  if (!cu_seqlens || !m->W || !m->attn_norm || !m->mlp_norm || !m->final_norm) return MOIN_ERR_INVALID_ARG;
  if (m->head_dim != 64 || m->n_kv_heads < 1 || (m->n_heads % m->n_kv_heads) != 0) return MOIN_ERR_BAD_SHAPE;
  if ((m->hidden % 64) != 0 || (m->ffn % 64) != 0 || (m->vocab % 8) != 0) return MOIN_ERR_BAD_SHAPE;
  if (logits_mode < MOIN_LOGITS_ALL || logits_mode > MOIN_LOGITS_NONE) return MOIN_ERR_INVALID_ARG;
  if (logits_mode != MOIN_LOGITS_NONE && (!logits || !m->lm_head)) return MOIN_ERR_INVALID_ARG;
  if (max_seqlen < 1 || max_seqlen > T) max_seqlen = T;
  const int lb = taps ? taps->layer_begin : 0, le = taps ? taps->layer_end : m->n_layers;
  if (lb < 0 || le > m->n_layers || lb > le) return MOIN_ERR_INVALID_ARG;
  const bool from_hidden = taps && taps->hidden_in;
  if (!from_hidden && (!tokens || !m->embed)) return MOIN_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MOIN_ERR_WORKSPACE;
  DecoderWorkspace w = carve(m, R, T, T, workspace);
  if (workspace_bytes < w.total) return MOIN_ERR_WORKSPACE;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  cudaStream_t s = (cudaStream_t)stream;
  const int H = m->hidden, nh = m->n_heads, nkv = m->n_kv_heads, F = m->ffn;
  const int qd = nh * 64, kvd = nkv * 64;

  { ProfScope prof(MOIN_K_GLUE, 2, s);
  token_meta_kernel<<<R, 256, 0, s>>>(cu_seqlens, req_expert, token_expert_in, R, w.pos, w.token_expert, w.last_row);
  rope_table_kernel<<<(max_seqlen * 32 + 255) / 256, 256, 0, s>>>(w.rope, max_seqlen, 32, (double)m->rope_base); }
  moin_plan plan;
  memset(&plan, 0, sizeof(plan));
  const bool lora = m->pools != nullptr && (req_expert != nullptr || token_expert_in != nullptr);
  if (lora) {
    plan.buffer = w.plan; plan.buffer_bytes = w.plan_bytes; plan.T = T; plan.E = m->E;
    // one expert per request: the run lengths are the request lengths; one per token: they depend on the ids, so
    // the plan decides after it has grouped them (reads its header back: one synchronisation of the stream)
    plan.mode = token_expert_in ? MOIN_PLAN_AUTO : ((T / R >= 64) ? MOIN_PLAN_TILES : MOIN_PLAN_SEGMENTS);
    st = moin_plan_build(w.token_expert, &plan, stream);
    if (st) return st;
  }
  if (from_hidden) {
    cudaError_t e = cudaMemcpyAsync(w.res, taps->hidden_in, (size_t)T * H * 4, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return record_cuda(e);
  } else {
    ProfScope prof(MOIN_K_GLUE, 1, s);
    embed_kernel<<<T, 256, 0, s>>>(tokens, (const __nv_bfloat16*)m->embed, H, m->vocab, w.res);
  }
  // weight of projection p: the caller's bf16 matrix, or - quantised base - its codes dequantised into scratch slot
  // `slot` on the call's stream (the group calls join their side streams before they return, so a slot is free again)
  moin_status wst = MOIN_OK;
  auto weight = [&](int layer, int p, int d_in, int d_out, int slot) -> const void* {
    const int i = layer * 7 + p;
    if (!m->W8 || !m->W8[i]) return m->W[i];
    if (!m->W_scale || !m->W_scale[i]) { wst = MOIN_ERR_INVALID_ARG; return nullptr; }
    moin_status e = moin_dequant_fp8(m->W8[i], m->W_scale[i], d_out, d_in, w.wq[slot], stream);
    if (e) wst = e;
    return w.wq[slot];
  };
  auto proj = [&](int layer, int p, const void* in, int d_in, int d_out, void* out) -> moin_status {
    const void* W = weight(layer, p, d_in, d_out, 0);
    if (wst) return wst;
    return moin_lora_linear(lora ? &plan : nullptr, in, W, lora ? &m->pools[layer * 7 + p] : nullptr,
                            m->lora_scale, T, d_in, d_out, out, w.lora, w.lora_bytes, stream);
  };
  // projections of a block that read the same input and do not depend on one another go out as one group
  auto proj_group = [&](int layer, int p0, int n, const void* in, const int* d_in, const int* d_out,
                        void* const* outs) -> moin_status {
    if (!lora) {
      for (int i = 0; i < n; ++i) {
        moin_status e = proj(layer, p0 + i, in, d_in[i], d_out[i], outs[i]);
        if (e) return e;
      }
      return MOIN_OK;
    }
    moin_lora_job jobs[MOIN_MAX_GROUP];
    for (int i = 0; i < n; ++i) jobs[i] = {in, weight(layer, p0 + i, d_in[i], d_out[i], i), &m->pools[layer * 7 + p0 + i], outs[i]};
    if (wst) return wst;
    return moin_lora_linear_group(&plan, jobs, n, m->lora_scale, w.lora, w.lora_bytes, stream);
  };
  const float scale_log2 = 1.4426950408889634f / sqrtf(64.f);
  const __nv_bfloat16* pending = nullptr;
  for (int l = lb; l < le; ++l) {
    { ProfScope prof(MOIN_K_GLUE, 1, s);
      add_rmsnorm_kernel<<<T, 256, 0, s>>>(w.res, pending, (const __nv_bfloat16*)m->attn_norm[l], w.xn, H, m->rms_eps, nullptr); }
    {
      const int din[3] = {H, H, H}, dout[3] = {qd, kvd, kvd};
      void* const outs[3] = {w.q, w.k, w.v};
      if ((st = proj_group(l, 0, 3, w.xn, din, dout, outs))) return st;
    }
    // rotary embedding: the keys are rotated in place once (every query head and every later query reads them);
    // the queries are rotated inside the attention kernel as it loads them
    { ProfScope prof(MOIN_K_GLUE, 1, s);
      rope_kernel<<<(int)(((long)T * nkv * 32 + 255) / 256), 256, 0, s>>>(w.k, w.pos, w.rope, T, nkv); }
    if (hs->gemm_impl != 1 && attention_tc_supported(nh, nkv, m->head_dim)) {   // tcgen05 kernel
      ProfScope prof(MOIN_K_ATTENTION, 1, s);
      if ((st = launch_attention_tc(hs, w.q, w.k, w.v, cu_seqlens, w.att, w.rope, R, T, max_seqlen, nh, nkv,
                                    scale_log2, s)))
        return st;
    } else {   // warp-MMA kernel: other head groupings, or forced by MOIN_OPT_GEMM_IMPL = 1
      ProfScope prof(MOIN_K_ATTENTION, 1, s);
      attention_kernel<<<dim3((max_seqlen + 63) / 64, nh, R), 128, 0, s>>>(w.q, w.k, w.v, cu_seqlens, w.att, nh, nkv, scale_log2,
                                                                         w.rope);
    }
    if ((st = proj(l, 3, w.att, qd, H, w.o))) return st;
    { ProfScope prof(MOIN_K_GLUE, 1, s);
      add_rmsnorm_kernel<<<T, 256, 0, s>>>(w.res, w.o, (const __nv_bfloat16*)m->mlp_norm[l], w.xn, H, m->rms_eps, nullptr); }
    {
      const int din[2] = {H, H}, dout[2] = {F, F};
      void* const outs[2] = {w.gate, w.up};
      if ((st = proj_group(l, 4, 2, w.xn, din, dout, outs))) return st;
    }
    { ProfScope prof(MOIN_K_GLUE, 1, s);
      swiglu_kernel<<<(int)(((long)T * F / 8 + 255) / 256), 256, 0, s>>>(w.gate, w.up, (long)T * F / 8); }
    if ((st = proj(l, 6, w.gate, F, H, w.o))) return st;
    pending = w.o;
  }
  if (pending) { ProfScope prof(MOIN_K_GLUE, 1, s);
    add_rmsnorm_kernel<<<T, 256, 0, s>>>(w.res, pending, nullptr, nullptr, H, m->rms_eps, nullptr); }
  if (taps && taps->hidden_out) {
    cudaError_t e = cudaMemcpyAsync(taps->hidden_out, w.res, (size_t)T * H * 4, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return record_cuda(e);
  }
  if (logits_mode == MOIN_LOGITS_ALL) {
    { ProfScope prof(MOIN_K_GLUE, 1, s);
      add_rmsnorm_kernel<<<T, 256, 0, s>>>(w.res, nullptr, (const __nv_bfloat16*)m->final_norm, w.xn, H, m->rms_eps, nullptr); }
    st = moin_lora_linear(nullptr, w.xn, m->lm_head, nullptr, 0.f, T, H, m->vocab, logits, w.lora, w.lora_bytes, stream);
    if (st) return st;
  } else if (logits_mode == MOIN_LOGITS_LAST) {
    cudaError_t e = cudaMemsetAsync(w.xlast, 0, (size_t)R * H * 2, s);
    if (e != cudaSuccess) return record_cuda(e);
    { ProfScope prof(MOIN_K_GLUE, 1, s);
      add_rmsnorm_kernel<<<R, 256, 0, s>>>(w.res, nullptr, (const __nv_bfloat16*)m->final_norm, w.xlast, H, m->rms_eps, w.last_row); }
    st = moin_lora_linear(nullptr, w.xlast, m->lm_head, nullptr, 0.f, R, H, m->vocab, logits, w.lora, w.lora_bytes, stream);
    if (st) return st;
  }
  return record_cuda(cudaGetLastError());
}

extern "C" moin_status moin_decoder_forward(const moin_model* m, const int32_t* tokens, const int32_t* cu_seqlens,
                                            const int32_t* req_expert, int32_t R, int32_t T, int32_t max_seqlen,
                                            void* logits, int32_t logits_mode, const moin_decoder_taps* taps,
                                            void* workspace, size_t workspace_bytes, moin_stream stream) {
  return decoder_forward_impl(m, tokens, cu_seqlens, req_expert, nullptr, R, T, max_seqlen, logits, logits_mode, taps,
                              workspace, workspace_bytes, stream);
}

extern "C" moin_status moin_decoder_forward_per_token(const moin_model* m, const int32_t* tokens,
                                                      const int32_t* cu_seqlens, const int32_t* token_expert, int32_t R,
                                                      int32_t T, int32_t max_seqlen, void* logits, int32_t logits_mode,
                                                      const moin_decoder_taps* taps, void* workspace,
                                                      size_t workspace_bytes, moin_stream stream) {
  if (!token_expert) return MOIN_ERR_INVALID_ARG;
  return decoder_forward_impl(m, tokens, cu_seqlens, nullptr, token_expert, R, T, max_seqlen, logits, logits_mode, taps,
                              workspace, workspace_bytes, stream);
}

extern "C" moin_status moin_dequant_fp8(const void* codes, const float* scale, int32_t d_out, int32_t d_in, void* W,
                                        moin_stream stream) {
  if (!codes || !scale || !W || d_out < 0 || d_in < 0) return MOIN_ERR_INVALID_ARG;
  if ((d_in % 16) != 0) return MOIN_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(codes) & 15u) || (reinterpret_cast<uintptr_t>(W) & 15u)) return MOIN_ERR_MISALIGNED;
  const long n16 = (long)d_out * d_in / 16;
  if (n16 == 0) return MOIN_OK;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  ProfScope prof(MOIN_K_GLUE, 1, (cudaStream_t)stream);
  dequant_fp8_kernel<<<(unsigned)((n16 + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      (const uint4*)codes, scale, d_in / 16, n16, (uint4*)W);
  return record_cuda(cudaGetLastError());
}
