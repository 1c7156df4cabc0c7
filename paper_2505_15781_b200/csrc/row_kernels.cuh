// Row-wise kernels between the GEMMs: embedding gather, split-K reduction
// fused with residual add + RMSNorm, RoPE + K/V slot scatter, SwiGLU, the
// head-row gather and the vocabulary softmax statistics.  T is the activation
// / cache element type (float in check mode, else fp16 or bf16); the residual
// stream and all statistics are fp32.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>
#include "head_stat.cuh"
#include "pdl.cuh"

namespace dkv {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

// Sum over a block of 256 threads; result valid in every thread.
__device__ __forceinline__ float block_sum_256(float v, float* s8) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s8[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) t += s8[i];
  return t;
}

// fp16 copy of a bf16 weight matrix [rows, k] (values below 2^-14 lose bits: |error| <= 2^-25) in blocks of 128 rows x 64 columns, block (i, j) at
// (i * ceil(k / 64) + j) * 8192 elements, rows inside a block 64 elements apart, zeros past the
// matrix: what the projection GEMM loads per weight half and k-block is one contiguous 16 KB piece.
// With gu_blk > 0 the matrix is [gate (gu_f rows); up (gu_f rows)] and the copy's rows are regrouped
// [gu_blk gate rows | gu_blk up rows] per 2 * gu_blk, so that the GEMM epilogue finds gate_j and up_j
// of a feature in the two accumulators of one thread.
// grid (ceil(k / 64), ceil(rows / 128)), 256 threads; k a multiple of 8.
__global__ void __launch_bounds__(256) k_block_f16(const __nv_bfloat16* __restrict__ in, __half* __restrict__ out,
                                                   int rows, int k, int gu_f, int gu_blk) {
  const long long blk = static_cast<long long>(blockIdx.y) * gridDim.x + blockIdx.x;
  uint4* o = reinterpret_cast<uint4*>(out + blk * (128 * 64));
  for (int e = threadIdx.x; e < 128 * 8; e += 256) {          // 8 vectors of 8 elements per row
    const int r = e >> 3, c8 = e & 7;
    const int dst = blockIdx.y * 128 + r, col = blockIdx.x * 64 + c8 * 8;
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    if (dst < rows && col < k) {
      long long src = dst;
      if (gu_blk > 0) {
        const int tile = dst / (2 * gu_blk), half = (dst / gu_blk) & 1, i = dst % gu_blk;
        src = static_cast<long long>(half) * gu_f + tile * gu_blk + i;
      }
      const uint4 v = *reinterpret_cast<const uint4*>(in + src * k + col);
      const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&v);
      __half2* h = reinterpret_cast<__half2*>(&w);
#pragma unroll
      for (int j = 0; j < 4; ++j) h[j] = __float22half2_rn(__bfloat1622float2(b[j]));
    }
    o[e] = w;
  }
}

// cos/sin table for RoPE: tab[pos * half + i] = (cos, sin)(pos * theta^(-2i/d_h)), computed in double.
__global__ void k_rope_table(float2* tab, int seq_len, int half, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= seq_len * half) return;
  const int pos = idx / half, i = idx % half;
  const double inv_freq = pow(theta, -static_cast<double>(i) / static_cast<double>(half));
  const double a = static_cast<double>(pos) * inv_freq;
  tab[idx] = make_float2(static_cast<float>(cos(a)), static_cast<float>(sin(a)));
}

// 8 consecutive elements of an embedding row as floats (16-byte loads)
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
  const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __bfloat1622float2(b[j]);
    v[2 * j] = f.x;
    v[2 * j + 1] = f.y;
  }
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 o;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
  for (int j = 0; j < 4; ++j) h[j] = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
  *reinterpret_cast<uint4*>(p) = o;
}
__device__ __forceinline__ void store8(__half* p, const float (&v)[8]) {
  uint4 o;
  __half2* h = reinterpret_cast<__half2*>(&o);
#pragma unroll
  for (int j = 0; j < 4; ++j) h[j] = __floats2half2_rn(v[2 * j], v[2 * j + 1]);
  *reinterpret_cast<uint4*>(p) = o;
}

// h[r] = E[tokens[act_idx[r]]] and the operand of the first QKV projection (one CTA per row, 16-byte
// accesses, d a multiple of 8).  ssq == NULL: xn[r] = RMSNorm(h[r]) * gain.  ssq != NULL: xn[r] =
// h[r] .* gain and ssq[r] = sum h[r]^2; the GEMM that reads xn divides by the RMS in its epilogue.
template <typename TW, typename T>
__global__ void __launch_bounds__(256)
k_embed_norm(const TW* __restrict__ embed, const int32_t* __restrict__ tokens, const int32_t* __restrict__ act_idx,
             const int* __restrict__ r_dev, const float* __restrict__ gain, float eps, int d, float* __restrict__ h,
             T* __restrict__ xn, float* __restrict__ ssq) {
  __shared__ float s8[8];
  pdl_enter(2);
  const int r = blockIdx.x;
  if (r >= *r_dev) return;
  const int tok = tokens[act_idx[r]];
  const TW* e = embed + static_cast<long long>(tok) * d;
  float* hr = h + static_cast<long long>(r) * d;
  T* xr = xn + static_cast<long long>(r) * d;
  constexpr int KEEP = 4;                     // row pieces of 2048 elements kept in registers (d <= 8192)
  float v[KEEP][8];
  float ss = 0.f;
  auto first_pass = [&](int c, float (&t)[8]) {
    load8(e + c, t);
    store8(hr + c, t);
#pragma unroll
    for (int j = 0; j < 8; ++j) ss += t[j] * t[j];
    if (ssq) {                                 // h .* gain needs no statistic of the row
      float g[8], o[8];
      load8(gain + c, g);
#pragma unroll
      for (int j = 0; j < 8; ++j) o[j] = t[j] * g[j];
      store8(xr + c, o);
    }
  };
#pragma unroll
  for (int i = 0; i < KEEP; ++i) {
    const int c = threadIdx.x * 8 + i * 2048;
    if (c < d) first_pass(c, v[i]);
  }
  for (int c = threadIdx.x * 8 + KEEP * 2048; c < d; c += 2048) {
    float t[8];
    first_pass(c, t);
  }
  ss = block_sum_256(ss, s8);
  if (ssq) {
    if (threadIdx.x == 0) ssq[r] = ss;
    return;
  }
  const float inv = rsqrtf(ss / static_cast<float>(d) + eps);
  auto second_pass = [&](int c, float (&t)[8]) {
    float g[8];
    load8(gain + c, g);
#pragma unroll
    for (int j = 0; j < 8; ++j) t[j] = t[j] * inv * g[j];
    store8(xr + c, t);
  };
#pragma unroll
  for (int i = 0; i < KEEP; ++i) {
    const int c = threadIdx.x * 8 + i * 2048;
    if (c < d) second_pass(c, v[i]);
  }
  for (int c = threadIdx.x * 8 + KEEP * 2048; c < d; c += 2048) {
    float t[8];
    load8(hr + c, t);
    second_pass(c, t);
  }
}

__device__ __forceinline__ void store4(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(__nv_bfloat16* p, float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&lo);
  v.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = v;
}
__device__ __forceinline__ void store4(__half* p, float a, float b, float c, float d) {
  __half2 lo = __floats2half2_rn(a, b), hi = __floats2half2_rn(c, d);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&lo);
  v.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = v;
}
__device__ __forceinline__ void add4(float4& a, const float4 b) {
  a.x += b.x;
  a.y += b.y;
  a.z += b.z;
  a.w += b.w;
}

// h[r] += sum_s part[s][r];  xn[r] = RMSNorm(h[r]) * gain     (one CTA per row;
// float4 accesses, d a multiple of 4; up to 4 x 256 float4 per pass are kept in
// flight per thread block so the split-K partials are read with wide parallelism)
// ssq != NULL: xn[r] = h[r] .* gain and ssq[r] = sum h[r]^2 instead (the consuming GEMM divides by the RMS).
template <typename T>
__global__ void __launch_bounds__(256)
k_resid_norm(float* __restrict__ h, const float* __restrict__ part, int splits, long long split_stride,
             const int* __restrict__ r_dev, const float* __restrict__ gain, float eps, int d,
             T* __restrict__ xn, float* __restrict__ ssq) {
  __shared__ float s8[8];
  pdl_enter(7);
  const int r = blockIdx.x;
  if (r >= *r_dev) return;
  const int nvec = d >> 2;
  float4* hr = reinterpret_cast<float4*>(h + static_cast<long long>(r) * d);
  const float4* pr = reinterpret_cast<const float4*>(part + static_cast<long long>(r) * d);
  const long long stride4 = split_stride >> 2;
  float ss = 0.f;
  float4 acc[4];     // after the loop: the row's values of the last (for d <= 4096 the only) pass
  int idx[4];
  const float4* g4 = reinterpret_cast<const float4*>(gain);
  float4 gv[4];
  for (int base = 0; base < nvec; base += 4 * 256) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      idx[j] = base + j * 256 + threadIdx.x;
      acc[j] = idx[j] < nvec ? hr[idx[j]] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // all partials of a group of up to nine splits are requested before the first is added: the
    // kernel is bound by how many loads it keeps in flight, not by their number
    for (int s0 = 0; s0 < splits; s0 += 9) {
      float4 v[9][4];
#pragma unroll
      for (int u = 0; u < 9; ++u) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          v[u][j] = (s0 + u < splits && idx[j] < nvec) ? pr[(s0 + u) * stride4 + idx[j]] : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 9; ++u) {
#pragma unroll
        for (int j = 0; j < 4; ++j) add4(acc[j], v[u][j]);
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (idx[j] < nvec) {
        hr[idx[j]] = acc[j];
        ss += acc[j].x * acc[j].x + acc[j].y * acc[j].y + acc[j].z * acc[j].z + acc[j].w * acc[j].w;
        gv[j] = g4[idx[j]];          // in flight during the block reduction
      }
    }
  }
  ss = block_sum_256(ss, s8);
  float inv = rsqrtf(ss / static_cast<float>(d) + eps);
  if (ssq) {
    if (threadIdx.x == 0) ssq[r] = ss;
    inv = 1.f;
  }
  T* xr = xn + static_cast<long long>(r) * d;
  if (nvec <= 4 * 256) {
    // one pass held the whole row: normalise from registers instead of reading h back
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (idx[j] < nvec)
        store4(xr + 4 * idx[j], acc[j].x * inv * gv[j].x, acc[j].y * inv * gv[j].y, acc[j].z * inv * gv[j].z,
               acc[j].w * inv * gv[j].w);
    return;
  }
  for (int i = threadIdx.x; i < nvec; i += 256) {
    const float4 v = hr[i];
    const float4 g = g4[i];
    store4(xr + 4 * i, v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
  }
}

// Split-K reduction of the QKV projection, RoPE on q and k at the row's
// original position, q to the compact buffer, k and v into the row's own
// cache slot [b][kv_head][pos][d_h].  grid (rows, y): the y blocks of a row stride over its units; one unit =
// 4 consecutive rotation pairs of one q/k head, or 4 consecutive v columns.
template <typename T>
__global__ void __launch_bounds__(256)
k_qkv_rope_scatter(const float* __restrict__ part, int splits, long long split_stride,
                   const int* __restrict__ r_dev, const int32_t* __restrict__ act_idx,
                   const float2* __restrict__ rope_tab, int seq_len, int n_q_heads, int n_kv_heads, int head_dim,
                   T* __restrict__ q, T* __restrict__ k_slots, T* __restrict__ v_slots) {
  pdl_enter(4);
  const int r = blockIdx.x;
  if (r >= *r_dev) return;
  const int half = head_dim >> 1;
  const int upr = half >> 2;                                  // units per q/k head
  const int units_qk = (n_q_heads + n_kv_heads) * upr;
  const int d_q = n_q_heads * head_dim, d_kv = n_kv_heads * head_dim;
  const int units = units_qk + (d_kv >> 2);
  const int flat = act_idx[r];
  const int b = flat / seq_len, pos = flat % seq_len;
  const int ncol = d_q + 2 * d_kv;
  const float* pr = part + static_cast<long long>(r) * ncol;
  for (int u = blockIdx.y * 256 + threadIdx.x; u < units; u += gridDim.y * 256) {
  if (u < units_qk) {
    const int hh = u / upr, i = (u % upr) * 4;
    const int col = hh * head_dim + i;                        // q heads first, then k heads
    float4 x1 = make_float4(0.f, 0.f, 0.f, 0.f), x2 = x1;
    for (int s = 0; s < splits; ++s) {
      add4(x1, *reinterpret_cast<const float4*>(pr + s * split_stride + col));
      add4(x2, *reinterpret_cast<const float4*>(pr + s * split_stride + col + half));
    }
    const float4* tab = reinterpret_cast<const float4*>(rope_tab + static_cast<long long>(pos) * half + i);
    const float4 t0 = tab[0], t1 = tab[1];                    // (cos, sin) of i, i+1 | i+2, i+3
    T* dst = (hh < n_q_heads)
                 ? q + static_cast<long long>(r) * d_q + hh * head_dim
                 : k_slots + ((static_cast<long long>(b) * n_kv_heads + (hh - n_q_heads)) * seq_len + pos) * head_dim;
    store4(dst + i, x1.x * t0.x - x2.x * t0.y, x1.y * t0.z - x2.y * t0.w, x1.z * t1.x - x2.z * t1.y,
           x1.w * t1.z - x2.w * t1.w);
    store4(dst + i + half, x2.x * t0.x + x1.x * t0.y, x2.y * t0.z + x1.y * t0.w, x2.z * t1.x + x1.z * t1.y,
           x2.w * t1.z + x1.w * t1.w);
  } else {
    const int e = (u - units_qk) * 4;
    const int hk = e / head_dim, i = e % head_dim;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < splits; ++s) add4(v, *reinterpret_cast<const float4*>(pr + s * split_stride + d_q + d_kv + e));
    store4(v_slots + ((static_cast<long long>(b) * n_kv_heads + hk) * seq_len + pos) * head_dim + i, v.x, v.y, v.z,
           v.w);
  }
  }
}

// u[r, j] = SiLU(gate[r, j]) * up[r, j] from the split-K partials of [gate | up];
// grid (rows, y): the y blocks of a row stride over groups of 4 consecutive columns.
// tiled = blk > 0: the columns are regrouped [blk gate | blk up] per 2 * blk (the weight layout of the fused epilogue).
template <typename T>
__global__ void __launch_bounds__(256)
k_swiglu(const float* __restrict__ part, int splits, long long split_stride, const int* __restrict__ r_dev, int f,
         int tiled, T* __restrict__ u) {
  pdl_enter(9);
  const int r = blockIdx.x;
  if (r >= *r_dev) return;
  const float* pr = part + static_cast<long long>(r) * (2 * f);
  for (int j = (blockIdx.y * 256 + threadIdx.x) * 4; j < f; j += gridDim.y * 1024) {
  const int cg = tiled ? (j / tiled) * 2 * tiled + (j % tiled) : j;   // column of gate_j
  const int cu = tiled ? cg + tiled : f + j;                          // column of up_j
  float4 g = make_float4(0.f, 0.f, 0.f, 0.f), up = g;
  for (int s = 0; s < splits; ++s) {
    add4(g, *reinterpret_cast<const float4*>(pr + s * split_stride + cg));
    add4(up, *reinterpret_cast<const float4*>(pr + s * split_stride + cu));
  }
  store4(u + static_cast<long long>(r) * f + j, g.x / (1.f + expf(-g.x)) * up.x, g.y / (1.f + expf(-g.y)) * up.y,
         g.z / (1.f + expf(-g.z)) * up.z, g.w / (1.f + expf(-g.w)) * up.w);
  }
}

// xh[i] = xn[head_row[i]] for i < n_head (device count), 16-byte copies (d a multiple of 8 elements of
// 2 bytes, or of 4 floats).  With ssq != NULL (xn holds h .* gain) also head_rs[i] = the row's
// 1 / RMS from its ssq_parts partial sums of squares [ssq_parts][ssq_ld].
template <typename T>
__global__ void __launch_bounds__(256)
k_head_gather(const T* __restrict__ xn, const int32_t* __restrict__ head_row, const int* __restrict__ n_head_dev,
              int d, T* __restrict__ xh, const float* __restrict__ ssq, int ssq_parts, long long ssq_ld, float eps,
              float* __restrict__ head_rs) {
  pdl_enter(11);
  const int i = blockIdx.x;
  if (i >= *n_head_dev) return;
  const int row = head_row[i];
  const uint4* src = reinterpret_cast<const uint4*>(xn + static_cast<long long>(row) * d);
  uint4* dst = reinterpret_cast<uint4*>(xh + static_cast<long long>(i) * d);
  const int n16 = d * static_cast<int>(sizeof(T)) / 16;
  for (int c = threadIdx.x; c < n16; c += 256) dst[c] = src[c];
  if (ssq && threadIdx.x == 0) {
    float ss = 0.f;
    for (int t = 0; t < ssq_parts; ++t) ss += ssq[t * ssq_ld + row];
    head_rs[i] = rsqrtf(ss / static_cast<float>(d) + eps);
  }
}

// Sum split-K partials of the head GEMM into the logits buffer (only needed when splits > 1
// or when the caller wants the logits in its own buffer).
__global__ void __launch_bounds__(256)
k_reduce_partials(const float* __restrict__ part, int splits, long long split_stride, int r_bound,
                  const int* __restrict__ r_dev, int n, float* __restrict__ out) {
  pdl_enter(14);
  int rows = r_bound;
  if (r_dev) rows = min(rows, *r_dev);
  const long long total = static_cast<long long>(rows) * n;
  for (long long e = blockIdx.x * 256LL + threadIdx.x; e < total; e += static_cast<long long>(gridDim.x) * 256LL) {
    float v = 0.f;
    for (int s = 0; s < splits; ++s) v += part[s * split_stride + e];
    out[e] = v;
  }
}

constexpr int SCORE_MAXPROB = 0;      // largest softmax probability
constexpr int SCORE_MARGIN = 1;       // difference of the two largest probabilities
constexpr int SCORE_NEG_ENTROPY = 2;  // sum p log p

// From the largest logit m, the second largest m2 (of the other ids),
// S = sum exp(l - m) and T = sum exp(l - m) (l - m): the score the selection ranks.
__device__ __forceinline__ float head_score(int score, float m, float m2, float S, float T) {
  if (score == SCORE_MARGIN) return (1.f - expf(m2 - m)) / S;
  if (score == SCORE_NEG_ENTROPY) return T / S - logf(S);
  return 1.f / S;
}

// Per head row: argmax token (mask_id excluded, lowest id on ties) and the
// score of the row (Sec. 3.1), written at the row's original position.  One
// CTA of 512 threads per head row; logits [n_head, vocab] fp32.
__global__ void __launch_bounds__(512)
k_head_stats(const float* __restrict__ logits, const int* __restrict__ n_head_dev,
             const int32_t* __restrict__ head_pos, int vocab, int mask_id, int score, float* __restrict__ conf,
             int32_t* __restrict__ pred) {
  __shared__ float s_m[16];
  __shared__ int s_i[16];
  __shared__ float s_s[16], s_t[16], s_m2[16];
  pdl_enter(12);
  const int i = blockIdx.x;
  if (i >= *n_head_dev) return;
  const float* l = logits + static_cast<long long>(i) * vocab;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float m = -CUDART_INF_F;
  int mi = 0x7fffffff;
  for (int c = tid; c < vocab; c += 512) {
    if (c == mask_id) continue;
    const float v = l[c];
    if (v > m || (v == m && c < mi)) {
      m = v;
      mi = c;
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const int oi = __shfl_xor_sync(0xffffffffu, mi, o);
    if (om > m || (om == m && oi < mi)) {
      m = om;
      mi = oi;
    }
  }
  if (lane == 0) {
    s_m[warp] = m;
    s_i[warp] = mi;
  }
  __syncthreads();
  m = s_m[0];
  mi = s_i[0];
  for (int w = 1; w < 16; ++w) {
    if (s_m[w] > m || (s_m[w] == m && s_i[w] < mi)) {
      m = s_m[w];
      mi = s_i[w];
    }
  }
  float s = 0.f, t = 0.f, m2 = -CUDART_INF_F;
  for (int c = tid; c < vocab; c += 512) {
    if (c == mask_id) continue;
    const float v = l[c];
    const float e = expf(v - m);
    s += e;
    t += e * (v - m);
    if (c != mi) m2 = fmaxf(m2, v);
  }
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    t += __shfl_xor_sync(0xffffffffu, t, o);
    m2 = fmaxf(m2, __shfl_xor_sync(0xffffffffu, m2, o));
  }
  if (lane == 0) {
    s_s[warp] = s;
    s_t[warp] = t;
    s_m2[warp] = m2;
  }
  __syncthreads();
  if (tid == 0) {
    float S = 0.f, T = 0.f, M2 = -CUDART_INF_F;
    for (int w = 0; w < 16; ++w) {
      S += s_s[w];
      T += s_t[w];
      M2 = fmaxf(M2, s_m2[w]);
    }
    const int flat = head_pos[i];
    conf[flat] = head_score(score, m, M2, S, T);
    pred[flat] = mi;
  }
}

// Combine the statistics the head GEMM left per CTA and lane quarter (arrays [n_groups][ld], one column
// per head row): one pass per head row with an online merge per thread, then a merge across the block; the score is
// written at the row's original position.  One CTA of 256 threads per row.  The launch asks for enough
// dynamic shared memory that an SM holds one block: launched early behind the head GEMM, the blocks would
// otherwise pile up on the few SMs with room and run several times longer.
__global__ void __launch_bounds__(256)
k_head_combine(const float* __restrict__ st_max, const float* __restrict__ st_sum, const int* __restrict__ st_arg,
               const float* __restrict__ st_m2, const float* __restrict__ st_t, int score, int n_groups, int ld,
               const int* __restrict__ n_head_dev, const int32_t* __restrict__ head_pos, float* __restrict__ conf,
               int32_t* __restrict__ pred) {
  __shared__ HeadStat s_w[8];
  pdl_enter(15);
  const int i = blockIdx.x;
  if (i >= *n_head_dev) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  HeadStat acc = head_stat_empty();
  for (int g0 = tid; g0 < n_groups; g0 += 4 * 256) {
    // four groups' loads in flight before any is merged
    HeadStat v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int g = g0 + u * 256;
      v[u] = head_stat_empty();
      if (g < n_groups) {
        const long long at = static_cast<long long>(g) * ld + i;
        v[u].m = __ldcg(st_max + at);
        v[u].arg = __ldcg(st_arg + at);
        v[u].s = __ldcg(st_sum + at);
        if (score != SCORE_MAXPROB) {
          v[u].m2 = __ldcg(st_m2 + at);
          v[u].t = __ldcg(st_t + at);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) acc = head_stat_merge(acc, v[u]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc = head_stat_merge(acc, head_stat_shfl_xor(acc, o));
  if (lane == 0) s_w[warp] = acc;
  __syncthreads();
  if (tid == 0) {
    HeadStat r = s_w[0];
    for (int w = 1; w < 8; ++w) r = head_stat_merge(r, s_w[w]);
    const int flat = head_pos[i];
    conf[flat] = head_score(score, r.m, r.m2, r.s, r.t);
    pred[flat] = r.arg;
  }
}

}  // namespace dkv
