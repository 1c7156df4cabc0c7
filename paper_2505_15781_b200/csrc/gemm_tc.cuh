// Projection GEMM on tcgen05 tensor cores (both operands bf16, or both fp16;
// fp32 accumulate in TMEM).
//
// out[r, n] = sum_k x[r, k] * w[n, k]       x [rows, K], w [N, K], both K-major.
//
// The weight matrix is the MMA "A" operand (128 weight rows = 128 TMEM lanes
// per MMA, `halves` MMAs side by side = 128 or 256 weight rows per tile) and
// the active rows of the step are the MMA "B" operand (br rows = br TMEM
// columns, a runtime multiple of 16).  With few active rows this is a
// weight-streaming kernel: every weight byte is pulled through a deep TMA ring
// exactly once, whatever the number of rows (up to 256 per tile); a 256-row
// weight tile halves how often the activation rows are re-read from L2.
//
// The kernel is persistent: CTA i works on units i, i + gridDim.x, ... where a
// unit is (weight tile, row tile, K split).  The TMA ring keeps running across
// units and, when tensor memory has room for two accumulators, the epilogue of
// one unit overlaps the main loop of the next.
//
// Epilogues.  Every mode can scale row r of the result by a per-row factor (the
// RMSNorm of the operand applied AFTER the product: norm(h) W^T = (h .* g) W^T / rms(h), so the
// producer of the operand writes h .* g and the sums of squares, and this kernel divides).  Beyond
// the plain fp32 partial sums there are fused row epilogues that need the COMPLETE sum over K and
// a whole head or row: the CTAs that share a weight tile (its K splits) first leave their partial
// sums in scratch (they stay in L2), count themselves on a per-tile counter, wait for the others
// (a bounded spin: all CTAs of such a launch are resident at once, the host launches this mode
// only when units <= SMs), and then each of them finishes a slice of the tile's rows:
//   FUSE_RESID  h += sum; the row's sum of squares over the tile's columns; h .* gain as the
//               next GEMM's 16-bit operand  (residual + RMSNorm around the O and down projections)
//   FUSE_QKV    sum -> RoPE at the row's original position -> q to the compact buffer, k and v
//               into the row's own cache slot  (Algorithm 1: the fresh K/V join the cache)
// so the split-K reduction, the residual, the norm statistics, RoPE and the K/V scatter need no
// kernel of their own.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = TMEM allocation and
// MMA issue, warps 2..9 = epilogue: two warps per TMEM lane quarter, which take
// alternate 16-column groups of the accumulator (the epilogue of a launch with
// one unit per CTA is a dependent chain of tensor-memory loads and stores per
// warp; eight warps halve it).
#pragma once
#include "head_stat.cuh"
#include "pdl.cuh"
#include "ptx.cuh"

namespace dkv {

constexpr int GEMM_BM = 128;  // weight rows per MMA (MMA M)
constexpr int GEMM_BK = 64;   // 16-bit elements per k-block (= one 128-byte swizzle row)
constexpr int GEMM_THREADS = 320;   // TMA warp, MMA warp, 8 epilogue warps
constexpr long long GEMM_WAIT_CYCLES = 4000000000LL;  // ~2 s at 2 GHz: far beyond any legitimate wait

constexpr int DEV_ERR_ROWS_BOUND = 1;   // status bit: more active rows than the caller's bound
constexpr int DEV_ERR_FEW_CAND = 2;     // fewer candidates than k
constexpr int DEV_ERR_HEAD_ROW = 4;     // a head row is not an active row
constexpr int DEV_ERR_WAIT = 8;         // a bounded wait inside a kernel ran out

constexpr int GEMM_A_BYTES = GEMM_BM * GEMM_BK * 2;  // 16 KB of weights per 128-row half per stage
constexpr int GEMM_MAX_STAGES = 12;
constexpr int GEMM_BAR_BYTES = 512;      // barriers, the TMEM slot and the abort flag
constexpr int GEMM_SCALE_BYTES = 1024;   // per-row scales of the unit's row tile (256 floats)

constexpr int FUSE_NONE = 0;
constexpr int FUSE_RESID = 1;
constexpr int FUSE_QKV = 2;

// Shared/tensor-memory plan for a row tile of `br` rows (a multiple of 16, at
// most 256) and `halves` (1 or 2) 128-row weight halves per tile.
struct GemmTcPlan {
  int br, halves, stage_bytes, stages, col_stride, n_bufs, tmem_cols, smem_bytes, ctas_per_sm;
};
inline GemmTcPlan gemm_tc_plan(int br, int halves, int ctas_per_sm) {
  GemmTcPlan p;
  p.br = br;
  p.halves = halves;
  p.stage_bytes = halves * GEMM_A_BYTES + br * GEMM_BK * 2;
  p.col_stride = 32;
  while (p.col_stride < br) p.col_stride *= 2;
  // 512 TMEM columns per SM, shared by the CTAs resident on it
  if (halves * p.col_stride > 512 / ctas_per_sm) ctas_per_sm = 1;
  const int tmem_budget = 512 / ctas_per_sm;
  p.n_bufs = (2 * halves * p.col_stride <= tmem_budget) ? 2 : 1;
  p.tmem_cols = p.n_bufs * halves * p.col_stride;     // a power of two >= 32
  const int budget = (ctas_per_sm >= 2 ? 110 : 220) * 1024;
  p.stages = budget / p.stage_bytes;
  if (p.stages > GEMM_MAX_STAGES) p.stages = GEMM_MAX_STAGES;
  if (p.stages < 2) p.stages = 2;
  p.smem_bytes = p.stages * p.stage_bytes + 1024 /*alignment slack*/ + GEMM_BAR_BYTES + GEMM_SCALE_BYTES;
  p.ctas_per_sm = ctas_per_sm;
  return p;
}

struct GemmTcParams {
  int n;                   // weight rows (output features)
  int kb_total;            // ceil(K / 64)
  int kb_per_split;        // k-blocks per split (the last split may have fewer)
  int splits;
  int r_bound;             // host-side bound on the rows
  const int* r_dev;        // exact row count on the device (nullable)
  float* out;              // [splits][split_stride] partial sums, row stride ldo
  long long split_stride;  // in floats
  int ldo;
  int* status;             // device status word (nullable)
  int x_bf16;              // 16-bit format of BOTH operands: 1 = bf16, 0 = fp16
  int br;                  // rows per tile (MMA N): multiple of 16, <= 256; equals the row box of tm_x
  int halves;              // 128-row weight halves per tile: 1 or 2
  int stages, stage_bytes;
  int col_stride;          // TMEM columns per accumulator (power of two >= br)
  int n_bufs;              // accumulator buffers in TMEM: 1 or 2
  int tmem_cols;           // TMEM allocation = n_bufs * halves * col_stride
  int r_tiles;             // ceil(r_bound / br)
  int units;               // weight tiles * r_tiles * splits
  // SwiGLU mode (halves = 2, splits = 1, weight tiles = [128 gate rows | 128 up rows]): the epilogue
  // combines the two accumulators of a thread and writes u = SiLU(gate) * up as 16-bit [r][ld_u]
  void* swiglu_out;
  int ld_u;
  // vocabulary-head mode: instead of the products, each epilogue warp writes, for its 32 weight
  // rows (= 32 token ids) and every row r, the largest logit, its id and sum exp(logit - max)
  int head_mode;
  int mask_id;             // token id left out of the statistics
  float* st_max;           // [4 * gridDim.x][r_bound]: per CTA and lane quarter, over all its weight tiles
  float* st_sum;
  int* st_arg;
  float* st_m2;            // second largest logit of the 32 ids (scores other than the max probability)
  float* st_t;             // sum exp(l - max)(l - max)
  int w_blocked;           // 1: tm_w maps a copy stored in 128 x 64 blocks, [ceil(n / 128)][kb_total] of them
  int w_static;            // 1: the weights were complete long before this launch, so they may be
                           // fetched before the wait on the stream predecessor
  // per-row scale of the result: NULL = none; rs_parts > 0: rs_src is [rs_parts][rs_ld] partial sums of
  // squares of the operand rows and the scale is rsqrt(sum / rs_d + rs_eps); rs_parts == 0: rs_src [rows]
  // holds the ready factors
  const float* rs_src;
  int rs_parts;
  long long rs_ld;
  float rs_inv_d, rs_eps;
  // fused row epilogue across the CTAs of a weight tile (FUSE_*); needs units <= resident CTAs
  int fuse_mode;
  unsigned int* tile_cnt;  // this launch's arrival counters, one per (weight tile, row tile): all zero at its start
  unsigned int* tile_cnt_next;   // the other set of counters (256): the previous fused launch's, zeroed by this
                                 // launch for the next one, so that no counter has to be reset behind a wait
  long long tail_wait_cycles;  // bound of the wait for the tile's other CTAs (GEMM_WAIT_CYCLES unless a test shortens it)
  int tail_extra;          // arrivals expected beyond the tile's K splits: 0; a test of the error path sets 1,
                           // so that the wait can only run out
  // FUSE_RESID
  float* h;                // [rows][n] residual stream, updated in place
  const float* gain;       // [n] gains of the norm that follows
  void* xn_out;            // [rows][n] 16-bit: h .* gain
  float* ssq_out;          // [weight tiles][ssq_ld]: each row's sum of squares over the tile's columns
  long long ssq_ld;
  // FUSE_QKV (n = (n_q_heads + 2 n_kv_heads) * head_dim, heads never straddle a weight tile)
  const int32_t* act_idx;  // [rows] flattened position b * seq_len + pos of each row
  const float2* rope_tab;  // [seq_len][head_dim / 2] (cos, sin)
  int seq_len, n_q_heads, n_kv_heads, head_dim;
  void* q_out;             // [rows][n_q_heads * head_dim] 16-bit
  void* k_slots;           // [batch][n_kv_heads][seq_len][head_dim] 16-bit, this layer
  void* v_slots;
};

__device__ __forceinline__ void named_bar_sync(int id, int n_threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint16_t to_bits16(float v, int bf16) {
  return bf16 ? __bfloat16_as_ushort(__float2bfloat16_rn(v)) : __half_as_ushort(__float2half_rn(v));
}
__device__ __forceinline__ uint2 pack4_16(float a, float b, float c, float d, int bf16) {
  uint2 o;
  if (bf16) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    o.x = *reinterpret_cast<uint32_t*>(&lo);
    o.y = *reinterpret_cast<uint32_t*>(&hi);
  } else {
    __half2 lo = __floats2half2_rn(a, b), hi = __floats2half2_rn(c, d);
    o.x = *reinterpret_cast<uint32_t*>(&lo);
    o.y = *reinterpret_cast<uint32_t*>(&hi);
  }
  return o;
}

// Second phase of the fused row epilogues, run by the 8 epilogue warps of every CTA of a weight tile
// once all K splits of the tile have left their partial sums in scratch: this CTA finishes rows
// [row_lo, row_hi) of the tile.  One warp per row, each lane two groups of four columns; a warp works
// on FUSE_ROWS rows at once and requests the partials of four splits of all of them before it adds any
// (the phase is bound by how many L2 loads are in flight, not by their number).
constexpr int FUSE_ROWS = 2;

// sums over the K splits of the float4 at element offset at[i] (i < FUSE_ROWS * 2), added onto acc[i];
// the partials of up to five splits of all four items are requested before any is added
constexpr int FUSE_BATCH = 5;
__device__ __forceinline__ void sum_splits(const GemmTcParams& p, const long long (&at)[FUSE_ROWS * 2],
                                           const bool (&on)[FUSE_ROWS * 2], float4 (&acc)[FUSE_ROWS * 2]) {
  for (int s0 = 0; s0 < p.splits; s0 += FUSE_BATCH) {
    float4 v[FUSE_BATCH][FUSE_ROWS * 2];
#pragma unroll
    for (int u = 0; u < FUSE_BATCH; ++u) {
#pragma unroll
      for (int i = 0; i < FUSE_ROWS * 2; ++i)
        v[u][i] = (on[i] && s0 + u < p.splits)
                      ? __ldcg(reinterpret_cast<const float4*>(p.out + (s0 + u) * p.split_stride + at[i]))
                      : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < FUSE_BATCH; ++u) {
#pragma unroll
      for (int i = 0; i < FUSE_ROWS * 2; ++i) {
        acc[i].x += v[u][i].x;
        acc[i].y += v[u][i].y;
        acc[i].z += v[u][i].z;
        acc[i].w += v[u][i].w;
      }
    }
  }
}

// (`g`: the lane's gains, loaded by the caller before the wait for the tile's splits — nothing that does
// not depend on the sums may add a round trip through L2 after them)
__device__ __forceinline__ void fused_rows_resid(const GemmTcParams& p, int n0, int tile_rows, int row_lo, int row_hi,
                                                 int ewarp, int lane, const float4 (&g)[2]) {
  const int tile_n = n0 / tile_rows;
  for (int rb = row_lo + ewarp * FUSE_ROWS; rb < row_hi; rb += 8 * FUSE_ROWS) {
    long long at[FUSE_ROWS * 2];
    bool on[FUSE_ROWS * 2];
    float4 acc[FUSE_ROWS * 2];
#pragma unroll
    for (int i = 0; i < FUSE_ROWS * 2; ++i) {
      const int r = rb + (i >> 1), n = n0 + (i & 1) * 128 + lane * 4;
      on[i] = r < row_hi && (i & 1) * 128 < tile_rows && n < p.n;
      at[i] = static_cast<long long>(r) * p.ldo + n;
      acc[i] = on[i] ? __ldcg(reinterpret_cast<const float4*>(p.h + at[i])) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    sum_splits(p, at, on, acc);
#pragma unroll
    for (int rr = 0; rr < FUSE_ROWS; ++rr) {
      float ss = 0.f;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int i = rr * 2 + hf;
        if (on[i]) {
          const float4 a = acc[i];
          *reinterpret_cast<float4*>(p.h + at[i]) = a;
          ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
          *reinterpret_cast<uint2*>(static_cast<uint16_t*>(p.xn_out) + at[i]) =
              pack4_16(a.x * g[hf].x, a.y * g[hf].y, a.z * g[hf].z, a.w * g[hf].w, p.x_bf16);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (lane == 0 && rb + rr < row_hi && n0 < p.n) p.ssq_out[tile_n * p.ssq_ld + rb + rr] = ss;   // (a pair's second CTA may own no column)
    }
  }
}

// A tile of 256 columns holds 256 / head_dim whole heads and a head's rotation pairs are (i, i + head_dim/2):
// head_dim / 8 lanes per head, each with pairs i..i+3, is exactly one warp per row (head_dim 64 or 128).
// `flat0`: the flattened positions of the warp's first FUSE_ROWS rows, loaded by the caller before the
// wait for the tile's splits; the positions of the next pass are requested while this pass runs, and
// a pass asks for its rotation factors BEFORE its partial sums: neither the position nor the table
// entry may add a round trip through L2 after the sums.
__device__ __forceinline__ void fused_rows_qkv(const GemmTcParams& p, int n0, int tile_rows, int row_lo, int row_hi,
                                               int ewarp, int lane, const int (&flat0)[FUSE_ROWS]) {
  const int hd = p.head_dim, half = hd >> 1;
  const int lanes_per_head = hd >> 3;
  const int hh = lane / lanes_per_head, i0 = (lane - hh * lanes_per_head) * 4;
  const int col0 = n0 + hh * hd;                         // first column of this lane's head
  const bool head_on = hh * hd < tile_rows && col0 < p.n;
  const int head = col0 / hd;                            // q heads, then k heads, then v heads
  const int d_q = p.n_q_heads * hd;
  const bool is_q = head < p.n_q_heads;
  const bool rot = head < p.n_q_heads + p.n_kv_heads;
  const int hk = head - p.n_q_heads - (rot ? 0 : p.n_kv_heads);
  int flat_next[FUSE_ROWS];
#pragma unroll
  for (int rr = 0; rr < FUSE_ROWS; ++rr) flat_next[rr] = flat0[rr];
  for (int rb = row_lo + ewarp * FUSE_ROWS; rb < row_hi; rb += 8 * FUSE_ROWS) {
    long long at[FUSE_ROWS * 2];
    bool on[FUSE_ROWS * 2];
    float4 acc[FUSE_ROWS * 2];
    int bq[FUSE_ROWS], posq[FUSE_ROWS];
    float4 t0q[FUSE_ROWS], t1q[FUSE_ROWS];
#pragma unroll
    for (int rr = 0; rr < FUSE_ROWS; ++rr) {
      const int flat = flat_next[rr];
      const int rn = rb + 8 * FUSE_ROWS + rr;                  // the same warp's row of the next pass
      flat_next[rr] = rn < row_hi ? p.act_idx[rn] : 0;
      bq[rr] = flat / p.seq_len;
      posq[rr] = flat - bq[rr] * p.seq_len;
      t0q[rr] = t1q[rr] = make_float4(1.f, 0.f, 1.f, 0.f);
      if (rot && head_on && rb + rr < row_hi) {
        const float4* tab = reinterpret_cast<const float4*>(p.rope_tab + static_cast<long long>(posq[rr]) * half + i0);
        t0q[rr] = __ldg(tab);                                  // (cos, sin) of i0, i0+1
        t1q[rr] = __ldg(tab + 1);                              // (cos, sin) of i0+2, i0+3
      }
    }
#pragma unroll
    for (int i = 0; i < FUSE_ROWS * 2; ++i) {
      const int r = rb + (i >> 1);
      on[i] = head_on && r < row_hi;
      at[i] = static_cast<long long>(r) * p.ldo + col0 + i0 + (i & 1) * half;     // x1 group, x2 group
      acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    sum_splits(p, at, on, acc);
#pragma unroll
    for (int rr = 0; rr < FUSE_ROWS; ++rr) {
      const int r = rb + rr;
      if (!on[rr * 2]) continue;
      const int b = bq[rr], pos = posq[rr];
      float4 x1 = acc[rr * 2], x2 = acc[rr * 2 + 1];
      if (rot) {
        const float4 t0 = t0q[rr], t1 = t1q[rr];
        const float4 y1 = make_float4(x1.x * t0.x - x2.x * t0.y, x1.y * t0.z - x2.y * t0.w,
                                      x1.z * t1.x - x2.z * t1.y, x1.w * t1.z - x2.w * t1.w);
        const float4 y2 = make_float4(x2.x * t0.x + x1.x * t0.y, x2.y * t0.z + x1.y * t0.w,
                                      x2.z * t1.x + x1.z * t1.y, x2.w * t1.z + x1.w * t1.w);
        x1 = y1;
        x2 = y2;
      }
      uint16_t* dst = is_q ? static_cast<uint16_t*>(p.q_out) + static_cast<long long>(r) * d_q + head * hd
                           : static_cast<uint16_t*>(rot ? p.k_slots : p.v_slots) +
                                 ((static_cast<long long>(b) * p.n_kv_heads + hk) * p.seq_len + pos) * hd;
      *reinterpret_cast<uint2*>(dst + i0) = pack4_16(x1.x, x1.y, x1.z, x1.w, p.x_bf16);
      *reinterpret_cast<uint2*>(dst + i0 + half) = pack4_16(x2.x, x2.y, x2.z, x2.w, p.x_bf16);
    }
  }
}

// Cross-CTA hand-over of the fused row epilogues, run by the 256 epilogue threads of a CTA after its
// partial sums of the unit are in scratch: the CTA counts itself on the tile's counter and waits
// (bounded) until all K splits of the tile are there; then it finishes its own slice of the tile's
// rows.  `tile` indexes the counters; the tile's columns are [n0, n0 + tile_rows).  The counters are
// not reset here: fused launches alternate between two sets, and each zeroes the other set once its
// predecessors have completed.  Returns false when a wait ran out (the abort flag is set).
__device__ __forceinline__ bool fused_tail(const GemmTcParams& p, int tile, int split, int n0, int tile_rows, int r0,
                                           int r_valid, volatile int* abort_flag, int et, int ewarp, int lane) {
  unsigned int* cnt = p.tile_cnt + tile;
  // this CTA's share of the tile's rows, and what its warps need beside the sums (gains; the first
  // rows' positions), requested before the wait
  const int n_rows = max(0, min(p.br, r_valid - r0));
  const int per = (n_rows + p.splits - 1) / p.splits;
  const int row_lo = r0 + min(n_rows, split * per), row_hi = r0 + min(n_rows, (split + 1) * per);
  float4 gains[2];
  int flat0[FUSE_ROWS];
#pragma unroll
  for (int hf = 0; hf < 2; ++hf) {
    const int n = n0 + hf * 128 + lane * 4;
    gains[hf] = (p.fuse_mode == FUSE_RESID && hf * 128 < tile_rows && n < p.n)
                    ? __ldg(reinterpret_cast<const float4*>(p.gain + n))
                    : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int rr = 0; rr < FUSE_ROWS; ++rr) {
    const int r = row_lo + ewarp * FUSE_ROWS + rr;
    flat0[rr] = (p.fuse_mode == FUSE_QKV && r < row_hi) ? p.act_idx[r] : 0;
  }
  __threadfence();
  named_bar_sync(2, 256);
  bool fail = false;
  if (et == 0) {
    atomicAdd(cnt, 1u);
    const long long t0 = clock64();
    while (ld_acquire_gpu(cnt) < static_cast<unsigned int>(p.splits + p.tail_extra)) {
      if (*abort_flag || clock64() - t0 > p.tail_wait_cycles) {
        fail = true;
        *abort_flag = 1;
        break;
      }
    }
  }
  // (thread 0's acquire and the barrier order the other splits' sums before every thread's loads)
  if (bar_red_or(2, 256, fail)) return false;
  if (p.fuse_mode == FUSE_RESID) fused_rows_resid(p, n0, tile_rows, row_lo, row_hi, ewarp, lane, gains);
  else fused_rows_qkv(p, n0, tile_rows, row_lo, row_hi, ewarp, lane, flat0);
  return true;
}

template <int HALVES>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, GemmTcParams p) {
  const int STAGES = p.stages;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment for the 128-byte swizzle atoms
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * p.stage_bytes);
  // bars: [0,S) full, [S,2S) empty, [2S,2S+2) accumulator full, [2S+2,2S+4) accumulator empty
  uint64_t* acc_full = bars + 2 * STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int a_bytes = HALVES * GEMM_A_BYTES;
  const int tile_rows = HALVES * GEMM_BM;

  // unit u -> (weight tile, row tile, split); consecutive units differ in the split first
  auto decode = [&](int u, int& n0, int& r0, int& split, int& kb0, int& n_kb) {
    split = u % p.splits;
    const int t = u / p.splits;
    r0 = (t % p.r_tiles) * p.br;
    n0 = (t / p.r_tiles) * tile_rows;
    kb0 = split * p.kb_per_split;
    n_kb = max(0, min(p.kb_total, kb0 + p.kb_per_split) - kb0);
  };

  // The TMA producer (thread 0).  The weights never change, so the ring is first filled with weight
  // tiles alone; only the activation rows have to wait for the kernel that produces them.  That first
  // fill needs nothing but the producer's own barriers: it is issued before the CTA's set-up
  // (tensor-memory allocation, the block-wide barrier) completes.
  const uint64_t pol_w = l2_policy_evict_first();   // weights are streamed once per step
  const uint64_t pol_x = l2_policy_evict_last();    // the few activation rows are re-read by every CTA
  struct Cursor {
    int u, i, n0, r0, split, kb0, n_kb;
    bool decoded;      // the unit's fields are valid (the divisions of decode() run once per unit, not per k-block)
  } cur, head;
  cur.u = blockIdx.x;
  cur.i = 0;
  cur.decoded = false;
  auto settle = [&](Cursor& c) {   // move to the next k-block that exists (or past the end)
    while (c.u < p.units) {
      if (!c.decoded) {
        decode(c.u, c.n0, c.r0, c.split, c.kb0, c.n_kb);
        c.decoded = true;
      }
      if (c.i < c.n_kb) return true;
      c.u += gridDim.x;
      c.i = 0;
      c.decoded = false;
    }
    return false;
  };
  auto load_a = [&](const Cursor& c, int s) {
    const uint32_t full = smem_u32(&bars[s]);
    mbar_expect_tx(full, static_cast<uint32_t>(p.stage_bytes));
    const uint32_t a_dst = smem_base + s * p.stage_bytes;
    for (int h = 0; h < HALVES; ++h)
      if (p.w_blocked)      // block (row block, k-block) of a blocked copy: rows block * 128 .. + 127 of its map
        tma_load_2d_hint(a_dst + h * GEMM_A_BYTES, &tm_w, full, 0,
                         (c.n0 + h * GEMM_BM) * p.kb_total + (c.kb0 + c.i) * GEMM_BM, pol_w);
      else
        tma_load_2d_hint(a_dst + h * GEMM_A_BYTES, &tm_w, full, (c.kb0 + c.i) * GEMM_BK, c.n0 + h * GEMM_BM, pol_w);
  };
  auto load_b = [&](const Cursor& c, int s) {
    tma_load_2d_hint(smem_base + s * p.stage_bytes + a_bytes, &tm_x, smem_u32(&bars[s]), (c.kb0 + c.i) * GEMM_BK,
                     c.r0, pol_x);
  };
  head = cur;
  int pre = 0;

  pdl_launch();   // the next kernel in the stream may start its own prologue
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tm_w);
    tma_prefetch_desc(&tm_x);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[STAGES + s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&acc_full[b]), 1);
      mbar_init(smem_u32(&acc_empty[b]), 8);   // one arrival per epilogue warp
    }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
    Cursor c = cur;
    while (p.w_static && pre < STAGES && settle(c)) {   // all stages are free at the start: no wait needed
      load_a(c, pre);
      ++pre;
      ++c.i;
    }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // (only the one recording thread looks at the trace switch, a word in global memory: the single-thread
  // roles must not wait for that load)
  const unsigned long long t_enter = (threadIdx.x == 64 && trace_on()) ? global_timer_ns() : 0ull;

  if (warp == 0) {
    // ------------------------------------------------------- TMA producer
    if (lane == 0) {
      pdl_wait();
      Cursor c = head;
      for (int it = 0; it < pre; ++it) {
        settle(c);
        load_b(c, it);
        ++c.i;
      }
      // ring position without divisions: stage s, phase bit ph (flips on every wrap)
      int s = pre == STAGES ? 0 : pre;
      uint32_t ph = pre == STAGES ? 1u : 0u;
      bool ok = true;
      while (ok && settle(c)) {
        ok = mbar_wait_bounded(smem_u32(&bars[STAGES + s]), ph ^ 1, abort_flag, GEMM_WAIT_CYCLES);
        if (!ok) break;
        load_a(c, s);
        load_b(c, s);
        ++c.i;
        if (++s == STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    // --------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_f16(GEMM_BM, p.br, p.x_bf16);
      int s = 0, j = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x, ++j) {
        int n0, r0, split, kb0, n_kb;
        decode(u, n0, r0, split, kb0, n_kb);
        const int buf = j % p.n_bufs;
        const uint32_t use = static_cast<uint32_t>(j / p.n_bufs);
        // the epilogue must have drained this accumulator buffer (first use passes)
        ok = mbar_wait_bounded(smem_u32(&acc_empty[buf]), (use & 1) ^ 1, abort_flag, GEMM_WAIT_CYCLES);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_base = tmem_base + static_cast<uint32_t>(buf * HALVES * p.col_stride);
        for (int i = 0; i < n_kb; ++i) {
          // everything that depends only on the stage is computed BEFORE the wait: what this thread
          // executes between the arrival of a stage and its MMAs is on the main loop's critical path
          const uint32_t a_addr = smem_base + s * p.stage_bytes;
          const uint64_t bdesc = umma_desc_sw128(a_addr + a_bytes);
          uint64_t adesc[HALVES];
#pragma unroll
          for (int h = 0; h < HALVES; ++h) adesc[h] = umma_desc_sw128(a_addr + h * GEMM_A_BYTES);
          const uint32_t full_bar = smem_u32(&bars[s]), empty_bar = smem_u32(&bars[STAGES + s]);
          const uint32_t acc0 = i > 0 ? 1u : 0u;
          ok = mbar_wait_bounded(full_bar, ph, abort_flag, GEMM_WAIT_CYCLES);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int h = 0; h < HALVES; ++h) {
#pragma unroll
            for (int k4 = 0; k4 < GEMM_BK / 16; ++k4) {
              // advance 16 elements = 32 bytes inside the swizzle row: +2 in the (addr >> 4) field
              umma_f16(d_base + static_cast<uint32_t>(h * p.col_stride), adesc[h] + 2 * k4, bdesc + 2 * k4, idesc,
                       k4 > 0 ? 1u : acc0);
            }
          }
          umma_commit(empty_bar);   // frees the smem stage when the MMAs are done
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (ok) umma_commit(smem_u32(&acc_full[buf]));  // accumulator complete (also when n_kb == 0)
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;           // TMEM lane quarter this warp may read
    const int cs = (warp - 2) >> 2;   // which of the alternating 16-column groups this warp takes
    const int et = threadIdx.x - 64;  // 0..255 among the epilogue threads
    float* s_rs = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + GEMM_BAR_BYTES);   // [256] row scales
    pdl_wait();              // the row count and the output buffer belong to earlier kernels
    // (every earlier launch has completed: the counters of the previous fused launch are free to be
    // zeroed for the next one)
    if (p.fuse_mode != FUSE_NONE && et == 255)
      for (int i = blockIdx.x; i < 256; i += gridDim.x) p.tile_cnt_next[i] = 0u;
    if (threadIdx.x == 64 && trace_on()) trace_store(3, t_enter);
    int r_valid = p.r_bound;
    if (p.r_dev) r_valid = min(r_valid, *p.r_dev);
    // head mode: the statistics of this warp's token ids over ALL weight tiles of the CTA, per row
    // (lane l < 16 keeps row cs * 16 + 32 * i + l in run<i>); written once after the last tile
    HeadStat run0 = head_stat_empty(), run1 = run0, run2 = run0, run3 = run0;
    int j = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x, ++j) {
      int n0, r0, split, kb0, n_kb;
      decode(u, n0, r0, split, kb0, n_kb);
      const int buf = j % p.n_bufs;
      const uint32_t use = static_cast<uint32_t>(j / p.n_bufs);
      // The row scales of this unit's row tile (1 when the launch has none), computed while the MMAs run.
      if (j > 0) named_bar_sync(1, 256);          // everyone is done with the previous unit's scales
      {
        float sc = 1.f;
        const int r = r0 + et;
        if (p.rs_src && r < r_valid) {
          if (p.rs_parts > 0) {
            float ss = 0.f;
            for (int i = 0; i < p.rs_parts; ++i) ss += __ldcg(p.rs_src + i * p.rs_ld + r);
            sc = rsqrtf(ss * p.rs_inv_d + p.rs_eps);
          } else {
            sc = __ldcg(p.rs_src + r);
          }
        }
        s_rs[et] = sc;
      }
      named_bar_sync(1, 256);
      ok = mbar_wait_bounded(smem_u32(&acc_full[buf]), use & 1, abort_flag, GEMM_WAIT_CYCLES);
      if (!ok) break;
      tc_fence_after();
      float* out = p.out + static_cast<long long>(split) * p.split_stride;
      if (p.swiglu_out) {
        // gate and up of feature j live in the same lane and column of the tile's two accumulators
        const int jf = (n0 >> 1) + q * 32 + lane;
        const uint32_t t_gate = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                static_cast<uint32_t>(buf * 2 * p.col_stride);
        const uint32_t t_up = t_gate + static_cast<uint32_t>(p.col_stride);
        for (int c = cs * 16; c < p.br; c += 32) {
          if (r0 + c >= r_valid) break;
          uint32_t vg[16], vu[16];
          tmem_ld_x16(t_gate + c, vg);
          tmem_ld_x16(t_up + c, vu);
          tmem_ld_wait();
          if (jf < p.ld_u) {
            // SiLU with the fast exponential and reciprocal: their error (~2^-21) is far below the
            // 16-bit rounding of the product, and the epilogue is bound by its instruction count
            // (hence also: one pointer, the format test outside the loop, no row test for whole groups)
            uint16_t* dst = static_cast<uint16_t*>(p.swiglu_out) + static_cast<long long>(r0 + c) * p.ld_u + jf;
            const int n_ok = min(16, r_valid - (r0 + c));
            uint16_t bits[16];
            if (p.x_bf16) {
#pragma unroll
              for (int jj = 0; jj < 16; ++jj) {
                const float sc = s_rs[c + jj];
                const float gt = __uint_as_float(vg[jj]) * sc;
                bits[jj] = __bfloat16_as_ushort(__float2bfloat16_rn(__fdividef(gt, 1.f + __expf(-gt)) * (__uint_as_float(vu[jj]) * sc)));
              }
            } else {
#pragma unroll
              for (int jj = 0; jj < 16; ++jj) {
                const float sc = s_rs[c + jj];
                const float gt = __uint_as_float(vg[jj]) * sc;
                bits[jj] = __half_as_ushort(__float2half_rn(__fdividef(gt, 1.f + __expf(-gt)) * (__uint_as_float(vu[jj]) * sc)));
              }
            }
            if (n_ok == 16) {
#pragma unroll
              for (int jj = 0; jj < 16; ++jj) dst[static_cast<long long>(jj) * p.ld_u] = bits[jj];
            } else {
#pragma unroll
              for (int jj = 0; jj < 16; ++jj)
                if (jj < n_ok) dst[static_cast<long long>(jj) * p.ld_u] = bits[jj];
            }
          }
        }
      } else
      for (int h = 0; h < HALVES; ++h) {
        const int n = n0 + h * GEMM_BM + q * 32 + lane;
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                static_cast<uint32_t>((buf * HALVES + h) * p.col_stride);
        for (int c = cs * 16; c < p.br; c += 32) {
          if (r0 + c >= r_valid) break;
          uint32_t v[16];
          if (n_kb > 0) {
            tmem_ld_x16(t_addr + c, v);
            tmem_ld_wait();
#pragma unroll
            for (int jj = 0; jj < 16; ++jj) v[jj] = __float_as_uint(__uint_as_float(v[jj]) * s_rs[c + jj]);
          } else {
#pragma unroll
            for (int jj = 0; jj < 16; ++jj) v[jj] = 0u;
          }
          if (p.head_mode) {
            // softmax statistics over this warp's 32 token ids, per row, by warp shuffles
            const bool live = n < p.n && n != p.mask_id;
            HeadStat mine = head_stat_empty();
#pragma unroll
            for (int jj = 0; jj < 16; ++jj) {
              const float val = live ? __uint_as_float(v[jj]) : -INFINITY;
              float m = val;
              int arg = live ? n : 0x7fffffff;
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) {
                const float om = __shfl_xor_sync(0xffffffffu, m, o);
                const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
                if (om > m || (om == m && oa < arg)) {
                  m = om;
                  arg = oa;
                }
              }
              float e = live ? expf(val - m) : 0.f;     // m is finite unless all 32 ids are dead (then e = 0)
              float m2 = -INFINITY, tt = 0.f;
              if (p.st_m2) {
                m2 = (live && n != arg) ? val : -INFINITY;
                tt = live ? e * (val - m) : 0.f;
              }
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
              if (p.st_m2) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                  m2 = fmaxf(m2, __shfl_xor_sync(0xffffffffu, m2, o));
                  tt += __shfl_xor_sync(0xffffffffu, tt, o);
                }
              }
              if (lane == jj) {      // lane jj keeps row c + jj
                mine.m = m;
                mine.s = e;
                mine.arg = arg;
                mine.m2 = m2;
                mine.t = tt;
              }
            }
            // joined with what this warp has seen of the row in earlier weight tiles
            const int ci = c >> 5;
            if (ci == 0) run0 = head_stat_merge(run0, mine);
            else if (ci == 1) run1 = head_stat_merge(run1, mine);
            else if (ci == 2) run2 = head_stat_merge(run2, mine);
            else run3 = head_stat_merge(run3, mine);
          } else if (n < p.n) {
            float* dst = out + static_cast<long long>(r0 + c) * p.ldo + n;
            if (r0 + c + 16 <= r_valid) {           // whole group valid: no per-row test
#pragma unroll
              for (int jj = 0; jj < 16; ++jj) dst[static_cast<long long>(jj) * p.ldo] = __uint_as_float(v[jj]);
            } else {
#pragma unroll
              for (int jj = 0; jj < 16; ++jj)
                if (r0 + c + jj < r_valid) dst[static_cast<long long>(jj) * p.ldo] = __uint_as_float(v[jj]);
            }
          }
        }
      }
      // this warp is done reading the buffer: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));

      if (p.fuse_mode != FUSE_NONE &&
          !fused_tail(p, u / p.splits, split, n0, tile_rows, r0, r_valid, abort_flag, et, warp - 2, lane)) {
        ok = false;
        break;
      }
    }
    if (p.head_mode && ok && lane < 16) {
      // one entry per (CTA, lane quarter) and row: arrays [gridDim.x * 4][r_bound] (one row tile)
      const long long at = static_cast<long long>(blockIdx.x * 4 + q) * p.r_bound;
#pragma unroll
      for (int ci = 0; ci < 4; ++ci) {
        const HeadStat& r = ci == 0 ? run0 : ci == 1 ? run1 : ci == 2 ? run2 : run3;
        const int row = cs * 16 + 32 * ci + lane;
        if (row < r_valid) {
          p.st_max[at + row] = r.m;
          p.st_sum[at + row] = r.s;
          p.st_arg[at + row] = r.arg;
          if (p.st_m2) {
            p.st_m2[at + row] = r.m2;
            p.st_t[at + row] = r.t;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait ran out.  Give copies in flight time to land before the shared
    // memory is released, and report through the status word.
    if (threadIdx.x == 0) {
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {
      }
      if (p.status) atomicOr(p.status, DEV_ERR_WAIT);
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

}  // namespace dkv
