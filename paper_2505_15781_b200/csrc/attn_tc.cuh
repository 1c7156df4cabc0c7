// Bidirectional attention of the active queries over all cache slots (Eq. 4)
// on tcgen05 tensor cores, head_dim 128, 16-bit operands (fp16 or bf16).
//
// One CTA = one (sequence, KV head, tile of 128 "rows"), a row being a (query
// row, query head of the KV head's group) pair, so GQA groups share the K/V
// tiles.  Q, K and V tiles are TMA-loaded (128-byte swizzle); K/V come straight
// from the position-addressed slot cache, BKV slots per iteration, double
// buffered; the K/V maps are 3-D [head][slot][head_dim], so a tile that reaches past the last slot is
// zero-filled and never sees a neighbouring head's or layer's memory.  Two shapes of the same kernel: <128 slots, two softmax warpgroups>,
// one CTA per SM, for launches that do not fill the GPU twice (shortest latency
// per CTA), and <64 slots, one warpgroup>, two CTAs per SM, for large launches:
// within one CTA the tensor pipe, the special-function unit and the tensor-memory
// round trips of an iteration depend on each other, so a second resident CTA is
// what keeps the units busy.  Per iteration: S = Q K^T (accumulator in tensor memory, double
// buffered) -> the four softmax warps (one thread per row) read S, keep the
// running max / sum, rescale the output accumulator in tensor memory and write
// P to shared memory -> O += P V with V as an MN-major operand in its natural
// [slot][head_dim] layout.  No mask: every query sees every slot.
//
// Warp roles (320 threads): warp 0 = TMA, warp 1 = TMEM allocation + MMA issue,
// warps 2..9 = softmax / correction / epilogue: two warpgroups, each thread owns
// one row and one half of the tile's columns (two warps per scheduler hide each
// other's latencies); the halves exchange only their row maxima.
#pragma once
#include "pdl.cuh"
#include "ptx.cuh"

namespace dkv {

constexpr int ATC_M = 128;        // rows per CTA (MMA M)
constexpr int ATC_BKV = 128;      // slots per iteration of the one-CTA-per-SM shape
constexpr int ATC_DH = 128;
constexpr int ATC_THREADS = 320;     // TMA warp, MMA warp, two softmax warpgroups (the larger shape)
constexpr int ATC_TILE = 128 * 128;                 // bytes of a [128 rows x 64 columns] 16-bit tile
// Q (2 tiles) | K,V: 2 stages x (2 + 2) half tiles of [BKV slots x 64 columns] | P (NPB buffers of NWG
// tiles) | barriers | row maxima / sums exchanged by two warpgroups.  There is no room for alignment
// slack: the dynamic shared memory must start on a 1024-byte boundary (checked).
// The one-CTA-per-SM shape keeps TWO P buffers: its launches are chains of dependent iterations, and
// with one buffer the softmax of tile j+1 could not publish its P before P_j V_j had completed.
template <int NWG>
__host__ __device__ constexpr int attn_tc_pbufs() {
  return NWG == 2 ? 2 : 1;
}
template <int BKV, int NWG>
constexpr int attn_tc_smem() {
  return 2 * ATC_TILE + 2 * 4 * BKV * 128 + attn_tc_pbufs<NWG>() * NWG * ATC_TILE + 256 +
         (NWG == 2 ? 2 * 2 * 128 * 4 : 0);
}
constexpr int ATC_SMEM = attn_tc_smem<128, 2>();
constexpr long long ATC_WAIT_CYCLES = 4000000000LL;

struct AttnTcParams {
  void* o;                  // [R, H_q, 128] 16-bit
  const int32_t* row_off;   // [B+1]
  int seq_len, n_q_heads, n_kv_heads;   // seq_len = attended slots = the slot extent of the K/V tensor maps
  int group;                // query heads per KV head
  int rows_q;               // query rows per tile = 128 / group
  int kv_head0;             // first KV head of this layer inside the K/V tensor maps
  float scale_log2;
  int bf16;                 // 1: bf16 operands, 0: fp16
  int* status;
};

// tcgen05.st: 32 lanes x 16 consecutive 32-bit columns from registers
__device__ __forceinline__ void tmem_st_x16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 3-D tiled load (query rows x heads of the group x 64 columns)
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// MN-major operand stored as rows (K index) of 128 bytes (64 MN elements), 128-byte swizzle:
// 8-row groups are 1024 bytes apart (stride offset), the next 64 MN elements are `lbo` bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// instruction descriptor: fp32 accumulate, A K-major, B K-major (b_mn = 0) or MN-major (b_mn = 1)
__host__ __device__ constexpr uint32_t umma_idesc_f16_b(int m, int n, int bf16, int b_mn) {
  return (1u << 4) | (static_cast<uint32_t>(bf16) << 7) | (static_cast<uint32_t>(bf16) << 10) |
         (static_cast<uint32_t>(b_mn) << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}

// 2^x on the special-function unit (one instruction; flushes subnormal results, exact 0 for -inf)
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack16(float lo, float hi, int bf16) {
  if (bf16) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
  }
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int BKV, int NWG>
__global__ void __launch_bounds__(64 + 128 * NWG, NWG == 2 ? 1 : 2)
k_attn_tc(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
          const __grid_constant__ CUtensorMap tm_v, AttnTcParams p) {
  static_assert(BKV == 64 * NWG, "each softmax thread owns 64 slots of a tile");
  constexpr int KVT = BKV * 128;                        // bytes of a [BKV slots x 64 columns] half tile
  constexpr int TMEM_COLS = (2 * BKV + ATC_DH) > 256 ? 512 : 256;
  constexpr int NPB = attn_tc_pbufs<NWG>();             // P buffers
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  uint8_t* smem_al = smem_raw;
  const uint32_t sQ = smem_base;                       // 2 halves (head_dim 0..63, 64..127)
  const uint32_t sKV = sQ + 2 * ATC_TILE;              // stage s: K half0, K half1, V half0, V half1
  const uint32_t sP = sKV + 8 * KVT;                   // NPB buffers of NWG half tiles of 64 slots
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + 2 * ATC_TILE + 8 * KVT + NPB * NWG * ATC_TILE);
  // K and V tiles have barriers of their own: a K tile is free as soon as its S = Q K^T is done,
  // one iteration before the V tile of the same slots, so the next K load starts that much earlier
  uint64_t* q_full = bars;           // 1
  uint64_t* k_full = bars + 1;       // 2
  uint64_t* k_empty = bars + 3;      // 2
  uint64_t* v_full = bars + 5;       // 2
  uint64_t* v_empty = bars + 7;      // 2
  uint64_t* s_full = bars + 9;       // 2
  uint64_t* p_ready = bars + 11;     // 2: P buffer b holds the probabilities of its next tile
  uint64_t* p_free = bars + 13;      // 2: the P V MMAs that read buffer b (and all MMAs before them) are done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 15);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* xch = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + 256);   // NWG == 2: [2][2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(q_full), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&k_full[s]), 1);
      mbar_init(smem_u32(&k_empty[s]), 1);
      mbar_init(smem_u32(&v_full[s]), 1);
      mbar_init(smem_u32(&v_empty[s]), 1);
      mbar_init(smem_u32(&s_full[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&p_ready[b]), 4 * NWG);
      mbar_init(smem_u32(&p_free[b]), 1);
    }
    // swizzled tiles need the 1024-byte alignment; without it nothing is loaded and the launch reports
    *abort_flag = (smem_base & 1023u) ? 1 : 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tS = tmem_base;                // 2 x BKV columns
  const uint32_t tO = tmem_base + 2 * BKV;      // 128 columns

  pdl_enter(5);   // q, the slots and row_off come from earlier kernels

  const int b = blockIdx.z, hk = blockIdx.y;
  const int n_a = p.row_off[b + 1] - p.row_off[b];
  const int q0 = blockIdx.x * p.rows_q;
  const bool active = q0 < n_a && !*abort_flag;   // uniform over the CTA
  const int n_iter = active ? (p.seq_len + BKV - 1) / BKV : 0;
  const int kv_head = p.kv_head0 + b * p.n_kv_heads + hk;    // index into the maps' outermost dimension

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA
    if (lane == 0 && active) {
      mbar_expect_tx(smem_u32(q_full), static_cast<uint32_t>(2 * p.rows_q * p.group * 128));
      for (int half = 0; half < 2; ++half)
        tma_load_3d(sQ + half * ATC_TILE, &tm_q, smem_u32(q_full), half * 64, hk * p.group, p.row_off[b] + q0);
      for (int j = 0; j < n_iter; ++j) {
        const int s = j & 1;
        const uint32_t base = sKV + s * 4 * KVT;
        const int row = j * BKV;      // slots past seq_len are zero-filled by the copy (3-D map)
        if (!mbar_wait_bounded(smem_u32(&k_empty[s]), ((j >> 1) & 1) ^ 1, abort_flag, ATC_WAIT_CYCLES)) break;
        const uint32_t kf = smem_u32(&k_full[s]);
        mbar_expect_tx(kf, 2 * KVT);
        for (int half = 0; half < 2; ++half) tma_load_3d(base + half * KVT, &tm_k, kf, half * 64, row, kv_head);
        if (!mbar_wait_bounded(smem_u32(&v_empty[s]), ((j >> 1) & 1) ^ 1, abort_flag, ATC_WAIT_CYCLES)) break;
        const uint32_t vf = smem_u32(&v_full[s]);
        mbar_expect_tx(vf, 2 * KVT);
        for (int half = 0; half < 2; ++half) tma_load_3d(base + (2 + half) * KVT, &tm_v, vf, half * 64, row, kv_head);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA
    if (lane == 0 && active) {
      const uint32_t idesc_s = umma_idesc_f16_b(ATC_M, BKV, p.bf16, 0);
      const uint32_t idesc_o = umma_idesc_f16_b(ATC_M, ATC_DH, p.bf16, 1);
      bool ok = mbar_wait_bounded(smem_u32(q_full), 0, abort_flag, ATC_WAIT_CYCLES);
      auto issue_s = [&](int j) {   // S_j = Q K_j^T into S buffer j & 1
        const uint32_t base = sKV + (j & 1) * 4 * KVT;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t adesc = umma_desc_sw128(sQ + (kk >> 2) * ATC_TILE) + 2 * (kk & 3);
          const uint64_t bdesc = umma_desc_sw128(base + (kk >> 2) * KVT) + 2 * (kk & 3);
          umma_f16(tS + (j & 1) * BKV, adesc, bdesc, idesc_s, kk > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&k_empty[j & 1]));   // K_j has been consumed
        umma_commit(smem_u32(&s_full[j & 1]));
      };
      if (ok && n_iter > 0) {
        ok = mbar_wait_bounded(smem_u32(&k_full[0]), 0, abort_flag, ATC_WAIT_CYCLES);
        if (ok) {
          tc_fence_after();
          issue_s(0);
        }
      }
      for (int j = 0; j < n_iter && ok; ++j) {
        if (j + 1 < n_iter) {
          ok = mbar_wait_bounded(smem_u32(&k_full[(j + 1) & 1]), ((j + 1) >> 1) & 1, abort_flag, ATC_WAIT_CYCLES);
          if (!ok) break;
          tc_fence_after();
          issue_s(j + 1);   // its S buffer was drained before p_ready of iteration j-1
        }
        const int pb = j % NPB;
        ok = mbar_wait_bounded(smem_u32(&p_ready[pb]), (j / NPB) & 1, abort_flag, ATC_WAIT_CYCLES) &&
             mbar_wait_bounded(smem_u32(&v_full[j & 1]), (j >> 1) & 1, abort_flag, ATC_WAIT_CYCLES);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vbase = sKV + (j & 1) * 4 * KVT + 2 * KVT;
#pragma unroll
        for (int ks = 0; ks < BKV / 16; ++ks) {   // 16 slots per MMA
          const uint64_t adesc = umma_desc_sw128(sP + (pb * NWG + (ks >> 2)) * ATC_TILE) + 2 * (ks & 3);
          const uint64_t bdesc = umma_desc_sw128_mn(vbase + ks * 2048, KVT);
          umma_f16(tO, adesc, bdesc, idesc_o, (j > 0 || ks > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&v_empty[j & 1]));   // V_j and P_j have been consumed
        umma_commit(smem_u32(&p_free[pb]));
      }
    }
  } else if (active) {
    // ------------------------------------------ softmax / correction / epilogue
    const int q = warp & 3;                      // TMEM lane quarter this warp may touch
    const int wg = (NWG == 2) ? ((warp - 2) >> 2) : 0;   // which 64 slots of a tile this thread owns
    const int row = q * 32 + lane;               // TMEM lane = row of the tile
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    constexpr int O_COLS = ATC_DH / NWG;         // head_dim columns this thread rescales and writes out
    float m_run = -INFINITY, l_run = 0.f;        // l_run: this thread's share of the row sum
    bool ok = true;
    for (int j = 0; j < n_iter; ++j) {
      ok = ok && mbar_wait_bounded(smem_u32(&s_full[j & 1]), (j >> 1) & 1, abort_flag, ATC_WAIT_CYCLES);
      // The raw scores stay in the registers the tensor-memory loads filled.  Independent chains
      // (the loops run across the four 16-column groups), the scale folded into one FMA per element,
      // slots past the sequence masked only in the last tile.
      uint32_t raw[4][16];
      float mx = -INFINITY;
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld_x16(tS + (j & 1) * BKV + lane_addr + wg * 64 + c * 16, raw[c]);
        tmem_ld_wait();
        if (j == n_iter - 1 && (p.seq_len & (BKV - 1))) {
          const int n_valid = p.seq_len - j * BKV - wg * 64;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int e = 0; e < 16; ++e)
              if (c * 16 + e >= n_valid) raw[c][e] = 0xff800000u;   // -inf
          }
        }
        float mx8[8];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          mx8[2 * c] = __uint_as_float(raw[c][0]);
          mx8[2 * c + 1] = __uint_as_float(raw[c][8]);
        }
#pragma unroll
        for (int e = 1; e < 8; ++e) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            mx8[2 * c] = fmaxf(mx8[2 * c], __uint_as_float(raw[c][e]));
            mx8[2 * c + 1] = fmaxf(mx8[2 * c + 1], __uint_as_float(raw[c][8 + e]));
          }
        }
        mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                   fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7]))) * p.scale_log2;   // scale > 0
      }
      float m_tile = mx;
      if constexpr (NWG == 2) {
        // the two halves of a row agree on its maximum; the same barrier carries a failed wait to
        // all 256 threads, so that they leave the loop together and nobody is left at a barrier
        float* xb = xch + (j & 1) * 256;
        xb[wg * 128 + row] = mx;
        if (bar_red_or(1, 256, !ok)) {
          ok = false;
          break;
        }
        m_tile = fmaxf(mx, xb[(wg ^ 1) * 128 + row]);
      } else {
        if (!ok) break;          // rows are independent: no barrier to leave behind
      }
      // m_run is the exponent the probabilities are taken against.  It follows the row maximum only
      // when that has grown by more than 2^8: until then p = 2^(s - m_run) <= 256 is exact enough in
      // 16 bits and nothing has to be rescaled; the final division by the row sum makes the result the
      // same.  Both halves of a row see the same maximum, hence take the same decision.
      const float m_new = (m_tile > m_run + 8.f) ? m_tile : m_run;     // m_tile is finite: the tile holds a slot
      const float alpha = ex2_approx(m_run - m_new);
      m_run = m_new;
      float sum8[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) sum8[c] = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float p0 = ex2_approx(fmaf(__uint_as_float(raw[c][e]), p.scale_log2, -m_new));
          const float p1 = ex2_approx(fmaf(__uint_as_float(raw[c][8 + e]), p.scale_log2, -m_new));
          raw[c][e] = __float_as_uint(p0);
          raw[c][8 + e] = __float_as_uint(p1);
          sum8[2 * c] += p0;
          sum8[2 * c + 1] += p1;
        }
      }
      const float sum = ((sum8[0] + sum8[1]) + (sum8[2] + sum8[3])) + ((sum8[4] + sum8[5]) + (sum8[6] + sum8[7]));
      l_run = l_run * alpha + sum;
      const int pb = j % NPB;
      if (j >= NPB) {
        // the P V MMAs that read this P buffer (tile j - NPB) must be complete before it is overwritten
        ok = mbar_wait_bounded(smem_u32(&p_free[pb]), ((j - NPB) / NPB) & 1, abort_flag, ATC_WAIT_CYCLES);
        if (!ok) continue;        // two warpgroups: reported to everyone at the next iteration's barrier
      }
      if (j > 0) {
        // the accumulator only needs touching when some row of this warp moved its exponent; then
        // P_{j-1} V_{j-1} (and with it every earlier MMA) must be complete first
        if (!__all_sync(0xffffffffu, alpha == 1.f)) {
          ok = mbar_wait_bounded(smem_u32(&p_free[(j - 1) % NPB]), ((j - 1) / NPB) & 1, abort_flag, ATC_WAIT_CYCLES);
          if (!ok) continue;
          tc_fence_after();
#pragma unroll
          for (int hf = 0; hf < O_COLS / 64; ++hf) {
            uint32_t acc[4][16];
            const uint32_t col0 = (NWG == 2 ? wg * 64 : hf * 64);
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_x16(tO + lane_addr + col0 + c * 16, acc[c]);
            tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
#pragma unroll
              for (int e = 0; e < 16; ++e) acc[c][e] = __float_as_uint(__uint_as_float(acc[c][e]) * alpha);
              tmem_st_x16(tO + lane_addr + col0 + c * 16, acc[c]);
            }
          }
          tmem_st_wait();
        }
      }
      // P_j -> shared memory, K-major rows of 128 bytes with the 128-byte swizzle; the thread's
      // 64 slots are one 64-column half tile
      uint8_t* prow = smem_al + (sP - smem_base) + (pb * NWG + wg) * ATC_TILE + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {            // 16-byte chunks of 8 slots
        const uint32_t* sv = &raw[ch >> 1][(ch & 1) * 8];
        uint4 w;
        w.x = pack16(__uint_as_float(sv[0]), __uint_as_float(sv[1]), p.bf16);
        w.y = pack16(__uint_as_float(sv[2]), __uint_as_float(sv[3]), p.bf16);
        w.z = pack16(__uint_as_float(sv[4]), __uint_as_float(sv[5]), p.bf16);
        w.w = pack16(__uint_as_float(sv[6]), __uint_as_float(sv[7]), p.bf16);
        *reinterpret_cast<uint4*>(prow + ((ch ^ (row & 7)) << 4)) = w;
      }
      fence_proxy_async_smem();      // the MMA reads P through the async proxy
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&p_ready[pb]));
    }
    // Leaving the loop with two warpgroups: either every thread finished it or a failed wait was seen
    // by all of them at a barrier; the barrier below is reached by all 256 threads in every case.
    if (n_iter > 0) {
      ok = ok && mbar_wait_bounded(smem_u32(&p_free[(n_iter - 1) % NPB]), ((n_iter - 1) / NPB) & 1, abort_flag,
                                   ATC_WAIT_CYCLES);
      float l_row = l_run;
      if constexpr (NWG == 2) {
        xch[wg * 128 + row] = l_run;
        if (bar_red_or(1, 256, !ok)) ok = false;
        l_row += xch[(wg ^ 1) * 128 + row];
      }
      if (ok) {
        tc_fence_after();
        const int qi = row / p.group, g = row - qi * p.group;
        const bool valid = row < p.rows_q * p.group && q0 + qi < n_a;
        const float inv = 1.f / l_row;
        uint8_t* orow = static_cast<uint8_t*>(p.o) +
                        ((static_cast<long long>(p.row_off[b] + q0 + qi) * p.n_q_heads + hk * p.group + g) * ATC_DH) * 2;
        // the thread's columns in groups of 64: all four tensor-memory loads of a group are in flight
        // before the one wait (one round trip instead of four)
#pragma unroll
        for (int c0 = wg * O_COLS; c0 < wg * O_COLS + O_COLS; c0 += 64) {
          uint32_t v[4][16];
#pragma unroll
          for (int g = 0; g < 4; ++g) tmem_ld_x16(tO + lane_addr + c0 + g * 16, v[g]);
          tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint4 w0, w1;
              w0.x = pack16(__uint_as_float(v[g][0]) * inv, __uint_as_float(v[g][1]) * inv, p.bf16);
              w0.y = pack16(__uint_as_float(v[g][2]) * inv, __uint_as_float(v[g][3]) * inv, p.bf16);
              w0.z = pack16(__uint_as_float(v[g][4]) * inv, __uint_as_float(v[g][5]) * inv, p.bf16);
              w0.w = pack16(__uint_as_float(v[g][6]) * inv, __uint_as_float(v[g][7]) * inv, p.bf16);
              w1.x = pack16(__uint_as_float(v[g][8]) * inv, __uint_as_float(v[g][9]) * inv, p.bf16);
              w1.y = pack16(__uint_as_float(v[g][10]) * inv, __uint_as_float(v[g][11]) * inv, p.bf16);
              w1.z = pack16(__uint_as_float(v[g][12]) * inv, __uint_as_float(v[g][13]) * inv, p.bf16);
              w1.w = pack16(__uint_as_float(v[g][14]) * inv, __uint_as_float(v[g][15]) * inv, p.bf16);
              *reinterpret_cast<uint4*>(orow + (c0 + g * 16) * 2) = w0;
              *reinterpret_cast<uint4*>(orow + (c0 + g * 16) * 2 + 16) = w1;
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
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
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace dkv
