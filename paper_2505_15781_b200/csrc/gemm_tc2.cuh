// The projection GEMM on CTA pairs (tcgen05 cta_group::2).  Same orientation as
// k_gemm_tc (weights = MMA A operand / TMEM lanes, the step's rows = MMA N), but
// one MMA spans two SMs: M = 256 weight rows, 128 per CTA, and each CTA stages
// only HALF of the row tile (the B operand is read from both CTAs' shared
// memory).  Per 32 KB of weights a CTA therefore holds br * 64 bytes of rows
// instead of br * 128: the ring is deeper at the same shared memory and the
// L2 -> SM traffic of the rows halves, which is what bounds the one-CTA kernel
// above ~128 rows.  A pair's tile is 512 weight rows (two MMAs side by side).  Which 128 rows a CTA
// stages for MMA h is a matter of its TMA coordinate only: rank r takes rows [r*256 + h*128, +128), so
// a CTA always owns 256 consecutive rows of the weight matrix.  Two uses: the unsplit gate/up
// projection with the SwiGLU epilogue (the weight copy is grouped [128 gate | 128 up] per 256 rows,
// so that each CTA holds the gate rows (MMA 0) and the up rows (MMA 1) of the same 128 features),
// and the QKV / O / down projections of steps with more than one row tile, with plain fp32 partial
// sums and, for O and down, the fused residual tail of k_gemm_tc (each CTA of a pair then counts as
// a 256-column weight tile of its own).  The split-K launches of the cached steps gain nothing from pairs.
//
// Roles per CTA (320 threads): warp 0 = TMA producer of its own half of the
// operands, completion counted on the LEADER's barrier (cta_group::2 loads);
// warp 1 = tensor-memory allocation in both CTAs (collective), MMA issue in the
// leader only, commits multicast to both CTAs' barriers; warps 2..9 = epilogue
// over the CTA's own 128 accumulator lanes (two warps per lane quarter, alternate
// 16-column groups).  Every wait is clock-bounded.
#pragma once
#include "gemm_tc.cuh"

namespace dkv {

constexpr int GEMM2_TILE_ROWS = 512;   // weight rows per pair tile

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_pair_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                              uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair when the MMAs issued so far are done
__device__ __forceinline__ void umma_pair_commit(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(static_cast<uint16_t>(3))
      : "memory");
}
// this CTA's tile -> its own shared memory; completion bytes counted on an mbarrier of the pair (cluster address)
__device__ __forceinline__ void tma_pair_load_2d_hint(uint32_t dst, const CUtensorMap* tm, uint32_t bar_cluster, int c0,
                                                      int c1, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar_cluster), "r"(c0), "r"(c1), "l"(policy)
      : "memory");
}

// Plan for a row tile of `br` rows (a multiple of 16, at most 256); per CTA a stage holds 2 x 16 KB
// of weights and br / 2 rows.
inline GemmTcPlan gemm_tc2_plan(int br) {
  GemmTcPlan p;
  p.br = br;
  p.halves = 2;
  p.stage_bytes = 2 * GEMM_A_BYTES + static_cast<int>(((br / 2) * GEMM_BK * 2 + 1023) / 1024 * 1024);
  p.col_stride = 32;
  while (p.col_stride < br) p.col_stride *= 2;
  p.n_bufs = (2 * 2 * p.col_stride <= 512) ? 2 : 1;
  p.tmem_cols = p.n_bufs * 2 * p.col_stride;
  p.stages = (220 * 1024) / p.stage_bytes;
  if (p.stages > GEMM_MAX_STAGES) p.stages = GEMM_MAX_STAGES;
  p.smem_bytes = p.stages * p.stage_bytes + 1024 + GEMM_BAR_BYTES + GEMM_SCALE_BYTES;
  p.ctas_per_sm = 1;
  return p;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
k_gemm_tc2(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, GemmTcParams p) {
  const int STAGES = p.stages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * p.stage_bytes);
  // full[S] (waited on in the leader only), empty[S], accumulator full[2] (both CTAs, by multicast
  // commits), accumulator empty[2] (leader only; the epilogue warps of both CTAs arrive on it)
  uint64_t* full = bars;
  uint64_t* empty = bars + STAGES;
  uint64_t* acc_full = bars + 2 * STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int a_bytes = 2 * GEMM_A_BYTES;
  const int b_rows = p.br >> 1;                     // rows of the row tile staged by this CTA
  const int b_bytes = b_rows * GEMM_BK * 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full[s]), 1);
      mbar_init(smem_u32(&empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&acc_full[b]), 1);
      mbar_init(smem_u32(&acc_empty[b]), 16);   // eight epilogue warps in each of the two CTAs
    }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), p.tmem_cols);   // collective over the pair
    tmem_relinquish_pair();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_w);
    tma_prefetch_desc(&tm_x);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();       // the peer's barriers exist before anything is signalled on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // unit u -> (pair tile of 512 weight rows, row tile, split); consecutive units differ in the split first
  auto decode = [&](int u, int& n0, int& r0, int& split, int& kb0, int& n_kb) {
    split = u % p.splits;
    const int t = u / p.splits;
    r0 = (t % p.r_tiles) * p.br;
    n0 = (t / p.r_tiles) * GEMM2_TILE_ROWS;
    kb0 = split * p.kb_per_split;
    n_kb = max(0, min(p.kb_total, kb0 + p.kb_per_split) - kb0);
  };

  pdl_launch();

  if (warp == 0) {
    // ------------------------------------------------------- TMA producer (each CTA its own halves)
    if (lane == 0) {
      const uint64_t pol_w = l2_policy_evict_first();
      const uint64_t pol_x = l2_policy_evict_last();
      struct Cursor {
        int u, i, n0, r0, split, kb0, n_kb;
        bool decoded;
      } cur;
      cur.u = pair;
      cur.i = 0;
      cur.decoded = false;
      auto settle = [&](Cursor& c) {
        while (c.u < p.units) {
          if (!c.decoded) {
            decode(c.u, c.n0, c.r0, c.split, c.kb0, c.n_kb);
            c.decoded = true;
          }
          if (c.i < c.n_kb) return true;
          c.u += n_pairs;
          c.i = 0;
          c.decoded = false;
        }
        return false;
      };
      auto load_a = [&](const Cursor& c, int s) {
        // the leader announces the bytes of BOTH CTAs' loads of this stage
        if (rank == 0) mbar_expect_tx(smem_u32(&full[s]), static_cast<uint32_t>(2 * (a_bytes + b_bytes)));
        const uint32_t lf = mapa_shared(smem_u32(&full[s]), 0);
        const uint32_t a_dst = smem_base + s * p.stage_bytes;
        for (int h = 0; h < 2; ++h)
          if (p.w_blocked)
            tma_pair_load_2d_hint(a_dst + h * GEMM_A_BYTES, &tm_w, lf, 0,
                                  (c.n0 + static_cast<int>(rank) * 256 + h * GEMM_BM) * p.kb_total +
                                      (c.kb0 + c.i) * GEMM_BM, pol_w);
          else
            tma_pair_load_2d_hint(a_dst + h * GEMM_A_BYTES, &tm_w, lf, (c.kb0 + c.i) * GEMM_BK,
                                  c.n0 + static_cast<int>(rank) * 256 + h * GEMM_BM, pol_w);
      };
      auto load_b = [&](const Cursor& c, int s) {
        const uint32_t lf = mapa_shared(smem_u32(&full[s]), 0);
        tma_pair_load_2d_hint(smem_base + s * p.stage_bytes + a_bytes, &tm_x, lf, (c.kb0 + c.i) * GEMM_BK,
                              c.r0 + static_cast<int>(rank) * b_rows, pol_x);
      };
      Cursor head = cur;
      int pre = 0;
      Cursor c = cur;
      while (p.w_static && pre < STAGES && settle(c)) {   // all stages are free at the start
        load_a(c, pre);
        ++pre;
        ++c.i;
      }
      pdl_wait();
      c = head;
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
        ok = mbar_wait_bounded(smem_u32(&empty[s]), ph ^ 1, abort_flag, GEMM_WAIT_CYCLES);
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
    // --------------------------------------------------------- MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = umma_idesc_f16(256, p.br, p.x_bf16);
      int s = 0, j = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int u = pair; u < p.units && ok; u += n_pairs, ++j) {
        int n0, r0, split, kb0, n_kb;
        decode(u, n0, r0, split, kb0, n_kb);
        const int buf = j % p.n_bufs;
        const uint32_t use = static_cast<uint32_t>(j / p.n_bufs);
        ok = mbar_wait_bounded(smem_u32(&acc_empty[buf]), (use & 1) ^ 1, abort_flag, GEMM_WAIT_CYCLES);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_base = tmem_base + static_cast<uint32_t>(buf * 2 * p.col_stride);
        for (int i = 0; i < n_kb; ++i) {
          // everything that depends only on the stage is computed BEFORE the wait: what this thread
          // executes between the arrival of a stage and its MMAs is on the main loop's critical path
          const uint32_t a_addr = smem_base + s * p.stage_bytes;
          const uint64_t bdesc = umma_desc_sw128(a_addr + a_bytes);
          const uint64_t adesc0 = umma_desc_sw128(a_addr), adesc1 = umma_desc_sw128(a_addr + GEMM_A_BYTES);
          const uint32_t full_bar = smem_u32(&full[s]), empty_bar = smem_u32(&empty[s]);
          const uint32_t acc0 = i > 0 ? 1u : 0u;
          ok = mbar_wait_bounded(full_bar, ph, abort_flag, GEMM_WAIT_CYCLES);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k4 = 0; k4 < GEMM_BK / 16; ++k4)
            umma_pair_f16(d_base, adesc0 + 2 * k4, bdesc + 2 * k4, idesc, k4 > 0 ? 1u : acc0);
#pragma unroll
          for (int k4 = 0; k4 < GEMM_BK / 16; ++k4)
            umma_pair_f16(d_base + static_cast<uint32_t>(p.col_stride), adesc1 + 2 * k4, bdesc + 2 * k4, idesc,
                          k4 > 0 ? 1u : acc0);
          umma_pair_commit(empty_bar);      // frees the stage in both CTAs
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (ok) umma_pair_commit(smem_u32(&acc_full[buf]));
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (both CTAs, own 128 lanes)
    const int q = warp & 3;
    const int cs = (warp - 2) >> 2;   // which of the alternating 16-column groups this warp takes
    const int et = threadIdx.x - 64;  // 0..255 among the epilogue threads
    float* s_rs = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + GEMM_BAR_BYTES);   // [256] row scales
    pdl_wait();
    // (every earlier launch has completed: the counters of the previous fused launch are free to be
    // zeroed for the next one)
    if (p.fuse_mode != FUSE_NONE && et == 255)
      for (int i = blockIdx.x; i < 256; i += gridDim.x) p.tile_cnt_next[i] = 0u;
    int r_valid = p.r_bound;
    if (p.r_dev) r_valid = min(r_valid, *p.r_dev);
    int j = 0;
    bool ok = true;
    for (int u = pair; u < p.units && ok; u += n_pairs, ++j) {
      int n0, r0, split, kb0, n_kb;
      decode(u, n0, r0, split, kb0, n_kb);
      const int buf = j % p.n_bufs;
      const uint32_t use = static_cast<uint32_t>(j / p.n_bufs);
      // the row scales of this unit's row tile (1 when the launch has none), computed while the MMAs run
      if (j > 0) named_bar_sync(1, 256);
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
      const int row_in_tile = static_cast<int>(rank) * GEMM_BM + q * 32 + lane;
      const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(buf * 2 * p.col_stride);
      if (p.swiglu_out) {
        // the gate/up copy is grouped [128 gate rows | 128 up rows] per 256 rows and this CTA staged the
        // gate rows (MMA 0) and the up rows (MMA 1) of features (n0 / 2) + rank * 128 + [0, 128)
        const int jf = (n0 >> 1) + row_in_tile;
        for (int c = cs * 16; c < p.br; c += 32) {
          if (r0 + c >= r_valid) break;
          uint32_t vg[16], vu[16];
          tmem_ld_x16(t_lane + c, vg);
          tmem_ld_x16(t_lane + p.col_stride + c, vu);
          tmem_ld_wait();
          if (jf < p.ld_u) {
            // SiLU with the fast exponential and reciprocal (error ~2^-21, far below the 16-bit rounding
            // of the product); one pointer, the format test outside the loop, no row test for whole groups
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
      } else {
        // plain partial sums: this CTA holds weight rows n0 + rank * 256 + h * 128 + [0, 128) in MMA h,
        // i.e. 256 consecutive output columns, like one tile of the one-CTA kernel
        float* out = p.out + static_cast<long long>(split) * p.split_stride;
        for (int h = 0; h < 2; ++h) {
          const int n = n0 + static_cast<int>(rank) * 256 + h * GEMM_BM + q * 32 + lane;
          const uint32_t t_addr = t_lane + static_cast<uint32_t>(h * p.col_stride);
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
            if (n < p.n) {
              float* dst = out + static_cast<long long>(r0 + c) * p.ldo + n;
              if (r0 + c + 16 <= r_valid) {
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
      }
      // this warp is done reading the buffer: tell the leader's MMA thread
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&acc_empty[buf]), 0));

      // fused row epilogue across the K splits: each CTA of the pair is one 256-column tile of its own
      if (p.fuse_mode != FUSE_NONE &&
          !fused_tail(p, (u / p.splits) * 2 + static_cast<int>(rank), split, n0 + static_cast<int>(rank) * 256, 256, r0,
                      r_valid, abort_flag, et, warp - 2, lane)) {
        ok = false;
        break;
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
  // neither CTA may leave (or free tensor memory) while the other can still read its shared
  // memory through an MMA or signal its barriers
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, p.tmem_cols);
  }
}

}  // namespace dkv
