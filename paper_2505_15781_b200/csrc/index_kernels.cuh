// Integer kernels: the cache policy's active set with its ascending
// compaction (Eq. 4, refresh / Prefill / PD rules of Sec. 3.3, Greedy window of
// Sec. 3.4), the head-row list, and the confidence top-k unmask selection of
// Sec. 3.1.
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "gemm_tc.cuh"  // DEV_ERR_* bits
#include "pdl.cuh"

namespace dkv {

constexpr int ACT_FULL = 0;       // every position
constexpr int ACT_GEN_ONLY = 1;   // positions >= prompt_len
constexpr int ACT_FROM_MASK = 2;  // positions whose bit is set in mask_src
constexpr int ACT_GREEDY = 3;     // D_t, D_{t-1} and the window around the centres
constexpr int ACT_PROMPT_ONLY = 4;  // positions < prompt_len (the isolated prefill pass)

struct CompactParams {
  int mode;
  int batch, seq_len, prompt_len;
  const uint8_t* mask_src;   // ACT_FROM_MASK: M_{t-1} (delay 1) or M_t (delay 0)
  const uint8_t* mask_cur;   // M_t (head rows, copy to mask_store)
  uint8_t* mask_store;       // where M_t is kept for the next step
  const int32_t* d_cur;      // [batch, k] D_t or NULL
  const int32_t* d_prev;     // [batch, k] D_{t-1} or NULL
  int32_t* d_store;          // where D_t is kept for the next step (or NULL)
  int k;
  int w_lo, w_hi;            // window = [c - w_lo, c + w_hi]
  int center_cur;            // 1: centres are D_t, 0: D_{t-1}
  int head_from_d;           // 1: head rows are D_t; 0: M_t inside [cand_lo, cand_hi)
  int shift;                 // 1: the logits of position j are read at row j-1 (that row is then active too)
  int right;                 // 1: a row is also active while the position to its right is (Appendix B, Un&Right-Shift)
  int cand_lo, cand_hi;
  int step;                  // t, stamped into written_step
  int rows_bound;            // per-sequence bound promised by the host
  int head_bound;
  int32_t* act_idx;          // [batch*seq_len] flattened positions, ascending
  int32_t* row_off;          // [batch+1]
  int32_t* inv;              // [batch, seq_len] compact row or -1
  int32_t* head_row;         // [.] compact row of each head row
  int32_t* head_pos;         // [.] flattened position of each head row
  int32_t* head_off;         // [batch+1]
  int32_t* written_step;     // [batch, seq_len]
  float* conf;               // [batch, seq_len] reset to -inf
  int32_t* pred;             // [batch, seq_len] reset to -1
  int* status;
  unsigned long long* active_total;  // running sum of active rows over steps (exact, for the cache ratio)
};

__device__ __forceinline__ bool in_list(const int32_t* d, int k, int pos) {
  for (int j = 0; j < k; ++j)
    if (d[j] == pos) return true;
  return false;
}

// Is `pos` a position whose confidence / token is wanted at this step?
__device__ __forceinline__ bool is_target(const CompactParams& p, int b, int pos) {
  if (pos < 0 || pos >= p.seq_len) return false;
  if (p.head_from_d) return p.d_cur && in_list(p.d_cur + b * p.k, p.k, pos);
  return pos >= p.cand_lo && pos < p.cand_hi && p.mask_cur[b * p.seq_len + pos] != 0;
}

// The row whose logits serve target position j is j itself, or j-1 with shifted outputs.
__device__ __forceinline__ bool is_head(const CompactParams& p, int b, int pos) {
  return is_target(p, b, pos + p.shift);
}

__device__ __forceinline__ bool policy_active(const CompactParams& p, int b, int pos) {
  switch (p.mode) {
    case ACT_FULL: return true;
    case ACT_GEN_ONLY: return pos >= p.prompt_len;
    case ACT_PROMPT_ONLY: return pos < p.prompt_len;
    case ACT_FROM_MASK: return p.mask_src[b * p.seq_len + pos] != 0;
    default: {
      const int32_t* dc = p.d_cur ? p.d_cur + b * p.k : nullptr;
      const int32_t* dp = p.d_prev ? p.d_prev + b * p.k : nullptr;
      if (dc && in_list(dc, p.k, pos)) return true;
      if (dp && in_list(dp, p.k, pos)) return true;
      const int32_t* cen = p.center_cur ? dc : dp;
      if (cen) {
        for (int j = 0; j < p.k; ++j) {
          const int c = cen[j];
          if (c >= 0 && pos >= c - p.w_lo && pos <= c + p.w_hi) return true;
        }
      }
      return false;
    }
  }
}

__device__ __forceinline__ bool is_active(const CompactParams& p, int b, int pos) {
  if (p.shift && is_head(p, b, pos)) return true;
  if (policy_active(p, b, pos)) return true;
  return p.right && pos + 1 < p.seq_len && policy_active(p, b, pos + 1);
}

// One CTA per sequence.  256 threads.
__global__ void __launch_bounds__(256) k_compact(CompactParams p) {
  __shared__ int s_warp_a[8], s_warp_h[8];
  __shared__ int s_base_a, s_base_h, s_run_a, s_run_h;
  pdl_enter(1);
  const int b = blockIdx.x;
  const int L = p.seq_len;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // offsets of this sequence = number of active / head rows of the sequences before it.  In the
  // common modes these counts need no per-position predicate: all rows / generation rows / prompt
  // rows are a product, the mask-driven set is the number of non-zero bytes of the flat mask in
  // front of this sequence (16-byte loads), and the head rows are the masked positions of each
  // earlier sequence's candidate range.  Greedy and the shifted variants take the general loop.
  int ca = 0, ch = 0;
  const bool general = p.mode == ACT_GREEDY || p.shift || p.right || p.head_from_d;
  if (general) {
    for (int bb = 0; bb < b; ++bb) {
      for (int pos = tid; pos < L; pos += 256) {
        ca += is_active(p, bb, pos) ? 1 : 0;
        ch += is_head(p, bb, pos) ? 1 : 0;
      }
    }
  } else {
    if (p.mode == ACT_FROM_MASK) {
      const long long n = static_cast<long long>(b) * L;
      const uint4* m16 = reinterpret_cast<const uint4*>(p.mask_src);
      const long long n16 = (reinterpret_cast<uintptr_t>(p.mask_src) & 15) ? 0 : n / 16;   // a caller's mask may be unaligned
      for (long long i = tid; i < n16; i += 256) {
        const uint4 v = m16[i];
        ca += __popc(__vcmpne4(v.x, 0u) & 0x01010101u) + __popc(__vcmpne4(v.y, 0u) & 0x01010101u) +
              __popc(__vcmpne4(v.z, 0u) & 0x01010101u) + __popc(__vcmpne4(v.w, 0u) & 0x01010101u);
      }
      for (long long i = n16 * 16 + tid; i < n; i += 256) ca += p.mask_src[i] != 0 ? 1 : 0;
    } else if (tid == 0) {
      ca = b * (p.mode == ACT_FULL ? L : (p.mode == ACT_GEN_ONLY ? L - p.prompt_len : p.prompt_len));
    }
    for (int bb = 0; bb < b; ++bb)
      for (int pos = p.cand_lo + tid; pos < p.cand_hi; pos += 256) ch += p.mask_cur[bb * L + pos] != 0 ? 1 : 0;
  }
  for (int o = 16; o > 0; o >>= 1) {
    ca += __shfl_xor_sync(0xffffffffu, ca, o);
    ch += __shfl_xor_sync(0xffffffffu, ch, o);
  }
  if (lane == 0) {
    s_warp_a[warp] = ca;
    s_warp_h[warp] = ch;
  }
  __syncthreads();
  if (tid == 0) {
    int a = 0, h = 0;
    for (int i = 0; i < 8; ++i) {
      a += s_warp_a[i];
      h += s_warp_h[i];
    }
    s_base_a = a;
    s_base_h = h;
    s_run_a = 0;
    s_run_h = 0;
  }
  __syncthreads();
  const int base_a = s_base_a, base_h = s_base_h;

  for (int c0 = 0; c0 < L; c0 += 256) {
    const int pos = c0 + tid;
    const bool valid = pos < L;
    const bool fa = valid && is_active(p, b, pos);
    const bool fh = valid && is_head(p, b, pos);
    const unsigned ba = __ballot_sync(0xffffffffu, fa);
    const unsigned bh = __ballot_sync(0xffffffffu, fh);
    if (lane == 0) {
      s_warp_a[warp] = __popc(ba);
      s_warp_h[warp] = __popc(bh);
    }
    __syncthreads();
    int pa = s_run_a, ph = s_run_h;
    for (int i = 0; i < warp; ++i) {
      pa += s_warp_a[i];
      ph += s_warp_h[i];
    }
    const unsigned lower = (1u << lane) - 1u;
    const int ia = pa + __popc(ba & lower);
    const int ih = ph + __popc(bh & lower);
    if (valid) {
      const int flat = b * L + pos;
      if (fa) {
        p.act_idx[base_a + ia] = flat;
        p.written_step[flat] = p.step;
      }
      p.inv[flat] = fa ? base_a + ia : -1;
      if (fh) {
        if (!fa && p.status) atomicOr(p.status, DEV_ERR_HEAD_ROW);
        p.head_row[base_h + ih] = fa ? base_a + ia : 0;
        p.head_pos[base_h + ih] = flat + p.shift;
      }
      p.conf[flat] = -CUDART_INF_F;
      p.pred[flat] = -1;
      if (p.mask_store) p.mask_store[flat] = p.mask_cur[flat];
    }
    __syncthreads();
    if (tid == 0) {
      int a = 0, h = 0;
      for (int i = 0; i < 8; ++i) {
        a += s_warp_a[i];
        h += s_warp_h[i];
      }
      s_run_a += a;
      s_run_h += h;
    }
    __syncthreads();
  }
  if (tid == 0) {
    p.row_off[b] = base_a;
    p.head_off[b] = base_h;
    if (b == p.batch - 1) {
      p.row_off[p.batch] = base_a + s_run_a;
      p.head_off[p.batch] = base_h + s_run_h;
      if (p.active_total) atomicAdd(p.active_total, static_cast<unsigned long long>(base_a + s_run_a));
    }
    if (p.status && (s_run_a > p.rows_bound || s_run_h > p.head_bound)) atomicOr(p.status, DEV_ERR_ROWS_BOUND);
  }
  if (p.d_store && p.d_cur && tid < p.k) p.d_store[b * p.k + tid] = p.d_cur[b * p.k + tid];
}

// Top-k unmask selection, one CTA per sequence (256 threads).  When `given`
// is not NULL the positions are taken from it instead of being selected.
__global__ void __launch_bounds__(256)
k_select_unmask(const float* __restrict__ conf, const int32_t* __restrict__ pred, int seq_len, int cand_lo,
                int cand_hi, int k, const int32_t* __restrict__ given, int32_t* tokens, uint8_t* masked,
                int32_t* chosen, int* status) {
  __shared__ float s_c[8];
  __shared__ int s_p[8];
  pdl_enter(13);
  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long base = static_cast<long long>(b) * seq_len;
  for (int j = 0; j < k; ++j) {
    if (given) {
      if (tid == 0) {
        const int pos = given[b * k + j];
        if (pos >= 0 && pos < seq_len) {
          tokens[base + pos] = pred[base + pos];
          masked[base + pos] = 0;
        }
        if (chosen) chosen[b * k + j] = pos;
      }
      continue;
    }
    float bc = -CUDART_INF_F;
    int bp = -1;
    for (int pos = cand_lo + tid; pos < cand_hi; pos += 256) {
      if (!masked[base + pos]) continue;
      float c = conf[base + pos];
      if (c != c) c = -CUDART_INF_F;                  // NaN counts as -inf
      if (bp < 0 || c > bc) {                         // ascending scan keeps the lower position on ties
        bc = c;
        bp = pos;
      }
    }
    for (int o = 16; o > 0; o >>= 1) {
      const float oc = __shfl_xor_sync(0xffffffffu, bc, o);
      const int op = __shfl_xor_sync(0xffffffffu, bp, o);
      if (op >= 0 && (bp < 0 || oc > bc || (oc == bc && op < bp))) {
        bc = oc;
        bp = op;
      }
    }
    if (lane == 0) {
      s_c[warp] = bc;
      s_p[warp] = bp;
    }
    __syncthreads();
    if (tid == 0) {
      float c = s_c[0];
      int pz = s_p[0];
      for (int i = 1; i < 8; ++i) {
        if (s_p[i] >= 0 && (pz < 0 || s_c[i] > c || (s_c[i] == c && s_p[i] < pz))) {
          c = s_c[i];
          pz = s_p[i];
        }
      }
      if (pz >= 0) {
        tokens[base + pz] = pred[base + pz];
        masked[base + pz] = 0;
      } else if (status) {
        atomicOr(status, DEV_ERR_FEW_CAND);
      }
      if (chosen) chosen[b * k + j] = pz;
    }
    __syncthreads();
  }
}

}  // namespace dkv
