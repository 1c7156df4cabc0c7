// Mergeable softmax statistics of the vocabulary head: shared by the head GEMM's epilogue, which
// produces and pre-merges them, and the kernel that combines them per head row.
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>

namespace dkv {

// Softmax statistics of a set of token ids: the largest logit m (its id: lowest on ties), the second
// largest m2 (over the other ids), S = sum exp(l - m) and T = sum exp(l - m)(l - m).  merge() joins the
// statistics of two disjoint sets; it is exact in (m, arg, m2) and order-independent there.
struct HeadStat {
  float m, m2, s, t;
  int arg;
};
__device__ __forceinline__ HeadStat head_stat_empty() {
  HeadStat e;
  e.m = -CUDART_INF_F;
  e.m2 = -CUDART_INF_F;
  e.s = 0.f;
  e.t = 0.f;
  e.arg = 0x7fffffff;
  return e;
}
__device__ __forceinline__ HeadStat head_stat_merge(const HeadStat& a, const HeadStat& b) {
  const bool b_wins = b.m > a.m || (b.m == a.m && b.arg < a.arg);
  const HeadStat& hi = b_wins ? b : a;
  const HeadStat& lo = b_wins ? a : b;
  HeadStat r;
  r.m = hi.m;
  r.arg = hi.arg;
  r.m2 = fmaxf(fmaxf(hi.m2, lo.m2), lo.m);
  if (lo.m == -CUDART_INF_F) {          // an empty side (also when both are empty): nothing to rescale
    r.s = hi.s;
    r.t = hi.t;
  } else {
    const float dm = lo.m - hi.m;        // <= 0
    const float w = expf(dm);
    r.s = hi.s + w * lo.s;
    r.t = hi.t + w * (lo.t + lo.s * dm);
  }
  return r;
}
__device__ __forceinline__ HeadStat head_stat_shfl_xor(const HeadStat& v, int o) {
  HeadStat r;
  r.m = __shfl_xor_sync(0xffffffffu, v.m, o);
  r.m2 = __shfl_xor_sync(0xffffffffu, v.m2, o);
  r.s = __shfl_xor_sync(0xffffffffu, v.s, o);
  r.t = __shfl_xor_sync(0xffffffffu, v.t, o);
  r.arg = __shfl_xor_sync(0xffffffffu, v.arg, o);
  return r;
}

}  // namespace dkv
