// Measurement aid: the ring of the projection GEMM without its arithmetic.  Every CTA streams its own
// slice of a large buffer (the "weights": unique bytes from HBM) and, per stage, a piece of a small
// buffer that every CTA re-reads (the "rows": L2 hits) into a ring of shared-memory stages with bulk
// copies; a consumer thread frees a stage the moment it is full.  The launch's duration is what the
// memory system alone allows for that access pattern: the ceiling the weight-streaming launches are
// held against.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "ptx.cuh"

namespace dkv {

struct StreamProbeParams {
  const uint8_t* a;        // streamed buffer; CTA i reads [i * a_per_cta, + n_chunks * a_chunk)
  const uint8_t* b;        // re-read buffer of b_span bytes (NULL: none)
  long long a_per_cta;
  long long b_span;        // a multiple of b_chunk
  int n_chunks;            // stages' worth of data per CTA
  int a_chunk, b_chunk;    // bytes per stage from a and from b (multiples of 16)
  int stages;
  long long wait_cycles;
  int* status;             // bit 3 (DEV_ERR_WAIT) is set when a wait ran out
};

__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}

__global__ void __launch_bounds__(64, 1) k_stream_probe(StreamProbeParams p) {
  extern __shared__ __align__(1024) uint8_t probe_smem[];
  const int stage_bytes = p.a_chunk + p.b_chunk;
  uint64_t* bars = reinterpret_cast<uint64_t*>(probe_smem + static_cast<size_t>(p.stages) * stage_bytes);   // full[S], empty[S]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * p.stages);
  if (threadIdx.x == 0) {
    for (int s = 0; s < 2 * p.stages; ++s) mbar_init(smem_u32(&bars[s]), 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  __syncthreads();
  const uint8_t* a = p.a + p.a_per_cta * blockIdx.x;
  int done = 0;       // chunks whose copies were issued (producer) / seen complete (consumer)
  if (threadIdx.x == 0) {
    for (int i = 0; i < p.n_chunks; ++i, ++done) {
      const int s = i % p.stages;
      if (i >= p.stages &&
          !mbar_wait_bounded(smem_u32(&bars[p.stages + s]), ((i / p.stages) & 1) ^ 1, abort_flag, p.wait_cycles))
        break;
      const uint32_t full = smem_u32(&bars[s]);
      mbar_expect_tx(full, static_cast<uint32_t>(stage_bytes));
      const uint32_t dst = smem_u32(probe_smem + static_cast<size_t>(s) * stage_bytes);
      for (int off = 0; off < p.a_chunk; off += 16384)
        bulk_load_1d(dst + off, a + static_cast<long long>(i) * p.a_chunk + off, min(16384, p.a_chunk - off), full);
      if (p.b_chunk) bulk_load_1d(dst + p.a_chunk, p.b + (static_cast<long long>(i) * p.b_chunk) % p.b_span, p.b_chunk, full);
    }
  } else if (threadIdx.x == 32) {
    for (int i = 0; i < p.n_chunks; ++i, ++done) {
      const int s = i % p.stages;
      if (!mbar_wait_bounded(smem_u32(&bars[s]), (i / p.stages) & 1, abort_flag, p.wait_cycles)) break;
      mbar_arrive(smem_u32(&bars[p.stages + s]));
    }
  }
  __syncthreads();
  if (*abort_flag) {
    // a wait ran out: give copies in flight time to land before the shared memory is released
    if (threadIdx.x == 0) {
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {
      }
      if (p.status) atomicOr(p.status, 8);
    }
    __syncthreads();
  }
}

}  // namespace dkv
