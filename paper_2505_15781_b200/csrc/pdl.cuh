// Programmatic dependent launch: a kernel launched with the stream-serialization
// attribute may start before its predecessor in the stream has finished.
// pdl_launch() lets the successor start early; pdl_wait() blocks until every
// predecessor has completed and its writes are visible.  Both are no-ops for a
// kernel launched without the attribute.
#pragma once

namespace dkv {

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Optional timeline trace (diagnostics): when a buffer has been set, block 0 of
// every kernel records when it started and when its predecessor's data was
// ready (nanoseconds of the global timer).  The difference between the two is
// how far ahead of its dependency the kernel was launched.
struct TraceRec {
  unsigned long long t_enter, t_ready;
  int kernel_id, pad;
};
__device__ TraceRec* g_trace_buf = nullptr;
__device__ int g_trace_cap = 0;
__device__ unsigned int g_trace_n = 0;

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool trace_on() {
  return g_trace_buf != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
}
__device__ __forceinline__ void trace_store(int kernel_id, unsigned long long t_enter) {
  const unsigned int i = atomicAdd(&g_trace_n, 1u);
  if (i < static_cast<unsigned int>(g_trace_cap)) {
    TraceRec r;
    r.t_enter = t_enter;
    r.t_ready = global_timer_ns();
    r.kernel_id = kernel_id;
    r.pad = 0;
    g_trace_buf[i] = r;
  }
}

// the common case: nothing useful to do before the predecessor's data is ready
__device__ __forceinline__ void pdl_enter(int kernel_id = 0) {
  const bool tr = threadIdx.x == 0 && trace_on();   // (one thread reads the switch, a word in global memory)
  const unsigned long long t0 = tr ? global_timer_ns() : 0ull;
  pdl_launch();
  pdl_wait();
  if (tr) trace_store(kernel_id, t0);
}

}  // namespace dkv
