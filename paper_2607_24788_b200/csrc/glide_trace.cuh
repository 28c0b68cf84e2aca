// Debug-only per-warp event trace of the streaming decode kernel.  Nothing here is part of a normal build:
// without -DGLIDE_TRACE the macro expands to nothing and the export below does not exist.
#pragma once

#ifdef GLIDE_TRACE
namespace glide {
__device__ unsigned long long *g_stream_trace = nullptr;   // [warps][64] of (code << 56 | globaltimer ns)
}
#define GLIDE_TRACE_DECL int trace_n = 0
#define GLIDE_TRACE_EVENT(code)                                                                        \
  do {                                                                                                 \
    if (glide::g_stream_trace && (threadIdx.x & 31) == 0 && trace_n < 64) {                            \
      unsigned long long now;                                                                          \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));                                          \
      glide::g_stream_trace[(size_t(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 64 + trace_n++] = \
          (static_cast<unsigned long long>(code) << 56) | (now & 0x00ffffffffffffffull);               \
    }                                                                                                  \
  } while (0)
// host side: point the kernels at a device buffer of [grid * warps][64] 64-bit words (nullptr switches tracing off)
extern "C" int glide_debug_set_stream_trace(void *dev_buf) {
  return cudaMemcpyToSymbol(glide::g_stream_trace, &dev_buf, sizeof(void *)) == cudaSuccess ? 0 : 6;
}
#else
#define GLIDE_TRACE_DECL do { } while (0)
#define GLIDE_TRACE_EVENT(code) do { } while (0)
#endif
