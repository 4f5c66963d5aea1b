// Shared device helpers of the Virtual-Expert MoE-layer kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace swapmoe {

constexpr int kMaxE = 256;       // experts per layer
constexpr int kMaxSlots = 64;    // K + spare slots
constexpr int kMaxTopK = 4;
constexpr int kTokTile = 32;     // tokens per CTA in the router and permute kernels
constexpr int kSegAlign = 128;   // slot segments start at multiples of this many rows

typedef __nv_bfloat16 bf16;

// One GEMM work item: a block of rows of one slot's segment in the padded workspace.
struct __align__(16) TileDesc {
  int32_t phys;   // arena entry holding the slot's weights
  int32_t row0;   // first row in the padded workspace
  int32_t rows;   // valid rows (<= tile height)
  int32_t slot;   // logical slot
};

__device__ __forceinline__ void load4(const float* p, float v[4]) {
  const float4 q = *reinterpret_cast<const float4*>(p);
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void load4(const bf16* p, float v[4]) {
  const uint2 q = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(q.x << 16);
  v[1] = __uint_as_float(q.x & 0xFFFF0000u);
  v[2] = __uint_as_float(q.y << 16);
  v[3] = __uint_as_float(q.y & 0xFFFF0000u);
}
__device__ __forceinline__ void store4(float* p, const float v[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ void store4(bf16* p, const float v[4]) {
  *reinterpret_cast<uint2*>(p) = make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
}
__device__ __forceinline__ void store8(float* p, const float v[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8(bf16* p, const float v[8]) {
  *reinterpret_cast<uint4*>(p) = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]),
                                            pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may
// start while its predecessor is still running; it must execute pdl_wait() before it reads or
// writes any global memory the predecessors touch.  pdl_trigger() lets the NEXT kernel's
// blocks be scheduled (they stop at their own pdl_wait()).  Both are no-ops otherwise.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Timeline tracing (built only with -DSWAPMOE_TRACE, see build.py): a kernel stamps %globaltimer
// into g_trace[kernel][CTA][slot]; swapmoe_debug_trace copies the table out.  Kernel ids: 0 router,
// 1 permute, 2 grouped GEMM-1, 3 grouped GEMM-2.  SWAPMOE_STAMP is called by ONE thread of a CTA.
constexpr int kTraceKernels = 4, kTraceCtas = 160, kTraceSlots = 16;
#ifdef SWAPMOE_TRACE
static __device__ unsigned long long g_trace[kTraceKernels][kTraceCtas][kTraceSlots];
#define SWAPMOE_STAMP(kern, slot)                                                     \
  do {                                                                                \
    if (blockIdx.x < kTraceCtas) {                                                    \
      unsigned long long t_;                                                          \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)::"memory");                \
      g_trace[kern][blockIdx.x][slot] = t_;                                           \
    }                                                                                 \
  } while (0)
#else
#define SWAPMOE_STAMP(kern, slot) do { } while (0)
#endif

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace swapmoe
