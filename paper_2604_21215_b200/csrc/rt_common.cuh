// Shared device helpers of the RT prefill kernels (sm_100a).
#pragma once
#include <utility>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rt.h"

namespace rt {

constexpr int kHeadDim = 64;
constexpr float kLog2e = 1.4426950408889634f;

// First bytes of every workspace: device status and the grid-barrier words.
struct SyncArea {
  int status;               // rt_status written by a kernel whose bounded wait ran out
  unsigned int abort_flag;  // set together with status; every waiter leaves when it sees it
  unsigned int bar_count;   // barrier arrivals since the start of the API call (zeroed once per call)
  unsigned int pad0;
  // time CTA 0 spent in each phase of the leaf kernel since the start of the API call, in ns:
  // [2*i] = work of phase i (A..E), [2*i+1] = wait at the barrier that ends it
  unsigned long long phase_ns[10];
  unsigned int pad[40];
};
static_assert(sizeof(SyncArea) == 256, "SyncArea is one 256-byte block");

// ---- storage type <-> float ------------------------------------------------------------
template <typename T> struct Vec4;   // 4 consecutive elements
template <> struct Vec4<float> {
  float4 v;
  __device__ __forceinline__ void to_float(float (&f)[4]) const { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
};
template <> struct Vec4<__nv_bfloat16> {
  uint2 v;
  __device__ __forceinline__ void to_float(float (&f)[4]) const {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
  }
};

__device__ __forceinline__ float to_f(float a) { return a; }
__device__ __forceinline__ float to_f(__nv_bfloat16 a) { return __bfloat162float(a); }
template <typename T> __device__ __forceinline__ T from_f(float a);
template <> __device__ __forceinline__ float from_f<float>(float a) { return a; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float a) { return __float2bfloat16_rn(a); }
// value after one round trip through the storage type
template <typename T> __device__ __forceinline__ float round_T(float a) { return to_f(from_f<T>(a)); }

// gains: NULL pointer = ones
template <typename T> __device__ __forceinline__ float gain_at(const T* g, int i) { return g ? to_f(g[i]) : 1.0f; }

// ---- cache-bypassing loads for data another CTA of the same kernel has just written -----
__device__ __forceinline__ float ldcg_f(const float* p) { return __ldcg(p); }
__device__ __forceinline__ float4 ldcg_f4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float ldcg_T(const float* p) { return __ldcg(p); }
__device__ __forceinline__ float ldcg_T(const __nv_bfloat16* p) {
  unsigned short u = __ldcg(reinterpret_cast<const unsigned short*>(p));
  return __uint_as_float(static_cast<unsigned>(u) << 16);
}
__device__ __forceinline__ float2 ldcg_T2(const float* p) { return __ldcg(reinterpret_cast<const float2*>(p)); }
__device__ __forceinline__ float2 ldcg_T2(const __nv_bfloat16* p) {
  unsigned u = __ldcg(reinterpret_cast<const unsigned*>(p));
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}

// ---- warp reductions -------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Sums 32 per-lane values across the warp with 31 shuffles: afterwards lane i holds the
// warp-wide sum of a[i] in a[0].
__device__ __forceinline__ void warp_transpose_sum32(float (&a)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < off; ++i) {
      const float send = upper ? a[i] : a[i + off];
      const float keep = upper ? a[i + off] : a[i];
      a[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
}

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add_u32(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // every device-side wait gives up after 2 s

// Barrier over all CTAs of a cooperative launch.  `target` is this CTA's running arrival
// target (starts at the arrivals counted before this launch).  Returns false when
// the wait ran out or another CTA reported a failure: the caller must then return at once.
__device__ __forceinline__ bool grid_barrier(SyncArea* s, unsigned& target, unsigned n_ctas, int* s_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    target += n_ctas;
    __threadfence();
    red_release_add_u32(&s->bar_count, 1u);
    int ok = 1;
    unsigned spins = 0;
    unsigned long long t_start = 0;
    while (ld_acquire_u32(&s->bar_count) < target) {
      if ((++spins & 1023u) == 0) {
        if (*reinterpret_cast<volatile unsigned*>(&s->abort_flag)) { ok = 0; break; }
        const unsigned long long now = globaltimer_ns();
        if (t_start == 0) t_start = now;
        else if (now - t_start > kWaitLimitNs) {
          s->status = RT_ERR_TIMEOUT;
          __threadfence();
          atomicExch(&s->abort_flag, 1u);
          ok = 0;
          break;
        }
      }
    }
    *s_flag = ok;
  }
  __syncthreads();
  return *s_flag != 0;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

// ---- programmatic dependent launch ------------------------------------------------------------
// A kernel launched with launch_chained(..., true) may be scheduled while its predecessor in the stream is still
// running; it must call grid_dep_sync() before it reads or writes anything the predecessor touches, in every CTA and
// before any early return (a grid whose CTAs left without waiting would count as finished too early for ITS
// successor).  Launched the ordinary way, both calls do nothing.
__device__ __forceinline__ void grid_dep_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // let the successor be scheduled behind us
  asm volatile("griddepcontrol.wait;" ::: "memory");                   // until the predecessor's writes are visible
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool chained,
                                  Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = chained ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace rt
