// Shared device helpers for the LSP decode kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace lsp {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(bf16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }

// Running state of the vocab reduction for one row: largest logit m1 (at id i1, lowest id on ties),
// largest logit among the other ids m2, and s = sum_v exp(z_v - m1).  Eq. 1's margin is m1 - m2 and the
// softmax max-probability is 1 / s.
struct Top2 {
  float m1;
  int i1;
  float m2;
  float s;
};

__device__ __forceinline__ Top2 top2_empty() { return Top2{-INFINITY, 0x7fffffff, -INFINITY, 0.f}; }

__device__ __forceinline__ void top2_push(Top2& t, float z, int id) {
  // ids arrive in ascending order within a thread, so a strict test keeps the lowest id on ties.
  if (z > t.m1) {
    t.s = t.s * __expf(t.m1 - z) + 1.f;
    t.m2 = t.m1;
    t.m1 = z;
    t.i1 = id;
  } else {
    t.s += __expf(z - t.m1);
    t.m2 = fmaxf(t.m2, z);
  }
}

__device__ __forceinline__ Top2 top2_merge(const Top2& a, const Top2& b) {
  const bool b_wins = (b.m1 > a.m1) || (b.m1 == a.m1 && b.i1 < a.i1);
  const Top2& w = b_wins ? b : a;
  const Top2& l = b_wins ? a : b;
  Top2 r;
  r.m1 = w.m1;
  r.i1 = w.i1;
  r.m2 = fmaxf(w.m2, l.m1);
  // exp(-inf - x) = 0 handles an empty side; guard the (-inf) - (-inf) case
  r.s = w.s + ((l.m1 == -INFINITY) ? 0.f : l.s * __expf(l.m1 - w.m1));
  return r;
}

__device__ __forceinline__ Top2 top2_shfl_xor(const Top2& t, int mask) {
  Top2 o;
  o.m1 = __shfl_xor_sync(0xffffffffu, t.m1, mask);
  o.i1 = __shfl_xor_sync(0xffffffffu, t.i1, mask);
  o.m2 = __shfl_xor_sync(0xffffffffu, t.m2, mask);
  o.s = __shfl_xor_sync(0xffffffffu, t.s, mask);
  return o;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Programmatic dependent launch.  Every kernel of a step is launched with the programmatic-serialisation attribute
// (launch_k below): it lets the next kernel's blocks be scheduled, and run their set-up, while the previous kernel
// drains.  pdl_begin() is the first statement of every kernel: it releases the following launch at once (that launch
// waits itself) and then waits until the preceding kernel has completed and its writes are visible.  Kernels with a
// set-up that touches no global memory call pdl_release() first and pdl_wait() after the set-up.  Both are no-ops in a
// kernel launched without the attribute.
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_begin() { pdl_release(); pdl_wait(); }

// Launches kernel(args...) on stream; pdl = 1 adds the programmatic-serialisation attribute.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(int pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                            Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// The same with thread block clusters of `cluster` CTAs along x (0 or 1 = none).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(int pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                            int cluster, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// Per-step descriptor the host uploads before each pass (int32 arrays of batch+1 entries each).
struct StepDesc {
  const int* F;        // cache length per sequence
  const int* pend;     // pending block length
  const int* N;        // active (masked) positions
  const int* row_off;  // first packed row of the sequence in this pass   [batch+1]
  const int* head_off; // first packed head row (masked rows only)        [batch+1]
  const int* Fp;       // token boundary (first masked position)
  const int* Lc;       // lengths to commit (commit kernel only)
};

}  // namespace lsp
