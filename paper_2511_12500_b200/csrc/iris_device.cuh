// Device-side primitives: pointer translation, ordered loads/stores/atomics, bounded waits.
// These are the CUDA counterparts of the paper's device API (Table 3): every remote operation is
// "translate the pointer, then do the memory operation" (Section 3.3).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstdint>

#include "iris_internal.h"

namespace iris {

// Listing 1 (__translate): offset inside from_rank's heap, re-based on to_rank's heap.
__device__ __forceinline__ uint64_t translate(uint64_t ptr, int from_rank, int to_rank, const HeapTable& t) {
  return t.base[to_rank] + (ptr - t.base[from_rank]);
}

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// ---- ordered 32-bit accesses -------------------------------------------------------------
__device__ __forceinline__ int32_t ld_acquire_gpu(const int32_t* p) {
  int32_t v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int32_t ld_relaxed_gpu(const int32_t* p) {
  int32_t v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu(int32_t* p, int32_t v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Ready flags: gpu scope while every slot lives on this device, system scope when the heap spans processes or
// devices (the writer's release has to reach a reader on another GPU, and the reader's acquire has to see it).
__device__ __forceinline__ void st_release_flag(int32_t* p, int32_t v, int sys) {
  if (sys) asm volatile("st.release.sys.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
  else st_release_gpu(p, v);
}
__device__ __forceinline__ int32_t ld_acquire_flag(const int32_t* p, int sys) {
  if (!sys) return ld_acquire_gpu(p);
  int32_t v;
  asm volatile("ld.acquire.sys.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
// Orders generic-proxy accesses against async-proxy (TMA / bulk copy) accesses.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

#define IRIS_ATOM_CASE(SEMV, SCOPEV, SEMS, SCOPES)                                                          \
  if (sem == SEMV && scope == SCOPEV) {                                                                     \
    if (IS_CAS)                                                                                             \
      asm volatile("atom." SEMS "." SCOPES ".global.cas.b32 %0, [%1], %2, %3;"                              \
                   : "=r"(old) : "l"(p), "r"(cmp), "r"(val) : "memory");                                    \
    else                                                                                                    \
      asm volatile("atom." SEMS "." SCOPES ".global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); \
    return old;                                                                                             \
  }

// atomic add / cas with run-time memory order and scope (Table 3 note: sem x scope).
template <bool IS_CAS>
__device__ __forceinline__ int32_t atomic_rmw(int32_t* p, int32_t cmp, int32_t val, int sem, int scope) {
  int32_t old = 0;
  IRIS_ATOM_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_BLOCK, "relaxed", "cta")
  IRIS_ATOM_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_GPU, "relaxed", "gpu")
  IRIS_ATOM_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_SYS, "relaxed", "sys")
  IRIS_ATOM_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_BLOCK, "acquire", "cta")
  IRIS_ATOM_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_GPU, "acquire", "gpu")
  IRIS_ATOM_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_SYS, "acquire", "sys")
  IRIS_ATOM_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_BLOCK, "release", "cta")
  IRIS_ATOM_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_GPU, "release", "gpu")
  IRIS_ATOM_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_SYS, "release", "sys")
  IRIS_ATOM_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_BLOCK, "acq_rel", "cta")
  IRIS_ATOM_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_GPU, "acq_rel", "gpu")
  IRIS_ATOM_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_SYS, "acq_rel", "sys")
  return old;
}
#undef IRIS_ATOM_CASE

__device__ __forceinline__ int32_t cas_release_gpu(int32_t* p, int32_t cmp, int32_t val) {
  int32_t old;
  asm volatile("atom.release.gpu.global.cas.b32 %0, [%1], %2, %3;" : "=r"(old) : "l"(p), "r"(cmp), "r"(val) : "memory");
  return old;
}
__device__ __forceinline__ int32_t cas_acquire_gpu(int32_t* p, int32_t cmp, int32_t val) {
  int32_t old;
  asm volatile("atom.acquire.gpu.global.cas.b32 %0, [%1], %2, %3;" : "=r"(old) : "l"(p), "r"(cmp), "r"(val) : "memory");
  return old;
}

// ---- 16-byte global accesses ---------------------------------------------------------------
__device__ __forceinline__ uint4 ld_global_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_global_v4(void* p, const uint4& v) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---- consumer arithmetic: two packed 16-bit elements, summed in fp32, rounded once (RNE) ----------
template <bool BF16>
__device__ __forceinline__ uint32_t add2(uint32_t c, uint32_t b) {
  if (BF16) {
    const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&c));
    const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b));
    __nv_bfloat162 r = __floats2bfloat162_rn(x.x + y.x, x.y + y.y);
    return *reinterpret_cast<uint32_t*>(&r);
  } else {
    const float2 x = __half22float2(*reinterpret_cast<const __half2*>(&c));
    const float2 y = __half22float2(*reinterpret_cast<const __half2*>(&b));
    __half2 r = __floats2half2_rn(x.x + y.x, x.y + y.y);
    return *reinterpret_cast<uint32_t*>(&r);
  }
}

// ---- device-detected errors ------------------------------------------------------------------
// First reporter wins; the record is {code, kernel, block, tile, slot, seen, expected, 0}.
__device__ __forceinline__ void report_timeout(int32_t* status, int kernel, int tile, int slot, int seen, int expected) {
  if (atomicCAS(status, 0, IRIS_ERR_TIMEOUT) == 0) {
    status[1] = kernel;
    status[2] = (int)blockIdx.x;
    status[3] = tile;
    status[4] = slot;
    status[5] = seen;
    status[6] = expected;
    __threadfence();
  }
}

}  // namespace iris
