// Memory access helpers (relaxed gpu-scope / system-scope loads and stores), error reporting,
// statistics and the debug profile clock of the persistent search kernel.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

// ------------------------------------------------------------------------------------------
// memory access helpers: query/cache state is shared between SMs, so it is always read and
// written at the L2 (relaxed, gpu scope); host-mapped words use system scope.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ u32 ld_u32(const u32 *p) {
  u32 v; asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ u64 ld_u64(const u64 *p) {
  u64 v; asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void st_u32(u32 *p, u32 v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_u64(u64 *p, u64 v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint4 ld_v4(const u32 *p) {
  uint4 v;
  asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ld_sys_v4(const u32 *p) {
  uint4 v;
  asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_sys_u32(u32 *p, u32 v) {
  asm volatile("st.relaxed.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_sys_u64(u64 *p, u64 v) {
  asm volatile("st.relaxed.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ u64 globaltimer() {
  u64 t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t;
}
__device__ __forceinline__ u32 lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ u32 hash32(u32 v) { v *= 0x9E3779B1u; v ^= v >> 15; return v * 0x85EBCA77u; }

// ------------------------------------------------------------------------------------------
// errors and statistics
// ------------------------------------------------------------------------------------------
__device__ __noinline__ void raise(const Ctx &c, u32 status, u32 a = 0, u32 b = 0, u32 d = 0, u32 e = 0) {
  if (atomicCAS(&c.ctl->status, 0u, status) == 0u) {
    c.ctl->dbg[0] = a; c.ctl->dbg[1] = b; c.ctl->dbg[2] = d; c.ctl->dbg[3] = e;
    c.ctl->dbg[4] = blockIdx.x; c.ctl->dbg[5] = threadIdx.x;
    __threadfence();
  }
  st_u32(&c.ctl->stop, 2u);
}
// warp-uniform variants: every lane gets lane 0's view, and the shuffle is a convergence point
__device__ __forceinline__ bool warp_stopped(const Ctx &c) {
  return __shfl_sync(0xffffffffu, ld_u32(&c.ctl->stop), 0) != 0u;
}
__device__ __forceinline__ u32 uld(const u32 *p) { return __shfl_sync(0xffffffffu, ld_u32(p), 0); }
__device__ __forceinline__ void stat_add(const Ctx &c, u32 idx, u32 v) {
  if (v) atomicAdd((unsigned long long *)&c.ctl->stats[idx], (unsigned long long)v);
}
// Debug profile: charge the time since `t` to stats[idx] and restart the clock.
__device__ __forceinline__ void phase_mark(const Ctx &c, u64 &t, u32 idx, u32 lane) {
  if (!c.prof) return;
  const u64 now = globaltimer();
  if (lane == 0) atomicAdd((unsigned long long *)&c.ctl->stats[idx], now - t);
  t = now;
}

}  // namespace gorio
