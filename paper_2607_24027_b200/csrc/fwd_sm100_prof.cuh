// Development instrumentation of the fused tcgen05 kernel.  Included by fwd_sm100.cu only when the
// library is built with -DSOL_PROFILE (per-role wait accounting) or -DSOL_ITEMTRACE (a timeline of the
// first work items of CTA 0 in an otherwise unchanged build); the product build sees none of it.
#pragma once

#include <cuda_runtime.h>

namespace sol {
namespace prof {

#ifdef SOL_PROFILE
// How many cycles each role spends in each kind of wait.  Slot meaning is listed next to every use in
// the kernel; read back with sol_attn_debug_profile().
constexpr int kProfCtas = 512, kProfRoles = 4, kProfSlots = 12;
__device__ long long g_prof[kProfCtas * kProfRoles * kProfSlots];
struct Prof {
  long long v[kProfSlots];
  long long t0;
  __device__ Prof() {
    for (int i = 0; i < kProfSlots; ++i) v[i] = 0;
    t0 = clock64();
  }
  __device__ void flush(int role) {
    v[kProfSlots - 1] = clock64() - t0;
    if (blockIdx.x < kProfCtas)
      for (int i = 0; i < kProfSlots; ++i) g_prof[(blockIdx.x * kProfRoles + role) * kProfSlots + i] = v[i];
  }
};
#endif

#ifdef SOL_ITEMTRACE
// [item][slot] = clock64() for the first work items of CTA 0; [cta] = {start, router end, items, softmax end}
constexpr int kItItems = 96, kItSlots = 16;
__device__ long long g_itrace[kItItems * kItSlots];
__device__ long long g_ctatrace[256 * 4];
__device__ __forceinline__ long long gtimer() {
  long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
#endif

}  // namespace prof
}  // namespace sol

#ifdef SOL_PROFILE
#define SOL_WAIT(bar, parity, slot) \
  ([&]() { const long long t_ = clock64(); const bool ok_ = mbar_wait((bar), (parity), &sm.abort_flag, wait_limit); prof.v[slot] += clock64() - t_; return ok_; }())
#define PROF_DECL prof::Prof prof;
#define PROF_COUNT(slot) (++prof.v[slot])
#define PROF_FLUSH(role) prof.flush(role)
#define PROF_ACC(slot) (&prof.v[slot])
#define PROF_T0 const long long prof_t0 = clock64();
#define PROF_ADD(slot) prof.v[slot] += clock64() - prof_t0;
// Debug builds only: copies the per-CTA, per-role wait-cycle counters of the last launch to the host.
extern "C" int sol_attn_debug_profile(long long* host_out, int n_values) {
  const size_t total = sizeof(long long) * sol::prof::kProfCtas * sol::prof::kProfRoles * sol::prof::kProfSlots;
  const size_t want = sizeof(long long) * (size_t)n_values;
  return (int)cudaMemcpyFromSymbol(host_out, sol::prof::g_prof, want < total ? want : total);
}
#endif

#ifdef SOL_ITEMTRACE
#define ITRACE(item, slot) \
  do { if (blockIdx.x == 0 && (item) < prof::kItItems) prof::g_itrace[(item) * prof::kItSlots + (slot)] = clock64(); } while (0)
#define ITRACE_VAL(item, slot, val) \
  do { if (blockIdx.x == 0 && (item) < prof::kItItems) prof::g_itrace[(item) * prof::kItSlots + (slot)] = (val); } while (0)
#define CTATRACE(slot, val) \
  do { if (blockIdx.x < 256) prof::g_ctatrace[blockIdx.x * 4 + (slot)] = (val); } while (0)
extern "C" int sol_attn_debug_itemtrace(long long* host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, sol::prof::g_itrace,
                                   sizeof(long long) * sol::prof::kItItems * sol::prof::kItSlots);
}
extern "C" int sol_attn_debug_ctatrace(long long* host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, sol::prof::g_ctatrace, sizeof(long long) * 256 * 4);
}
#endif
