// Debug builds (-DAPEX_TIMELINE, relocatable device code) record time stamps of the expert-FFN kernels.
#ifndef APEX_TIMELINE_CUH
#define APEX_TIMELINE_CUH
#ifdef APEX_TIMELINE
namespace apex {
extern __device__ unsigned long long g_timeline[1024 * 16];
__device__ __forceinline__ unsigned long long globaltimer_ns_raw() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
}  // namespace apex
#endif
#endif  // APEX_TIMELINE_CUH
