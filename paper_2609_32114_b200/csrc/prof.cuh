// Optional phase timestamps for kernel tuning.  Compiled in only with -DHA_LA_PROFILE_PHASES (the developer build
// `python -m paper_2609_32114_b200.build --profile`, read back by `python -m paper_2609_32114_b200.prof_phases`);
// in the normal build every macro expands to nothing.
#pragma once
#ifdef HA_LA_PROFILE_PHASES
#define HA_PROF_DECL(name)                                                                        \
  static __device__ long long g_prof_##name[1024];                                                \
  extern "C" int ha_la_debug_read_prof_##name(long long* out) {                                   \
    return cudaMemcpyFromSymbol(out, g_prof_##name, sizeof(long long) * 1024) == cudaSuccess ? 0 : 4; \
  }
#ifdef HA_LA_PROFILE_COARSE
#define HA_PROF(name, slot) do { } while (0)
#else
#define HA_PROF(name, slot)                                                            \
  do {                                                                                 \
    if (threadIdx.x == 0 && blockIdx.x == 0 && (slot) < 1024) g_prof_##name[slot] = clock64(); \
  } while (0)
#endif
// the same for a thread of the caller's choice (CTA 0 only)
#define HA_PROF_ANY(name, slot)                                                        \
  do {                                                                                 \
    if (blockIdx.x == 0 && (slot) < 1024) g_prof_##name[slot] = clock64();             \
  } while (0)
// records the SM id of CTA `blockIdx.x` at slot base + blockIdx.x % count
#define HA_PROF_SMID(name, base, count)                                                \
  do {                                                                                 \
    if (threadIdx.x == 0) {                                                            \
      unsigned smid_;                                                                  \
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid_));                               \
      g_prof_##name[(base) + blockIdx.x % (count)] = smid_;                            \
    }                                                                                  \
  } while (0)
// stores the global nanosecond timer at `slot` (any CTA; the caller picks who records)
#define HA_PROF_GT(name, slot)                                                         \
  do {                                                                                 \
    unsigned long long gt_;                                                            \
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_));                            \
    if ((slot) >= 0 && (slot) < 1024) g_prof_##name[slot] = (long long)gt_;            \
  } while (0)
#else
#define HA_PROF_GT(name, slot) do { } while (0)
#define HA_PROF_ANY(name, slot) do { } while (0)
#define HA_PROF_SMID(name, base, count) do { } while (0)
#define HA_PROF_DECL(name)
#define HA_PROF(name, slot) do { } while (0)
#endif
