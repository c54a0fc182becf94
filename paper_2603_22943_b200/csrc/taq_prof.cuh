// Optional per-CTA phase stamps for the tensor-core kernels.  Compiled in only with -DTAQ_PROFILE (the normal build
// contains none of it): every CTA owns 128 slots of a caller-provided buffer; TAQ_PROF(slot) stores the SM clock,
// TAQ_GPROF(slot) the global nanosecond timer.  Every kernel file has its own buffer pointer, registered with
// taq_profile_set_<name>() (TAQ_PROF_DEFINE(name) at file scope creates both).
#pragma once
#ifdef TAQ_PROFILE
#define TAQ_PROF_DEFINE(name)                                                                                         \
    static __device__ unsigned long long* g_profile = nullptr;                                                        \
    extern "C" int taq_profile_set_##name(unsigned long long* buf_dev) { return (int)cudaMemcpyToSymbol(g_profile, &buf_dev, sizeof(buf_dev)); }
#define TAQ_PROF_INIT                                                                                                 \
    unsigned long long* prof_base = g_profile;                                                                  \
    if (prof_base) prof_base += (size_t)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) * 128;
#define TAQ_PROF(slot) do { if (prof_base) prof_base[(slot)] = (unsigned long long)clock64(); } while (0)
#define TAQ_GPROF(slot)                                                       \
    do {                                                                      \
        if (prof_base) {                                                      \
            unsigned long long t_;                                            \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));            \
            prof_base[(slot)] = t_;                                           \
        }                                                                     \
    } while (0)
#else
#define TAQ_PROF_DEFINE(name)
#define TAQ_PROF_INIT
#define TAQ_PROF(slot) do { } while (0)
#define TAQ_GPROF(slot) do { } while (0)
#endif
