// Global-memory vector loads and stores with explicit cache-hint sets, as inline PTX.
//
// A "policy" picks the qualifiers on ld.global / st.global. Streaming kernels touch every byte
// once, so the hints only decide how much of L1/L2 the stream is allowed to occupy:
//   0  ld.global                    st.global                      (default caching)
//   1  ld.global.nc                 st.global                      (read-only data path)
//   2  ld.global.cs                 st.global.cs                   (evict-first streaming)
//   3  ld.global.L1::no_allocate    st.global.cs
//   4  ld.global.L1::no_allocate + L2 evict_first policy on loads and stores
//   5  loads as 4 (read-once data leaves L2 first), plain st.global (written data stays)
//   6  loads as 4, stores with an L2 evict_last policy (written data is kept for the next kernel)
//   7  loads as 4; stores in two phases: L2 evict_first while the kernel is still consuming what
//      its predecessor left in L2 (its own output must not push those lines out), plain
//      st.global afterwards (so that the kernel's last-written lines are what it leaves behind)
//   8  as 7 with L2 evict_last in the second phase (the consumer's evict_first loads demote the
//      lines again once they have been read)
// 16-byte accesses are .v4.b32; 32-byte accesses are the 256-bit .v8.b32 form of sm_100.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace streamops {

constexpr int kNumPolicies = 9;

template <int VB> struct Vec;
template <> struct alignas(16) Vec<16> { uint32_t w[4]; };
template <> struct alignas(32) Vec<32> { uint32_t w[8]; };

__device__ __forceinline__ uint64_t make_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t make_evict_last_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// The L2 policy operands a kernel needs for its policy: one for loads, one for stores, and for
// the two-phase policy the one its stores switch to after the first phase.
struct L2Policies { uint64_t ld, st, st_late; };
template <int POL> __device__ __forceinline__ L2Policies make_l2_policies() {
    L2Policies p{0, 0, 0};
    if constexpr (POL >= 4) p.ld = make_evict_first_policy();
    if constexpr (POL == 4 || POL == 7 || POL == 8) p.st = p.ld;
    if constexpr (POL == 6) p.st = make_evict_last_policy();
    if constexpr (POL == 8) p.st_late = make_evict_last_policy();
    return p;
}

#define STREAMOPS_LD16(QUAL, TAIL, ...)                                                          \
    asm volatile("ld.global" QUAL ".v4.b32 {%0,%1,%2,%3}, [%4]" TAIL ";"                         \
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3])                        \
                 : "l"(p) __VA_ARGS__)
#define STREAMOPS_LD32(QUAL, TAIL, ...)                                                          \
    asm volatile("ld.global" QUAL ".v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8]" TAIL ";"             \
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]),         \
                   "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])                                      \
                 : "l"(p) __VA_ARGS__)
#define STREAMOPS_ST16(QUAL, TAIL, ...)                                                          \
    asm volatile("st.global" QUAL ".v4.b32 [%0], {%1,%2,%3,%4}" TAIL ";"                         \
                 :: "l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]) __VA_ARGS__       \
                 : "memory")
#define STREAMOPS_ST32(QUAL, TAIL, ...)                                                          \
    asm volatile("st.global" QUAL ".v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8}" TAIL ";"             \
                 :: "l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]),     \
                    "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7]) __VA_ARGS__                            \
                 : "memory")

template <int POL>
__device__ __forceinline__ void ldg(Vec<16> &v, const void *p, uint64_t l2pol) {
    if constexpr (POL == 0) STREAMOPS_LD16("", "");
    else if constexpr (POL == 1) STREAMOPS_LD16(".nc", "");
    else if constexpr (POL == 2) STREAMOPS_LD16(".cs", "");
    else if constexpr (POL == 3) STREAMOPS_LD16(".L1::no_allocate", "");
    else STREAMOPS_LD16(".L1::no_allocate.L2::cache_hint", ", %5", , "l"(l2pol));   // 4, 5, 6
}
template <int POL>
__device__ __forceinline__ void ldg(Vec<32> &v, const void *p, uint64_t l2pol) {
    if constexpr (POL == 0) STREAMOPS_LD32("", "");
    else if constexpr (POL == 1) STREAMOPS_LD32(".nc", "");
    else if constexpr (POL == 2) STREAMOPS_LD32(".cs", "");
    else if constexpr (POL == 3) STREAMOPS_LD32(".L1::no_allocate", "");
    else STREAMOPS_LD32(".L1::no_allocate.L2::cache_hint", ", %9", , "l"(l2pol));
}
template <int POL>
__device__ __forceinline__ void stg(void *p, const Vec<16> &v, uint64_t l2pol) {
    if constexpr (POL == 0 || POL == 1 || POL == 5) STREAMOPS_ST16("", "");
    else if constexpr (POL == 2 || POL == 3) STREAMOPS_ST16(".cs", "");
    else STREAMOPS_ST16(".L2::cache_hint", ", %5", , "l"(l2pol));
}
template <int POL>
__device__ __forceinline__ void stg(void *p, const Vec<32> &v, uint64_t l2pol) {
    if constexpr (POL == 0 || POL == 1 || POL == 5) STREAMOPS_ST32("", "");
    else if constexpr (POL == 2 || POL == 3) STREAMOPS_ST32(".cs", "");
    else STREAMOPS_ST32(".L2::cache_hint", ", %9", , "l"(l2pol));
}

// Views of a vector's words as elements. A double is a register pair, so these are free.
template <typename T> struct Lanes;
template <> struct Lanes<double> {
    static __device__ __forceinline__ double get(const uint32_t *w, int i) {
        return __hiloint2double((int)w[2 * i + 1], (int)w[2 * i]);
    }
    static __device__ __forceinline__ void set(uint32_t *w, int i, double v) {
        w[2 * i] = (uint32_t)__double2loint(v);
        w[2 * i + 1] = (uint32_t)__double2hiint(v);
    }
};
template <> struct Lanes<float> {
    static __device__ __forceinline__ float get(const uint32_t *w, int i) { return __uint_as_float(w[i]); }
    static __device__ __forceinline__ void set(uint32_t *w, int i, float v) { w[i] = __float_as_uint(v); }
};

}  // namespace streamops
