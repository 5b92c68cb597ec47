// Small pieces shared by the tridiagonalisation kernels: thread-private traffic with tensor memory
// and the two reciprocals that sit on every step's critical path.
#pragma once

#include <cstdint>

#include "eosq_sm100.cuh"

namespace eosq {

// 16 columns of the thread's lane; the wait carries the registers, so that no use of them can be
// scheduled ahead of it.
__device__ __forceinline__ void tt_wait16(uint32_t (&r)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                   "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :
                 : "memory");
}
__device__ __forceinline__ void tt_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        :
        : "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ double tt_get(const uint32_t (&r)[16], int e) {
    return __hiloint2double(static_cast<int>(r[2 * e + 1]), static_cast<int>(r[2 * e]));
}
__device__ __forceinline__ void tt_put(uint32_t (&r)[16], int e, double v) {
    r[2 * e] = static_cast<uint32_t>(__double2loint(v));
    r[2 * e + 1] = static_cast<uint32_t>(__double2hiint(v));
}
// 1 / sqrt(x) and 1 / x to a few ulp: the hardware's estimates (about 2^-22) and two Newton steps.
// Both sit on the chain that every step waits for; x is a sum of squares well inside the normal range
// (a subnormal or huge x only costs accuracy on a matrix whose scale is already hopeless).
__device__ __forceinline__ double tt_rsqrt(double x) {
    double y;
    asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
    const double hx = 0.5 * x;
    double e = fma(-hx * y, y, 0.5);
    y = fma(y, e, y);
    e = fma(-hx * y, y, 0.5);
    return fma(y, e, y);
}
__device__ __forceinline__ double tt_rcp(double x) {
    double r;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(x));
    double e = fma(-x, r, 1.0);
    r = fma(r, e, r);
    e = fma(-x, r, 1.0);
    return fma(r, e, r);
}
}  // namespace eosq
