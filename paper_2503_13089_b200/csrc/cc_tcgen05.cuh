// Building blocks shared by the tensor-core kernels (tcgen05 / TMEM, sm_100a): shared-memory matrix
// descriptors for the canonical no-swizzle K-major layout, bounded mbarrier waits, TMEM loads.
#pragma once

#include <stdint.h>

namespace {

constexpr long long WAIT_LIMIT = 4000000000LL;   // clock cycles (about 2 s)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Byte offset of element (row r, column k) of an R-row FP16 operand in the canonical K-major layout
// without swizzle: 8-row x 16-byte core matrices, 128 bytes apart along the rows, R*16 bytes
// apart along k.
__device__ __forceinline__ int canon_bytes(int r, int k, int R) {
    return (k >> 3) * (R * 16) + (r >> 3) * 128 + (r & 7) * 16 + (k & 7) * 2;
}

__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fff);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;   // between the two core matrices along K
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;   // between 8-row groups
    d |= (uint64_t)1 << 46;                             // descriptor version of sm_100
    return d;                                           // layout type 0: no swizzle
}

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when the CTA is aborting (this or another waiter timed out).
// Every lane of a warp waits on the same barrier word with the same parity, so the branches are
// uniform across the warp and say so (bra.uni): the compiler then needs no convergence barriers
// around the loop, which sits on the critical path of every tile.
// `ok` is left alone by a wait that succeeds and cleared by one that gives up.
__device__ __forceinline__ void mbar_wait_acc(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t& ok,
                                              long long limit = WAIT_LIMIT) {
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .u64 t0, t1;\n\t"
        ".reg .u32 n, f;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "@p bra.uni MBW_DONE;\n\t"
        "mov.u64 t0, %%clock64;\n\t"
        "mov.u32 n, 0;\n"
        "MBW_LOOP:\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "@p bra.uni MBW_DONE;\n\t"
        "add.u32 n, n, 1;\n\t"
        "and.b32 f, n, 15;\n\t"                    // a failed try has already slept in hardware: look up every 16
        "setp.ne.u32 q, f, 0;\n\t"
        "@q bra.uni MBW_LOOP;\n\t"
        "ld.volatile.shared.u32 f, [%3];\n\t"
        "setp.ne.u32 q, f, 0;\n\t"
        "@q bra.uni MBW_DONE;\n\t"                 // another waiter gave up: p is false
        "mov.u64 t1, %%clock64;\n\t"
        "sub.u64 t1, t1, t0;\n\t"
        "setp.le.u64 q, t1, %4;\n\t"
        "@q bra.uni MBW_LOOP;\n\t"
        "mov.u32 f, 1;\n\t"
        "st.volatile.shared.u32 [%3], f;\n"          // time-out: p is false
        "MBW_DONE:\n\t"
        "@!p mov.u32 %0, 0;\n\t"
        "}"
        : "+r"(ok)
        : "r"(bar), "r"(parity), "r"(smem_u32(const_cast<int*>(abort_flag))), "l"(limit)
        : "memory");
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    uint32_t ok = 1u;
    mbar_wait_acc(bar, parity, abort_flag, ok);
    return ok != 0u;
}

#define TMEM_LD32(v, taddr)                                                                                      \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                       \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                       \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                      \
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),  \
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),      \
                   "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),    \
                   "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),    \
                   "=r"(v[29]), "=r"(v[30]), "=r"(v[31])                                                         \
                 : "r"(taddr))
// The loaded registers are only valid after the wait; naming them as in/out operands keeps the
// compiler from moving their uses above it.
#define TMEM_WAIT32(v)                                                                                           \
    asm volatile("tcgen05.wait::ld.sync.aligned;"                                                                \
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),  \
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]),      \
                   "+r"(v[15]), "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]),    \
                   "+r"(v[22]), "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]),    \
                   "+r"(v[29]), "+r"(v[30]), "+r"(v[31])                                                         \
                 :: "memory")
// One wait for two loads: both register sets are named.
#define TMEM_WAIT64(v, w)                                                                                        \
    asm volatile("tcgen05.wait::ld.sync.aligned;"                                                                \
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),  \
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]),      \
                   "+r"(v[15]), "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]),    \
                   "+r"(v[22]), "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]),    \
                   "+r"(v[29]), "+r"(v[30]), "+r"(v[31]),                                                        \
                   "+r"(w[0]), "+r"(w[1]), "+r"(w[2]), "+r"(w[3]), "+r"(w[4]), "+r"(w[5]), "+r"(w[6]), "+r"(w[7]),  \
                   "+r"(w[8]), "+r"(w[9]), "+r"(w[10]), "+r"(w[11]), "+r"(w[12]), "+r"(w[13]), "+r"(w[14]),      \
                   "+r"(w[15]), "+r"(w[16]), "+r"(w[17]), "+r"(w[18]), "+r"(w[19]), "+r"(w[20]), "+r"(w[21]),    \
                   "+r"(w[22]), "+r"(w[23]), "+r"(w[24]), "+r"(w[25]), "+r"(w[26]), "+r"(w[27]), "+r"(w[28]),    \
                   "+r"(w[29]), "+r"(w[30]), "+r"(w[31])                                                         \
                 :: "memory")


}  // namespace
