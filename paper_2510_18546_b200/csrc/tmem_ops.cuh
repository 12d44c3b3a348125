// tcgen05.ld / tcgen05.st wrappers with explicit register lists (32x32b shape: thread t of the
// warp reads/writes TMEM lane (32 * (warp % 4) + t), one 32-bit column per register).
// A load wrapper either ends with tcgen05.wait::ld inside the same asm statement, or is split into
// an "issue" and an "arrived" part; the values may be used only after the wait, and the "arrived"
// part ties them to the wait so that the compiler cannot schedule a consumer before it.
#pragma once
#include <stdint.h>

namespace enl {

#define ENL_R32_OUT(v) \
    "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), \
    "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), \
    "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), \
    "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
#define ENL_R32_INOUT(v) \
    "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), \
    "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]), "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), \
    "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), \
    "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
#define ENL_R32_IN(v) \
    "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), \
    "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), \
    "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), \
    "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
#define ENL_X32_LIST \
    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, " \
    "%25, %26, %27, %28, %29, %30, %31}"

// loads columns [taddr, taddr + 32) of the calling thread's lane and waits for them
__device__ __forceinline__ void tmem_ld32_wait(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 " ENL_X32_LIST ", [%32];\n\t"
                 "tcgen05.wait::ld.sync.aligned;\n\t"
                 : ENL_R32_OUT(v) : "r"(taddr) : "memory");
}

// The same load without the wait.  tmem_ld_wait() waits for every load the thread has issued;
// tmem_ld32_arrived(v) must follow it for each register block before the block is read.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 " ENL_X32_LIST ", [%32];\n\t"
                 : ENL_R32_OUT(v) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;\n\t" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32_arrived(uint32_t (&v)[32])
{
    asm volatile("" : ENL_R32_INOUT(v) : : "memory");
}

// stores 32 columns starting at taddr (no wait; call tmem_st_wait before signalling)
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], " ENL_X32_LIST ";\n\t"
                 : : ENL_R32_IN(v), "r"(taddr) : "memory");
}

// stores 16 columns starting at taddr (no wait; call tmem_st_wait before signalling)
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};\n\t"
        :
        : "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_st_wait()
{
    asm volatile("tcgen05.wait::st.sync.aligned;\n\t" ::: "memory");
}

#undef ENL_R32_OUT
#undef ENL_R32_INOUT
#undef ENL_R32_IN
#undef ENL_X32_LIST

}  // namespace enl
