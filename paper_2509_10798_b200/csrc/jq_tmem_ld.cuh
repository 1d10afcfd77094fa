// tcgen05.ld wrappers: shape 32x32b, every thread of a warp reads 16 consecutive 32-bit columns of its
// own tensor-memory lane (lane = 32 * (warp % 4) + lane id).
// The load is asynchronous.  It is issued by JQ_TMEM_LD16 and completed by JQ_TMEM_WAIT16, which names
// the destination registers as read-write operands: the compiler then cannot move a use of them in
// front of the wait, while everything that does not touch them may be scheduled between the two.
#pragma once

#define JQ_TMEM_LD16(taddr, v) \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];" \
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]) \
                 : "r"(taddr) : "memory")

#define JQ_TMEM_WAIT16(v) \
    asm volatile("tcgen05.wait::ld.sync.aligned;" \
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]) \
                 : : "memory")
