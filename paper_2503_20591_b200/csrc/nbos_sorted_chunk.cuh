// Pair steps of the placement kernel for host tables stored in ascending key order.
//
// In that order a feasible host enters a request's best three exactly while the request has
// fewer than three hosts, so the only question per (request, host) pair is the capacity test of
// Section 3.2.1 (with the SR limit of Section 3.4.1 folded into the host's gmax field). The
// packed form answers it with a subtraction of the two 32-bit words and one 3-input logic
// operation whose "result != 0" predicate is chained through the pairs of a chunk: the chained
// predicate stays true only if every pair failed. No counter and no compare with the current
// third best: three instructions per pair, or two where both words go through one 64-bit
// subtraction.
//
// Pipe balance. 32-bit integer multiply-add (mad.lo with -1: a subtraction) runs on the
// multiply pipe, logic operations on the integer ALU; both pipes take a warp instruction every
// second cycle, so a kernel that loads only one of them leaves half of the integer issue rate
// unused. Five of eight requests use two multiply-pipe subtractions + one logic operation,
// three use one 64-bit subtraction (one integer-ALU instruction when measured alone) + one
// logic operation. The split was chosen by timing: all requests in the first form measured 4 %
// slower, all in the second 15 % slower, half and half 3 % slower.
//
// One asm statement covers a whole chunk (W hosts x Q requests) because a predicate cannot
// leave an asm statement. Operand layout (fixed, unused ones are passed as zero):
//   %0 flag (out)   %1..%8 request word 0   %9..%16 request word 1
//   %17,%18 host 0 (word 0, word 1)  %19,%20 host 1  %21,%22 host 2  %23,%24 host 3
//   %25 guard mask of word 0   %26 guard mask of word 1
#ifndef NBOS_SORTED_CHUNK_CUH_
#define NBOS_SORTED_CHUNK_CUH_

namespace nbos {

// one mask: e = ~(d0 & d1) & guards  (lop3 0x2a), predicate = (e != 0) & predicate
#define NBOS_SP_MM(P, a, b, x, y)                                   \
    "mad.lo.u32 d0, %" #a ", 0xffffffff, %" #x ";\n\t"              \
    "mad.lo.u32 d1, %" #b ", 0xffffffff, %" #y ";\n\t"              \
    "lop3.and.b32 e|" #P ", d0, d1, %25, 0x2a, " #P ";\n\t"
// The same with both words in one 64-bit subtraction. No borrow leaves word 0: a host word
// always has its top guard bit set, a request word never (asks are clamped below the field
// range; a retired request carries exactly the guard mask, which every host word contains).
#define NBOS_SP_64(P, a, b, x, y)                                   \
    "mov.b64 hh, {%" #x ", %" #y "};\n\t"                           \
    "mov.b64 rr, {%" #a ", %" #b "};\n\t"                           \
    "sub.u64 dd, hh, rr;\n\t"                                       \
    "mov.b64 {d0, d1}, dd;\n\t"                                     \
    "lop3.and.b32 e|" #P ", d0, d1, %25, 0x2a, " #P ";\n\t"
// two masks: e0 = ~d0 & guards0 (0x0c), e = e0 | (~d1 & guards1) (0xf2)
#define NBOS_SP2_MM(P, a, b, x, y)                                  \
    "mad.lo.u32 d0, %" #a ", 0xffffffff, %" #x ";\n\t"              \
    "mad.lo.u32 d1, %" #b ", 0xffffffff, %" #y ";\n\t"              \
    "lop3.b32 e0, d0, %25, 0, 0x0c;\n\t"                            \
    "lop3.and.b32 e|" #P ", e0, d1, %26, 0xf2, " #P ";\n\t"

// rows: one host (x, y) against the first Q requests. F32 is the form with two 32-bit
// subtractions, F64 the one used for three requests of eight. Four predicate chains (p0..p3)
// take turns, so that consecutive logic operations do not wait for one another.
#define NBOS_ROW1(F32, F64, x, y) F32(p0, 1, 9, x, y)
#define NBOS_ROW2(F32, F64, x, y) NBOS_ROW1(F32, F64, x, y) F64(p1, 2, 10, x, y)
#define NBOS_ROW4(F32, F64, x, y) NBOS_ROW2(F32, F64, x, y) F32(p2, 3, 11, x, y) F32(p3, 4, 12, x, y)
#define NBOS_ROW8(F32, F64, x, y)                                                                    \
    NBOS_ROW4(F32, F64, x, y) F64(p0, 5, 13, x, y) F32(p1, 6, 14, x, y) F32(p2, 7, 15, x, y) F64(p3, 8, 16, x, y)
#define NBOS_HOSTS1(ROW, F32, F64) ROW(F32, F64, 17, 18)
#define NBOS_HOSTS4(ROW, F32, F64) \
    ROW(F32, F64, 17, 18) ROW(F32, F64, 19, 20) ROW(F32, F64, 21, 22) ROW(F32, F64, 23, 24)

#define NBOS_CHUNK_ASM(BODY)                                                                       \
    asm volatile(                                                                                  \
        "{\n\t.reg .pred p0, p1, p2, p3;\n\t.reg .u32 d0, d1, e0, e;\n\t.reg .b64 hh, rr, dd;\n\t"  \
        "setp.eq.u32 p0, 0, 0;\n\tsetp.eq.u32 p1, 0, 0;\n\t"                                       \
        "setp.eq.u32 p2, 0, 0;\n\tsetp.eq.u32 p3, 0, 0;\n\t" BODY                                  \
        "and.pred p0, p0, p1;\n\tand.pred p2, p2, p3;\n\tand.pred p0, p0, p2;\n\t"                \
        "selp.u32 %0, 0, 1, p0;\n\t}"                                                              \
        : "=r"(any_fit)                                                                            \
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]),  \
          "r"(b[0]), "r"(b[1]), "r"(b[2]), "r"(b[3]), "r"(b[4]), "r"(b[5]), "r"(b[6]), "r"(b[7]),  \
          "r"(x[0]), "r"(y[0]), "r"(x[1]), "r"(y[1]), "r"(x[2]), "r"(y[2]), "r"(x[3]), "r"(y[3]),  \
          "r"(guards0), "r"(guards1))

// True when at least one of the W x Q (host, request) pairs of the chunk passes the capacity test.
template <int Q, int W, bool TWO_MASKS>
__device__ __forceinline__ bool sorted_chunk_any_fit(const unsigned int (&r0)[Q], const unsigned int (&r1)[Q],
                                                     const uint4 (&h)[W], unsigned int guards0,
                                                     unsigned int guards1)
{
    static_assert((Q == 1 || Q == 2 || Q == 4 || Q == 8) && (W == 1 || W == 4), "chunk shape");
    unsigned int a[8], b[8], x[4], y[4];
#pragma unroll
    for (int q = 0; q < 8; ++q) { a[q] = q < Q ? r0[q] : 0u; b[q] = q < Q ? r1[q] : 0u; }
#pragma unroll
    for (int u = 0; u < 4; ++u) { x[u] = u < W ? h[u].x : 0u; y[u] = u < W ? h[u].y : 0u; }
    unsigned int any_fit;
#define NBOS_CHUNK_CASE(QV, ROW)                                                                    \
    if constexpr (Q == QV) {                                                                        \
        if constexpr (TWO_MASKS) {                                                                  \
            if constexpr (W == 4) NBOS_CHUNK_ASM(NBOS_HOSTS4(ROW, NBOS_SP2_MM, NBOS_SP2_MM));       \
            else NBOS_CHUNK_ASM(NBOS_HOSTS1(ROW, NBOS_SP2_MM, NBOS_SP2_MM));                        \
        } else {                                                                                    \
            if constexpr (W == 4) NBOS_CHUNK_ASM(NBOS_HOSTS4(ROW, NBOS_SP_MM, NBOS_SP_64));         \
            else NBOS_CHUNK_ASM(NBOS_HOSTS1(ROW, NBOS_SP_MM, NBOS_SP_64));                          \
        }                                                                                           \
    }
    NBOS_CHUNK_CASE(1, NBOS_ROW1)
    NBOS_CHUNK_CASE(2, NBOS_ROW2)
    NBOS_CHUNK_CASE(4, NBOS_ROW4)
    NBOS_CHUNK_CASE(8, NBOS_ROW8)
#undef NBOS_CHUNK_CASE
    return any_fit != 0u;
}

}  // namespace nbos

#endif  // NBOS_SORTED_CHUNK_CUH_
