// Pair step of the placement kernel in its ranked form (see RankLayout in nbos_internal.h).
//
// A host and a request are one 64-bit value each: the four capacities of Section 3.2.1 and the
// rank in the order of Section 3.4.1, every field under a guard bit. host - request leaves all
// guards set exactly when the host fits the ask (coarsely, never rejecting a host that fits) and
// ranks before the request's current third best. So a (request, host) pair costs one 64-bit
// subtraction and one 3-input logic operation, ~(lo & hi) & guards, whose "result != 0"
// predicate is chained through the pairs of a chunk: the chain stays true only while every pair
// failed. Nothing else happens per pair; when some pair of a chunk passed, the caller re-tests
// the chunk exactly and updates the best three.
//
// Pipe balance. The 64-bit subtraction is one integer-ALU instruction, and so is the logic
// operation; the same subtraction done as two 32-bit multiply-adds with -1 (no borrow crosses
// bit 31: a host word always has its top guard set, a request word never) runs on the multiply
// pipe instead. Both pipes take a warp instruction every second cycle, so the requests of a
// chunk are split between the two forms (NBOS_RANKED_FORMS, request by request: W = one 64-bit
// subtraction, M = two multiply-adds).
//
// One asm statement covers a whole chunk (W hosts x Q requests) because a predicate cannot leave
// an asm statement. Operands: %0 flag (out), %1..%8 requests, %9..%12 hosts, %13 guard mask.
#ifndef NBOS_RANKED_CHUNK_CUH_
#define NBOS_RANKED_CHUNK_CUH_

namespace nbos {

#define NBOS_RK_W(P, r, h)                                          \
    "sub.u64 dd, %" #h ", %" #r ";\n\t"                             \
    "mov.b64 {d0, d1}, dd;\n\t"                                     \
    "lop3.and.b32 e|" #P ", d0, d1, %13, 0x2a, " #P ";\n\t"
#define NBOS_RK_M(P, r, h)                                          \
    "mov.b64 {r0, r1}, %" #r ";\n\t"                                \
    "mov.b64 {h0, h1}, %" #h ";\n\t"                                \
    "mad.lo.u32 d0, r0, 0xffffffff, h0;\n\t"                        \
    "mad.lo.u32 d1, r1, 0xffffffff, h1;\n\t"                        \
    "lop3.and.b32 e|" #P ", d0, d1, %13, 0x2a, " #P ";\n\t"

// form of request 1..8 of a row: bit q-1 of NBOS_RK_PATTERN set = request q takes the 64-bit
// subtraction (chosen by timing)
#ifndef NBOS_RK_PATTERN
#define NBOS_RK_PATTERN 0x92
#endif
#if NBOS_RK_PATTERN & 0x01
#define NBOS_RK_F1 NBOS_RK_W
#else
#define NBOS_RK_F1 NBOS_RK_M
#endif
#if NBOS_RK_PATTERN & 0x02
#define NBOS_RK_F2 NBOS_RK_W
#else
#define NBOS_RK_F2 NBOS_RK_M
#endif
#if NBOS_RK_PATTERN & 0x04
#define NBOS_RK_F3 NBOS_RK_W
#else
#define NBOS_RK_F3 NBOS_RK_M
#endif
#if NBOS_RK_PATTERN & 0x08
#define NBOS_RK_F4 NBOS_RK_W
#else
#define NBOS_RK_F4 NBOS_RK_M
#endif
#if NBOS_RK_PATTERN & 0x10
#define NBOS_RK_F5 NBOS_RK_W
#else
#define NBOS_RK_F5 NBOS_RK_M
#endif
#if NBOS_RK_PATTERN & 0x20
#define NBOS_RK_F6 NBOS_RK_W
#else
#define NBOS_RK_F6 NBOS_RK_M
#endif
#if NBOS_RK_PATTERN & 0x40
#define NBOS_RK_F7 NBOS_RK_W
#else
#define NBOS_RK_F7 NBOS_RK_M
#endif
#if NBOS_RK_PATTERN & 0x80
#define NBOS_RK_F8 NBOS_RK_W
#else
#define NBOS_RK_F8 NBOS_RK_M
#endif

// rows: one host against the first Q requests; four predicate chains take turns
#define NBOS_RK_ROW1(h) NBOS_RK_F1(p0, 1, h)
#define NBOS_RK_ROW2(h) NBOS_RK_ROW1(h) NBOS_RK_F2(p1, 2, h)
#define NBOS_RK_ROW4(h) NBOS_RK_ROW2(h) NBOS_RK_F3(p2, 3, h) NBOS_RK_F4(p3, 4, h)
#define NBOS_RK_ROW8(h) \
    NBOS_RK_ROW4(h) NBOS_RK_F5(p0, 5, h) NBOS_RK_F6(p1, 6, h) NBOS_RK_F7(p2, 7, h) NBOS_RK_F8(p3, 8, h)
#define NBOS_RK_HOSTS1(ROW) ROW(9)
#define NBOS_RK_HOSTS4(ROW) ROW(9) ROW(10) ROW(11) ROW(12)

#define NBOS_RK_CHUNK_ASM(BODY)                                                                      \
    asm volatile(                                                                                    \
        "{\n\t.reg .pred p0, p1, p2, p3;\n\t.reg .u32 d0, d1, r0, r1, h0, h1, e;\n\t.reg .b64 dd;\n\t" \
        "setp.eq.u32 p0, 0, 0;\n\tsetp.eq.u32 p1, 0, 0;\n\t"                                         \
        "setp.eq.u32 p2, 0, 0;\n\tsetp.eq.u32 p3, 0, 0;\n\t" BODY                                    \
        "and.pred p0, p0, p1;\n\tand.pred p2, p2, p3;\n\tand.pred p0, p0, p2;\n\t"                  \
        "selp.u32 %0, 0, 1, p0;\n\t}"                                                                \
        : "=r"(any_pass)                                                                             \
        : "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(a[4]), "l"(a[5]), "l"(a[6]), "l"(a[7]),    \
          "l"(x[0]), "l"(x[1]), "l"(x[2]), "l"(x[3]), "r"(guards))

// True when at least one of the W x Q (host, request) pairs of the chunk keeps all its guards.
template <int Q, int W>
__device__ __forceinline__ bool ranked_chunk_any_pass(const unsigned long long (&rq)[Q],
                                                      const unsigned long long (&h)[W], unsigned int guards)
{
    static_assert((Q == 1 || Q == 2 || Q == 4 || Q == 8) && (W == 1 || W == 4), "chunk shape");
    unsigned long long a[8], x[4];
#pragma unroll
    for (int q = 0; q < 8; ++q) a[q] = q < Q ? rq[q] : 0ull;
#pragma unroll
    for (int u = 0; u < 4; ++u) x[u] = u < W ? h[u] : 0ull;
    unsigned int any_pass;
#define NBOS_RK_CASE(QV, ROW)                                                   \
    if constexpr (Q == QV) {                                                    \
        if constexpr (W == 4) NBOS_RK_CHUNK_ASM(NBOS_RK_HOSTS4(ROW));           \
        else NBOS_RK_CHUNK_ASM(NBOS_RK_HOSTS1(ROW));                            \
    }
    NBOS_RK_CASE(1, NBOS_RK_ROW1)
    NBOS_RK_CASE(2, NBOS_RK_ROW2)
    NBOS_RK_CASE(4, NBOS_RK_ROW4)
    NBOS_RK_CASE(8, NBOS_RK_ROW8)
#undef NBOS_RK_CASE
    return any_pass != 0u;
}

// ---- first level: one 32-bit word per host and per request ---------------------------------
// e = ~(host - request) & guards is non-zero when some guard fell. The subtraction is written
// as a multiply-add with -1 (multiply pipe), the logic operation runs on the integer ALU: one
// instruction on each pipe per pair. Operands: %0 flag (out), %1..%8 requests, %9..%24 hosts,
// %25 guard mask.
#define NBOS_R1_PAIR(P, r, h)                                       \
    "mad.lo.u32 d0, %" #r ", 0xffffffff, %" #h ";\n\t"              \
    "lop3.and.b32 e|" #P ", d0, %25, 0, 0x0c, " #P ";\n\t"
// rows: one host against the first Q requests, all on the predicate chain of the host's group of
// four (P); the four chains of a 16-host chunk are independent, so their logic operations do
// not wait for one another
#define NBOS_R1_ROW1(P, h) NBOS_R1_PAIR(P, 1, h)
#define NBOS_R1_ROW2(P, h) NBOS_R1_ROW1(P, h) NBOS_R1_PAIR(P, 2, h)
#define NBOS_R1_ROW4(P, h) NBOS_R1_ROW2(P, h) NBOS_R1_PAIR(P, 3, h) NBOS_R1_PAIR(P, 4, h)
#define NBOS_R1_ROW8(P, h) \
    NBOS_R1_ROW4(P, h) NBOS_R1_PAIR(P, 5, h) NBOS_R1_PAIR(P, 6, h) NBOS_R1_PAIR(P, 7, h) NBOS_R1_PAIR(P, 8, h)
// small chunks (one group): the requests take turns on the four chains instead
#define NBOS_R1_RR1(h) NBOS_R1_PAIR(p0, 1, h)
#define NBOS_R1_RR2(h) NBOS_R1_RR1(h) NBOS_R1_PAIR(p1, 2, h)
#define NBOS_R1_RR4(h) NBOS_R1_RR2(h) NBOS_R1_PAIR(p2, 3, h) NBOS_R1_PAIR(p3, 4, h)
#define NBOS_R1_RR8(h) \
    NBOS_R1_RR4(h) NBOS_R1_PAIR(p0, 5, h) NBOS_R1_PAIR(p1, 6, h) NBOS_R1_PAIR(p2, 7, h) NBOS_R1_PAIR(p3, 8, h)
#define NBOS_R1_HOSTS1(RR) RR(9) "and.pred p0, p0, p1;\n\tand.pred p2, p2, p3;\n\tand.pred p0, p0, p2;\n\t" \
    "setp.eq.u32 p1, 0, 0;\n\tsetp.eq.u32 p2, 0, 0;\n\tsetp.eq.u32 p3, 0, 0;\n\t"
#define NBOS_R1_HOSTS4(RR) RR(9) RR(10) RR(11) RR(12) "and.pred p0, p0, p1;\n\tand.pred p2, p2, p3;\n\tand.pred p0, p0, p2;\n\t" \
    "setp.eq.u32 p1, 0, 0;\n\tsetp.eq.u32 p2, 0, 0;\n\tsetp.eq.u32 p3, 0, 0;\n\t"
// hosts interleaved over the groups, so that neighbouring instructions belong to different chains
#define NBOS_R1_HOSTS8(ROW) \
    ROW(p0, 9) ROW(p1, 13) ROW(p0, 10) ROW(p1, 14) ROW(p0, 11) ROW(p1, 15) ROW(p0, 12) ROW(p1, 16)
#define NBOS_R1_HOSTS16(ROW)                                                                     \
    ROW(p0, 9) ROW(p1, 13) ROW(p2, 17) ROW(p3, 21) ROW(p0, 10) ROW(p1, 14) ROW(p2, 18) ROW(p3, 22) \
    ROW(p0, 11) ROW(p1, 15) ROW(p2, 19) ROW(p3, 23) ROW(p0, 12) ROW(p1, 16) ROW(p2, 20) ROW(p3, 24)

// the flag has bit v set when some pair of host group v (hosts 4v .. 4v+3 of the chunk) passed
#define NBOS_R1_CHUNK_ASM(BODY)                                                                      \
    asm volatile(                                                                                    \
        "{\n\t.reg .pred p0, p1, p2, p3;\n\t.reg .u32 d0, e, f0, f1, f2, f3;\n\t"                    \
        "setp.eq.u32 p0, 0, 0;\n\tsetp.eq.u32 p1, 0, 0;\n\t"                                         \
        "setp.eq.u32 p2, 0, 0;\n\tsetp.eq.u32 p3, 0, 0;\n\t" BODY                                    \
        "selp.u32 f0, 0, 1, p0;\n\tselp.u32 f1, 0, 2, p1;\n\t"                                       \
        "selp.u32 f2, 0, 4, p2;\n\tselp.u32 f3, 0, 8, p3;\n\t"                                       \
        "or.b32 f0, f0, f1;\n\tor.b32 f2, f2, f3;\n\tor.b32 %0, f0, f2;\n\t}"                       \
        : "=r"(groups_passed)                                                                        \
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]),    \
          "r"(x[0]), "r"(x[1]), "r"(x[2]), "r"(x[3]), "r"(x[4]), "r"(x[5]), "r"(x[6]), "r"(x[7]),    \
          "r"(x[8]), "r"(x[9]), "r"(x[10]), "r"(x[11]), "r"(x[12]), "r"(x[13]), "r"(x[14]), "r"(x[15]), \
          "r"(guards))

// Bit v of the result is set when at least one pair of hosts 4v .. 4v+3 (W hosts in all) with the Q
// requests keeps all guards of its first-level word.
template <int Q, int W>
__device__ __forceinline__ unsigned int ranked_l1_chunk_groups_passed(const unsigned int (&r1)[Q], const unsigned int (&h)[W],
                                                         unsigned int guards)
{
    static_assert((Q == 1 || Q == 2 || Q == 4 || Q == 8) && (W == 1 || W == 4 || W == 8 || W == 16), "chunk shape");
    unsigned int a[8], x[16];
#pragma unroll
    for (int q = 0; q < 8; ++q) a[q] = q < Q ? r1[q] : 0u;
#pragma unroll
    for (int u = 0; u < 16; ++u) x[u] = u < W ? h[u] : 0u;
    unsigned int groups_passed;
#define NBOS_R1_CASE(QV, ROW, RR)                                               \
    if constexpr (Q == QV) {                                                    \
        if constexpr (W == 16) NBOS_R1_CHUNK_ASM(NBOS_R1_HOSTS16(ROW));         \
        else if constexpr (W == 8) NBOS_R1_CHUNK_ASM(NBOS_R1_HOSTS8(ROW));      \
        else if constexpr (W == 4) NBOS_R1_CHUNK_ASM(NBOS_R1_HOSTS4(RR));       \
        else NBOS_R1_CHUNK_ASM(NBOS_R1_HOSTS1(RR));                             \
    }
    NBOS_R1_CASE(1, NBOS_R1_ROW1, NBOS_R1_RR1)
    NBOS_R1_CASE(2, NBOS_R1_ROW2, NBOS_R1_RR2)
    NBOS_R1_CASE(4, NBOS_R1_ROW4, NBOS_R1_RR4)
    NBOS_R1_CASE(8, NBOS_R1_ROW8, NBOS_R1_RR8)
#undef NBOS_R1_CASE
    return groups_passed;
}

}  // namespace nbos

#endif  // NBOS_RANKED_CHUNK_CUH_
