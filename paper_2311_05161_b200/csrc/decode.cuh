// dINT4 code expansion shared by the linear kernels: sixteen-entry byte tables in four
// registers, looked up with the byte-permute instruction (Eq. 6 folded into an integer table).
#pragma once

#include "common.cuh"

namespace w4a8 {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// 16-byte global load that does not allocate in L1 (each code byte is used once per CTA).
__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Eight codes (nibble i = code of k0 + i) -> eight INT8 levels, bytes in k order.  Tables from
// build_level_tables: eleven logic instructions.
__device__ __forceinline__ void decode8(uint32_t w, const uint32_t (&t)[4], uint32_t &o0,
                                        uint32_t &o1)
{
    const uint32_t idx = w & 0x77777777u;
    const uint32_t e = w << 4;
    const uint32_t idx_hi = idx >> 16;
    const uint32_t a0 = prmt(t[0], t[1], idx), b0 = prmt(t[2], t[3], idx);
    const uint32_t a1 = prmt(t[0], t[1], idx_hi), b1 = prmt(t[2], t[3], idx_hi);
    const uint32_t m0 = prmt(e, w, 0xD9C8u), m1 = prmt(e, w, 0xFBEAu);   // bit 3 -> byte mask
    o0 = (a0 & ~m0) | (b0 & m0);
    o1 = (a1 & ~m1) | (b1 & m1);
}

// Cheaper expansion for special values step/2 and step/4.  The levels are stored with an offset
// `off` = 13 * 2^shift, so every table byte lies in [0, 2 off] <= 104 and has its top bit clear.
// A permute whose selector nibble has bit 3 set returns the selected byte's sign spread over the
// byte, which is zero for such a table.  So the raw code nibbles pick from the table of codes
// 0..7 and give 0 for codes 8..15, and the nibbles with bit 3 flipped do the opposite on the
// table of codes 8..15: no mask, no select.  Every sum of products then carries
// off * (sum of the token's INT8 values), which the caller takes out again.  Integer arithmetic
// modulo 2^32 throughout, so the result is exact whenever the true sum fits.
__device__ __forceinline__ void build_offset_tables(int z, const LevelTables &lt, int shift,
                                                    uint32_t (&t)[4])
{
    const uint32_t off = 13u << shift;
    const uint32_t kc = (128u - off) * 0x01010101u;      // the tables' 0x80 bias minus the offset
    const uint32_t zz = (uint32_t)z * lt.zmul;
    t[0] = lt.base[0] - zz - kc;
    t[1] = lt.base[1] - zz - kc;
    t[2] = lt.base[2] - zz - kc;
    // codes 12 and 13, then the two special values +1 and -1
    t[3] = ((lt.base[3] - (zz & 0xFFFFu) - (kc & 0xFFFFu)) & 0xFFFFu) | ((off + 1u) << 16) |
           ((off - 1u) << 24);
}

// The offset form of decode8 with both halves merged (one of the two permute results is zero in
// every byte).  The merge is written as a multiply-add by `one`, a register that holds 1 and that
// the compiler cannot see through, so it runs on the FMA pipe: seven instructions on the logic
// pipe, which is what bounds the expansion.
__device__ __forceinline__ void decode8_offset(uint32_t w, const uint32_t (&t)[4], uint32_t one,
                                               uint32_t &o0, uint32_t &o1)
{
    const uint32_t wx = w ^ 0x88888888u;
    const uint32_t a0 = prmt(t[0], t[1], w), b0 = prmt(t[2], t[3], wx);
    const uint32_t a1 = prmt(t[0], t[1], w >> 16), b1 = prmt(t[2], t[3], wx >> 16);
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(o0) : "r"(a0), "r"(one), "r"(b0));
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(o1) : "r"(a1), "r"(one), "r"(b1));
}

}  // namespace w4a8
