// GF(2^128) arithmetic for GHASH (SP 800-38D sec. 6.3-6.4) on a GPU without a
// carry-less multiply instruction.
//
// Representation ("natural domain"): a field element is four 32-bit words,
// bit j of word k being the coefficient of x^(32k+j).  A 16-byte block read as
// four little-endian words reaches this form by reversing the bits inside every
// byte (GHASH numbers the bits of a block left to right).  In this domain the
// field product is the ordinary polynomial product reduced modulo
// x^128 + x^7 + x^2 + x + 1.
//
// A 32x32 -> 64 carry-less product is built from 16 ordinary integer multiplies
// of operands masked to every fourth bit: with at most 8 ones per operand no
// 4-bit slot can overflow, so the low bit of every slot is the XOR the
// carry-less product wants.  The four products of one residue class are
// combined with XOR (adding them could overflow a slot), then masked.
// 128x128 uses two Karatsuba levels (9 such products).
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define GIFT_HD __host__ __device__ __forceinline__
#else
#define GIFT_HD inline
#endif

namespace gift {

struct u128 {
    uint32_t w[4];
};

GIFT_HD uint32_t brev32(uint32_t x)
{
#if defined(__CUDA_ARCH__)
    return __brev(x);
#else
    x = ((x >> 1) & 0x55555555u) | ((x & 0x55555555u) << 1);
    x = ((x >> 2) & 0x33333333u) | ((x & 0x33333333u) << 2);
    x = ((x >> 4) & 0x0F0F0F0Fu) | ((x & 0x0F0F0F0Fu) << 4);
    x = ((x >> 8) & 0x00FF00FFu) | ((x & 0x00FF00FFu) << 8);
    return (x >> 16) | (x << 16);
#endif
}

GIFT_HD uint32_t bswap32(uint32_t x)
{
#if defined(__CUDA_ARCH__)
    return __byte_perm(x, 0, 0x0123);
#else
    return (x >> 24) | ((x >> 8) & 0xFF00u) | ((x << 8) & 0xFF0000u) | (x << 24);
#endif
}

// funnel shift left: high word of ((hi:lo) << s), 0 < s < 32
GIFT_HD uint32_t fshl(uint32_t lo, uint32_t hi, uint32_t s)
{
#if defined(__CUDA_ARCH__)
    return __funnelshift_l(lo, hi, s);
#else
    return (hi << s) | (lo >> (32 - s));
#endif
}

GIFT_HD uint64_t mulwide(uint32_t a, uint32_t b)
{
    return (uint64_t)a * (uint64_t)b;
}

// A multiplier of 1 that the compiler cannot see through.  On this GPU logic, permute and
// shift instructions share one pipe, which binds the cipher kernel, while the multiply pipe
// is mostly idle.  An add written as a*1 + b stays a multiply-add instruction only if the
// factor is not a compile-time constant; constant memory that the host could rewrite is
// opaque enough.  The value never changes.
#if defined(__CUDACC__)
static __constant__ uint32_t gift_kmul[1] = {1u};
#endif
static const uint32_t gift_kmul_host[1] = {1u};
#if defined(__CUDA_ARCH__)
#define GIFT_KMUL(i) gift_kmul[i]
#else
#define GIFT_KMUL(i) gift_kmul_host[i]
#endif

// a + b on the multiply pipe
GIFT_HD uint32_t add_mul(uint32_t a, uint32_t b)
{
    return a * GIFT_KMUL(0) + b;
}

// Reverse the bits inside each byte of a little-endian word: block bytes <-> natural domain.
GIFT_HD uint32_t reflect_bytes(uint32_t x)
{
    return bswap32(brev32(x));
}

GIFT_HD u128 block_to_field(uint32_t d0, uint32_t d1, uint32_t d2, uint32_t d3)
{
    u128 r;
    r.w[0] = reflect_bytes(d0);
    r.w[1] = reflect_bytes(d1);
    r.w[2] = reflect_bytes(d2);
    r.w[3] = reflect_bytes(d3);
    return r;
}

GIFT_HD u128 xor128(const u128& a, const u128& b)
{
    u128 r;
    r.w[0] = a.w[0] ^ b.w[0];
    r.w[1] = a.w[1] ^ b.w[1];
    r.w[2] = a.w[2] ^ b.w[2];
    r.w[3] = a.w[3] ^ b.w[3];
    return r;
}

#define GIFT_M0 0x11111111u
#define GIFT_M1 0x22222222u
#define GIFT_M2 0x44444444u
#define GIFT_M3 0x88888888u

// One multiplier operand split for the masked-integer product: bm[j] = b & M_j.
struct split32 {
    uint32_t m[4];
};

GIFT_HD split32 split_word(uint32_t b)
{
    split32 s;
    s.m[0] = b & GIFT_M0;
    s.m[1] = b & GIFT_M1;
    s.m[2] = b & GIFT_M2;
    s.m[3] = b & GIFT_M3;
    return s;
}

// 32x32 -> 64 carry-less product of a with a pre-split b.
GIFT_HD uint64_t clmul32(uint32_t a, const split32& b)
{
    const uint32_t a0 = a & GIFT_M0, a1 = a & GIFT_M1, a2 = a & GIFT_M2, a3 = a & GIFT_M3;
    // class r collects the products a_i * b_j with i + j == r (mod 4).  The four masked
    // classes occupy disjoint bits, so they are merged with integer adds, issued as
    // multiply-adds to keep them off the logic pipe.  Each 32-bit half is merged on its
    // own: no carry can cross.
    uint64_t c = mulwide(a0, b.m[0]) ^ mulwide(a1, b.m[3]) ^ mulwide(a2, b.m[2]) ^ mulwide(a3, b.m[1]);
    uint32_t lo = (uint32_t)c & GIFT_M0, hi = (uint32_t)(c >> 32) & GIFT_M0;
    c = mulwide(a0, b.m[1]) ^ mulwide(a1, b.m[0]) ^ mulwide(a2, b.m[3]) ^ mulwide(a3, b.m[2]);
    lo = add_mul((uint32_t)c & GIFT_M1, lo);
    hi = add_mul((uint32_t)(c >> 32) & GIFT_M1, hi);
    c = mulwide(a0, b.m[2]) ^ mulwide(a1, b.m[1]) ^ mulwide(a2, b.m[0]) ^ mulwide(a3, b.m[3]);
    lo = add_mul((uint32_t)c & GIFT_M2, lo);
    hi = add_mul((uint32_t)(c >> 32) & GIFT_M2, hi);
    c = mulwide(a0, b.m[3]) ^ mulwide(a1, b.m[2]) ^ mulwide(a2, b.m[1]) ^ mulwide(a3, b.m[0]);
    lo = add_mul((uint32_t)c & GIFT_M3, lo);
    hi = add_mul((uint32_t)(c >> 32) & GIFT_M3, hi);
    return ((uint64_t)hi << 32) | lo;
}

// A fixed multiplier prepared for repeated use: the nine Karatsuba leaf
// operands of b, each split into its four masked classes (36 words).
//   leaves: b0, b1, b0^b1 | b2, b3, b2^b3 | b0^b2, b1^b3, b0^b1^b2^b3
struct mulop {
    split32 leaf[9];
};

GIFT_HD mulop prepare_mulop(const u128& b)
{
    mulop p;
    const uint32_t b0 = b.w[0], b1 = b.w[1], b2 = b.w[2], b3 = b.w[3];
    p.leaf[0] = split_word(b0);
    p.leaf[1] = split_word(b1);
    p.leaf[2] = split_word(b0 ^ b1);
    p.leaf[3] = split_word(b2);
    p.leaf[4] = split_word(b3);
    p.leaf[5] = split_word(b2 ^ b3);
    p.leaf[6] = split_word(b0 ^ b2);
    p.leaf[7] = split_word(b1 ^ b3);
    p.leaf[8] = split_word(b0 ^ b1 ^ b2 ^ b3);
    return p;
}

// 64x64 -> 128 carry-less product (one Karatsuba level) of (x0,x1) with leaves l[0..2].
GIFT_HD void clmul64(uint32_t x0, uint32_t x1, const split32* l, uint32_t r[4])
{
    const uint64_t p0 = clmul32(x0, l[0]);
    const uint64_t p2 = clmul32(x1, l[1]);
    const uint64_t pm = clmul32(x0 ^ x1, l[2]);
    const uint64_t mid = pm ^ p0 ^ p2;
    r[0] = (uint32_t)p0;
    r[1] = (uint32_t)(p0 >> 32) ^ (uint32_t)mid;
    r[2] = (uint32_t)p2 ^ (uint32_t)(mid >> 32);
    r[3] = (uint32_t)(p2 >> 32);
}

// 128x128 -> 256 carry-less product, unreduced.
GIFT_HD void clmul128(const u128& a, const mulop& b, uint32_t r[8])
{
    uint32_t z0[4], z2[4], zm[4];
    clmul64(a.w[0], a.w[1], &b.leaf[0], z0);
    clmul64(a.w[2], a.w[3], &b.leaf[3], z2);
    clmul64(a.w[0] ^ a.w[2], a.w[1] ^ a.w[3], &b.leaf[6], zm);
    const uint32_t m0 = zm[0] ^ z0[0] ^ z2[0], m1 = zm[1] ^ z0[1] ^ z2[1];
    const uint32_t m2 = zm[2] ^ z0[2] ^ z2[2], m3 = zm[3] ^ z0[3] ^ z2[3];
    r[0] = z0[0];
    r[1] = z0[1];
    r[2] = z0[2] ^ m0;
    r[3] = z0[3] ^ m1;
    r[4] = z2[0] ^ m2;
    r[5] = z2[1] ^ m3;
    r[6] = z2[2];
    r[7] = z2[3];
}

// Reduce a 256-bit polynomial modulo x^128 + x^7 + x^2 + x + 1: the high half h folds
// down as h * (1 + x + x^2 + x^7), every shifted copy built with funnel shifts across the
// words; the few bits pushed past x^127 wrap around once more.  (Written with wide
// multiplies by 2^s instead, the reduction spilled registers and was slower.)
GIFT_HD u128 reduce256(const uint32_t r[8])
{
    const uint32_t h0 = r[4], h1 = r[5], h2 = r[6], h3 = r[7];
    uint32_t t0 = h0 ^ (h0 << 1) ^ (h0 << 2) ^ (h0 << 7);
    uint32_t t1 = h1 ^ fshl(h0, h1, 1) ^ fshl(h0, h1, 2) ^ fshl(h0, h1, 7);
    uint32_t t2 = h2 ^ fshl(h1, h2, 1) ^ fshl(h1, h2, 2) ^ fshl(h1, h2, 7);
    uint32_t t3 = h3 ^ fshl(h2, h3, 1) ^ fshl(h2, h3, 2) ^ fshl(h2, h3, 7);
    const uint32_t ov = (h3 >> 31) ^ (h3 >> 30) ^ (h3 >> 25);
    t0 ^= ov ^ (ov << 1) ^ (ov << 2) ^ (ov << 7);
    u128 zz;
    zz.w[0] = r[0] ^ t0; zz.w[1] = r[1] ^ t1; zz.w[2] = r[2] ^ t2; zz.w[3] = r[3] ^ t3;
    return zz;
}

GIFT_HD u128 gfmul(const u128& a, const mulop& b)
{
    uint32_t r[8];
    clmul128(a, b, r);
    return reduce256(r);
}

GIFT_HD u128 gfmul(const u128& a, const u128& b)
{
    return gfmul(a, prepare_mulop(b));
}

GIFT_HD u128 gf_one()
{
    u128 r;
    r.w[0] = 1u; r.w[1] = 0u; r.w[2] = 0u; r.w[3] = 0u;
    return r;
}

GIFT_HD u128 gf_zero()
{
    u128 r;
    r.w[0] = 0u; r.w[1] = 0u; r.w[2] = 0u; r.w[3] = 0u;
    return r;
}

}  // namespace gift
