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
// A 32x32 -> 64 carry-less product is built from ordinary integer multiplies of
// operands masked to every fourth bit: with at most 8 ones per operand no 4-bit
// slot can overflow, so the low bit of every slot is the XOR the carry-less
// product wants.  The low word of the product takes 16 such 32-bit multiplies;
// the high word is obtained as the low word of the product of the bit-reversed
// operands (16 more), never from the high word of a wide multiply (see
// clmul32_low).  128x128 uses two Karatsuba levels (9 such leaves).
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
// has room.  An add written as a*1 + b stays a multiply-add instruction only if the factor
// is not a compile-time constant; constant memory that the host could rewrite is opaque
// enough.  The value never changes.
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

// One 32-bit leaf of a fixed multiplier, split for the masked-integer product in both bit
// orders: f[j] = b & M_j and r[j] = (rev32(b) << 1) & M_j.
struct alignas(16) leaf_op {
    uint32_t f[4];
    uint32_t r[4];
};

GIFT_HD leaf_op split_leaf(uint32_t b)
{
    const uint32_t rb = brev32(b) << 1;      // the shift of hi_from_rev, taken here once per key
    leaf_op s;
    s.f[0] = b & GIFT_M0; s.f[1] = b & GIFT_M1; s.f[2] = b & GIFT_M2; s.f[3] = b & GIFT_M3;
    s.r[0] = rb & GIFT_M0; s.r[1] = rb & GIFT_M1; s.r[2] = rb & GIFT_M2; s.r[3] = rb & GIFT_M3;
    return s;
}

// Low 32 bits of the carry-less product of a with a pre-split b (bm[j] = b & M_j).
//
// Class r collects the products a_i * b_j with i + j == r (mod 4); bit 4k + r of their XOR
// is the wanted coefficient.  Only the LOW word of every integer product is used (a plain
// 32-bit multiply): reading the high word of a 32x32 -> 64 product costs this GPU two extra
// issue slots per read, which the wide form paid 72 times per block.  In the low word a slot
// k holds at most k + 1 <= 8 ones per product, so two products can be ADDED by the
// multiplier itself without a slot running over (14 at most below the top slot, and what
// the top slot carries out falls off bit 31); the two sums are then XORed and masked by one
// logic instruction.  The four masked classes occupy disjoint bits and are merged by adds,
// issued as multiply-adds to keep them off the logic pipe.
GIFT_HD uint32_t clmul32_low(uint32_t a, const uint32_t bm[4])
{
    const uint32_t a0 = a & GIFT_M0, a1 = a & GIFT_M1, a2 = a & GIFT_M2, a3 = a & GIFT_M3;
    const uint32_t c0 = ((a0 * bm[0] + a1 * bm[3]) ^ (a2 * bm[2] + a3 * bm[1])) & GIFT_M0;
    const uint32_t c1 = ((a0 * bm[1] + a1 * bm[0]) ^ (a2 * bm[3] + a3 * bm[2])) & GIFT_M1;
    const uint32_t c2 = ((a0 * bm[2] + a1 * bm[1]) ^ (a2 * bm[0] + a3 * bm[3])) & GIFT_M2;
    const uint32_t c3 = ((a0 * bm[3] + a1 * bm[2]) ^ (a2 * bm[1] + a3 * bm[0])) & GIFT_M3;
    return add_mul(c3, add_mul(c2, add_mul(c1, c0)));
}

// A 64-bit carry-less product P = a (x) b is kept as two words: lo = P mod x^32 and hr, the
// low word of rev32(a) (x) (rev32(b) << 1).  Reversing all 63 bits of P gives
// rev32(a) (x) rev32(b), whose low word shifted up by one is the high word of P read
// backwards: hi = rev32(hr)  (see hi_from_rev).  The high half thus comes from a second
// low-word product instead of from the high word of a wide multiply.  XOR is linear in both
// forms, so sums of products stay in this split form until the very end.
GIFT_HD uint32_t hi_from_rev(uint32_t hr)
{
    return brev32(hr);
}

// A fixed multiplier prepared for repeated use: the nine Karatsuba leaf operands of b.
//   leaves: b0, b1, b0^b1 | b2, b3, b2^b3 | b0^b2, b1^b3, b0^b1^b2^b3
struct mulop {
    leaf_op leaf[9];
};

GIFT_HD mulop prepare_mulop(const u128& b)
{
    mulop p;
    const uint32_t b0 = b.w[0], b1 = b.w[1], b2 = b.w[2], b3 = b.w[3];
    p.leaf[0] = split_leaf(b0);
    p.leaf[1] = split_leaf(b1);
    p.leaf[2] = split_leaf(b0 ^ b1);
    p.leaf[3] = split_leaf(b2);
    p.leaf[4] = split_leaf(b3);
    p.leaf[5] = split_leaf(b2 ^ b3);
    p.leaf[6] = split_leaf(b0 ^ b2);
    p.leaf[7] = split_leaf(b1 ^ b3);
    p.leaf[8] = split_leaf(b0 ^ b1 ^ b2 ^ b3);
    return p;
}

// 64x64 -> 128 carry-less product (one Karatsuba level) of (x0,x1), given with its word-wise
// bit reversals (rx0,rx1), with leaves l[0..2].  The result has words 0..3; n[k] is the part
// of word k in natural bit order (k = 0..2) and r[k] the part still in reversed form
// (k = 1..3): word k = n[k] ^ hi_from_rev(r[k]).
GIFT_HD void clmul64(uint32_t x0, uint32_t x1, uint32_t rx0, uint32_t rx1, const leaf_op* l, uint32_t n[3], uint32_t r[4])
{
    const uint32_t p0l = clmul32_low(x0, l[0].f), p0r = clmul32_low(rx0, l[0].r);
    const uint32_t p2l = clmul32_low(x1, l[1].f), p2r = clmul32_low(rx1, l[1].r);
    const uint32_t pml = clmul32_low(x0 ^ x1, l[2].f), pmr = clmul32_low(rx0 ^ rx1, l[2].r);
    n[0] = p0l;
    n[1] = pml ^ p0l ^ p2l;       // low word of the middle term
    n[2] = p2l;
    r[0] = 0u;
    r[1] = p0r;
    r[2] = pmr ^ p0r ^ p2r;       // high word of the middle term
    r[3] = p2r;
}

// 128x128 -> 256 carry-less product, unreduced.
GIFT_HD void clmul128(const u128& a, const mulop& b, uint32_t out[8])
{
    const uint32_t ra0 = brev32(a.w[0]), ra1 = brev32(a.w[1]), ra2 = brev32(a.w[2]), ra3 = brev32(a.w[3]);
    uint32_t z0n[3], z0r[4], z2n[3], z2r[4], zmn[3], zmr[4];
    clmul64(a.w[0], a.w[1], ra0, ra1, &b.leaf[0], z0n, z0r);
    clmul64(a.w[2], a.w[3], ra2, ra3, &b.leaf[3], z2n, z2r);
    clmul64(a.w[0] ^ a.w[2], a.w[1] ^ a.w[3], ra0 ^ ra2, ra1 ^ ra3, &b.leaf[6], zmn, zmr);
    // middle term m = zm ^ z0 ^ z2, word k of it lands in word k + 2 of the result
    const uint32_t mn0 = zmn[0] ^ z0n[0] ^ z2n[0], mn1 = zmn[1] ^ z0n[1] ^ z2n[1], mn2 = zmn[2] ^ z0n[2] ^ z2n[2];
    const uint32_t mr1 = zmr[1] ^ z0r[1] ^ z2r[1], mr2 = zmr[2] ^ z0r[2] ^ z2r[2], mr3 = zmr[3] ^ z0r[3] ^ z2r[3];
    out[0] = z0n[0];
    out[1] = z0n[1] ^ hi_from_rev(z0r[1]);
    out[2] = z0n[2] ^ mn0 ^ hi_from_rev(z0r[2]);
    out[3] = mn1 ^ hi_from_rev(z0r[3] ^ mr1);
    out[4] = z2n[0] ^ mn2 ^ hi_from_rev(mr2);
    out[5] = z2n[1] ^ hi_from_rev(z2r[1] ^ mr3);
    out[6] = z2n[2] ^ hi_from_rev(z2r[2]);
    out[7] = hi_from_rev(z2r[3]);
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
