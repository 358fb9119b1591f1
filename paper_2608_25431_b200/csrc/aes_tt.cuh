// AES-128 forward cipher (FIPS-197 sec. 5.1) in table form.
//
// The state is four little-endian words, one per column (row r in byte r).
// T0[x] packs the MixColumns image of S[x] for a row-0 byte: bytes
// (2*S[x], S[x], S[x], 3*S[x]); the tables for rows 1..3 are T0 rotated left by
// 8, 16 and 24 bits.  One round of SubBytes + ShiftRows + MixColumns +
// AddRoundKey is then, per output column c,
//     T0[s_c.b0] ^ T1[s_(c+1).b1] ^ T2[s_(c+2).b2] ^ T3[s_(c+3).b3] ^ rk[c].
// The table storage is a policy (`Tab`): plain arrays on the host, a
// bank-conflict-free replicated layout in shared memory on the device.
#pragma once
#include <stdint.h>

#include "gf128.cuh"

namespace gift {

// Select four bytes out of the eight of (a, b): nibble i of sel picks result byte i,
// values 0-3 from a, 4-7 from b.
GIFT_HD uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
#if defined(__CUDA_ARCH__)
    return __byte_perm(a, b, sel);
#else
    const uint64_t both = ((uint64_t)b << 32) | a;
    uint32_t r = 0;
    for (int i = 0; i < 4; i++) {
        const uint32_t n = (sel >> (4 * i)) & 7u;
        r |= (uint32_t)((both >> (8 * n)) & 0xFFu) << (8 * i);
    }
    return r;
#endif
}

GIFT_HD uint32_t rotl32(uint32_t x, int s)
{
    return s == 0 ? x : ((x << s) | (x >> (32 - s)));
}

// ---- table construction from the definition (FIPS-197 sec. 4.2, 5.1.1) ----

GIFT_HD uint32_t gf256_xtime(uint32_t a)
{
    return ((a << 1) ^ ((a & 0x80u) ? 0x1Bu : 0u)) & 0xFFu;
}

GIFT_HD uint32_t gf256_mul(uint32_t a, uint32_t b)
{
    uint32_t p = 0;
    for (int i = 0; i < 8; i++) {
        if (b & 1u) p ^= a;
        a = gf256_xtime(a);
        b >>= 1;
    }
    return p;
}

// S-box entry: x^254 (the inverse, with 0 -> 0) followed by the affine map.
GIFT_HD uint32_t sbox_entry(uint32_t x)
{
    // x^254 = x^(2+4+8+16+32+64+128)
    uint32_t sq = gf256_mul(x, x);      // x^2
    uint32_t inv = sq;
    for (int i = 0; i < 6; i++) {
        sq = gf256_mul(sq, sq);
        inv = gf256_mul(inv, sq);
    }
    uint32_t s = inv ^ (inv << 1) ^ (inv << 2) ^ (inv << 3) ^ (inv << 4);
    s = (s ^ (s >> 8)) & 0xFFu;         // the affine map is a sum of byte rotations
    return s ^ 0x63u;
}

GIFT_HD uint32_t t0_entry(uint32_t x)
{
    const uint32_t s = sbox_entry(x);
    const uint32_t s2 = gf256_xtime(s);
    return s2 | (s << 8) | (s << 16) | ((s2 ^ s) << 24);
}

// ---- table policy for host code and for slow paths that read global memory ----
struct PlainTab {
    const uint32_t* t0;   // 256 words
    template <int T, int K>
    GIFT_HD uint32_t look(uint32_t w) const
    {
        return rotl32(t0[(w >> (8 * K)) & 0xFFu], 8 * T);
    }
    // a word with S[byte K of w] in byte 1
    template <int K>
    GIFT_HD uint32_t sub(uint32_t w) const
    {
        return t0[(w >> (8 * K)) & 0xFFu];
    }
};

// KeyExpansion (FIPS-197 sec. 5.2), Nk = 4: rk[4*r .. 4*r+3] is round key r as LE column words.
template <class Tab>
GIFT_HD void aes128_expand_key(const Tab& tb, const uint32_t key[4], uint32_t rk[44])
{
    rk[0] = key[0]; rk[1] = key[1]; rk[2] = key[2]; rk[3] = key[3];
    uint32_t rcon = 1;
    for (int i = 4; i < 44; i += 4) {
        const uint32_t t = rk[i - 1];
        // SubWord(RotWord(t)): result byte j = S[t.byte((j+1)&3)]
        const uint32_t sw = ((tb.template sub<1>(t) >> 8) & 0xFFu) |
                            (((tb.template sub<2>(t) >> 8) & 0xFFu) << 8) |
                            (((tb.template sub<3>(t) >> 8) & 0xFFu) << 16) |
                            (((tb.template sub<0>(t) >> 8) & 0xFFu) << 24);
        rk[i] = rk[i - 4] ^ sw ^ rcon;
        rk[i + 1] = rk[i - 3] ^ rk[i];
        rk[i + 2] = rk[i - 2] ^ rk[i + 1];
        rk[i + 3] = rk[i - 1] ^ rk[i + 2];
        rcon = gf256_xtime(rcon);
    }
}

// One full round on the state s with round key k[0..3].
template <class Tab>
GIFT_HD void aes_round(const Tab& tb, uint32_t s[4], const uint32_t* k)
{
    const uint32_t a = s[0], b = s[1], c = s[2], d = s[3];
    s[0] = tb.template look<0, 0>(a) ^ tb.template look<1, 1>(b) ^ tb.template look<2, 2>(c) ^
           tb.template look<3, 3>(d) ^ k[0];
    s[1] = tb.template look<0, 0>(b) ^ tb.template look<1, 1>(c) ^ tb.template look<2, 2>(d) ^
           tb.template look<3, 3>(a) ^ k[1];
    s[2] = tb.template look<0, 0>(c) ^ tb.template look<1, 1>(d) ^ tb.template look<2, 2>(a) ^
           tb.template look<3, 3>(b) ^ k[2];
    s[3] = tb.template look<0, 0>(d) ^ tb.template look<1, 1>(a) ^ tb.template look<2, 2>(b) ^
           tb.template look<3, 3>(c) ^ k[3];
}

// The last round: SubBytes + ShiftRows + AddRoundKey, no MixColumns.
template <class Tab>
GIFT_HD void aes_last_round(const Tab& tb, uint32_t s[4], const uint32_t* k)
{
    const uint32_t a = s[0], b = s[1], c = s[2], d = s[3];
    // sub<K>(w) carries S[w.byte K] in byte 1; gather the four bytes of each column
    uint32_t lo, hi;
    lo = prmt(tb.template sub<0>(a), tb.template sub<1>(b), 0x0051u);   // b0 = x.b1, b1 = y.b1
    hi = prmt(tb.template sub<2>(c), tb.template sub<3>(d), 0x0051u);
    s[0] = prmt(lo, hi, 0x5410u) ^ k[0];
    lo = prmt(tb.template sub<0>(b), tb.template sub<1>(c), 0x0051u);
    hi = prmt(tb.template sub<2>(d), tb.template sub<3>(a), 0x0051u);
    s[1] = prmt(lo, hi, 0x5410u) ^ k[1];
    lo = prmt(tb.template sub<0>(c), tb.template sub<1>(d), 0x0051u);
    hi = prmt(tb.template sub<2>(a), tb.template sub<3>(b), 0x0051u);
    s[2] = prmt(lo, hi, 0x5410u) ^ k[2];
    lo = prmt(tb.template sub<0>(d), tb.template sub<1>(a), 0x0051u);
    hi = prmt(tb.template sub<2>(b), tb.template sub<3>(c), 0x0051u);
    s[3] = prmt(lo, hi, 0x5410u) ^ k[3];
}

// Whole cipher on one block held as four LE column words.
template <class Tab>
GIFT_HD void aes128_encrypt(const Tab& tb, const uint32_t* rk, uint32_t s[4])
{
    s[0] ^= rk[0]; s[1] ^= rk[1]; s[2] ^= rk[2]; s[3] ^= rk[3];
#pragma unroll
    for (int r = 1; r < 10; r++) aes_round(tb, s, rk + 4 * r);
    aes_last_round(tb, s, rk + 40);
}

// ---- inverse cipher (FIPS-197 sec. 5.3), used only by the token mode ----
//
// Written out plainly: InvShiftRows + InvSubBytes through a 256-byte inverse S-box,
// AddRoundKey, and InvMixColumns computed on four packed bytes at a time.  Token batches
// are small (the kernel is bound by launch latency), so no tables are built for it.

// multiply each of the four packed bytes by x in GF(2^8)
GIFT_HD uint32_t xtime4(uint32_t w)
{
    return ((w & 0x7F7F7F7Fu) << 1) ^ (((w >> 7) & 0x01010101u) * 0x1Bu);
}

GIFT_HD uint32_t rotr32(uint32_t x, int s)
{
    return (x >> s) | (x << (32 - s));
}

// One column: out row r = 0e*a_r ^ 0b*a_(r+1) ^ 0d*a_(r+2) ^ 09*a_(r+3)
GIFT_HD uint32_t inv_mix_column(uint32_t w)
{
    const uint32_t w2 = xtime4(w), w4 = xtime4(w2), w8 = xtime4(w4);
    const uint32_t w9 = w8 ^ w, wb = w9 ^ w2, wd = w9 ^ w4, we = w8 ^ w4 ^ w2;
    return we ^ rotr32(wb, 8) ^ rotr32(wd, 16) ^ rotr32(w9, 24);
}

GIFT_HD void aes128_decrypt(const uint8_t* isbox, const uint32_t* rk, uint32_t s[4])
{
    s[0] ^= rk[40]; s[1] ^= rk[41]; s[2] ^= rk[42]; s[3] ^= rk[43];
    for (int round = 9; round >= 0; round--) {
        uint32_t t[4];
        // InvShiftRows then InvSubBytes: output column c, row r comes from column (c - r) mod 4
        for (int c = 0; c < 4; c++) {
            t[c] = (uint32_t)isbox[s[c] & 0xFFu] |
                   ((uint32_t)isbox[(s[(c + 3) & 3] >> 8) & 0xFFu] << 8) |
                   ((uint32_t)isbox[(s[(c + 2) & 3] >> 16) & 0xFFu] << 16) |
                   ((uint32_t)isbox[(s[(c + 1) & 3] >> 24) & 0xFFu] << 24);
        }
        for (int c = 0; c < 4; c++) {
            const uint32_t v = t[c] ^ rk[4 * round + c];
            s[c] = round != 0 ? inv_mix_column(v) : v;
        }
    }
}

// ---- CTR with GCM's counter layout (SP 800-38D sec. 7.1) ----
//
// Counter block = nonce (12 bytes) || BE32(ctr).  Only the last column varies
// between the blocks of a segment, so the first AddRoundKey of columns 0..2 and
// three of the four lookups of every round-1 output column are the same for all
// of them.  `CtrPrefix` holds what is constant: s3 base and the round-1 column
// constants.  Round-1 output column c takes byte (3-c) of the varying word.
struct CtrPrefix {
    uint32_t k03;     // rk[3]: XORed with the byte-swapped counter to give the varying word
    uint32_t c1[4];   // rk[4+c] ^ the three constant lookups of round-1 column c
};

template <class Tab>
GIFT_HD CtrPrefix ctr_prefix(const Tab& tb, const uint32_t* rk, const uint32_t nonce[3])
{
    const uint32_t a = nonce[0] ^ rk[0], b = nonce[1] ^ rk[1], c = nonce[2] ^ rk[2];
    CtrPrefix p;
    p.k03 = rk[3];
    p.c1[0] = tb.template look<0, 0>(a) ^ tb.template look<1, 1>(b) ^ tb.template look<2, 2>(c) ^ rk[4];
    p.c1[1] = tb.template look<0, 0>(b) ^ tb.template look<1, 1>(c) ^ tb.template look<3, 3>(a) ^ rk[5];
    p.c1[2] = tb.template look<0, 0>(c) ^ tb.template look<2, 2>(a) ^ tb.template look<3, 3>(b) ^ rk[6];
    p.c1[3] = tb.template look<1, 1>(a) ^ tb.template look<2, 2>(b) ^ tb.template look<3, 3>(c) ^ rk[7];
    return p;
}

// Keystream block for counter value ctr (the GCM data blocks use ctr = 2, 3, ...).
template <class Tab>
GIFT_HD void ctr_keystream(const Tab& tb, const uint32_t* rk, const CtrPrefix& p, uint32_t ctr,
                           uint32_t ks[4])
{
    const uint32_t d = bswap32(ctr) ^ p.k03;
    ks[0] = p.c1[0] ^ tb.template look<3, 3>(d);
    ks[1] = p.c1[1] ^ tb.template look<2, 2>(d);
    ks[2] = p.c1[2] ^ tb.template look<1, 1>(d);
    ks[3] = p.c1[3] ^ tb.template look<0, 0>(d);
#pragma unroll
    for (int r = 2; r < 10; r++) aes_round(tb, ks, rk + 4 * r);
    aes_last_round(tb, ks, rk + 40);
}

// ---- CTR across 256 consecutive counters ----
//
// Inside a group of 256 consecutive counter values only the counter's lowest byte changes,
// which is byte 3 of the varying state word.  After round 1 only column 0 depends on it;
// in round 2 every output column takes exactly one byte of column 0, so three of its four
// lookups are the same for the whole group.  `CtrGroup` caches what is constant per group:
// the round-2 constants.  Per block that leaves 1 lookup in round 1 and 4 in round 2.
struct CtrGroup {
    uint32_t grp;      // ctr >> 8 the cache belongs to
    uint32_t c2[4];    // round-2 output column c without the lookup that depends on column 0
};

template <class Tab>
GIFT_HD void ctr_group_setup(const Tab& tb, const uint32_t* rk, const CtrPrefix& p, uint32_t ctr, CtrGroup& g)
{
    const uint32_t d = bswap32(ctr) ^ p.k03;                 // bytes 0..2 are what the group shares
    const uint32_t k1 = p.c1[1] ^ tb.template look<2, 2>(d);  // round-1 columns 1..3
    const uint32_t k2 = p.c1[2] ^ tb.template look<1, 1>(d);
    const uint32_t k3 = p.c1[3] ^ tb.template look<0, 0>(d);
    g.grp = ctr >> 8;
    g.c2[0] = tb.template look<1, 1>(k1) ^ tb.template look<2, 2>(k2) ^ tb.template look<3, 3>(k3) ^ rk[8];
    g.c2[1] = tb.template look<0, 0>(k1) ^ tb.template look<1, 1>(k2) ^ tb.template look<2, 2>(k3) ^ rk[9];
    g.c2[2] = tb.template look<0, 0>(k2) ^ tb.template look<1, 1>(k3) ^ tb.template look<3, 3>(k1) ^ rk[10];
    g.c2[3] = tb.template look<0, 0>(k3) ^ tb.template look<2, 2>(k1) ^ tb.template look<3, 3>(k2) ^ rk[11];
}

// Keystream block for counter value ctr, which must lie in the group g was set up for.
template <class Tab>
GIFT_HD void ctr_keystream_grouped(const Tab& tb, const uint32_t* rk, const CtrPrefix& p, const CtrGroup& g,
                                   uint32_t ctr, uint32_t ks[4])
{
    const uint32_t d = bswap32(ctr) ^ p.k03;
    const uint32_t x0 = p.c1[0] ^ tb.template look<3, 3>(d);          // round 1, column 0
    ks[0] = g.c2[0] ^ tb.template look<0, 0>(x0);                      // round 2
    ks[1] = g.c2[1] ^ tb.template look<3, 3>(x0);
    ks[2] = g.c2[2] ^ tb.template look<2, 2>(x0);
    ks[3] = g.c2[3] ^ tb.template look<1, 1>(x0);
#pragma unroll
    for (int r = 3; r < 10; r++) aes_round(tb, ks, rk + 4 * r);
    aes_last_round(tb, ks, rk + 40);
}

}  // namespace gift
