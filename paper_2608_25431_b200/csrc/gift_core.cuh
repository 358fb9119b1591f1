// Per-lane work of the segment cipher: CTR keystream, XOR, GHASH accumulation
// over a contiguous run of 16-byte blocks of one segment, and the power-of-H
// fix-up that makes run results order-free.
//
// GHASH of a segment with n ciphertext blocks C_1..C_n and empty AAD is
//     S = sum_i C_i * H^(n-i+2)  +  LEN * H          (SP 800-38D sec. 6.4, 7.1)
// so any subset of blocks can be hashed on its own, as long as each partial sum
// is multiplied by the right power of H before the sums are XORed together.  A
// run is split over the 32 lanes of a warp, each lane keeping U interleaved
// Horner chains with stride 32*U blocks: A <- A * H^(32U) + C.  A chain whose
// last block has 1-based index i in the segment contributes A * H^(n-i+2).
// Arbitrary powers come from a per-key table pow[m][d] = H^(d * 256^m).
//
// Everything here compiles for host and device so that the host-side checks can
// run the same arithmetic without a GPU.
#pragma once
#include <stdint.h>

#include "aes_tt.cuh"
#include "gf128.cuh"

namespace gift {

enum { MODE_ENCRYPT = 0, MODE_DECRYPT = 1, MODE_VERIFY = 2 };

constexpr int POW_LEVELS = 4;          // exponents up to 2^32 - 1

// Per-user key material read by the hot loop.  512 bytes, 16-byte aligned fields.
struct KeyHot {
    uint32_t rk[44];                   // AES-128 round keys, LE column words
    uint32_t h[4];                     // hash subkey H = E_K(0), natural domain
    mulop hs;                          // H^32, prepared multiplier (the stride of a lane's hash chain)
    uint32_t valid;                    // 1 when a key is installed
    uint32_t pad[7];
};
static_assert(sizeof(KeyHot) == 512, "KeyHot layout");

// H^e from the per-key table of POW_LEVELS x 256 entries, e >= 0.
GIFT_HD u128 mul_by_power(const u128& a, const u128* powtab, uint64_t e)
{
    u128 r = a;
#pragma unroll 1
    for (int m = 0; m < POW_LEVELS; m++) {
        const uint32_t d = (uint32_t)(e >> (8 * m)) & 0xFFu;
        if (d) r = gfmul(r, powtab[m * 256 + d]);
    }
    return r;
}

// Ask for the table entries that mul_by_power(.., e) will read, ahead of time (the exponent of
// a lane's chain is known before its first block is hashed; the entries then arrive while the
// rows are processed instead of sitting, one after the other, on the tail of the piece).
GIFT_HD void pow_prefetch(const u128* powtab, uint64_t e)
{
#if defined(__CUDA_ARCH__)
#pragma unroll
    for (int m = 0; m < POW_LEVELS; m++) {
        const uint32_t d = (uint32_t)(e >> (8 * m)) & 0xFFu;
        if (d) asm volatile("prefetch.global.L1 [%0];" ::"l"(powtab + m * 256 + d));
    }
#else
    (void)powtab; (void)e;
#endif
}

// ---- static work split --------------------------------------------------------------------
//
// The accepted segments' weights are laid end to end and resident warp w takes the weight
// range [w*slice, (w+1)*slice).  A segment's weight is its rows of 32 blocks plus SEG_WEIGHT
// for what a piece of work costs beyond its rows; its first SEG_WEIGHT units stand for that
// overhead, the rest map to its blocks.  A slice boundary inside a segment is rounded down to
// a whole row, so every piece starts on a row.
constexpr uint32_t SEG_WEIGHT = 64u;
constexpr uint32_t MIN_SLICE = 256u;

GIFT_HD uint64_t seg_weight(uint64_t nblk)
{
    return ((nblk + 31u) & ~(uint64_t)31u) + SEG_WEIGHT;     // an empty segment still needs its tag
}

// First block of the piece that starts at weight distance d from the segment's start.
GIFT_HD uint64_t slice_cut(uint64_t d, uint64_t nblk)
{
    if (d <= SEG_WEIGHT) return 0;
    const uint64_t b = d - SEG_WEIGHT;
    return b >= nblk ? nblk : (b & ~(uint64_t)31u);
}

// The blocks [first, end) of a segment that belong to the slice [g0, g1), for a segment of nblk
// blocks whose weight range is [p0, p1), and the number of slices that meet the segment: each
// of those reports once, with or without blocks, and the last report completes the segment.
struct SlicePiece {
    uint64_t first, end;
    uint32_t reporters;
};

GIFT_HD SlicePiece slice_piece(uint64_t g0, uint64_t g1, uint64_t p0, uint64_t p1, uint64_t nblk, uint64_t slice)
{
    SlicePiece r;
    r.first = g0 <= p0 ? 0 : slice_cut(g0 - p0, nblk);
    r.end = g1 >= p1 ? nblk : slice_cut(g1 - p0, nblk);
    r.reporters = (g0 <= p0 && g1 >= p1) ? 1u : (uint32_t)((p1 - 1) / slice - p0 / slice) + 1u;
    return r;
}

// Where the bytes of a segment live: flat (one offset) or through a page table.
struct SegAddr {
    const int32_t* table;     // nullptr: flat
    uint64_t page_bytes;
    uint64_t origin;          // flat: byte offset of the segment; paged: index of its first table entry
};

// Walks a segment's bytes in increasing order without dividing per block.
struct Cursor {
    SegAddr a;
    uint64_t pidx;            // page number within the segment
    uint64_t within;          // byte position inside that page (flat: inside the segment)
    uint64_t loaded;          // page whose base is cached
    uint64_t base;

    GIFT_HD void seek(const SegAddr& addr, uint64_t k)
    {
        a = addr;
        loaded = ~(uint64_t)0;
        if (a.table) {
            pidx = k / a.page_bytes;
            within = k - pidx * a.page_bytes;
            base = 0;
        } else {
            pidx = 0;
            within = k;
            base = a.origin;
        }
    }
    GIFT_HD void advance(uint64_t bytes) { within += bytes; }
    GIFT_HD uint64_t offset()
    {
        if (a.table) {
            while (within >= a.page_bytes) {
                within -= a.page_bytes;
                pidx++;
            }
            if (pidx != loaded) {
                base = (uint64_t)(uint32_t)a.table[a.origin + pidx] * a.page_bytes;
                loaded = pidx;
            }
        }
        return base + within;
    }
};

struct Block {
    uint32_t d[4];
};

GIFT_HD Block load_block(const uint8_t* p)
{
    Block b;
#if defined(__CUDA_ARCH__)
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    b.d[0] = v.x; b.d[1] = v.y; b.d[2] = v.z; b.d[3] = v.w;
#else
    for (int k = 0; k < 4; k++)
        b.d[k] = (uint32_t)p[4 * k] | ((uint32_t)p[4 * k + 1] << 8) | ((uint32_t)p[4 * k + 2] << 16) |
                 ((uint32_t)p[4 * k + 3] << 24);
#endif
    return b;
}

GIFT_HD void store_block(uint8_t* p, const Block& b)
{
#if defined(__CUDA_ARCH__)
    *reinterpret_cast<uint4*>(p) = make_uint4(b.d[0], b.d[1], b.d[2], b.d[3]);
#else
    for (int k = 0; k < 4; k++) {
        p[4 * k] = (uint8_t)b.d[k];
        p[4 * k + 1] = (uint8_t)(b.d[k] >> 8);
        p[4 * k + 2] = (uint8_t)(b.d[k] >> 16);
        p[4 * k + 3] = (uint8_t)(b.d[k] >> 24);
    }
#endif
}

// First n (< 16) bytes of a block, the rest zero.
GIFT_HD Block load_partial(const uint8_t* p, uint32_t n)
{
    Block b;
    b.d[0] = b.d[1] = b.d[2] = b.d[3] = 0;
    for (uint32_t k = 0; k < n; k++) b.d[k >> 2] |= (uint32_t)p[k] << (8 * (k & 3));
    return b;
}

GIFT_HD void store_partial(uint8_t* p, const Block& b, uint32_t n)
{
    for (uint32_t k = 0; k < n; k++) p[k] = (uint8_t)(b.d[k >> 2] >> (8 * (k & 3)));
}

GIFT_HD void mask_partial(Block& b, uint32_t n)
{
    for (uint32_t k = n; k < 16; k++) b.d[k >> 2] &= ~(0xFFu << (8 * (k & 3)));
}

// One lane's share of a run.
//   seg_nblk   number of 16-byte blocks of the whole segment (last may be partial)
//   run_first  0-based index of the run's first block in the segment
//   run_n      blocks in the run
//   tail       len % 16 of the segment (0: last block is full)
// Returns the lane's GHASH contribution, already multiplied by its power of H.
template <int U, int MODE, class Tab>
GIFT_HD u128 run_lane(const Tab& tb, const uint32_t* rk, const CtrPrefix& pre, const mulop& hs,
                      const u128* powtab, const uint8_t* src, uint8_t* dst, const SegAddr& addr,
                      uint64_t seg_nblk, uint64_t run_first, uint32_t run_n, uint32_t tail, int lane)
{
    u128 acc[U];
    Cursor cur[U];
#pragma unroll
    for (int u = 0; u < U; u++) {
        acc[u] = gf_zero();
        cur[u].seek(addr, (run_first + (uint64_t)(32 * u + lane)) * 16);
    }
#pragma unroll 1
    for (uint32_t base = 0; base < run_n; base += 32 * U) {
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint32_t i = base + 32 * u + (uint32_t)lane;
            if (i < run_n) {
                const uint64_t gb = run_first + i;
                const uint64_t off = cur[u].offset();
                const bool partial = tail != 0 && gb == seg_nblk - 1;
                Block d = partial ? load_partial(src + off, tail) : load_block(src + off);
                Block c = d;
                if (MODE != MODE_VERIFY) {
                    uint32_t ks[4];
                    ctr_keystream(tb, rk, pre, (uint32_t)(gb + 2), ks);
                    Block o;
                    o.d[0] = d.d[0] ^ ks[0]; o.d[1] = d.d[1] ^ ks[1];
                    o.d[2] = d.d[2] ^ ks[2]; o.d[3] = d.d[3] ^ ks[3];
                    if (partial) {
                        store_partial(dst + off, o, tail);
                        mask_partial(o, tail);
                    } else {
                        store_block(dst + off, o);
                    }
                    if (MODE == MODE_ENCRYPT) c = o;
                }
                acc[u] = xor128(gfmul(acc[u], hs), block_to_field(c.d[0], c.d[1], c.d[2], c.d[3]));
                cur[u].advance((uint64_t)(32 * U) * 16);
            }
        }
    }
    u128 sum = gf_zero();
#pragma unroll
    for (int u = 0; u < U; u++) {
        const uint32_t first = 32 * u + (uint32_t)lane;
        if (first < run_n) {
            const uint32_t i_last = first + ((run_n - 1 - first) / (32 * U)) * (32 * U);
            const uint64_t e = seg_nblk - run_first - i_last + 1;     // = n - i + 2, i 1-based
            sum = xor128(sum, mul_by_power(acc[u], powtab, e));
        }
    }
    return sum;
}

// The same work as run_lane with one chain per lane, arranged for the hot loop:
//  - rows of 32 blocks in which every lane has a full block run without predicates, the
//    lane pointer advancing by 512 bytes per row; in paged mode this needs pages that are
//    a multiple of 512 bytes, so that a row never straddles a page (otherwise the caller
//    uses run_lane);
//  - the loop is software pipelined: the keystream of row j and the hash update of row
//    j-1 are independent, so the table lookups of the cipher and the multiplies and logic
//    of the hash can interleave inside one warp;
//  - the ragged last row (and a partial last block) goes through predicated code once.
template <int MODE, bool PEEL, class Tab>
GIFT_HD u128 run_lane_rows(const Tab& tb, const uint32_t* rk, const CtrPrefix& pre, const mulop& hs,
                           const u128* powtab, const uint8_t* src, uint8_t* dst, const SegAddr& addr,
                           uint64_t seg_nblk, uint64_t run_first, uint32_t run_n, uint32_t tail, int lane)
{
    const bool has_partial = tail != 0 && run_n != 0 && run_first + run_n == seg_nblk;
    const uint32_t n_full = run_n - (has_partial ? 1u : 0u);
    const uint32_t rows = n_full >> 5;                      // rows in which all 32 lanes hold a full block
    u128 acc = gf_zero();
    uint32_t ctr = (uint32_t)(run_first + 2) + (uint32_t)lane;

    // position of the run's first row
    uint64_t pidx = 0, within = run_first * 16, base;
    uint32_t rows_in_page = 0xFFFFFFFFu;                    // flat: never wraps
    if (addr.table) {
        pidx = within / addr.page_bytes;
        within -= pidx * addr.page_bytes;
        base = (uint64_t)(uint32_t)addr.table[addr.origin + pidx] * addr.page_bytes;
        rows_in_page = (uint32_t)((addr.page_bytes - within) >> 9);
    } else {
        base = addr.origin;
    }
    uint64_t off = base + within + (uint64_t)lane * 16;     // this lane's block of the current row

    {
        // the exponent this lane's chain will need at the end (see below)
        const uint32_t n_mine = rows + ((rows * 32 + (uint32_t)lane) < run_n ? 1u : 0u);
        if (n_mine) pow_prefetch(powtab, seg_nblk - run_first - ((uint32_t)lane + (n_mine - 1) * 32) + 1);
    }
    Block c_prev;
    c_prev.d[0] = c_prev.d[1] = c_prev.d[2] = c_prev.d[3] = 0;
    bool pending = false;
    CtrGroup grp;
    grp.grp = ~(ctr >> 8);                                  // forces the first set-up
    grp.c2[0] = grp.c2[1] = grp.c2[2] = grp.c2[3] = 0;
    uint32_t j = 0;
    if (PEEL && rows != 0) {
        // The first row on its own, without the hash update of a previous row (which would
        // multiply zero): worth it where a piece is a handful of rows, i.e. in small calls; in
        // large ones the extra copy of the cipher code costs more than the multiply it saves.
        const Block d = load_block(src + off);
        Block c = d;
        if (MODE != MODE_VERIFY) {
            uint32_t ks[4];
            ctr_group_setup(tb, rk, pre, ctr, grp);
            ctr_keystream_grouped(tb, rk, pre, grp, ctr, ks);
            Block o;
            o.d[0] = d.d[0] ^ ks[0]; o.d[1] = d.d[1] ^ ks[1];
            o.d[2] = d.d[2] ^ ks[2]; o.d[3] = d.d[3] ^ ks[3];
            store_block(dst + off, o);
            if (MODE == MODE_ENCRYPT) c = o;
        }
        c_prev = c;
        pending = true;
        ctr += 32;
        off += 512;
        if (--rows_in_page == 0) {
            pidx++;
            if (1 < rows || (uint64_t)rows * 32 < run_n) {
                base = (uint64_t)(uint32_t)addr.table[addr.origin + pidx] * addr.page_bytes;
                off = base + (uint64_t)lane * 16;
            }
            rows_in_page = (uint32_t)(addr.page_bytes >> 9);
        }
        j = 1;
    }
#pragma unroll 1
    for (; j < rows; j++) {
        const Block d = load_block(src + off);
        Block c = d;
        if (MODE != MODE_VERIFY) {
            uint32_t ks[4];
            // the counter advances by 32 per row: a lane enters a new group of 256 every 8 rows
            if ((ctr >> 8) != grp.grp) ctr_group_setup(tb, rk, pre, ctr, grp);
            ctr_keystream_grouped(tb, rk, pre, grp, ctr, ks);
            Block o;
            o.d[0] = d.d[0] ^ ks[0]; o.d[1] = d.d[1] ^ ks[1];
            o.d[2] = d.d[2] ^ ks[2]; o.d[3] = d.d[3] ^ ks[3];
            store_block(dst + off, o);
            if (MODE == MODE_ENCRYPT) c = o;
        }
        // hash update of the previous row (the first pass multiplies zero, which stays zero)
        acc = xor128(gfmul(acc, hs), block_to_field(c_prev.d[0], c_prev.d[1], c_prev.d[2], c_prev.d[3]));
        c_prev = c;
        pending = true;
        // (the advance stays behind the hash update: its branch would otherwise split the block in
        // which the compiler interleaves cipher and hash; measured 405 instead of 436 GB/s)
        ctr += 32;
        off += 512;
        if (--rows_in_page == 0) {                          // next page (uniform across the warp)
            pidx++;
            if (j + 1 < rows || (uint64_t)rows * 32 < run_n) {
                base = (uint64_t)(uint32_t)addr.table[addr.origin + pidx] * addr.page_bytes;
                off = base + (uint64_t)lane * 16;
            }
            rows_in_page = (uint32_t)(addr.page_bytes >> 9);
        }
    }
    if (pending) acc = xor128(gfmul(acc, hs), block_to_field(c_prev.d[0], c_prev.d[1], c_prev.d[2], c_prev.d[3]));

    // ragged last row: some lanes hold one more block, one of them possibly the partial block
    const uint32_t i = rows * 32 + (uint32_t)lane;
    uint32_t count = rows;                                  // blocks this lane has hashed
    if (i < run_n) {
        const bool partial = has_partial && i == run_n - 1;
        const Block d = partial ? load_partial(src + off, tail) : load_block(src + off);
        Block c = d;
        if (MODE != MODE_VERIFY) {
            uint32_t ks[4];
            ctr_keystream(tb, rk, pre, ctr, ks);
            Block o;
            o.d[0] = d.d[0] ^ ks[0]; o.d[1] = d.d[1] ^ ks[1];
            o.d[2] = d.d[2] ^ ks[2]; o.d[3] = d.d[3] ^ ks[3];
            if (partial) {
                store_partial(dst + off, o, tail);
                mask_partial(o, tail);
            } else {
                store_block(dst + off, o);
            }
            if (MODE == MODE_ENCRYPT) c = o;
        }
        acc = xor128(gfmul(acc, hs), block_to_field(c.d[0], c.d[1], c.d[2], c.d[3]));
        count++;
    }
    if (count == 0) return gf_zero();
    const uint32_t i_last = (uint32_t)lane + (count - 1) * 32;
    const uint64_t e = seg_nblk - run_first - i_last + 1;
    return mul_by_power(acc, powtab, e);
}

// Tag from the combined hash S of all runs: T = (S + A*H^(n+2) + LEN*H) ^ E_K(J0), as four LE
// words.  A is an optional 16-byte block of additional authenticated data (SP 800-38D
// sec. 7.1: the AAD blocks precede the ciphertext in GHASH); aad == nullptr means none.
template <class Tab>
GIFT_HD void finish_tag(const Tab& tb, const uint32_t* rk, const uint32_t h[4], const uint32_t nonce[3],
                        uint64_t len_bytes, const u128& s, uint32_t tag[4], const uint8_t* aad = nullptr,
                        const u128* powtab = nullptr)
{
    // length block [8*|A|]_64 || [8*|C|]_64, big-endian bytes, as LE words then natural domain
    const uint64_t bits = len_bytes * 8;
    const u128 lenf = block_to_field(0u, aad ? bswap32(128u) : 0u, bswap32((uint32_t)(bits >> 32)),
                                     bswap32((uint32_t)bits));
    u128 hh;
    hh.w[0] = h[0]; hh.w[1] = h[1]; hh.w[2] = h[2]; hh.w[3] = h[3];
    u128 t = xor128(s, gfmul(lenf, hh));
    if (aad) {
        const Block a = load_block(aad);
        const uint64_t nblk = (len_bytes + 15) >> 4;
        t = xor128(t, mul_by_power(block_to_field(a.d[0], a.d[1], a.d[2], a.d[3]), powtab, nblk + 2));
    }
    uint32_t j0[4] = {nonce[0], nonce[1], nonce[2], 0x01000000u};     // nonce || 00 00 00 01
    aes128_encrypt(tb, rk, j0);
    tag[0] = reflect_bytes(t.w[0]) ^ j0[0];
    tag[1] = reflect_bytes(t.w[1]) ^ j0[1];
    tag[2] = reflect_bytes(t.w[2]) ^ j0[2];
    tag[3] = reflect_bytes(t.w[3]) ^ j0[3];
}

// Key schedule, hash subkey and its powers for one user (runs once per key change).
template <class Tab>
GIFT_HD void derive_key_hot(const Tab& tb, const uint32_t key[4], KeyHot* out, u128* h_out)
{
    aes128_expand_key(tb, key, out->rk);
    uint32_t z[4] = {0u, 0u, 0u, 0u};
    aes128_encrypt(tb, out->rk, z);
    const u128 h = block_to_field(z[0], z[1], z[2], z[3]);
    out->h[0] = h.w[0]; out->h[1] = h.w[1]; out->h[2] = h.w[2]; out->h[3] = h.w[3];
    u128 p = h;
    for (int k = 0; k < 5; k++) p = gfmul(p, p);       // H^32
    out->hs = prepare_mulop(p);
    out->valid = 1u;
    for (int k = 0; k < 7; k++) out->pad[k] = 0u;
    *h_out = h;
}

// Level m of the power table: pow[m][d] = (H^(256^m))^d for d = 0..255.
GIFT_HD void build_pow_level(const u128& h, int m, u128* level)
{
    u128 b = h;
    for (int k = 0; k < 8 * m; k++) b = gfmul(b, b);
    const mulop bp = prepare_mulop(b);
    u128 p = gf_one();
    level[0] = p;
    for (int d = 1; d < 256; d++) {
        p = gfmul(p, bp);
        level[d] = p;
    }
}

}  // namespace gift
