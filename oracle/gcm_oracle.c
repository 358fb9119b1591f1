/*
 * CPU oracle for per-user segment encryption (test infrastructure, not product).
 *
 * A plain, slow restatement of the definitions the GPU path must reproduce bit
 * for bit: the AES-128 forward cipher (FIPS-197), counter mode with GCM's
 * counter layout (SP 800-38A sec. 6.5, SP 800-38D sec. 7.1), GHASH and the tag
 * (SP 800-38D sec. 6.3, 6.4, 7.1), and the per-segment semantics of the
 * paper's encryption-as-isolation workflow (paper sec. 3, steps 3-5: decrypt
 * with the claimed owner's key, a lie about ownership ends in a decryption
 * failure; sec. 3 step 4: every private byte has one owner; sec. 4.2: unowned
 * memory may not be read).
 *
 * Nothing here is tuned: the S-box is computed from its definition, the
 * GF(2^128) product is the bit-serial algorithm, there are no tables beyond
 * the 256-byte S-box, no blocking and no fusion.  The only parallelism is an
 * OpenMP loop over independent segments.  The GPU library shares no code,
 * header, table or constant with this file.  Only tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.
 *
 * Pins (tests/test_oracle_*.py): OpenSSL equivalence for the block cipher, CTR
 * and whole-message GCM (with and without AAD); the published worked examples
 * under tests/golden/; field axioms and closed forms for GF(2^128) and GHASH.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* AES-128, FIPS-197                                                         */
/* ------------------------------------------------------------------------ */

/* GF(2^8) product modulo x^8 + x^4 + x^3 + x + 1 (FIPS-197 sec. 4.2). */
static uint8_t gf256_mul(uint8_t a, uint8_t b)
{
    uint8_t p = 0;
    for (int i = 0; i < 8; i++) {
        if (b & 1) p ^= a;
        uint8_t hi = a & 0x80;
        a = (uint8_t)(a << 1);
        if (hi) a ^= 0x1b;
        b >>= 1;
    }
    return p;
}

/* Multiplication by x (02) and by x+1 (03) in GF(2^8), FIPS-197 sec. 4.2.1. */
static uint8_t mul2(uint8_t a) { return (uint8_t)((a << 1) ^ ((a & 0x80) ? 0x1b : 0)); }
static uint8_t mul3(uint8_t a) { return (uint8_t)(mul2(a) ^ a); }

static uint8_t SBOX[256];
static int sbox_ready = 0;

/* S-box from its definition (FIPS-197 sec. 5.1.1): multiplicative inverse in
 * GF(2^8), 0 -> 0, followed by the affine map
 * b'_i = b_i ^ b_(i+4) ^ b_(i+5) ^ b_(i+6) ^ b_(i+7) ^ c_i,  c = 0x63. */
static void build_sbox(void)
{
    for (int x = 0; x < 256; x++) {
        uint8_t inv = 0;
        if (x != 0) {
            for (int y = 1; y < 256; y++) {
                if (gf256_mul((uint8_t)x, (uint8_t)y) == 1) { inv = (uint8_t)y; break; }
            }
        }
        uint8_t out = 0;
        for (int i = 0; i < 8; i++) {
            int bit = ((inv >> i) & 1) ^ ((inv >> ((i + 4) & 7)) & 1) ^
                      ((inv >> ((i + 5) & 7)) & 1) ^ ((inv >> ((i + 6) & 7)) & 1) ^
                      ((inv >> ((i + 7) & 7)) & 1) ^ ((0x63 >> i) & 1);
            out |= (uint8_t)(bit << i);
        }
        SBOX[x] = out;
    }
}

void gift_oracle_init(void)
{
    if (!sbox_ready) {
        build_sbox();
        sbox_ready = 1;
    }
}

void gift_oracle_sbox(uint8_t out[256])
{
    gift_oracle_init();
    memcpy(out, SBOX, 256);
}

/* KeyExpansion for Nk = 4, Nr = 10 (FIPS-197 sec. 5.2).  Words are kept as
 * four bytes in memory order, so rk[16*r .. 16*r+15] is round key r. */
void gift_oracle_aes128_key_expand(const uint8_t key[16], uint8_t rk[176])
{
    gift_oracle_init();
    memcpy(rk, key, 16);
    uint8_t rcon = 0x01;
    for (int i = 4; i < 44; i++) {
        uint8_t t[4];
        memcpy(t, rk + 4 * (i - 1), 4);
        if (i % 4 == 0) {
            /* RotWord then SubWord then Rcon */
            uint8_t t0 = t[0];
            t[0] = SBOX[t[1]] ^ rcon;
            t[1] = SBOX[t[2]];
            t[2] = SBOX[t[3]];
            t[3] = SBOX[t0];
            rcon = gf256_mul(rcon, 0x02);
        }
        for (int k = 0; k < 4; k++) rk[4 * i + k] = rk[4 * (i - 4) + k] ^ t[k];
    }
}

/* Cipher (FIPS-197 sec. 5.1).  State s[r][c] = in[r + 4c]. */
static void aes128_cipher(const uint8_t rk[176], const uint8_t in[16], uint8_t out[16])
{
    uint8_t s[4][4];
    for (int c = 0; c < 4; c++)
        for (int r = 0; r < 4; r++) s[r][c] = in[r + 4 * c] ^ rk[r + 4 * c];

    for (int round = 1; round <= 10; round++) {
        /* SubBytes */
        for (int r = 0; r < 4; r++)
            for (int c = 0; c < 4; c++) s[r][c] = SBOX[s[r][c]];
        /* ShiftRows: row r rotates left by r */
        for (int r = 1; r < 4; r++) {
            uint8_t row[4];
            for (int c = 0; c < 4; c++) row[c] = s[r][(c + r) & 3];
            for (int c = 0; c < 4; c++) s[r][c] = row[c];
        }
        /* MixColumns: circulant (02 03 01 01), skipped in the last round */
        if (round != 10) {
            for (int c = 0; c < 4; c++) {
                uint8_t a0 = s[0][c], a1 = s[1][c], a2 = s[2][c], a3 = s[3][c];
                s[0][c] = mul2(a0) ^ mul3(a1) ^ a2 ^ a3;
                s[1][c] = a0 ^ mul2(a1) ^ mul3(a2) ^ a3;
                s[2][c] = a0 ^ a1 ^ mul2(a2) ^ mul3(a3);
                s[3][c] = mul3(a0) ^ a1 ^ a2 ^ mul2(a3);
            }
        }
        /* AddRoundKey */
        for (int c = 0; c < 4; c++)
            for (int r = 0; r < 4; r++) s[r][c] ^= rk[16 * round + r + 4 * c];
    }
    for (int c = 0; c < 4; c++)
        for (int r = 0; r < 4; r++) out[r + 4 * c] = s[r][c];
}

void gift_oracle_aes128_encrypt_block(const uint8_t key[16], const uint8_t in[16], uint8_t out[16])
{
    uint8_t rk[176];
    gift_oracle_aes128_key_expand(key, rk);
    aes128_cipher(rk, in, out);
}

/* InvCipher (FIPS-197 sec. 5.3): the rounds of Cipher undone in reverse order
 * with InvShiftRows, InvSubBytes, AddRoundKey and InvMixColumns. */
static uint8_t INV_SBOX[256];
static int inv_sbox_ready = 0;

static void aes128_inv_cipher(const uint8_t rk[176], const uint8_t in[16], uint8_t out[16])
{
    if (!inv_sbox_ready) {
        for (int x = 0; x < 256; x++) INV_SBOX[SBOX[x]] = (uint8_t)x;
        inv_sbox_ready = 1;
    }
    uint8_t s[4][4];
    for (int c = 0; c < 4; c++)
        for (int r = 0; r < 4; r++) s[r][c] = in[r + 4 * c] ^ rk[160 + r + 4 * c];
    for (int round = 9; round >= 0; round--) {
        /* InvShiftRows: row r rotates right by r */
        for (int r = 1; r < 4; r++) {
            uint8_t row[4];
            for (int c = 0; c < 4; c++) row[(c + r) & 3] = s[r][c];
            for (int c = 0; c < 4; c++) s[r][c] = row[c];
        }
        /* InvSubBytes */
        for (int r = 0; r < 4; r++)
            for (int c = 0; c < 4; c++) s[r][c] = INV_SBOX[s[r][c]];
        /* AddRoundKey */
        for (int c = 0; c < 4; c++)
            for (int r = 0; r < 4; r++) s[r][c] ^= rk[16 * round + r + 4 * c];
        /* InvMixColumns: circulant (0e 0b 0d 09), skipped after the last AddRoundKey */
        if (round != 0) {
            for (int c = 0; c < 4; c++) {
                uint8_t a0 = s[0][c], a1 = s[1][c], a2 = s[2][c], a3 = s[3][c];
                s[0][c] = gf256_mul(a0, 0x0e) ^ gf256_mul(a1, 0x0b) ^ gf256_mul(a2, 0x0d) ^ gf256_mul(a3, 0x09);
                s[1][c] = gf256_mul(a0, 0x09) ^ gf256_mul(a1, 0x0e) ^ gf256_mul(a2, 0x0b) ^ gf256_mul(a3, 0x0d);
                s[2][c] = gf256_mul(a0, 0x0d) ^ gf256_mul(a1, 0x09) ^ gf256_mul(a2, 0x0e) ^ gf256_mul(a3, 0x0b);
                s[3][c] = gf256_mul(a0, 0x0b) ^ gf256_mul(a1, 0x0d) ^ gf256_mul(a2, 0x09) ^ gf256_mul(a3, 0x0e);
            }
        }
    }
    for (int c = 0; c < 4; c++)
        for (int r = 0; r < 4; r++) out[r + 4 * c] = s[r][c];
}

void gift_oracle_aes128_decrypt_block(const uint8_t key[16], const uint8_t in[16], uint8_t out[16])
{
    uint8_t rk[176];
    gift_oracle_aes128_key_expand(key, rk);
    aes128_inv_cipher(rk, in, out);
}

/* ------------------------------------------------------------------------ */
/* CTR (SP 800-38A sec. 6.5) with the 32-bit increment of SP 800-38D sec. 6.2 */
/* ------------------------------------------------------------------------ */

/* inc32: the last four bytes are a big-endian counter that wraps modulo 2^32. */
static void inc32(uint8_t cb[16])
{
    for (int i = 15; i >= 12; i--) {
        cb[i]++;
        if (cb[i] != 0) break;
    }
}

static void ctr32_xor_rk(const uint8_t rk[176], const uint8_t icb[16],
                         const uint8_t* in, uint8_t* out, uint64_t len)
{
    uint8_t cb[16], ks[16];
    memcpy(cb, icb, 16);
    uint64_t done = 0;
    while (done < len) {
        aes128_cipher(rk, cb, ks);
        uint64_t n = len - done < 16 ? len - done : 16;
        for (uint64_t k = 0; k < n; k++) out[done + k] = in[done + k] ^ ks[k];
        done += n;
        inc32(cb);
    }
}

/* Raw CTR starting from an arbitrary 16-byte initial counter block. */
void gift_oracle_ctr32_xor(const uint8_t key[16], const uint8_t icb[16],
                           const uint8_t* in, uint8_t* out, uint64_t len)
{
    uint8_t rk[176];
    gift_oracle_aes128_key_expand(key, rk);
    ctr32_xor_rk(rk, icb, in, out, len);
}

/* ------------------------------------------------------------------------ */
/* GF(2^128) and GHASH (SP 800-38D sec. 6.3, 6.4)                             */
/* ------------------------------------------------------------------------ */

/* A block as two 64-bit halves read big-endian: bit i of the block (numbered
 * left to right, bit 0 = most significant bit of byte 0 = coefficient of x^0)
 * is bit 63-i of hi for i < 64 and bit 127-i of lo otherwise. */
static uint64_t get_be64(const uint8_t* p)
{
    uint64_t v = 0;
    for (int i = 0; i < 8; i++) v = (v << 8) | p[i];
    return v;
}

static void put_be64(uint8_t* p, uint64_t v)
{
    for (int i = 0; i < 8; i++) p[i] = (uint8_t)(v >> (56 - 8 * i));
}

/* Z = X * Y, Algorithm 1 of SP 800-38D:  Z = 0, V = Y;  for i = 0..127:
 * if x_i then Z ^= V;  V = V >> 1 (towards higher bit numbers), and if the
 * bit shifted out was 1 then V ^= R with R = 11100001 || 0^120. */
void gift_oracle_gf128_mul(const uint8_t x[16], const uint8_t y[16], uint8_t z[16])
{
    uint64_t xh = get_be64(x), xl = get_be64(x + 8);
    uint64_t vh = get_be64(y), vl = get_be64(y + 8);
    uint64_t zh = 0, zl = 0;
    for (int i = 0; i < 128; i++) {
        int xi = i < 64 ? (int)((xh >> (63 - i)) & 1) : (int)((xl >> (127 - i)) & 1);
        if (xi) { zh ^= vh; zl ^= vl; }
        int out = (int)(vl & 1);
        vl = (vl >> 1) | (vh << 63);
        vh >>= 1;
        if (out) vh ^= ((uint64_t)0xe1) << 56;
    }
    put_be64(z, zh);
    put_be64(z + 8, zl);
}

/* Y_i = (Y_(i-1) ^ X_i) * H over the 16-byte blocks of data, the last one
 * zero padded (Algorithm 2 applied to a padded string). */
static void ghash_update(uint8_t y[16], const uint8_t h[16], const uint8_t* data, uint64_t len)
{
    uint64_t done = 0;
    while (done < len) {
        uint8_t blk[16] = {0};
        uint64_t n = len - done < 16 ? len - done : 16;
        memcpy(blk, data + done, n);
        for (int k = 0; k < 16; k++) y[k] ^= blk[k];
        gift_oracle_gf128_mul(y, h, y);
        done += n;
    }
}

/* GHASH_H(A || 0-pad || C || 0-pad || [8|A|]_64 || [8|C|]_64), sec. 7.1 step 5. */
void gift_oracle_ghash(const uint8_t h[16], const uint8_t* aad, uint64_t alen,
                       const uint8_t* c, uint64_t clen, uint8_t out[16])
{
    uint8_t y[16] = {0}, lenblk[16];
    ghash_update(y, h, aad, alen);
    ghash_update(y, h, c, clen);
    put_be64(lenblk, alen * 8);
    put_be64(lenblk + 8, clen * 8);
    ghash_update(y, h, lenblk, 16);
    memcpy(out, y, 16);
}

/* ------------------------------------------------------------------------ */
/* AES-128-GCM with a 96-bit IV and a 128-bit tag (SP 800-38D sec. 7)         */
/* ------------------------------------------------------------------------ */

static void gcm_tag(const uint8_t rk[176], const uint8_t nonce[12], const uint8_t* aad,
                    uint64_t alen, const uint8_t* ct, uint64_t len, uint8_t tag[16])
{
    uint8_t zero[16] = {0}, h[16], j0[16], s[16], ekj0[16];
    aes128_cipher(rk, zero, h);            /* H = E_K(0^128) */
    memcpy(j0, nonce, 12);                 /* J0 = IV || 0^31 || 1 */
    j0[12] = 0; j0[13] = 0; j0[14] = 0; j0[15] = 1;
    gift_oracle_ghash(h, aad, alen, ct, len, s);
    aes128_cipher(rk, j0, ekj0);
    for (int k = 0; k < 16; k++) tag[k] = s[k] ^ ekj0[k];   /* T = GCTR_K(J0, S) */
}

static void gcm_ctr(const uint8_t rk[176], const uint8_t nonce[12],
                    const uint8_t* in, uint8_t* out, uint64_t len)
{
    uint8_t icb[16];
    memcpy(icb, nonce, 12);                /* inc32(J0) = IV || 0^30 || 10 */
    icb[12] = 0; icb[13] = 0; icb[14] = 0; icb[15] = 2;
    ctr32_xor_rk(rk, icb, in, out, len);
}

void gift_oracle_gcm_encrypt(const uint8_t key[16], const uint8_t nonce[12],
                             const uint8_t* aad, uint64_t alen,
                             const uint8_t* pt, uint64_t len, uint8_t* ct, uint8_t tag[16])
{
    uint8_t rk[176];
    gift_oracle_aes128_key_expand(key, rk);
    gcm_ctr(rk, nonce, pt, ct, len);
    gcm_tag(rk, nonce, aad, alen, ct, len, tag);
}

/* Returns 0 and writes the plaintext if the tag matches; returns 1 and writes
 * nothing otherwise (sec. 7.2: the tag is checked over the received ciphertext). */
int gift_oracle_gcm_decrypt(const uint8_t key[16], const uint8_t nonce[12],
                            const uint8_t* aad, uint64_t alen,
                            const uint8_t* ct, uint64_t len, const uint8_t tag[16], uint8_t* pt)
{
    uint8_t rk[176], t[16];
    gift_oracle_aes128_key_expand(key, rk);
    gcm_tag(rk, nonce, aad, alen, ct, len, t);
    uint8_t diff = 0;
    for (int k = 0; k < 16; k++) diff |= (uint8_t)(t[k] ^ tag[k]);
    if (diff) return 1;
    gcm_ctr(rk, nonce, ct, pt, len);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Segment tables: the paper's workflow over ownership segments               */
/* ------------------------------------------------------------------------ */

/* One ownership segment (paper sec. 4.1, insight 1: one record per contiguous
 * same-owner region).  40 bytes, same field order as the caller's table. */
typedef struct {
    int32_t  owner;      /* claimed owner */
    uint32_t flags;      /* reserved, must be 0 */
    uint64_t offset;     /* flat mode: byte offset into the buffer */
    uint64_t len;        /* payload bytes, any value >= 0 */
    uint8_t  nonce[12];
    uint32_t page0;      /* paged mode: first entry of this segment in the page table */
} oracle_seg;

enum {
    ST_TAG_MISMATCH = 1, ST_OWNER_MISMATCH = 2, ST_UNOWNED = 4, ST_NO_KEY = 8, ST_BAD_DESC = 16,
    ST_OVERLAP = 32
};
enum { OWNER_PARAM = -1, OWNER_NONE = -2, OWNER_CONFLICT = -3 };

#define GCM_MAX_LEN ((((uint64_t)1) << 36) - 32)

typedef struct {
    const uint8_t* src; uint8_t* dst; uint64_t buf_bytes;
    const int32_t* page_table; uint32_t n_pages; uint64_t page_bytes;   /* page_table NULL: flat */
    int32_t* owner_map; uint32_t n_units; uint64_t unit_bytes;           /* owner_map NULL: none */
    const uint8_t* keys; const uint8_t* has_key; uint32_t max_users;     /* keys[u*16], has_key[u] */
} seg_env;

/* Descriptor validity: alignment, range, page entries, reserved flags. */
static int seg_bad_desc(const seg_env* e, const oracle_seg* s)
{
    if (s->flags != 0) return 1;
    if (s->len > GCM_MAX_LEN) return 1;
    if (e->page_table == NULL) {
        if (s->offset % 16 != 0) return 1;
        if (s->offset > e->buf_bytes || s->len > e->buf_bytes - s->offset) return 1;
        if (e->owner_map != NULL && s->len > 0) {
            uint64_t u1 = (s->offset + s->len + e->unit_bytes - 1) / e->unit_bytes;
            if (u1 > e->n_units) return 1;
        }
    } else {
        uint64_t np = (s->len + e->page_bytes - 1) / e->page_bytes;
        if ((uint64_t)s->page0 + np > e->n_pages) return 1;
        for (uint64_t p = 0; p < np; p++) {
            int32_t t = e->page_table[s->page0 + p];
            if (t < 0) return 1;
            if (((uint64_t)t + 1) * e->page_bytes > e->buf_bytes) return 1;
            if (e->owner_map != NULL && (uint64_t)t >= e->n_units) return 1;
        }
    }
    return 0;
}

/* The ownership units a segment covers: flat mode, the units of unit_bytes
 * that its byte range touches; paged mode, one unit per page it occupies,
 * indexed by the physical page number.  An empty segment covers nothing. */
static uint64_t seg_unit_count(const seg_env* e, const oracle_seg* s)
{
    if (s->len == 0) return 0;
    if (e->page_table == NULL) {
        uint64_t u0 = s->offset / e->unit_bytes;
        uint64_t u1 = (s->offset + s->len + e->unit_bytes - 1) / e->unit_bytes;
        return u1 - u0;
    }
    return (s->len + e->page_bytes - 1) / e->page_bytes;
}

static uint64_t seg_unit(const seg_env* e, const oracle_seg* s, uint64_t k)
{
    if (e->page_table == NULL) return s->offset / e->unit_bytes + k;
    return (uint64_t)e->page_table[s->page0 + k];
}

static int seg_has_key(const seg_env* e, int32_t owner)
{
    return owner >= 0 && (uint32_t)owner < e->max_users && e->has_key[owner];
}

/* Gather a segment's bytes out of the flat or paged buffer, and scatter back. */
static void seg_gather(const seg_env* e, const oracle_seg* s, const uint8_t* base, uint8_t* out)
{
    if (e->page_table == NULL) { memcpy(out, base + s->offset, s->len); return; }
    for (uint64_t k = 0; k < s->len; k += e->page_bytes) {
        uint64_t n = s->len - k < e->page_bytes ? s->len - k : e->page_bytes;
        uint64_t page = (uint64_t)e->page_table[s->page0 + k / e->page_bytes];
        memcpy(out + k, base + page * e->page_bytes, n);
    }
}

static void seg_scatter(const seg_env* e, const oracle_seg* s, uint8_t* base, const uint8_t* in)
{
    if (e->page_table == NULL) { memcpy(base + s->offset, in, s->len); return; }
    for (uint64_t k = 0; k < s->len; k += e->page_bytes) {
        uint64_t n = s->len - k < e->page_bytes ? s->len - k : e->page_bytes;
        uint64_t page = (uint64_t)e->page_table[s->page0 + k / e->page_bytes];
        memcpy(base + page * e->page_bytes, in + k, n);
    }
}

static int env_bad(const seg_env* e)
{
    if (e->page_table != NULL && (e->page_bytes == 0 || e->page_bytes % 16 != 0)) return 1;
    if (e->owner_map != NULL && e->page_table == NULL && e->unit_bytes == 0) return 1;
    return 0;
}

/* bad[i] = 1 where segment i has an invalid descriptor (used by the overlap definition,
 * which leaves such segments out). */
int gift_oracle_seg_bad_desc(uint64_t buf_bytes, const oracle_seg* segs, uint32_t nseg,
                             const int32_t* page_table, uint32_t n_pages, uint64_t page_bytes,
                             int has_labels, uint32_t n_units, uint64_t unit_bytes, uint8_t* bad)
{
    static int32_t dummy;
    seg_env e = { NULL, NULL, buf_bytes, page_table, n_pages, page_bytes,
                  has_labels ? &dummy : NULL, n_units, unit_bytes, NULL, NULL, 0 };
    if (env_bad(&e)) return -1;
    for (uint32_t i = 0; i < nseg; i++) bad[i] = (uint8_t)seg_bad_desc(&e, &segs[i]);
    return 0;
}

/* Export (paper sec. 3 steps 5-6, sec. 4.1 on key selection from the
 * ownership state): a segment is encrypted only if every unit it covers is
 * owned by the claimed owner, who must have a key.  Otherwise its destination
 * bytes are left as they were, its tag is zero and the status says why.
 * aad16, when not NULL, holds 16 bytes of additional authenticated data per
 * segment (SP 800-38D sec. 7.1). */
int gift_oracle_seg_encrypt(const uint8_t* src, uint8_t* dst, uint64_t buf_bytes,
                            const oracle_seg* segs, uint32_t nseg,
                            const int32_t* page_table, uint32_t n_pages, uint64_t page_bytes,
                            const int32_t* owner_map, uint32_t n_units, uint64_t unit_bytes,
                            const uint8_t* keys, const uint8_t* has_key, uint32_t max_users,
                            uint8_t* tags_out, uint32_t* status, const uint8_t* aad16,
                            const uint8_t* overlap)
{
    seg_env e = { src, dst, buf_bytes, page_table, n_pages, page_bytes,
                  (int32_t*)owner_map, n_units, unit_bytes, keys, has_key, max_users };
    if (env_bad(&e)) return -1;
    gift_oracle_init();
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < (int64_t)nseg; i++) {
        const oracle_seg* s = &segs[i];
        uint32_t st = 0;
        memset(tags_out + 16 * i, 0, 16);
        if (seg_bad_desc(&e, s)) { status[i] = ST_BAD_DESC; continue; }
        if (overlap != NULL && overlap[i]) { status[i] = ST_OVERLAP; continue; }   /* refused like a bad descriptor */
        if (owner_map != NULL) {
            uint64_t nu = seg_unit_count(&e, s);
            for (uint64_t k = 0; k < nu; k++) {
                int32_t l = owner_map[seg_unit(&e, s, k)];
                if (l <= OWNER_NONE) st |= ST_UNOWNED;                       /* unowned or conflicted */
                else if (l == OWNER_PARAM || l != s->owner) st |= ST_OWNER_MISMATCH;
            }
        }
        if (!seg_has_key(&e, s->owner)) st |= ST_NO_KEY;
        status[i] = st;
        if (st != 0) continue;
        uint8_t* tmp = (uint8_t*)malloc(s->len ? s->len : 1);
        if (!tmp) { failed = 1; continue; }
        seg_gather(&e, s, src, tmp);
        gift_oracle_gcm_encrypt(keys + 16 * (uint64_t)s->owner, s->nonce, aad16 ? aad16 + 16 * i : NULL,
                                aad16 ? 16 : 0, tmp, s->len, tmp, tags_out + 16 * i);
        seg_scatter(&e, s, dst, tmp);
        free(tmp);
    }
    return failed ? -2 : 0;
}

/* Import (paper sec. 3 steps 3-4): decrypt with the claimed owner's key.  A
 * matching tag yields the plaintext and records the claimed owner on the
 * covered units.  A mismatch, or a claimed owner without a key, is a
 * decryption failure: the destination bytes of the segment become zero and
 * the covered units become unowned.  Units are written in two passes so that
 * a unit covered by any failed segment ends up unowned.
 * mode 0: decrypt; mode 1: verify only (status, nothing else written). */
int gift_oracle_seg_decrypt(const uint8_t* src, uint8_t* dst, uint64_t buf_bytes,
                            const oracle_seg* segs, uint32_t nseg,
                            const int32_t* page_table, uint32_t n_pages, uint64_t page_bytes,
                            int32_t* owner_map, uint32_t n_units, uint64_t unit_bytes,
                            const uint8_t* keys, const uint8_t* has_key, uint32_t max_users,
                            const uint8_t* tags_in, uint32_t* status, int mode, const uint8_t* aad16,
                            const uint8_t* overlap)
{
    seg_env e = { src, dst, buf_bytes, page_table, n_pages, page_bytes,
                  owner_map, n_units, unit_bytes, keys, has_key, max_users };
    if (env_bad(&e)) return -1;
    gift_oracle_init();
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < (int64_t)nseg; i++) {
        const oracle_seg* s = &segs[i];
        if (seg_bad_desc(&e, s)) { status[i] = ST_BAD_DESC; continue; }
        if (overlap != NULL && overlap[i]) { status[i] = ST_OVERLAP; continue; }
        if (!seg_has_key(&e, s->owner)) {
            status[i] = ST_NO_KEY;
            if (mode == 0) {
                uint8_t* z = (uint8_t*)calloc(s->len ? s->len : 1, 1);
                if (!z) { failed = 1; continue; }
                seg_scatter(&e, s, dst, z);
                free(z);
            }
            continue;
        }
        uint8_t* tmp = (uint8_t*)malloc(s->len ? s->len : 1);
        if (!tmp) { failed = 1; continue; }
        seg_gather(&e, s, src, tmp);
        int bad = gift_oracle_gcm_decrypt(keys + 16 * (uint64_t)s->owner, s->nonce, aad16 ? aad16 + 16 * i : NULL,
                                          aad16 ? 16 : 0, tmp, s->len, tags_in + 16 * i, tmp);
        status[i] = bad ? ST_TAG_MISMATCH : 0;
        if (mode == 0) {
            if (bad) memset(tmp, 0, s->len);
            seg_scatter(&e, s, dst, tmp);
        }
        free(tmp);
    }
    if (mode == 0 && owner_map != NULL) {
        for (int pass = 0; pass < 2; pass++) {
            for (uint32_t i = 0; i < nseg; i++) {
                const oracle_seg* s = &segs[i];
                if (status[i] == ST_BAD_DESC || status[i] == ST_OVERLAP) continue;
                int ok = status[i] == 0;
                if ((pass == 0) != ok) continue;
                uint64_t nu = seg_unit_count(&e, s);
                for (uint64_t k = 0; k < nu; k++)
                    owner_map[seg_unit(&e, s, k)] = ok ? s->owner : OWNER_NONE;
            }
        }
    }
    return failed ? -2 : 0;
}

/* ------------------------------------------------------------------------ */
/* Token mode (paper sec. 4.5, "Token encryption")                            */
/* ------------------------------------------------------------------------ */

/* Each 64-bit token is extended to 128 bits with a 64-bit nonce and passed
 * through the block cipher under its owner's key, so that equal tokens do not
 * give equal ciphertexts and the framework can still split and append
 * sequences token by token.  Layout taken here: bytes 0-7 the token, bytes
 * 8-15 the nonce, both little-endian.  The end-of-sequence token gets a fixed
 * public marker instead of a ciphertext (16 bytes 0xFF) so that the framework
 * can see that generation has ended.  Decryption applies the inverse cipher
 * and drops the nonce; the marker decrypts to the end-of-sequence token.
 * Status: ST_NO_KEY when the owner has no key (output zero). */
static void put_le64(uint8_t* p, uint64_t v)
{
    for (int i = 0; i < 8; i++) p[i] = (uint8_t)(v >> (8 * i));
}

static uint64_t get_le64(const uint8_t* p)
{
    uint64_t v = 0;
    for (int i = 7; i >= 0; i--) v = (v << 8) | p[i];
    return v;
}

void gift_oracle_tok_encrypt(const uint64_t* tokens, const uint64_t* nonces, const int32_t* owners,
                             uint32_t n, uint64_t eos_token, const uint8_t* keys,
                             const uint8_t* has_key, uint32_t max_users, uint8_t* out16, uint32_t* status)
{
    gift_oracle_init();
    for (uint32_t i = 0; i < n; i++) {
        uint8_t* o = out16 + 16 * (uint64_t)i;
        int ok = owners[i] >= 0 && (uint32_t)owners[i] < max_users && has_key[owners[i]];
        status[i] = ok ? 0 : ST_NO_KEY;
        if (!ok) { memset(o, 0, 16); continue; }
        if (tokens[i] == eos_token) { memset(o, 0xFF, 16); continue; }
        uint8_t blk[16];
        put_le64(blk, tokens[i]);
        put_le64(blk + 8, nonces[i]);
        gift_oracle_aes128_encrypt_block(keys + 16 * (uint64_t)owners[i], blk, o);
    }
}

void gift_oracle_tok_decrypt(const uint8_t* in16, const int32_t* owners, uint32_t n, uint64_t eos_token,
                             const uint8_t* keys, const uint8_t* has_key, uint32_t max_users,
                             uint64_t* tokens_out, uint64_t* nonces_out, uint32_t* status)
{
    gift_oracle_init();
    for (uint32_t i = 0; i < n; i++) {
        const uint8_t* c = in16 + 16 * (uint64_t)i;
        int ok = owners[i] >= 0 && (uint32_t)owners[i] < max_users && has_key[owners[i]];
        status[i] = ok ? 0 : ST_NO_KEY;
        tokens_out[i] = 0;
        if (nonces_out) nonces_out[i] = 0;
        if (!ok) continue;
        int marker = 1;
        for (int k = 0; k < 16; k++) marker &= c[k] == 0xFF;
        if (marker) { tokens_out[i] = eos_token; continue; }
        uint8_t blk[16];
        gift_oracle_aes128_decrypt_block(keys + 16 * (uint64_t)owners[i], c, blk);
        tokens_out[i] = get_le64(blk);
        if (nonces_out) nonces_out[i] = get_le64(blk + 8);
    }
}

