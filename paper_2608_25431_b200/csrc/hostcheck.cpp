// Host build of the device arithmetic, for tests that run without a GPU.
//
// gf128.cuh, aes_tt.cuh and gift_core.cuh compile for both host and device.
// This file exposes them through a C interface so that the field product, the
// table cipher, the key derivation, the power table and the whole
// run / lane / chain decomposition of a segment can be compared with the CPU
// oracle before any kernel runs.  It is not part of libgift.so.
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "gift_core.cuh"
#include "gift_csr.cuh"

using namespace gift;

static uint32_t g_t0[256];
static bool g_ready = false;

static const PlainTab& tab()
{
    static PlainTab t;
    if (!g_ready) {
        for (uint32_t x = 0; x < 256; x++) g_t0[x] = t0_entry(x);
        g_ready = true;
    }
    t.t0 = g_t0;
    return t;
}

static void key_words(const uint8_t* k, uint32_t w[4])
{
    Block b = load_block(k);
    for (int i = 0; i < 4; i++) w[i] = b.d[i];
}

extern "C" {

void hc_t0_table(uint32_t out[256])
{
    tab();
    memcpy(out, g_t0, sizeof(g_t0));
}

void hc_gfmul(const uint8_t* x, const uint8_t* y, uint8_t* z)
{
    Block a = load_block(x), b = load_block(y);
    u128 fa = block_to_field(a.d[0], a.d[1], a.d[2], a.d[3]);
    u128 fb = block_to_field(b.d[0], b.d[1], b.d[2], b.d[3]);
    u128 r = gfmul(fa, fb);
    Block o;
    for (int i = 0; i < 4; i++) o.d[i] = reflect_bytes(r.w[i]);
    store_block(z, o);
}

void hc_expand_key(const uint8_t* key, uint8_t* rk176)
{
    uint32_t k[4], rk[44];
    key_words(key, k);
    aes128_expand_key(tab(), k, rk);
    for (int i = 0; i < 44; i++) {
        rk176[4 * i] = (uint8_t)rk[i]; rk176[4 * i + 1] = (uint8_t)(rk[i] >> 8);
        rk176[4 * i + 2] = (uint8_t)(rk[i] >> 16); rk176[4 * i + 3] = (uint8_t)(rk[i] >> 24);
    }
}

void hc_aes_encrypt(const uint8_t* key, const uint8_t* in, uint8_t* out)
{
    uint32_t k[4], rk[44];
    key_words(key, k);
    aes128_expand_key(tab(), k, rk);
    Block b = load_block(in);
    aes128_encrypt(tab(), rk, b.d);
    store_block(out, b);
}

void hc_aes_decrypt(const uint8_t* key, const uint8_t* in, uint8_t* out)
{
    uint32_t k[4], rk[44];
    key_words(key, k);
    aes128_expand_key(tab(), k, rk);
    uint8_t isbox[256];
    for (uint32_t x = 0; x < 256; x++) isbox[sbox_entry(x)] = (uint8_t)x;
    Block b = load_block(in);
    aes128_decrypt(isbox, rk, b.d);
    store_block(out, b);
}

// H^e through the 4-level power table, as block bytes.
void hc_power(const uint8_t* key, uint64_t e, uint8_t* out)
{
    uint32_t k[4];
    key_words(key, k);
    KeyHot hot;
    u128 h;
    derive_key_hot(tab(), k, &hot, &h);
    std::vector<u128> pow(POW_LEVELS * 256);
    for (int m = 0; m < POW_LEVELS; m++) build_pow_level(h, m, &pow[m * 256]);
    u128 r = mul_by_power(gf_one(), pow.data(), e);
    Block o;
    for (int i = 0; i < 4; i++) o.d[i] = reflect_bytes(r.w[i]);
    store_block(out, o);
}

uint64_t hc_seg_weight(uint64_t nblk) { return seg_weight(nblk); }

uint32_t hc_min_slice(void) { return MIN_SLICE; }

// out = {first, end, reporters} of slice [g0, g1) in the segment with weight range [p0, p1)
void hc_slice_piece(uint64_t g0, uint64_t g1, uint64_t p0, uint64_t p1, uint64_t nblk, uint64_t slice, uint64_t out[3])
{
    const SlicePiece r = slice_piece(g0, g1, p0, p1, nblk, slice);
    out[0] = r.first; out[1] = r.end; out[2] = r.reporters;
}

}  // extern "C"

// One whole segment, decomposed exactly as the kernel does: runs of run_blocks
// blocks, 32 lanes per run, U chains per lane (U == 0: the row loop; U == 3: the row loop with
// its first row peeled off, as small calls run it).  mode: 0 encrypt, 1 decrypt, 2 verify.
// table == NULL: flat at byte offset origin; else paged from table entry origin.
template <int U>
static void seg_emulate(const uint8_t* key, const uint8_t* nonce12, const uint8_t* src, uint8_t* dst,
                        const int32_t* table, uint64_t page_bytes, uint64_t origin, uint64_t len,
                        uint32_t run_blocks, int mode, uint8_t* tag16)
{
    uint32_t k[4];
    key_words(key, k);
    KeyHot hot;
    u128 h;
    derive_key_hot(tab(), k, &hot, &h);
    u128 p64 = h;
    for (int i = 0; i < 6; i++) p64 = gfmul(p64, p64);
    const mulop hs64 = prepare_mulop(p64);      // H^64: the stride of two chains per lane
    std::vector<u128> pow(POW_LEVELS * 256);
    for (int m = 0; m < POW_LEVELS; m++) build_pow_level(h, m, &pow[m * 256]);
    uint32_t nonce[3];
    Block nb = load_partial(nonce12, 12);
    nonce[0] = nb.d[0]; nonce[1] = nb.d[1]; nonce[2] = nb.d[2];
    const CtrPrefix pre = ctr_prefix(tab(), hot.rk, nonce);
    SegAddr addr = {table, page_bytes, origin};
    const uint64_t nblk = (len + 15) / 16;
    const uint32_t tail = (uint32_t)(len % 16);
    u128 s = gf_zero();
    for (uint64_t first = 0; first < nblk; first += run_blocks) {
        const uint32_t n = (uint32_t)(nblk - first < run_blocks ? nblk - first : run_blocks);
        for (int lane = 0; lane < 32; lane++) {
            u128 c;
            if (U == 3) {
                if (mode == 0)
                    c = run_lane_rows<MODE_ENCRYPT, true>(tab(), hot.rk, pre, hot.hs, pow.data(), src, dst, addr,
                                                   nblk, first, n, tail, lane);
                else if (mode == 1)
                    c = run_lane_rows<MODE_DECRYPT, true>(tab(), hot.rk, pre, hot.hs, pow.data(), src, dst, addr,
                                                   nblk, first, n, tail, lane);
                else
                    c = run_lane_rows<MODE_VERIFY, true>(tab(), hot.rk, pre, hot.hs, pow.data(), src, dst, addr,
                                                  nblk, first, n, tail, lane);
            } else if (U == 0) {          // the row-wise, software-pipelined loop (chains == 0 selects it)
                if (mode == 0)
                    c = run_lane_rows<MODE_ENCRYPT, false>(tab(), hot.rk, pre, hot.hs, pow.data(), src, dst, addr,
                                                    nblk, first, n, tail, lane);
                else if (mode == 1)
                    c = run_lane_rows<MODE_DECRYPT, false>(tab(), hot.rk, pre, hot.hs, pow.data(), src, dst, addr,
                                                    nblk, first, n, tail, lane);
                else
                    c = run_lane_rows<MODE_VERIFY, false>(tab(), hot.rk, pre, hot.hs, pow.data(), src, dst, addr,
                                                   nblk, first, n, tail, lane);
            } else if (mode == 0)
                c = run_lane<(U == 2 ? 2 : 1), MODE_ENCRYPT>(tab(), hot.rk, pre, (U == 2 ? hs64 : hot.hs), pow.data(), src, dst, addr,
                                              nblk, first, n, tail, lane);
            else if (mode == 1)
                c = run_lane<(U == 2 ? 2 : 1), MODE_DECRYPT>(tab(), hot.rk, pre, (U == 2 ? hs64 : hot.hs), pow.data(), src, dst, addr,
                                              nblk, first, n, tail, lane);
            else
                c = run_lane<(U == 2 ? 2 : 1), MODE_VERIFY>(tab(), hot.rk, pre, (U == 2 ? hs64 : hot.hs), pow.data(), src, dst, addr,
                                             nblk, first, n, tail, lane);
            s = xor128(s, c);
        }
    }
    uint32_t tag[4];
    finish_tag(tab(), hot.rk, hot.h, nonce, len, s, tag);
    Block t;
    for (int i = 0; i < 4; i++) t.d[i] = tag[i];
    store_block(tag16, t);
}

extern "C" {

void hc_segment(const uint8_t* key, const uint8_t* nonce12, const uint8_t* src, uint8_t* dst,
                const int32_t* table, uint64_t page_bytes, uint64_t origin, uint64_t len,
                uint32_t run_blocks, int chains, int mode, uint8_t* tag16)
{
    if (chains == 0)
        seg_emulate<0>(key, nonce12, src, dst, table, page_bytes, origin, len, run_blocks, mode, tag16);
    else if (chains == 1)
        seg_emulate<1>(key, nonce12, src, dst, table, page_bytes, origin, len, run_blocks, mode, tag16);
    else if (chains == 2)
        seg_emulate<2>(key, nonce12, src, dst, table, page_bytes, origin, len, run_blocks, mode, tag16);
    else
        seg_emulate<3>(key, nonce12, src, dst, table, page_bytes, origin, len, run_blocks, mode, tag16);
}


// 1 if ptr[0..n) is a valid CSR pointer array for `limit` indexed items, by the pair checks the
// label kernels use.
int hc_csr_ok(const int32_t* ptr, uint32_t n, uint32_t limit)
{
    if (n == 0) return 0;
    if (n == 1) return csr_single_ok(ptr[0], limit) ? 1 : 0;
    for (uint32_t k = 0; k + 1 < n; k++)
        if (!csr_pair_ok(ptr[k], ptr[k + 1], k == 0, k + 2 == n, limit)) return 0;
    return 1;
}

}
