"""Pins for the CPU oracle's cipher: the standards' worked examples, OpenSSL, and algebra.

Each pin is chosen so that a plausible slip in the oracle (a wrong S-box constant, a
transposed state, a mis-ordered counter, a reversed bit order in GF(2^128), a dropped
length block) fails at least one of them.
"""
import os

import numpy as np
import pytest
from cryptography.hazmat.primitives.ciphers import Cipher, algorithms, modes
from cryptography.hazmat.primitives.ciphers.aead import AESGCM

from oracle import gcm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "standards_kat.txt")


def _hex(s):
    s = s.strip()
    return b"" if s == "-" else bytes.fromhex(s)


def _kat(kind):
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = [p.strip() for p in line.split("|")]
            if parts[0] == kind:
                rows.append(parts[1:])
    assert rows, kind
    return rows


def _ecb(key, block):
    return Cipher(algorithms.AES(key), modes.ECB()).encryptor().update(block)


# ---- published worked examples ------------------------------------------------

@pytest.mark.parametrize("row", _kat("block"), ids=lambda r: r[0])
def test_kat_block(row):
    _, key, pt, ct = row
    assert gcm.aes128_encrypt_block(_hex(key), _hex(pt)) == _hex(ct)
    assert _ecb(_hex(key), _hex(pt)) == _hex(ct)          # the fixture itself, via OpenSSL


@pytest.mark.parametrize("row", _kat("keyexp"), ids=lambda r: r[0])
def test_kat_key_expansion(row):
    _, key, idx, word = row
    rk = gcm.key_expand(_hex(key)).tobytes()
    i = int(idx)
    assert rk[4 * i: 4 * i + 4] == _hex(word)


@pytest.mark.parametrize("row", _kat("ctr"), ids=lambda r: r[0])
def test_kat_ctr(row):
    _, key, icb, pt, ct = row
    assert gcm.ctr32_xor(_hex(key), _hex(icb), _hex(pt)) == _hex(ct)
    assert Cipher(algorithms.AES(_hex(key)), modes.CTR(_hex(icb))).encryptor().update(_hex(pt)) == _hex(ct)


@pytest.mark.parametrize("row", _kat("gfmul"), ids=lambda r: r[0])
def test_kat_gfmul(row):
    _, x, h, z = row
    assert gcm.gf128_mul(_hex(x), _hex(h)) == _hex(z)


@pytest.mark.parametrize("row", _kat("ghash"), ids=lambda r: r[0])
def test_kat_ghash(row):
    _, h, aad, c, out = row
    assert gcm.ghash(_hex(h), _hex(aad), _hex(c)) == _hex(out)


@pytest.mark.parametrize("row", _kat("gcm"), ids=lambda r: r[0])
def test_kat_gcm(row):
    _, key, iv, aad, pt, ct, tag = row
    c, t = gcm.gcm_encrypt(_hex(key), _hex(iv), _hex(pt), _hex(aad))
    assert c == _hex(ct) and t == _hex(tag)
    assert AESGCM(_hex(key)).encrypt(_hex(iv), _hex(pt), _hex(aad) or None) == _hex(ct) + _hex(tag)
    assert gcm.gcm_decrypt(_hex(key), _hex(iv), _hex(ct), _hex(tag), _hex(aad)) == _hex(pt)


# ---- S-box: properties fixed by its definition ---------------------------------

def test_sbox_properties():
    s = gcm.sbox()
    assert sorted(s.tolist()) == list(range(256))              # a permutation
    assert s[0] == 0x63                                        # inverse(0) = 0, affine constant
    assert all(s[x] != x and s[x] != (x ^ 0xFF) for x in range(256))   # no fixed / opposite points
    assert s[0x53] == 0xED                                     # FIPS-197 sec. 5.1.1 worked example


# ---- OpenSSL equivalence on random and structured inputs -----------------------

def test_block_vs_openssl():
    rng = np.random.default_rng(1)
    cases = [(bytes(16), bytes(16)), (b"\xff" * 16, b"\xff" * 16)]
    for i in range(128):                                       # single-bit keys and blocks
        one = (1 << i).to_bytes(16, "big")
        cases += [(one, bytes(16)), (bytes(16), one)]
    cases += [(rng.bytes(16), rng.bytes(16)) for _ in range(2000)]
    for k, b in cases:
        assert gcm.aes128_encrypt_block(k, b) == _ecb(k, b)


def test_ctr_vs_openssl_lengths_and_wrap():
    rng = np.random.default_rng(2)
    for n in list(range(0, 50)) + [255, 256, 257, 4095, 4096, 4097]:
        k, icb, d = rng.bytes(16), rng.bytes(16), rng.bytes(n)
        ref = Cipher(algorithms.AES(k), modes.CTR(icb)).encryptor().update(d)
        if int.from_bytes(icb[12:], "big") + (n + 15) // 16 < 2 ** 32:
            assert gcm.ctr32_xor(k, icb, d) == ref
        assert gcm.ctr32_xor(k, icb, gcm.ctr32_xor(k, icb, d)) == d     # involution
    # 32-bit wrap: the counter field wraps without carrying into the nonce (SP 800-38D inc32)
    k = rng.bytes(16)
    icb = rng.bytes(12) + b"\xff\xff\xff\xff"
    d = rng.bytes(48)
    out = gcm.ctr32_xor(k, icb, d)
    ks0 = _ecb(k, icb)
    ks1 = _ecb(k, icb[:12] + bytes(4))
    ks2 = _ecb(k, icb[:12] + b"\x00\x00\x00\x01")
    assert out == bytes(a ^ b for a, b in zip(d, ks0 + ks1 + ks2))


def test_gcm_vs_openssl():
    rng = np.random.default_rng(3)
    lens = [0, 1, 15, 16, 17, 31, 32, 33, 64, 100, 144, 255, 256, 1000, 4096, 4100, 64004]
    for n in lens:
        for alen in (0, 0, 13, 16, 20):
            k, iv, pt, aad = rng.bytes(16), rng.bytes(12), rng.bytes(n), rng.bytes(alen)
            ref = AESGCM(k).encrypt(iv, pt, aad or None)
            ct, tag = gcm.gcm_encrypt(k, iv, pt, aad)
            assert ct + tag == ref, (n, alen)
            assert gcm.gcm_decrypt(k, iv, ct, tag, aad) == pt
    # the CTR stream of GCM starts at nonce || 00000002 (J0 + 1)
    k, iv, pt = rng.bytes(16), rng.bytes(12), rng.bytes(100)
    ct, _ = gcm.gcm_encrypt(k, iv, pt)
    assert ct == gcm.ctr32_xor(k, iv + b"\x00\x00\x00\x02", pt)


def test_gcm_rejects_any_single_bit_flip():
    rng = np.random.default_rng(4)
    k, iv, pt = rng.bytes(16), rng.bytes(12), rng.bytes(64)
    ct, tag = gcm.gcm_encrypt(k, iv, pt)
    for i in range(64 * 8):
        bad = bytearray(ct)
        bad[i // 8] ^= 1 << (i % 8)
        assert gcm.gcm_decrypt(k, iv, bytes(bad), tag) is None
    for i in range(128):
        bad = bytearray(tag)
        bad[i // 8] ^= 1 << (i % 8)
        assert gcm.gcm_decrypt(k, iv, ct, bytes(bad)) is None
    other = rng.bytes(16)
    assert gcm.gcm_decrypt(other, iv, ct, tag) is None


# ---- GF(2^128): axioms and closed forms -----------------------------------------

ONE = b"\x80" + bytes(15)          # the polynomial 1: bit 0 is the leftmost bit
X = b"\x40" + bytes(15)            # the polynomial x


def _xor(a, b):
    return bytes(p ^ q for p, q in zip(a, b))


def test_gf128_axioms():
    rng = np.random.default_rng(5)
    for _ in range(100):
        a, b, c = rng.bytes(16), rng.bytes(16), rng.bytes(16)
        assert gcm.gf128_mul(a, b) == gcm.gf128_mul(b, a)
        assert gcm.gf128_mul(gcm.gf128_mul(a, b), c) == gcm.gf128_mul(a, gcm.gf128_mul(b, c))
        assert gcm.gf128_mul(a, _xor(b, c)) == _xor(gcm.gf128_mul(a, b), gcm.gf128_mul(a, c))
        assert gcm.gf128_mul(a, ONE) == a
        assert gcm.gf128_mul(a, bytes(16)) == bytes(16)
        # squaring is linear in characteristic 2
        sq = lambda v: gcm.gf128_mul(v, v)
        assert sq(_xor(a, b)) == _xor(sq(a), sq(b))


def test_gf128_times_x_is_one_shift_step():
    rng = np.random.default_rng(6)
    for _ in range(200):
        a = rng.bytes(16)
        v = int.from_bytes(a, "big")
        out = v >> 1
        if v & 1:
            out ^= 0xE1 << 120
        assert gcm.gf128_mul(a, X) == out.to_bytes(16, "big")
    # x^128 = 1 + x + x^2 + x^7, i.e. the byte 0xE1 followed by zeros
    p = ONE
    for _ in range(128):
        p = gcm.gf128_mul(p, X)
    assert p == b"\xe1" + bytes(15)


def test_gf128_vs_integer_polynomial_arithmetic():
    """Independent model: carry-less product of Python integers reduced mod x^128+x^7+x^2+x+1."""
    def to_poly(b):            # coefficient of x^j = bit j of the block, left to right
        v = int.from_bytes(b, "big")
        return sum(((v >> (127 - j)) & 1) << j for j in range(128))

    def from_poly(p):
        v = sum(((p >> j) & 1) << (127 - j) for j in range(128))
        return v.to_bytes(16, "big")

    def mulmod(a, b):
        r = 0
        for j in range(128):
            if (b >> j) & 1:
                r ^= a << j
        mod = (1 << 128) | 0x87
        for j in range(254, 127, -1):
            if (r >> j) & 1:
                r ^= mod << (j - 128)
        return r

    rng = np.random.default_rng(7)
    for _ in range(100):
        a, b = rng.bytes(16), rng.bytes(16)
        assert gcm.gf128_mul(a, b) == from_poly(mulmod(to_poly(a), to_poly(b)))


def test_ghash_closed_form_and_chunk_combine():
    rng = np.random.default_rng(8)
    h = rng.bytes(16)
    powers = [ONE]
    for _ in range(16):
        powers.append(gcm.gf128_mul(powers[-1], h))
    m = 9
    c = rng.bytes(16 * m)
    blocks = [c[16 * i: 16 * i + 16] for i in range(m)]
    lenblk = (0).to_bytes(8, "big") + (8 * len(c)).to_bytes(8, "big")
    # closed form: S = sum_i C_i * H^(m-i+2) + LEN * H    (i = 1..m)
    s = gcm.gf128_mul(lenblk, powers[1])
    for i, blk in enumerate(blocks, start=1):
        s = _xor(s, gcm.gf128_mul(blk, powers[m - i + 2]))
    assert gcm.ghash(h, b"", c) == s

    # every split point: partial Horner sums of the two chunks recombine with a power of H
    def horner(bl):
        y = bytes(16)
        for blk in bl:
            y = gcm.gf128_mul(_xor(y, blk), h)
        return y              # last block carries H^1

    for cut in range(0, m + 1):
        left, right = horner(blocks[:cut]), horner(blocks[cut:])
        whole = _xor(gcm.gf128_mul(left, powers[m - cut]), right)
        total = gcm.gf128_mul(_xor(whole, lenblk), h)
        assert total == gcm.ghash(h, b"", c), cut


def test_ghash_zero_padding_and_aad_layout():
    rng = np.random.default_rng(9)
    h = rng.bytes(16)
    a, c = rng.bytes(5), rng.bytes(21)
    lenblk = (8 * 5).to_bytes(8, "big") + (8 * 21).to_bytes(8, "big")
    y = bytes(16)
    for blk in (a + bytes(11), c[:16], c[16:] + bytes(11), lenblk):
        y = gcm.gf128_mul(_xor(y, blk), h)
    assert gcm.ghash(h, a, c) == y


# ---- inverse cipher and token mode ------------------------------------------------

def test_inverse_cipher_vs_openssl_and_published_example():
    rng = np.random.default_rng(10)
    for row in _kat("block"):
        _, key, pt, ct = row
        assert gcm.aes128_decrypt_block(_hex(key), _hex(ct)) == _hex(pt)      # FIPS-197 App. C.1 inverse cipher
    for _ in range(500):
        k, b = rng.bytes(16), rng.bytes(16)
        dec = Cipher(algorithms.AES(k), modes.ECB()).decryptor().update(b)
        assert gcm.aes128_decrypt_block(k, b) == dec
        assert gcm.aes128_decrypt_block(k, gcm.aes128_encrypt_block(k, b)) == b


def test_token_mode_layout_marker_and_round_trip():
    rng = np.random.default_rng(11)
    ids = np.arange(4, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(64), dtype=np.uint8).reshape(4, 16)
    eos = 2
    toks = np.array([17, 2, 17, 31999, 2**63 + 5, 17], dtype=np.uint64)
    nonces = rng.integers(0, 2**63, size=6, dtype=np.uint64)
    owners = np.array([0, 1, 0, 3, 2, 9], dtype=np.int32)          # user 9 has no key
    ct, st = gcm.tok_encrypt(toks, nonces, owners, eos, ids, keys, 16)
    assert st.tolist() == [0, 0, 0, 0, 0, 8] and not ct[5].any()
    assert (ct[1] == 0xFF).all()                                   # the end-of-sequence marker
    # one cipher block per token: bytes 0-7 token, 8-15 nonce, little-endian, under the owner's key
    blk = int(toks[0]).to_bytes(8, "little") + int(nonces[0]).to_bytes(8, "little")
    assert ct[0].tobytes() == _ecb(keys[0].tobytes(), blk)
    assert ct[0].tobytes() != ct[2].tobytes()                      # same token, same key, other nonce
    t2, n2, st2 = gcm.tok_decrypt(ct, owners, eos, ids, keys, 16)
    assert st2.tolist() == [0, 0, 0, 0, 0, 8]
    assert t2[:5].tolist() == toks[:5].tolist() and t2[5] == 0
    assert n2[[0, 2, 3, 4]].tolist() == nonces[[0, 2, 3, 4]].tolist()
    # a wrong claimed owner yields another token, never the plaintext (paper sec. 3, step 3)
    wrong = owners.copy()
    wrong[0] = 1
    t3, _, _ = gcm.tok_decrypt(ct, wrong, eos, ids, keys, 16)
    assert t3[0] != toks[0]
