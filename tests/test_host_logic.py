"""Host-side checks that need no GPU: the C-ABI surface, and the device arithmetic compiled
for the host (field product, table cipher, key schedule, power table and the whole
run / lane / chain decomposition of a segment) against the CPU oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import gcm
from paper_2608_25431_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _u8(b):
    return np.frombuffer(bytes(b), dtype=np.uint8).copy()


@pytest.fixture(scope="module")
def hc():
    return C.CDLL(B.build_hostcheck())


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "gift.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(gift_[a-z_]+)\s*\(", header)))
    assert "gift_seg_encrypt" in declared and "gift_propagate_labels" in declared
    lib = C.CDLL(B.build_lib())          # loading needs no GPU; nothing is called
    for name in declared:
        assert hasattr(lib, name), name
    from paper_2608_25431_b200 import binding
    assert sorted(binding.EXPORTS) == declared
    for name in declared:                          # the binding offers every call under its C name
        assert callable(getattr(binding, name)), name


def test_binding_fails_loudly_without_gpu():
    import torch
    from paper_2608_25431_b200 import binding
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        binding.Ctx(4)


def test_t0_table_matches_sbox_definition(hc):
    t0 = np.zeros(256, dtype=np.uint32)
    hc.hc_t0_table(_p(t0))
    s = gcm.sbox().astype(np.uint32)
    s2 = ((s << 1) ^ np.where(s & 0x80, 0x1B, 0)) & 0xFF
    assert np.array_equal(t0, s2 | (s << 8) | (s << 16) | ((s2 ^ s) << 24))


def test_field_product_matches_oracle(hc):
    rng = np.random.default_rng(0)
    special = [bytes(16), b"\x80" + bytes(15), b"\xff" * 16, bytes(15) + b"\x01", b"\x40" + bytes(15)]
    pairs = [(a, b) for a in special for b in special] + [(rng.bytes(16), rng.bytes(16)) for _ in range(500)]
    for a, b in pairs:
        z = np.zeros(16, dtype=np.uint8)
        hc.hc_gfmul(_p(_u8(a)), _p(_u8(b)), _p(z))
        assert z.tobytes() == gcm.gf128_mul(a, b)


def test_table_cipher_and_key_schedule_match_oracle(hc):
    rng = np.random.default_rng(1)
    for _ in range(300):
        k, b = _u8(rng.bytes(16)), _u8(rng.bytes(16))
        o = np.zeros(16, dtype=np.uint8)
        hc.hc_aes_encrypt(_p(k), _p(b), _p(o))
        assert o.tobytes() == gcm.aes128_encrypt_block(k, b)
        rk = np.zeros(176, dtype=np.uint8)
        hc.hc_expand_key(_p(k), _p(rk))
        assert rk.tobytes() == gcm.key_expand(k).tobytes()


def test_inverse_cipher_matches_oracle(hc):
    rng = np.random.default_rng(5)
    for _ in range(300):
        k, b = _u8(rng.bytes(16)), _u8(rng.bytes(16))
        o = np.zeros(16, dtype=np.uint8)
        hc.hc_aes_decrypt(_p(k), _p(b), _p(o))
        assert o.tobytes() == gcm.aes128_decrypt_block(k, b)


def test_power_table_matches_square_and_multiply(hc):
    rng = np.random.default_rng(2)
    k = _u8(rng.bytes(16))
    h = gcm.aes128_encrypt_block(k, bytes(16))

    def power(e):
        r, b = b"\x80" + bytes(15), h
        while e:
            if e & 1:
                r = gcm.gf128_mul(r, b)
            b = gcm.gf128_mul(b, b)
            e >>= 1
        return r

    for e in [0, 1, 2, 31, 32, 33, 255, 256, 257, 65535, 65536, 1 << 24, (1 << 32) - 1, 123456789]:
        o = np.zeros(16, dtype=np.uint8)
        hc.hc_power(_p(k), C.c_uint64(e), _p(o))
        assert o.tobytes() == power(e), e


@pytest.mark.parametrize("chains", [0, 1, 2, 3])      # 0: row loop, 1-2: chains per lane, 3: row loop with the first row peeled
def test_run_decomposition_reproduces_gcm(hc, chains):
    """Every (length, run length) split of a segment into runs, lanes and chains gives the oracle's bytes and tag."""
    rng = np.random.default_rng(3 + chains)
    for n in [0, 1, 15, 16, 17, 31, 32, 33, 511, 512, 513, 1024, 1040, 2048 + 7, 4096, 5000, 70000]:
        for run_blocks in (32, 64, 96, 1024):
            k, nonce = _u8(rng.bytes(16)), _u8(rng.bytes(12))
            pt = _u8(rng.bytes(n + 32))
            ct = np.full(n + 32, 0xEE, dtype=np.uint8)
            tag = np.zeros(16, dtype=np.uint8)
            hc.hc_segment(_p(k), _p(nonce), _p(pt), _p(ct), None, C.c_uint64(0), C.c_uint64(16), C.c_uint64(n),
                          C.c_uint32(run_blocks), chains, 0, _p(tag))
            ref_ct, ref_tag = gcm.gcm_encrypt(k, nonce, pt[16:16 + n])
            assert ct[16:16 + n].tobytes() == ref_ct and tag.tobytes() == ref_tag, (n, run_blocks)
            assert (ct[:16] == 0xEE).all() and (ct[16 + n:] == 0xEE).all()      # nothing outside the segment
            out = np.full(n + 32, 0xEE, dtype=np.uint8)
            tag2 = np.zeros(16, dtype=np.uint8)
            hc.hc_segment(_p(k), _p(nonce), _p(ct), _p(out), None, C.c_uint64(0), C.c_uint64(16), C.c_uint64(n),
                          C.c_uint32(run_blocks), chains, 1, _p(tag2))
            assert out[16:16 + n].tobytes() == pt[16:16 + n].tobytes() and tag2.tobytes() == ref_tag
            tag3 = np.zeros(16, dtype=np.uint8)
            hc.hc_segment(_p(k), _p(nonce), _p(ct), _p(out), None, C.c_uint64(0), C.c_uint64(16), C.c_uint64(n),
                          C.c_uint32(run_blocks), chains, 2, _p(tag3))
            assert tag3.tobytes() == ref_tag


@pytest.mark.parametrize("pb,chains", [(160, 2), (160, 1), (512, 0), (1024, 0), (1536, 0), (512, 3), (1536, 3)])
def test_paged_addressing_reproduces_gcm(hc, pb, chains):
    rng = np.random.default_rng(9)
    for n in [100, 160, 161, 1000, 3000, 3200, 5 * pb, 5 * pb + 1, 7 * pb - 1]:
        npg = (n + pb - 1) // pb
        if npg + 3 > 40:
            continue
        table = rng.permutation(40).astype(np.int32)
        buf = _u8(rng.bytes(40 * pb))
        out = buf.copy()
        tag = np.zeros(16, dtype=np.uint8)
        k, nonce = _u8(rng.bytes(16)), _u8(rng.bytes(12))
        hc.hc_segment(_p(k), _p(nonce), _p(buf), _p(out), _p(table), C.c_uint64(pb), C.c_uint64(3), C.c_uint64(n),
                      C.c_uint32(64), chains, 0, _p(tag))
        sl = [(int(table[3 + i]) * pb, min(pb, n - i * pb)) for i in range(npg)]
        plain = b"".join(buf[o:o + l].tobytes() for o, l in sl)
        got = b"".join(out[o:o + l].tobytes() for o, l in sl)
        ref_ct, ref_tag = gcm.gcm_encrypt(k, nonce, plain)
        assert got == ref_ct and tag.tobytes() == ref_tag, n
        touched = np.zeros(40 * pb, dtype=bool)
        for o, l in sl:
            touched[o:o + l] = True
        assert np.array_equal(out[~touched], buf[~touched])


def test_static_work_split_tiles_every_segment_exactly(hc):
    """The kernel's split arithmetic, compiled for the host: for random tables and warp counts
    the pieces of every accepted segment tile [0, nblk) in order, start on whole rows, and
    exactly the predicted number of slices report on it (the last report finishes its tag)."""
    hc.hc_seg_weight.restype = C.c_uint64
    hc.hc_seg_weight.argtypes = [C.c_uint64]
    hc.hc_min_slice.restype = C.c_uint32
    hc.hc_slice_piece.argtypes = [C.c_uint64] * 6 + [C.c_void_p]
    rng = np.random.default_rng(31)
    out = np.zeros(3, dtype=np.uint64)

    def check(nblks, accepted, n_warps):
        w = np.array([hc.hc_seg_weight(int(n)) if a else 0 for n, a in zip(nblks, accepted)], dtype=np.uint64)
        prefix = np.concatenate([[0], np.cumsum(w)]).astype(np.uint64)
        total = int(prefix[-1])
        slice_ = max((total + n_warps - 1) // n_warps, hc.hc_min_slice())
        pieces = [[] for _ in nblks]
        reports = np.zeros(len(nblks), dtype=np.int64)
        predicted = np.zeros(len(nblks), dtype=np.int64)
        for wi in range(n_warps):
            g0 = wi * slice_
            if g0 >= total:
                break
            g1 = min(g0 + slice_, total)
            s = int(np.searchsorted(prefix[:-1], g0, side="right")) - 1      # largest s with prefix[s] <= g0
            while s < len(nblks) and int(prefix[s]) < g1:
                p0, p1 = int(prefix[s]), int(prefix[s + 1])
                if p1 > p0:
                    hc.hc_slice_piece(g0, g1, p0, p1, int(nblks[s]), slice_, _p(out))
                    first, end, rep = int(out[0]), int(out[1]), int(out[2])
                    assert first <= end <= nblks[s]
                    assert first % 32 == 0 or first == nblks[s]
                    if end > first:
                        pieces[s].append((first, end))
                    reports[s] += 1
                    assert predicted[s] in (0, rep)
                    predicted[s] = rep
                s += 1
        for s, n in enumerate(nblks):
            if not accepted[s]:
                assert reports[s] == 0
                continue
            assert reports[s] == predicted[s] >= 1, (s, reports[s], predicted[s])
            pos = 0
            for a, b in pieces[s]:                                             # warps visit a segment in order
                assert a == pos
                pos = b
            assert pos == n

    check(np.full(256, 4001), np.ones(256, bool), 3552)                        # the decode-row table
    check(np.array([0]), np.array([True]), 3552)
    check(np.array([5, 0, 0, 70000]), np.array([True, True, False, True]), 4)
    for _ in range(120):
        n = int(rng.integers(1, 300))
        kind = int(rng.integers(0, 4))
        if kind == 0:
            nb = rng.integers(0, 6, size=n)
        elif kind == 1:
            nb = rng.integers(0, 5000, size=n)
        elif kind == 2:
            nb = rng.choice([0, 1, 31, 32, 33, 1024, 16384, 100000], size=n)
        else:
            nb = (rng.pareto(1.0, size=n) * 50).astype(np.int64)
        check(nb.astype(np.int64), rng.random(n) < 0.9, int(rng.choice([1, 7, 3552, 4736])))


def test_csr_pointer_check_matches_oracle_reading(hc):
    """The pair checks the label kernels apply to untrusted CSR pointer arrays accept exactly the
    tables the oracle's reading accepts (hand cases, then random ones)."""
    from oracle import labels as L
    hc.hc_csr_ok.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32]

    def ok(ptr, limit):
        a = np.asarray(ptr, dtype=np.int32)
        return bool(hc.hc_csr_ok(_p(a), a.size, limit))

    hand = [([0, 2, 5, 6], 6, True), ([0, 5, 2, 6], 6, False), ([0, 2, 5, 7], 6, False), ([-1, 2, 5, 6], 6, False),
            ([0, 0, 0], 0, True), ([3], 3, True), ([4], 3, False), ([-1], 3, False), ([1, 1], 0, False),
            ([0, 2**31 - 1, 5], 6, False), ([2, 3], 3, True)]
    for ptr, limit, want in hand:
        assert ok(ptr, limit) == want == L.csr_ok(ptr, limit), (ptr, limit)
    rng = np.random.default_rng(91)
    for _ in range(500):
        n = int(rng.integers(1, 12))
        limit = int(rng.integers(0, 30))
        ptr = np.sort(rng.integers(0, limit + 1, size=n)).astype(np.int32)
        if rng.random() < 0.5:
            ptr[int(rng.integers(0, n))] = int(rng.integers(-3, limit + 4))
        assert ok(ptr, limit) == L.csr_ok(ptr, limit), (ptr, limit)
