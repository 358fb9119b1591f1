"""ctypes wrapper around the C oracle (gcm_oracle.c).  Test infrastructure only.

Every function takes and returns numpy arrays / bytes; nothing here adds arithmetic of
its own, it only marshals arguments for the C definitions.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

ST_TAG_MISMATCH, ST_OWNER_MISMATCH, ST_UNOWNED, ST_NO_KEY, ST_BAD_DESC = 1, 2, 4, 8, 16
OWNER_PARAM, OWNER_NONE, OWNER_CONFLICT = -1, -2, -3

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.gift_oracle_init()
    return _lib


def _u8(b) -> np.ndarray:
    if isinstance(b, (bytes, bytearray)):
        return np.frombuffer(bytes(b), dtype=np.uint8).copy()
    a = np.ascontiguousarray(b)
    return a.view(np.uint8).reshape(-1)


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def sbox() -> np.ndarray:
    out = np.zeros(256, dtype=np.uint8)
    lib().gift_oracle_sbox(_p(out))
    return out


def key_expand(key) -> np.ndarray:
    k = _u8(key)
    assert k.size == 16
    rk = np.zeros(176, dtype=np.uint8)
    lib().gift_oracle_aes128_key_expand(_p(k), _p(rk))
    return rk


def aes128_encrypt_block(key, block) -> bytes:
    k, b = _u8(key), _u8(block)
    assert k.size == 16 and b.size == 16
    out = np.zeros(16, dtype=np.uint8)
    lib().gift_oracle_aes128_encrypt_block(_p(k), _p(b), _p(out))
    return out.tobytes()


def aes128_decrypt_block(key, block) -> bytes:
    k, b = _u8(key), _u8(block)
    assert k.size == 16 and b.size == 16
    out = np.zeros(16, dtype=np.uint8)
    lib().gift_oracle_aes128_decrypt_block(_p(k), _p(b), _p(out))
    return out.tobytes()


def ctr32_xor(key, icb, data) -> bytes:
    k, i, d = _u8(key), _u8(icb), _u8(data)
    assert k.size == 16 and i.size == 16
    out = np.zeros(max(d.size, 1), dtype=np.uint8)
    lib().gift_oracle_ctr32_xor(_p(k), _p(i), _p(d), _p(out), C.c_uint64(d.size))
    return out[: d.size].tobytes()


def gf128_mul(x, y) -> bytes:
    a, b = _u8(x), _u8(y)
    assert a.size == 16 and b.size == 16
    out = np.zeros(16, dtype=np.uint8)
    lib().gift_oracle_gf128_mul(_p(a), _p(b), _p(out))
    return out.tobytes()


def ghash(h, aad, c) -> bytes:
    hh, a, cc = _u8(h), _u8(aad), _u8(c)
    out = np.zeros(16, dtype=np.uint8)
    lib().gift_oracle_ghash(_p(hh), _p(a), C.c_uint64(a.size), _p(cc), C.c_uint64(cc.size), _p(out))
    return out.tobytes()


def gcm_encrypt(key, nonce, pt, aad=b""):
    k, n, p, a = _u8(key), _u8(nonce), _u8(pt), _u8(aad)
    assert k.size == 16 and n.size == 12
    ct = np.zeros(max(p.size, 1), dtype=np.uint8)
    tag = np.zeros(16, dtype=np.uint8)
    lib().gift_oracle_gcm_encrypt(_p(k), _p(n), _p(a), C.c_uint64(a.size), _p(p), C.c_uint64(p.size),
                                  _p(ct), _p(tag))
    return ct[: p.size].tobytes(), tag.tobytes()


def gcm_decrypt(key, nonce, ct, tag, aad=b""):
    """Plaintext bytes, or None when the tag does not match."""
    k, n, c, t, a = _u8(key), _u8(nonce), _u8(ct), _u8(tag), _u8(aad)
    assert k.size == 16 and n.size == 12 and t.size == 16
    pt = np.zeros(max(c.size, 1), dtype=np.uint8)
    lib().gift_oracle_gcm_decrypt.restype = C.c_int
    bad = lib().gift_oracle_gcm_decrypt(_p(k), _p(n), _p(a), C.c_uint64(a.size), _p(c),
                                        C.c_uint64(c.size), _p(t), _p(pt))
    return None if bad else pt[: c.size].tobytes()


def _key_table(user_ids, keys, max_users):
    tab = np.zeros((max_users, 16), dtype=np.uint8)
    has = np.zeros(max_users, dtype=np.uint8)
    for u, k in zip(np.asarray(user_ids).tolist(), np.asarray(keys).reshape(-1, 16)):
        tab[u] = k
        has[u] = 1
    return tab, has


def _tables(page_table, page_bytes, owner_map, unit_bytes):
    if page_table is None:
        pt, npg = None, 0
    else:
        pt = np.ascontiguousarray(page_table, dtype=np.int32)
        npg = pt.size
    if owner_map is None:
        om, nu = None, 0
    else:
        assert owner_map.dtype == np.int32 and owner_map.flags.c_contiguous
        om, nu = owner_map, owner_map.size
    return pt, npg, om, nu


def _aad(aad, n):
    if aad is None:
        return None
    a = np.ascontiguousarray(aad, dtype=np.uint8).reshape(-1)
    assert a.size == 16 * n
    return a


def overlapping(segs, buf_bytes, page_table=None, page_bytes=0, owner_map=None, unit_bytes=0):
    """uint8[nseg]: 1 where a segment shares a byte with another segment of the table, or holds one
    byte of the buffer twice (paper sec. 4.3 rule step 3: distinct memory; sec. 3 step 4: one owner
    per byte).  Written out from the definition: count, for every byte of the buffer, how many
    times the valid segments of the table cover it; a segment overlaps when one of its bytes is
    covered more than once.  Segments with an invalid descriptor and empty segments take no part."""
    segs = np.ascontiguousarray(segs)
    n = segs.size
    pt, npg, om, nu = _tables(page_table, page_bytes, owner_map, unit_bytes)
    bad = np.zeros(max(n, 1), dtype=np.uint8)
    f = lib().gift_oracle_seg_bad_desc
    f.restype = C.c_int
    rc = f(C.c_uint64(buf_bytes), _p(segs), C.c_uint32(n), _p(pt) if pt is not None else None, C.c_uint32(npg),
           C.c_uint64(page_bytes), C.c_int(1 if om is not None else 0), C.c_uint32(nu), C.c_uint64(unit_bytes), _p(bad))
    if rc != 0:
        raise ValueError("oracle overlapping: bad call (%d)" % rc)

    def pieces(i):
        """(start, stop) byte ranges of segment i in the buffer."""
        ln = int(segs["len"][i])
        if pt is None:
            return [(int(segs["offset"][i]), int(segs["offset"][i]) + ln)]
        out = []
        for k in range(0, ln, page_bytes):
            base = int(pt[int(segs["page0"][i]) + k // page_bytes]) * page_bytes
            out.append((base, base + min(page_bytes, ln - k)))
        return out

    cover = np.zeros(buf_bytes, dtype=np.uint16)
    for i in range(n):
        if not bad[i]:
            for a, b in pieces(i):
                cover[a:b] += 1
    flags = np.zeros(n, dtype=np.uint8)
    for i in range(n):
        if not bad[i] and any((cover[a:b] > 1).any() for a, b in pieces(i)):
            flags[i] = 1
    return flags


def seg_encrypt(src, dst, segs, user_ids, keys, max_users, page_table=None, page_bytes=0,
                owner_map=None, unit_bytes=0, aad=None, check_overlap=False):
    """Encrypt every segment of `segs` from src into dst (may be the same array).

    Returns (tags uint8[nseg,16], status uint32[nseg]).
    """
    assert src.dtype == np.uint8 and dst.dtype == np.uint8 and src.size == dst.size
    segs = np.ascontiguousarray(segs)
    assert segs.dtype.itemsize == 40
    tab, has = _key_table(user_ids, keys, max_users)
    pt, npg, om, nu = _tables(page_table, page_bytes, owner_map, unit_bytes)
    n = segs.size
    tags = np.zeros((max(n, 1), 16), dtype=np.uint8)
    status = np.zeros(max(n, 1), dtype=np.uint32)
    ovl = overlapping(segs, src.size, page_table, page_bytes, owner_map, unit_bytes) if check_overlap and n else None
    f = lib().gift_oracle_seg_encrypt
    f.restype = C.c_int
    rc = f(_p(src), _p(dst), C.c_uint64(src.size), _p(segs), C.c_uint32(n),
           _p(pt) if pt is not None else None, C.c_uint32(npg), C.c_uint64(page_bytes),
           _p(om) if om is not None else None, C.c_uint32(nu), C.c_uint64(unit_bytes),
           _p(tab), _p(has), C.c_uint32(max_users), _p(tags), _p(status),
           _p(_aad(aad, n)) if aad is not None else None, _p(ovl) if ovl is not None else None)
    if rc != 0:
        raise ValueError("oracle seg_encrypt: bad call (%d)" % rc)
    return tags[:n], status[:n]


def seg_decrypt(src, dst, segs, tags, user_ids, keys, max_users, page_table=None, page_bytes=0,
                owner_map=None, unit_bytes=0, verify_only=False, aad=None, check_overlap=False):
    """Decrypt (or only verify) every segment; owner_map, when given, is updated in place.

    Returns status uint32[nseg].
    """
    assert src.dtype == np.uint8 and src.flags.c_contiguous
    if dst is None:
        dst = src
    segs = np.ascontiguousarray(segs)
    tab, has = _key_table(user_ids, keys, max_users)
    pt, npg, om, nu = _tables(page_table, page_bytes, owner_map, unit_bytes)
    n = segs.size
    tg = np.ascontiguousarray(tags, dtype=np.uint8).reshape(-1)
    if tg.size == 0:
        tg = np.zeros(16, dtype=np.uint8)
    status = np.zeros(max(n, 1), dtype=np.uint32)
    ovl = overlapping(segs, src.size, page_table, page_bytes, owner_map, unit_bytes) if check_overlap and n else None
    f = lib().gift_oracle_seg_decrypt
    f.restype = C.c_int
    rc = f(_p(src), _p(dst), C.c_uint64(src.size), _p(segs), C.c_uint32(n),
           _p(pt) if pt is not None else None, C.c_uint32(npg), C.c_uint64(page_bytes),
           _p(om) if om is not None else None, C.c_uint32(nu), C.c_uint64(unit_bytes),
           _p(tab), _p(has), C.c_uint32(max_users), _p(tg), _p(status), C.c_int(1 if verify_only else 0),
           _p(_aad(aad, n)) if aad is not None else None, _p(ovl) if ovl is not None else None)
    if rc != 0:
        raise ValueError("oracle seg_decrypt: bad call (%d)" % rc)
    return status[:n]


def tok_encrypt(tokens, nonces, owners, eos_token, user_ids, keys, max_users):
    """Token mode: (ciphertext uint8[n,16], status uint32[n])."""
    t = np.ascontiguousarray(tokens, dtype=np.uint64)
    nn = np.ascontiguousarray(nonces, dtype=np.uint64)
    o = np.ascontiguousarray(owners, dtype=np.int32)
    tab, has = _key_table(user_ids, keys, max_users)
    n = t.size
    out = np.zeros((max(n, 1), 16), dtype=np.uint8)
    status = np.zeros(max(n, 1), dtype=np.uint32)
    lib().gift_oracle_tok_encrypt(_p(t), _p(nn), _p(o), C.c_uint32(n), C.c_uint64(int(eos_token)), _p(tab), _p(has),
                                  C.c_uint32(max_users), _p(out), _p(status))
    return out[:n], status[:n]


def tok_decrypt(ct, owners, eos_token, user_ids, keys, max_users):
    """Token mode: (tokens uint64[n], nonces uint64[n], status uint32[n])."""
    c = np.ascontiguousarray(ct, dtype=np.uint8).reshape(-1, 16)
    o = np.ascontiguousarray(owners, dtype=np.int32)
    tab, has = _key_table(user_ids, keys, max_users)
    n = c.shape[0]
    toks = np.zeros(max(n, 1), dtype=np.uint64)
    nonces = np.zeros(max(n, 1), dtype=np.uint64)
    status = np.zeros(max(n, 1), dtype=np.uint32)
    lib().gift_oracle_tok_decrypt(_p(c), _p(o), C.c_uint32(n), C.c_uint64(int(eos_token)), _p(tab), _p(has),
                                  C.c_uint32(max_users), _p(toks), _p(nonces), _p(status))
    return toks[:n], nonces[:n], status[:n]


def threads() -> int:
    """Number of OpenMP threads the segment loops use."""
    try:
        omp = C.CDLL("libgomp.so.1")
        omp.omp_get_max_threads.restype = C.c_int
        return int(omp.omp_get_max_threads())
    except OSError:
        return len(os.sched_getaffinity(0))
