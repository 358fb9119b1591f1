"""Pins for the oracle's segment semantics (export / import of ownership segments).

The cipher itself is pinned in test_oracle_crypto.py; here every segment result is
re-derived with OpenSSL on bytes gathered by the test, and the status / fallback rules
are checked against hand-built cases.
"""
import numpy as np
from cryptography.hazmat.primitives.ciphers.aead import AESGCM

from oracle import gcm
from paper_2608_25431_b200 import workloads as W


def _gather(w, buf, i):
    s = w.segs[i]
    n = int(s["len"])
    if w.page_table is None:
        o = int(s["offset"])
        return buf[o: o + n].tobytes()
    out = bytearray()
    pb = w.page_bytes
    for k in range(0, n, pb):
        page = int(w.page_table[int(s["page0"]) + k // pb])
        out += buf[page * pb: page * pb + min(pb, n - k)].tobytes()
    return bytes(out)


def _enc(w, src, dst, **kw):
    return gcm.seg_encrypt(src, dst, kw.pop("segs", w.segs), w.user_ids, kw.pop("keys", w.keys),
                           w.max_users, w.page_table, w.page_bytes,
                           kw.pop("owner_map", w.owner_map), w.unit_bytes)


def _check_against_openssl(w, ct, tags, idx):
    for i in idx:
        s = w.segs[i]
        ref = AESGCM(w.keys[int(s["owner"])].tobytes()).encrypt(s["nonce"].tobytes(), _gather(w, w.buf, i), None)
        assert _gather(w, ct, i) + tags[i].tobytes() == ref, i


def test_flat_segments_match_openssl_and_round_trip():
    w = W.config1()
    ct = w.buf.copy()
    tags, st = _enc(w, w.buf, ct)
    assert not st.any()
    _check_against_openssl(w, ct, tags, range(len(w.segs)))
    pt = ct.copy()
    st = gcm.seg_decrypt(ct, pt, w.segs, tags, w.user_ids, w.keys, w.max_users)
    assert not st.any() and np.array_equal(pt, w.buf)


def test_partial_last_block_rows():
    w = W.config2(n_users=6, vocab=100)
    ct = w.buf.copy()
    tags, st = _enc(w, w.buf, ct)
    assert not st.any()
    _check_against_openssl(w, ct, tags, range(6))
    rows_pt = w.buf.reshape(6, -1)
    rows_ct = ct.reshape(6, -1)
    assert np.array_equal(rows_pt[:, 204:], rows_ct[:, 204:])      # pad bytes outside segments untouched


def test_paged_segments_match_openssl_in_place():
    w = W.config4(total_bytes=3 << 20, cap_bytes=1 << 20, n_users=16)
    ct = w.buf.copy()
    tags, st = _enc(w, ct, ct)                                     # in place
    assert not st.any()
    big = np.argsort(w.segs["len"])[-3:]
    some = np.random.default_rng(0).choice(len(w.segs), size=min(20, len(w.segs)), replace=False)
    _check_against_openssl(w, ct, tags, list(big) + list(some))
    st = gcm.seg_decrypt(ct, ct, w.segs, tags, w.user_ids, w.keys, w.max_users, w.page_table, w.page_bytes)
    assert not st.any() and np.array_equal(ct, w.buf)


def test_table_order_is_irrelevant():
    w = W.config1()
    ct = w.buf.copy()
    tags, _ = _enc(w, w.buf, ct)
    perm = np.random.default_rng(1).permutation(len(w.segs))
    ct2 = w.buf.copy()
    tags2, _ = _enc(w, w.buf, ct2, segs=w.segs[perm])
    assert np.array_equal(ct, ct2) and np.array_equal(tags[perm], tags2)


def test_changing_one_users_key_touches_only_that_user():
    w = W.config1()
    ct = w.buf.copy()
    tags, _ = _enc(w, w.buf, ct)
    keys2 = w.keys.copy()
    keys2[3] ^= 0x5A
    ct2 = w.buf.copy()
    tags2, _ = _enc(w, w.buf, ct2, keys=keys2)
    for i, s in enumerate(w.segs):
        o, n = int(s["offset"]), int(s["len"])
        same = np.array_equal(ct[o:o + n], ct2[o:o + n]) and np.array_equal(tags[i], tags2[i])
        assert same == (int(s["owner"]) != 3)


def test_export_status_rules():
    w = W.config2(n_users=8, vocab=64)
    ST = gcm
    om = w.owner_map.copy()
    om[1] = 5                   # another user's label on row 1
    om[2] = gcm.OWNER_NONE      # unowned
    om[3] = gcm.OWNER_PARAM     # parameters can never be exported
    om[4] = gcm.OWNER_CONFLICT
    segs = w.segs.copy()
    segs["offset"][5] += 8      # misaligned
    segs["len"][6] = w.buf.size # out of range
    ids, keys = w.user_ids[:7], w.keys[:7]          # user 7 has no key
    dst = np.full_like(w.buf, 0xEE)
    tags, st = gcm.seg_encrypt(w.buf, dst, segs, ids, keys, w.max_users, None, 0, om, w.unit_bytes)
    assert st.tolist() == [0, ST.ST_OWNER_MISMATCH, ST.ST_UNOWNED, ST.ST_OWNER_MISMATCH, ST.ST_UNOWNED,
                           ST.ST_BAD_DESC, ST.ST_BAD_DESC, ST.ST_NO_KEY]
    rows = dst.reshape(8, -1)
    assert (rows[1:] == 0xEE).all() and not tags[1:].any()          # failed: bytes as they were, zero tag
    assert (rows[0, int(segs["len"][0]):] == 0xEE).all() and tags[0].any()
    # a claimed owner that disagrees with a uniform map is a mismatch too
    segs = w.segs.copy()
    segs["owner"][0] = 1
    _, st = gcm.seg_encrypt(w.buf, dst, segs, w.user_ids, w.keys, w.max_users, None, 0, w.owner_map, w.unit_bytes)
    assert st[0] == ST.ST_OWNER_MISMATCH and not st[1:].any()


def test_import_failure_zero_fills_and_unowns():
    w = W.config2(n_users=6, vocab=64)
    ct = w.buf.copy()
    tags, _ = _enc(w, w.buf, ct)
    bad_ct = ct.copy()
    bad_ct[int(w.segs["offset"][1]) + 17] ^= 0x04                   # flipped ciphertext bit
    bad_tags = tags.copy()
    bad_tags[2, 9] ^= 0x80                                           # flipped tag bit
    segs = w.segs.copy()
    segs["owner"][3] = 0                                             # claims another user's key
    om = np.full(6, 99, dtype=np.int32)
    out = np.full_like(ct, 0xEE)
    st = gcm.seg_decrypt(bad_ct, out, segs, bad_tags, w.user_ids, w.keys, w.max_users,
                         owner_map=om, unit_bytes=w.unit_bytes)
    assert st.tolist() == [0, 1, 1, 1, 0, 0]
    rows, ref = out.reshape(6, -1), w.buf.reshape(6, -1)
    n = int(w.segs["len"][0])
    for i in range(6):
        if st[i]:
            assert not rows[i, :n].any()
        else:
            assert np.array_equal(rows[i, :n], ref[i, :n])
        assert (rows[i, n:] == 0xEE).all()
    assert om.tolist() == [0, gcm.OWNER_NONE, gcm.OWNER_NONE, gcm.OWNER_NONE, 4, 5]
    # verify-only: same statuses, nothing written
    out2 = np.full_like(ct, 0xEE)
    om2 = np.full(6, 99, dtype=np.int32)
    st2 = gcm.seg_decrypt(bad_ct, out2, segs, bad_tags, w.user_ids, w.keys, w.max_users,
                          owner_map=om2, unit_bytes=w.unit_bytes, verify_only=True)
    assert st2.tolist() == st.tolist() and (out2 == 0xEE).all() and (om2 == 99).all()


def test_empty_segment_tag_is_encrypted_j0():
    w = W.config1()
    segs = w.segs[:1].copy()
    segs["len"] = 0
    tags, st = gcm.seg_encrypt(w.buf, w.buf.copy(), segs, w.user_ids, w.keys, w.max_users)
    j0 = segs["nonce"][0].tobytes() + b"\x00\x00\x00\x01"
    assert st[0] == 0 and tags[0].tobytes() == gcm.aes128_encrypt_block(w.keys[0], j0)


def test_workload_generators_are_seeded():
    a, b = W.config4(total_bytes=1 << 20, cap_bytes=1 << 18, n_users=8), W.config4(total_bytes=1 << 20, cap_bytes=1 << 18, n_users=8)
    assert np.array_equal(a.buf, b.buf) and np.array_equal(a.segs, b.segs)
    w5 = W.config5(layers=1, n_users=8, chunk_tokens=4, fill=False)
    assert len(w5.segs) == 8 and w5.buf_bytes == 20 * W.KV_TOKEN_BYTES
    w3 = W.config3(layers=1, n_users=2, min_len=17, max_len=40, fill=True)
    assert w3.buf.size == len(w3.segs) * W.KV_PAGE_BYTES
    assert sorted(w3.page_table.tolist()) == list(range(len(w3.segs)))


def test_segment_aad_matches_openssl_and_binds_the_tag():
    w = W.config1()
    rng = np.random.default_rng(3)
    aad = np.frombuffer(rng.bytes(16 * len(w.segs)), dtype=np.uint8).reshape(-1, 16)
    ct = w.buf.copy()
    tags, st = gcm.seg_encrypt(w.buf, ct, w.segs, w.user_ids, w.keys, w.max_users, aad=aad)
    assert not st.any()
    for i, s in enumerate(w.segs):
        o, n = int(s["offset"]), int(s["len"])
        ref = AESGCM(w.keys[int(s["owner"])].tobytes()).encrypt(s["nonce"].tobytes(), w.buf[o:o + n].tobytes(),
                                                                aad[i].tobytes())
        assert ct[o:o + n].tobytes() + tags[i].tobytes() == ref
    plain_tags, _ = gcm.seg_encrypt(w.buf, w.buf.copy(), w.segs, w.user_ids, w.keys, w.max_users)
    assert not np.array_equal(tags, plain_tags)                      # the data is authenticated, not ignored
    st = gcm.seg_decrypt(ct, ct.copy(), w.segs, tags, w.user_ids, w.keys, w.max_users, aad=aad)
    assert not st.any()
    moved = aad.copy()
    moved[2, 0] ^= 1                                                 # presented in another role
    st = gcm.seg_decrypt(ct, ct.copy(), w.segs, tags, w.user_ids, w.keys, w.max_users, aad=moved)
    assert st.tolist() == [0, 0, 1, 0, 0, 0, 0, 0]


def _seg_table(rows):
    """rows: (owner, offset, len, page0)"""
    t = np.zeros(len(rows), dtype=W.SEG_DTYPE)
    for i, (owner, off, ln, page0) in enumerate(rows):
        t[i]["owner"], t[i]["offset"], t[i]["len"], t[i]["page0"] = owner, off, ln, page0
        t[i]["nonce"] = np.arange(12, dtype=np.uint8) + i
    return t


def test_overlap_definition_on_hand_built_tables():
    """Which segments share bytes is written down by hand for every table below."""
    # flat, 256-byte buffer
    flat = _seg_table([
        (0, 0, 32, 0),        # 0: [0, 32)    overlaps 1
        (1, 16, 32, 0),       # 1: [16, 48)   overlaps 0 and 2
        (2, 32, 48, 0),       # 2: [32, 80)   overlaps 1 and contains 3
        (3, 48, 16, 0),       # 3: [48, 64)   inside 2
        (0, 80, 16, 0),       # 4: [80, 96)   touches 2, shares no byte
        (1, 96, 0, 0),        # 5: empty, at the start of 6: never overlaps
        (2, 96, 20, 0),       # 6: [96, 116)  alone
        (3, 100, 16, 0),      # 7: offset not a multiple of 16: bad descriptor, takes no part (would hit 6)
        (0, 128, 40, 0),      # 8: [128, 168) identical to 9
        (1, 128, 40, 0),      # 9
        (2, 240, 32, 0),      # 10: runs past the buffer: bad descriptor
        (3, 240, 16, 0),      # 11: [240, 256) alone (10 does not count)
    ])
    assert gcm.overlapping(flat, 256).tolist() == [1, 1, 1, 1, 0, 0, 0, 0, 1, 1, 0, 0]
    # paged, 8 physical pages of 64 bytes; chains listed in the page table
    table = np.array([0, 1,      # seg 0: pages 0, 1
                      2, 1,      # seg 1: pages 2, 1   (page 1 shared with seg 0)
                      3,         # seg 2: page 3       alone
                      4, 4,      # seg 3: page 4 twice (overlaps itself)
                      5, 6,      # seg 4: 70 bytes: page 5 and six bytes of page 6
                      6,         # seg 5: page 6       (shares its first bytes with seg 4)
                      7, 9,      # seg 6: page 9 does not exist: bad descriptor
                      7], dtype=np.int32)   # seg 7: page 7 alone (seg 6 does not count)
    paged = _seg_table([(0, 0, 128, 0), (1, 0, 100, 2), (2, 0, 64, 4), (3, 0, 128, 5), (0, 0, 70, 7),
                        (1, 0, 10, 9), (2, 0, 128, 10), (3, 0, 5, 12)])
    assert gcm.overlapping(paged, 8 * 64, table, 64).tolist() == [1, 1, 0, 1, 1, 1, 0, 0]


def test_overlapping_segments_are_refused_untouched():
    rng = np.random.default_rng(5)
    ids = np.arange(4, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(64), dtype=np.uint8).reshape(4, 16)
    segs = _seg_table([(0, 0, 32, 0), (1, 16, 32, 0), (2, 64, 32, 0), (3, 96, 16, 0)])
    buf = np.frombuffer(rng.bytes(128), dtype=np.uint8).copy()
    out = buf.copy()
    tags, st = gcm.seg_encrypt(buf, out, segs, ids, keys, 4, check_overlap=True)
    assert st.tolist() == [32, 32, 0, 0]
    assert np.array_equal(out[:64], buf[:64]) and not tags[:2].any()          # refused: bytes as they were, tag zero
    ct, tag = gcm.gcm_encrypt(keys[2], segs["nonce"][2], buf[64:96])
    assert out[64:96].tobytes() == ct and tags[2].tobytes() == tag
    # without the check the same table is taken as it comes (undefined mix, not tested); decrypt side:
    om = np.full(8, 7, dtype=np.int32)
    back = out.copy()
    st = gcm.seg_decrypt(out, back, segs, tags, ids, keys, 4, owner_map=om, unit_bytes=16, check_overlap=True)
    assert st.tolist() == [32, 32, 0, 0]
    assert np.array_equal(back[:64], out[:64]) and np.array_equal(back[64:112], buf[64:112])
    assert om.tolist() == [7, 7, 7, 7, 2, 2, 3, 7]                            # refused segments leave labels alone
