"""GPU parity: the CUDA path through the C-ABI against the CPU oracle, bit for bit.

Ciphertext, tags, status words and owner maps are unique results, so every comparison is
exact equality on the same seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import (dev, gpu_decrypt, gpu_encrypt, make_ctx, np_, oracle_decrypt, oracle_encrypt, st_)

pytestmark = pytest.mark.gpu

# default (tables of up to 1024 segments run as one fused launch), two AES tables, and the
# split form (plan / scan / cipher launches) forced for small tables too
VARIANTS = [0, binding.CTX_TWO_TABLES, binding.CTX_SPLIT_LAUNCH, binding.CTX_TWO_TABLES | binding.CTX_SPLIT_LAUNCH]


def _roundtrip_exact(w, flags=0, in_place=False):
    ctx = make_ctx(w, flags)
    src = dev(w.buf)
    dst = src if in_place else torch.full_like(src, 0xEE)
    tags, st = gpu_encrypt(ctx, w, src, None if in_place else dst)
    ref_ct = w.buf.copy() if in_place else np.full_like(w.buf, 0xEE)
    ref_tags, ref_st = oracle_encrypt(w, w.buf, ref_ct)
    assert np.array_equal(st_(st), ref_st)
    assert np.array_equal(np_(tags), ref_tags)
    assert np.array_equal(np_(dst), ref_ct)
    # decrypt back
    om_gpu = torch.full((w.owner_map.size,), 77, dtype=torch.int32, device="cuda") if w.owner_map is not None else None
    out = dst if in_place else torch.full_like(src, 0xEE)
    st2 = gpu_decrypt(ctx, w, dst, tags, None if in_place else out, owner_map=om_gpu)
    om_ref = np.full(w.owner_map.size, 77, dtype=np.int32) if w.owner_map is not None else None
    ref_pt = ref_ct.copy() if in_place else np.full_like(w.buf, 0xEE)
    ref_st2 = oracle_decrypt(w, ref_ct, ref_pt, ref_tags, owner_map=om_ref)
    assert np.array_equal(st_(st2), ref_st2) and not ref_st2.any()
    assert np.array_equal(np_(out), ref_pt)
    if om_ref is not None:
        assert np.array_equal(np_(om_gpu), om_ref)
    # verify-only agrees and writes nothing
    st3 = gpu_decrypt(ctx, w, dev(ref_ct), tags, verify_only=True)
    assert not st_(st3).any()
    ctx.close()
    return ref_ct, ref_tags


@pytest.mark.parametrize("flags", VARIANTS)
def test_config1_tiny_round_trip(flags):
    w = W.config1()
    ref_ct, _ = _roundtrip_exact(w, flags)
    for salt in (1, 2):
        _roundtrip_exact(W.config1(seed_salt=salt), flags)


@pytest.mark.parametrize("flags", VARIANTS)
def test_config2_decode_rows(flags):
    _roundtrip_exact(W.config2(), flags)


def test_config3_kv_handoff_two_layers():
    _roundtrip_exact(W.config3(layers=2))


def test_config4_zipf_in_place():
    w = W.config4()
    _roundtrip_exact(w, in_place=True)


def test_lengths_ragged_and_empty():
    """Every length 0..600 plus block and run boundaries, back to back at 16-byte aligned offsets."""
    rng = np.random.default_rng(11)
    lens = list(range(0, 600)) + [4095, 4096, 4097, 65535, 65536, 65537, 70000, 262144 + 5]
    offs, o = [], 0
    for n in lens:
        offs.append(o)
        o += (n + 15) // 16 * 16 + 16 * int(rng.integers(0, 3))
    segs = np.zeros(len(lens), dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, 5, size=len(lens))
    segs["offset"] = offs
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * len(lens)), dtype=np.uint8).reshape(-1, 12)
    ids, keys = np.arange(5, dtype=np.int32), np.frombuffer(rng.bytes(80), dtype=np.uint8).reshape(5, 16)
    buf = np.frombuffer(rng.bytes(o + 64), dtype=np.uint8).copy()
    w = W.Workload("ragged", ids, keys, 5, buf, buf.size, segs)
    for flags in VARIANTS[:3]:
        _roundtrip_exact(w, flags)


def test_empty_call_and_argument_errors():
    w = W.config1()
    ctx = make_ctx(w)
    src = dev(w.buf)
    tags = torch.zeros((1, 16), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.seg_encrypt(src, src, torch.zeros(40, dtype=torch.uint8, device="cuda"), 0, tags, st)    # nseg = 0: no-op
    with pytest.raises(binding.GiftError) as e:
        ctx.seg_encrypt(src[1:], src[1:], torch.zeros(40, dtype=torch.uint8, device="cuda"), 1, tags, st)
    assert e.value.code == binding.E_ALIGN
    with pytest.raises(binding.GiftError) as e:
        ctx.set_keys(np.array([99], dtype=np.int32), np.zeros((1, 16), dtype=np.uint8))
    assert e.value.code == binding.E_RANGE
    with pytest.raises(binding.GiftError):
        binding.Ctx(4, 0, 0x40)                   # no such flag
    assert binding.version() >= 200 and ctx.launch_count() > 0
    ctx.close()


def test_large_segments_many_runs_and_high_powers():
    """One 64 MiB segment (the largest the workloads draw), one of 3 MiB + 7 and small ones:
    exercises the cross-run combine and exponents up to 2^22."""
    rng = np.random.default_rng(12)
    lens = [64 << 20, (3 << 20) + 7, 16, 1 << 20, 100]
    offs = np.concatenate([[0], np.cumsum([(n + 15) // 16 * 16 for n in lens])[:-1]])
    total = int(offs[-1]) + 112
    segs = np.zeros(len(lens), dtype=W.SEG_DTYPE)
    segs["owner"] = [0, 1, 2, 1, 0]
    segs["offset"] = offs
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * len(lens)), dtype=np.uint8).reshape(-1, 12)
    ids, keys = np.arange(3, dtype=np.int32), np.frombuffer(rng.bytes(48), dtype=np.uint8).reshape(3, 16)
    buf = np.frombuffer(rng.bytes(total), dtype=np.uint8).copy()
    w = W.Workload("large", ids, keys, 3, buf, buf.size, segs)
    _roundtrip_exact(w, in_place=True)


def test_one_segment_beyond_2_pow_24_blocks_uses_the_top_power_level():
    """256 MiB + 4 KiB + 5 bytes in one segment: the first blocks' exponents exceed 2^24, the
    fourth digit of the power table, which no workload of the paper's sizes reaches."""
    rng = np.random.default_rng(13)
    n = (256 << 20) + 4096 + 5
    segs = np.zeros(1, dtype=W.SEG_DTYPE)
    segs["owner"], segs["offset"], segs["len"] = 1, 0, n
    segs["nonce"] = np.frombuffer(rng.bytes(12), dtype=np.uint8).reshape(1, 12)
    ids, keys = np.arange(2, dtype=np.int32), np.frombuffer(rng.bytes(32), dtype=np.uint8).reshape(2, 16)
    buf = np.frombuffer(rng.bytes((n + 15) // 16 * 16), dtype=np.uint8).copy()
    w = W.Workload("huge", ids, keys, 2, buf, buf.size, segs)
    ctx = make_ctx(w)
    d = dev(w.buf)
    tags, st = gpu_encrypt(ctx, w, d)
    ref_ct = w.buf.copy()
    ref_tags, ref_st = oracle_encrypt(w, w.buf, ref_ct)            # one oracle pass: about 20 s on one core
    assert not ref_st.any() and not st_(st).any()
    assert np.array_equal(np_(tags), ref_tags)
    assert np.array_equal(np_(d), ref_ct)
    st2 = gpu_decrypt(ctx, w, d, tags)                             # and back, against the original bytes
    assert not st_(st2).any() and np.array_equal(np_(d), w.buf)
    ctx.close()


@pytest.mark.parametrize("flags", [0, binding.CTX_SPLIT_LAUNCH])
def test_export_status_rules_match_oracle(flags):
    w = W.config2(n_users=8, vocab=64)
    om = w.owner_map.copy()
    om[1], om[2], om[3], om[4] = 5, binding.OWNER_NONE, binding.OWNER_PARAM, binding.OWNER_CONFLICT
    segs = w.segs.copy()
    segs["offset"][5] += 8
    segs["len"][6] = w.buf.size
    segs["flags"][0] = 0
    ids, keys = w.user_ids[:7], w.keys[:7]
    ctx = make_ctx(w, flags, user_ids=ids, keys=keys)
    src = dev(w.buf)
    dst = torch.full_like(src, 0xEE)
    tags, st = gpu_encrypt(ctx, w, src, dst, segs=segs, owner_map=om)
    ref = np.full_like(w.buf, 0xEE)
    ref_tags, ref_st = oracle_encrypt(w, w.buf, ref, segs=segs, owner_map=om, user_ids=ids, keys=keys)
    assert ref_st.tolist() == [0, 2, 4, 2, 4, 16, 16, 8]
    assert np.array_equal(st_(st), ref_st) and np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(dst), ref)
    # mixed labels inside one multi-unit segment, reserved flag, paged out-of-range entry
    w4 = W.config4(total_bytes=2 << 20, cap_bytes=1 << 20, n_users=8)
    om4 = w4.owner_map.copy()
    big = int(np.argmax(w4.segs["len"]))
    pages = w4.page_table[int(w4.segs["page0"][big]): int(w4.segs["page0"][big]) + int(w4.extra["npages"][big])]
    if len(pages) > 1:
        om4[pages[-1]] = (int(w4.segs["owner"][big]) + 1) % 8
    segs4 = w4.segs.copy()
    segs4["flags"][0] = 1
    pt4 = w4.page_table.copy()
    victim = 1 if big != 1 else 2
    pt4[int(segs4["page0"][victim])] = len(pt4) + 5
    w4.page_table = pt4
    ctx4 = make_ctx(w4, flags)
    src4 = dev(w4.buf)
    tags4, st4 = gpu_encrypt(ctx4, w4, src4, None, segs=segs4, owner_map=om4)
    ref4 = w4.buf.copy()
    ref_tags4, ref_st4 = oracle_encrypt(w4, ref4, ref4, segs=segs4, owner_map=om4)
    assert ref_st4[0] == 16 and (int(segs4["len"][victim]) == 0 or ref_st4[victim] == 16)
    assert np.array_equal(st_(st4), ref_st4) and np.array_equal(np_(tags4), ref_tags4)
    assert np.array_equal(np_(src4), ref4)
    ctx.close()
    ctx4.close()


@pytest.mark.parametrize("flags", [0, binding.CTX_SPLIT_LAUNCH])
def test_import_failures_zero_fill_and_unown(flags):
    w = W.config2(n_users=12, vocab=500)
    ctx = make_ctx(w, flags, user_ids=w.user_ids[:11], keys=w.keys[:11])       # user 11 has no key
    ct = w.buf.copy()
    ref_tags, _ = oracle_encrypt(w, w.buf, ct, owner_map=None)
    bad_ct = ct.copy()
    bad_ct[int(w.segs["offset"][1]) + 17] ^= 0x04
    bad_ct[int(w.segs["offset"][2]) + int(w.segs["len"][2]) - 1] ^= 0x80       # last byte of a partial block
    bad_tags = ref_tags.copy()
    bad_tags[3, 9] ^= 0x80
    segs = w.segs.copy()
    segs["owner"][4] = 0                      # claims another user's key
    segs["nonce"][5, 0] ^= 1                  # wrong nonce
    om_ref = np.full(12, 99, dtype=np.int32)
    ref = np.full_like(ct, 0xEE)
    ids, keys = w.user_ids[:11], w.keys[:11]
    from oracle import gcm
    ref_st = gcm.seg_decrypt(bad_ct, ref, segs, bad_tags, ids, keys, w.max_users, None, 0, om_ref, w.unit_bytes)
    assert ref_st.tolist() == [0, 1, 1, 1, 1, 1, 0, 0, 0, 0, 0, 8]
    om = torch.full((12,), 99, dtype=torch.int32, device="cuda")
    out = torch.full((ct.size,), 0xEE, dtype=torch.uint8, device="cuda")
    st = gpu_decrypt(ctx, w, dev(bad_ct), dev(bad_tags), out, segs=segs, owner_map=om)
    assert np.array_equal(st_(st), ref_st) and np.array_equal(np_(out), ref) and np.array_equal(np_(om), om_ref)
    st = gpu_decrypt(ctx, w, dev(bad_ct), dev(bad_tags), segs=segs, verify_only=True)
    assert np.array_equal(st_(st), ref_st)
    ctx.close()


def test_every_single_bit_flip_is_detected():
    rng = np.random.default_rng(13)
    key = np.frombuffer(rng.bytes(16), dtype=np.uint8).reshape(1, 16)
    n = 64 * 8 + 128
    segs = np.zeros(n, dtype=W.SEG_DTYPE)
    segs["offset"] = np.arange(n) * 64
    segs["len"] = 64
    segs["nonce"] = np.frombuffer(rng.bytes(12), dtype=np.uint8)
    pt = np.tile(np.frombuffer(rng.bytes(64), dtype=np.uint8), n)
    w = W.Workload("flips", np.zeros(1, dtype=np.int32), key, 1, pt, pt.size, segs)
    ctx = make_ctx(w)
    buf = dev(pt)
    tags, st = gpu_encrypt(ctx, w, buf)
    assert not st_(st).any()
    ct, tg = np_(buf).copy(), np_(tags).copy()
    for i in range(64 * 8):
        ct[i * 64 + i // 8] ^= 1 << (i % 8)
    for i in range(128):
        tg[64 * 8 + i, i // 8] ^= 1 << (i % 8)
    st = gpu_decrypt(ctx, w, dev(ct), dev(tg), verify_only=True)
    assert (st_(st) == 1).all()
    ctx.close()


def test_key_change_touches_only_that_user_and_clear_keys():
    w = W.config1()
    ctx = make_ctx(w)
    a = dev(w.buf)
    tags_a, _ = gpu_encrypt(ctx, w, a)
    keys2 = w.keys.copy()
    keys2[3] ^= 0x5A
    ctx.set_keys(np.array([3], dtype=np.int32), keys2[3:4])
    b = dev(w.buf)
    tags_b, _ = gpu_encrypt(ctx, w, b)
    a, b, ta, tb = np_(a), np_(b), np_(tags_a), np_(tags_b)
    for i, s in enumerate(w.segs):
        o, n = int(s["offset"]), int(s["len"])
        same = np.array_equal(a[o:o + n], b[o:o + n]) and np.array_equal(ta[i], tb[i])
        assert same == (int(s["owner"]) != 3)
    ctx.clear_keys(np.array([2], dtype=np.int32))
    c = dev(w.buf)
    _, st = gpu_encrypt(ctx, w, c)
    assert st_(st).tolist() == [0, 0, 8, 0, 0, 0, 0, 0]
    ctx.close()


def test_bound_aad_matches_oracle_and_detects_a_changed_role():
    from oracle import gcm
    for w in (W.config1(), W.config4(total_bytes=6 << 20, cap_bytes=2 << 20, n_users=8)):
        n = len(w.segs)
        rng = np.random.default_rng(31)
        aad = np.frombuffer(rng.bytes(16 * n), dtype=np.uint8).reshape(n, 16).copy()
        ctx = make_ctx(w)
        d_aad = dev(aad)
        ctx.bind_aad(d_aad)
        buf = dev(w.buf)
        tags, st = gpu_encrypt(ctx, w, buf)
        ref = w.buf.copy()
        ref_tags, ref_st = gcm.seg_encrypt(ref, ref, w.segs, w.user_ids, w.keys, w.max_users, w.page_table,
                                           w.page_bytes, w.owner_map, w.unit_bytes, aad=aad)
        assert np.array_equal(st_(st), ref_st) and np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(buf), ref)
        st = gpu_decrypt(ctx, w, buf, tags, verify_only=True)
        assert not st_(st).any()
        moved = aad.copy()
        moved[n // 2, 5] ^= 0x10
        ctx.bind_aad(dev(moved))
        st = gpu_decrypt(ctx, w, buf, tags, verify_only=True)
        expect = gcm.seg_decrypt(ref, ref.copy(), w.segs, ref_tags, w.user_ids, w.keys, w.max_users, w.page_table,
                                 w.page_bytes, verify_only=True, aad=moved)
        assert np.array_equal(st_(st), expect) and expect[n // 2] == 1 and expect.sum() == 1
        if n > 2:                                # a table longer than the bound array is refused before any launch
            ctx.bind_aad(dev(aad[: n - 1].copy()))
            with pytest.raises(binding.GiftError) as e:
                gpu_encrypt(ctx, w, dev(w.buf))
            assert e.value.code == binding.E_RANGE
        ctx.bind_aad(None)                       # unbound again: plain tags
        buf2 = dev(w.buf)
        tags2, _ = gpu_encrypt(ctx, w, buf2)
        plain_tags, _ = oracle_encrypt(w, w.buf.copy(), w.buf.copy())
        assert np.array_equal(np_(tags2), plain_tags)
        ctx.close()
