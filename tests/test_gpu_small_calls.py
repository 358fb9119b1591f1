"""The single-launch form that tables of at most 1024 segments take, against the oracle.

A small call (the rows of a decode step, paper sec. 3 steps 5-6) runs as one kernel: every
CTA recomputes the work split and every warp checks the segments it touches itself.  These
tests cross the 1024-segment threshold, mix refused segments in, alternate with the
three-launch form on the same context (the hash accumulators and tickets must be back at
zero after every call), and compare everything with the oracle bit for bit."""
import numpy as np
import pytest
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import dev, gpu_decrypt, gpu_encrypt, make_ctx, np_, st_

pytestmark = pytest.mark.gpu


def _flat(rng, nseg, n_users, max_len, unit=256):
    lens = rng.integers(0, max_len + 1, size=nseg)
    lens[rng.choice(nseg, size=max(1, nseg // 50), replace=False)] = 0
    starts, o = [], 0
    for n in lens:
        o = (o + unit - 1) // unit * unit
        starts.append(o)
        o += int(n)
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, n_users, size=nseg)
    segs["offset"] = starts
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * nseg), dtype=np.uint8).reshape(nseg, 12)
    total = (o + unit) // unit * unit
    buf = np.frombuffer(rng.bytes(total), dtype=np.uint8).copy()
    om = np.full(total // unit, binding.OWNER_NONE, dtype=np.int32)
    for i in range(nseg):
        if lens[i]:
            om[starts[i] // unit: (starts[i] + int(lens[i]) + unit - 1) // unit] = segs["owner"][i]
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    return W.Workload("small_flat", ids, keys, n_users, buf, buf.size, segs, owner_map=om, unit_bytes=unit)


def _check_export_and_import(ctx, w, rng, have=None):
    have = w.user_ids if have is None else have
    keys = w.keys[: len(have)]
    d = dev(w.buf)
    tags, st = gpu_encrypt(ctx, w, d)
    ref = w.buf.copy()
    ref_tags, ref_st = gcm.seg_encrypt(ref, ref, w.segs, have, keys, w.max_users, w.page_table, w.page_bytes,
                                       w.owner_map, w.unit_bytes)
    assert np.array_equal(st_(st), ref_st)
    assert np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(d), ref)
    bad = ref.copy()
    for _ in range(3):
        bad[int(rng.integers(0, bad.size))] ^= 1 << int(rng.integers(0, 8))
    om_ref = np.full(w.owner_map.size, 55, dtype=np.int32)
    out_ref = bad.copy()
    st_ref = gcm.seg_decrypt(out_ref, out_ref, w.segs, ref_tags, have, keys, w.max_users, w.page_table, w.page_bytes,
                             om_ref, w.unit_bytes)
    om = torch.full((w.owner_map.size,), 55, dtype=torch.int32, device="cuda")
    d_bad = dev(bad)
    st2 = gpu_decrypt(ctx, w, d_bad, dev(ref_tags), owner_map=om)
    assert np.array_equal(st_(st2), st_ref)
    assert np.array_equal(np_(d_bad), out_ref) and np.array_equal(np_(om), om_ref)
    st3 = gpu_decrypt(ctx, w, dev(bad), dev(ref_tags), verify_only=True)
    assert np.array_equal(st_(st3), st_ref)


@pytest.mark.parametrize("nseg", [1, 2, 31, 32, 33, 257, 1023, 1024, 1025, 1100])
def test_tables_around_the_threshold_match_oracle(nseg):
    rng = np.random.default_rng(W.SEED_BASE + 300 + nseg)
    w = _flat(rng, nseg, 6, 9000 if nseg > 300 else 70000)
    # a few refused segments: a foreign unit, an unowned unit, a bad offset, a user without a key
    om, segs = w.owner_map, w.segs
    nz = np.nonzero(segs["len"] > 0)[0]
    if len(nz) >= 4:
        a, b, c, d_ = nz[0], nz[len(nz) // 3], nz[len(nz) // 2], nz[-1]
        om[int(segs["offset"][a]) // w.unit_bytes] = (int(segs["owner"][a]) + 1) % 6
        om[int(segs["offset"][b]) // w.unit_bytes] = binding.OWNER_NONE
        segs["offset"][c] += 8
        segs["owner"][d_] = 5
    ctx = make_ctx(w, user_ids=w.user_ids[:5], keys=w.keys[:5])         # user 5 has no key
    for _ in range(2):                                                  # twice: scratch must be clean again
        _check_export_and_import(ctx, w, rng, have=w.user_ids[:5])
    ctx.close()


def test_fused_and_split_calls_alternate_on_one_context():
    """A 64 MiB segment is cut into many pieces (accumulator and ticket in use) in a table of 3
    segments (fused form); then 3 000 segments (split form); then the small table again."""
    rng = np.random.default_rng(W.SEED_BASE + 350)
    n_users = 4
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()

    def table(lens):
        offs = np.concatenate([[0], np.cumsum([(n + 15) // 16 * 16 for n in lens])[:-1]])
        segs = np.zeros(len(lens), dtype=W.SEG_DTYPE)
        segs["owner"] = rng.integers(0, n_users, size=len(lens))
        segs["offset"] = offs
        segs["len"] = lens
        segs["nonce"] = np.frombuffer(rng.bytes(12 * len(lens)), dtype=np.uint8).reshape(-1, 12)
        total = int(offs[-1]) + (int(lens[-1]) + 15) // 16 * 16 + 16
        buf = rng.integers(0, 256, size=total, dtype=np.uint8)
        return W.Workload("alt", ids, keys, n_users, buf, buf.size, segs)

    small = table([(32 << 20) + 3, 5, (8 << 20)])
    many = table(list(rng.integers(0, 40000, size=3000)))
    ctx = make_ctx(small)
    for w in (small, many, small, small, many):
        d = dev(w.buf)
        tags, st = gpu_encrypt(ctx, w, d)
        ref = w.buf.copy()
        ref_tags, ref_st = gcm.seg_encrypt(ref, ref, w.segs, ids, keys, n_users)
        assert not st_(st).any() and not ref_st.any()
        assert np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(d), ref)
        st2 = gpu_decrypt(ctx, w, d, tags)
        assert not st_(st2).any() and np.array_equal(np_(d), w.buf)
    ctx.close()


def test_paged_small_table_with_bad_page_entries_and_labels():
    w = W.config4(total_bytes=12 << 20, cap_bytes=4 << 20, n_users=8)
    assert len(w.segs) <= 1024
    rng = np.random.default_rng(W.SEED_BASE + 360)
    pt = w.page_table.copy()
    lens = w.segs["len"]
    multi = [i for i in range(len(w.segs)) if lens[i] > 2 * w.page_bytes]
    pt[int(w.segs["page0"][multi[0]]) + 1] = -4                         # a bad entry in the middle of a chain
    w.page_table = pt
    om = w.owner_map
    om[pt[int(w.segs["page0"][multi[1]]) + 2]] = binding.OWNER_CONFLICT  # a conflicted page deep in a chain
    ctx = make_ctx(w)
    _check_export_and_import(ctx, w, rng)
    ctx.close()


def test_many_short_segments_take_the_peeled_large_table_kernel():
    """6 000 flat segments of at most 3 KiB in a buffer that leaves less than 4 KiB per segment: the
    three-launch form with the kernel that peels the first row of every piece."""
    rng = np.random.default_rng(W.SEED_BASE + 370)
    nseg, n_users = 6000, 5
    lens = rng.integers(0, 3073, size=nseg)
    offs = np.concatenate([[0], np.cumsum((lens + 15) // 16 * 16)[:-1]])
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, n_users, size=nseg)
    segs["offset"] = offs
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * nseg), dtype=np.uint8).reshape(nseg, 12)
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    total = int(offs[-1]) + (int(lens[-1]) + 15) // 16 * 16 + 16
    assert total // nseg <= 4096
    buf = rng.integers(0, 256, size=total, dtype=np.uint8)
    w = W.Workload("short", ids, keys, n_users, buf, buf.size, segs)
    ctx = make_ctx(w)
    d = dev(buf)
    tags, st = gpu_encrypt(ctx, w, d)
    ref = buf.copy()
    ref_tags, ref_st = gcm.seg_encrypt(ref, ref, segs, ids, keys, n_users)
    assert not ref_st.any() and not st_(st).any()
    assert np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(d), ref)
    bad = ref.copy()
    bad[int(offs[77]) + 3] ^= 2
    st2 = gpu_decrypt(ctx, w, dev(bad), dev(ref_tags), verify_only=True)
    assert st_(st2).sum() == 1 and st_(st2)[77] == 1
    st3 = gpu_decrypt(ctx, w, d, tags)
    assert not st_(st3).any() and np.array_equal(np_(d), buf)
    ctx.close()
