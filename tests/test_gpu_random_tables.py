"""Seeded random segment tables, flat and paged with odd page sizes, against the oracle.

Page sizes that are not multiples of 512 bytes take the generic lane loop of the cipher
kernel (a row of 32 blocks may straddle pages there); multiples of 512 take the row loop."""
import numpy as np
import pytest
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import dev, gpu_decrypt, gpu_encrypt, make_ctx, np_, st_

pytestmark = pytest.mark.gpu


def _random_workload(rng, paged, page_bytes):
    n_users = int(rng.integers(1, 9))
    nseg = int(rng.integers(1, 40))
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    lens = rng.choice([0, 1, 15, 16, 17, 48, 500, 511, 512, 513, 2047, 4096, 4097, 9000, 33000], size=nseg)
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, n_users, size=nseg)
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * nseg), dtype=np.uint8).reshape(nseg, 12)
    if paged:
        npages = (lens + page_bytes - 1) // page_bytes
        total = int(npages.sum()) + 3
        table = rng.permutation(total).astype(np.int32)
        segs["page0"] = np.concatenate([[0], np.cumsum(npages)[:-1]])
        buf = np.frombuffer(rng.bytes(total * page_bytes), dtype=np.uint8).copy()
        om = np.full(total, binding.OWNER_NONE, dtype=np.int32)
        for i in range(nseg):
            om[table[int(segs["page0"][i]): int(segs["page0"][i]) + int(npages[i])]] = segs["owner"][i]
        w = W.Workload("rand_paged", ids, keys, n_users, buf, buf.size, segs, page_table=table,
                       page_bytes=page_bytes, owner_map=om, unit_bytes=page_bytes)
    else:
        unit = int(rng.choice([64, 256]))           # 256 and above: small tables take the fused launch
        offs, o = [], 0
        for n in lens:
            o = (o + unit - 1) // unit * unit            # unit-aligned starts: every unit has one owner
            offs.append(o)
            o += int(n) + 16 * int(rng.integers(0, 3))
        segs["offset"] = offs
        buf = np.frombuffer(rng.bytes((o + unit) // unit * unit), dtype=np.uint8).copy()
        om = np.full(buf.size // unit, binding.OWNER_NONE, dtype=np.int32)
        for i in range(nseg):
            if lens[i]:
                om[offs[i] // unit: (offs[i] + int(lens[i]) + unit - 1) // unit] = segs["owner"][i]
        w = W.Workload("rand_flat", ids, keys, n_users, buf, buf.size, segs, owner_map=om, unit_bytes=unit)
    # a few corrupted labels and one user without a key
    for u in rng.choice(om.size, size=min(3, om.size), replace=False):
        om[u] = rng.choice([binding.OWNER_NONE, binding.OWNER_PARAM, binding.OWNER_CONFLICT, 0])
    return w


@pytest.mark.parametrize("paged,page_bytes", [(False, 0), (True, 16), (True, 48), (True, 1040), (True, 512),
                                              (True, 1536), (True, 4096)])
def test_random_tables_match_oracle(paged, page_bytes):
    rng = np.random.default_rng(W.SEED_BASE + 70 + page_bytes)
    for trial in range(6):
        w = _random_workload(rng, paged, page_bytes)
        have = w.user_ids[:-1] if len(w.user_ids) > 1 and trial % 2 else w.user_ids      # sometimes a missing key
        flags = binding.CTX_SPLIT_LAUNCH if trial % 3 == 2 else 0          # mostly the fused single launch
        ctx = make_ctx(w, flags, user_ids=have, keys=w.keys[: len(have)])
        buf = dev(w.buf)
        tags, st = gpu_encrypt(ctx, w, buf)
        ref = w.buf.copy()
        ref_tags, ref_st = gcm.seg_encrypt(ref, ref, w.segs, have, w.keys[: len(have)], w.max_users, w.page_table,
                                           w.page_bytes, w.owner_map, w.unit_bytes)
        assert np.array_equal(st_(st), ref_st), (paged, page_bytes, trial)
        assert np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(buf), ref)
        # import with a few flipped bits; labels are rewritten by the call
        bad = ref.copy()
        for _ in range(2):
            bad[int(rng.integers(0, bad.size))] ^= 1 << int(rng.integers(0, 8))
        om_ref = np.full(w.owner_map.size, 55, dtype=np.int32)
        out_ref = bad.copy()
        st_ref = gcm.seg_decrypt(out_ref, out_ref, w.segs, ref_tags, have, w.keys[: len(have)], w.max_users,
                                 w.page_table, w.page_bytes, om_ref, w.unit_bytes)
        om = torch.full((w.owner_map.size,), 55, dtype=torch.int32, device="cuda")
        d_bad = dev(bad)
        st2 = gpu_decrypt(ctx, w, d_bad, dev(ref_tags), owner_map=om)
        assert np.array_equal(st_(st2), st_ref), (paged, page_bytes, trial)
        assert np.array_equal(np_(d_bad), out_ref) and np.array_equal(np_(om), om_ref)
        ctx.close()


def test_many_tiny_segments():
    """200 000 segments of 0..80 bytes: one run each; stresses the work list, the scan and the scratch growth."""
    rng = np.random.default_rng(W.SEED_BASE + 90)
    nseg, n_users = 200_000, 64
    lens = rng.integers(0, 81, size=nseg)
    offs = np.arange(nseg, dtype=np.uint64) * np.uint64(96)
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, n_users, size=nseg)
    segs["offset"] = offs
    segs["len"] = lens
    segs["nonce"][:, :4] = np.arange(nseg, dtype="<u4")[:, None].view(np.uint8).reshape(nseg, 4)
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    buf = np.frombuffer(rng.bytes(nseg * 96), dtype=np.uint8).copy()
    w = W.Workload("tiny", ids, keys, n_users, buf, buf.size, segs)
    ctx = make_ctx(w)
    d = dev(buf)
    tags, st = gpu_encrypt(ctx, w, d)
    ref = buf.copy()
    ref_tags, ref_st = gcm.seg_encrypt(ref, ref, segs, ids, keys, n_users)
    assert not ref_st.any() and np.array_equal(st_(st), ref_st)
    assert np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(d), ref)
    st2 = gpu_decrypt(ctx, w, d, tags)
    assert not st_(st2).any() and np.array_equal(np_(d), buf)
    ctx.close()


def test_mid_size_flat_table_with_ragged_lengths():
    """3 000 flat segments of 0..300 000 bytes (any byte length): about 450 MB, so that every
    resident warp gets a slice of a few thousand blocks whose ends fall at arbitrary places
    inside segments with partial last rows and partial last blocks."""
    rng = np.random.default_rng(4242)
    nseg, n_users = 3000, 7
    lens = rng.integers(0, 300_001, size=nseg)
    lens[rng.choice(nseg, size=40, replace=False)] = 0
    offs = np.concatenate([[0], np.cumsum((lens + 15) // 16 * 16)[:-1]])
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, n_users, size=nseg)
    segs["offset"] = offs
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * nseg), dtype=np.uint8).reshape(nseg, 12)
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    total = int(offs[-1] + (lens[-1] + 15) // 16 * 16) + 64
    buf = rng.integers(0, 256, size=total, dtype=np.uint8)
    w = W.Workload("mid_flat", ids, keys, n_users, buf, buf.size, segs)
    ctx = make_ctx(w)
    d = dev(w.buf)
    tags, st = gpu_encrypt(ctx, w, d)
    ref = w.buf.copy()
    ref_tags, ref_st = gcm.seg_encrypt(ref, ref, w.segs, ids, keys, n_users)
    assert not ref_st.any() and not st_(st).any()
    assert np.array_equal(np_(tags), ref_tags)
    assert np.array_equal(np_(d), ref)
    st2 = gpu_decrypt(ctx, w, d, tags)
    assert not st_(st2).any() and np.array_equal(np_(d), w.buf)
    ctx.close()
