"""Seeded random tables of every kind against the oracle: flat and paged, tiny to multi-megabyte
segments, table sizes around the single-launch threshold, corrupted labels, reserved flags set,
users without keys, both AES table counts and both launch forms; export, import of tampered
bytes and verify, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import dev, gpu_decrypt, gpu_encrypt, make_ctx, np_, st_

pytestmark = pytest.mark.gpu


def _one_table(rng):
    paged = bool(rng.integers(0, 2)); n_users = int(rng.integers(1, 9)); nseg = int(rng.choice([1, 3, 40, 700, 1024, 1025, 2500]))
    big = rng.random() < 0.3
    choices = [0, 1, 15, 16, 17, 48, 500, 512, 513, 4096, 4097, 9000, 33000] + ([300000, 1 << 20, (3 << 20) + 5] if big and nseg <= 40 else [])
    lens = rng.choice(choices, size=nseg)
    ids = np.arange(n_users, dtype=np.int32); keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE); segs["owner"] = rng.integers(0, n_users, size=nseg); segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * nseg), dtype=np.uint8).reshape(nseg, 12)
    if paged:
        pb = int(rng.choice([16, 48, 512, 1040, 1536, 4096, 65536]))
        npages = (lens + pb - 1) // pb; total = int(npages.sum()) + 3
        table = rng.permutation(total).astype(np.int32); segs["page0"] = np.concatenate([[0], np.cumsum(npages)[:-1]])
        buf = np.frombuffer(rng.bytes(total * pb), dtype=np.uint8).copy(); om = np.full(total, -2, dtype=np.int32)
        for i in range(nseg): om[table[int(segs["page0"][i]): int(segs["page0"][i]) + int(npages[i])]] = segs["owner"][i]
        w = W.Workload("fz", ids, keys, n_users, buf, buf.size, segs, page_table=table, page_bytes=pb, owner_map=om, unit_bytes=pb)
    else:
        unit = int(rng.choice([64, 256, 4096])); offs, o = [], 0
        for n in lens:
            o = (o + unit - 1) // unit * unit; offs.append(o); o += int(n)
        segs["offset"] = offs; buf = np.frombuffer(rng.bytes((o + unit) // unit * unit), dtype=np.uint8).copy()
        om = np.full(buf.size // unit, -2, dtype=np.int32)
        for i in range(nseg):
            if lens[i]: om[offs[i] // unit: (offs[i] + int(lens[i]) + unit - 1) // unit] = segs["owner"][i]
        w = W.Workload("fz", ids, keys, n_users, buf, buf.size, segs, owner_map=om, unit_bytes=unit)
    for u in rng.choice(om.size, size=min(4, om.size), replace=False): om[u] = rng.choice([-2, -1, -3, 0])
    if nseg > 2: segs["flags"][int(rng.integers(0, nseg))] = int(rng.integers(0, 2))
    have = ids[:-1] if n_users > 1 and rng.random() < 0.4 else ids
    flags = int(rng.choice([0, 0, binding.CTX_SPLIT_LAUNCH, binding.CTX_TWO_TABLES]))
    ctx = make_ctx(w, flags, user_ids=have, keys=keys[: len(have)])
    d = dev(w.buf); tags, st = gpu_encrypt(ctx, w, d); ref = w.buf.copy()
    rt, rs = gcm.seg_encrypt(ref, ref, w.segs, have, keys[: len(have)], n_users, w.page_table, w.page_bytes, w.owner_map, w.unit_bytes)
    assert np.array_equal(st_(st), rs) and np.array_equal(np_(tags), rt) and np.array_equal(np_(d), ref), ("enc", paged, nseg, flags)
    bad = ref.copy()
    for _ in range(3): bad[int(rng.integers(0, bad.size))] ^= 1 << int(rng.integers(0, 8))
    om_ref = np.full(om.size, 55, dtype=np.int32); out_ref = bad.copy()
    sr = gcm.seg_decrypt(out_ref, out_ref, w.segs, rt, have, keys[: len(have)], n_users, w.page_table, w.page_bytes, om_ref, w.unit_bytes)
    omd = torch.full((om.size,), 55, dtype=torch.int32, device="cuda"); db = dev(bad)
    s2 = gpu_decrypt(ctx, w, db, dev(rt), owner_map=omd)
    assert np.array_equal(st_(s2), sr) and np.array_equal(np_(db), out_ref) and np.array_equal(np_(omd), om_ref), ("dec", paged, nseg, flags)
    s3 = gpu_decrypt(ctx, w, dev(bad), dev(rt), verify_only=True)
    assert np.array_equal(st_(s3), sr), ("ver", paged, nseg, flags)
    ctx.close()


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_tables_of_every_kind_match_oracle(seed):
    rng = np.random.default_rng(W.SEED_BASE + 500 + seed)
    for _ in range(60):
        _one_table(rng)
    assert binding.gift_last_error_detail() == ""
