"""The allocation-free export call (gift_seg_encrypt_static) against the oracle and gift_seg_encrypt.

Some users of the library cannot call cudaMalloc at the moment they export data (all device
memory already belongs to their own pool, or an allocation there would stall every stream),
so this entry point keeps its scratch in a fixed array inside the library.  The test calls
it through the C-ABI twice in a row and compares ciphertext, tags and status words with the
CPU oracle and with the regular entry point; results are unique, so every comparison is
exact equality.  It also runs a table that is larger than anything the context has seen, which
would make the regular entry point grow its scratch, and checks that free device memory
does not move.  The file is named to be collected last."""
import numpy as np
import pytest
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu


def _segs_dev(segs):
    return torch.from_numpy(np.ascontiguousarray(segs).view(np.uint8).copy()).cuda()


def _run(fn, w, src, segs, owner_map):
    n = len(segs)
    dst = torch.full_like(src, 0xEE)
    tags = torch.full((n, 16), 0xAB, dtype=torch.uint8, device="cuda")
    status = torch.full((n,), 0xDEAD, dtype=torch.int32, device="cuda")
    fn(src, dst, _segs_dev(segs), n, tags, status,
       page_table=torch.from_numpy(w.page_table).cuda() if w.page_table is not None else None,
       page_bytes=w.page_bytes, owner_map=torch.from_numpy(owner_map).cuda() if owner_map is not None else None,
       unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    return dst.cpu().numpy(), tags.cpu().numpy(), status.cpu().numpy().astype(np.uint32)


def _oracle(w, src, segs, owner_map, aad=None):
    dst = np.full_like(src, 0xEE)
    tags, st = gcm.seg_encrypt(src, dst, segs, w.user_ids, w.keys, w.max_users, w.page_table, w.page_bytes,
                               owner_map, w.unit_bytes, aad=aad)
    return dst, tags, st


def test_static_scratch_export_matches_oracle_and_regular_export_twice():
    # paged KV blocks with multi-run segments, one refused segment, and a second, different call
    w = W.config4(total_bytes=24 << 20, cap_bytes=8 << 20, n_users=32)
    ctx = binding.Ctx(w.max_users)
    ctx.set_keys(w.user_ids, w.keys)
    src = torch.from_numpy(w.buf).cuda()
    om = w.owner_map.copy()
    victim = int(np.argmax(w.segs["len"] > 0))
    om[w.page_table[int(w.segs["page0"][victim])]] = binding.OWNER_NONE      # this segment must be refused
    calls = [(w.segs, src), (W.bump_epoch(w.segs)[::-1].copy(), torch.flip(src, dims=[0]).contiguous())]
    for segs, data in calls:
        want = _oracle(w, data.cpu().numpy(), segs, om)
        got = _run(ctx.seg_encrypt_static, w, data, segs, om)
        ref = _run(ctx.seg_encrypt, w, data, segs, om)
        for a, b, c in zip(want, got, ref):
            assert np.array_equal(a, b) and np.array_equal(a, c)
        assert want[2].any() and not want[2].all()           # the refused segment is reported
    # a flat table too, and the size limit
    w1 = W.config1()
    ctx1 = binding.Ctx(w1.max_users)
    ctx1.set_keys(w1.user_ids, w1.keys)
    src1 = torch.from_numpy(w1.buf).cuda()
    want = _oracle(w1, w1.buf, w1.segs, None)
    for fn in (ctx1.seg_encrypt_static, ctx1.seg_encrypt_static, ctx1.seg_encrypt):
        got = _run(fn, w1, src1, w1.segs, None)
        for a, b in zip(want, got):
            assert np.array_equal(a, b)
    big = torch.zeros(40 * (binding.STATIC_MAX_SEGS + 1), dtype=torch.uint8, device="cuda")
    tags = torch.zeros((binding.STATIC_MAX_SEGS + 1, 16), dtype=torch.uint8, device="cuda")
    status = torch.zeros(binding.STATIC_MAX_SEGS + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.GiftError) as e:
        ctx1.seg_encrypt_static(src1, src1, big, binding.STATIC_MAX_SEGS + 1, tags, status)
    assert e.value.code == binding.E_RANGE
    ctx.close()
    ctx1.close()


def test_static_scratch_export_honours_bound_aad():
    """Tags made by the static entry on a context with bound AAD verify with gift_verify_tags on the
    same context, and equal the oracle's tags with that AAD."""
    w = W.config4(total_bytes=6 << 20, cap_bytes=2 << 20, n_users=8)
    n = len(w.segs)
    rng = np.random.default_rng(41)
    aad = np.frombuffer(rng.bytes(16 * n), dtype=np.uint8).reshape(n, 16).copy()
    ctx = binding.Ctx(w.max_users)
    ctx.set_keys(w.user_ids, w.keys)
    d_aad = torch.from_numpy(aad).cuda()
    ctx.bind_aad(d_aad)
    src = torch.from_numpy(w.buf).cuda()
    want = _oracle(w, w.buf, w.segs, w.owner_map, aad=aad)
    for _ in range(2):
        got = _run(ctx.seg_encrypt_static, w, src, w.segs, w.owner_map)
        for a, b in zip(want, got):
            assert np.array_equal(a, b)
    ct, tags = torch.from_numpy(got[0]).cuda(), torch.from_numpy(got[1]).cuda()
    status = torch.full((n,), 9, dtype=torch.int32, device="cuda")
    ctx.verify_tags(ct, _segs_dev(w.segs), n, tags, status, page_table=torch.from_numpy(w.page_table).cuda(),
                    page_bytes=w.page_bytes)
    torch.cuda.synchronize()
    assert not status.any().item()
    ctx.close()


def test_static_scratch_export_allocates_nothing_for_a_table_larger_than_any_before():
    """5 000 small flat segments on a context whose scratch holds 1 024: the regular entry point
    would reallocate, the static one must leave free device memory where it was."""
    rng = np.random.default_rng(43)
    nseg, n_users = 5000, 9
    lens = rng.integers(16, 4097, size=nseg)
    offs = np.concatenate([[0], np.cumsum((lens + 15) // 16 * 16)[:-1]])
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, n_users, size=nseg)
    segs["offset"] = offs
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * nseg), dtype=np.uint8).reshape(nseg, 12)
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    total = int(offs[-1]) + (int(lens[-1]) + 15) // 16 * 16
    buf = rng.integers(0, 256, size=total, dtype=np.uint8)
    w = W.Workload("static_many", ids, keys, n_users, buf, buf.size, segs)
    ctx = binding.Ctx(n_users)                  # never reserved: its own scratch holds 1 024 segments
    ctx.set_keys(ids, keys)
    src = torch.from_numpy(buf).cuda()
    dst = torch.full_like(src, 0xEE)
    d_segs = _segs_dev(segs)
    tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    status = torch.zeros(nseg, dtype=torch.int32, device="cuda")
    ctx.seg_encrypt_static(src, dst, d_segs, nseg, tags, status)       # warm-up: symbol look-up, kernel load
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(2):
        tags.zero_()
        ctx.seg_encrypt_static(src, dst, d_segs, nseg, tags, status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    want = _oracle(w, buf, segs, None)
    assert np.array_equal(dst.cpu().numpy(), want[0]) and np.array_equal(tags.cpu().numpy(), want[1])
    assert not status.any().item() and not want[2].any()
    ctx2 = binding.Ctx(n_users)                 # the regular entry point on a second context agrees
    ctx2.set_keys(ids, keys)
    ref = _run(ctx2.seg_encrypt, w, src, segs, None)
    assert np.array_equal(ref[0], want[0]) and np.array_equal(ref[1], want[1])
    ctx.close()
    ctx2.close()


def test_no_cuda_call_of_the_library_failed_silently():
    """Clean-up paths go on after a failing CUDA call but remember it; by the end of a run (this
    file is collected last) nothing must have been remembered."""
    assert binding.gift_last_error_detail() == ""
