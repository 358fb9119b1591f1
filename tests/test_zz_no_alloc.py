"""The allocation-free export call (gift_seg_encrypt_static) against gift_seg_encrypt.

Some users of the library cannot call cudaMalloc at the moment they export data (all device
memory already belongs to their own pool, or an allocation there would stall every stream),
so this entry point keeps its scratch in a fixed array inside the library.  The test calls
it through the C-ABI twice in a row and compares ciphertext, tags and status words with the
regular entry point; results are unique, so the comparison is exact equality.  The file is
named to be collected last."""
import numpy as np
import pytest
import torch

from paper_2608_25431_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu


def _segs_dev(segs):
    return torch.from_numpy(np.ascontiguousarray(segs).view(np.uint8).copy()).cuda()


def _run(ctx, fn, w, src, segs, owner_map):
    n = len(segs)
    dst = torch.full_like(src, 0xEE)
    tags = torch.full((n, 16), 0xAB, dtype=torch.uint8, device="cuda")
    status = torch.full((n,), 0xDEAD, dtype=torch.int32, device="cuda")
    fn(src, dst, _segs_dev(segs), n, tags, status,
       page_table=torch.from_numpy(w.page_table).cuda() if w.page_table is not None else None,
       page_bytes=w.page_bytes, owner_map=torch.from_numpy(owner_map).cuda(), unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    return dst.cpu().numpy(), tags.cpu().numpy(), status.cpu().numpy()


def test_static_scratch_export_matches_regular_export_twice():
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
        ref = _run(ctx, ctx.seg_encrypt, w, data, segs, om)
        got = _run(ctx, ctx.seg_encrypt_static, w, data, segs, om)
        for a, b in zip(ref, got):
            assert np.array_equal(a, b)
        assert ref[2].any() and not ref[2].all()             # the refused segment is reported by both
    # a flat table too, and the size limit
    w1 = W.config1()
    ctx1 = binding.Ctx(w1.max_users)
    ctx1.set_keys(w1.user_ids, w1.keys)
    src1 = torch.from_numpy(w1.buf).cuda()
    n = len(w1.segs)
    out = []
    for fn in (ctx1.seg_encrypt, ctx1.seg_encrypt_static):
        dst = torch.full_like(src1, 0xEE)
        tags = torch.zeros((n, 16), dtype=torch.uint8, device="cuda")
        status = torch.zeros(n, dtype=torch.int32, device="cuda")
        fn(src1, dst, _segs_dev(w1.segs), n, tags, status)
        torch.cuda.synchronize()
        out.append((dst.cpu().numpy(), tags.cpu().numpy(), status.cpu().numpy()))
    for a, b in zip(*out):
        assert np.array_equal(a, b)
    big = torch.zeros(40 * (binding.STATIC_MAX_SEGS + 1), dtype=torch.uint8, device="cuda")
    tags = torch.zeros((binding.STATIC_MAX_SEGS + 1, 16), dtype=torch.uint8, device="cuda")
    status = torch.zeros(binding.STATIC_MAX_SEGS + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.GiftError) as e:
        ctx1.seg_encrypt_static(src1, src1, big, binding.STATIC_MAX_SEGS + 1, tags, status)
    assert e.value.code == binding.E_RANGE
    ctx.close()
    ctx1.close()
