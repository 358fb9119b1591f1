"""The optional overlap check of a segment table (GIFT_CTX_CHECK_OVERLAP) against the oracle's definition."""
import numpy as np
import pytest
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import dev, gpu_decrypt, gpu_encrypt, make_ctx, np_, st_

pytestmark = pytest.mark.gpu


def _flat_with_overlaps(rng, nseg, n_users):
    lens = rng.integers(0, 3000, size=nseg)
    starts, o = [], 0
    for n in lens:
        starts.append(o)
        o += (int(n) + 15) // 16 * 16
    starts = np.array(starts, dtype=np.int64)
    # pull some segments back onto their predecessors, duplicate some, leave most alone
    for i in rng.choice(np.arange(1, nseg), size=max(1, nseg // 12), replace=False):
        starts[i] = max(0, starts[i] - 16 * int(rng.integers(1, 40)))
    for i in rng.choice(np.arange(1, nseg), size=max(1, nseg // 40), replace=False):
        starts[i], lens[i] = starts[i - 1], lens[i - 1]
    segs = np.zeros(nseg, dtype=W.SEG_DTYPE)
    segs["owner"] = rng.integers(0, n_users, size=nseg)
    segs["offset"] = starts
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * nseg), dtype=np.uint8).reshape(nseg, 12)
    segs["offset"][nseg // 2] += 4                                      # one bad descriptor among them
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    buf = np.frombuffer(rng.bytes(o + 64), dtype=np.uint8).copy()
    return W.Workload("ovl_flat", ids, keys, n_users, buf, buf.size, segs)


@pytest.mark.parametrize("nseg,flags", [(40, 0), (700, 0), (700, binding.CTX_SPLIT_LAUNCH), (5000, 0)])
def test_flat_overlaps_are_refused_exactly(nseg, flags):
    rng = np.random.default_rng(W.SEED_BASE + 400 + nseg)
    w = _flat_with_overlaps(rng, nseg, 5)
    ctx = make_ctx(w, flags | binding.CTX_CHECK_OVERLAP)
    src = dev(w.buf)
    dst = torch.full_like(src, 0xEE)
    tags, st = gpu_encrypt(ctx, w, src, dst)
    ref = np.full_like(w.buf, 0xEE)
    ref_tags, ref_st = gcm.seg_encrypt(w.buf, ref, w.segs, w.user_ids, w.keys, w.max_users, check_overlap=True)
    assert (ref_st == 32).sum() >= 2 and (ref_st == 0).sum() > nseg // 2 and (ref_st == 16).sum() >= 1
    assert np.array_equal(st_(st), ref_st)
    assert np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(dst), ref)
    # import of what was exported, same table: the same segments are refused and left alone
    out = torch.full_like(src, 0x77)
    st2 = gpu_decrypt(ctx, w, dst, tags, out)
    ref_out = np.full_like(w.buf, 0x77)
    ref_st2 = gcm.seg_decrypt(ref, ref_out, w.segs, ref_tags, w.user_ids, w.keys, w.max_users, check_overlap=True)
    assert np.array_equal(st_(st2), ref_st2) and np.array_equal(np_(out), ref_out)
    ctx.close()


def test_paged_overlaps_shared_and_repeated_pages():
    w = W.config4(total_bytes=10 << 20, cap_bytes=2 << 20, n_users=8)
    pt = w.page_table.copy()
    lens, page0 = w.segs["len"], w.segs["page0"]
    multi = [i for i in range(len(w.segs)) if lens[i] > 2 * w.page_bytes]
    single = [i for i in range(len(w.segs)) if 0 < lens[i] <= w.page_bytes]
    a, b, c = multi[0], multi[1], multi[2]
    pt[int(page0[a]) + 1] = pt[int(page0[b])]            # a's second page is b's first
    pt[int(page0[c]) + 1] = pt[int(page0[c])]            # c names one page twice
    pt[int(page0[single[0]])] = pt[int(page0[single[1]])]   # two short segments on one page
    w.page_table = pt
    om = w.owner_map                                      # label the shared pages consistently with one claimant
    for flags in (0, binding.CTX_SPLIT_LAUNCH):
        ctx = make_ctx(w, flags | binding.CTX_CHECK_OVERLAP)
        d = dev(w.buf)
        tags, st = gpu_encrypt(ctx, w, d)
        ref = w.buf.copy()
        ref_tags, ref_st = gcm.seg_encrypt(ref, ref, w.segs, w.user_ids, w.keys, w.max_users, w.page_table,
                                           w.page_bytes, om, w.unit_bytes, check_overlap=True)
        for i in (a, b, c, single[0], single[1]):
            assert ref_st[i] == 32
        assert (ref_st == 32).sum() == 5
        assert np.array_equal(st_(st), ref_st) and np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(d), ref)
        ctx.close()


def test_without_the_flag_no_overlap_status_appears():
    rng = np.random.default_rng(W.SEED_BASE + 450)
    w = _flat_with_overlaps(rng, 60, 3)
    ctx = make_ctx(w)
    _, st = gpu_encrypt(ctx, w, dev(w.buf), torch.zeros(w.buf.size, dtype=torch.uint8, device="cuda"))
    assert not (st_(st) & 32).any()
    ctx.close()


def test_overlap_check_limits_and_the_static_entry():
    """Flat tables beyond 65 536 segments are refused when the check is on; the allocation-free entry takes
    flat tables with the check and refuses paged ones (their check needs memory that grows)."""
    rng = np.random.default_rng(W.SEED_BASE + 460)
    w = _flat_with_overlaps(rng, 300, 3)
    ctx = make_ctx(w, binding.CTX_CHECK_OVERLAP)
    src = dev(w.buf)
    n = len(w.segs)
    from gpu_harness import segs_dev
    dst = torch.full_like(src, 0xEE)
    tags = torch.zeros((n, 16), dtype=torch.uint8, device="cuda")
    st = torch.zeros(n, dtype=torch.int32, device="cuda")
    ctx.seg_encrypt_static(src, dst, segs_dev(w.segs), n, tags, st)
    torch.cuda.synchronize()
    ref = np.full_like(w.buf, 0xEE)
    ref_tags, ref_st = gcm.seg_encrypt(w.buf, ref, w.segs, w.user_ids, w.keys, w.max_users, check_overlap=True)
    assert np.array_equal(st_(st), ref_st) and np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(dst), ref)
    big_n = 65537
    big = torch.zeros(40 * big_n, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.GiftError) as e:
        ctx.seg_encrypt(src, dst, big, big_n, torch.zeros((big_n, 16), dtype=torch.uint8, device="cuda"),
                        torch.zeros(big_n, dtype=torch.int32, device="cuda"))
    assert e.value.code == binding.E_RANGE
    w4 = W.config4(total_bytes=4 << 20, cap_bytes=1 << 20, n_users=4)
    ctx4 = make_ctx(w4, binding.CTX_CHECK_OVERLAP)
    n4 = len(w4.segs)
    with pytest.raises(binding.GiftError) as e:
        ctx4.seg_encrypt_static(dev(w4.buf), dev(w4.buf), segs_dev(w4.segs), n4,
                                torch.zeros((n4, 16), dtype=torch.uint8, device="cuda"),
                                torch.zeros(n4, dtype=torch.int32, device="cuda"),
                                page_table=dev(w4.page_table), page_bytes=w4.page_bytes)
    assert e.value.code == binding.E_INVAL
    ctx.close()
    ctx4.close()
