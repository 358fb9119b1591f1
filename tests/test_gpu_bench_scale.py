"""Parity at the full sizes the benchmark times, in the same launch configuration.

The buffers are too large for the oracle to process whole, so a seeded sample of segments
(the largest, the smallest and random ones, plus every tampered one) is compared with the
oracle byte for byte, and properties that hold at any size are checked on the device:
every status word, decrypt(encrypt(x)) == x over the whole buffer, verify == all clear."""
import numpy as np
import pytest
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding, device_fill, workloads as W

pytestmark = pytest.mark.gpu


def _need(nbytes):
    free, _ = torch.cuda.mem_get_info()
    if free < nbytes:
        pytest.skip("needs %.1f GiB of free device memory" % (nbytes / 2**30))


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _segs_dev(segs):
    return torch.from_numpy(np.ascontiguousarray(segs).view(np.uint8).copy()).cuda()


def _gather(w, buf, i):
    """Bytes of segment i out of a device buffer, as a numpy array."""
    s = w.segs[i]
    n = int(s["len"])
    if w.page_table is None:
        o = int(s["offset"])
        return buf[o:o + n].cpu().numpy()
    pb = w.page_bytes
    npg = (n + pb - 1) // pb
    pages = torch.from_numpy(w.page_table[int(s["page0"]): int(s["page0"]) + npg].astype(np.int64)).cuda()
    return buf.view(-1, pb)[pages].reshape(-1)[:n].cpu().numpy()


def _sample(w, rng, extra=()):
    order = np.argsort(w.segs["len"], kind="stable")
    pick = set(order[:8].tolist()) | set(order[-8:].tolist()) | set(int(x) for x in extra)
    pick |= set(rng.choice(len(w.segs), size=min(64, len(w.segs)), replace=False).tolist())
    return sorted(pick)


def _check_sample(w, sample, plain, cipher_buf, tags):
    tags = tags.cpu().numpy()
    for i in sample:
        s = w.segs[i]
        ct, tag = gcm.gcm_encrypt(w.keys[int(s["owner"])], s["nonce"], plain[i])
        assert _gather(w, cipher_buf, i).tobytes() == ct, i
        assert tags[i].tobytes() == tag, i


def _full_round_trip(w, fill):
    nseg = len(w.segs)
    ctx = binding.Ctx(w.max_users)
    ctx.set_keys(w.user_ids, w.keys)
    buf = torch.empty(w.buf_bytes, dtype=torch.uint8, device="cuda")
    fill(buf)
    rng = np.random.default_rng(W.SEED_BASE + 77)
    sample = _sample(w, rng)
    plain = {i: _gather(w, buf, i) for i in sample}
    checksum = buf.view(torch.int64).sum().item()
    segs, table = _segs_dev(w.segs), (_dev(w.page_table) if w.page_table is not None else None)
    om = _dev(w.owner_map)
    tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    status = torch.full((nseg,), 7, dtype=torch.int32, device="cuda")
    ctx.seg_encrypt(buf, buf, segs, nseg, tags, status, page_table=table, page_bytes=w.page_bytes,
                    owner_map=om, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    assert not status.any().item()
    _check_sample(w, sample, plain, buf, tags)
    ctx.verify_tags(buf, segs, nseg, tags, status, page_table=table, page_bytes=w.page_bytes)
    assert not status.any().item()
    om2 = torch.full_like(om, binding.OWNER_NONE)
    ctx.seg_decrypt(buf, buf, segs, nseg, tags, status, page_table=table, page_bytes=w.page_bytes,
                    owner_map=om2, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    assert not status.any().item()
    assert buf.view(torch.int64).sum().item() == checksum
    for i in sample:
        assert np.array_equal(_gather(w, buf, i), plain[i]), i
    covered = torch.zeros_like(om, dtype=torch.bool)
    assert torch.equal(om2[om2 != binding.OWNER_NONE], om[om2 != binding.OWNER_NONE])
    del covered
    ctx.close()
    return True


def test_config3_full_32_layers():
    w = W.config3(layers=32, fill=False)
    _need(w.buf_bytes + (3 << 30))
    assert _full_round_trip(w, lambda b: device_fill.fill_bf16_normal(b, W.SEED_BASE + 3, 1.0))


def test_config4_full_8gib_zipf():
    w = W.config4(total_bytes=8 << 30, cap_bytes=64 << 20, fill=False)
    _need(w.buf_bytes + (3 << 30))
    assert int(w.segs["len"].max()) == 64 << 20
    assert _full_round_trip(w, lambda b: device_fill.fill_bytes(b, W.SEED_BASE + 4))


def test_config5_full_tamper_detection_exact():
    w = W.config5(layers=32, chunk_tokens=512, fill=False)
    _need(w.buf_bytes + (4 << 30))
    x = w.extra
    nseg = len(w.segs)
    ctx = binding.Ctx(w.max_users)
    ctx.set_keys(w.user_ids, w.keys)
    buf = torch.empty(w.buf_bytes, dtype=torch.uint8, device="cuda")
    device_fill.fill_bf16_normal(buf, W.SEED_BASE + 5, 1.0)
    rng = np.random.default_rng(W.SEED_BASE + 78)
    sample = _sample(w, rng, extra=x["poisoned"][::8])
    plain = {i: _gather(w, buf, i) for i in sample}
    segs, om = _segs_dev(w.segs), _dev(w.owner_map)
    tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    status = torch.full((nseg,), 7, dtype=torch.int32, device="cuda")
    ctx.seg_encrypt(buf, buf, segs, nseg, tags, status, owner_map=om, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    assert not status.any().item()
    _check_sample(w, sample, plain, buf, tags)
    # tamper: 1 % of the segments, in thirds a ciphertext bit, a tag bit, a wrong claimed owner
    bad = w.segs.copy()
    for s, kind, bit, tbit, wrong in zip(x["poisoned"], x["poison_kind"], x["poison_bit"], x["poison_tagbit"], x["poison_owner"]):
        if kind == 0:
            buf[int(bad["offset"][s]) + int(bit) // 8] ^= 1 << (int(bit) % 8)
        elif kind == 1:
            tags[int(s), int(tbit) // 8] ^= 1 << (int(tbit) % 8)
        else:
            bad["owner"][s] = wrong
    om2 = torch.full_like(om, 12345)
    ctx.seg_decrypt(buf, buf, _segs_dev(bad), nseg, tags, status, owner_map=om2, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    st = status.cpu().numpy()
    assert np.array_equal(np.nonzero(st)[0], x["poisoned"]) and (st[x["poisoned"]] == binding.ST_TAG_MISMATCH).all()
    om2 = om2.cpu().numpy()
    T, L = x["T"], x["layers"]
    for i in sample:
        s = w.segs[i]
        got = _gather(w, buf, i)
        u0, nu = int(s["offset"]) // w.unit_bytes, int(s["len"]) // w.unit_bytes
        if st[i]:
            assert not got.any() and (om2[u0:u0 + nu] == binding.OWNER_NONE).all()
        else:
            assert np.array_equal(got, plain[i]) and (om2[u0:u0 + nu] == int(s["owner"])).all()
    ctx.close()
