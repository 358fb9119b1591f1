"""Two-level ownership index: host-side rule steps (1)-(3) and slice runs against brute force (no GPU),
and on the GPU the owner expansion plus an end-to-end export of slot-level ownership slices."""
import itertools

import numpy as np
import pytest

from oracle import gcm, ownership_index as OI
from paper_2608_25431_b200 import binding as B


def _recs_args():
    recs = [dict(base=0x1000, shape=(4, 8), elem=2), dict(base=0x2000, shape=(4, 8), elem=2),
            dict(base=0x2020, shape=(16,), elem=4), dict(base=0x9000, shape=(2, 3, 2, 16, 8), elem=2)]
    return recs


def _to_c(recs, args):
    cr = [B.TensorRec.make(r["base"], r["shape"], r["elem"], [0]) for r in recs]
    ca = [B.KernelArg.make(a["base"], a["shape"], a["alias_group"]) for a in args]
    return cr, ca


def test_rule_steps_1_to_3_match_brute_force():
    recs = _recs_args()
    cases = [
        # AddResidual in place: O aliases I (declared), R separate
        [dict(base=0x1000, shape=(4, 8), alias_group=1), dict(base=0x1000, shape=(4, 8), alias_group=1),
         dict(base=0x2000, shape=(4, 8), alias_group=0)],
        # the same without the declaration: unintended aliasing
        [dict(base=0x1000, shape=(4, 8), alias_group=0), dict(base=0x1000, shape=(4, 8), alias_group=0)],
        # a tensor the monitor does not know, and a wrong shape
        [dict(base=0x1234, shape=(4, 8), alias_group=0), dict(base=0x2000, shape=(8, 4), alias_group=0)],
        # partially overlapping records (0x2000..0x2040 and 0x2020..0x2060)
        [dict(base=0x2000, shape=(4, 8), alias_group=0), dict(base=0x2020, shape=(16,), alias_group=0)],
        [dict(base=0x9000, shape=(2, 3, 2, 16, 8), alias_group=0), dict(base=0x1000, shape=(4, 8), alias_group=2)],
        [],
    ]
    for args in cases:
        cr, ca = _to_c(recs, args)
        idx, st = B.resolve_args(cr, ca)
        ridx, rst = OI.resolve_args(recs, args)
        assert idx == ridx and st == rst, args
    assert B.resolve_args(*_to_c(recs, cases[1]))[1] == [B.ARG_ALIAS, B.ARG_ALIAS]
    assert B.resolve_args(*_to_c(recs, cases[2]))[1] == [B.ARG_UNKNOWN, B.ARG_SHAPE]


def test_slice_runs_match_brute_force():
    shape, elem = (2, 3, 2, 16, 8), 2                       # [layer][block][kv][slot][dim], 16-byte rows
    rec = B.TensorRec.make(0, shape, elem, [0, 1, 3])
    slices = [((1, 2, 0, 0, 0), (2, 3, 2, 8, 8)),            # C[1,2,:,0:8,:]
              ((1, 2, 0, 8, 0), (2, 3, 2, 16, 8)),           # C[1,2,:,8:16,:]
              ((0, 0, 0, 0, 0), (2, 3, 2, 16, 8)),           # everything: one run
              ((0, 1, 0, 0, 0), (2, 2, 2, 16, 8)),           # C[:,1,:,:,:]
              ((0, 0, 1, 4, 0), (2, 3, 2, 8, 8)),            # C[:,:,1,4:8,:]
              ((1, 0, 0, 3, 0), (2, 3, 1, 4, 8))]            # single slots
    for lo, hi in slices:
        run, table = B.slice_runs(rec, lo, hi)
        rrun, rtable = OI.slice_runs(shape, elem, lo, hi)
        assert run == rrun and np.array_equal(table, rtable), (lo, hi)
    with pytest.raises(B.GiftError) as e:                    # half a row: not a multiple of 16 bytes
        B.slice_runs(rec, (0, 0, 0, 0, 0), (1, 1, 1, 1, 4))
    assert e.value.code == B.E_ALIGN
    with pytest.raises(B.GiftError):
        B.slice_runs(rec, (0, 0, 0, 0, 0), (3, 1, 1, 1, 8))  # out of range


@pytest.mark.gpu
def test_owner_expansion_and_slot_level_export_on_gpu():
    import torch
    rng = np.random.default_rng(0x61F70000 + 60)
    shape, elem = (2, 6, 2, 16, 64), 2                       # [layer][block][kv][slot][dim] bf16
    odims = [0, 1, 3]                                        # owner per (layer, block, slot)
    n_users = 5
    # slot-level ownership: the two halves of every block belong to different users
    half_owner = rng.integers(0, n_users, size=(2, 6, 2)).astype(np.int32)
    lvl2 = np.repeat(half_owner, 8, axis=2)                  # (layer, block, slot)
    total = int(np.prod(shape)) * elem
    buf = np.frombuffer(rng.bytes(total), dtype=np.uint8).copy()
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16)
    ctx = B.Ctx(n_users)
    ctx.set_keys(ids, keys)
    d_lvl2 = torch.from_numpy(lvl2.reshape(-1)).cuda()
    rec = B.TensorRec.make(0, shape, elem, odims, d_lvl2.data_ptr())

    # every (layer, block, half) is one ownership slice C[l,b,:,h*8:(h+1)*8,:]: 2 runs of 1 KiB
    from paper_2608_25431_b200 import workloads as W
    segs, table = [], []
    for l, b, h in itertools.product(range(2), range(6), range(2)):
        run, t = B.slice_runs(rec, (l, b, 0, 8 * h, 0), (l + 1, b + 1, 2, 8 * h + 8, 64))
        assert run == 8 * 64 * 2 and len(t) == 2
        segs.append((int(half_owner[l, b, h]), len(table), run * len(t), (l, b, h)))
        table += t.tolist()
    run_bytes = 8 * 64 * 2
    st = np.zeros(len(segs), dtype=W.SEG_DTYPE)
    st["owner"] = [s[0] for s in segs]
    st["page0"] = [s[1] for s in segs]
    st["len"] = [s[2] for s in segs]
    st["nonce"] = W.nonce_triple([s[3][0] for s in segs], [s[3][1] for s in segs], [s[3][2] for s in segs])

    n_units = total // run_bytes
    unit_owner = torch.full((n_units,), -7, dtype=torch.int32, device="cuda")
    ctx.expand_owners(rec, run_bytes, unit_owner)
    torch.cuda.synchronize()
    ref_units = OI.expand_owners(shape, elem, odims, lvl2, run_bytes)
    assert np.array_equal(unit_owner.cpu().numpy(), ref_units)
    for rb in (128, 256, 16 * 64 * 2, 2 * 16 * 64 * 2):    # part of a slot record ... a whole block (both halves)
        uo = torch.full((total // rb,), -7, dtype=torch.int32, device="cuda")
        ctx.expand_owners(rec, rb, uo)
        torch.cuda.synchronize()
        ref = OI.expand_owners(shape, elem, odims, lvl2, rb)
        assert np.array_equal(uo.cpu().numpy(), ref)
        if rb >= 16 * 64 * 2:
            assert (ref == B.OWNER_CONFLICT).any()           # blocks whose halves have different owners
    with pytest.raises(B.GiftError):                         # neither a part of a record nor whole records
        ctx.expand_owners(rec, 192, torch.zeros(total // 192, dtype=torch.int32, device="cuda"))

    d_buf = torch.from_numpy(buf).cuda()
    tags = torch.zeros((len(segs), 16), dtype=torch.uint8, device="cuda")
    status = torch.full((len(segs),), 9, dtype=torch.int32, device="cuda")
    ctx.seg_encrypt(d_buf, d_buf, torch.from_numpy(st.view(np.uint8).copy()).cuda(), len(segs), tags, status,
                    page_table=torch.from_numpy(np.array(table, dtype=np.int32)).cuda(), page_bytes=run_bytes,
                    owner_map=unit_owner, unit_bytes=run_bytes)
    torch.cuda.synchronize()
    assert not status.cpu().numpy().any()                    # every slice is owned by the user it is exported for
    out = d_buf.cpu().numpy().reshape(shape + (elem,))
    plain = buf.reshape(shape + (elem,))
    tags = tags.cpu().numpy()
    for i, (owner, _, _, (l, b, h)) in enumerate(segs):
        pt = plain[l, b, :, 8 * h: 8 * h + 8].tobytes()
        ct, tag = gcm.gcm_encrypt(keys[owner], st["nonce"][i], pt)
        assert out[l, b, :, 8 * h: 8 * h + 8].tobytes() == ct and tags[i].tobytes() == tag
    # claiming a slice for the other half's owner is refused by the label check
    st2 = st.copy()
    other = [(i, s) for i, s in enumerate(segs) if segs[i ^ 1][0] != s[0]]
    i0 = other[0][0]
    st2["owner"][i0] = segs[i0 ^ 1][0]
    ctx.seg_encrypt(d_buf, d_buf, torch.from_numpy(st2.view(np.uint8).copy()).cuda(), len(segs), torch.zeros_like(torch.from_numpy(tags)).cuda(),
                    status, page_table=torch.from_numpy(np.array(table, dtype=np.int32)).cuda(), page_bytes=run_bytes,
                    owner_map=unit_owner, unit_bytes=run_bytes)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[i0] == B.ST_OWNER_MISMATCH
    ctx.close()
