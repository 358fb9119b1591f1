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


# ---- pins of the brute-force oracle: every expected value below was worked out by hand ----
#
# Tensor of paper sec. 4.2's example, C[layer][block][kv][slot][dim] with shape (2, 3, 2, 16, 8) and
# 2-byte elements.  Byte strides: dim 2, slot 16, kv 256, block 512, layer 1536; 3072 bytes in all.

def test_oracle_slice_runs_hand_computed():
    shape, elem = (2, 3, 2, 16, 8), 2
    hand = [
        # C[1,2,:,0:8,:]: slots 0..7 of one kv half are 8*16 = 128 contiguous bytes; the two halves start
        # at 1536 + 2*512 + {0, 256} = 2560 and 2816, i.e. runs number 20 and 22
        (((1, 2, 0, 0, 0), (2, 3, 2, 8, 8)), 128, [20, 22]),
        # C[1,2,:,8:16,:]: the other eight slots, 128 bytes further on
        (((1, 2, 0, 8, 0), (2, 3, 2, 16, 8)), 128, [21, 23]),
        # C[:,1,:,:,:]: a whole block (512 bytes) per layer, at 512 and 1536 + 512 = 2048
        (((0, 1, 0, 0, 0), (2, 2, 2, 16, 8)), 512, [1, 4]),
        # C[:,:,1,4:8,:]: four slots = 64 bytes at layer*1536 + block*512 + 256 + 4*16
        (((0, 0, 1, 4, 0), (2, 3, 2, 8, 8)), 64, [5, 13, 21, 29, 37, 45]),
        # C[1,:,0,3,:]: single slots of 16 bytes at 1536 + block*512 + 48 = 1584, 2096, 2608
        (((1, 0, 0, 3, 0), (2, 3, 1, 4, 8)), 16, [99, 131, 163]),
        # the whole tensor is one run
        (((0, 0, 0, 0, 0), (2, 3, 2, 16, 8)), 3072, [0]),
    ]
    rec = B.TensorRec.make(0, shape, elem, [0, 1, 3])
    for (lo, hi), run, table in hand:
        orun, otable = OI.slice_runs(shape, elem, lo, hi)
        assert orun == run and otable.tolist() == table, (lo, hi)
        crun, ctable = B.slice_runs(rec, lo, hi)                 # the library's host call agrees with the same values
        assert crun == run and ctable.tolist() == table, (lo, hi)
    # the byte offsets themselves for the smallest case: three rows of eight 2-byte elements
    assert OI.slice_byte_offsets(shape, elem, (1, 0, 0, 3, 0), (2, 3, 1, 4, 8)).tolist() == \
        list(range(1584, 1600)) + list(range(2096, 2112)) + list(range(2608, 2624))


def test_oracle_expand_owners_hand_computed():
    # shape (2, 3, 2, 4, 2), 2-byte elements: a slot row is 4 bytes, a kv half 16, a block 32, a layer 96.
    # Ownership by (layer, block, slot): the three extents differ, so a transposed broadcast cannot pass.
    shape, elem, odims = (2, 3, 2, 4, 2), 2, [0, 1, 3]
    P, X = -1, -3                                               # PARAM, CONFLICT
    lvl2 = [[[1, 1, 2, 2], [3, 3, 3, 3], [0, 1, 0, 1]],
            [[4, 4, 4, 4], [P, P, 5, 5], [2, 2, 2, 2]]]
    hand = {
        # one label per slot row: the level-2 record, once per kv half
        4: [1, 1, 2, 2, 1, 1, 2, 2] + [3] * 8 + [0, 1, 0, 1, 0, 1, 0, 1] +
           [4] * 8 + [P, P, 5, 5, P, P, 5, 5] + [2] * 8,
        # two slots per run: they agree, or the run is CONFLICT
        8: [1, 2, 1, 2, 3, 3, 3, 3, X, X, X, X, 4, 4, 4, 4, P, 5, P, 5, 2, 2, 2, 2],
        # a kv half (four slots) per run
        16: [X, X, 3, 3, X, X, 4, 4, X, X, 2, 2],
        # a whole block per run
        32: [X, 3, X, 4, X, 2],
        # half a slot row: part of one record, the label twice
        2: [v for v in ([1, 1, 2, 2, 1, 1, 2, 2] + [3] * 8 + [0, 1, 0, 1, 0, 1, 0, 1] +
                        [4] * 8 + [P, P, 5, 5, P, P, 5, 5] + [2] * 8) for _ in (0, 1)],
    }
    for run_bytes, want in hand.items():
        assert OI.expand_owners(shape, elem, odims, lvl2, run_bytes).tolist() == want, run_bytes
    # ownership by rows only (odims = (0)): every byte of a layer carries the layer's label
    assert OI.expand_owners(shape, elem, [0], [7, 9], 48).tolist() == [7, 7, 9, 9]
    # ownership by the innermost of the recorded dimensions only (odims = (3)): label = slot's
    assert OI.expand_owners((1, 1, 2, 4, 2), elem, [3], [5, 6, 7, 8], 4).tolist() == [5, 6, 7, 8, 5, 6, 7, 8]


def test_oracle_resolve_args_hand_computed():
    OK_, UNK, SHP, ALI = 0, 1, 2, 4
    recs = [dict(base=0x1000, shape=(4, 8), elem=2),             # 0: [0x1000, 0x1040)
            dict(base=0x2000, shape=(4, 8), elem=2),             # 1: [0x2000, 0x2040)
            dict(base=0x2020, shape=(16,), elem=4),              # 2: [0x2020, 0x2060)  overlaps 1 partially
            dict(base=0x9000, shape=(2, 3, 2, 16, 8), elem=2),   # 3: [0x9000, 0x9C00)
            dict(base=0x9010, shape=(4,), elem=4),               # 4: [0x9010, 0x9020)  inside 3
            dict(base=0x1040, shape=(8,), elem=2)]               # 5: [0x1040, 0x1050)  touches 0, no common byte

    def arg(k, group=0, shape=None):
        return dict(base=recs[k]["base"], shape=recs[k]["shape"] if shape is None else shape, alias_group=group)

    hand = [
        ([arg(1), arg(2)], [1, 2], [ALI, ALI]),                  # partial overlap, either order
        ([arg(2), arg(1)], [2, 1], [ALI, ALI]),
        ([arg(3), arg(4)], [3, 4], [ALI, ALI]),                  # one inside the other, either order
        ([arg(4), arg(3)], [4, 3], [ALI, ALI]),
        ([arg(3, 7), arg(4, 7)], [3, 4], [OK_, OK_]),            # declared as aliases: accepted
        ([arg(3, 7), arg(4, 8)], [3, 4], [ALI, ALI]),            # different groups: not the same declaration
        ([arg(0), arg(5)], [0, 5], [OK_, OK_]),                  # adjacent ranges share no byte
        ([arg(0), arg(1), arg(2), arg(5)], [0, 1, 2, 5], [OK_, ALI, ALI, OK_]),
        ([arg(1, 0, (8, 4)), arg(2)], [1, 2], [SHP | ALI, ALI]), # wrong shape and overlapping
        ([dict(base=0x2010, shape=(4, 8), alias_group=0), arg(2)], [-1, 2], [UNK, OK_]),   # unknown base: no record, no range
    ]
    for args, want_idx, want_st in hand:
        assert OI.resolve_args(recs, args) == (want_idx, want_st), args
        cr = [B.TensorRec.make(r["base"], r["shape"], r["elem"], [0]) for r in recs]
        ca = [B.KernelArg.make(a["base"], a["shape"], a["alias_group"]) for a in args]
        assert B.resolve_args(cr, ca) == (want_idx, want_st), args


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
