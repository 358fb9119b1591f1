"""GPU parity for the flow rules and for the mixed batch with tampering (config 5)."""
import numpy as np
import pytest
import torch

from oracle import labels as L
from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import (dev, gpu_decrypt, gpu_encrypt, make_ctx, np_, oracle_decrypt, oracle_encrypt, st_)

pytestmark = pytest.mark.gpu


def _rule(ctx, kind, ins, n_out, out=None, **kw):
    d_ins = [dev(np.asarray(m, dtype=np.int32)) if not torch.is_tensor(m) else m for m in ins]
    out = torch.full((n_out,), 12345, dtype=torch.int32, device="cuda") if out is None else out
    viol = torch.full((2,), 7, dtype=torch.int32, device="cuda")
    dk = {k: (dev(np.asarray(v, dtype=np.int32)) if v is not None else None) for k, v in kw.items() if k != "param_mask"}
    ctx.propagate_labels(kind, d_ins, out, viol, n_out=n_out, param_mask=kw.get("param_mask", 0), **dk)
    torch.cuda.synchronize()
    return np_(out), np_(viol).astype(np.uint32)


@pytest.fixture(scope="module")
def ctx():
    c = binding.Ctx(4)
    yield c
    c.close()


def test_pointwise_rules_match_oracle(ctx):
    rng = np.random.default_rng(21)
    for n in (1, 31, 32, 33, 1000, 70001):
        a = rng.choice([0, 1, 2, 3, L.PARAM, L.NONE, L.CONFLICT], size=n, p=[.3, .2, .2, .1, .1, .05, .05]).astype(np.int32)
        b = np.where(rng.random(n) < 0.9, a, rng.integers(0, 4, size=n)).astype(np.int32)
        out, viol = _rule(ctx, binding.RULE_IDENTITY, [a], n)
        ro, rv = L.propagate(L.IDENTITY, [a], n)
        assert np.array_equal(out, ro) and np.array_equal(viol, rv)
        for pm, par in ((0b100, L.PARAM), (0b100, 1), (0, None)):
            ins = [a, b] + ([np.array([par], np.int32)] if par is not None else [])
            out, viol = _rule(ctx, binding.RULE_ROWWISE, ins, n, param_mask=pm)
            ro, rv = L.propagate(L.ROWWISE, ins, n, param_mask=pm)
            assert np.array_equal(out, ro) and np.array_equal(viol, rv)
        g = rng.integers(-2, n + 2, size=n + 5).astype(np.int32)
        out, viol = _rule(ctx, binding.RULE_BROADCAST, [a], n + 5, gather=g)
        ro, rv = L.propagate(L.BROADCAST, [a], n + 5, gather=g)
        assert np.array_equal(out, ro) and np.array_equal(viol, rv)


def test_broadcast_reads_a_snapshot_when_aliased(ctx):
    m = dev(np.arange(1000, dtype=np.int32))
    g = np.arange(1000, dtype=np.int32)[::-1].copy()
    out, viol = _rule(ctx, binding.RULE_BROADCAST, [m], 1000, out=m, gather=g)
    assert np.array_equal(out, g) and viol.tolist() == [0, 0xFFFFFFFF]


def test_segreduce_matches_oracle_including_attack_and_uncovered_outputs(ctx):
    rng = np.random.default_rng(22)
    n_req = 300
    ntok = rng.choice([1, 1, 1, 40, 513], size=n_req)
    head, tail = 3, 4                                   # outputs no request covers
    seg_ptr = (head + np.concatenate([[0], np.cumsum(ntok)])).astype(np.int32)
    n_out = int(seg_ptr[-1]) + tail
    tok = np.full(n_out, L.NONE, dtype=np.int32)
    for r in range(n_req):
        tok[seg_ptr[r]:seg_ptr[r + 1]] = r % 50
    nb = rng.integers(0, 70, size=n_req)
    src_ptr = np.concatenate([[0], np.cumsum(nb)]).astype(np.int32)
    kv_owner = np.repeat(np.arange(n_req) % 50, nb).astype(np.int32)
    src_idx = np.arange(kv_owner.size, dtype=np.int32)
    for e in rng.choice(src_idx.size, size=25, replace=False):        # redirected block-table entries
        src_idx[e] = rng.integers(-1, kv_owner.size + 1)
    tok[seg_ptr[7]] = L.PARAM
    out, viol = _rule(ctx, binding.RULE_SEGREDUCE, [tok, kv_owner], n_out, seg_ptr=seg_ptr, src_ptr=src_ptr, src_idx=src_idx)
    ro, rv = L.propagate(L.SEGREDUCE, [tok, kv_owner], n_out, seg_ptr=seg_ptr, src_ptr=src_ptr, src_idx=src_idx)
    assert np.array_equal(out, ro) and np.array_equal(viol, rv) and rv[0] > head + tail


def test_segreduce_with_malformed_index_arrays_rejects_the_launch(ctx):
    """Pointer arrays that are no valid CSR description (decreasing, negative, past the end) must end as
    CONFLICT on every output, never as a stray read or write; twice, with a good table in between."""
    rng = np.random.default_rng(23)
    n_out, n_req = 5000, 120
    cuts = np.sort(rng.choice(np.arange(1, n_out), size=n_req - 1, replace=False))
    seg_ptr = np.concatenate([[0], cuts, [n_out]]).astype(np.int32)
    nb = rng.integers(0, 9, size=n_req)
    src_ptr = np.concatenate([[0], np.cumsum(nb)]).astype(np.int32)
    kv = rng.integers(0, 4, size=int(src_ptr[-1]) + 3).astype(np.int32)
    src_idx = rng.integers(0, kv.size, size=int(src_ptr[-1])).astype(np.int32)
    tok = rng.integers(0, 4, size=n_out).astype(np.int32)

    def both(sp, srp):
        out, viol = _rule(ctx, binding.RULE_SEGREDUCE, [tok, kv], n_out, seg_ptr=sp, src_ptr=srp, src_idx=src_idx)
        ro, rv = L.propagate(L.SEGREDUCE, [tok, kv], n_out, seg_ptr=sp, src_ptr=srp, src_idx=src_idx)
        assert np.array_equal(out, ro) and np.array_equal(viol, rv)
        return rv

    good = both(seg_ptr, src_ptr)
    bad_tables = []
    sp = seg_ptr.copy(); sp[40], sp[41] = sp[41], sp[40]; bad_tables.append((sp, src_ptr))           # decreasing pair
    sp = seg_ptr.copy(); sp[-1] = n_out + 1000; bad_tables.append((sp, src_ptr))                     # past the outputs
    sp = seg_ptr.copy(); sp[0] = -5; bad_tables.append((sp, src_ptr))                                # negative start
    srp = src_ptr.copy(); srp[-1] += 7; bad_tables.append((seg_ptr, srp))                            # past src_idx
    srp = src_ptr.copy(); srp[10] = 2**31 - 1; bad_tables.append((seg_ptr, srp))                     # a huge entry in the middle
    for sp, srp in bad_tables:
        rv = both(sp, srp)
        assert rv.tolist() == [n_out, 0]
        assert both(seg_ptr, src_ptr).tolist() == good.tolist()                                      # the flag does not stick


def test_config5_rules_tamper_detection_and_reencrypt():
    w = W.config5(layers=2)
    x = w.extra
    ctx = make_ctx(w)
    T = x["T"]
    # --- the four flow rules in sequence on the token owner map -------------------------------
    cur = x["token_owner"].copy()
    d_cur = dev(cur)
    chain = [
        (binding.RULE_IDENTITY, L.IDENTITY, lambda m: [m], {}),
        (binding.RULE_ROWWISE, L.ROWWISE, lambda m: [m, np.array([L.PARAM], np.int32)], {"param_mask": 0b10}),
        (binding.RULE_SEGREDUCE, L.SEGREDUCE, lambda m: [m, x["kv_owner"]],
         {"seg_ptr": x["seg_ptr"], "src_ptr": x["src_ptr"], "src_idx": x["block_table"]}),
        (binding.RULE_BROADCAST, L.BROADCAST, lambda m: [m], {"gather": x["gather"]}),
    ]
    for gk, ok, mk, kw in chain:
        ins = mk(cur)
        out, viol = _rule(ctx, gk, ins, T, **kw)
        ro, rv = L.propagate(ok, ins, T, **kw)
        assert np.array_equal(out, ro) and np.array_equal(viol, rv) and rv[0] == 0
        cur = ro
    assert np.array_equal(cur, x["token_owner"])
    # the redirected block tables: exactly the attacked requests' tokens conflict
    ins = [x["token_owner"], x["kv_owner"]]
    kw = {"seg_ptr": x["seg_ptr"], "src_ptr": x["src_ptr"], "src_idx": x["block_table_attacked"]}
    out, viol = _rule(ctx, binding.RULE_SEGREDUCE, ins, T, **kw)
    ro, rv = L.propagate(L.SEGREDUCE, ins, T, **kw)
    assert np.array_equal(out, ro) and np.array_equal(viol, rv)
    bad_req = np.unique(np.searchsorted(x["seg_ptr"], np.nonzero(out == L.CONFLICT)[0], side="right") - 1)
    assert np.array_equal(bad_req, x["redirected_requests"])

    # --- export, tamper, import, re-export --------------------------------------------------
    buf = dev(w.buf)
    tags, st = gpu_encrypt(ctx, w, buf)
    ref_ct = w.buf.copy()
    ref_tags, ref_st = oracle_encrypt(w, ref_ct, ref_ct)
    assert not ref_st.any() and np.array_equal(st_(st), ref_st)
    assert np.array_equal(np_(tags), ref_tags) and np.array_equal(np_(buf), ref_ct)

    segs = w.segs.copy()
    bad_ct, bad_tags = ref_ct.copy(), ref_tags.copy()
    for s, kind, bit, tbit, wrong in zip(x["poisoned"], x["poison_kind"], x["poison_bit"], x["poison_tagbit"], x["poison_owner"]):
        if kind == 0:
            bad_ct[int(segs["offset"][s]) + bit // 8] ^= 1 << (bit % 8)
        elif kind == 1:
            bad_tags[s, tbit // 8] ^= 1 << (tbit % 8)
        else:
            segs["owner"][s] = wrong
    om = torch.full((w.owner_map.size,), L.NONE, dtype=torch.int32, device="cuda")
    d_ct = dev(bad_ct)
    st = gpu_decrypt(ctx, w, d_ct, dev(bad_tags), segs=segs, owner_map=om)
    om_ref = np.full(w.owner_map.size, L.NONE, dtype=np.int32)
    ref_pt = bad_ct.copy()
    ref_st = oracle_decrypt(w, ref_pt, ref_pt, bad_tags, segs=segs, owner_map=om_ref)
    flagged = np.nonzero(st_(st))[0]
    assert np.array_equal(flagged, x["poisoned"])                      # exactly the seeded 1 %
    assert np.array_equal(st_(st), ref_st) and np.array_equal(np_(d_ct), ref_pt) and np.array_equal(np_(om), om_ref)
    good = np.ones(len(segs), dtype=bool)
    good[x["poisoned"]] = False
    for s in np.nonzero(good)[0][:: max(1, len(segs) // 64)]:           # untouched segments carry the plaintext
        o, n = int(segs["offset"][s]), int(segs["len"][s])
        assert np.array_equal(ref_pt[o:o + n], w.buf[o:o + n])
    # re-export under fresh nonces with the labels the import recorded: poisoned segments are refused
    segs2 = W.bump_epoch(w.segs)
    tags2, st2 = gpu_encrypt(ctx, w, d_ct, None, segs=segs2, owner_map=np_(om))
    ref2 = ref_pt.copy()
    ref_tags2, ref_st2 = oracle_encrypt(w, ref2, ref2, segs=segs2, owner_map=om_ref)
    assert np.array_equal(st_(st2), ref_st2) and np.array_equal(np_(tags2), ref_tags2) and np.array_equal(np_(d_ct), ref2)
    assert np.array_equal(np.nonzero(ref_st2)[0], x["poisoned"]) and (ref_st2[x["poisoned"]] == 4).all()
    assert not np.array_equal(ref_tags2[good], ref_tags[good])
    ctx.close()


def test_swap_space_labels_match_oracle(ctx):
    rng = np.random.default_rng(23)
    n_units = 5000
    om = rng.choice([0, 1, 2, 3, L.NONE, L.PARAM], size=n_units, p=[.2, .2, .2, .2, .15, .05]).astype(np.int32)
    units = rng.permutation(n_units)[:1200].astype(np.int32)
    units[7], units[900] = -3, n_units + 4                        # bad list entries
    d_om, d_units = dev(om), dev(units)
    saved = torch.full((1200,), 77, dtype=torch.int32, device="cuda")
    viol = torch.full((2,), 5, dtype=torch.int32, device="cuda")
    ctx.labels_swap_out(d_om, d_units, saved, viol)
    torch.cuda.synchronize()
    ref_om = om.copy()
    ref_saved, ref_viol = L.swap_out(ref_om, units)
    assert np.array_equal(np_(saved), ref_saved) and np.array_equal(np_(viol).astype(np.uint32), ref_viol)
    assert np.array_equal(np_(d_om), ref_om)
    back = rng.permutation(n_units)[:1200].astype(np.int32)       # they return to other slots, some still occupied
    ctx.labels_swap_in(d_om, dev(back), saved, viol)
    torch.cuda.synchronize()
    ref_viol = L.swap_in(ref_om, back, ref_saved)
    assert np.array_equal(np_(d_om), ref_om) and np.array_equal(np_(viol).astype(np.uint32), ref_viol)
    assert ref_viol[0] > 0
