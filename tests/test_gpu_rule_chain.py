"""The fused rule chain gives what the oracle's rules give when applied one after another."""
import numpy as np
import pytest
import torch

from oracle import labels as L
from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import dev, np_

pytestmark = pytest.mark.gpu

OKIND = {binding.RULE_IDENTITY: L.IDENTITY, binding.RULE_ROWWISE: L.ROWWISE,
         binding.RULE_SEGREDUCE: L.SEGREDUCE, binding.RULE_BROADCAST: L.BROADCAST}
INDEX_KEYS = ("seg_ptr", "src_ptr", "src_idx", "gather")


@pytest.fixture(scope="module")
def ctx():
    c = binding.Ctx(4)
    yield c
    c.close()


def run_chain(ctx, stages, maps):
    """stages: list of (kind, [input names or arrays], output name, n_out, kwargs of numpy index arrays).
    maps: name -> numpy int32 array (the initial contents; outputs must be present with their size).
    Returns (device results by name, viol) and (oracle results by name, viol)."""
    d_maps = {k: dev(v.astype(np.int32)) for k, v in maps.items()}
    o_maps = {k: v.astype(np.int32).copy() for k, v in maps.items()}
    rules, o_viol = [], []
    for kind, ins, out, n_out, kw in stages:
        r = {"kind": kind, "in_maps": [d_maps[i] for i in ins], "out_map": d_maps[out], "n_out": n_out,
             "param_mask": kw.get("param_mask", 0)}
        for k in INDEX_KEYS:
            if kw.get(k) is not None:
                r[k] = dev(np.asarray(kw[k], dtype=np.int32))
        rules.append(r)
        ro, rv = L.propagate(OKIND[kind], [o_maps[i] for i in ins], n_out, **kw)
        o_maps[out][:n_out] = ro
        o_viol.append(rv)
    viol = torch.full((2 * len(stages),), 7, dtype=torch.int32, device="cuda")
    ctx.propagate_chain(rules, viol)
    torch.cuda.synchronize()
    return {k: np_(v) for k, v in d_maps.items()}, np_(viol).astype(np.uint32), o_maps, np.concatenate(o_viol)


def test_config5_four_rules_in_one_launch(ctx):
    x = W.config5(layers=2).extra
    T = x["T"]
    for table, expect_conflicts in ((x["block_table"], False), (x["block_table_attacked"], True)):
        maps = {"tok": x["token_owner"], "a": np.zeros(T), "b": np.zeros(T), "c": np.zeros(T), "d": np.zeros(T),
                "w": np.array([L.PARAM]), "kv": x["kv_owner"]}
        stages = [
            (binding.RULE_IDENTITY, ["tok"], "a", T, {}),
            (binding.RULE_ROWWISE, ["a", "w"], "b", T, {"param_mask": 0b10}),
            (binding.RULE_SEGREDUCE, ["b", "kv"], "c", T, {"seg_ptr": x["seg_ptr"], "src_ptr": x["src_ptr"], "src_idx": table}),
            (binding.RULE_BROADCAST, ["c"], "d", T, {"gather": x["gather"]}),
        ]
        before = ctx.launch_count()
        got, viol, ref, rviol = run_chain(ctx, stages, maps)
        assert ctx.launch_count() == before + 1
        for k in maps:
            assert np.array_equal(got[k], ref[k]), k
        assert np.array_equal(viol, rviol)
        if expect_conflicts:
            assert viol[4] > 0 and viol[6] > 0                  # the attacked requests, and what the gather spreads
            bad_req = np.unique(np.searchsorted(x["seg_ptr"], np.nonzero(got["c"] == L.CONFLICT)[0], side="right") - 1)
            assert np.array_equal(bad_req, x["redirected_requests"])
        else:
            assert not viol[0::2].any() and np.array_equal(got["d"], x["token_owner"])


def test_random_chains_with_in_place_stages_and_ragged_sizes(ctx):
    rng = np.random.default_rng(77)
    for n in (1, 33, 8191, 8192, 8193, 100_003):
        a = rng.choice([0, 1, 2, 3, L.PARAM, L.NONE, L.CONFLICT], size=n, p=[.3, .2, .2, .1, .1, .05, .05])
        b = np.where(rng.random(n) < 0.95, a, rng.integers(0, 4, size=n))
        n_req = max(1, n // 37)
        cuts = np.sort(rng.choice(np.arange(n + 1), size=n_req + 1, replace=(n + 1 < n_req + 1)))
        nb = rng.integers(0, 5, size=n_req)
        src_ptr = np.concatenate([[0], np.cumsum(nb)])
        src_idx = rng.integers(-1, n + 1, size=int(src_ptr[-1]))
        g = rng.integers(-1, n + 1, size=n)
        maps = {"a": a, "b": b, "t": np.zeros(n), "u": np.zeros(n), "p": np.array([L.PARAM])}
        stages = [
            (binding.RULE_ROWWISE, ["a", "b", "p"], "a", n, {"param_mask": 0b100}),      # in place
            (binding.RULE_BROADCAST, ["a"], "t", n, {"gather": g}),
            (binding.RULE_SEGREDUCE, ["t", "b"], "t", n, {"seg_ptr": cuts, "src_ptr": src_ptr, "src_idx": src_idx}),  # in0 in place
            (binding.RULE_IDENTITY, ["t"], "u", n, {}),
            (binding.RULE_ROWWISE, ["u", "a"], "u", n, {}),
        ]
        got, viol, ref, rviol = run_chain(ctx, stages, maps)
        for k in maps:
            assert np.array_equal(got[k], ref[k]), (n, k)
        assert np.array_equal(viol, rviol), n


def test_chain_with_a_malformed_reduction_table_rejects_that_rule_only(ctx):
    rng = np.random.default_rng(78)
    n = 3000
    a = rng.integers(0, 3, size=n)
    cuts = np.sort(rng.choice(np.arange(n + 1), size=41, replace=False))
    src_ptr = np.arange(41) * 2
    src_idx = rng.integers(0, n, size=80)
    bad_cuts = cuts.copy()
    bad_cuts[5], bad_cuts[6] = bad_cuts[6], bad_cuts[5]
    for seg_ptr in (bad_cuts, cuts, bad_cuts, cuts):
        maps = {"a": a, "t": np.zeros(n), "u": np.zeros(n)}
        stages = [
            (binding.RULE_IDENTITY, ["a"], "t", n, {}),
            (binding.RULE_SEGREDUCE, ["t", "a"], "u", n, {"seg_ptr": seg_ptr, "src_ptr": src_ptr, "src_idx": src_idx}),
            (binding.RULE_IDENTITY, ["u"], "t", n, {}),
        ]
        got, viol, ref, rviol = run_chain(ctx, stages, maps)
        for k in maps:
            assert np.array_equal(got[k], ref[k]), k
        assert np.array_equal(viol, rviol)
        if seg_ptr is bad_cuts:
            assert viol[2] == n and viol[3] == 0 and (got["u"] == L.CONFLICT).all()


def test_chain_argument_errors(ctx):
    m = dev(np.arange(64, dtype=np.int32))
    g = dev(np.arange(64, dtype=np.int32))
    viol = torch.zeros(32, dtype=torch.int32, device="cuda")
    ident = {"kind": binding.RULE_IDENTITY, "in_maps": [m], "out_map": m}
    with pytest.raises(binding.GiftError):                   # more rules than a chain holds
        ctx.propagate_chain([ident] * 9, viol)
    with pytest.raises(binding.GiftError):                   # gather source overlaps the output
        ctx.propagate_chain([{"kind": binding.RULE_BROADCAST, "in_maps": [m], "out_map": m, "gather": g}], viol)
    before = ctx.launch_count()
    ctx.propagate_chain([], viol)                            # nothing to do: no launch
    assert ctx.launch_count() == before
    torch.cuda.synchronize()
    assert np.array_equal(np_(m), np.arange(64))
