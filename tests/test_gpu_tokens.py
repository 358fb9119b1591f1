"""Token mode (per-token block cipher with nonce, end-of-sequence marker) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu


def _run(n, n_users, seed, with_missing_key=True):
    rng = np.random.default_rng(W.SEED_BASE + 40 + seed)
    ids = np.arange(n_users, dtype=np.int32)
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16)
    eos = 2
    toks = rng.integers(0, 32000, size=n, dtype=np.uint64)          # vocabulary-sized ids in 64-bit tokens
    toks[rng.random(n) < 0.02] = eos
    toks[rng.random(n) < 0.01] = np.uint64(2**64 - 1)
    nonces = rng.integers(0, 2**64, size=n, dtype=np.uint64)
    owners = rng.integers(0, n_users, size=n).astype(np.int32)
    max_users = n_users + 2
    if with_missing_key and n > 3:
        owners[1], owners[2], owners[3] = n_users, -1, max_users + 5      # no key, parameter id, out of range
    ctx = binding.Ctx(max_users)
    ctx.set_keys(ids, keys)
    d = lambda a: torch.from_numpy(a).cuda()
    out = torch.full((max(n, 1), 16), 0x5A, dtype=torch.uint8, device="cuda")
    st = torch.full((max(n, 1),), 77, dtype=torch.int32, device="cuda")
    ctx.tok_encrypt(d(toks.view(np.int64)), d(nonces.view(np.int64)), d(owners), eos, out, st)
    torch.cuda.synchronize()
    ref_ct, ref_st = gcm.tok_encrypt(toks, nonces, owners, eos, ids, keys, max_users)
    assert np.array_equal(out[:n].cpu().numpy(), ref_ct)
    assert np.array_equal(st[:n].cpu().numpy().astype(np.uint32), ref_st)
    t_out = torch.full((max(n, 1),), -1, dtype=torch.int64, device="cuda")
    n_out = torch.full((max(n, 1),), -1, dtype=torch.int64, device="cuda")
    claimed = owners.copy()
    if n > 10:
        claimed[7] = (claimed[7] + 1) % n_users                    # a wrong claim: another token comes out
    ctx.tok_decrypt(out, d(claimed), eos, t_out, st, nonces_out=n_out)
    torch.cuda.synchronize()
    rt, rn, rst = gcm.tok_decrypt(ref_ct, claimed, eos, ids, keys, max_users)
    assert np.array_equal(t_out[:n].cpu().numpy().view(np.uint64), rt)
    assert np.array_equal(n_out[:n].cpu().numpy().view(np.uint64), rn)
    assert np.array_equal(st[:n].cpu().numpy().astype(np.uint32), rst)
    good = (rst == 0) & (claimed == owners)
    assert np.array_equal(rt[good], toks[good])
    if n > 10 and toks[7] != eos:
        assert rt[7] != toks[7]
    ctx.tok_decrypt(out, d(claimed), eos, t_out, st)              # nonces are optional
    torch.cuda.synchronize()
    assert np.array_equal(t_out[:n].cpu().numpy().view(np.uint64), rt)
    ctx.close()


@pytest.mark.parametrize("n", [1, 2, 127, 128, 129, 256, 100003])
def test_token_round_trip_matches_oracle(n):
    _run(n, 16, n % 7)


def test_decode_step_and_prefill_batch_shapes():
    _run(256, 256, 1, with_missing_key=False)        # one sampled token per user of a decode step
    _run(131328, 512, 2)                             # the mixed batch of config 5: 256 x 512 + 256 tokens
