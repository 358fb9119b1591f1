"""Pins for the label oracle: lattice laws, the paper's scenarios, and brute-force taint.

The brute force is the element-level tracking the paper contrasts itself with (sec. 4.1,
insight 1): toy versions of the kernels run over arrays whose elements carry *sets* of
owners, every arithmetic result taking the union of its operands' sets.  Collapsing each
output segment's set must give what the segment-level rule gives.
"""
import itertools

import numpy as np

from oracle import labels as L

P, N, C = L.PARAM, L.NONE, L.CONFLICT


def test_join_is_a_semilattice_with_param_as_identity():
    vals = [P, N, C, 0, 1, 2]
    for a, b, c in itertools.product(vals, repeat=3):
        assert L.join(a, b) == L.join(b, a)
        assert L.join(L.join(a, b), c) == L.join(a, L.join(b, c))
    for a in vals:
        assert L.join(a, P) == (a if a > N else C)
        assert L.join(a, a) == (a if a > N else C)
    assert L.join(0, 1) == C and L.join(N, 0) == C and L.join(3, 3) == 3
    # order independence == "no NONE/CONFLICT, and min == max over user labels"
    rng = np.random.default_rng(0)
    for _ in range(200):
        ls = rng.choice([P, N, 0, 0, 1, P], size=rng.integers(1, 6)).tolist()
        users = [l for l in ls if l >= 0]
        expect = C if any(l <= N for l in ls) else (P if not users else (users[0] if min(users) == max(users) else C))
        assert L.join_all(ls) == expect
        assert L.join_all(reversed(ls)) == expect


# ---- element-level taint brute force ---------------------------------------------

def _collapse(sets):
    """Label of a segment from the union of its elements' owner sets."""
    u = set().union(*sets)
    if N in u or C in u:
        return C
    u.discard(P)
    if not u:
        return P
    return u.pop() if len(u) == 1 else C


def _tainted(labels_per_row, width):
    return [[{int(l)} for _ in range(width)] for l in labels_per_row]


def test_rowwise_matches_taint_of_add_bias_relu_matmul_argmax_residual():
    rng = np.random.default_rng(1)
    B, H, H2 = 6, 5, 3
    for trial in range(30):
        rows = rng.choice([0, 1, 2, P, N], size=B, p=[.3, .3, .2, .1, .1]).astype(np.int32)
        res = rows.copy()
        if trial % 3 == 0:
            res[rng.integers(0, B)] = 7                         # residual row of another user
        bias_label = P if trial % 4 else 1                       # a "bias" that is user data
        I, R = _tainted(rows, H), _tainted(res, H)
        bias = [{bias_label} for _ in range(H)]
        Wm = [[{P} for _ in range(H2)] for _ in range(H)]
        # AddBias + ReLU: O[i][j] = relu(I[i][j] + b[j])
        add_bias = [[I[i][j] | bias[j] for j in range(H)] for i in range(B)]
        out, viol = L.propagate(L.ROWWISE, [rows, np.array([bias_label], np.int32)], B, param_mask=0b10)
        for i in range(B):
            expect = _collapse(add_bias[i])
            if bias_label != P:
                assert out[i] == C                              # step (4): parameter operand mislabelled
            else:
                assert out[i] == expect
        assert viol[0] == (out == C).sum()
        # MatrixMultiply: O[i][k] = sum_j I[i][j] * W[j][k]
        mm = [[set().union(*[I[i][j] | Wm[j][k] for j in range(H)]) for k in range(H2)] for i in range(B)]
        out, _ = L.propagate(L.ROWWISE, [rows, np.array([P], np.int32)], B, param_mask=0b10)
        assert [int(o) for o in out] == [_collapse(mm[i]) for i in range(B)]
        # FindMax: O[i] = argmax_j I[i][j]
        am = [[set().union(*I[i])] for i in range(B)]
        out, _ = L.propagate(L.ROWWISE, [rows], B)
        assert [int(o) for o in out] == [_collapse(am[i]) for i in range(B)]
        # AddResidual: O[i][j] = I[i][j] + R[i][j]
        ar = [[I[i][j] | R[i][j] for j in range(H)] for i in range(B)]
        out, _ = L.propagate(L.ROWWISE, [rows, res], B)
        assert [int(o) for o in out] == [_collapse(ar[i]) for i in range(B)]


def test_rowwise_is_independent_of_hidden_size():
    rows = np.array([0, 1, 1, 2], np.int32)
    a, _ = L.propagate(L.ROWWISE, [rows, np.array([P], np.int32)], 4, param_mask=2)
    assert a.tolist() == rows.tolist()          # one label per row whatever the row width


def test_segreduce_matches_taint_of_paged_attention_and_flags_redirected_block():
    rng = np.random.default_rng(2)
    n_req, n_blocks, D = 4, 10, 3
    # Alice = request 0 (user 0), Bob = request 1 (user 1) ...; one query token per request
    q_owner = np.arange(n_req, dtype=np.int32)
    kv_owner = np.array([0, 0, 1, 1, 1, 2, 2, 3, 3, N], dtype=np.int32)
    tables = [[0, 1], [2, 3, 4], [5, 6], [7, 8]]

    def run(tabs):
        seg_ptr = np.arange(n_req + 1, dtype=np.int32)
        src_ptr = np.concatenate([[0], np.cumsum([len(t) for t in tabs])]).astype(np.int32)
        src_idx = np.array([b for t in tabs for b in t], dtype=np.int32)
        out, viol = L.propagate(L.SEGREDUCE, [q_owner, kv_owner], n_req, seg_ptr=seg_ptr, src_ptr=src_ptr,
                                src_idx=src_idx)
        # brute force: out[r][d] = sum over blocks, tokens of softmax(q.k) * v
        Q = _tainted(q_owner, D)
        KV = _tainted(kv_owner, D)
        expect = []
        for r in range(n_req):
            acc = [set() for _ in range(D)]
            for b in tabs[r]:
                score = set().union(*Q[r]) | set().union(*KV[b])
                for d in range(D):
                    acc[d] |= score | KV[b][d]
            expect.append(_collapse(acc))
        assert [int(o) for o in out] == expect
        return out, viol

    out, viol = run(tables)
    assert out.tolist() == [0, 1, 2, 3] and viol.tolist() == [0, 0xFFFFFFFF]
    # the confused-deputy attack of paper sec. 2.2: Bob's block table is redirected to Alice's block
    attacked = [list(t) for t in tables]
    attacked[1][1] = 0
    out, viol = run(attacked)
    assert out.tolist() == [0, C, 2, 3] and viol.tolist() == [1, 1]
    # reading a block nobody owns is a violation as well (sec. 4.2, unowned memory)
    attacked = [list(t) for t in tables]
    attacked[3].append(9)
    out, viol = run(attacked)
    assert out[3] == C and viol.tolist() == [1, 3]


def test_segreduce_cost_scales_with_blocks_not_width():
    # a prefill chunk: all tokens of a request share the request's joined label
    tok = np.array([0, 0, 0, 1, 1], np.int32)
    kv = np.array([0, 1], np.int32)
    out, _ = L.propagate(L.SEGREDUCE, [tok, kv], 5, seg_ptr=np.array([0, 3, 5], np.int32),
                         src_ptr=np.array([0, 1, 2], np.int32), src_idx=np.array([0, 1], np.int32))
    assert out.tolist() == [0, 0, 0, 1, 1]


def test_identity_and_broadcast_match_taint_of_copy_and_gather():
    rng = np.random.default_rng(3)
    src = rng.choice([0, 1, 2, P, N, C], size=12).astype(np.int32)
    out, viol = L.propagate(L.IDENTITY, [src], 12)
    expect = [_collapse([{int(l)}]) for l in src]
    assert out.tolist() == expect and viol[0] == expect.count(C)
    gather = rng.integers(-1, 13, size=20).astype(np.int32)
    out, viol = L.propagate(L.BROADCAST, [src], 20, gather=gather)
    expect = [_collapse([{int(src[g])}]) if 0 <= g < 12 else C for g in gather]
    assert out.tolist() == expect
    first = expect.index(C) if C in expect else 0xFFFFFFFF
    assert viol.tolist() == [expect.count(C), first]


def test_rules_read_a_snapshot_when_aliased():
    m = np.array([0, 1, 2, 3], np.int32)
    out, _ = L.propagate(L.BROADCAST, [m], 4, gather=np.array([3, 2, 1, 0], np.int32))
    assert out.tolist() == [3, 2, 1, 0]


def test_swap_space_keeps_ownership_with_the_blocks():
    om = np.array([0, 0, 1, 1, 2, N, N, N], np.int32)
    saved, viol = L.swap_out(om, [2, 3, 0])                       # Bob's two blocks and one of Alice's leave
    assert saved.tolist() == [1, 1, 0] and viol.tolist() == [0, 0xFFFFFFFF]
    assert om.tolist() == [N, 0, N, N, 2, N, N, N]                # freed slots are unreadable
    viol = L.swap_in(om, [6, 7, 5], saved)                        # they come back to other slots
    assert viol.tolist() == [0, 0xFFFFFFFF] and om.tolist() == [N, 0, N, N, 2, 0, 1, 1]
    viol = L.swap_in(om, [4, 9], np.array([1, 1], np.int32))      # onto a live block, and out of range
    assert viol.tolist() == [2, 0] and om[4] == C


def test_segreduce_with_a_malformed_table_rejects_the_whole_launch():
    """Hand-built: index arrays that are no valid CSR description make every output CONFLICT."""
    in0 = np.array([1, 1, 2, 2, 2, 3], dtype=np.int32)
    in1 = np.array([1, 2, 3], dtype=np.int32)
    good = dict(seg_ptr=[0, 2, 5, 6], src_ptr=[0, 1, 2, 3], src_idx=[0, 1, 2])
    out, viol = L.propagate(L.SEGREDUCE, [in0, in1], 6, **good)
    assert out.tolist() == [1, 1, 2, 2, 2, 3] and viol.tolist() == [0, 0xFFFFFFFF]
    all_conflict = [L.CONFLICT] * 6
    for bad in (dict(good, seg_ptr=[0, 5, 2, 6]),            # decreasing: two requests would claim rows 2..4
                dict(good, seg_ptr=[0, 2, 5, 7]),            # runs past the outputs
                dict(good, seg_ptr=[-1, 2, 5, 6]),           # negative start
                dict(good, src_ptr=[0, 1, 2, 4]),            # runs past src_idx
                dict(good, src_ptr=[0, 2, 1, 3]),            # decreasing
                dict(good, src_ptr=[-2, 1, 2, 3])):
        out, viol = L.propagate(L.SEGREDUCE, [in0, in1], 6, **bad)
        assert out.tolist() == all_conflict and viol.tolist() == [6, 0], bad
    assert L.csr_ok([0, 0, 0], 0) and L.csr_ok([3], 3) and not L.csr_ok([4], 3) and not L.csr_ok([], 3)
    # a valid table that leaves outputs uncovered is not malformed: only those outputs conflict
    out, viol = L.propagate(L.SEGREDUCE, [in0, in1], 6, seg_ptr=[1, 2, 5], src_ptr=[0, 1, 2], src_idx=[0, 1])
    assert out.tolist() == [L.CONFLICT, 1, 2, 2, 2, L.CONFLICT] and viol.tolist() == [2, 0]
