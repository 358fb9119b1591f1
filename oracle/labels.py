"""Ownership labels and flow rules, written out from the paper's description.

Test infrastructure only.  Labels are int32: a user id >= 0, PARAM (-1, the special
id of model parameters, paper sec. 4.2), NONE (-2, memory no record covers, which may
not be read, sec. 4.2 "Unowned memory") and CONFLICT (-3, an output whose sources do
not share one owner).

A rule follows step (5) of "Generating IFT rules" (paper sec. 4.3): for every
subscript, the non-parameter sources must share one owner, which the destinations
receive; step (4): operands declared as parameters must be labelled PARAM.  The paper
rejects the whole launch on a violation (sec. 4.1, insight 3); here every output is
still written, violations are marked CONFLICT and counted, and committing is the
caller's decision.  All rules read a snapshot of their inputs.
"""
from __future__ import annotations

import numpy as np

PARAM, NONE, CONFLICT = -1, -2, -3
IDENTITY, ROWWISE, SEGREDUCE, BROADCAST = 0, 1, 2, 3


def join(a: int, b: int) -> int:
    """Least upper bound of two labels: PARAM is neutral, equal users stay, the rest conflicts."""
    if a <= NONE or b <= NONE:
        return CONFLICT
    if a == PARAM:
        return b
    if b == PARAM:
        return a
    return a if a == b else CONFLICT


def join_all(labels) -> int:
    acc = PARAM
    for l in labels:
        acc = join(acc, int(l))
    return acc


def _viol(out: np.ndarray) -> np.ndarray:
    bad = np.nonzero(out == CONFLICT)[0]
    return np.array([bad.size, bad[0] if bad.size else 0xFFFFFFFF], dtype=np.uint32)


def csr_ok(ptr, limit: int) -> bool:
    """ptr[0] >= 0, ptr non-decreasing, ptr[-1] <= limit."""
    p = [int(x) for x in ptr]
    if len(p) == 0 or p[0] < 0 or p[-1] > limit:
        return False
    for k in range(1, len(p)):
        if p[k] < p[k - 1]:
            return False
    return True


def propagate(kind: int, inputs, n_out: int, *, param_mask: int = 0, seg_ptr=None, src_ptr=None,
              src_idx=None, gather=None):
    """Apply one flow rule; returns (out int32[n_out], viol uint32[2] = count, first index)."""
    ins = [np.array(m, dtype=np.int32, copy=True) for m in inputs]     # snapshot
    out = np.empty(n_out, dtype=np.int32)
    if kind == IDENTITY:
        # copy kernels: the destination unit takes the source unit's owner
        for j in range(n_out):
            out[j] = join(int(ins[0][j]), PARAM)
    elif kind == ROWWISE:
        # row j of the output depends on row j of every row operand; parameter operands
        # (bit k of param_mask) are whole tensors that must carry the PARAM label
        params_ok = all(int(ins[k][0]) == PARAM for k in range(len(ins)) if (param_mask >> k) & 1)
        rows = [k for k in range(len(ins)) if not (param_mask >> k) & 1]
        for j in range(n_out):
            out[j] = join_all(ins[k][j] for k in rows) if params_ok else CONFLICT
    elif kind == SEGREDUCE:
        # decoding-stage attention: the outputs of request s depend on its own rows and on
        # every KV block its block table names (paper sec. 7.2: the rule walks each block)
        out[:] = CONFLICT
        # The index arrays come from the untrusted framework (paper sec. 4.3: the rule checks the
        # arguments of the launch it is given).  Reading taken: a table that is not a valid CSR
        # description (a pointer array that is negative, decreasing, or that runs past what it
        # indexes) rejects the launch as a whole, i.e. every output is CONFLICT.
        if not (csr_ok(seg_ptr, n_out) and csr_ok(src_ptr, len(src_idx))):
            return out, _viol(out)
        covered = np.zeros(n_out, dtype=bool)
        for s in range(len(seg_ptr) - 1):
            srcs = [ins[0][t] for t in range(seg_ptr[s], seg_ptr[s + 1])]
            for e in range(src_ptr[s], src_ptr[s + 1]):
                b = int(src_idx[e])
                srcs.append(ins[1][b] if 0 <= b < len(ins[1]) else NONE)
            m = join_all(srcs)
            for t in range(seg_ptr[s], seg_ptr[s + 1]):
                out[t] = m
                covered[t] = True
        out[~covered] = CONFLICT      # an output no request covers has no defined source
    elif kind == BROADCAST:
        for j in range(n_out):
            g = int(gather[j])
            out[j] = join(int(ins[0][g]), PARAM) if 0 <= g < len(ins[0]) else CONFLICT
    else:
        raise ValueError("unknown rule kind")
    return out, _viol(out)


def swap_out(owner_map, units):
    """Secure swap space (paper sec. 4.5): save the labels of the listed units and unown them.

    Returns (saved int32[n], viol uint32[2]); owner_map is updated in place."""
    saved = np.empty(len(units), dtype=np.int32)
    bad = []
    for i, u in enumerate(units):
        u = int(u)
        if u < 0 or u >= len(owner_map):
            saved[i] = CONFLICT
            bad.append(i)
            continue
        saved[i] = owner_map[u]
        owner_map[u] = NONE
    return saved, np.array([len(bad), bad[0] if bad else 0xFFFFFFFF], dtype=np.uint32)


def swap_in(owner_map, units, saved):
    """Put saved labels back at the units the blocks return to; an occupied unit is a violation."""
    bad = []
    for i, u in enumerate(units):
        u = int(u)
        if u < 0 or u >= len(owner_map):
            bad.append(i)
            continue
        if owner_map[u] != NONE:
            owner_map[u] = CONFLICT
            bad.append(i)
        else:
            owner_map[u] = saved[i]
    return np.array([len(bad), bad[0] if bad else 0xFFFFFFFF], dtype=np.uint32)
