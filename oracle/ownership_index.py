"""Two-level ownership index and rule steps (1)-(3), by brute force (test infrastructure only).

Paper sec. 4.2: a tensor record holds base address, shape, element size and the
ownership-related dimensions; an ownership record maps the subscripts of those dimensions to
an owner.  Paper sec. 4.3: a rule first finds the records of the accessed tensors by base
address, then checks shapes, then checks that tensors occupy distinct memory unless meant
to alias.  Everything here enumerates bytes or elements explicitly with numpy.
"""
from __future__ import annotations

import numpy as np

ARG_OK, ARG_UNKNOWN, ARG_SHAPE, ARG_ALIAS = 0, 1, 2, 4


def resolve_args(recs, args):
    """recs: list of dict(base, shape, elem); args: list of dict(base, shape, alias_group)."""
    idx, st = [], []
    for a in args:
        k = next((i for i, r in enumerate(recs) if r["base"] == a["base"]), -1)
        idx.append(k)
        if k < 0:
            st.append(ARG_UNKNOWN)
        else:
            st.append(ARG_OK if tuple(recs[k]["shape"]) == tuple(a["shape"]) else ARG_SHAPE)
    for i in range(len(args)):
        for j in range(i + 1, len(args)):
            if idx[i] < 0 or idx[j] < 0:
                continue
            ri, rj = recs[idx[i]], recs[idx[j]]
            bytes_i = set(range(ri["base"], ri["base"] + int(np.prod(ri["shape"])) * ri["elem"]))
            bytes_j = range(rj["base"], rj["base"] + int(np.prod(rj["shape"])) * rj["elem"])
            overlap = any(b in bytes_i for b in (bytes_j[0], bytes_j[-1])) or \
                (bytes_j[0] <= ri["base"] <= bytes_j[-1])
            intended = args[i]["alias_group"] != 0 and args[i]["alias_group"] == args[j]["alias_group"]
            if overlap and not intended:
                st[i] |= ARG_ALIAS
                st[j] |= ARG_ALIAS
    return idx, st


def slice_byte_offsets(shape, elem, lo, hi):
    """Byte offsets (from the tensor base) of the slice [lo, hi), in row-major order."""
    total = int(np.prod(shape)) * elem
    offs = np.arange(total, dtype=np.int64).reshape(tuple(shape) + (elem,))
    sl = tuple(slice(int(l), int(h)) for l, h in zip(lo, hi))
    return offs[sl].reshape(-1)


def slice_runs(shape, elem, lo, hi):
    """(run_bytes, page numbers): maximal equal-length contiguous runs of the slice."""
    b = slice_byte_offsets(shape, elem, lo, hi)
    breaks = np.nonzero(np.diff(b) != 1)[0] + 1
    starts = np.concatenate([[0], breaks])
    lens = np.diff(np.concatenate([starts, [b.size]]))
    assert (lens == lens[0]).all()
    run = int(lens[0])
    first = b[starts]
    assert (first % run == 0).all()
    return run, (first // run).astype(np.int32)


def expand_owners(shape, elem, odims, owners_level2, run_bytes):
    """One label per run of run_bytes bytes: the label all its bytes share, else CONFLICT (-3)."""
    oshape = [shape[d] for d in odims]
    lvl2 = np.asarray(owners_level2, dtype=np.int32).reshape(oshape)
    view = [shape[d] if d in odims else 1 for d in range(len(shape))]
    full = np.broadcast_to(lvl2.reshape(view), shape).reshape(-1)          # label of every element
    per_byte = np.repeat(full, elem)
    runs = per_byte.reshape(-1, run_bytes)
    same = (runs == runs[:, :1]).all(axis=1)
    return np.where(same, runs[:, 0], -3).astype(np.int32)
