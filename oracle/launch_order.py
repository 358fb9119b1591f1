"""Multi-stream launch-order check (paper sec. 4.4, "Concurrency control"), plain Python.

Test infrastructure only.  The monitor keeps, per memory segment, the last writer kernel
and the last reader kernels, each a (stream, sequence) pair, and per stream the last
completed kernel; a kernel counts as completed once a synchronisation operation on its
stream has been seen after its launch.  Two invariants prevent read-write races, a third
handles write-write races "in a similar manner":
  - launching a reader of M: the last writer of M, if on another stream, must have completed;
  - launching a writer of M: every last reader of M on another stream must have completed,
    and so must the last writer of M if it is on another stream.
The trace is walked in launch order; a launch that breaks an invariant is flagged (the
paper's monitor would hold it back), and the records are updated as if it had run.
"""
from __future__ import annotations

import numpy as np

RAW, WAR, WAW = 1, 2, 4          # read of an in-flight write, write under an in-flight read, write-write


def check(kind, stream, acc_ptr, acc_seg, acc_write, n_streams, n_segments):
    """kind[e]: 0 launch, 1 synchronisation of stream[e]; launch e accesses acc_seg[acc_ptr[e]:acc_ptr[e+1]].

    Returns (flags uint32[n_events], summary uint32[2] = flagged launches, first flagged event).
    """
    n = len(kind)
    last_sync = [-1] * n_streams              # latest synchronisation seen on each stream
    last_writer = [-1] * n_segments
    last_reader = [[-1] * n_streams for _ in range(n_segments)]
    flags = np.zeros(n, dtype=np.uint32)

    def completed(k):                         # k: event index of an earlier launch
        return last_sync[int(stream[k])] > k

    for e in range(n):
        s = int(stream[e])
        if kind[e] == 1:
            last_sync[s] = e
            continue
        f = 0
        for a in range(acc_ptr[e], acc_ptr[e + 1]):
            m, w = int(acc_seg[a]), int(acc_write[a])
            lw = last_writer[m]
            if lw >= 0 and int(stream[lw]) != s and not completed(lw):
                f |= WAW if w else RAW
            if w:
                for s2 in range(n_streams):
                    lr = last_reader[m][s2]
                    if s2 != s and lr >= 0 and not completed(lr):
                        f |= WAR
        for a in range(acc_ptr[e], acc_ptr[e + 1]):
            m, w = int(acc_seg[a]), int(acc_write[a])
            if w:
                last_writer[m] = e
            else:
                last_reader[m][s] = e
        flags[e] = f
    bad = np.nonzero(flags)[0]
    return flags, np.array([bad.size, bad[0] if bad.size else 0xFFFFFFFF], dtype=np.uint32)
