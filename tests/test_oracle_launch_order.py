"""Pins for the launch-order oracle: the legal and illegal orders the paper describes."""
import numpy as np

from oracle import launch_order as LO
from paper_2608_25431_b200 import workloads as W


def _trace(events, n_streams=2, n_segments=4):
    """events: ('L', stream, reads, writes) or ('S', stream)."""
    kind, stream, ptr, seg, wr = [], [], [0], [], []
    for ev in events:
        kind.append(0 if ev[0] == "L" else 1)
        stream.append(ev[1])
        if ev[0] == "L":
            for m in ev[2]:
                seg.append(m); wr.append(0)
            for m in ev[3]:
                seg.append(m); wr.append(1)
        ptr.append(len(seg))
    return LO.check(np.array(kind), np.array(stream), np.array(ptr), np.array(seg, dtype=np.int64),
                    np.array(wr, dtype=np.int64), n_streams, n_segments)


def test_read_of_in_flight_write_on_another_stream_is_flagged():
    # the paper's example: attention reads user A's KV block while a background stream overwrites it
    flags, summ = _trace([("L", 1, [], [0]), ("L", 0, [0], [1])])
    assert flags.tolist() == [0, LO.RAW] and summ.tolist() == [1, 1]
    flags, _ = _trace([("L", 1, [], [0]), ("S", 1), ("L", 0, [0], [1])])          # writer completed first
    assert flags.tolist() == [0, 0, 0]
    flags, _ = _trace([("L", 1, [], [0]), ("S", 0), ("L", 0, [0], [1])])          # wrong stream synchronised
    assert flags.tolist() == [0, 0, LO.RAW]
    flags, _ = _trace([("L", 0, [], [0]), ("L", 0, [0], [1])])                    # same stream: ordered anyway
    assert flags.tolist() == [0, 0]


def test_write_under_in_flight_read_and_write_write():
    flags, _ = _trace([("L", 0, [2], []), ("L", 1, [], [2])])
    assert flags.tolist() == [0, LO.WAR]
    flags, _ = _trace([("L", 0, [2], []), ("S", 0), ("L", 1, [], [2])])
    assert flags.tolist() == [0, 0, 0]
    flags, _ = _trace([("L", 0, [], [2]), ("L", 1, [], [2])])
    assert flags.tolist() == [0, LO.WAW]
    flags, _ = _trace([("L", 0, [2], [2]), ("L", 1, [2], [2])])                   # in-place kernels on two streams
    assert flags.tolist() == [0, LO.RAW | LO.WAR | LO.WAW]
    # readers on two streams: both must have completed before a third stream writes
    flags, _ = _trace([("L", 0, [1], []), ("L", 1, [1], []), ("S", 0), ("L", 2, [], [1])], n_streams=3)
    assert flags.tolist() == [0, 0, 0, LO.WAR]
    flags, _ = _trace([("L", 0, [1], []), ("L", 1, [1], []), ("S", 0), ("S", 1), ("L", 2, [], [1])], n_streams=3)
    assert flags.tolist() == [0, 0, 0, 0, 0]


def test_collective_buffer_order_is_legal():
    # writer on stream 1, transfer (reader) on stream 2 after it completed, next writer after the transfer completed
    flags, _ = _trace([("L", 1, [], [3]), ("S", 1), ("L", 2, [3], []), ("S", 2), ("L", 1, [], [3])], n_streams=3)
    assert not flags.any()
    flags, _ = _trace([("L", 1, [], [3]), ("S", 1), ("L", 2, [3], []), ("L", 1, [], [3])], n_streams=3)
    assert flags.tolist() == [0, 0, 0, LO.WAR]


def test_generated_traces_are_clean_without_planted_races_and_flagged_with():
    t = W.launch_trace(400, 64, 3, race_frac=0.0)
    flags, summ = LO.check(t["kind"], t["stream"], t["acc_ptr"], t["acc_seg"], t["acc_write"], 3, 64)
    assert not flags.any() and summ.tolist() == [0, 0xFFFFFFFF]
    t = W.launch_trace(400, 64, 3, race_frac=0.3)
    flags, summ = LO.check(t["kind"], t["stream"], t["acc_ptr"], t["acc_seg"], t["acc_write"], 3, 64)
    assert summ[0] > 0 and flags[summ[1]] != 0 and not flags[: summ[1]].any()
    seg_ptr, seg_ev, seg_wr = W.trace_by_segment(t["acc_ptr"], t["acc_seg"], t["acc_write"], 64)
    assert seg_ptr[-1] == len(t["acc_seg"])
    for m in range(64):
        assert (np.diff(seg_ev[seg_ptr[m]:seg_ptr[m + 1]]) >= 0).all()          # launch order inside a segment
