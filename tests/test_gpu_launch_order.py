"""The launch-order check on the GPU against the sequential oracle."""
import numpy as np
import pytest
import torch

from oracle import launch_order as LO
from paper_2608_25431_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Ctx(4)
    yield c
    c.close()


def _gpu(ctx, t):
    seg_ptr, seg_ev, seg_wr = W.trace_by_segment(t["acc_ptr"], t["acc_seg"], t["acc_write"], t["n_segments"])
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    n = len(t["kind"])
    flags = torch.full((max(n, 1),), 99, dtype=torch.int32, device="cuda")
    summ = torch.full((2,), 5, dtype=torch.int32, device="cuda")
    ctx.check_launch_order(d(t["kind"]), d(t["stream"]), d(seg_ptr), d(seg_ev), d(seg_wr), t["n_streams"], flags, summ)
    torch.cuda.synchronize()
    return flags[:n].cpu().numpy().astype(np.uint32), summ.cpu().numpy().astype(np.uint32)


@pytest.mark.parametrize("n_launch,n_seg,n_streams,race", [(1, 4, 1, 0.0), (50, 8, 2, 0.2), (2000, 128, 3, 0.2),
                                                             (3000, 64, 8, 0.1), (20000, 1024, 4, 0.1),
                                                             (5000, 100, 32, 0.05), (4000, 256, 3, 0.0)])
def test_flags_match_oracle(ctx, n_launch, n_seg, n_streams, race):
    t = W.launch_trace(n_launch, n_seg, n_streams, race_frac=race, seed_salt=n_launch % 5)
    ref_flags, ref_summ = LO.check(t["kind"], t["stream"], t["acc_ptr"], t["acc_seg"], t["acc_write"],
                                   n_streams, n_seg)
    flags, summ = _gpu(ctx, t)
    assert np.array_equal(flags, ref_flags) and np.array_equal(summ, ref_summ)
    if race == 0.0:
        assert summ.tolist() == [0, 0xFFFFFFFF]
    elif n_launch >= 2000:
        assert summ[0] > 0


def test_in_place_kernels_and_the_papers_example(ctx):
    def trace(events, n_streams, n_segments):
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
        return {"kind": np.array(kind, np.uint8), "stream": np.array(stream, np.int32),
                "acc_ptr": np.array(ptr, np.int32), "acc_seg": np.array(seg, np.int32),
                "acc_write": np.array(wr, np.uint8), "n_streams": n_streams, "n_segments": n_segments}

    cases = [
        [("L", 1, [], [0]), ("L", 0, [0], [1])],                                   # attention reads what the swap stream overwrites
        [("L", 1, [], [0]), ("S", 1), ("L", 0, [0], [1])],
        [("L", 0, [2], [2]), ("L", 1, [2], [2])],
        [("L", 1, [], [3]), ("S", 1), ("L", 2, [3], []), ("S", 2), ("L", 1, [], [3])],   # collective buffer, legal
        [("L", 1, [], [3]), ("S", 1), ("L", 2, [3], []), ("L", 1, [], [3])],
        [("S", 0), ("S", 1)],
    ]
    for ev in cases:
        t = trace(ev, 3, 4)
        ref_flags, ref_summ = LO.check(t["kind"], t["stream"], t["acc_ptr"], t["acc_seg"], t["acc_write"], 3, 4)
        flags, summ = _gpu(ctx, t)
        assert np.array_equal(flags, ref_flags) and np.array_equal(summ, ref_summ)
