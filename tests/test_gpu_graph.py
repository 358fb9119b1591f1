"""A whole export call captured in a CUDA graph and replayed: same bytes as the oracle.

The call enqueues a memset and four kernels and neither allocates (once the scratch is
reserved) nor synchronises, so it can be captured; replaying the graph removes the
per-launch host cost for small, frequent calls such as a decode step's rows."""
import numpy as np
import pytest
import torch

from paper_2608_25431_b200 import binding, workloads as W

from gpu_harness import oracle_encrypt

pytestmark = pytest.mark.gpu


def test_captured_export_replays_bit_exact():
    w = W.config2(n_users=32, vocab=1000)
    n = len(w.segs)
    ctx = binding.Ctx(w.max_users)
    ctx.set_keys(w.user_ids, w.keys)
    ctx.reserve(n)
    src = torch.from_numpy(w.buf).cuda()
    dst = torch.zeros_like(src)
    segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    om = torch.from_numpy(w.owner_map).cuda()
    tags = torch.zeros((n, 16), dtype=torch.uint8, device="cuda")
    status = torch.zeros(n, dtype=torch.int32, device="cuda")

    def call():
        ctx.seg_encrypt(src, dst, segs, n, tags, status, owner_map=om, unit_bytes=w.unit_bytes)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call()                                   # warm-up outside the capture (function attributes, scratch)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        call()
    rng = np.random.default_rng(5)
    for rep in range(3):
        data = np.frombuffer(rng.bytes(w.buf.size), dtype=np.uint8).copy()
        src.copy_(torch.from_numpy(data))
        dst.zero_()
        tags.zero_()
        status.fill_(9)
        g.replay()
        torch.cuda.synchronize()
        ref = np.zeros_like(data)
        ref_tags, ref_st = oracle_encrypt(w, data, ref)
        assert np.array_equal(status.cpu().numpy().astype(np.uint32), ref_st)
        assert np.array_equal(tags.cpu().numpy(), ref_tags)
        assert np.array_equal(dst.cpu().numpy(), ref)
    ctx.close()
