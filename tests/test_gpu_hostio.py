"""Chunked export from pinned host memory gives the oracle's bytes, tags and status words."""
import numpy as np
import pytest
import torch

from paper_2608_25431_b200 import hostio, workloads as W

from gpu_harness import oracle_encrypt

pytestmark = pytest.mark.gpu


def test_layer_chunked_export_matches_oracle():
    w = W.config3(layers=5, n_users=6, min_len=40, max_len=300)
    nseg, n_slots = len(w.segs), w.extra["n_slots"]
    om = w.owner_map.copy()
    refused = 3 * n_slots + 1                                 # one block of layer 3 is unowned
    om[w.page_table[refused]] = -2
    ref = w.buf.copy()
    ref_tags, ref_st = oracle_encrypt(w, ref, ref, owner_map=om)
    assert ref_st[refused] == 4 and ref_st.sum() == 4

    h_src = torch.from_numpy(w.buf).pin_memory()
    h_dst = torch.zeros(w.buf_bytes, dtype=torch.uint8).pin_memory()
    h_tags = torch.zeros((nseg, 16), dtype=torch.uint8).pin_memory()
    h_status = torch.full((nseg,), 9, dtype=torch.int32).pin_memory()
    d_buf = torch.zeros(w.buf_bytes, dtype=torch.uint8, device="cuda")
    d_segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    d_tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    d_status = torch.zeros(nseg, dtype=torch.int32, device="cuda")
    exp = hostio.HostExporter(w.max_users, w.user_ids, w.keys, 0, 3, 0, n_slots)
    chunks = hostio.layer_chunks(5, n_slots, n_slots * w.page_bytes)
    for _ in range(2):                                        # twice: contexts and scratch are reused
        h_dst.zero_()
        exp.export(h_src, h_dst, d_buf, chunks, d_segs, d_tags, d_status, h_tags, h_status,
                   page_table=torch.from_numpy(w.page_table).cuda(), page_bytes=w.page_bytes,
                   owner_map=torch.from_numpy(om).cuda(), unit_bytes=w.unit_bytes)
        torch.cuda.synchronize()
        assert np.array_equal(h_status.numpy().astype(np.uint32), ref_st)
        assert np.array_equal(h_tags.numpy(), ref_tags)
        assert np.array_equal(h_dst.numpy(), ref)
    assert exp.launch_count() > 0
    exp.close()
