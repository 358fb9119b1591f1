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
    # the way back: upload ciphertext and tags, decrypt on the device, only status words return;
    # one tampered block must come back as zeros and unowned
    bad = ref.copy()
    bad[3 * w.page_bytes + 5] ^= 1
    victim = int(np.nonzero(w.page_table == 3)[0][0])
    h_ct = torch.from_numpy(bad).pin_memory()
    h_tg = torch.from_numpy(ref_tags).pin_memory()
    om_dev = torch.full((om.size,), -2, dtype=torch.int32, device="cuda")
    h_status.fill_(9)
    exp.import_(h_ct, h_tg, d_buf, chunks, d_segs, d_tags, d_status, h_status,
                page_table=torch.from_numpy(w.page_table).cuda(), page_bytes=w.page_bytes,
                owner_map=om_dev, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    from gpu_harness import oracle_decrypt
    om_ref = np.full(om.size, -2, dtype=np.int32)
    pt_ref = bad.copy()
    st_ref = oracle_decrypt(w, pt_ref, pt_ref, ref_tags, owner_map=om_ref)
    assert st_ref[victim] == 1 and st_ref[refused] == 1          # the tampered block, and the one never exported
    assert np.array_equal(h_status.numpy().astype(np.uint32), st_ref)
    assert np.array_equal(d_buf.cpu().numpy(), pt_ref) and np.array_equal(om_dev.cpu().numpy(), om_ref)
    exp.close()


def test_two_steps_in_flight_match_oracle():
    w = W.config4(total_bytes=6 << 20, cap_bytes=2 << 20, n_users=8)
    nseg = len(w.segs)
    pipe = hostio.StepPipeline(w.max_users, w.user_ids, w.keys, w.buf_bytes, nseg)
    d_segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    table, om = torch.from_numpy(w.page_table).cuda(), torch.from_numpy(w.owner_map).cuda()
    rng = np.random.default_rng(8)
    inputs = [torch.from_numpy(np.frombuffer(rng.bytes(w.buf_bytes), dtype=np.uint8).copy()).pin_memory()
              for _ in range(3)]
    slots = []
    for h in inputs[:2]:                                     # two steps in flight at once
        slots.append(pipe.step(h, d_segs, nseg, page_table=table, page_bytes=w.page_bytes, owner_map=om,
                               unit_bytes=w.unit_bytes))
    pipe.wait()
    torch.cuda.synchronize()
    assert slots == [0, 1]
    for h, k in zip(inputs[:2], slots):
        ref = h.numpy().copy()
        ref_tags, ref_st = oracle_encrypt(w, ref, ref)
        assert np.array_equal(pipe.h_out[k].numpy(), ref) and np.array_equal(pipe.h_tags[k].numpy(), ref_tags)
        assert np.array_equal(pipe.h_status[k].numpy().astype(np.uint32), ref_st)
    k = pipe.step(inputs[2], d_segs, nseg, page_table=table, page_bytes=w.page_bytes, owner_map=om,
                  unit_bytes=w.unit_bytes)                   # slot 0 again
    pipe.wait()
    torch.cuda.synchronize()
    ref = inputs[2].numpy().copy()
    ref_tags, _ = oracle_encrypt(w, ref, ref)
    assert k == 0 and np.array_equal(pipe.h_out[0].numpy(), ref) and np.array_equal(pipe.h_tags[0].numpy(), ref_tags)
    pipe.close()


def test_direct_output_into_pinned_host_memory_matches_oracle():
    """The cipher kernel stores ciphertext straight into pinned host memory; the staged plaintext stays."""
    w = W.config3(layers=3, n_users=5, min_len=40, max_len=300)
    nseg, n_slots = len(w.segs), w.extra["n_slots"]
    ref = w.buf.copy()
    ref_tags, ref_st = oracle_encrypt(w, ref, ref)
    assert not ref_st.any()
    h_src = torch.from_numpy(w.buf).pin_memory()
    h_dst = torch.zeros(w.buf_bytes, dtype=torch.uint8).pin_memory()
    h_tags = torch.zeros((nseg, 16), dtype=torch.uint8).pin_memory()
    h_status = torch.full((nseg,), 9, dtype=torch.int32).pin_memory()
    d_buf = torch.zeros(w.buf_bytes, dtype=torch.uint8, device="cuda")
    d_segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    d_tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    d_status = torch.zeros(nseg, dtype=torch.int32, device="cuda")
    exp = hostio.HostExporter(w.max_users, w.user_ids, w.keys, 0, 2, 0, n_slots)
    chunks = hostio.layer_chunks(3, n_slots, n_slots * w.page_bytes)
    exp.export(h_src, h_dst, d_buf, chunks, d_segs, d_tags, d_status, h_tags, h_status,
               page_table=torch.from_numpy(w.page_table).cuda(), page_bytes=w.page_bytes, direct_out=True)
    torch.cuda.synchronize()
    assert not h_status.any().item()
    assert np.array_equal(h_tags.numpy(), ref_tags)
    assert np.array_equal(h_dst.numpy(), ref)
    assert np.array_equal(d_buf.cpu().numpy(), w.buf)         # the device copy is still plaintext
    exp.close()
