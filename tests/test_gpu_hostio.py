"""The host-boundary calls gift_export_to_host / gift_import_from_host against the oracle.

Only ciphertext may reach the host side: bytes that no accepted segment covers, a refused
segment's bytes among them, must arrive as zeros, and the plaintext staged on the device must
stay as it was."""
import numpy as np
import pytest
import torch

from paper_2608_25431_b200 import binding, hostio, workloads as W

from gpu_harness import make_ctx, oracle_decrypt, oracle_encrypt

pytestmark = pytest.mark.gpu


def _pinned(a):
    return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()


def test_layer_chunked_export_and_import_match_oracle():
    w = W.config3(layers=5, n_users=6, min_len=40, max_len=300)
    nseg, n_slots = len(w.segs), w.extra["n_slots"]
    om = w.owner_map.copy()
    refused = 3 * n_slots + 1                                 # one block of layer 3 is unowned
    om[w.page_table[refused]] = -2
    ref = np.zeros_like(w.buf)                                # out of place into zeros: what the host may see
    ref_tags, ref_st = oracle_encrypt(w, w.buf, ref, owner_map=om)
    assert ref_st[refused] == 4 and ref_st.sum() == 4
    page = int(w.page_table[refused])
    assert not ref[page * w.page_bytes:(page + 1) * w.page_bytes].any()

    h_src = _pinned(w.buf)
    h_dst = torch.full((w.buf_bytes,), 0x5A, dtype=torch.uint8).pin_memory()
    h_tags = torch.zeros((nseg, 16), dtype=torch.uint8).pin_memory()
    h_status = torch.full((nseg,), 9, dtype=torch.int32).pin_memory()
    d_plain = torch.zeros(w.buf_bytes, dtype=torch.uint8, device="cuda")
    d_cipher = torch.full((w.buf_bytes,), 0xC3, dtype=torch.uint8, device="cuda")
    d_segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    d_tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    d_status = torch.zeros(nseg, dtype=torch.int32, device="cuda")
    table, d_om = torch.from_numpy(w.page_table).cuda(), torch.from_numpy(om).cuda()
    ctx = make_ctx(w)
    chunks = hostio.layer_chunks(5, n_slots, n_slots * w.page_bytes)
    for _ in range(2):                                        # twice: streams and scratch are reused
        h_dst.fill_(0x5A)
        ctx.export_to_host(h_src, h_dst, d_plain, d_cipher, d_segs, nseg, chunks, d_tags, d_status, h_tags, h_status,
                           page_table=table, page_bytes=w.page_bytes, owner_map=d_om, unit_bytes=w.unit_bytes)
        torch.cuda.synchronize()
        assert np.array_equal(h_status.numpy().astype(np.uint32), ref_st)
        assert np.array_equal(h_tags.numpy(), ref_tags)
        assert np.array_equal(h_dst.numpy(), ref)             # the refused block arrives as zeros, not as plaintext
        assert np.array_equal(d_plain.cpu().numpy(), w.buf)   # the staged plaintext is untouched
    # plaintext already on the device: no upload
    h_dst.fill_(0x5A)
    ctx.export_to_host(None, h_dst, d_plain, d_cipher, d_segs, nseg, chunks, d_tags, d_status, h_tags, h_status,
                       page_table=table, page_bytes=w.page_bytes, owner_map=d_om, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    assert np.array_equal(h_dst.numpy(), ref) and np.array_equal(h_tags.numpy(), ref_tags)

    # the way back: upload ciphertext and tags, decrypt on the device, only status words return;
    # one tampered block must come back as zeros and unowned
    bad = ref.copy()
    bad[3 * w.page_bytes + 5] ^= 1
    victim = int(np.nonzero(w.page_table == 3)[0][0])
    d_buf = torch.full((w.buf_bytes,), 0x11, dtype=torch.uint8, device="cuda")
    om_dev = torch.full((om.size,), -2, dtype=torch.int32, device="cuda")
    h_status.fill_(9)
    ctx.import_from_host(_pinned(bad), _pinned(ref_tags), d_buf, d_segs, nseg, chunks, d_tags, d_status, h_status,
                         page_table=table, page_bytes=w.page_bytes, owner_map=om_dev, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    om_ref = np.full(om.size, -2, dtype=np.int32)
    pt_ref = bad.copy()
    st_ref = oracle_decrypt(w, pt_ref, pt_ref, ref_tags, owner_map=om_ref)
    assert st_ref[victim] == 1 and st_ref[refused] == 1          # the tampered block, and the one never exported
    assert np.array_equal(h_status.numpy().astype(np.uint32), st_ref)
    assert np.array_equal(d_buf.cpu().numpy(), pt_ref) and np.array_equal(om_dev.cpu().numpy(), om_ref)
    assert ctx.launch_count() > 0
    ctx.close()


def test_whole_buffer_exports_two_in_flight_match_oracle():
    """Page chains scattered over the pool cannot be cut into byte ranges: one chunk per export,
    two exports in flight on two streams with their own buffers."""
    w = W.config4(total_bytes=6 << 20, cap_bytes=2 << 20, n_users=8)
    nseg = len(w.segs)
    ctx = make_ctx(w)
    slots = hostio.ExportSlots(w.buf_bytes, nseg, 2)
    d_segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    tables = dict(page_table=torch.from_numpy(w.page_table).cuda(), page_bytes=w.page_bytes,
                  owner_map=torch.from_numpy(w.owner_map).cuda(), unit_bytes=w.unit_bytes)
    rng = np.random.default_rng(8)
    inputs = [_pinned(np.frombuffer(rng.bytes(w.buf_bytes), dtype=np.uint8).copy()) for _ in range(3)]
    chunks = hostio.whole_buffer(w.buf_bytes, nseg)
    used = [slots.export(ctx, h, d_segs, nseg, chunks, **tables) for h in inputs[:2]]
    slots.wait()
    torch.cuda.synchronize()
    assert used == [0, 1]
    for h, k in zip(inputs[:2], used):
        ref = np.zeros(w.buf_bytes, dtype=np.uint8)
        ref_tags, ref_st = oracle_encrypt(w, h.numpy(), ref)
        assert np.array_equal(slots.h_out[k].numpy(), ref) and np.array_equal(slots.h_tags[k].numpy(), ref_tags)
        assert np.array_equal(slots.h_status[k].numpy().astype(np.uint32), ref_st)
    k = slots.export(ctx, inputs[2], d_segs, nseg, chunks, **tables)        # slot 0 again
    slots.wait()
    torch.cuda.synchronize()
    ref = np.zeros(w.buf_bytes, dtype=np.uint8)
    ref_tags, _ = oracle_encrypt(w, inputs[2].numpy(), ref)
    assert k == 0 and np.array_equal(slots.h_out[0].numpy(), ref) and np.array_equal(slots.h_tags[0].numpy(), ref_tags)
    ctx.close()


def test_flat_chunks_with_uncovered_bytes_and_bound_aad():
    """Flat rows cut into three chunks; the gaps between rows and a refused row must reach the host as zeros;
    a bound AAD array is indexed by the segment's position in the whole table."""
    from oracle import gcm
    w = W.config2(n_users=12, vocab=700)
    nseg = len(w.segs)
    om = w.owner_map.copy()
    om[7] = binding.OWNER_PARAM                                # row 7 may not be exported
    rng = np.random.default_rng(77)
    aad = np.frombuffer(rng.bytes(16 * nseg), dtype=np.uint8).reshape(nseg, 16).copy()
    ref = np.zeros_like(w.buf)
    ref_tags, ref_st = gcm.seg_encrypt(w.buf, ref, w.segs, w.user_ids, w.keys, w.max_users, None, 0, om, w.unit_bytes,
                                       aad=aad)
    assert ref_st[7] == 2 and ref_st.sum() == 2
    pitch = w.unit_bytes
    chunks = [(0, 4 * pitch, 0, 4), (4 * pitch, 9 * pitch, 4, 9), (9 * pitch, w.buf_bytes, 9, nseg)]
    ctx = make_ctx(w)
    d_aad = torch.from_numpy(aad).cuda()
    ctx.bind_aad(d_aad)
    h_dst = torch.full((w.buf_bytes,), 0x5A, dtype=torch.uint8).pin_memory()
    h_tags = torch.zeros((nseg, 16), dtype=torch.uint8).pin_memory()
    h_status = torch.full((nseg,), 9, dtype=torch.int32).pin_memory()
    d_plain = torch.zeros(w.buf_bytes, dtype=torch.uint8, device="cuda")
    d_cipher = torch.empty(w.buf_bytes, dtype=torch.uint8, device="cuda")
    d_segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    d_tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    d_status = torch.zeros(nseg, dtype=torch.int32, device="cuda")
    ctx.export_to_host(_pinned(w.buf), h_dst, d_plain, d_cipher, d_segs, nseg, chunks, d_tags, d_status, h_tags,
                       h_status, owner_map=torch.from_numpy(om).cuda(), unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    assert np.array_equal(h_status.numpy().astype(np.uint32), ref_st)
    assert np.array_equal(h_tags.numpy(), ref_tags) and np.array_equal(h_dst.numpy(), ref)
    row7 = h_dst.numpy()[7 * pitch: 8 * pitch]
    assert not row7.any() and w.buf[7 * pitch: 8 * pitch].any()
    with pytest.raises(binding.GiftError):                     # a chunk that runs past the table
        ctx.export_to_host(None, h_dst, d_plain, d_cipher, d_segs, nseg, [(0, pitch, 0, nseg + 1)], d_tags, d_status,
                           h_tags, h_status)
    ctx.close()


def test_cipher_kernel_can_write_straight_into_pinned_host_memory():
    """gift_seg_encrypt takes page-locked host memory as dst; the device copy stays plaintext."""
    w = W.config3(layers=3, n_users=5, min_len=40, max_len=300)
    nseg = len(w.segs)
    ref = w.buf.copy()
    ref_tags, ref_st = oracle_encrypt(w, ref, ref)
    assert not ref_st.any()
    h_dst = torch.zeros(w.buf_bytes, dtype=torch.uint8).pin_memory()
    d_buf = torch.from_numpy(w.buf).cuda()
    d_segs = torch.from_numpy(w.segs.view(np.uint8).copy()).cuda()
    d_tags = torch.zeros((nseg, 16), dtype=torch.uint8, device="cuda")
    d_status = torch.zeros(nseg, dtype=torch.int32, device="cuda")
    ctx = make_ctx(w)
    ctx.seg_encrypt(d_buf, h_dst, d_segs, nseg, d_tags, d_status, page_table=torch.from_numpy(w.page_table).cuda(),
                    page_bytes=w.page_bytes)
    torch.cuda.synchronize()
    assert not d_status.any().item()
    assert np.array_equal(d_tags.cpu().numpy(), ref_tags)
    assert np.array_equal(h_dst.numpy(), ref)
    assert np.array_equal(d_buf.cpu().numpy(), w.buf)
    ctx.close()
