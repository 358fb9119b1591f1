"""Export from pinned host memory, chunked so that copies overlap the cipher.

A caller whose plaintext sits in pinned host memory (a swapped-out KV pool, paper sec. 4.5)
needs host -> device copy, export, device -> host copy.  Done in one piece the three stages
run back to back and PCIe idles while the cipher runs and the other way round.  Here the
buffer is cut into chunks that no segment straddles (for the layer-major KV pool: one
layer per chunk); chunk i uses stream i mod k, so the upload of one chunk, the cipher of
the previous one and the download of the one before overlap.  Each stream has its own
context, because a context's scratch belongs to one stream at a time.

Only orchestration lives here: every byte is produced by gift_seg_encrypt.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import torch

from . import binding


@dataclass
class Chunk:
    byte_lo: int      # buffer range [byte_lo, byte_hi) that holds all bytes of the chunk's segments
    byte_hi: int
    seg_lo: int       # rows [seg_lo, seg_hi) of the segment table
    seg_hi: int


def layer_chunks(n_layers: int, segs_per_layer: int, bytes_per_layer: int) -> List[Chunk]:
    """Chunks of a layer-major pool whose segment table is layer-major too."""
    return [Chunk(l * bytes_per_layer, (l + 1) * bytes_per_layer, l * segs_per_layer, (l + 1) * segs_per_layer)
            for l in range(n_layers)]


class HostExporter:
    """k contexts and streams that export chunks of a host buffer through one device buffer.

    `import_` is the opposite direction (paper sec. 3, steps 3-4): ciphertext and tags arrive
    from pinned host memory, every chunk is uploaded and decrypted with the claimed owners'
    keys on its stream, the plaintext stays on the device and only the status words go back.
    """

    def __init__(self, max_users: int, user_ids, keys, device: int = 0, n_streams: int = 3, flags: int = 0,
                 max_segs_per_chunk: int = 1024):
        self.ctxs = [binding.Ctx(max_users, device, flags) for _ in range(n_streams)]
        for c in self.ctxs:
            c.set_keys(user_ids, keys)
            c.reserve(max_segs_per_chunk)
        self.streams = [torch.cuda.Stream(device=device) for _ in range(n_streams)]

    def close(self):
        for c in self.ctxs:
            c.close()

    def launch_count(self) -> int:
        return sum(c.launch_count() for c in self.ctxs)

    def export(self, h_src: torch.Tensor, h_dst: torch.Tensor, d_buf: torch.Tensor, chunks: List[Chunk],
               d_segs: torch.Tensor, d_tags: torch.Tensor, d_status: torch.Tensor, h_tags: torch.Tensor,
               h_status: torch.Tensor, page_table: Optional[torch.Tensor] = None, page_bytes: int = 0,
               owner_map: Optional[torch.Tensor] = None, unit_bytes: int = 0, direct_out: bool = False):
        """Enqueue upload, export and download of every chunk; returns without waiting.

        h_src, h_dst: pinned uint8 host tensors of the buffer's size; d_buf: device staging of
        the same size; d_segs: the whole table on the device as uint8[nseg*40].  With
        direct_out the cipher kernel stores the ciphertext straight into h_dst (pinned memory is
        device-visible), so the staged plaintext stays intact and no download copy runs.
        """
        cur = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(cur)
        for i, ch in enumerate(chunks):
            st = self.streams[i % len(self.streams)]
            ctx = self.ctxs[i % len(self.ctxs)]
            st.wait_event(start)
            with torch.cuda.stream(st):
                d_buf[ch.byte_lo:ch.byte_hi].copy_(h_src[ch.byte_lo:ch.byte_hi], non_blocking=True)
                n = ch.seg_hi - ch.seg_lo
                ctx.seg_encrypt(d_buf, h_dst if direct_out else d_buf, d_segs[ch.seg_lo * 40: ch.seg_hi * 40], n,
                                d_tags[ch.seg_lo:ch.seg_hi], d_status[ch.seg_lo:ch.seg_hi],
                                page_table=page_table, page_bytes=page_bytes, owner_map=owner_map,
                                unit_bytes=unit_bytes, stream=st.cuda_stream)
                if not direct_out:
                    h_dst[ch.byte_lo:ch.byte_hi].copy_(d_buf[ch.byte_lo:ch.byte_hi], non_blocking=True)
                h_tags[ch.seg_lo:ch.seg_hi].copy_(d_tags[ch.seg_lo:ch.seg_hi], non_blocking=True)
                h_status[ch.seg_lo:ch.seg_hi].copy_(d_status[ch.seg_lo:ch.seg_hi], non_blocking=True)
        for st in self.streams:
            cur.wait_stream(st)

    def import_(self, h_src: torch.Tensor, h_tags: torch.Tensor, d_buf: torch.Tensor, chunks: List[Chunk],
                d_segs: torch.Tensor, d_tags: torch.Tensor, d_status: torch.Tensor, h_status: torch.Tensor,
                page_table: Optional[torch.Tensor] = None, page_bytes: int = 0,
                owner_map: Optional[torch.Tensor] = None, unit_bytes: int = 0):
        """Enqueue upload and in-place decryption of every chunk; returns without waiting."""
        cur = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(cur)
        for i, ch in enumerate(chunks):
            st = self.streams[i % len(self.streams)]
            ctx = self.ctxs[i % len(self.ctxs)]
            st.wait_event(start)
            with torch.cuda.stream(st):
                d_buf[ch.byte_lo:ch.byte_hi].copy_(h_src[ch.byte_lo:ch.byte_hi], non_blocking=True)
                d_tags[ch.seg_lo:ch.seg_hi].copy_(h_tags[ch.seg_lo:ch.seg_hi], non_blocking=True)
                n = ch.seg_hi - ch.seg_lo
                ctx.seg_decrypt(d_buf, d_buf, d_segs[ch.seg_lo * 40: ch.seg_hi * 40], n,
                                d_tags[ch.seg_lo:ch.seg_hi], d_status[ch.seg_lo:ch.seg_hi],
                                page_table=page_table, page_bytes=page_bytes, owner_map=owner_map,
                                unit_bytes=unit_bytes, stream=st.cuda_stream)
                h_status[ch.seg_lo:ch.seg_hi].copy_(d_status[ch.seg_lo:ch.seg_hi], non_blocking=True)
        for st in self.streams:
            cur.wait_stream(st)


class StepPipeline:
    """Whole-buffer export steps kept two in flight: for tables whose segments cannot be cut
    into contiguous chunks (page chains scattered over the pool).  Step i runs upload, export
    and download on stream i mod 2 with its own context and device buffers, so the download
    of one step overlaps the upload of the next."""

    def __init__(self, max_users: int, user_ids, keys, buf_bytes: int, nseg: int, device: int = 0, flags: int = 0):
        self.ctxs = [binding.Ctx(max_users, device, flags) for _ in range(2)]
        for c in self.ctxs:
            c.set_keys(user_ids, keys)
            c.reserve(nseg)
        self.streams = [torch.cuda.Stream(device=device) for _ in range(2)]
        dev = torch.device("cuda", device)
        self.bufs = [torch.empty(buf_bytes, dtype=torch.uint8, device=dev) for _ in range(2)]
        self.tags = [torch.empty((nseg, 16), dtype=torch.uint8, device=dev) for _ in range(2)]
        self.status = [torch.empty(nseg, dtype=torch.int32, device=dev) for _ in range(2)]
        self.h_out = [torch.empty(buf_bytes, dtype=torch.uint8, pin_memory=True) for _ in range(2)]
        self.h_tags = [torch.empty((nseg, 16), dtype=torch.uint8, pin_memory=True) for _ in range(2)]
        self.h_status = [torch.empty(nseg, dtype=torch.int32, pin_memory=True) for _ in range(2)]
        self.step_no = 0

    def close(self):
        for c in self.ctxs:
            c.close()

    def launch_count(self) -> int:
        return sum(c.launch_count() for c in self.ctxs)

    def step(self, h_src: torch.Tensor, d_segs: torch.Tensor, nseg: int, page_table=None, page_bytes: int = 0,
             owner_map=None, unit_bytes: int = 0):
        """Enqueue one export step; returns the slot (0/1) whose host outputs it will fill."""
        k = self.step_no & 1
        self.step_no += 1
        st = self.streams[k]
        st.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(st):
            self.bufs[k].copy_(h_src, non_blocking=True)
            self.ctxs[k].seg_encrypt(self.bufs[k], self.bufs[k], d_segs, nseg, self.tags[k], self.status[k],
                                     page_table=page_table, page_bytes=page_bytes, owner_map=owner_map,
                                     unit_bytes=unit_bytes, stream=st.cuda_stream)
            self.h_out[k].copy_(self.bufs[k], non_blocking=True)
            self.h_tags[k].copy_(self.tags[k], non_blocking=True)
            self.h_status[k].copy_(self.status[k], non_blocking=True)
        return k

    def wait(self):
        for st in self.streams:
            torch.cuda.current_stream().wait_stream(st)

