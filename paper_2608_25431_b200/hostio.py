"""Helpers around the host-boundary calls gift_export_to_host / gift_import_from_host.

The overlap of upload, cipher and download lives in the library (three internal streams per
context, see include/gift.h).  What is left here is how to cut a pool into chunks, and a
holder for the buffers of a caller that keeps two whole-buffer exports in flight.
"""
from __future__ import annotations

from typing import List, Tuple

import torch

from . import binding

Chunk = Tuple[int, int, int, int]      # (byte_lo, byte_hi, seg_lo, seg_hi)


def layer_chunks(n_layers: int, segs_per_layer: int, bytes_per_layer: int) -> List[Chunk]:
    """Chunks of a layer-major pool whose segment table is layer-major too."""
    return [(l * bytes_per_layer, (l + 1) * bytes_per_layer, l * segs_per_layer, (l + 1) * segs_per_layer)
            for l in range(n_layers)]


def whole_buffer(buf_bytes: int, nseg: int) -> List[Chunk]:
    """One chunk: for tables whose segments cannot be cut into contiguous byte ranges
    (page chains scattered over the pool)."""
    return [(0, buf_bytes, 0, nseg)]


class ExportSlots:
    """Device and pinned host buffers for k whole-buffer exports in flight.

    Export i uses slot i mod k and its own CUDA stream, so that the download of one export
    overlaps the upload of the next (the context's internal streams serve them in turn)."""

    def __init__(self, buf_bytes: int, nseg: int, k: int = 2, device: int = 0):
        dev = torch.device("cuda", device)
        self.k = k
        self.streams = [torch.cuda.Stream(device=dev) for _ in range(k)]
        self.d_plain = [torch.empty(buf_bytes, dtype=torch.uint8, device=dev) for _ in range(k)]
        self.d_cipher = [torch.empty(buf_bytes, dtype=torch.uint8, device=dev) for _ in range(k)]
        self.d_tags = [torch.empty((nseg, 16), dtype=torch.uint8, device=dev) for _ in range(k)]
        self.d_status = [torch.empty(nseg, dtype=torch.int32, device=dev) for _ in range(k)]
        self.h_out = [torch.empty(buf_bytes, dtype=torch.uint8, pin_memory=True) for _ in range(k)]
        self.h_tags = [torch.empty((nseg, 16), dtype=torch.uint8, pin_memory=True) for _ in range(k)]
        self.h_status = [torch.empty(nseg, dtype=torch.int32, pin_memory=True) for _ in range(k)]
        self.n = 0

    def export(self, ctx: binding.Ctx, h_src: torch.Tensor, d_segs: torch.Tensor, nseg: int, chunks, **tables) -> int:
        """Enqueue one export; returns the slot whose host outputs it will fill."""
        s = self.n % self.k
        self.n += 1
        st = self.streams[s]
        st.wait_stream(torch.cuda.current_stream())
        ctx.export_to_host(h_src, self.h_out[s], self.d_plain[s], self.d_cipher[s], d_segs, nseg, chunks,
                           self.d_tags[s], self.d_status[s], self.h_tags[s], self.h_status[s],
                           stream=st.cuda_stream, **tables)
        return s

    def wait(self):
        for st in self.streams:
            torch.cuda.current_stream().wait_stream(st)
