"""Seeded synthetic inputs shaped like the serving workloads of the paper.

This module only draws random inputs and lays out tables; it holds none of the
method's arithmetic (no cipher, no hash, no label join) and imports neither the
CUDA binding nor the CPU oracle, so both can be fed from it.

The paper evaluates on ShareGPT, HumanEval and LongBench traces with OPT and
Qwen2.5 weights (paper sec. 7, "Performance Evaluation"); none of that is
needed here.  These generators stand in for those workloads by shape only:
token/logit rows of a decode step, paged KV-cache blocks of a LLaMA-7B-shaped
model handed from prefill to decode, Zipf-skewed ownership, and a mixed
prefill/decode batch with seeded tampering.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

# One row of the segment table: {owner, flags, offset, len, nonce[12], page0}, 40 bytes.
SEG_DTYPE = np.dtype([
    ("owner", "<i4"), ("flags", "<u4"), ("offset", "<u8"), ("len", "<u8"),
    ("nonce", "u1", (12,)), ("page0", "<u4"),
])
assert SEG_DTYPE.itemsize == 40

SEED_BASE = 0x61F70000

# LLaMA-7B KV shape: 32 layers, 32 heads x 128 dims, K and V, bf16.
KV_LAYERS = 32
KV_BLOCK_TOKENS = 16
KV_TOKEN_BYTES = 2 * 32 * 128 * 2            # K and V of one token in one layer: 16 KiB
KV_PAGE_BYTES = KV_BLOCK_TOKENS * KV_TOKEN_BYTES   # 256 KiB per block per layer


@dataclass
class Workload:
    """Inputs of one call: keys, a payload buffer, a segment table and optional tables."""
    name: str
    user_ids: np.ndarray                 # int32 [U]
    keys: np.ndarray                     # uint8 [U, 16]
    max_users: int
    buf: Optional[np.ndarray]            # uint8 [buf_bytes] plaintext (None: fill on device)
    buf_bytes: int
    segs: np.ndarray                     # SEG_DTYPE [nseg]
    page_table: Optional[np.ndarray] = None   # int32 [n_pages] or None (flat)
    page_bytes: int = 0
    owner_map: Optional[np.ndarray] = None    # int32 [n_units] or None
    unit_bytes: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def payload_bytes(self) -> int:
        return int(self.segs["len"].sum())


def _rng(config: int, salt: int = 0) -> np.random.Generator:
    return np.random.default_rng(SEED_BASE + config + (salt << 8))


def _keys(rng: np.random.Generator, n_users: int):
    keys = np.frombuffer(rng.bytes(16 * n_users), dtype=np.uint8).reshape(n_users, 16).copy()
    return np.arange(n_users, dtype=np.int32), keys


def nonce_triple(a, b, c) -> np.ndarray:
    """12-byte nonces LE32(a) || LE32(b) || LE32(c), broadcast over arrays."""
    a, b, c = np.broadcast_arrays(np.asarray(a, dtype="<u4"), np.asarray(b, dtype="<u4"),
                                  np.asarray(c, dtype="<u4"))
    out = np.empty(a.shape + (12,), dtype=np.uint8)
    out[..., 0:4] = a[..., None].view(np.uint8).reshape(a.shape + (4,))
    out[..., 4:8] = b[..., None].view(np.uint8).reshape(a.shape + (4,))
    out[..., 8:12] = c[..., None].view(np.uint8).reshape(a.shape + (4,))
    return out


def bf16_normal(rng: np.random.Generator, n: int, std: float) -> np.ndarray:
    """n bf16 values N(0, std) as uint16 bit patterns (round-to-nearest-even from fp32)."""
    x = rng.standard_normal(n, dtype=np.float32) * np.float32(std)
    u = x.view(np.uint32)
    u = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (u >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# Config 1: tiny round trip
# --------------------------------------------------------------------------
def config1(seed_salt: int = 0) -> Workload:
    """8 users, one contiguous uint8 buffer of 8 back-to-back segments, lengths 16*U{1..512}."""
    rng = _rng(1, seed_salt)
    uids, keys = _keys(rng, 8)
    lens = 16 * rng.integers(1, 513, size=8)
    offs = np.concatenate([[0], np.cumsum(lens)[:-1]])
    total = int(lens.sum())
    buf = np.frombuffer(rng.bytes(total), dtype=np.uint8).copy()
    segs = np.zeros(8, dtype=SEG_DTYPE)
    segs["owner"] = uids
    segs["offset"] = offs
    segs["len"] = lens
    segs["nonce"] = np.frombuffer(rng.bytes(12 * 8), dtype=np.uint8).reshape(8, 12)
    return Workload("c1_tiny", uids, keys, 8, buf, total, segs)


# --------------------------------------------------------------------------
# Config 2: decode-step output rows
# --------------------------------------------------------------------------
def config2(n_users: int = 256, vocab: int = 32000, step: int = 7, seed_salt: int = 0) -> Workload:
    """One row per user: vocab bf16 logits N(0, std 3), one int32 sampled token, 12 pad bytes.

    The segment is the 2*vocab + 4 payload bytes of the row, so its last cipher block is
    partial; rows sit at a 16-byte-aligned pitch.
    """
    rng = _rng(2, seed_salt)
    uids, keys = _keys(rng, n_users)
    seg_len = 2 * vocab + 4
    pitch = (seg_len + 15) // 16 * 16
    buf = np.zeros(n_users * pitch, dtype=np.uint8)
    rows = buf.reshape(n_users, pitch)
    rows[:, : 2 * vocab] = bf16_normal(rng, n_users * vocab, 3.0).reshape(n_users, vocab).view(np.uint8)
    rows[:, 2 * vocab: 2 * vocab + 4] = rng.integers(0, vocab, size=n_users).astype("<i4")[:, None].view(
        np.uint8).reshape(n_users, 4)
    segs = np.zeros(n_users, dtype=SEG_DTYPE)
    segs["owner"] = uids
    segs["offset"] = np.arange(n_users, dtype=np.uint64) * np.uint64(pitch)
    segs["len"] = seg_len
    segs["nonce"] = nonce_triple(uids, step, 0)
    owner_map = uids.copy()          # one ownership unit per row
    return Workload("c2_decode_rows", uids, keys, n_users, buf, buf.size, segs,
                    owner_map=owner_map, unit_bytes=pitch)


# --------------------------------------------------------------------------
# Config 3: prefill -> decode KV-cache handoff
# --------------------------------------------------------------------------
def config3(layers: int = 2, n_users: int = 16, min_len: int = 256, max_len: int = 2048,
            fill: bool = True, seed_salt: int = 0) -> Workload:
    """Paged KV pool pool[layer][slot] of 256 KiB blocks; one segment per (user, layer, block).

    Slots are one random permutation split among the users (the same slot numbers in
    every layer); page index = layer * n_slots + slot; nonce = (user, layer, block).
    Unfilled token slots of a user's last block are zero.  With fill=False the payload
    is left for the caller to generate on the device (bench scale).
    """
    rng = _rng(3, seed_salt)
    uids, keys = _keys(rng, n_users)
    prompt = rng.integers(min_len, max_len + 1, size=n_users)
    nblk = (prompt + KV_BLOCK_TOKENS - 1) // KV_BLOCK_TOKENS
    n_slots = int(nblk.sum())
    perm = rng.permutation(n_slots).astype(np.int64)
    first = np.concatenate([[0], np.cumsum(nblk)[:-1]])
    user_of_entry = np.repeat(uids, nblk)                       # per (user, block) in user order
    block_of_entry = np.concatenate([np.arange(n) for n in nblk])
    nseg = layers * n_slots
    # Page table: entry (layer, e) -> layer * n_slots + perm[e]
    page_table = (np.arange(layers, dtype=np.int64)[:, None] * n_slots + perm[None, :]).reshape(-1)
    segs = np.zeros(nseg, dtype=SEG_DTYPE)
    segs["owner"] = np.tile(user_of_entry, layers)
    segs["len"] = KV_PAGE_BYTES
    segs["page0"] = np.arange(nseg, dtype=np.uint32)
    lay = np.repeat(np.arange(layers), n_slots)
    segs["nonce"] = nonce_triple(segs["owner"], lay, np.tile(block_of_entry, layers))
    owner_map = np.empty(nseg, dtype=np.int32)
    owner_map[page_table] = segs["owner"]
    buf_bytes = nseg * KV_PAGE_BYTES
    buf = None
    if fill:
        buf = np.zeros(buf_bytes, dtype=np.uint8)
        pages = buf.reshape(nseg, KV_BLOCK_TOKENS, KV_TOKEN_BYTES)
        for u in range(n_users):
            tail = int(prompt[u]) - (int(nblk[u]) - 1) * KV_BLOCK_TOKENS   # tokens in last block
            for l in range(layers):
                e0 = int(first[u])
                idx = page_table[l * n_slots + e0: l * n_slots + e0 + int(nblk[u])]
                vals = bf16_normal(rng, int(nblk[u]) * KV_PAGE_BYTES // 2, 1.0).view(np.uint8)
                blk = vals.reshape(int(nblk[u]), KV_BLOCK_TOKENS, KV_TOKEN_BYTES)
                blk[-1, tail:, :] = 0
                pages[idx] = blk
    return Workload("c3_kv_handoff", uids, keys, n_users, buf, buf_bytes, segs,
                    page_table=page_table.astype(np.int32), page_bytes=KV_PAGE_BYTES,
                    owner_map=owner_map, unit_bytes=KV_PAGE_BYTES,
                    extra={"prompt": prompt, "nblk": nblk, "n_slots": n_slots, "layers": layers,
                           "first": first, "perm": perm})


# --------------------------------------------------------------------------
# Config 4: Zipf-skewed ownership over a paged pool
# --------------------------------------------------------------------------
def config4(total_bytes: int = 64 << 20, cap_bytes: int = 4 << 20, n_users: int = 1024,
            fill: bool = True, seed_salt: int = 0) -> Workload:
    """Segment lengths 16*min(zipf(1.2), cap) drawn until the running total reaches total_bytes.

    Segment i < n_users belongs to user i, later ones to a uniform user.  Every segment is a
    chain of 256 KiB pages at a random permutation of pool slots; its last page is partial.
    """
    rng = _rng(4, seed_salt)
    uids, keys = _keys(rng, n_users)
    lens = []
    tot = 0
    cap_blocks = cap_bytes // 16
    while tot < total_bytes:
        draw = rng.zipf(1.2, size=256)
        for d in draw:
            l = 16 * int(min(int(d), cap_blocks))
            lens.append(l)
            tot += l
            if tot >= total_bytes:
                break
    lens = np.array(lens, dtype=np.int64)
    nseg = lens.size
    owners = np.empty(nseg, dtype=np.int32)
    owners[: min(nseg, n_users)] = uids[: min(nseg, n_users)]
    if nseg > n_users:
        owners[n_users:] = rng.integers(0, n_users, size=nseg - n_users)
    npages = (lens + KV_PAGE_BYTES - 1) // KV_PAGE_BYTES
    n_slots = int(npages.sum())
    page_table = rng.permutation(n_slots).astype(np.int32)
    page0 = np.concatenate([[0], np.cumsum(npages)[:-1]])
    segs = np.zeros(nseg, dtype=SEG_DTYPE)
    segs["owner"] = owners
    segs["len"] = lens
    segs["page0"] = page0
    segs["nonce"] = nonce_triple(owners, np.arange(nseg), 0)
    owner_map = np.empty(n_slots, dtype=np.int32)
    owner_map[page_table] = np.repeat(owners, npages)
    buf_bytes = n_slots * KV_PAGE_BYTES
    buf = None
    if fill:
        buf = np.frombuffer(rng.bytes(buf_bytes), dtype=np.uint8).copy()
    return Workload("c4_zipf", uids, keys, n_users, buf, buf_bytes, segs,
                    page_table=page_table, page_bytes=KV_PAGE_BYTES,
                    owner_map=owner_map, unit_bytes=KV_PAGE_BYTES,
                    extra={"npages": npages})


# --------------------------------------------------------------------------
# Config 5: mixed prefill/decode batch, flow rules, tampering
# --------------------------------------------------------------------------
def config5(layers: int = 2, n_users: int = 512, chunk_tokens: int = 32, fill: bool = True,
            poison_frac: float = 0.01, seed_salt: int = 0) -> Workload:
    """Flat handoff buffer [layer][token][16 KiB]; request r owns a contiguous token range.

    Even requests are prefill chunks (chunk_tokens tokens), odd ones decode steps (1 token).
    One segment per (request, layer).  `extra` carries what the flow rules need (token owner
    map, request->token CSR, a KV-block owner map with request->block CSR tables, a broadcast
    gather) and the seeded tampering plan: poison_frac of the segments, in thirds a flipped
    ciphertext bit, a flipped tag bit, a claimed owner replaced by another user; and the same
    fraction of block-table entries redirected to another user's block.
    """
    rng = _rng(5, seed_salt)
    uids, keys = _keys(rng, n_users)
    ntok = np.where(np.arange(n_users) % 2 == 0, chunk_tokens, 1).astype(np.int64)
    tok0 = np.concatenate([[0], np.cumsum(ntok)[:-1]])
    T = int(ntok.sum())
    nseg = layers * n_users
    segs = np.zeros(nseg, dtype=SEG_DTYPE)
    lay = np.repeat(np.arange(layers), n_users)
    req = np.tile(np.arange(n_users), layers)
    segs["owner"] = uids[req]
    segs["offset"] = (lay.astype(np.uint64) * np.uint64(T) + tok0[req].astype(np.uint64)) * np.uint64(KV_TOKEN_BYTES)
    segs["len"] = ntok[req] * KV_TOKEN_BYTES
    segs["nonce"] = nonce_triple(uids[req], lay, 0)
    buf_bytes = layers * T * KV_TOKEN_BYTES
    token_owner = np.repeat(uids, ntok).astype(np.int32)
    owner_map = np.tile(token_owner, layers)          # crypto units: one per (layer, token)
    buf = None
    if fill:
        buf = bf16_normal(rng, buf_bytes // 2, 1.0).view(np.uint8)

    # Flow-rule inputs.  Each request reads a context of KV blocks it owns.
    ctx_blocks = rng.integers(1, 9, size=n_users)
    n_kv = int(ctx_blocks.sum())
    kv_perm = rng.permutation(n_kv).astype(np.int32)
    kv_owner = np.empty(n_kv, dtype=np.int32)
    src_ptr = np.concatenate([[0], np.cumsum(ctx_blocks)]).astype(np.int32)
    kv_owner[kv_perm] = np.repeat(uids, ctx_blocks)
    block_table = kv_perm.copy()
    n_redirect = max(1, int(round(poison_frac * n_kv)))
    red_entries = rng.choice(n_kv, size=n_redirect, replace=False)
    block_table_attacked = block_table.copy()
    for e in red_entries:
        r = int(np.searchsorted(src_ptr, e, side="right") - 1)
        victim = int(rng.integers(0, n_users - 1))
        victim += victim >= r
        block_table_attacked[e] = kv_perm[src_ptr[victim]]     # first block of another user
    seg_ptr = np.concatenate([[0], np.cumsum(ntok)]).astype(np.int32)
    gather = np.repeat(seg_ptr[1:] - 1, ntok).astype(np.int32)   # every token <- request's last token

    # Tampering plan.
    n_poison = max(3, int(round(poison_frac * nseg)))
    poisoned = np.sort(rng.choice(nseg, size=n_poison, replace=False))
    kinds = np.arange(n_poison) % 3            # 0: ciphertext bit, 1: tag bit, 2: wrong owner
    rng.shuffle(kinds)
    bitpos = np.array([int(rng.integers(0, int(segs["len"][s]) * 8)) for s in poisoned], dtype=np.int64)
    tagbit = rng.integers(0, 128, size=n_poison)
    wrong = np.array([(int(segs["owner"][s]) + 1 + int(rng.integers(0, n_users - 1))) % n_users
                      for s in poisoned], dtype=np.int32)
    return Workload("c5_mixed", uids, keys, n_users, buf, buf_bytes, segs,
                    owner_map=owner_map, unit_bytes=KV_TOKEN_BYTES,
                    extra={"layers": layers, "T": T, "ntok": ntok, "tok0": tok0,
                           "token_owner": token_owner, "seg_ptr": seg_ptr,
                           "kv_owner": kv_owner, "src_ptr": src_ptr, "block_table": block_table,
                           "block_table_attacked": block_table_attacked,
                           "redirected_requests": np.unique(
                               np.searchsorted(src_ptr, red_entries, side="right") - 1),
                           "gather": gather,
                           "poisoned": poisoned, "poison_kind": kinds, "poison_bit": bitpos,
                           "poison_tagbit": tagbit, "poison_owner": wrong})


def bump_epoch(segs: np.ndarray) -> np.ndarray:
    """Copy of a segment table whose nonces differ from the original: bit 31 of the second word.

    Re-encrypting the same position under the same key must never reuse a nonce.
    """
    out = segs.copy()
    out["nonce"][:, 7] ^= 0x80
    return out


# --------------------------------------------------------------------------
# Launch traces for the multi-stream launch-order check (paper sec. 4.4)
# --------------------------------------------------------------------------
def launch_trace(n_launches: int = 2000, n_segments: int = 512, n_streams: int = 3, race_frac: float = 0.02,
                 seed_salt: int = 0):
    """A seeded trace of kernel launches and synchronisations over n_streams streams.

    Stream 0 is the compute stream: each launch reads a handful of KV-block segments and
    writes one or two.  The other streams swap KV blocks in the background (one write, or
    one read, per launch).  A well-behaved framework synchronises a background stream before
    the compute stream touches what it wrote, and the other way round; with probability
    race_frac that synchronisation is left out, which plants a race.
    Returns a dict of numpy arrays: kind, stream (per event), acc_ptr, acc_seg, acc_write.
    """
    rng = _rng(6, seed_salt)
    kind, stream, acc_ptr, acc_seg, acc_write = [], [], [0], [], []
    dirty = {}          # segment -> (stream, event) of an access not yet synchronised

    def emit_sync(s):
        kind.append(1)
        stream.append(s)
        acc_ptr.append(len(acc_seg))
        for m in [m for m, (st, _) in dirty.items() if st == s]:
            del dirty[m]

    def emit_launch(s, reads, writes):
        for m in list(reads) + list(writes):
            if m in dirty and dirty[m][0] != s and rng.random() >= race_frac:
                emit_sync(dirty[m][0])
        kind.append(0)
        stream.append(s)
        for m in reads:
            acc_seg.append(int(m))
            acc_write.append(0)
        for m in writes:
            acc_seg.append(int(m))
            acc_write.append(1)
        acc_ptr.append(len(acc_seg))
        e = len(kind) - 1
        for m in list(reads) + list(writes):
            dirty[int(m)] = (s, e)

    for _ in range(n_launches):
        if n_streams > 1 and rng.random() < 0.25:
            s = int(rng.integers(1, n_streams))
            m = int(rng.integers(0, n_segments))
            if rng.random() < 0.5:
                emit_launch(s, [], [m])         # swap in: overwrite a block
            else:
                emit_launch(s, [m], [])         # swap out: read a block
        else:
            reads = rng.choice(n_segments, size=min(n_segments, int(rng.integers(1, 9))), replace=False)
            writes = rng.choice(n_segments, size=min(n_segments, int(rng.integers(1, 3))), replace=False)
            emit_launch(0, reads, writes)
        if rng.random() < 0.02:
            emit_sync(int(rng.integers(0, n_streams)))
    return {"kind": np.array(kind, dtype=np.uint8), "stream": np.array(stream, dtype=np.int32),
            "acc_ptr": np.array(acc_ptr, dtype=np.int32), "acc_seg": np.array(acc_seg, dtype=np.int32),
            "acc_write": np.array(acc_write, dtype=np.uint8), "n_streams": n_streams, "n_segments": n_segments}


def trace_by_segment(acc_ptr, acc_seg, acc_write, n_segments):
    """The accesses of a launch trace grouped per segment in launch order (the history that
    the extended ownership records accumulate): (seg_ptr int32[n_segments+1],
    seg_event int32[A], seg_write uint8[A]).  A stable sort only; no checking logic."""
    n_events = len(acc_ptr) - 1
    ev = np.repeat(np.arange(n_events, dtype=np.int32), np.diff(acc_ptr))
    order = np.argsort(np.asarray(acc_seg), kind="stable")
    counts = np.bincount(np.asarray(acc_seg, dtype=np.int64), minlength=n_segments)
    seg_ptr = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    return seg_ptr, ev[order].astype(np.int32), np.asarray(acc_write, dtype=np.uint8)[order]
