"""Thin ctypes binding over libgift.so: argument marshalling only.

Function names follow include/gift.h.  Data arguments are torch CUDA tensors (their
data_ptr() is passed through); key material is passed from host numpy arrays.  There is
no fallback: if the library has not been built, or no CUDA device is present, the first
call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("GIFT_LIB", os.path.join(_HERE, "libgift.so"))

OK, E_INVAL, E_NOMEM, E_CUDA, E_RANGE, E_ALIGN = 0, -1, -2, -3, -4, -5
ST_TAG_MISMATCH, ST_OWNER_MISMATCH, ST_UNOWNED, ST_NO_KEY, ST_BAD_DESC, ST_OVERLAP = 1, 2, 4, 8, 16, 32
CTX_TWO_TABLES, CTX_CHECK_OVERLAP, CTX_SPLIT_LAUNCH = 1, 2, 4
OWNER_PARAM, OWNER_NONE, OWNER_CONFLICT = -1, -2, -3
RULE_IDENTITY, RULE_ROWWISE, RULE_SEGREDUCE, RULE_BROADCAST = 0, 1, 2, 3
STATIC_MAX_SEGS = 65536

EXPORTS = [
    "gift_ctx_create", "gift_ctx_destroy", "gift_ctx_reserve", "gift_set_keys", "gift_clear_keys",
    "gift_ctx_bind_aad", "gift_seg_encrypt", "gift_seg_encrypt_static", "gift_seg_decrypt", "gift_verify_tags",
    "gift_propagate_labels", "gift_propagate_chain", "gift_tok_encrypt", "gift_tok_decrypt", "gift_check_launch_order",
    "gift_resolve_args", "gift_slice_runs", "gift_expand_owners", "gift_labels_swap_out", "gift_labels_swap_in",
    "gift_strerror", "gift_version", "gift_launch_count", "gift_timing_enable", "gift_timing_read",
    "gift_export_to_host", "gift_import_from_host", "gift_last_error_detail",
]


class GiftError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        detail = ""
        if code in (E_CUDA, E_NOMEM):
            detail = ": " + lib().gift_last_error_detail().decode()
        super().__init__("%s failed: %s (%d)%s" % (where, strerror(code), code, detail))


class _Pages(C.Structure):
    _fields_ = [("table", C.c_void_p), ("n", C.c_uint32), ("page_bytes", C.c_uint64)]


class _Labels(C.Structure):
    _fields_ = [("owner_map", C.c_void_p), ("n_units", C.c_uint32), ("unit_bytes", C.c_uint64)]


class _Rule(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("n_out", C.c_uint32), ("n_in", C.c_uint32), ("n_seg", C.c_uint32),
                ("n_in0", C.c_uint32), ("n_in1", C.c_uint32), ("n_src", C.c_uint32),
                ("seg_ptr", C.c_void_p), ("src_ptr", C.c_void_p), ("src_idx", C.c_void_p),
                ("gather", C.c_void_p), ("param_mask", C.c_uint32)]


class Chunk(C.Structure):
    """gift_chunk: the segments [seg_lo, seg_hi) of the table and the byte range that holds them."""
    _fields_ = [("byte_lo", C.c_uint64), ("byte_hi", C.c_uint64), ("seg_lo", C.c_uint32), ("seg_hi", C.c_uint32)]


class _Trace(C.Structure):
    _fields_ = [("n_events", C.c_uint32), ("n_streams", C.c_uint32), ("n_segments", C.c_uint32),
                ("kind", C.c_void_p), ("stream", C.c_void_p), ("seg_ptr", C.c_void_p),
                ("seg_event", C.c_void_p), ("seg_write", C.c_void_p)]


RACE_RAW, RACE_WAR, RACE_WAW = 1, 2, 4
ARG_OK, ARG_UNKNOWN, ARG_SHAPE, ARG_ALIAS = 0, 1, 2, 4
MAX_DIMS = 5


class TensorRec(C.Structure):
    """gift_tensor_rec: base address, shape, element size, ownership-related dimensions, level-2 owners."""
    _fields_ = [("base", C.c_uint64), ("ndim", C.c_uint32), ("elem_size", C.c_uint32),
                ("shape", C.c_uint64 * MAX_DIMS), ("odim_mask", C.c_uint32), ("owners", C.c_void_p)]

    @classmethod
    def make(cls, base, shape, elem_size, odims, owners_ptr=None):
        r = cls()
        r.base, r.ndim, r.elem_size = int(base), len(shape), int(elem_size)
        for d, n in enumerate(shape):
            r.shape[d] = int(n)
        r.odim_mask = sum(1 << d for d in odims)
        r.owners = owners_ptr
        return r


class KernelArg(C.Structure):
    _fields_ = [("base", C.c_uint64), ("ndim", C.c_uint32), ("alias_group", C.c_uint32),
                ("shape", C.c_uint64 * MAX_DIMS)]

    @classmethod
    def make(cls, base, shape, alias_group=0):
        a = cls()
        a.base, a.ndim, a.alias_group = int(base), len(shape), int(alias_group)
        for d, n in enumerate(shape):
            a.shape[d] = int(n)
        return a


def resolve_args(recs, args):
    """Steps (1)-(3) of a flow rule on host records: (record index per argument, status bits per argument)."""
    rarr = (TensorRec * max(1, len(recs)))(*recs)
    aarr = (KernelArg * max(1, len(args)))(*args)
    idx = (C.c_int32 * max(1, len(args)))()
    st = (C.c_uint32 * max(1, len(args)))()
    f = lib().gift_resolve_args
    f.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
    _check(f(rarr, len(recs), aarr, len(args), idx, st), "gift_resolve_args")
    return list(idx)[: len(args)], list(st)[: len(args)]


def slice_runs(rec, lo, hi):
    """(run_bytes, page numbers) of the slice [lo, hi) of a recorded tensor."""
    lo_a = (C.c_uint64 * MAX_DIMS)(*[int(x) for x in lo])
    hi_a = (C.c_uint64 * MAX_DIMS)(*[int(x) for x in hi])
    run, n = C.c_uint64(), C.c_uint32()
    f = lib().gift_slice_runs
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32]
    _check(f(C.byref(rec), lo_a, hi_a, C.byref(run), C.byref(n), None, 0), "gift_slice_runs")
    table = np.zeros(max(1, n.value), dtype=np.int32)
    _check(f(C.byref(rec), lo_a, hi_a, C.byref(run), C.byref(n), table.ctypes.data_as(C.c_void_p), table.size),
           "gift_slice_runs")
    return run.value, table[: n.value]

_lib = None


def lib():
    """Load libgift.so; raises if it is missing (build it with `python -m paper_2608_25431_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libgift.so is not built: run python -m paper_2608_25431_b200.build "
                               "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        l.gift_ctx_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_uint32, C.c_uint32]
        l.gift_ctx_destroy.argtypes = [C.c_void_p]
        l.gift_ctx_reserve.argtypes = [C.c_void_p, C.c_uint32]
        l.gift_set_keys.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
        l.gift_clear_keys.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
        l.gift_seg_encrypt.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint32,
                                       C.POINTER(_Pages), C.POINTER(_Labels), C.c_void_p, C.c_void_p, C.c_void_p]
        l.gift_seg_decrypt.argtypes = l.gift_seg_encrypt.argtypes
        l.gift_seg_encrypt_static.argtypes = l.gift_seg_encrypt.argtypes
        l.gift_verify_tags.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint32,
                                       C.POINTER(_Pages), C.c_void_p, C.c_void_p, C.c_void_p]
        l.gift_propagate_labels.argtypes = [C.c_void_p, C.POINTER(_Rule), C.POINTER(C.c_void_p), C.c_void_p,
                                            C.c_void_p, C.c_void_p]
        l.gift_propagate_chain.argtypes = [C.c_void_p, C.POINTER(_Rule), C.POINTER(C.POINTER(C.c_void_p)),
                                           C.POINTER(C.c_void_p), C.c_uint32, C.c_void_p, C.c_void_p]
        l.gift_tok_encrypt.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint64,
                                       C.c_void_p, C.c_void_p, C.c_void_p]
        l.gift_tok_decrypt.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint64, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p]
        l.gift_check_launch_order.argtypes = [C.c_void_p, C.POINTER(_Trace), C.c_void_p, C.c_void_p, C.c_void_p]
        l.gift_last_error_detail.restype = C.c_char_p
        l.gift_strerror.restype = C.c_char_p
        l.gift_strerror.argtypes = [C.c_int]
        l.gift_version.restype = C.c_uint32
        l.gift_launch_count.restype = C.c_uint64
        l.gift_launch_count.argtypes = [C.c_void_p]
        l.gift_timing_enable.argtypes = [C.c_void_p, C.c_int]
        l.gift_timing_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_uint32)]
        l.gift_ctx_bind_aad.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32]
        l.gift_export_to_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                          C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.POINTER(_Pages),
                                          C.POINTER(_Labels), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.gift_import_from_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p,
                                            C.c_uint32, C.c_void_p, C.c_uint32, C.POINTER(_Pages), C.POINTER(_Labels),
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = l
    return _lib


def strerror(code: int) -> str:
    return lib().gift_strerror(code).decode()


def version() -> int:
    return int(lib().gift_version())


def _check(rc, where):
    if rc != OK:
        raise GiftError(rc, where)


def _stream_ptr(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return C.c_void_p(int(stream))


def _dev(t):
    """Device-visible pointer of a contiguous CUDA tensor, or of a pinned host tensor (page-locked
    host memory has the same address on the device under unified addressing), or None."""
    if t is None:
        return None
    if not (t.is_cuda or t.is_pinned()) or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor or a pinned host tensor")
    return C.c_void_p(t.data_ptr())


class Ctx:
    """A libgift context: per-user keys on one device.  See include/gift.h for semantics."""

    def __init__(self, max_users: int, device: int = 0, flags: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("libgift needs a CUDA device; there is no CPU fallback")
        self._h = C.c_void_p()
        _check(lib().gift_ctx_create(C.byref(self._h), device, max_users, flags), "gift_ctx_create")
        self.max_users = max_users
        self.device = device

    def close(self):
        if self._h:
            lib().gift_ctx_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def bind_aad(self, aad16):
        """aad16: CUDA uint8 tensor [n, 16] authenticated with the segments of the calls that follow, or None."""
        self._aad = aad16            # keep the tensor alive while it is bound
        n = 0 if aad16 is None else aad16.numel() // 16
        _check(lib().gift_ctx_bind_aad(self._h, _dev(aad16), n), "gift_ctx_bind_aad")

    def reserve(self, max_segs: int):
        _check(lib().gift_ctx_reserve(self._h, max_segs), "gift_ctx_reserve")

    def set_keys(self, user_ids, keys16, stream=None):
        ids = np.ascontiguousarray(user_ids, dtype=np.int32)
        keys = np.ascontiguousarray(keys16, dtype=np.uint8).reshape(-1)
        if keys.size != 16 * ids.size:
            raise ValueError("keys16 must hold 16 bytes per user id")
        _check(lib().gift_set_keys(self._h, ids.ctypes.data_as(C.c_void_p), keys.ctypes.data_as(C.c_void_p),
                                   ids.size, _stream_ptr(stream)), "gift_set_keys")

    def clear_keys(self, user_ids, stream=None):
        ids = np.ascontiguousarray(user_ids, dtype=np.int32)
        _check(lib().gift_clear_keys(self._h, ids.ctypes.data_as(C.c_void_p), ids.size, _stream_ptr(stream)),
               "gift_clear_keys")

    @staticmethod
    def _tables(page_table, page_bytes, owner_map, unit_bytes):
        pg = lb = None
        if page_table is not None:
            pg = _Pages(page_table.data_ptr(), page_table.numel(), page_bytes)
        if owner_map is not None:
            lb = _Labels(owner_map.data_ptr(), owner_map.numel(), unit_bytes)
        return pg, lb

    def seg_encrypt(self, src, dst, segs, nseg, tags_out, status, page_table=None, page_bytes=0,
                    owner_map=None, unit_bytes=0, stream=None):
        pg, lb = self._tables(page_table, page_bytes, owner_map, unit_bytes)
        _check(lib().gift_seg_encrypt(self._h, _dev(src), _dev(dst), src.numel() * src.element_size(), _dev(segs),
                                      nseg, C.byref(pg) if pg else None, C.byref(lb) if lb else None,
                                      _dev(tags_out), _dev(status), _stream_ptr(stream)), "gift_seg_encrypt")

    def seg_encrypt_static(self, src, dst, segs, nseg, tags_out, status, page_table=None, page_bytes=0,
                           owner_map=None, unit_bytes=0, stream=None):
        """gift_seg_encrypt_static: same results as seg_encrypt, but allocates nothing.

        For callers that cannot call cudaMalloc when they export data; at most
        STATIC_MAX_SEGS segments per call, and calls that overlap on the GPU race on the
        library's fixed scratch array (see include/gift.h)."""
        pg, lb = self._tables(page_table, page_bytes, owner_map, unit_bytes)
        _check(lib().gift_seg_encrypt_static(self._h, _dev(src), _dev(dst), src.numel() * src.element_size(),
                                             _dev(segs), nseg, C.byref(pg) if pg else None,
                                             C.byref(lb) if lb else None, _dev(tags_out), _dev(status),
                                             _stream_ptr(stream)), "gift_seg_encrypt_static")

    def seg_decrypt(self, src, dst, segs, nseg, tags_in, status, page_table=None, page_bytes=0,
                    owner_map=None, unit_bytes=0, stream=None):
        pg, lb = self._tables(page_table, page_bytes, owner_map, unit_bytes)
        _check(lib().gift_seg_decrypt(self._h, _dev(src), _dev(dst), src.numel() * src.element_size(), _dev(segs),
                                      nseg, C.byref(pg) if pg else None, C.byref(lb) if lb else None,
                                      _dev(tags_in), _dev(status), _stream_ptr(stream)), "gift_seg_decrypt")

    def verify_tags(self, src, segs, nseg, tags_in, status, page_table=None, page_bytes=0, stream=None):
        pg, _ = self._tables(page_table, page_bytes, None, 0)
        _check(lib().gift_verify_tags(self._h, _dev(src), src.numel() * src.element_size(), _dev(segs), nseg,
                                      C.byref(pg) if pg else None, _dev(tags_in), _dev(status),
                                      _stream_ptr(stream)), "gift_verify_tags")

    def propagate_labels(self, kind, in_maps, out_map, viol, *, n_out=None, param_mask=0, seg_ptr=None,
                         src_ptr=None, src_idx=None, gather=None, stream=None):
        n_out = out_map.numel() if n_out is None else n_out
        n_seg = seg_ptr.numel() - 1 if seg_ptr is not None else 0
        rule = _Rule(kind, n_out, len(in_maps), n_seg,
                     in_maps[0].numel(), in_maps[1].numel() if len(in_maps) > 1 else 0,
                     src_idx.numel() if src_idx is not None else 0,
                     seg_ptr.data_ptr() if seg_ptr is not None else None,
                     src_ptr.data_ptr() if src_ptr is not None else None,
                     src_idx.data_ptr() if src_idx is not None else None,
                     gather.data_ptr() if gather is not None else None, param_mask)
        arr = (C.c_void_p * len(in_maps))(*[m.data_ptr() for m in in_maps])
        _check(lib().gift_propagate_labels(self._h, C.byref(rule), arr, _dev(out_map), _dev(viol),
                                           _stream_ptr(stream)), "gift_propagate_labels")

    def prepare_chain(self, rules):
        """Marshal a rule chain once; the returned callable (viol, stream=None) runs
        gift_propagate_chain on it.  `rules` is a list of dicts with the keyword arguments of
        propagate_labels (kind, in_maps, out_map and the rule's index arrays).  The tensors
        named in `rules` must stay alive and in place while the callable is used."""
        n = len(rules)
        arr = (_Rule * max(n, 1))()
        ins = (C.POINTER(C.c_void_p) * max(n, 1))()
        outs = (C.c_void_p * max(n, 1))()
        keep = [rules]
        for k, r in enumerate(rules):
            in_maps, out_map = r["in_maps"], r["out_map"]
            seg_ptr, src_ptr = r.get("seg_ptr"), r.get("src_ptr")
            src_idx, gather = r.get("src_idx"), r.get("gather")
            n_out = r.get("n_out", out_map.numel())
            arr[k] = _Rule(r["kind"], n_out, len(in_maps), seg_ptr.numel() - 1 if seg_ptr is not None else 0,
                           in_maps[0].numel(), in_maps[1].numel() if len(in_maps) > 1 else 0,
                           src_idx.numel() if src_idx is not None else 0,
                           seg_ptr.data_ptr() if seg_ptr is not None else None,
                           src_ptr.data_ptr() if src_ptr is not None else None,
                           src_idx.data_ptr() if src_idx is not None else None,
                           gather.data_ptr() if gather is not None else None, r.get("param_mask", 0))
            a = (C.c_void_p * len(in_maps))(*[m.data_ptr() for m in in_maps])
            keep.append(a)
            ins[k] = C.cast(a, C.POINTER(C.c_void_p))
            outs[k] = out_map.data_ptr()
        fn, h = lib().gift_propagate_chain, self._h

        def run(viol, stream=None, _keep=keep):
            _check(fn(h, arr, ins, outs, n, _dev(viol), _stream_ptr(stream)), "gift_propagate_chain")
        return run

    def propagate_chain(self, rules, viol, stream=None):
        """gift_propagate_chain on `rules` (see prepare_chain); viol holds 2 * len(rules) words."""
        self.prepare_chain(rules)(viol, stream)

    def tok_encrypt(self, tokens, nonces, owners, eos_token, out16, status, stream=None):
        _check(lib().gift_tok_encrypt(self._h, _dev(tokens), _dev(nonces), _dev(owners), tokens.numel(),
                                      int(eos_token), _dev(out16), _dev(status), _stream_ptr(stream)),
               "gift_tok_encrypt")

    def tok_decrypt(self, in16, owners, eos_token, tokens_out, status, nonces_out=None, stream=None):
        _check(lib().gift_tok_decrypt(self._h, _dev(in16), _dev(owners), owners.numel(), int(eos_token),
                                      _dev(tokens_out), _dev(nonces_out), _dev(status), _stream_ptr(stream)),
               "gift_tok_decrypt")

    def check_launch_order(self, kind, stream_ids, seg_ptr, seg_event, seg_write, n_streams, flags, summary,
                           stream=None):
        import torch
        if seg_event.numel() == 0:       # no accesses at all: the library still wants valid pointers
            seg_event = torch.zeros(1, dtype=torch.int32, device=seg_ptr.device)
            seg_write = torch.zeros(1, dtype=torch.uint8, device=seg_ptr.device)
        t = _Trace(kind.numel(), n_streams, seg_ptr.numel() - 1, kind.data_ptr(), stream_ids.data_ptr(),
                   seg_ptr.data_ptr(), seg_event.data_ptr(), seg_write.data_ptr())
        _check(lib().gift_check_launch_order(self._h, C.byref(t), _dev(flags), _dev(summary), _stream_ptr(stream)),
               "gift_check_launch_order")

    def expand_owners(self, rec, run_bytes, unit_owner, stream=None):
        f = lib().gift_expand_owners
        f.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint32, C.c_void_p]
        _check(f(self._h, C.byref(rec), int(run_bytes), _dev(unit_owner), unit_owner.numel(), _stream_ptr(stream)),
               "gift_expand_owners")

    def labels_swap_out(self, owner_map, units, saved, viol, stream=None):
        f = lib().gift_labels_swap_out
        f.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p]
        _check(f(self._h, _dev(owner_map), owner_map.numel(), _dev(units), units.numel(), _dev(saved), _dev(viol),
                 _stream_ptr(stream)), "gift_labels_swap_out")

    def labels_swap_in(self, owner_map, units, saved, viol, stream=None):
        f = lib().gift_labels_swap_in
        f.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p]
        _check(f(self._h, _dev(owner_map), owner_map.numel(), _dev(units), units.numel(), _dev(saved), _dev(viol),
                 _stream_ptr(stream)), "gift_labels_swap_in")

    @staticmethod
    def chunk_array(chunks):
        """HOST array of gift_chunk from (byte_lo, byte_hi, seg_lo, seg_hi) tuples or Chunk objects."""
        arr = (Chunk * max(1, len(chunks)))()
        for k, ch in enumerate(chunks):
            arr[k] = ch if isinstance(ch, Chunk) else Chunk(*[int(v) for v in ch])
        return arr

    def export_to_host(self, h_src, h_dst, d_plain, d_cipher, segs, nseg, chunks, d_tags, d_status, h_tags, h_status,
                       page_table=None, page_bytes=0, owner_map=None, unit_bytes=0, stream=None):
        """gift_export_to_host; chunks is a list of (byte_lo, byte_hi, seg_lo, seg_hi) or a prepared chunk_array."""
        arr = chunks if isinstance(chunks, C.Array) else self.chunk_array(chunks)
        pg, lb = self._tables(page_table, page_bytes, owner_map, unit_bytes)
        _check(lib().gift_export_to_host(self._h, _dev(h_src), _dev(h_dst), _dev(d_plain), _dev(d_cipher),
                                         d_plain.numel() * d_plain.element_size(), _dev(segs), nseg, arr, len(arr) if len(chunks) else 0,
                                         C.byref(pg) if pg else None, C.byref(lb) if lb else None, _dev(d_tags),
                                         _dev(d_status), _dev(h_tags), _dev(h_status), _stream_ptr(stream)),
               "gift_export_to_host")

    def import_from_host(self, h_src, h_tags, d_buf, segs, nseg, chunks, d_tags, d_status, h_status,
                         page_table=None, page_bytes=0, owner_map=None, unit_bytes=0, stream=None):
        """gift_import_from_host; chunks as for export_to_host."""
        arr = chunks if isinstance(chunks, C.Array) else self.chunk_array(chunks)
        pg, lb = self._tables(page_table, page_bytes, owner_map, unit_bytes)
        _check(lib().gift_import_from_host(self._h, _dev(h_src), _dev(h_tags), _dev(d_buf),
                                           d_buf.numel() * d_buf.element_size(), _dev(segs), nseg, arr,
                                           len(arr) if len(chunks) else 0, C.byref(pg) if pg else None,
                                           C.byref(lb) if lb else None, _dev(d_tags), _dev(d_status), _dev(h_status),
                                           _stream_ptr(stream)), "gift_import_from_host")

    def launch_count(self) -> int:
        return int(lib().gift_launch_count(self._h))

    def timing_enable(self, on: bool = True):
        _check(lib().gift_timing_enable(self._h, 1 if on else 0), "gift_timing_enable")

    def timing_read(self):
        """(total milliseconds, launches) of the cipher kernel since the last read."""
        ms, n = C.c_double(), C.c_uint32()
        _check(lib().gift_timing_read(self._h, C.byref(ms), C.byref(n)), "gift_timing_read")
        return ms.value, n.value


PROBE_KINDS = {0: "lop3", 1: "mad.wide.u32", 2: "prmt", 3: "ld.shared.u32", 4: "shf", 5: "add.u32",
               6: "lop3+mad.wide", 7: "mad.lo.u32", 8: "lop3+ld.shared", 9: "mul.wide.u32",
               10: "lop3+mul.wide", 11: "lop3+mad.lo", 12: "lop3+add", 13: "prmt+mad.wide",
               14: "lop3(imm)+mad.wide", 15: "2 lop3+mad.wide", 16: "ld.shared+mad.wide", 17: "lop3+prmt", 18: "mul.hi.u32", 19: "lop3+mul.hi",
               20: "cipher mix (15 logic, 5 multiply, 4 lookups per 24)", 21: "2 lop3+mul.wide",
               22: "lop3+prmt+mul.wide", 23: "3 lop3+ld.shared", 24: "2 lop3+mul.wide+ld.shared+xor",
               25: "2 lop3 (low half)+mul.wide", 26: "2 lop3 (high half)+mul.wide", 27: "2 lop3+mad.lo",
               28: "3 lop3+mul.wide", 29: "lop3(low,high)+lop3+mul.wide", 30: "mad.lo(high)+2 lop3+mul.wide",
               31: "prmt(high)+lop3+mul.wide", 32: "mul.wide, 4 lop3, lop3(high)", 33: "brev", 34: "lop3+brev",
               35: "mma.sync m16n8k128 b1 and.popc (one lane-op per thread)", 36: "2 mad.lo + lop3 on their results"}


def probe_pipe(kind: int, iters: int = 2000, device: int = 0):
    """(lane-operations per SM clock, SM MHz seen) for one instruction kind.

    Diagnostics: calls libgift_probe.so (built by build.build_probe), which is not part of libgift.so."""
    from . import build
    probe = C.CDLL(build.build_probe())
    probe.gift_probe_pipe.argtypes = [C.c_int, C.c_int, C.c_uint32, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    ops, mhz = C.c_double(), C.c_double()
    rc = probe.gift_probe_pipe(device, kind, iters, C.byref(ops), C.byref(mhz))
    if rc != 0:
        raise RuntimeError("gift_probe_pipe failed (%d)" % rc)
    return ops.value, mhz.value


# ---------------------------------------------------------------------------------------
# The same calls under the names of include/gift.h, for callers that prefer the C spelling.
# ---------------------------------------------------------------------------------------
def gift_ctx_create(max_users: int, device: int = 0, flags: int = 0) -> Ctx:
    return Ctx(max_users, device, flags)


def gift_ctx_destroy(ctx: Ctx):
    ctx.close()


def gift_ctx_bind_aad(ctx: Ctx, aad16):
    ctx.bind_aad(aad16)


def gift_ctx_reserve(ctx: Ctx, max_segs: int):
    ctx.reserve(max_segs)


def gift_set_keys(ctx: Ctx, user_ids, keys16, stream=None):
    ctx.set_keys(user_ids, keys16, stream)


def gift_clear_keys(ctx: Ctx, user_ids, stream=None):
    ctx.clear_keys(user_ids, stream)


def gift_seg_encrypt(ctx: Ctx, *args, **kw):
    ctx.seg_encrypt(*args, **kw)


def gift_seg_encrypt_static(ctx: Ctx, *args, **kw):
    ctx.seg_encrypt_static(*args, **kw)


def gift_seg_decrypt(ctx: Ctx, *args, **kw):
    ctx.seg_decrypt(*args, **kw)


def gift_verify_tags(ctx: Ctx, *args, **kw):
    ctx.verify_tags(*args, **kw)


def gift_propagate_labels(ctx: Ctx, *args, **kw):
    ctx.propagate_labels(*args, **kw)


def gift_propagate_chain(ctx: Ctx, *args, **kw):
    ctx.propagate_chain(*args, **kw)


def gift_tok_encrypt(ctx: Ctx, *args, **kw):
    ctx.tok_encrypt(*args, **kw)


def gift_tok_decrypt(ctx: Ctx, *args, **kw):
    ctx.tok_decrypt(*args, **kw)


def gift_check_launch_order(ctx: Ctx, *args, **kw):
    ctx.check_launch_order(*args, **kw)


def gift_expand_owners(ctx: Ctx, *args, **kw):
    ctx.expand_owners(*args, **kw)


def gift_labels_swap_out(ctx: Ctx, *args, **kw):
    ctx.labels_swap_out(*args, **kw)


def gift_labels_swap_in(ctx: Ctx, *args, **kw):
    ctx.labels_swap_in(*args, **kw)


def gift_timing_enable(ctx: Ctx, on: bool = True):
    ctx.timing_enable(on)


def gift_timing_read(ctx: Ctx):
    return ctx.timing_read()


def gift_launch_count(ctx: Ctx) -> int:
    return ctx.launch_count()


def gift_export_to_host(ctx: Ctx, *args, **kw):
    ctx.export_to_host(*args, **kw)


def gift_import_from_host(ctx: Ctx, *args, **kw):
    ctx.import_from_host(*args, **kw)


def gift_last_error_detail() -> str:
    return lib().gift_last_error_detail().decode()


gift_resolve_args = resolve_args
gift_slice_runs = slice_runs
gift_strerror = strerror
gift_version = version
