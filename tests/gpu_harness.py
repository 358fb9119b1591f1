"""Helpers for the GPU parity tests: run a workload through the C-ABI binding and through the oracle."""
import numpy as np
import torch

from oracle import gcm
from paper_2608_25431_b200 import binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def segs_dev(segs):
    return torch.from_numpy(np.ascontiguousarray(segs).view(np.uint8).copy()).cuda()


def make_ctx(w, flags=0, user_ids=None, keys=None):
    ctx = binding.Ctx(w.max_users, 0, flags)
    ctx.set_keys(w.user_ids if user_ids is None else user_ids, w.keys if keys is None else keys)
    return ctx


def gpu_encrypt(ctx, w, src, dst=None, segs=None, owner_map="default"):
    """src, dst: CUDA uint8 tensors (dst None: in place).  Returns (tags, status) CUDA tensors."""
    segs = w.segs if segs is None else segs
    n = len(segs)
    om = w.owner_map if isinstance(owner_map, str) else owner_map
    tags = torch.full((max(n, 1), 16), 0xAB, dtype=torch.uint8, device="cuda")
    status = torch.full((max(n, 1),), 0xDEAD, dtype=torch.int32, device="cuda")
    ctx.seg_encrypt(src, src if dst is None else dst, segs_dev(segs), n, tags, status,
                    page_table=dev(w.page_table) if w.page_table is not None else None, page_bytes=w.page_bytes,
                    owner_map=dev(om) if om is not None else None, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    return tags[:n], status[:n]


def gpu_decrypt(ctx, w, src, tags, dst=None, segs=None, owner_map=None, verify_only=False):
    """owner_map: CUDA int32 tensor updated in place, or None.  Returns status CUDA tensor."""
    segs = w.segs if segs is None else segs
    n = len(segs)
    status = torch.full((max(n, 1),), 0xDEAD, dtype=torch.int32, device="cuda")
    tg = tags.contiguous() if tags.numel() else torch.zeros(16, dtype=torch.uint8, device="cuda")
    pt = dev(w.page_table) if w.page_table is not None else None
    if verify_only:
        ctx.verify_tags(src, segs_dev(segs), n, tg, status, page_table=pt, page_bytes=w.page_bytes)
    else:
        ctx.seg_decrypt(src, src if dst is None else dst, segs_dev(segs), n, tg, status, page_table=pt,
                        page_bytes=w.page_bytes, owner_map=owner_map, unit_bytes=w.unit_bytes)
    torch.cuda.synchronize()
    return status[:n]


def oracle_encrypt(w, src, dst, segs=None, owner_map="default", user_ids=None, keys=None):
    segs = w.segs if segs is None else segs
    om = w.owner_map if isinstance(owner_map, str) else owner_map
    return gcm.seg_encrypt(src, dst, segs, w.user_ids if user_ids is None else user_ids,
                           w.keys if keys is None else keys, w.max_users, w.page_table, w.page_bytes, om,
                           w.unit_bytes)


def oracle_decrypt(w, src, dst, tags, segs=None, owner_map=None, verify_only=False):
    segs = w.segs if segs is None else segs
    return gcm.seg_decrypt(src, dst, segs, tags, w.user_ids, w.keys, w.max_users, w.page_table, w.page_bytes,
                           owner_map, w.unit_bytes, verify_only=verify_only)


def np_(t):
    return t.detach().cpu().numpy()


def st_(t):
    return np_(t).astype(np.uint32)
