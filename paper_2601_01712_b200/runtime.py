"""Owners of device memory for the C-ABI library, built on PyTorch tensors.

PyTorch is used for allocation, streams and copies only; every step of the
model runs inside ``librelaygr.so``.  These classes marshal arguments and keep
the borrowed buffers alive, nothing else.
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as B
from . import synth


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


class Model:
    """Uploads one set of synthetic weights and creates the library context."""

    def __init__(self, shape: synth.ModelShape, weights: synth.Weights, device: str = "cuda:0"):
        self.shape = shape
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self._t = {}
        for name, a in weights.mat.items():
            if shape.dtype == synth.DTYPE_BF16:
                t = torch.from_numpy(weights.bits[name].view(np.int16)).to(self.device).view(torch.bfloat16)
            else:
                t = torch.from_numpy(a).to(self.device)
            self._t[name] = t.contiguous()
        for name, a in weights.vec.items():
            self._t[name] = torch.from_numpy(a).to(self.device).contiguous()
        self.cfg = B.ModelCfg(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.dtype,
                              shape.page_tokens, weights.mat["emb"].shape[0], shape.ln_eps, shape.attn_kind)
        w = B.Weights()
        for name in B.WEIGHT_FIELDS:
            setattr(w, name, self._t[name].data_ptr())
        self._w = w
        self.ctx = B.relaygr_create(self.cfg, w)
        self._ws = None
        self.page_bytes = B.relaygr_kv_page_bytes(self.ctx)

    def new_slot(self) -> "Model":
        """Another context on the same weights (a model slot): its own workspace, usable with the same pool."""
        other = object.__new__(Model)
        other.shape, other.device, other._t, other.cfg, other._w = self.shape, self.device, self._t, self.cfg, self._w
        other.ctx = B.relaygr_create(self.cfg, self._w)
        other._ws = None
        other.page_bytes = self.page_bytes
        return other

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.shape.dtype == synth.DTYPE_BF16 else torch.float32

    def reserve(self, max_rows: int, max_users: int, max_pages: int):
        """Allocate and lend the workspace for calls up to these sizes."""
        n = B.relaygr_workspace_bytes(self.ctx, max_rows, max_users, max_pages)
        if self._ws is None or self._ws.numel() < n:
            self._ws_raw = torch.empty(n + 1024, dtype=torch.uint8, device=self.device)
            pad = (-self._ws_raw.data_ptr()) % 1024
            self._ws = self._ws_raw[pad:pad + n]
            B.relaygr_set_workspace(self.ctx, self._ws.data_ptr(), self._ws.numel())
        return n

    def gather(self, ids: torch.Tensor, stream=None) -> torch.Tensor:
        out = torch.empty((ids.numel(), self.shape.d_model), dtype=self.torch_dtype, device=self.device)
        B.relaygr_gather(self.ctx, ids.data_ptr(), ids.numel(), out.data_ptr(), _stream_ptr(stream))
        return out

    def rank_full(self, batch: "DeviceBatch", scores: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        if scores is None:
            scores = torch.empty(int(batch.cand_off[-1]), dtype=torch.float32, device=self.device)
        B.relaygr_rank_full(self.ctx, batch.n_users, batch.prefix_ids.data_ptr(), batch.prefix_off,
                            batch.short_ids.data_ptr(), batch.short_off, batch.cand_ids.data_ptr(), batch.cand_off,
                            scores.data_ptr(), _stream_ptr(stream))
        return scores

    def device_status(self, stream=None) -> int:
        """Synchronises the stream and returns the kernels' status word (0 = healthy)."""
        return B.relaygr_device_status(self.ctx, _stream_ptr(stream))

    def launch_count(self) -> int:
        return B.relaygr_launch_count(self.ctx)

    def close(self):
        if self.ctx:
            B.relaygr_destroy(self.ctx)
            self.ctx = None


class DeviceBatch:
    """A jagged batch with id arrays on the device and offsets on the host."""

    def __init__(self, batch: synth.Batch, device):
        to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device) if len(a) else torch.zeros(1, dtype=torch.int32, device=device)
        self.users = batch.users
        self.n_users = batch.n_users
        self.prefix_ids, self.prefix_off = to(batch.prefix_ids), batch.prefix_off
        self.short_ids, self.short_off = to(batch.short_ids), batch.short_off
        self.cand_ids, self.cand_off = to(batch.cand_ids), batch.cand_off


class KvPool:
    """A device slab (and optionally a pinned host slab) lent to the library's pool."""

    def __init__(self, model: Model, hbm_pages: int, host_pages: int = 0):
        self.model = model
        pb = model.page_bytes
        self._slab_raw = torch.zeros(hbm_pages * pb + 1024, dtype=torch.uint8, device=model.device)
        pad = (-self._slab_raw.data_ptr()) % 1024        # the caching allocator only promises 512 bytes
        self.slab = self._slab_raw[pad:pad + hbm_pages * pb]
        self.host = None
        if host_pages:
            self.host = torch.empty(host_pages * pb, dtype=torch.uint8, pin_memory=True)     # allocated pinned, not copied into a pinned buffer
        self.pool = B.relaygr_kv_pool_create(model.ctx, self.slab.data_ptr(), self.slab.numel(),
                                             self.host.data_ptr() if self.host is not None else None,
                                             self.host.numel() if self.host is not None else 0)

    def alloc(self, user, prefix_len, page_ids=None, ok=(B.OK,)):
        return B.relaygr_kv_alloc(self.pool, int(user), int(prefix_len), page_ids, ok)

    def free(self, user, ok=(B.OK,)):
        return B.relaygr_kv_free(self.pool, int(user), ok)

    def evict(self, user, spill, side_stream=None, ok=(B.OK,)):
        return B.relaygr_kv_evict(self.pool, int(user), spill, _stream_ptr(side_stream), ok)

    def reload(self, user, side_stream=None, ok=(B.OK,)):
        return B.relaygr_kv_reload_from_host(self.pool, int(user), _stream_ptr(side_stream), ok)

    def lookup(self, user):
        return B.relaygr_kv_lookup(self.pool, int(user))

    def pages(self, user):
        return B.relaygr_kv_pages(self.pool, int(user))

    def stats(self):
        return B.relaygr_kv_stats(self.pool)

    def preinfer(self, batch: DeviceBatch, stream=None, ok=(B.OK,), slot: Optional[Model] = None):
        return B.relaygr_preinfer((slot or self.model).ctx, self.pool, batch.users, batch.prefix_ids.data_ptr(), batch.prefix_off,
                                  _stream_ptr(stream), ok)

    def rank(self, batch: DeviceBatch, scores: Optional[torch.Tensor] = None, stream=None, per_user_status=None, ok=(B.OK,),
             slot: Optional[Model] = None):
        if scores is None:
            scores = torch.empty(max(1, int(batch.cand_off[-1])), dtype=torch.float32, device=self.model.device)
        code = B.relaygr_rank((slot or self.model).ctx, self.pool, batch.users, batch.short_ids.data_ptr(), batch.short_off,
                              batch.cand_ids.data_ptr(), batch.cand_off, scores.data_ptr(), _stream_ptr(stream),
                              per_user_status, ok)
        return scores[:int(batch.cand_off[-1])] if code == B.OK else None

    def read_kv(self, user, prefix_len):
        """Copy a user's K and V rows out of its pages: two arrays [L, P, d] (model dtype), for tests."""
        sh = self.model.shape
        pages = self.pages(user)
        dt = self.model.torch_dtype
        slab = self.slab.view(dt).view(-1, sh.n_layers, 2, sh.page_tokens, sh.d_model)
        sel = slab[torch.from_numpy(pages.astype(np.int64)).to(slab.device)]       # [n, L, 2, 64, d]
        sel = sel.permute(1, 2, 0, 3, 4).reshape(sh.n_layers, 2, -1, sh.d_model)[:, :, :prefix_len]
        return sel[:, 0].contiguous(), sel[:, 1].contiguous()

    def close(self):
        if self.pool:
            B.relaygr_kv_pool_destroy(self.pool)
            self.pool = None
