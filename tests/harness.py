"""Shared helpers for the GPU parity tests: upload seeded inputs, drive the C-ABI binding, convert
cache layouts for comparison with the oracle.  No method arithmetic lives here."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import Cache, Precc, layer_desc

ATOL, RTOL = 2e-2, 1e-2          # the stated bar for attention outputs: |gpu - ref| <= ATOL + RTOL*|ref|


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def weights_np(w):
    return {k: f64(v) for k, v in w.items()}


def base_rows(cache_t: torch.Tensor) -> np.ndarray:
    """[n_blocks, n_kv, PAGE, hd] -> token-major [n_blocks*PAGE, n_kv*hd] (float64)."""
    nb, n_kv, pg, hd = cache_t.shape
    return f64(cache_t.permute(0, 2, 1, 3).reshape(nb * pg, n_kv * hd))


def lr_rows(cache_t: torch.Tensor, agent: int) -> np.ndarray:
    """[N, n_blocks, PAGE, r] -> [n_blocks*PAGE, r] of one agent."""
    return f64(cache_t[agent].reshape(-1, cache_t.shape[-1]))


def assert_close(got: np.ndarray, ref: np.ndarray, what: str, atol=ATOL, rtol=RTOL, norm_tol=2e-2):
    """The stated elementwise bar plus a per-row normalised bound (so long contexts are not vacuous)."""
    mask = ~np.isnan(ref)
    assert mask.any(), f"{what}: nothing to compare"
    g, r = got[mask], ref[mask]
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    err = np.abs(g - r)
    bad = err > atol + rtol * np.abs(r)
    assert not bad.any(), f"{what}: {bad.sum()} elements off, max abs err {err.max():.3e}"
    if norm_tol is not None:
        rows_ref = np.where(mask, ref, 0.0).reshape(-1, ref.shape[-1])
        rows_got = np.where(mask, got, 0.0).reshape(-1, ref.shape[-1])
        nr = np.linalg.norm(rows_ref, axis=1)
        ne = np.linalg.norm(rows_got - rows_ref, axis=1)
        keep = nr > 0
        rel = (ne[keep] / nr[keep]).max()
        assert rel <= norm_tol, f"{what}: per-row relative L2 error {rel:.3e} > {norm_tol}"
    return float(err.max())


class Layer:
    """One layer's device state built from seeded inputs through the library's own calls."""

    def __init__(self, px: Precc, geo: I.Geometry, seed: int, n_blocks: int, tag: str = "L0", fill=None,
                 softmax_scale: float = 0.0, scale_k=None, scale_v=None):
        self.px, self.geo = px, geo
        self.desc = layer_desc(geo, softmax_scale, scale_k, scale_v)
        self.w = I.layer_weights(geo, seed, tag)
        self.w_np = weights_np(self.w)
        dev = {k: v.cuda() for k, v in self.w.items()}
        self.B_k = dev["B_k"] if geo.rank_k else None
        self.B_v = dev["B_v"] if geo.rank_v else None
        self.A_packed = px.pack_adapters(geo, dev["A_k"], dev["A_v"])
        self.W_packed = px.pack_base_weights(geo, dev["W_k"], dev["W_v"])
        self.cache = Cache(geo, n_blocks, fill=fill)

    def append(self, H: torch.Tensor, start_slot=0, slot_mapping=None, agent_mask=(1 << 64) - 1):
        Hd = H.cuda()
        self.px.rebase_project(self.desc, Hd, self.W_packed, self.cache, start_slot, slot_mapping)
        self.px.lr_precompute(self.desc, Hd, self.A_packed, self.cache, start_slot, slot_mapping, agent_mask)

    def decode(self, q: torch.Tensor, agent_id, ctx_len, max_ctx=None, block_table=None, first_block=None, ws=None):
        qd = q.cuda()
        aid = torch.as_tensor(agent_id, dtype=torch.int32).cuda()
        cl = torch.as_tensor(ctx_len, dtype=torch.int32).cuda()
        max_ctx = int(max(ctx_len)) if max_ctx is None else max_ctx
        if ws is None:
            ws = self.px.decode_workspace(self.desc, qd.shape[0], max_ctx)
        out = torch.full_like(qd, float("nan"))
        bt = None if block_table is None else block_table.cuda()
        fb = None if first_block is None else torch.as_tensor(first_block, dtype=torch.int32).cuda()
        self.px.lr_attend_decode(self.desc, qd, aid, cl, max_ctx, self.B_k, self.B_v, self.cache, out, ws, bt, fb)
        torch.cuda.synchronize()
        return out

    def prefill(self, q: torch.Tensor, agent: int, T: int, block_table=None, first_block=0):
        qd = q.cuda()
        out = torch.full_like(qd, float("nan"))
        bt = None if block_table is None else block_table.cuda()
        self.px.lr_attend_prefill(self.desc, qd, agent, T, self.B_k, self.B_v, self.cache, out, bt, first_block)
        torch.cuda.synchronize()
        return out

    def prefill_ws(self, q: torch.Tensor, agent: int, T: int, ws, block_table=None, first_block=0):
        qd = q.cuda()
        out = torch.full_like(qd, float("nan"))
        bt = None if block_table is None else block_table.cuda()
        self.px.lr_attend_prefill_ws(self.desc, qd, agent, T, self.B_k, self.B_v, self.cache, out, ws, bt, first_block)
        torch.cuda.synchronize()
        return out
