"""Thin ctypes binding over the C-ABI library ``libprecc.so`` (see ``include/precc.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels behind the ABI.
PyTorch is used for device memory and streams.  There is no fallback: if the library is
missing or a call fails, a ``PreccError`` is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from .inputs import PAGE, Geometry

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libprecc.so")

EXPORTS = [
    "precc_create", "precc_destroy", "precc_last_error", "precc_error_name", "precc_sm_count", "precc_set_trace_buffer",
    "precc_poll_status", "precc_pack_kmajor", "precc_lr_precompute", "precc_rebase_project", "precc_turn_project",
    "precc_decode_workspace_bytes", "precc_workspace_init", "precc_lr_attend_decode",
    "precc_lr_attend_decode_static", "precc_lr_attend_prefill",
    "precc_rebase_project_rope", "precc_turn_project_rope", "precc_lr_attend_decode_rope", "precc_lr_attend_prefill_rope",
    "precc_turn_project_rows", "precc_partial_record_floats", "precc_lr_attend_decode_partial", "precc_combine_partials",
    "precc_set_wait_limit", "precc_selftest_wait_timeout",
    "precc_prefill_rope_scratch_bytes", "precc_lr_attend_prefill_rope_scratch",
    "precc_prefill_ws_bytes", "precc_lr_attend_prefill_ws",
]


class PreccError(RuntimeError):
    pass


class LayerDesc(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("n_agents", C.c_int32), ("rank_k", C.c_int32), ("rank_v", C.c_int32),
                ("lora_scale_k", C.c_float), ("lora_scale_v", C.c_float), ("softmax_scale", C.c_float)]


class CacheDesc(C.Structure):
    _fields_ = [("k_base", C.c_void_p), ("v_base", C.c_void_p), ("lr_k", C.c_void_p), ("lr_v", C.c_void_p),
                ("n_blocks", C.c_int64)]


_lib = None


class RopeDesc(C.Structure):
    _fields_ = [("table", C.c_void_p), ("max_pos", C.c_int32), ("positions", C.c_void_p), ("start_pos", C.c_int64)]


def load_library() -> C.CDLL:
    """dlopen the library (built in-tree by ``build.py``); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise PreccError(f"{LIB_PATH} not found: build it with `python -m paper_2609_34054_b200.build` "
                         "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_size_t
    lib.precc_create.argtypes = [C.POINTER(vp), i32]
    lib.precc_destroy.argtypes = [vp]
    lib.precc_last_error.argtypes = [vp]
    lib.precc_last_error.restype = C.c_char_p
    lib.precc_error_name.argtypes = [i32]
    lib.precc_error_name.restype = C.c_char_p
    lib.precc_sm_count.argtypes = [vp]
    lib.precc_set_trace_buffer.argtypes = [vp, vp, sz]
    lib.precc_poll_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    lib.precc_set_wait_limit.argtypes = [vp, u64]
    lib.precc_selftest_wait_timeout.argtypes = [vp, vp, vp]
    lib.precc_pack_kmajor.argtypes = [vp, vp, i32, i32, vp, i32, i32, vp]
    lib.precc_lr_precompute.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, i64, u64, C.POINTER(CacheDesc), vp]
    lib.precc_rebase_project.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, i64, C.POINTER(CacheDesc), vp]
    lib.precc_turn_project.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, i64, u64, C.POINTER(CacheDesc), vp]
    lib.precc_decode_workspace_bytes.argtypes = [C.POINTER(LayerDesc), i32, i32, i32]
    lib.precc_decode_workspace_bytes.restype = sz
    lib.precc_workspace_init.argtypes = [vp, vp, sz, vp]
    lib.precc_lr_attend_decode.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, vp, i32, vp, i32, vp, vp,
                                           C.POINTER(CacheDesc), vp, vp, sz, vp]
    lib.precc_lr_attend_decode_static.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, vp, i32, vp, i32, vp, vp,
                                                  C.POINTER(CacheDesc), vp, vp]
    lib.precc_lr_attend_prefill.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, i32, i32, vp, i32, i32, vp, vp,
                                            C.POINTER(CacheDesc), vp, vp]
    lib.precc_prefill_ws_bytes.argtypes = [vp, C.POINTER(LayerDesc), i32]
    lib.precc_prefill_ws_bytes.restype = sz
    lib.precc_lr_attend_prefill_ws.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, i32, i32, vp, i32, i32, vp, vp,
                                               C.POINTER(CacheDesc), vp, vp, sz, vp]
    rp = C.POINTER(RopeDesc)
    lib.precc_rebase_project_rope.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, i64, rp, C.POINTER(CacheDesc), vp]
    lib.precc_turn_project_rope.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, i64, u64, rp, C.POINTER(CacheDesc), vp]
    lib.precc_lr_attend_decode_rope.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, vp, i32, vp, i32, vp, vp, rp,
                                                C.POINTER(CacheDesc), vp, vp, sz, vp]
    lib.precc_lr_attend_prefill_rope.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, i32, i32, vp, i32, i32, vp, vp, rp,
                                                 C.POINTER(CacheDesc), vp, vp]
    lib.precc_prefill_rope_scratch_bytes.argtypes = [C.POINTER(LayerDesc), i32, i32]
    lib.precc_prefill_rope_scratch_bytes.restype = sz
    lib.precc_lr_attend_prefill_rope_scratch.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, i32, i32, vp, i32, i32, vp, vp, rp,
                                                         C.POINTER(CacheDesc), vp, vp, sz, vp]
    lib.precc_turn_project_rows.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, vp, vp, C.POINTER(CacheDesc), vp]
    lib.precc_partial_record_floats.argtypes = [C.POINTER(LayerDesc)]
    lib.precc_partial_record_floats.restype = sz
    lib.precc_lr_attend_decode_partial.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, vp, vp, vp, i32, vp, i32, vp,
                                                   C.POINTER(CacheDesc), vp, vp, sz, vp]
    lib.precc_combine_partials.argtypes = [vp, C.POINTER(LayerDesc), vp, i32, i32, vp, vp, vp, vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is C.c_int:  # default restype: the int32 status code
            fn.restype = i32
    _lib = lib
    return lib


def layer_desc(geo: Geometry, softmax_scale: float = 0.0, scale_k: Optional[float] = None,
               scale_v: Optional[float] = None) -> LayerDesc:
    return LayerDesc(geo.d_model, geo.n_q, geo.n_kv, geo.hd, geo.n_agents, geo.rank_k, geo.rank_v,
                     geo.scale_k if scale_k is None else scale_k, geo.scale_v if scale_v is None else scale_v,
                     softmax_scale)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise PreccError("tensor must be a contiguous CUDA tensor")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Cache:
    """Caller-owned caches of one layer in the library's HBM layouts."""

    def __init__(self, geo: Geometry, n_blocks: int, device="cuda", fill: Optional[float] = None):
        mk = (lambda *s: torch.full(s, fill, dtype=torch.bfloat16, device=device)) if fill is not None else \
             (lambda *s: torch.empty(s, dtype=torch.bfloat16, device=device))
        self.geo, self.n_blocks = geo, n_blocks
        self.k_base = mk(n_blocks, geo.n_kv, PAGE, geo.hd)
        self.v_base = mk(n_blocks, geo.n_kv, PAGE, geo.hd)
        self.lr_k = mk(geo.n_agents, n_blocks, PAGE, geo.rank_k) if geo.rank_k else None
        self.lr_v = mk(geo.n_agents, n_blocks, PAGE, geo.rank_v) if geo.rank_v else None

    @classmethod
    def from_tensors(cls, geo: Geometry, k_base, v_base, lr_k, lr_v) -> "Cache":
        self = cls.__new__(cls)
        self.geo, self.n_blocks = geo, k_base.shape[0]
        self.k_base, self.v_base, self.lr_k, self.lr_v = k_base, v_base, lr_k, lr_v
        return self

    def desc(self) -> CacheDesc:
        return CacheDesc(_ptr(self.k_base), _ptr(self.v_base), _ptr(self.lr_k), _ptr(self.lr_v), self.n_blocks)

    def nbytes(self) -> int:
        return sum(t.numel() * 2 for t in (self.k_base, self.v_base, self.lr_k, self.lr_v) if t is not None)


class Precc:
    """One library context on one CUDA device."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise PreccError("no CUDA device: the precc path has no CPU fallback")
        self.device = device
        torch.cuda.set_device(device)
        h = C.c_void_p()
        rc = self.lib.precc_create(C.byref(h), device)
        if rc != 0:
            raise PreccError(f"precc_create failed: {self.lib.precc_error_name(rc).decode()}")
        self.h = h
        self.sm_count = self.lib.precc_sm_count(h)

    def close(self):
        if getattr(self, "h", None):
            self.lib.precc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, what: str):
        if rc != 0:
            raise PreccError(f"{what}: {self.lib.precc_error_name(rc).decode()}: "
                             f"{self.lib.precc_last_error(self.h).decode()}")

    # ------------------------------------------------------------------ plumbing
    def set_trace_buffer(self, buf: Optional[torch.Tensor]):
        """int64 CUDA tensor [n_blocks, 8] receiving per-block phase timestamps of decode, or None."""
        if buf is None:
            self._check(self.lib.precc_set_trace_buffer(self.h, None, 0), "precc_set_trace_buffer")
        else:
            self._check(self.lib.precc_set_trace_buffer(self.h, _ptr(buf), buf.shape[0]), "precc_set_trace_buffer")

    def poll_status(self) -> int:
        st = C.c_uint32(0)
        self.lib.precc_poll_status(self.h, _stream(), C.byref(st))
        return st.value

    def set_wait_limit(self, sm_cycles: int):
        """Limit of the kernels' bounded waits in SM clock cycles (0 = the default of about a second)."""
        self._check(self.lib.precc_set_wait_limit(self.h, sm_cycles), "precc_set_wait_limit")

    def selftest_wait_timeout(self, done_flag: torch.Tensor):
        """Launch the kernel that waits on a barrier nothing completes; done_flag: uint32/int32 CUDA tensor of one element."""
        self._check(self.lib.precc_selftest_wait_timeout(self.h, _ptr(done_flag), _stream()), "precc_selftest_wait_timeout")

    def pack_kmajor(self, src: torch.Tensor, dst: torch.Tensor, dst_row0: int):
        d, n = src.shape
        self._check(self.lib.precc_pack_kmajor(self.h, _ptr(src), d, n, _ptr(dst), dst.shape[0], dst_row0, _stream()),
                    "precc_pack_kmajor")

    def pack_adapters(self, geo: Geometry, A_k: torch.Tensor, A_v: torch.Tensor) -> torch.Tensor:
        """[N, d, r] per projection -> packed [N*(r_k+r_v), d], rows ordered [projection][agent][r]."""
        rows = geo.n_agents * (geo.rank_k + geo.rank_v)
        dst = torch.empty((max(rows, 1), geo.d_model), dtype=torch.bfloat16, device=A_v.device if A_v is not None else A_k.device)
        at = 0
        for A, r in ((A_k, geo.rank_k), (A_v, geo.rank_v)):
            for k in range(geo.n_agents if r else 0):
                self.pack_kmajor(A[k], dst, at)
                at += r
        return dst

    def pack_base_weights(self, geo: Geometry, W_k: torch.Tensor, W_v: torch.Tensor) -> torch.Tensor:
        """[d, n_kv*hd] per projection -> packed [2*n_kv*hd, d]."""
        dst = torch.empty((2 * geo.kv_width, geo.d_model), dtype=torch.bfloat16, device=W_k.device)
        self.pack_kmajor(W_k, dst, 0)
        self.pack_kmajor(W_v, dst, geo.kv_width)
        return dst

    def pack_turn_weights(self, geo: Geometry, W_k, W_v, A_k, A_v) -> torch.Tensor:
        """Packed W rows followed by packed A rows: the operand of ``turn_project``."""
        n_lr = geo.n_agents * (geo.rank_k + geo.rank_v)
        dst = torch.empty((2 * geo.kv_width + n_lr, geo.d_model), dtype=torch.bfloat16, device=W_k.device)
        self.pack_kmajor(W_k, dst, 0)
        self.pack_kmajor(W_v, dst, geo.kv_width)
        at = 2 * geo.kv_width
        for A, r in ((A_k, geo.rank_k), (A_v, geo.rank_v)):
            for k in range(geo.n_agents if r else 0):
                self.pack_kmajor(A[k], dst, at)
                at += r
        return dst

    def turn_project(self, desc: LayerDesc, H: torch.Tensor, WA_packed: torch.Tensor, cache: Cache,
                     start_slot: int = 0, slot_mapping: Optional[torch.Tensor] = None, agent_mask: int = (1 << 64) - 1):
        cd = cache.desc()
        self._check(self.lib.precc_turn_project(self.h, C.byref(desc), _ptr(H), H.shape[0], _ptr(WA_packed),
                                                _ptr(slot_mapping), start_slot, agent_mask & ((1 << 64) - 1),
                                                C.byref(cd), _stream()), "precc_turn_project")

    def turn_project_rows(self, desc: LayerDesc, H: torch.Tensor, WA_packed: torch.Tensor, cache: Cache,
                          slot_mapping: torch.Tensor, row_masks: torch.Tensor, lr_copy_slots: Optional[torch.Tensor] = None):
        """Fused projection with one agent mask per row (row_masks: int64 tensor holding the uint64 bit masks);
        lr_copy_slots: optional int32 [M], a second slot that also receives each row's LR rows (< 0: none)."""
        if row_masks.dtype != torch.int64:
            raise PreccError("row_masks must be int64 (bit patterns of uint64 masks)")
        if lr_copy_slots is not None and lr_copy_slots.dtype != torch.int32:
            raise PreccError("lr_copy_slots must be int32")
        cd = cache.desc()
        self._check(self.lib.precc_turn_project_rows(self.h, C.byref(desc), _ptr(H), H.shape[0], _ptr(WA_packed),
                                                     _ptr(slot_mapping), _ptr(row_masks), _ptr(lr_copy_slots),
                                                     C.byref(cd), _stream()),
                    "precc_turn_project_rows")

    # ------------------------------------------------------------------ the four entry points
    def lr_precompute(self, desc: LayerDesc, H: torch.Tensor, A_packed: torch.Tensor, cache: Cache,
                      start_slot: int = 0, slot_mapping: Optional[torch.Tensor] = None, agent_mask: int = (1 << 64) - 1):
        cd = cache.desc()
        self._check(self.lib.precc_lr_precompute(self.h, C.byref(desc), _ptr(H), H.shape[0], _ptr(A_packed),
                                                 _ptr(slot_mapping), start_slot, agent_mask & ((1 << 64) - 1),
                                                 C.byref(cd), _stream()), "precc_lr_precompute")

    def rebase_project(self, desc: LayerDesc, H: torch.Tensor, W_packed: torch.Tensor, cache: Cache,
                       start_slot: int = 0, slot_mapping: Optional[torch.Tensor] = None):
        cd = cache.desc()
        self._check(self.lib.precc_rebase_project(self.h, C.byref(desc), _ptr(H), H.shape[0], _ptr(W_packed),
                                                  _ptr(slot_mapping), start_slot, C.byref(cd), _stream()),
                    "precc_rebase_project")

    # ------------------------------------------------------------------ rotary-key variant
    @staticmethod
    def _rope(table: torch.Tensor, positions: Optional[torch.Tensor] = None, start_pos: int = 0) -> RopeDesc:
        if table.dtype != torch.float32 or table.dim() != 3 or table.shape[2] != 2:
            raise PreccError("rope table must be fp32 [max_pos][hd/2][2]")
        return RopeDesc(_ptr(table), table.shape[0], _ptr(positions), start_pos)

    def rebase_project_rope(self, desc: LayerDesc, H: torch.Tensor, W_packed: torch.Tensor, cache: Cache, rope: torch.Tensor,
                            start_slot: int = 0, slot_mapping: Optional[torch.Tensor] = None, start_pos: int = 0,
                            positions: Optional[torch.Tensor] = None):
        cd, rd = cache.desc(), self._rope(rope, positions, start_pos)
        self._check(self.lib.precc_rebase_project_rope(self.h, C.byref(desc), _ptr(H), H.shape[0], _ptr(W_packed),
                                                       _ptr(slot_mapping), start_slot, C.byref(rd), C.byref(cd), _stream()),
                    "precc_rebase_project_rope")

    def turn_project_rope(self, desc: LayerDesc, H: torch.Tensor, WA_packed: torch.Tensor, cache: Cache, rope: torch.Tensor,
                          start_slot: int = 0, slot_mapping: Optional[torch.Tensor] = None, agent_mask: int = (1 << 64) - 1,
                          start_pos: int = 0, positions: Optional[torch.Tensor] = None):
        cd, rd = cache.desc(), self._rope(rope, positions, start_pos)
        self._check(self.lib.precc_turn_project_rope(self.h, C.byref(desc), _ptr(H), H.shape[0], _ptr(WA_packed),
                                                     _ptr(slot_mapping), start_slot, agent_mask & ((1 << 64) - 1),
                                                     C.byref(rd), C.byref(cd), _stream()), "precc_turn_project_rope")

    def lr_attend_decode_rope(self, desc: LayerDesc, q: torch.Tensor, agent_id: torch.Tensor, ctx_len: torch.Tensor,
                              max_ctx: int, B_k, B_v, rope: torch.Tensor, cache: Cache, out: torch.Tensor,
                              workspace: torch.Tensor, block_table: Optional[torch.Tensor] = None,
                              first_block: Optional[torch.Tensor] = None):
        cd, rd = cache.desc(), self._rope(rope)
        stride = block_table.shape[1] if block_table is not None else 0
        self._check(self.lib.precc_lr_attend_decode_rope(
            self.h, C.byref(desc), _ptr(q), q.shape[0], _ptr(agent_id), _ptr(ctx_len), _ptr(block_table), stride,
            _ptr(first_block), max_ctx, _ptr(B_k), _ptr(B_v), C.byref(rd), C.byref(cd), _ptr(out), _ptr(workspace),
            workspace.numel(), _stream()), "precc_lr_attend_decode_rope")

    def lr_attend_prefill_rope(self, desc: LayerDesc, q: torch.Tensor, agent: int, ctx_len: int, B_k, B_v, rope: torch.Tensor,
                               cache: Cache, out: torch.Tensor, block_table: Optional[torch.Tensor] = None, first_block: int = 0):
        cd, rd = cache.desc(), self._rope(rope)
        stride = block_table.numel() if block_table is not None else 0
        self._check(self.lib.precc_lr_attend_prefill_rope(
            self.h, C.byref(desc), _ptr(q), q.shape[0], agent, ctx_len, _ptr(block_table), stride, first_block,
            _ptr(B_k), _ptr(B_v), C.byref(rd), C.byref(cd), _ptr(out), _stream()), "precc_lr_attend_prefill_rope")

    def prefill_rope_scratch_bytes(self, desc: LayerDesc, ctx_len: int, S: int) -> int:
        return int(self.lib.precc_prefill_rope_scratch_bytes(C.byref(desc), ctx_len, S))

    def lr_attend_prefill_rope_scratch(self, desc: LayerDesc, q: torch.Tensor, agent: int, ctx_len: int, B_k, B_v, rope: torch.Tensor,
                                       cache: Cache, out: torch.Tensor, key_scratch: torch.Tensor,
                                       block_table: Optional[torch.Tensor] = None, first_block: int = 0):
        """Rotary prefill through a caller-provided scratch for the sequence's adapted keys (uint8 or bf16 tensor)."""
        cd, rd = cache.desc(), self._rope(rope)
        stride = block_table.numel() if block_table is not None else 0
        self._check(self.lib.precc_lr_attend_prefill_rope_scratch(
            self.h, C.byref(desc), _ptr(q), q.shape[0], agent, ctx_len, _ptr(block_table), stride, first_block,
            _ptr(B_k), _ptr(B_v), C.byref(rd), C.byref(cd), _ptr(out), _ptr(key_scratch),
            key_scratch.numel() * key_scratch.element_size(), _stream()), "precc_lr_attend_prefill_rope_scratch")

    # ------------------------------------------------------------------ context-sharded decode
    def partial_record_floats(self, desc: LayerDesc) -> int:
        return int(self.lib.precc_partial_record_floats(C.byref(desc)))

    def lr_attend_decode_partial(self, desc: LayerDesc, q: torch.Tensor, agent_id: torch.Tensor, ctx_len: torch.Tensor,
                                 max_ctx: int, B_k, cache: Cache, records: torch.Tensor, workspace: torch.Tensor,
                                 block_table: Optional[torch.Tensor] = None, first_block: Optional[torch.Tensor] = None):
        """This shard's split-KV record per (request, kv head) over its local tokens: records fp32 [B][n_kv][R]."""
        if records.dtype != torch.float32:
            raise PreccError("records must be fp32")
        cd = cache.desc()
        stride = block_table.shape[1] if block_table is not None else 0
        self._check(self.lib.precc_lr_attend_decode_partial(
            self.h, C.byref(desc), _ptr(q), q.shape[0], _ptr(agent_id), _ptr(ctx_len), _ptr(block_table), stride,
            _ptr(first_block), max_ctx, _ptr(B_k), C.byref(cd), _ptr(records), _ptr(workspace), workspace.numel(), _stream()),
            "precc_lr_attend_decode_partial")

    def combine_partials(self, desc: LayerDesc, records: torch.Tensor, agent_id: torch.Tensor, B_v, out: torch.Tensor):
        """records fp32 [n_shards][B][n_kv][R] (as an all-gather leaves them) -> out [B][n_q][hd]."""
        self._check(self.lib.precc_combine_partials(self.h, C.byref(desc), _ptr(records), records.shape[0], out.shape[0],
                                                    _ptr(agent_id), _ptr(B_v), _ptr(out), _stream()), "precc_combine_partials")

    def decode_workspace(self, desc: LayerDesc, max_batch: int, max_ctx: int) -> torch.Tensor:
        n = self.lib.precc_decode_workspace_bytes(C.byref(desc), max_batch, max_ctx, self.sm_count)
        if n == 0:
            raise PreccError("precc_decode_workspace_bytes: unsupported shape")
        ws = torch.empty(n, dtype=torch.uint8, device=f"cuda:{self.device}")
        self._check(self.lib.precc_workspace_init(self.h, _ptr(ws), n, _stream()), "precc_workspace_init")
        return ws

    def lr_attend_decode(self, desc: LayerDesc, q: torch.Tensor, agent_id: torch.Tensor, ctx_len: torch.Tensor,
                         max_ctx: int, B_k, B_v, cache: Cache, out: torch.Tensor, workspace: torch.Tensor,
                         block_table: Optional[torch.Tensor] = None, first_block: Optional[torch.Tensor] = None):
        cd = cache.desc()
        stride = block_table.shape[1] if block_table is not None else 0
        self._check(self.lib.precc_lr_attend_decode(
            self.h, C.byref(desc), _ptr(q), q.shape[0], _ptr(agent_id), _ptr(ctx_len), _ptr(block_table), stride,
            _ptr(first_block), max_ctx, _ptr(B_k), _ptr(B_v), C.byref(cd), _ptr(out), _ptr(workspace),
            workspace.numel(), _stream()), "precc_lr_attend_decode")

    def lr_attend_decode_static(self, desc: LayerDesc, q: torch.Tensor, agent_id: torch.Tensor, ctx_len: torch.Tensor,
                                max_ctx: int, B_k, B_v, cache: Cache, out: torch.Tensor,
                                block_table: Optional[torch.Tensor] = None, first_block: Optional[torch.Tensor] = None):
        """Decode attention for callers that may not allocate device memory (an engine whose KV pool owns
        all of HBM, code inside a stream capture, a loop that cannot afford cudaMalloc's synchronisation):
        the split-merge scratch is an array built into the library, so no workspace is passed.  All calls
        on a device share that array; do not let two of them overlap on the GPU."""
        cd = cache.desc()
        stride = block_table.shape[1] if block_table is not None else 0
        self._check(self.lib.precc_lr_attend_decode_static(
            self.h, C.byref(desc), _ptr(q), q.shape[0], _ptr(agent_id), _ptr(ctx_len), _ptr(block_table), stride,
            _ptr(first_block), max_ctx, _ptr(B_k), _ptr(B_v), C.byref(cd), _ptr(out), _stream()),
            "precc_lr_attend_decode_static")

    def lr_attend_prefill(self, desc: LayerDesc, q: torch.Tensor, agent: int, ctx_len: int, B_k, B_v, cache: Cache,
                          out: torch.Tensor, block_table: Optional[torch.Tensor] = None, first_block: int = 0):
        cd = cache.desc()
        stride = block_table.numel() if block_table is not None else 0
        self._check(self.lib.precc_lr_attend_prefill(
            self.h, C.byref(desc), _ptr(q), q.shape[0], agent, ctx_len, _ptr(block_table), stride, first_block,
            _ptr(B_k), _ptr(B_v), C.byref(cd), _ptr(out), _stream()), "precc_lr_attend_prefill")

    def prefill_ws_bytes(self, desc: LayerDesc, S: int) -> int:
        return int(self.lib.precc_prefill_ws_bytes(self.h, C.byref(desc), S))

    def lr_attend_prefill_ws(self, desc: LayerDesc, q: torch.Tensor, agent: int, ctx_len: int, B_k, B_v, cache: Cache,
                             out: torch.Tensor, workspace: Optional[torch.Tensor], block_table: Optional[torch.Tensor] = None,
                             first_block: int = 0):
        """Prefill with a caller-provided workspace (uint8 tensor of prefill_ws_bytes, or None): helper blocks on idle SMs."""
        cd = cache.desc()
        stride = block_table.numel() if block_table is not None else 0
        nbytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
        self._check(self.lib.precc_lr_attend_prefill_ws(
            self.h, C.byref(desc), _ptr(q), q.shape[0], agent, ctx_len, _ptr(block_table), stride, first_block,
            _ptr(B_k), _ptr(B_v), C.byref(cd), _ptr(out), _ptr(workspace), nbytes, _stream()), "precc_lr_attend_prefill_ws")
