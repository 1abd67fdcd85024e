"""ctypes binding of libkvmem_b200.so: argument marshalling only.

Every step of the recall path (index build, scoring, selection, view assembly, attention)
runs in the library's CUDA kernels; PyTorch supplies device memory and streams.  There is no
CPU fallback: if the shared library is missing or a call fails, an exception is raised.
Names mirror the C ABI declared in ``include/kvmem.h``.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import torch

from . import _build

OK = 0
E_INVALID, E_CAPACITY, E_STATE, E_CUDA, E_TIMEOUT, E_UNSUPPORTED, E_DEVICE_RANGE = -1, -2, -3, -4, -5, -6, -7


class KvmemError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"kvmem status {status}: {message}")
        self.status = status


class PoolConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "n_q_heads", "n_kv_heads", "head_dim", "block_tokens",
                                          "max_sessions", "max_blocks", "max_blocks_per_session", "device",
                                          "rope_max_positions")] + [("rope_theta", C.c_float),
                                                                   ("rope_in_block_keys", C.c_int32), ("fp8_pages", C.c_int32),
                                                                   ("fp8_k_scale", C.c_float), ("fp8_v_scale", C.c_float)]


class SelectParams(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("budget_blocks", "max_view_tokens", "mandatory_tokens",
                                          "n_sink_blocks", "n_recent_blocks")]


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Load (building first if sources are newer) the CUDA library.  Raises if that is impossible."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = _build.LIB_PATH
        if not os.path.exists(path) or os.environ.get("KVMEM_REBUILD"):
            _build.build()
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} is missing: build it with paper_2609_04852_b200._build.build()")
    L = C.CDLL(path)
    vp, i32, sz, f32 = C.c_void_p, C.c_int32, C.c_size_t, C.c_float
    cfgp, prmp = C.POINTER(PoolConfig), C.POINTER(SelectParams)
    sig = {
        "kvmem_pool_bytes": (sz, [cfgp]),
        "kvmem_budget_blocks": (i32, [prmp, i32, i32]),
        "kvmem_select_workspace_bytes": (sz, [cfgp, i32, i32]),
        "kvmem_attend_workspace_bytes": (sz, [cfgp, i32, i32]),
        "kvmem_last_error": (C.c_char_p, []),
        "kvmem_pool_create": (C.c_int, [cfgp, vp, sz, C.POINTER(vp)]),
        "kvmem_pool_destroy": (C.c_int, [vp]),
        "kvmem_session_reset": (C.c_int, [vp, i32, vp]),
        "kvmem_session_blocks": (i32, [vp, i32]),
        "kvmem_append_blocks": (C.c_int, [vp, i32, vp, vp, i32, C.POINTER(i32), vp]),
        "kvmem_score": (C.c_int, [vp, i32, i32, vp, i32, vp, f32, vp, sz, vp]),
        "kvmem_topk": (C.c_int, [vp, i32, i32, vp, i32, prmp, vp, i32, vp, vp]),
        "kvmem_score_host_workspace_bytes": (sz, [vp, i32, i32, i32]),
        "kvmem_score_host_staging_bytes": (sz, [vp, i32]),
        "kvmem_score_host_index": (C.c_int, [vp, vp, i32, i32, vp, i32, i32, vp, vp, sz, vp, sz, vp]),
        "kvmem_select": (C.c_int, [vp, i32, i32, vp, i32, prmp, vp, i32, vp, vp, vp, sz, vp]),
        "kvmem_materialize": (C.c_int, [vp, i32, i32, vp, i32, vp, vp, vp, i32, vp]),
        "kvmem_materialize_delta": (C.c_int, [vp, i32, i32, vp, vp, vp, i32, vp, vp, vp, i32, vp, vp]),
        "kvmem_view_attend": (C.c_int, [vp, i32, vp, i32, vp, vp, i32, vp, f32, vp, vp, vp, sz, vp]),
        "kvmem_get_index": (C.c_int, [vp, i32, C.POINTER(vp), C.POINTER(i32)]),
        "kvmem_get_block_table": (C.c_int, [vp, i32, C.POINTER(vp), C.POINTER(i32)]),
        "kvmem_device_status": (C.c_int, [vp, C.POINTER(i32), vp]),
        "kvmem_set_option": (C.c_int, [C.c_char_p, i32]),
        "kvmem_materialize_attend": (C.c_int, [vp, i32, i32, vp, i32, vp, i32, vp, vp, vp, i32, f32, vp, vp, vp, sz, vp]),
        "kvmem_append_blocks_rope": (C.c_int, [vp, i32, vp, vp, i32, C.POINTER(i32), C.POINTER(i32), vp]),
        "kvmem_rope_rotate": (C.c_int, [vp, vp, vp, C.c_int64, i32, vp, i32, vp]),
        "kvmem_materialize_rope": (C.c_int, [vp, i32, i32, vp, i32, vp, vp, vp, i32, i32, vp]),
        "kvmem_working_set_delta": (C.c_int, [vp, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp]),
        "kvmem_view_cache_bytes": (sz, [vp, i32]),
        "kvmem_view_cache_layout": (C.c_int, [vp, i32, C.POINTER(sz)]),
        "kvmem_view_cache_reset": (C.c_int, [vp, vp, sz, i32, vp]),
        "kvmem_view_cache_update": (C.c_int, [vp, i32, vp, vp, vp, sz, i32, i32, i32, vp, vp]),
        "kvmem_view_cache_attend": (C.c_int, [vp, vp, i32, vp, sz, i32, f32, vp, vp, vp, sz, vp]),
        "kvmem_paged_attend": (C.c_int, [vp, i32, i32, vp, i32, vp, i32, vp, f32, vp, vp, vp, sz, vp]),
        "kvmem_paged_attend_rope": (C.c_int, [vp, i32, i32, vp, i32, vp, i32, vp, i32, f32, vp, vp, vp, sz, vp]),
        "kvmem_materialize_attend_rope": (C.c_int, [vp, i32, i32, vp, i32, vp, i32, vp, vp, vp, i32, i32, f32, vp, vp, vp, sz, vp]),
        "kvmem_materialize_fp8": (C.c_int, [vp, i32, i32, vp, i32, vp, vp, vp, i32, f32, f32, vp]),
        "kvmem_materialize_fp8_rope": (C.c_int, [vp, i32, i32, vp, i32, vp, vp, vp, i32, i32, f32, f32, vp]),
        "kvmem_paged_attend_fp8": (C.c_int, [vp, i32, i32, vp, i32, vp, i32, vp, f32, vp, vp, vp, sz, vp]),
        "kvmem_paged_attend_fp8_rope": (C.c_int, [vp, i32, i32, vp, i32, vp, i32, vp, i32, f32, vp, vp, vp, sz, vp]),
        "kvmem_materialize_attend_fp8": (C.c_int, [vp, i32, i32, vp, i32, vp, i32, vp, vp, vp, i32, f32, vp, vp, vp, sz, vp]),
        "kvmem_view_attend_fp8": (C.c_int, [vp, i32, vp, i32, vp, vp, i32, vp, f32, f32, f32, vp, vp, vp, sz, vp]),
        "kvmem_view_attend_static": (C.c_int, [vp, i32, vp, i32, vp, vp, i32, vp, f32, vp, vp, vp]),
        "kvmem_selftest_wait_timeout": (C.c_int, [vp, C.c_uint32, vp, vp]),
        "kvmem_step_staging_bytes": (sz, [cfgp, i32, i32]),
        "kvmem_recall_step_host": (C.c_int, [vp, i32, i32, vp, i32, prmp, vp, i32, vp, vp, vp, i32, f32, vp, vp,
                                             vp, sz, vp, sz, vp, sz, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    if path == _build.LIB_PATH:
        _lib = L
    return L


EXPORTED = ("kvmem_pool_bytes", "kvmem_budget_blocks", "kvmem_select_workspace_bytes",
            "kvmem_attend_workspace_bytes", "kvmem_last_error", "kvmem_pool_create", "kvmem_pool_destroy",
            "kvmem_session_reset", "kvmem_session_blocks", "kvmem_append_blocks", "kvmem_select",
            "kvmem_materialize", "kvmem_view_attend", "kvmem_get_index", "kvmem_get_block_table",
            "kvmem_device_status", "kvmem_set_option", "kvmem_step_staging_bytes", "kvmem_recall_step_host",
            "kvmem_view_attend_static", "kvmem_materialize_attend",
            "kvmem_paged_attend", "kvmem_append_blocks_rope", "kvmem_rope_rotate", "kvmem_materialize_rope",
            "kvmem_working_set_delta", "kvmem_score", "kvmem_view_cache_bytes", "kvmem_view_cache_layout",
            "kvmem_view_cache_reset", "kvmem_view_cache_update", "kvmem_view_cache_attend", "kvmem_paged_attend_rope", "kvmem_topk", "kvmem_score_host_workspace_bytes",
            "kvmem_score_host_staging_bytes", "kvmem_score_host_index", "kvmem_materialize_fp8", "kvmem_view_attend_fp8",
            "kvmem_materialize_attend_rope", "kvmem_paged_attend_fp8", "kvmem_materialize_attend_fp8",
            "kvmem_paged_attend_fp8_rope", "kvmem_selftest_wait_timeout", "kvmem_materialize_delta",
            "kvmem_materialize_fp8_rope")


def _check(status: int) -> None:
    if status != OK:
        raise KvmemError(status, load_library().kvmem_last_error().decode())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype=None) -> int:
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


class HostStep:
    """kvmem_recall_step_host with its arguments checked and marshalled once; see Pool.host_step."""

    def __init__(self, pool, q_shape, params, sel_ids, n_sel, view, out_host, lse_host, scale, session_first):
        ns, M = q_shape[0], q_shape[1]
        for t, dt in ((out_host, torch.float32), (lse_host, torch.float32)):
            if t.is_cuda or not t.is_contiguous() or t.dtype != dt:
                raise ValueError("expected contiguous CPU tensors (fp32 outputs)")
        need = pool.lib.kvmem_step_staging_bytes(C.byref(pool.cfg), ns, M)
        if pool._staging is None or pool._staging.numel() < need:
            pool._staging = torch.empty(need, dtype=torch.uint8, device=pool.device)
        sws, aws = pool.select_workspace(ns, M), pool.attend_workspace(ns, M)
        self._keep = (pool, params, sel_ids, n_sel, view, out_host, lse_host, pool._staging, sws, aws)   # the buffers stay alive
        self._q_shape, self._fn = q_shape, pool.lib.kvmem_recall_step_host
        self._head = (pool.handle, session_first, ns)
        self._tail = (M, C.byref(params), _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                      _dev(view.k, torch.bfloat16), _dev(view.v, torch.bfloat16), view.cap_tokens, scale, out_host.data_ptr(),
                      lse_host.data_ptr(), pool._staging.data_ptr(), pool._staging.numel(), sws.data_ptr(), sws.numel(),
                      aws.data_ptr(), aws.numel())

    def __call__(self, q_host: torch.Tensor) -> None:
        if q_host.is_cuda or q_host.dtype != torch.bfloat16 or tuple(q_host.shape) != self._q_shape or not q_host.is_contiguous():
            raise ValueError("expected a contiguous CPU bf16 query of the planned shape")
        _check(self._fn(*self._head, q_host.data_ptr(), *self._tail, _stream()))


def budget_blocks(params: SelectParams, block_tokens: int, n_blocks: int) -> int:
    return int(load_library().kvmem_budget_blocks(C.byref(params), block_tokens, n_blocks))


def set_option(name: str, value: int) -> None:
    _check(load_library().kvmem_set_option(name.encode(), value))


@dataclass
class View:
    """Execution view buffers: bf16 [n_sessions][L][G][cap_tokens][d] each."""
    k: torch.Tensor
    v: torch.Tensor
    cap_tokens: int


class Pool:
    """A paged KV repository with its Mean-K index, living in one torch uint8 tensor."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, block_tokens: int,
                 max_sessions: int, max_blocks: int, max_blocks_per_session: int, device: int = 0,
                 rope_max_positions: int = 0, rope_theta: float = 0.0, rope_in_block_keys: bool = False,
                 fp8_pages: bool = False, fp8_k_scale: float = 1.0, fp8_v_scale: float = 1.0):
        self.lib = load_library()
        self.cfg = PoolConfig(n_layers, n_q_heads, n_kv_heads, head_dim, block_tokens, max_sessions, max_blocks,
                              max_blocks_per_session, device, rope_max_positions, rope_theta, int(rope_in_block_keys),
                              int(fp8_pages), fp8_k_scale, fp8_v_scale)
        nbytes = self.lib.kvmem_pool_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise KvmemError(E_INVALID, self.lib.kvmem_last_error().decode())
        self.device = torch.device("cuda", device)
        self.storage = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.handle = C.c_void_p()
        _check(self.lib.kvmem_pool_create(C.byref(self.cfg), self.storage.data_ptr(), nbytes, C.byref(self.handle)))
        self._select_ws: Optional[torch.Tensor] = None
        self._attend_ws: Optional[torch.Tensor] = None
        self._host_ws: Optional[torch.Tensor] = None
        self._host_staging: Optional[torch.Tensor] = None
        self._staging: Optional[torch.Tensor] = None

    # ---- lifetime
    def close(self) -> None:
        if self.handle:
            self.lib.kvmem_pool_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- repository
    def session_reset(self, session: int) -> None:
        _check(self.lib.kvmem_session_reset(self.handle, session, _stream()))

    def session_blocks(self, session: int) -> int:
        n = self.lib.kvmem_session_blocks(self.handle, session)
        if n < 0:
            _check(n)
        return n

    def append_blocks(self, session: int, k: torch.Tensor, v: torch.Tensor,
                      phys_ids: Optional[Sequence[int]] = None) -> None:
        c = self.cfg
        per_block = c.block_tokens * c.n_layers * c.n_kv_heads * c.head_dim
        if k.numel() % per_block or k.shape != v.shape:
            raise KvmemError(E_INVALID, "k and v must hold whole blocks of identical shape")
        n = k.numel() // per_block
        ids = None
        if phys_ids is not None:
            if len(phys_ids) != n:
                raise KvmemError(E_INVALID, "one page id per block")
            ids = (C.c_int32 * n)(*[int(x) for x in phys_ids])
        _check(self.lib.kvmem_append_blocks(self.handle, session, _dev(k, torch.bfloat16), _dev(v, torch.bfloat16),
                                            n, ids, _stream()))

    # ---- working-set delta
    def working_set_delta(self, prev_ids: torch.Tensor, n_prev: torch.Tensor, next_ids: torch.Tensor,
                          n_next: torch.Tensor):
        """Retained / incoming / outgoing blocks between two selections (ascending int32 id lists of equal stride).
        Returns (retained [ns][stride][3], incoming [ns][stride][2], outgoing [ns][stride], counts [ns][3])."""
        ns, stride = prev_ids.shape
        if next_ids.shape != prev_ids.shape:
            raise ValueError("both id lists must have the same [n_sessions][stride] shape")
        dev = prev_ids.device
        ret = torch.zeros(ns, stride, 3, dtype=torch.int32, device=dev)
        inc = torch.zeros(ns, stride, 2, dtype=torch.int32, device=dev)
        out = torch.zeros(ns, stride, dtype=torch.int32, device=dev)
        cnt = torch.zeros(ns, 3, dtype=torch.int32, device=dev)
        _check(self.lib.kvmem_working_set_delta(self.handle, ns, _dev(prev_ids, torch.int32), _dev(n_prev, torch.int32),
                                                _dev(next_ids, torch.int32), _dev(n_next, torch.int32), stride,
                                                ret.data_ptr(), inc.data_ptr(), out.data_ptr(), cnt.data_ptr(), _stream()))
        return ret, inc, out, cnt

    # ---- execution cache: working-set reuse with bounded delta re-RoPE
    def new_view_cache(self, cap_blocks: int, max_delta_ropes: int, first_position: int = 0) -> "ViewCache":
        return ViewCache(self, cap_blocks, max_delta_ropes, first_position)

    # ---- position-consistent keys
    def append_blocks_rope(self, session: int, k_roped: torch.Tensor, v: torch.Tensor, block_pos0: Sequence[int],
                           phys_ids: Optional[Sequence[int]] = None) -> None:
        """append_blocks for keys that carry RoPE: token t of block i was encoded at block_pos0[i] + t."""
        c = self.cfg
        per_block = c.block_tokens * c.n_layers * c.n_kv_heads * c.head_dim
        if k_roped.numel() % per_block or k_roped.shape != v.shape:
            raise KvmemError(E_INVALID, "k and v must hold whole blocks of identical shape")
        n = k_roped.numel() // per_block
        if len(block_pos0) != n or (phys_ids is not None and len(phys_ids) != n):
            raise KvmemError(E_INVALID, "one position (and page id) per block")
        ids = None if phys_ids is None else (C.c_int32 * n)(*[int(x) for x in phys_ids])
        pos = (C.c_int32 * n)(*[int(x) for x in block_pos0])
        _check(self.lib.kvmem_append_blocks_rope(self.handle, session, _dev(k_roped, torch.bfloat16),
                                                 _dev(v, torch.bfloat16), n, ids, pos, _stream()))

    def rope_rotate(self, x: torch.Tensor, positions: torch.Tensor, out: Optional[torch.Tensor] = None,
                    inverse: bool = False) -> torch.Tensor:
        """x bf16 [n_rows][n_vec][head_dim], positions int32 [n_rows] -> rotated copy (inverse: encoding removed)."""
        if out is None:
            out = torch.empty_like(x)
        n_rows, n_vec = x.shape[0], x.numel() // (x.shape[0] * self.cfg.head_dim)
        _check(self.lib.kvmem_rope_rotate(self.handle, _dev(x, torch.bfloat16), _dev(out, torch.bfloat16), n_rows, n_vec,
                                          _dev(positions, torch.int32), int(inverse), _stream()))
        return out

    def materialize_rope(self, sel_ids: torch.Tensor, n_sel: torch.Tensor, view: View, first_position: int = 0,
                         session_first: int = 0) -> None:
        """materialize with keys rotated to their compact positions first_position + j*B + t; values copied."""
        ns = n_sel.shape[0]
        _check(self.lib.kvmem_materialize_rope(self.handle, session_first, ns, _dev(sel_ids, torch.int32),
                                               sel_ids.shape[-1], _dev(n_sel, torch.int32), _dev(view.k, torch.bfloat16),
                                               _dev(view.v, torch.bfloat16), view.cap_tokens, first_position, _stream()))

    # ---- the recall step
    def select_workspace(self, n_sessions: int, n_q_tokens: int) -> torch.Tensor:
        need = self.lib.kvmem_select_workspace_bytes(C.byref(self.cfg), n_sessions, n_q_tokens)
        if need == 0:
            raise KvmemError(E_INVALID, self.lib.kvmem_last_error().decode())
        if self._select_ws is None or self._select_ws.numel() < need:
            self._select_ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._select_ws

    def attend_workspace(self, n_sessions: int, n_q_tokens: int) -> torch.Tensor:
        need = self.lib.kvmem_attend_workspace_bytes(C.byref(self.cfg), n_sessions, n_q_tokens)
        if need == 0:
            raise KvmemError(E_INVALID, self.lib.kvmem_last_error().decode())
        if self._attend_ws is None or self._attend_ws.numel() < need:
            self._attend_ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._attend_ws

    def score(self, q: torch.Tensor, scores: torch.Tensor, session_first: int = 0, score_scale: float = 1.0) -> None:
        """Block relevance only: q bf16 [n_sessions][M][L][H][d] -> scores fp32 [n_sessions][max_blocks_per_session]
        (times score_scale: a rank holding 1/N of a session's heads passes 1/N, so that the ranks' outputs sum to R)."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.select_workspace(ns, M)
        _check(self.lib.kvmem_score(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                    _dev(scores, torch.float32), score_scale, ws.data_ptr(), ws.numel(), _stream()))

    def topk(self, scores: torch.Tensor, params: SelectParams, sel_ids: torch.Tensor, n_sel: torch.Tensor,
             session_first: int = 0) -> None:
        """Selection from scores the caller already has: scores fp32 [n_sessions][stride] on the device."""
        ns = scores.shape[0]
        _check(self.lib.kvmem_topk(self.handle, session_first, ns, _dev(scores, torch.float32), scores.shape[1],
                                   C.byref(params), _dev(sel_ids, torch.int32), sel_ids.shape[-1],
                                   _dev(n_sel, torch.int32), _stream()))

    def score_host_index(self, index_host: torch.Tensor, n_blocks: int, q: torch.Tensor, scores: torch.Tensor,
                         tile_blocks: int = 4096) -> None:
        """Block relevance against an index in HOST memory (bf16 [L][G][stride][d], ideally pinned), streamed to the
        GPU in tiles of tile_blocks blocks; q bf16 [M][L][H][d] and scores fp32 [n_blocks] on the device."""
        if index_host.is_cuda or index_host.dtype != torch.bfloat16 or not index_host.is_contiguous():
            raise ValueError("index_host must be a contiguous CPU bf16 tensor")
        M = q.shape[0]
        need_ws = self.lib.kvmem_score_host_workspace_bytes(self.handle, n_blocks, M, tile_blocks)
        need_st = self.lib.kvmem_score_host_staging_bytes(self.handle, tile_blocks)
        if need_ws == 0 or need_st == 0:
            raise KvmemError(E_INVALID, self.lib.kvmem_last_error().decode())
        if self._host_ws is None or self._host_ws.numel() < need_ws:
            self._host_ws = torch.empty(need_ws, dtype=torch.uint8, device=self.device)
        if self._host_staging is None or self._host_staging.numel() < need_st:
            self._host_staging = torch.empty(need_st, dtype=torch.uint8, device=self.device)
        _check(self.lib.kvmem_score_host_index(self.handle, index_host.data_ptr(), n_blocks, index_host.shape[2],
                                               _dev(q, torch.bfloat16), M, tile_blocks, _dev(scores, torch.float32),
                                               self._host_staging.data_ptr(), self._host_staging.numel(),
                                               self._host_ws.data_ptr(), self._host_ws.numel(), _stream()))

    def select(self, q: torch.Tensor, params: SelectParams, sel_ids: torch.Tensor, n_sel: torch.Tensor,
               scores: Optional[torch.Tensor] = None, session_first: int = 0) -> None:
        """q bf16 [n_sessions][M][L][H][d]; sel_ids int32 [n_sessions][stride]; n_sel int32 [n_sessions]."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.select_workspace(ns, M)
        _check(self.lib.kvmem_select(self.handle, session_first, ns, _dev(q, torch.bfloat16), M, C.byref(params),
                                     _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                     None if scores is None else _dev(scores, torch.float32),
                                     ws.data_ptr(), ws.numel(), _stream()))

    def materialize(self, sel_ids: torch.Tensor, n_sel: torch.Tensor, view: View, session_first: int = 0) -> None:
        ns = n_sel.shape[0]
        _check(self.lib.kvmem_materialize(self.handle, session_first, ns, _dev(sel_ids, torch.int32),
                                          sel_ids.shape[-1], _dev(n_sel, torch.int32), _dev(view.k, torch.bfloat16),
                                          _dev(view.v, torch.bfloat16), view.cap_tokens, _stream()))

    def materialize_delta(self, prev_ids: torch.Tensor, n_prev: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor,
                          view: View, stats: Optional[torch.Tensor] = None, session_first: int = 0) -> None:
        """Move a view built from prev_ids to sel_ids: slots whose block stays are not touched, the others are fetched.
        stats int32 [n_sessions][3] (optional) receives (unchanged, retained and moved, incoming) per session."""
        ns = n_sel.shape[0]
        if prev_ids.shape != sel_ids.shape:
            raise ValueError("both id lists must have the same [n_sessions][stride] shape")
        _check(self.lib.kvmem_materialize_delta(self.handle, session_first, ns, _dev(prev_ids, torch.int32), _dev(n_prev, torch.int32),
                                                _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                                _dev(view.k, torch.bfloat16), _dev(view.v, torch.bfloat16), view.cap_tokens,
                                                None if stats is None else _dev(stats, torch.int32), _stream()))

    def view_attend(self, q: torch.Tensor, view: View, n_sel: torch.Tensor, out: torch.Tensor, lse: torch.Tensor,
                    scale: float = 0.0) -> None:
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_view_attend(self.handle, ns, _dev(q, torch.bfloat16), M, _dev(view.k, torch.bfloat16),
                                          _dev(view.v, torch.bfloat16), view.cap_tokens, _dev(n_sel, torch.int32),
                                          scale, _dev(out, torch.float32), _dev(lse, torch.float32),
                                          ws.data_ptr(), ws.numel(), _stream()))

    def materialize_attend(self, q: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor, view: View,
                           out: torch.Tensor, lse: torch.Tensor, scale: float = 0.0, session_first: int = 0) -> None:
        """materialize + view_attend in one pass over the selected blocks (same results, a third less HBM traffic)."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_materialize_attend(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                                 _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                                 _dev(view.k, torch.bfloat16), _dev(view.v, torch.bfloat16),
                                                 view.cap_tokens, scale, _dev(out, torch.float32),
                                                 _dev(lse, torch.float32), ws.data_ptr(), ws.numel(), _stream()))

    def paged_attend(self, q: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor, out: torch.Tensor,
                     lse: torch.Tensor, scale: float = 0.0, session_first: int = 0) -> None:
        """Copy-free execution view: attention straight over the selected blocks' pages (no view written)."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_paged_attend(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                           _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                           scale, _dev(out, torch.float32), _dev(lse, torch.float32),
                                           ws.data_ptr(), ws.numel(), _stream()))

    def paged_attend_rope(self, q: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor, out: torch.Tensor,
                          lse: torch.Tensor, first_position: int = 0, scale: float = 0.0, session_first: int = 0) -> None:
        """Copy-free view with position-consistent keys: raw key tiles are RoPE'd in shared memory on their way
        to the tensor cores (same results as materialize_rope + view_attend, no view written)."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_paged_attend_rope(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                                _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                                first_position, scale, _dev(out, torch.float32), _dev(lse, torch.float32),
                                                ws.data_ptr(), ws.numel(), _stream()))

    def materialize_attend_rope(self, q: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor, view: View,
                                out: torch.Tensor, lse: torch.Tensor, first_position: int = 0, scale: float = 0.0,
                                session_first: int = 0) -> None:
        """materialize_rope + view_attend in one call (one pass on a pool with the in-block key layout)."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_materialize_attend_rope(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                                      _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                                      _dev(view.k, torch.bfloat16), _dev(view.v, torch.bfloat16),
                                                      view.cap_tokens, first_position, scale, _dev(out, torch.float32),
                                                      _dev(lse, torch.float32), ws.data_ptr(), ws.numel(), _stream()))

    # ---- FP8 (E4M3) execution view
    def new_view_fp8(self, n_sessions: int, cap_tokens: int) -> Tuple[torch.Tensor, torch.Tensor]:
        """(keys uint8 [ns][L][G][cap][d], values uint8 [ns][L][G][cap/64][d][64]) for materialize_fp8."""
        c = self.cfg
        k8 = torch.zeros(n_sessions, c.n_layers, c.n_kv_heads, cap_tokens, c.head_dim, dtype=torch.uint8, device=self.device)
        v8t = torch.zeros(n_sessions, c.n_layers, c.n_kv_heads, cap_tokens // 64, c.head_dim, 64, dtype=torch.uint8,
                          device=self.device)
        return k8, v8t

    def materialize_fp8(self, sel_ids: torch.Tensor, n_sel: torch.Tensor, k8: torch.Tensor, v8t: torch.Tensor,
                        k_scale: float = 1.0, v_scale: float = 1.0, session_first: int = 0) -> None:
        ns = sel_ids.shape[0]
        _check(self.lib.kvmem_materialize_fp8(self.handle, session_first, ns, _dev(sel_ids, torch.int32), sel_ids.shape[-1],
                                              _dev(n_sel, torch.int32), _dev(k8, torch.uint8), _dev(v8t, torch.uint8),
                                              k8.shape[3], k_scale, v_scale, _stream()))

    def materialize_fp8_rope(self, sel_ids: torch.Tensor, n_sel: torch.Tensor, k8: torch.Tensor, v8t: torch.Tensor,
                             first_position: int = 0, k_scale: float = 1.0, v_scale: float = 1.0, session_first: int = 0) -> None:
        """Position-consistent FP8 view: keys rotated to their compact positions, then quantised; values as materialize_fp8."""
        ns = sel_ids.shape[0]
        _check(self.lib.kvmem_materialize_fp8_rope(self.handle, session_first, ns, _dev(sel_ids, torch.int32), sel_ids.shape[-1],
                                                   _dev(n_sel, torch.int32), _dev(k8, torch.uint8), _dev(v8t, torch.uint8),
                                                   k8.shape[3], first_position, k_scale, v_scale, _stream()))

    def view_attend_fp8(self, q: torch.Tensor, k8: torch.Tensor, v8t: torch.Tensor, n_sel: torch.Tensor, out: torch.Tensor,
                        lse: torch.Tensor, k_scale: float = 1.0, v_scale: float = 1.0, scale: float = 0.0) -> None:
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_view_attend_fp8(self.handle, ns, _dev(q, torch.bfloat16), M, _dev(k8, torch.uint8),
                                              _dev(v8t, torch.uint8), k8.shape[3], _dev(n_sel, torch.int32), scale, k_scale,
                                              v_scale, _dev(out, torch.float32), _dev(lse, torch.float32), ws.data_ptr(),
                                              ws.numel(), _stream()))

    def paged_attend_fp8(self, q: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor, out: torch.Tensor,
                         lse: torch.Tensor, scale: float = 0.0, session_first: int = 0) -> None:
        """Copy-free view over an FP8 repository (pool created with fp8_pages): attention straight over the pages."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_paged_attend_fp8(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                               _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                               scale, _dev(out, torch.float32), _dev(lse, torch.float32),
                                               ws.data_ptr(), ws.numel(), _stream()))

    def paged_attend_fp8_rope(self, q: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor, out: torch.Tensor,
                              lse: torch.Tensor, first_position: int = 0, scale: float = 0.0, session_first: int = 0) -> None:
        """Copy-free, position-consistent attention over an FP8 repository of in-block-rotated keys: the query is rotated
        back once per block (pool created with fp8_pages and rope_in_block_keys)."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_paged_attend_fp8_rope(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                                    _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                                    first_position, scale, _dev(out, torch.float32), _dev(lse, torch.float32),
                                                    ws.data_ptr(), ws.numel(), _stream()))

    def materialize_attend_fp8(self, q: torch.Tensor, sel_ids: torch.Tensor, n_sel: torch.Tensor, k8: torch.Tensor,
                               v8t: torch.Tensor, out: torch.Tensor, lse: torch.Tensor, scale: float = 0.0,
                               session_first: int = 0) -> None:
        """materialize_fp8 + view_attend_fp8 in one pass over an FP8 repository (pool created with fp8_pages)."""
        ns, M = q.shape[0], q.shape[1]
        ws = self.attend_workspace(ns, M)
        _check(self.lib.kvmem_materialize_attend_fp8(self.handle, session_first, ns, _dev(q, torch.bfloat16), M,
                                                     _dev(sel_ids, torch.int32), sel_ids.shape[-1], _dev(n_sel, torch.int32),
                                                     _dev(k8, torch.uint8), _dev(v8t, torch.uint8), k8.shape[3], scale,
                                                     _dev(out, torch.float32), _dev(lse, torch.float32),
                                                     ws.data_ptr(), ws.numel(), _stream()))

    def view_attend_static(self, q: torch.Tensor, view: View, n_sel: torch.Tensor, out: torch.Tensor,
                           lse: torch.Tensor, scale: float = 0.0) -> None:
        """view_attend without a caller workspace, for hosts that cannot allocate device memory: the
        split-K scratch is a fixed array inside the library (at most 8 (session, layer, KV head)
        triples per call; calls that overlap on the GPU race on it)."""
        ns, M = q.shape[0], q.shape[1]
        _check(self.lib.kvmem_view_attend_static(self.handle, ns, _dev(q, torch.bfloat16), M,
                                                 _dev(view.k, torch.bfloat16), _dev(view.v, torch.bfloat16),
                                                 view.cap_tokens, _dev(n_sel, torch.int32), scale,
                                                 _dev(out, torch.float32), _dev(lse, torch.float32), _stream()))

    def recall_step_host(self, q_host: torch.Tensor, params: SelectParams, sel_ids: torch.Tensor,
                         n_sel: torch.Tensor, view: View, out_host: torch.Tensor, lse_host: torch.Tensor,
                         scale: float = 0.0, session_first: int = 0) -> None:
        """Whole step with HOST query and results (the library does the copies and waits for the stream)."""
        ns, M = q_host.shape[0], q_host.shape[1]
        for t, dt in ((q_host, torch.bfloat16), (out_host, torch.float32), (lse_host, torch.float32)):
            if t.is_cuda or not t.is_contiguous() or t.dtype != dt:
                raise ValueError("expected contiguous CPU tensors (bf16 query, fp32 outputs)")
        need = self.lib.kvmem_step_staging_bytes(C.byref(self.cfg), ns, M)
        if self._staging is None or self._staging.numel() < need:
            self._staging = torch.empty(need, dtype=torch.uint8, device=self.device)
        sws, aws = self.select_workspace(ns, M), self.attend_workspace(ns, M)
        _check(self.lib.kvmem_recall_step_host(
            self.handle, session_first, ns, q_host.data_ptr(), M, C.byref(params), _dev(sel_ids, torch.int32),
            sel_ids.shape[-1], _dev(n_sel, torch.int32), _dev(view.k, torch.bfloat16), _dev(view.v, torch.bfloat16),
            view.cap_tokens, scale, out_host.data_ptr(), lse_host.data_ptr(), self._staging.data_ptr(),
            self._staging.numel(), sws.data_ptr(), sws.numel(), aws.data_ptr(), aws.numel(), _stream()))

    def host_step(self, q_shape, params: SelectParams, sel_ids: torch.Tensor, n_sel: torch.Tensor, view: View,
                  out_host: torch.Tensor, lse_host: torch.Tensor, scale: float = 0.0, session_first: int = 0) -> "HostStep":
        """recall_step_host with everything but the query marshalled once (a decode loop calls the same step with the
        same buffers every token): returns a callable that takes the pinned bf16 query of shape q_shape."""
        return HostStep(self, tuple(q_shape), params, sel_ids, n_sel, view, out_host, lse_host, scale, session_first)

    # ---- helpers that only allocate
    def new_view(self, n_sessions: int, cap_tokens: int) -> View:
        c = self.cfg
        shape = (n_sessions, c.n_layers, c.n_kv_heads, cap_tokens, c.head_dim)
        return View(torch.zeros(shape, dtype=torch.bfloat16, device=self.device),
                    torch.zeros(shape, dtype=torch.bfloat16, device=self.device), cap_tokens)

    def new_outputs(self, n_sessions: int, n_q_tokens: int) -> Tuple[torch.Tensor, torch.Tensor]:
        c = self.cfg
        out = torch.empty(n_sessions, n_q_tokens, c.n_layers, c.n_q_heads, c.head_dim, dtype=torch.float32,
                          device=self.device)
        lse = torch.empty(n_sessions, n_q_tokens, c.n_layers, c.n_q_heads, dtype=torch.float32, device=self.device)
        return out, lse

    # ---- inspection
    def index(self, session: int) -> torch.Tensor:
        """Copy of the session's Mean-K index: bf16 [L][G][n_blocks][d]."""
        ptr, n = C.c_void_p(), C.c_int32()
        _check(self.lib.kvmem_get_index(self.handle, session, C.byref(ptr), C.byref(n)))
        c = self.cfg
        off = (ptr.value - self.storage.data_ptr())
        elems = c.n_layers * c.n_kv_heads * c.max_blocks_per_session * c.head_dim
        full = self.storage[off:off + 2 * elems].view(torch.bfloat16).view(c.n_layers, c.n_kv_heads,
                                                                              c.max_blocks_per_session, c.head_dim)
        return full[:, :, :n.value, :].clone()

    def block_table(self, session: int) -> torch.Tensor:
        ptr, n = C.c_void_p(), C.c_int32()
        _check(self.lib.kvmem_get_block_table(self.handle, session, C.byref(ptr), C.byref(n)))
        off = ptr.value - self.storage.data_ptr()
        return self.storage[off:off + 4 * n.value].view(torch.int32).clone()

    def selftest_wait_timeout(self, limit_us: int = 1000) -> int:
        """Run the kernels' bounded wait to its limit on a barrier nobody arrives at; returns the nanoseconds it lasted.
        The status word then holds E_TIMEOUT until device_status() reads it."""
        waited = torch.zeros(1, dtype=torch.int64, device=self.device)
        _check(self.lib.kvmem_selftest_wait_timeout(self.handle, limit_us, waited.data_ptr(), _stream()))
        return int(waited.item())

    def device_status(self) -> int:
        st = C.c_int32()
        _check(self.lib.kvmem_device_status(self.handle, C.byref(st), _stream()))
        return st.value


class ViewCache:
    """The execution view kept across steps for one session: `cap_blocks` slots of one block each (keys
    encoded for their compact position, values unchanged), updated as a working-set delta."""

    def __init__(self, pool: Pool, cap_blocks: int, max_delta_ropes: int, first_position: int = 0):
        self.pool, self.cap, self.max_delta, self.first_position = pool, cap_blocks, max_delta_ropes, first_position
        need = pool.lib.kvmem_view_cache_bytes(pool.handle, cap_blocks)
        if need == 0:
            raise KvmemError(E_INVALID, "cap_blocks must be in [1, 32768]")
        self.buf = torch.empty(need, dtype=torch.uint8, device=pool.device)
        offs = (C.c_size_t * 6)()
        _check(pool.lib.kvmem_view_cache_layout(pool.handle, cap_blocks, offs))
        self.offsets = list(offs)
        self.stats = torch.zeros(4, dtype=torch.int32, device=pool.device)
        _check(pool.lib.kvmem_view_cache_reset(pool.handle, self.buf.data_ptr(), self.buf.numel(), cap_blocks, _stream()))

    def update(self, session: int, sel_ids: torch.Tensor, n_sel: torch.Tensor) -> None:
        """sel_ids int32 [>= n] ascending (one session's row), n_sel int32 [1]; stats land in self.stats."""
        p = self.pool
        _check(p.lib.kvmem_view_cache_update(p.handle, session, _dev(sel_ids, torch.int32), _dev(n_sel, torch.int32),
                                             self.buf.data_ptr(), self.buf.numel(), self.cap, self.max_delta,
                                             self.first_position, self.stats.data_ptr(), _stream()))

    def attend(self, q: torch.Tensor, out: torch.Tensor, lse: torch.Tensor, scale: float = 0.0) -> None:
        """q bf16 [M][L][H][d] (one session) -> out fp32 [M][L][H][d], lse fp32 [M][L][H]."""
        p = self.pool
        M = q.shape[0]
        ws = p.attend_workspace(1, M)
        _check(p.lib.kvmem_view_cache_attend(p.handle, _dev(q, torch.bfloat16), M, self.buf.data_ptr(), self.buf.numel(),
                                             self.cap, scale, _dev(out, torch.float32), _dev(lse, torch.float32),
                                             ws.data_ptr(), ws.numel(), _stream()))

    # ---- inspection (copies)
    def _ints(self, which: int, n: int) -> torch.Tensor:
        o = self.offsets[which]
        return self.buf[o:o + 4 * n].view(torch.int32).clone()

    def records(self):
        """(slot_block, slot_pos, slot_cnt, view_slots, n_view) as CPU tensors / int."""
        torch.cuda.synchronize(self.pool.device)
        return (self._ints(1, self.cap).cpu(), self._ints(2, self.cap).cpu(), self._ints(3, self.cap).cpu(),
                self._ints(4, self.cap).cpu(), int(self._ints(5, 1).cpu()[0]))

    def pages(self) -> torch.Tensor:
        """bf16 [cap][2][L][G][B][d]: the slots in the pool's page format (a view of the cache buffer)."""
        c = self.pool.cfg
        n = self.cap * 2 * c.n_layers * c.n_kv_heads * c.block_tokens * c.head_dim
        o = self.offsets[0]
        return self.buf[o:o + 2 * n].view(torch.bfloat16).view(self.cap, 2, c.n_layers, c.n_kv_heads, c.block_tokens, c.head_dim)
