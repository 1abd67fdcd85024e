"""ctypes wrapper of the CPU oracle (``kvmem_oracle.c``).  TEST INFRASTRUCTURE, NOT PRODUCT.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this.
It imports nothing from the CUDA package.  Arrays are NumPy; bf16 tensors travel as
``uint16`` bit patterns (``torch_tensor.view(torch.int16).numpy().view(np.uint16)``).

Parity pins: every function here is pinned by ``tests/test_oracle_pins.py`` (and the RoPE
functions by ``tests/test_oracle_rope_pins.py``) against closed
forms, invariants of the equations, special cases that reduce to textbook softmax
attention, and brute force on tiny inputs.  What stays *parity unpinned* is only what the
paper never prints: the authors' sink/recent sizes, whether their candidate set excludes
reserved blocks, their index element type, their query-head to KV-head mapping, their
tie-break, and their RoPE variant (pairing and base).  The readings taken are stated in ``kvmem_oracle.c``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvmem_oracle.c")
_LIB = os.path.join(_HERE, "libkvmem_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64, i32, dbl, p = C.c_int64, C.c_int, C.c_double, C.c_void_p
        L.kvo_mean_k_index.argtypes = [p, i64, i32, i32, i32, i32, p, i64, i64]
        L.kvo_mean_k_index.restype = None
        L.kvo_block_scores.argtypes = [p, p, i64, i64, i32, i32, i32, i32, i32, p, p]
        L.kvo_block_scores.restype = i32
        L.kvo_budget_blocks.argtypes = [i64, i32, i64, i64, i64]
        L.kvo_budget_blocks.restype = i64
        L.kvo_select.argtypes = [p, i64, i32, i64, i64, i64, i64, i64, p]
        L.kvo_select.restype = i64
        L.kvo_place_blocks.argtypes = [p, p, i64, i32, i32, i32, i32, p, p, p]
        L.kvo_place_blocks.restype = None
        L.kvo_gather.argtypes = [p, p, p, p, i64, i32, i32, i32, i32, p, p, i64]
        L.kvo_gather.restype = None
        L.kvo_attend.argtypes = [p, p, p, i64, i64, i32, i32, i32, i32, i32, dbl, p, p]
        L.kvo_attend.restype = None
        L.kvo_rope_table.argtypes = [i64, i32, dbl, p]
        L.kvo_rope_table.restype = None
        L.kvo_rope_rotate.argtypes = [p, p, i64, i32, i32, p, p, i64, i32]
        L.kvo_rope_rotate.restype = i32
        L.kvo_gather_rope.argtypes = [p, p, p, p, i64, i32, i32, i32, i32, p, p, i64, i64, p, i64, i32]
        L.kvo_gather_rope.restype = i32
        L.kvo_working_set_delta.argtypes = [p, i64, p, i64, p, p, p, p]
        L.kvo_working_set_delta.restype = None
        L.kvo_view_cache_update.argtypes = [p, p, p, p, i64, i32, i32, i32, i32, i64, i64, i64, p, i64, p, p, p, p, p, p, p, i32]
        L.kvo_attend_qrot.argtypes = [p, p, p, i64, i64, i32, i32, i32, i32, i32, i32, i64, p, dbl, p, p]
        L.kvo_attend_qrot.restype = None
        L.kvo_view_cache_update.restype = i32
        L.kvo_view_cache_view.argtypes = [p, p, p, i64, i32, i32, i32, i32, p, p, i64]
        L.kvo_view_cache_view.restype = None
        f32 = C.c_float
        L.kvo_quantize_e4m3.argtypes = [p, p, i64, f32]
        L.kvo_quantize_e4m3.restype = None
        L.kvo_dequantize_e4m3.argtypes = [p, p, i64, f32]
        L.kvo_dequantize_e4m3.restype = None
        L.kvo_gather_fp8.argtypes = [p, p, p, p, i64, i32, i32, i32, i32, f32, f32, p, p, i64]
        L.kvo_gather_fp8.restype = None
        L.kvo_attend_fp8.argtypes = [p, p, p, i64, i64, i32, i32, i32, i32, i32, dbl, dbl, dbl, p, p]
        L.kvo_attend_fp8.restype = None
        L.kvo_threads.argtypes = []
        L.kvo_threads.restype = i32
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a: np.ndarray) -> np.ndarray:
    assert a.dtype == np.uint16 and a.flags.c_contiguous, "bf16 bit patterns as contiguous uint16"
    return a


def threads() -> int:
    return int(lib().kvo_threads())


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32 (for use in tests)."""
    return (a.astype(np.uint32) << 16).view(np.float32)


def mean_k_index(K: np.ndarray, B: int, idx: Optional[np.ndarray] = None, b_first: int = 0) -> np.ndarray:
    """K: uint16 [n_blocks*B][L][G][d]  ->  idx uint16 [L][G][stride][d] (rows b_first.. filled)."""
    _u16(K)
    n_tok, L, G, d = K.shape
    assert n_tok % B == 0, "only whole blocks are indexed"
    nb = n_tok // B
    if idx is None:
        idx = np.zeros((L, G, b_first + nb, d), dtype=np.uint16)
    _u16(idx)
    assert idx.shape[0] == L and idx.shape[1] == G and idx.shape[3] == d and idx.shape[2] >= b_first + nb
    lib().kvo_mean_k_index(_ptr(K), nb, B, L, G, d, _ptr(idx), idx.shape[2], b_first)
    return idx


def block_scores(q: np.ndarray, idx: np.ndarray, NB: int) -> Tuple[np.ndarray, np.ndarray]:
    """q uint16 [M][L][H][d], idx uint16 [L][G][stride][d]  ->  (R fp32 [NB], R_g fp32 [G][NB])."""
    _u16(q), _u16(idx)
    M, L, H, d = q.shape
    G = idx.shape[1]
    assert idx.shape[0] == L and idx.shape[3] == d and H % G == 0 and NB <= idx.shape[2]
    R = np.zeros(NB, dtype=np.float32)
    Rg = np.zeros((G, NB), dtype=np.float32)
    rc = lib().kvo_block_scores(_ptr(q), _ptr(idx), NB, idx.shape[2], M, L, H, G, d, _ptr(R), _ptr(Rg))
    if rc != 0:
        raise MemoryError("oracle: logit buffer allocation failed")
    return R, Rg


def budget_blocks(NB: int, B: int, budget_blocks: int, max_view_tokens: int, mandatory_tokens: int = 0) -> int:
    return int(lib().kvo_budget_blocks(NB, B, budget_blocks, max_view_tokens, mandatory_tokens))


def select(R: np.ndarray, B: int, budget_blocks: int, max_view_tokens: int, mandatory_tokens: int = 0,
           n_sink_blocks: int = 0, n_recent_blocks: int = 0) -> np.ndarray:
    """R fp32 [NB] -> ascending int32 ids of the selected blocks."""
    assert R.dtype == np.float32 and R.flags.c_contiguous
    NB = R.shape[0]
    sel = np.zeros(max(NB, 1), dtype=np.int32)
    n = lib().kvo_select(_ptr(R), NB, B, budget_blocks, max_view_tokens, mandatory_tokens,
                         n_sink_blocks, n_recent_blocks, _ptr(sel))
    return sel[:n].copy()


@dataclass
class Repository:
    """Physical pages [n_pages][B][L][G][d] (uint16) for K and V."""
    pagesK: np.ndarray
    pagesV: np.ndarray

    @classmethod
    def empty(cls, n_pages: int, B: int, L: int, G: int, d: int) -> "Repository":
        return cls(np.zeros((n_pages, B, L, G, d), np.uint16), np.zeros((n_pages, B, L, G, d), np.uint16))

    def place(self, K: np.ndarray, V: np.ndarray, table: np.ndarray) -> None:
        """Copy whole blocks K, V (uint16 [n_blocks*B][L][G][d]) into pages table[0..n_blocks)."""
        _u16(K), _u16(V)
        _, B, L, G, d = self.pagesK.shape
        nb = K.shape[0] // B
        assert K.shape[0] == nb * B and table.dtype == np.int32 and table.shape[0] >= nb
        assert int(table[:nb].max(initial=-1)) < self.pagesK.shape[0] and int(table[:nb].min(initial=0)) >= 0
        lib().kvo_place_blocks(_ptr(K), _ptr(V), nb, B, L, G, d, _ptr(np.ascontiguousarray(table)),
                               _ptr(self.pagesK), _ptr(self.pagesV))


def gather(repo: Repository, table: np.ndarray, sel: np.ndarray, cap_tokens: int,
           viewK: Optional[np.ndarray] = None, viewV: Optional[np.ndarray] = None
           ) -> Tuple[np.ndarray, np.ndarray]:
    """Execution view uint16 [L][G][cap_tokens][d] x2 (tokens beyond len(sel)*B left as they were)."""
    _, B, L, G, d = repo.pagesK.shape
    assert table.dtype == np.int32 and sel.dtype == np.int32 and len(sel) * B <= cap_tokens
    if viewK is None:
        viewK = np.zeros((L, G, cap_tokens, d), np.uint16)
        viewV = np.zeros((L, G, cap_tokens, d), np.uint16)
    lib().kvo_gather(_ptr(repo.pagesK), _ptr(repo.pagesV), _ptr(np.ascontiguousarray(table)),
                     _ptr(np.ascontiguousarray(sel)), len(sel), B, L, G, d, _ptr(viewK), _ptr(viewV), cap_tokens)
    return viewK, viewV


def attend(q: np.ndarray, viewK: np.ndarray, viewV: np.ndarray, T: int, scale: Optional[float] = None
           ) -> Tuple[np.ndarray, np.ndarray]:
    """q uint16 [M][L][H][d]; views uint16 [L][G][cap][d]  ->  (O fp32 [M][L][H][d], LSE fp32 [M][L][H])."""
    _u16(q), _u16(viewK), _u16(viewV)
    M, L, H, d = q.shape
    G, cap = viewK.shape[1], viewK.shape[2]
    assert viewK.shape == viewV.shape and viewK.shape[0] == L and viewK.shape[3] == d and T <= cap
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    out = np.zeros((M, L, H, d), np.float32)
    lse = np.zeros((M, L, H), np.float32)
    lib().kvo_attend(_ptr(q), _ptr(viewK), _ptr(viewV), T, cap, M, L, H, G, d, float(scale), _ptr(out), _ptr(lse))
    return out, lse


# ---- position-consistent materialisation (RoPE) ------------------------------------------------

def rope_table(n_pos: int, d: int, theta: float) -> np.ndarray:
    """fp32 [n_pos][d/2][2] = (cos, sin) of position * theta^(-2i/d)."""
    tab = np.zeros((n_pos, d // 2, 2), np.float32)
    lib().kvo_rope_table(n_pos, d, float(theta), _ptr(tab))
    return tab


def rope_rotate(x: np.ndarray, pos: np.ndarray, tab: np.ndarray, inverse: bool = False) -> np.ndarray:
    """x uint16 [n_rows][n_vec][d]; every vector of row r rotated by pos[r] (inverse: by -pos[r])."""
    _u16(x)
    n_rows, n_vec, d = x.shape
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    assert pos.shape == (n_rows,) and tab.dtype == np.float32 and tab.shape[1] == d // 2
    y = np.zeros_like(x)
    rc = lib().kvo_rope_rotate(_ptr(x), _ptr(y), n_rows, n_vec, d, _ptr(pos), _ptr(tab), tab.shape[0], int(inverse))
    if rc != 0:
        raise ValueError("position outside the RoPE table")
    return y


def gather_rope(repo: Repository, table: np.ndarray, sel: np.ndarray, cap_tokens: int, first_pos: int,
                tab: np.ndarray, in_block: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """Execution view whose keys carry RoPE at their compact positions first_pos + j*B + t.  in_block: the pages
    hold keys already rotated by their offset t inside the block; the view rotates them by first_pos + j*B."""
    _, B, L, G, d = repo.pagesK.shape
    assert table.dtype == np.int32 and sel.dtype == np.int32 and len(sel) * B <= cap_tokens
    viewK = np.zeros((L, G, cap_tokens, d), np.uint16)
    viewV = np.zeros((L, G, cap_tokens, d), np.uint16)
    rc = lib().kvo_gather_rope(_ptr(repo.pagesK), _ptr(repo.pagesV), _ptr(np.ascontiguousarray(table)),
                               _ptr(np.ascontiguousarray(sel)), len(sel), B, L, G, d, _ptr(viewK), _ptr(viewV),
                               cap_tokens, first_pos, _ptr(tab), tab.shape[0], int(in_block))
    if rc != 0:
        raise ValueError("compact positions outside the RoPE table")
    return viewK, viewV


def attend_qrot(q: np.ndarray, viewK: np.ndarray, viewV: np.ndarray, T: int, block_tokens: int, first_pos: int,
                tab: np.ndarray, scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Attention over a plain gather of in-block-rotated keys, the query rotated back by each tile's position."""
    _u16(q), _u16(viewK), _u16(viewV)
    M, L, H, d = q.shape
    G, cap = viewK.shape[1], viewK.shape[2]
    assert first_pos + T <= tab.shape[0] and T <= cap
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    out = np.zeros((M, L, H, d), np.float32)
    lse = np.zeros((M, L, H), np.float32)
    lib().kvo_attend_qrot(_ptr(q), _ptr(viewK), _ptr(viewV), T, cap, M, L, H, G, d, block_tokens, first_pos, _ptr(tab),
                          float(scale), _ptr(out), _ptr(lse))
    return out, lse


# ---- working-set delta ---------------------------------------------------------------------------

def working_set_delta(prev: np.ndarray, nxt: np.ndarray):
    """Ascending int32 id lists -> (retained [nR][3] = id, old slot, new slot; incoming [nL][2] = id, new slot;
    outgoing [nE])."""
    prev, nxt = np.ascontiguousarray(prev, np.int32), np.ascontiguousarray(nxt, np.int32)
    ret = np.zeros((max(len(nxt), 1), 3), np.int32)
    inc = np.zeros((max(len(nxt), 1), 2), np.int32)
    out = np.zeros(max(len(prev), 1), np.int32)
    cnt = np.zeros(3, np.int32)
    lib().kvo_working_set_delta(_ptr(prev), len(prev), _ptr(nxt), len(nxt), _ptr(ret), _ptr(inc), _ptr(out), _ptr(cnt))
    return ret[: cnt[0]].copy(), inc[: cnt[1]].copy(), out[: cnt[2]].copy()


# ---- incremental contiguous view (Eq. "kvmem-working-set-delta", Sec. 4.4) ----------------------------

def view_delta_plan(prev: np.ndarray, nxt: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """What has to happen to every slot of a contiguous view that held the blocks `prev` (ascending ids, block prev[j] at
    tokens [j*B, (j+1)*B)) so that it holds `nxt`: action[j] = 0 the slot already holds nxt[j] (nothing moves),
    1 nxt[j] is a retained block (in W_next and W_prev) that sat in another slot, 2 nxt[j] is incoming (in W_next only).
    Returns (action int32 [len(nxt)], counts int32 [3] = slots unchanged, retained and moved, incoming)."""
    prev, nxt = np.ascontiguousarray(prev, np.int32), np.ascontiguousarray(nxt, np.int32)
    held = set(int(b) for b in prev)
    action = np.zeros(len(nxt), np.int32)
    for j, b in enumerate(nxt):
        if j < len(prev) and int(prev[j]) == int(b):
            action[j] = 0
        elif int(b) in held:
            action[j] = 1
        else:
            action[j] = 2
    counts = np.array([(action == 0).sum(), (action == 1).sum(), (action == 2).sum()], np.int32)
    return action, counts


def view_update(repo: Repository, table: np.ndarray, viewK: np.ndarray, viewV: np.ndarray, prev: np.ndarray,
                nxt: np.ndarray) -> np.ndarray:
    """Move a contiguous view (uint16 [L][G][cap][d] keys and values, in place) from the working set `prev` to `nxt`: a
    slot whose block stays is not touched; every other slot of `nxt` receives its block from the repository (with the
    whole history in one memory a moved retained block costs the same read and write whether it is shifted inside the
    view or fetched again, and fetching has no ordering hazard).  Tokens past len(nxt) * B are left as they were.
    Returns the counts of view_delta_plan."""
    _, B, L, G, d = repo.pagesK.shape
    action, counts = view_delta_plan(prev, nxt)
    assert len(nxt) * B <= viewK.shape[2]
    for j, b in enumerate(np.ascontiguousarray(nxt, np.int32)):
        if action[j] == 0:
            continue
        page = int(table[int(b)])
        viewK[:, :, j * B:(j + 1) * B, :] = repo.pagesK[page].transpose(1, 2, 0, 3)      # [B][L][G][d] -> [L][G][B][d]
        viewV[:, :, j * B:(j + 1) * B, :] = repo.pagesV[page].transpose(1, 2, 0, 3)
    return counts


# ---- execution cache: working-set reuse with bounded delta re-RoPE -----------------------------------

class ViewCache:
    """Oracle state of the execution cache (Sec. 4.4): `cap` slots of one block each, token-major
    [cap][B][L][G][d] keys (encoded for their compact position) and values, plus the slot records."""

    def __init__(self, repo: Repository, cap: int):
        _, B, L, G, d = repo.pagesK.shape
        self.cap, self.dims = cap, (B, L, G, d)
        self.K = np.zeros((cap, B, L, G, d), np.uint16)
        self.V = np.zeros((cap, B, L, G, d), np.uint16)
        self.slot_block = np.full(cap, -1, np.int32)
        self.slot_pos = np.zeros(cap, np.int32)
        self.slot_cnt = np.zeros(cap, np.int32)
        self.view_slots = np.full(cap, -1, np.int32)
        self.n_view = 0

    def update(self, repo: Repository, table: np.ndarray, sel: np.ndarray, max_delta: int, first_pos: int,
               tab: np.ndarray, in_block: bool = False) -> np.ndarray:
        """Move the cache to the working set `sel`; returns stats (unmoved, delta re-RoPEd, rebuilt, incoming)."""
        B, L, G, d = self.dims
        sel = np.ascontiguousarray(sel, np.int32)
        stats = np.zeros(4, np.int32)
        rc = lib().kvo_view_cache_update(_ptr(repo.pagesK), _ptr(repo.pagesV), _ptr(np.ascontiguousarray(table)), _ptr(sel),
                                         len(sel), B, L, G, d, self.cap, max_delta, first_pos, _ptr(tab), tab.shape[0],
                                         _ptr(self.K), _ptr(self.V), _ptr(self.slot_block), _ptr(self.slot_pos),
                                         _ptr(self.slot_cnt), _ptr(self.view_slots), _ptr(stats), int(in_block))
        if rc != 0:
            raise ValueError("selection larger than the cache, or compact positions outside the RoPE table")
        self.n_view = len(sel)
        return stats

    def view(self, cap_tokens: int) -> Tuple[np.ndarray, np.ndarray]:
        """The execution view in attention order: [L][G][cap_tokens][d] keys and values."""
        B, L, G, d = self.dims
        viewK = np.zeros((L, G, cap_tokens, d), np.uint16)
        viewV = np.zeros((L, G, cap_tokens, d), np.uint16)
        lib().kvo_view_cache_view(_ptr(self.K), _ptr(self.V), _ptr(self.view_slots), self.n_view, B, L, G, d,
                                  _ptr(viewK), _ptr(viewV), cap_tokens)
        return viewK, viewV


# ---- FP8 (E4M3) execution view ------------------------------------------------------------------------

def quantize_e4m3(x: np.ndarray, inv_scale: float = 1.0) -> np.ndarray:
    """bf16 bit patterns (uint16) -> E4M3 codes (uint8) of x * inv_scale, round to nearest even, saturating at 448."""
    x = np.ascontiguousarray(_u16(x))
    y = np.zeros(x.shape, np.uint8)
    lib().kvo_quantize_e4m3(_ptr(x), _ptr(y), x.size, float(inv_scale))
    return y


def dequantize_e4m3(y: np.ndarray, scale: float = 1.0) -> np.ndarray:
    y = np.ascontiguousarray(y, np.uint8)
    x = np.zeros(y.shape, np.float32)
    lib().kvo_dequantize_e4m3(_ptr(y), _ptr(x), y.size, float(scale))
    return x


def gather_fp8(repo: Repository, table: np.ndarray, sel: np.ndarray, cap_tokens: int, k_inv_scale: float = 1.0,
               v_inv_scale: float = 1.0) -> Tuple[np.ndarray, np.ndarray]:
    """FP8 execution view: keys uint8 [L][G][cap][d]; values uint8 [L][G][cap/64][d][64] (transposed per 64-token tile)."""
    _, B, L, G, d = repo.pagesK.shape
    assert cap_tokens % 64 == 0 and len(sel) * B <= cap_tokens and table.dtype == np.int32 and sel.dtype == np.int32
    vK = np.zeros((L, G, cap_tokens, d), np.uint8)
    vV = np.zeros((L, G, cap_tokens // 64, d, 64), np.uint8)
    lib().kvo_gather_fp8(_ptr(repo.pagesK), _ptr(repo.pagesV), _ptr(np.ascontiguousarray(table)),
                         _ptr(np.ascontiguousarray(sel)), len(sel), B, L, G, d, float(k_inv_scale), float(v_inv_scale),
                         _ptr(vK), _ptr(vV), cap_tokens)
    return vK, vV


def attend_fp8(q: np.ndarray, viewK8: np.ndarray, viewV8T: np.ndarray, T: int, k_scale: float = 1.0, v_scale: float = 1.0,
               scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """q uint16 [M][L][H][d] over an FP8 view -> (O fp32 [M][L][H][d], LSE fp32 [M][L][H])."""
    _u16(q)
    M, L, H, d = q.shape
    G, cap = viewK8.shape[1], viewK8.shape[2]
    assert viewK8.dtype == np.uint8 and viewV8T.dtype == np.uint8 and viewV8T.shape == (L, G, cap // 64, d, 64) and T <= cap
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    out = np.zeros((M, L, H, d), np.float32)
    lse = np.zeros((M, L, H), np.float32)
    lib().kvo_attend_fp8(_ptr(q), _ptr(viewK8), _ptr(viewV8T), T, cap, M, L, H, G, d, float(scale), float(k_scale),
                         float(v_scale), _ptr(out), _ptr(lse))
    return out, lse


def attend_fp8_qrot(q: np.ndarray, viewK8: np.ndarray, viewV8T: np.ndarray, T: int, block_tokens: int, first_pos: int,
                    tab: np.ndarray, k_scale: float = 1.0, v_scale: float = 1.0, scale: Optional[float] = None
                    ) -> Tuple[np.ndarray, np.ndarray]:
    """Attention over an FP8 view whose keys are the codes of in-block-rotated keys (RoPE(k, offset in block) / k_scale),
    with the query rotated back by each block's compact position (Sec. 4.4 position consistency on an FP8 KV cache,
    Sec. 6.1).  Every E4M3 value is exactly representable in bf16, so this is attend_qrot on the dequantised view:
    the codes widened (exactly) to bf16, the value tiles transposed back, k_scale folded into the softmax scale and
    v_scale applied to the output."""
    _u16(q)
    L, G, cap, d = viewK8.shape
    assert viewK8.dtype == np.uint8 and viewV8T.dtype == np.uint8 and viewV8T.shape == (L, G, cap // 64, d, 64)
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    kf = dequantize_e4m3(viewK8)
    vf = dequantize_e4m3(viewV8T).transpose(0, 1, 2, 4, 3).reshape(L, G, cap, d)
    kb = np.ascontiguousarray(kf).view(np.uint32) >> 16          # exact: an E4M3 value has 3 mantissa bits
    vb = np.ascontiguousarray(vf).view(np.uint32) >> 16
    assert np.array_equal(bf16_bits_to_f32(kb.astype(np.uint16)), kf)
    out, lse = attend_qrot(q, np.ascontiguousarray(kb.astype(np.uint16)), np.ascontiguousarray(vb.astype(np.uint16)), T,
                           block_tokens, first_pos, tab, float(scale) * float(k_scale))
    return out * np.float32(v_scale), lse
