"""The C-ABI shared library: it loads without a GPU, exports every symbol the header declares,
and its pure host helpers (sizes, budget clamp) agree with the definitions."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import kvmem_oracle as orc
from paper_2609_04852_b200 import PoolConfig, SelectParams, budget_blocks, load_library
from paper_2609_04852_b200 import _build, kvmem

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "kvmem.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvmem_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    _build.build()
    lib = load_library()
    declared = _declared_functions()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in kvmem.h but not exported"
    assert sorted(kvmem.EXPORTED) == declared, "binding and header disagree on the entry points"


def test_pool_bytes_follow_the_layout():
    lib = load_library()
    cfg = PoolConfig(1, 32, 8, 128, 64, 1, 16384, 16384, 0)
    nbytes = lib.kvmem_pool_bytes(C.byref(cfg))
    pages = 16384 * 2 * 8 * 64 * 128 * 2          # 4 GiB of K and V
    index = 8 * 16384 * 128 * 2                   # 32 MiB: one vector per (block, layer, KV head)
    assert pages + index <= nbytes <= pages + index + 16384 * 4 + 4096
    assert index // 16384 == 1 * 8 * 128 * 2      # bytes per block grow linearly with blocks (Sec. 6.5)
    bad = PoolConfig(1, 32, 5, 128, 64, 1, 8, 8, 0)
    assert lib.kvmem_pool_bytes(C.byref(bad)) == 0 and b"multiple" in lib.kvmem_last_error()
    assert lib.kvmem_select_workspace_bytes(C.byref(cfg), 1, 4) > 16 * 8 * 16384 * 4
    assert lib.kvmem_attend_workspace_bytes(C.byref(cfg), 1, 4) > 0
    assert lib.kvmem_step_staging_bytes(C.byref(cfg), 1, 4) >= 4 * 32 * 128 * (2 + 4) + 4 * 32 * 4


def test_budget_clamp_agrees_with_the_capacity_inequality_and_the_oracle():
    rng = np.random.default_rng(5)
    assert budget_blocks(SelectParams(4096, 262144, 0, 0, 0), 64, 16384) == 4096
    assert budget_blocks(SelectParams(4096, 262144, 1, 0, 0), 64, 16384) == 4095
    for _ in range(200):
        NB, B16, k, Ba, nq = (int(x) for x in rng.integers(0, 5000, 5))
        B = 16 * (1 + B16 % 16)
        got = budget_blocks(SelectParams(k, Ba, nq, 0, 0), B, NB)
        assert got == orc.budget_blocks(NB, B, k, Ba, nq)
        assert got == 0 or nq + B * got <= Ba


def test_calls_without_a_pool_fail_cleanly():
    lib = load_library()
    assert lib.kvmem_session_reset(None, 0, None) == kvmem.E_STATE
    assert lib.kvmem_pool_destroy(None) == kvmem.E_STATE
    assert lib.kvmem_set_option(b"no_such_option", 1) == kvmem.E_INVALID
    handle = C.c_void_p()
    cfg = PoolConfig(1, 32, 8, 128, 64, 1, 8, 8, 0)
    assert lib.kvmem_pool_create(C.byref(cfg), None, 0, C.byref(handle)) == kvmem.E_INVALID   # null storage
    assert not handle.value


def test_page_format_options_are_validated_and_sized_on_the_host():
    """The optional page formats (keys rotated by their in-block offset; FP8 repository) are configuration: what is
    accepted, what is refused and how many bytes the pool takes are decided on the host, before any GPU work."""
    lib = load_library()
    base = dict(n_layers=1, n_q_heads=32, n_kv_heads=8, head_dim=128, block_tokens=64, max_sessions=1, max_blocks=1024,
                max_blocks_per_session=1024, device=0)

    def cfg(**kw):
        c = PoolConfig()
        for k, v in {**base, **kw}.items():
            setattr(c, k, v)
        return c

    plain = lib.kvmem_pool_bytes(C.byref(cfg()))
    assert plain > 0
    # rotary table: 8 bytes x head_dim / 2 per position, plus the per-block original positions
    rope = lib.kvmem_pool_bytes(C.byref(cfg(rope_max_positions=4096, rope_theta=1.0e6)))
    assert rope - plain >= 4096 * 64 * 8 and rope - plain <= 4096 * 64 * 8 + 1024 * 4 + 1024
    in_block = lib.kvmem_pool_bytes(C.byref(cfg(rope_max_positions=4096, rope_theta=1.0e6, rope_in_block_keys=1)))
    assert in_block == rope                                        # a different content of the same pages
    assert lib.kvmem_pool_bytes(C.byref(cfg(rope_in_block_keys=1))) == 0 and b"rope_in_block_keys" in lib.kvmem_last_error()
    assert lib.kvmem_pool_bytes(C.byref(cfg(rope_max_positions=32, rope_theta=1.0e6, rope_in_block_keys=1))) == 0
    assert lib.kvmem_pool_bytes(C.byref(cfg(rope_max_positions=64, rope_theta=0.5))) == 0
    # FP8 repository: one byte per page element, the index stays bf16
    f8 = lib.kvmem_pool_bytes(C.byref(cfg(fp8_pages=1, fp8_k_scale=1.0, fp8_v_scale=0.5)))
    page_elems = 1024 * 2 * 8 * 64 * 128
    assert plain - f8 == page_elems                                # 2 bytes -> 1 byte per element
    for bad in (dict(fp8_pages=1, fp8_k_scale=0.0, fp8_v_scale=1.0), dict(fp8_pages=1, fp8_k_scale=1.0, fp8_v_scale=float("inf")),
                dict(fp8_pages=1, fp8_k_scale=1.0, fp8_v_scale=1.0, block_tokens=32),
                dict(fp8_pages=1, fp8_k_scale=1.0, fp8_v_scale=1.0, rope_max_positions=4096, rope_theta=1.0e6),
                dict(fp8_pages=2, fp8_k_scale=1.0, fp8_v_scale=1.0)):
        assert lib.kvmem_pool_bytes(C.byref(cfg(**bad))) == 0, bad
