"""Counter-based synthetic workspaces: the same bytes on CPU and on a GPU.

Every bulk value is a pure function of (seed, stream, element index): a 32-bit integer
mix of the index picks one of 65,536 equiprobable N(0,1) quantiles from a table that is
always computed on the CPU.  Only integer ops, a table lookup and one fp32 multiply-add
touch the data on the device, so a tensor generated with ``device="cuda"`` is bit-identical
to the one generated with ``device="cpu"``, and chunks can be generated independently.

Recipe (shapes follow the five benchmark configurations):
  * keys and values: i.i.d. N(0,1), rounded once to bf16, token-major ``[tokens][L][G][d]``;
  * per (session, layer, KV head) a unit vector ``u``; a *planted* block has every key
    shifted by ``a * u`` before the bf16 rounding (``a`` in units of sigma);
  * queries: ``z + sqrt(d) * u[g(h)]`` with ``z ~ N(0, I)``, so a planted block's mean key
    scores about ``a`` logits above the background;
  * planted block ids: the ``n_planted`` blocks with the smallest hash, in hash order
    (that order is the Zipf rank when the shift decays with rank);
  * page tables: identity, or one seeded permutation of all physical pages dealt out to
    the sessions.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Tuple

import torch

_M32 = 0xFFFFFFFF
_TABLE_BITS = 16
_CHUNK_CPU = 1 << 18   # elements hashed per pass: cache-sized on the host ...
_CHUNK_GPU = 1 << 24   # ... launch-amortising on a GPU; the values do not depend on it

# stream ids (mixed into the hash key)
_S_K, _S_V, _S_U, _S_Q, _S_PLANT, _S_PAGES = 1, 2, 3, 4, 5, 6


@dataclass(frozen=True)
class WorkloadSpec:
    name: str
    n_sessions: int
    n_blocks: int            # NB: logical blocks per session
    block_tokens: int        # B_blk
    n_q_tokens: int          # M
    n_q_heads: int           # H
    n_kv_heads: int          # G
    head_dim: int            # d
    n_layers: int            # L
    n_planted: int           # planted blocks per session
    shift: float             # planted shift a (sigma units) for rank 1
    zipf_s: float            # 0: constant shift; else a_rho = shift - zipf_s * ln(rho)
    budget_blocks: int       # k requested per session
    max_view_tokens: int     # B_a = min(B_model, B_gpu)
    seed: int
    permute_pages: bool
    attend: bool             # False for the chunked-scoring configuration
    n_query_sets: int = 16

    @property
    def tokens(self) -> int:
        return self.n_blocks * self.block_tokens

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def with_(self, **kw) -> "WorkloadSpec":
        return replace(self, **kw)


def _spec(name, ns, nb, m, planted, shift, zipf, k, seed, permute=False, attend=True):
    return WorkloadSpec(name=name, n_sessions=ns, n_blocks=nb, block_tokens=64, n_q_tokens=m,
                        n_q_heads=32, n_kv_heads=8, head_dim=128, n_layers=1, n_planted=planted,
                        shift=shift, zipf_s=zipf, budget_blocks=k, max_view_tokens=262144,
                        seed=seed, permute_pages=permute, attend=attend)


CONFIGS: Dict[str, WorkloadSpec] = {
    # 16,384-token history, 1 query token, 8 planted blocks at +3 sigma, k = 32
    "tiny": _spec("tiny", 1, 256, 1, 8, 3.0, 0.0, 32, seed=0),
    # 128K history, 1 + 3 MTP query tokens, 64 planted, k = 512
    "128k": _spec("128k", 1, 2048, 4, 64, 3.0, 0.0, 512, seed=1),
    # 1M history, Zipf(1.1)-weighted relevance over 1,024 planted blocks, k = 4,096 (window bound)
    "1m": _spec("1m", 1, 16384, 4, 1024, 8.0, 1.1, 4096, seed=2),
    # 8 independent 256K sessions, permuted physical pages, k = 1,024 each
    "batch8": _spec("batch8", 8, 4096, 1, 32, 3.0, 0.0, 1024, seed=3, permute=True),
    # 512-token chunk against the 1M index: score + select + materialize only
    "chunk512": _spec("chunk512", 1, 16384, 512, 1024, 3.0, 0.0, 4096, seed=4, attend=False),
}
# The paper's workspace-scaling experiment (its table of retrieval latency against workspace size): 32-token
# blocks, a 128-token query, a 64K-token execution view; the history is swept from 256K to 10M tokens
# (8,192 to 312,500 blocks) by the benchmark.  Base size 1M tokens.  Score + select + materialize only.
CONFIGS["table4"] = replace(_spec("table4", 1, 32768, 128, 256, 3.0, 0.0, 2048, seed=5, attend=False),
                            block_tokens=32, n_query_sets=4)


# ----------------------------------------------------------------------------- hashing

def _mix32(x: torch.Tensor) -> torch.Tensor:
    """Bijective 32-bit integer mix on int64 tensors holding values in [0, 2^32)."""
    x = (((x >> 16) ^ x) * 0x45D9F3B) & _M32
    x = (((x >> 16) ^ x) * 0x45D9F3B) & _M32
    return (x >> 16) ^ x


def _key(seed: int, stream: int, a: int = 0, b: int = 0) -> Tuple[int, int]:
    """Two 32-bit keys from small integers (pure Python, no tensors)."""
    def mix(v: int) -> int:
        v &= _M32
        v = (((v >> 16) ^ v) * 0x45D9F3B) & _M32
        v = (((v >> 16) ^ v) * 0x45D9F3B) & _M32
        return (v >> 16) ^ v
    k1 = mix(mix(mix(mix(seed + 0x9E3779B9) ^ stream) + a * 0x85EBCA6B) ^ (b * 0xC2B2AE35))
    k2 = mix(k1 ^ 0x27D4EB2F)
    return k1, k2


def _hash32(counter: torch.Tensor, key: Tuple[int, int]) -> torch.Tensor:
    lo = counter & _M32
    hi = counter >> 32
    x = lo ^ ((hi * 0x9E3779B1) & _M32) ^ key[0]
    x = _mix32(x)
    x = _mix32((x + key[1]) & _M32)
    return x


_table_cache: Dict[str, torch.Tensor] = {}


def _normal_table(device) -> torch.Tensor:
    """65,536 equiprobable N(0,1) quantile mid-points as fp32; always computed on the CPU."""
    dev = str(device)
    if "cpu" not in _table_cache:
        n = 1 << _TABLE_BITS
        p = (torch.arange(n, dtype=torch.float64) + 0.5) / n
        _table_cache["cpu"] = torch.special.ndtri(p).to(torch.float32)
    if dev not in _table_cache:
        _table_cache[dev] = _table_cache["cpu"].to(device)
    return _table_cache[dev]


def _normal(start: int, count: int, key: Tuple[int, int], device) -> torch.Tensor:
    """fp32 N(0,1) draws for element indices [start, start + count)."""
    table = _normal_table(device)
    out = torch.empty(count, dtype=torch.float32, device=device)
    chunk = _CHUNK_CPU if str(device) == "cpu" else _CHUNK_GPU
    for off in range(0, count, chunk):
        n = min(chunk, count - off)
        c = torch.arange(start + off, start + off + n, dtype=torch.int64, device=device)
        h = _hash32(c, key)
        out[off:off + n] = table[h >> (32 - _TABLE_BITS)]
    return out


# ----------------------------------------------------------------------------- recipe

def planted_directions(spec: WorkloadSpec, session: int) -> torch.Tensor:
    """Unit vectors u[l][g][:] (fp32, CPU)."""
    n = spec.n_layers * spec.n_kv_heads * spec.head_dim
    z = _normal(0, n, _key(spec.seed, _S_U, session), "cpu").to(torch.float64)
    z = z.view(spec.n_layers, spec.n_kv_heads, spec.head_dim)
    return (z / z.norm(dim=-1, keepdim=True)).to(torch.float32)


def planted_blocks(spec: WorkloadSpec, session: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """(ids int64 [n_planted] in rank order, shift fp32 [n_planted]) on the CPU."""
    if spec.n_planted == 0:
        return torch.empty(0, dtype=torch.int64), torch.empty(0, dtype=torch.float32)
    b = torch.arange(spec.n_blocks, dtype=torch.int64)
    h = _hash32(b, _key(spec.seed, _S_PLANT, session))
    ids = torch.argsort(h * spec.n_blocks + b)[: spec.n_planted]  # distinct sort keys
    rho = torch.arange(1, spec.n_planted + 1, dtype=torch.float64)
    a = torch.full_like(rho, spec.shift) - spec.zipf_s * torch.log(rho)
    return ids, a.to(torch.float32)


def kv_blocks(spec: WorkloadSpec, session: int, b0: int, b1: int, device="cpu"
              ) -> Tuple[torch.Tensor, torch.Tensor]:
    """K and V of logical blocks [b0, b1) of one session: bf16 ``[(b1-b0)*B][L][G][d]``."""
    B, L, G, d = spec.block_tokens, spec.n_layers, spec.n_kv_heads, spec.head_dim
    per_tok = L * G * d
    n_tok = (b1 - b0) * B
    start = b0 * B * per_tok
    k = _normal(start, n_tok * per_tok, _key(spec.seed, _S_K, session), device).view(n_tok, L, G, d)
    v = _normal(start, n_tok * per_tok, _key(spec.seed, _S_V, session), device).view(n_tok, L, G, d)
    ids, a = planted_blocks(spec, session)
    amp = torch.zeros(spec.n_blocks, dtype=torch.float32)
    amp[ids] = a
    amp = amp[b0:b1]
    if bool((amp != 0).any()):
        u = planted_directions(spec, session).to(device)
        amp_tok = amp.to(device).repeat_interleave(B).view(n_tok, 1, 1, 1)
        shift = amp_tok * u.view(1, L, G, d)   # fp32 multiply ...
        k = k + shift                           # ... then fp32 add: no fused op, same bits everywhere
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def make_queries(spec: WorkloadSpec, qset: int = 0, drift: float = 1.0) -> torch.Tensor:
    """Query set ``qset``: bf16 ``[n_sessions][M][L][H][d]`` on the CPU.

    ``drift`` < 1 models consecutive agent steps whose queries stay close: the free part of query set
    ``qset`` is sqrt(1 - drift^2) * (that of set 0) + drift * (its own), so consecutive selections overlap
    more the smaller ``drift`` is; 1.0 (default) gives independent query sets."""
    M, L, H, d, r = spec.n_q_tokens, spec.n_layers, spec.n_q_heads, spec.head_dim, spec.group
    out = torch.empty(spec.n_sessions, M, L, H, d, dtype=torch.float32)
    for s in range(spec.n_sessions):
        z = _normal(0, M * L * H * d, _key(spec.seed, _S_Q, s, qset), "cpu").view(M, L, H, d)
        if drift < 1.0 and qset != 0:
            z0 = _normal(0, M * L * H * d, _key(spec.seed, _S_Q, s, 0), "cpu").view(M, L, H, d)
            z = math.sqrt(1.0 - drift * drift) * z0 + drift * z
        u = planted_directions(spec, s)                       # [L][G][d]
        u_h = u.repeat_interleave(r, dim=1)                   # query head h looks at KV head h // r
        out[s] = z + math.sqrt(d) * u_h.view(1, L, H, d)
    return out.to(torch.bfloat16)


def page_table(spec: WorkloadSpec) -> torch.Tensor:
    """Physical page of every logical block: int32 ``[n_sessions][NB]`` on the CPU."""
    total = spec.n_sessions * spec.n_blocks
    if not spec.permute_pages:
        return torch.arange(total, dtype=torch.int32).view(spec.n_sessions, spec.n_blocks)
    p = torch.arange(total, dtype=torch.int64)
    h = _hash32(p, _key(spec.seed, _S_PAGES))
    perm = torch.argsort(h * total + p)
    return perm.to(torch.int32).view(spec.n_sessions, spec.n_blocks)


def select_params(spec: WorkloadSpec) -> Dict[str, int]:
    return dict(budget_blocks=spec.budget_blocks, max_view_tokens=spec.max_view_tokens,
                mandatory_tokens=0, n_sink_blocks=0, n_recent_blocks=0)
