"""Seeded synthetic inputs for the Block-attention prefilling hot path.

This module is the only code shared by the CUDA path and the CPU oracle.  It
holds no arithmetic of the method itself: it draws block lengths, pool indices
and i.i.d. N(0,1) values from numpy's PCG64 generator and converts them to
bfloat16 bit patterns (round-to-nearest-even).  RoPE is *not* applied here: an
isotropic Gaussian pair stays an isotropic Gaussian pair under any rotation, so
"K drawn N(0,1) and stored rotated at cache positions 0..L-1" has the same
distribution as K drawn N(0,1) directly, and the drawn array *is* the cached K.

The five workloads mirror RAG prompt shapes (Section 2.2, Section 3.6 of the
paper: 5-30 retrieved passages, a short user query as the final block).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

BA_MODE_BLOCK = 0
BA_MODE_FULL = 1


# ----------------------------------------------------------------------------
# bfloat16 <-> float conversions on bit patterns (format conversion only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bits (uint16), round-to-nearest-even; NaN kept quiet."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def normal_bf16(seed: int, shape) -> np.ndarray:
    """i.i.d. N(0,1) drawn in float32 from PCG64(seed), rounded once to bf16 bits."""
    rng = np.random.default_rng(seed)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    chunk = 1 << 24
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        out[lo:hi] = f32_to_bf16_bits(rng.standard_normal(hi - lo, dtype=np.float32))
    return out.reshape(shape)


# ----------------------------------------------------------------------------
# Workload descriptions
# ----------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rope_theta: float
    # ragged structure: block lengths in prompt order, blocks per sequence
    block_lens: List[int]
    seq_nblocks: List[int]
    seed: int
    n_layers: int = 1
    # shared-pool serving (config 5): lengths of the pool's blocks and, per
    # request, the pool indices of its cached blocks (in prompt order)
    pool_lens: Optional[List[int]] = None
    request_pool_idx: Optional[List[List[int]]] = None
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return len(self.seq_nblocks)

    @property
    def n_tokens(self) -> int:
        return int(sum(self.block_lens))

    @property
    def n_blocks(self) -> int:
        return len(self.block_lens)

    def final_lens(self) -> List[int]:
        out, b = [], 0
        for nb in self.seq_nblocks:
            out.append(self.block_lens[b + nb - 1])
            b += nb
        return out

    def cached_lens_per_seq(self) -> List[List[int]]:
        out, b = [], 0
        for nb in self.seq_nblocks:
            out.append(list(self.block_lens[b:b + nb - 1]))
            b += nb
        return out


def _ragged_to_total(rng: np.random.Generator, total: int, lo: int, hi: int) -> List[int]:
    """Draw lengths uniform in [lo, hi] until they reach `total`; the last draw
    is truncated so the sum is exactly `total` (it may fall below `lo`)."""
    lens, s = [], 0
    while s < total:
        l = int(rng.integers(lo, hi + 1))
        l = min(l, total - s)
        lens.append(l)
        s += l
    return lens


def config1() -> Workload:
    return Workload("cfg1_tiny", 4, 2, 64, 10000.0, [64, 64, 64, 64, 32], [5], seed=1001,
                    notes="4 cached blocks of 64 + final 32; block and full mode")


def config2() -> Workload:
    rng = np.random.default_rng(2002)
    lens = [int(x) for x in rng.integers(128, 385, size=10)] + [64]
    return Workload("cfg2_rag", 32, 8, 128, 500000.0, lens, [11], seed=2002,
                    notes="10 passages U[128,384] + 64-token query")


def config3(n_layers: int = 32) -> Workload:
    return Workload("cfg3_32k", 32, 8, 128, 500000.0, [1000] * 32 + [768], [33], seed=3003,
                    n_layers=n_layers, notes="32 x 1000 cached + final 768 (32768 tokens)")


def config4(batch: int = 8, seq_len: int = 16384) -> Workload:
    rng = np.random.default_rng(4004)
    lens, nb = [], []
    for _ in range(batch):
        l = _ragged_to_total(rng, seq_len, 64, 2048)
        lens += l
        nb.append(len(l))
    return Workload("cfg4_cold_prefill", 32, 8, 128, 500000.0, lens, nb, seed=4004,
                    notes="batch x seq_len tokens, ragged blocks U[64,2048], last block final")


def config5(n_requests: int = 16, pool_blocks: int = 512, per_request: int = 20,
            final_len: int = 128) -> Workload:
    rng = np.random.default_rng(5005)
    pool_lens = [int(x) for x in rng.integers(50, 501, size=pool_blocks)]
    req_idx = [[int(x) for x in rng.integers(0, pool_blocks, size=per_request)]
               for _ in range(n_requests)]
    lens, nb = [], []
    for r in range(n_requests):
        lens += [pool_lens[i] for i in req_idx[r]] + [final_len]
        nb.append(per_request + 1)
    return Workload("cfg5_pool_serving", 32, 8, 128, 500000.0, lens, nb, seed=5005,
                    pool_lens=pool_lens, request_pool_idx=req_idx,
                    notes="pool of cached blocks U[50,500]; 20 indices per request; final 128")


def random_ragged(seed: int, batch: int, max_blocks: int, max_len: int, n_q_heads: int,
                  n_kv_heads: int, head_dim: int, rope_theta: float = 10000.0,
                  edge_lens=(1, 63, 64, 65, 127, 128, 129)) -> Workload:
    """Property-test layouts: random block counts and lengths with tile-edge sizes mixed in."""
    rng = np.random.default_rng(seed)
    lens, nb = [], []
    for _ in range(batch):
        n = int(rng.integers(1, max_blocks + 1))
        for _ in range(n):
            if rng.random() < 0.4:
                l = int(rng.choice([e for e in edge_lens if e <= max_len] or [1]))
            else:
                l = int(rng.integers(1, max_len + 1))
            lens.append(l)
        nb.append(n)
    return Workload(f"ragged_{seed}", n_q_heads, n_kv_heads, head_dim, rope_theta, lens, nb,
                    seed=seed)


# ----------------------------------------------------------------------------
# Tensors for a workload
# ----------------------------------------------------------------------------
def prefill_inputs(w: Workload, layer: int = 0):
    """Q [T,Hq,D], K,V [T,Hkv,D] bf16 bits for a packed ragged prefill."""
    T = w.n_tokens
    s = w.seed * 1000 + layer * 7
    q = normal_bf16(s + 1, (T, w.n_q_heads, w.head_dim))
    k = normal_bf16(s + 2, (T, w.n_kv_heads, w.head_dim))
    v = normal_bf16(s + 3, (T, w.n_kv_heads, w.head_dim))
    return q, k, v


def warm_inputs(w: Workload, layer: int = 0):
    """Inputs of the warm-cache path.

    Returns a dict with bf16-bit arrays:
      k_cache, v_cache : [T_c, Hkv, D]  cached blocks, packed in prompt order with
                         the final blocks left out; K holds cache-time positions
      q_f, k_f, v_f    : [T_f, H, D]    final blocks packed over the batch
    When the workload has a pool, k_pool/v_pool [T_pool,Hkv,D] and src_off[Bc]
    (first pool row of each cached block) are returned instead of k_cache/v_cache.
    """
    s = w.seed * 1000 + layer * 7
    Tf = sum(w.final_lens())
    out = {
        "q_f": normal_bf16(s + 11, (Tf, w.n_q_heads, w.head_dim)),
        "k_f": normal_bf16(s + 12, (Tf, w.n_kv_heads, w.head_dim)),
        "v_f": normal_bf16(s + 13, (Tf, w.n_kv_heads, w.head_dim)),
    }
    if w.pool_lens is None:
        Tc = w.n_tokens - Tf
        out["k_cache"] = normal_bf16(s + 14, (Tc, w.n_kv_heads, w.head_dim))
        out["v_cache"] = normal_bf16(s + 15, (Tc, w.n_kv_heads, w.head_dim))
    else:
        Tp = int(sum(w.pool_lens))
        out["k_pool"] = normal_bf16(s + 16, (Tp, w.n_kv_heads, w.head_dim))
        out["v_pool"] = normal_bf16(s + 17, (Tp, w.n_kv_heads, w.head_dim))
        pool_off = np.concatenate([[0], np.cumsum(w.pool_lens)]).astype(np.int64)
        src = [pool_off[i] for req in w.request_pool_idx for i in req]
        out["src_off"] = np.asarray(src, dtype=np.int32)
    return out


def scatter_into_pages(packed: np.ndarray, cache_lens, page_rows: int, seed: int, spare_pages: int = 3):
    """Lays packed cached rows [T_c, ...] (uint16 bf16 bits) out as a pool of fixed-size pages: every
    cached block gets ceil(L / page_rows) pages, pages are numbered by a seeded permutation (with a few
    spare pages in between), rows of a last page beyond the block's end are filled with N(0,1) noise.
    Returns (pool [n_pages * page_rows, ...], page_cu int32 [n_blocks + 1], page_idx int32, n_pages)."""
    rng = np.random.default_rng(seed)
    counts = [(int(L) + page_rows - 1) // page_rows for L in cache_lens]
    page_cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    n_used = int(page_cu[-1])
    n_pages = n_used + spare_pages
    page_idx = rng.permutation(n_pages)[:n_used].astype(np.int32)
    pool = normal_bf16(seed + 1, (n_pages * page_rows,) + tuple(packed.shape[1:]))
    r = 0
    for c, L in enumerate(cache_lens):
        for k in range(counts[c]):
            n = min(page_rows, int(L) - k * page_rows)
            g = int(page_idx[page_cu[c] + k])
            pool[g * page_rows:g * page_rows + n] = packed[r:r + n]
            r += n
    return pool, page_cu, page_idx, n_pages
