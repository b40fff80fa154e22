"""Small conveniences on top of the binding: a context holder, tensor
conversion between bf16 bit patterns (numpy) and torch CUDA tensors, and
read-back of the segment tables.  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def bits_to_tensor(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 CPU tensor sharing the memory."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)


def bits_to_device(bits: np.ndarray, device="cuda:0") -> torch.Tensor:
    return bits_to_tensor(bits).to(device)


def device_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class Context:
    """Owns a ba_ctx.  One per stream."""

    def __init__(self, n_q_heads, n_kv_heads, head_dim, rope_theta, rope_layout=B.BA_ROPE_ADJACENT,
                 softmax_scale=0.0, device=0, max_blocks=4096, max_q_rows=1 << 20):
        self.cfg = B.ba_config(n_q_heads, n_kv_heads, head_dim, rope_layout, float(rope_theta),
                               float(softmax_scale), 0)
        self.device = device
        ws = B.ba_workspace_bytes(self.cfg, max_blocks, max_q_rows)
        self.ctx = B.ba_create(self.cfg, device, ws)

    @classmethod
    def for_workload(cls, w, **kw):
        return cls(w.n_q_heads, w.n_kv_heads, w.head_dim, w.rope_theta, **kw)

    def close(self):
        if getattr(self, "ctx", None) is not None:
            B.ba_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def segment(self, block_lens, seq_nblocks, mode, n_tokens=None, stream=None):
        """Returns (ba_segments, table buffer).  Keep the buffer alive while the tables are used."""
        if isinstance(block_lens, torch.Tensor):
            n_blocks, batch = block_lens.numel(), seq_nblocks.numel()
            assert n_tokens is not None
        else:
            block_lens = np.ascontiguousarray(block_lens, dtype=np.int32)
            seq_nblocks = np.ascontiguousarray(seq_nblocks, dtype=np.int32)
            n_blocks, batch = len(block_lens), len(seq_nblocks)
            if n_tokens is None:
                n_tokens = int(block_lens.sum())
        nbytes = B.ba_segments_bytes(batch, n_blocks, n_tokens)
        buf = torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{self.device}")
        seg = B.ba_segment(self.ctx, block_lens, seq_nblocks, batch, n_blocks, n_tokens, mode, buf, stream)
        return seg, buf

    def device_status(self) -> int:
        return B.ba_last_device_status(self.ctx)

    def launches(self) -> int:
        return B.ba_launch_count(self.ctx)

    def last_attend_shape(self) -> dict:
        return B.ba_last_attend_shape(self.ctx)


_TABLE_SIZES = {
    "cu_seq": ("batch", 1), "cu_cache_seq": ("batch", 1), "cu_final_seq": ("batch", 1),
    "cu_seq_block": ("batch", 1), "cu_block": ("n_blocks", 1), "block_delta": ("n_blocks", 0),
    "block_seq": ("n_blocks", 0), "block_kv_begin": ("n_blocks", 0), "block_part_off": ("n_blocks", 0),
    "cache_block": ("n_cached_blocks", 0), "cache_cu": ("n_cached_blocks", 1),
    "cache_delta": ("n_cached_blocks", 0), "tok_block": ("n_tokens", 0), "tok_pos": ("n_tokens", 0),
    "tok_pos_local": ("n_tokens", 0), "cu_qtile": ("n_blocks", 1), "cu_ftile": ("batch", 1), "cache_tile_cu": ("n_cached_blocks", 1),
    "cu_ktile": ("n_blocks", 1),
}


def read_tables(seg: B.ba_segments, buf: torch.Tensor) -> dict:
    """Copy the tables back to the host as numpy arrays (after synchronising)."""
    torch.cuda.synchronize(buf.device)
    host = buf.cpu().numpy()
    base = buf.data_ptr()
    out = {}
    for name, (dim, extra) in _TABLE_SIZES.items():
        n = getattr(seg, dim) + extra
        off = getattr(seg, name) - base
        out[name] = host[off:off + 4 * n].view(np.int32).copy()
    off = seg.block_is_final - base
    out["block_is_final"] = host[off:off + seg.n_blocks].copy()
    off = seg.totals - base
    out["totals"] = host[off:off + 32].view(np.int32).copy()
    return out
