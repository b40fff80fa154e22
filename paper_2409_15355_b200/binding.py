"""ctypes binding of the C ABI declared in include/ba.h.

Argument marshalling only: every step of the path runs in the CUDA library.
Tensors are torch CUDA tensors (torch is used for device memory and streams);
their data pointers are handed to the library unchanged.  There is no CPU
fallback: loading fails loudly when the library is missing, and ba_create fails
when no sm_100 device is present.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

from . import build as _build

BA_OK = 0
BA_ERR_INVALID_ARG, BA_ERR_SHAPE, BA_ERR_UNSUPPORTED, BA_ERR_WORKSPACE, BA_ERR_CUDA, BA_ERR_TIMEOUT = range(1, 7)
BA_MODE_BLOCK, BA_MODE_FULL = 0, 1
BA_ROPE_ADJACENT, BA_ROPE_HALF = 0, 1
BA_OUT_BF16, BA_OUT_F32 = 0, 1

EXPORTS = [
    "ba_create", "ba_destroy", "ba_status_string", "ba_workspace_bytes", "ba_last_device_status",
    "ba_launch_count", "ba_segments_bytes", "ba_segment", "ba_reencode_k", "ba_block_prefill",
    "ba_final_attend", "ba_reencode_k_noalloc", "ba_selftest_wait_expiry", "ba_reencode_k_deferred", "ba_flush",
    "ba_final_attend_fused", "ba_reencode_k_paged", "ba_final_attend_paged", "ba_final_attend_fused_paged",
    "ba_block_prefill_bwd", "ba_last_attend_shape", "ba_plan_final_attend",
]
BA_NOALLOC_MAX_BLOCKS = 4096


class ba_config(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("rope_layout", C.c_int32), ("rope_theta", C.c_double), ("softmax_scale", C.c_float),
                ("reserved", C.c_int32)]


class ba_segments(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_blocks", C.c_int32), ("n_tokens", C.c_int32),
                ("n_cached_blocks", C.c_int32), ("mode", C.c_int32), ("q_tile_tokens", C.c_int32),
                ("n_prompt_items", C.c_int32), ("n_final_items", C.c_int32),
                ("final_key_tiles", C.c_int32 * 6)] + [
        (n, C.c_void_p) for n in (
            "cu_seq", "cu_cache_seq", "cu_final_seq", "cu_seq_block", "cu_block", "block_delta",
            "block_seq", "block_kv_begin", "block_part_off", "block_is_final", "cache_block",
            "cache_cu", "cache_delta", "tok_block", "tok_pos", "tok_pos_local", "cu_qtile",
            "cu_ftile", "cache_tile_cu", "cu_ktile", "totals", "cache_rope")]


class ba_page_table(C.Structure):
    _fields_ = [("page_rows", C.c_int32), ("n_pages", C.c_int32), ("page_cu", C.c_void_p), ("page_idx", C.c_void_p)]


def make_page_table(page_rows: int, n_pages: int, page_cu, page_idx) -> "ba_page_table":
    """page_cu / page_idx: torch int32 CUDA tensors (kept alive by the caller)."""
    return ba_page_table(page_rows, n_pages, _ptr(page_cu), _ptr(page_idx))


class BaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (ba_status {status})")


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """dlopen libba.so (building it first if its sources changed) and declare prototypes."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = os.environ.get("BA_LIBRARY") or _build.build()   # BA_LIBRARY: use this prebuilt library as it is
    if not os.path.exists(path):
        raise FileNotFoundError(f"CUDA library not found: {path}")
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    lib.ba_create.argtypes = [C.POINTER(vp), C.POINTER(ba_config), C.c_int, sz]
    lib.ba_destroy.argtypes = [vp]
    lib.ba_status_string.argtypes = [C.c_int]
    lib.ba_status_string.restype = C.c_char_p
    lib.ba_workspace_bytes.argtypes = [C.POINTER(ba_config), i32, i32, C.POINTER(sz)]
    lib.ba_last_device_status.argtypes = [vp]
    lib.ba_launch_count.argtypes = [vp]
    lib.ba_launch_count.restype = C.c_int64
    lib.ba_last_attend_shape.argtypes = [vp, C.POINTER(i32 * 4)]
    lib.ba_plan_final_attend.argtypes = [i32, i32, i32, i32, C.POINTER(i32 * 3), i32, C.POINTER(i32 * 3)]
    lib.ba_segments_bytes.argtypes = [i32, i32, i32, C.POINTER(sz)]
    lib.ba_segment.argtypes = [vp, vp, vp, i32, i32, i32, C.c_int, vp, sz, C.POINTER(ba_segments), vp]
    lib.ba_reencode_k.argtypes = [vp, vp, vp, i32, vp, vp, vp, i32, i32, vp]
    lib.ba_reencode_k_noalloc.argtypes = [C.POINTER(ba_config), C.c_int, vp, vp, i32, vp, vp, vp, i32, i32, vp, vp]
    lib.ba_selftest_wait_expiry.argtypes = [vp, vp]
    lib.ba_reencode_k_deferred.argtypes = [vp, vp, vp, i32, vp, vp, vp, i32, i32, vp]
    lib.ba_flush.argtypes = [vp, vp]
    lib.ba_block_prefill.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(ba_segments), C.c_int, C.c_int, vp]
    lib.ba_final_attend.argtypes = [vp, vp, vp, vp, i32, vp, vp, i32, vp, i32, vp, vp,
                                    C.POINTER(ba_segments), C.c_int, C.c_int, vp]
    lib.ba_final_attend_fused.argtypes = [vp, vp, vp, vp, i32, vp, vp, i32, vp, i32, vp, vp, vp,
                                          C.POINTER(ba_segments), C.c_int, C.c_int, vp]
    pt = C.POINTER(ba_page_table)
    lib.ba_reencode_k_paged.argtypes = [vp, vp, pt, vp, vp, vp, i32, i32, vp]
    lib.ba_final_attend_paged.argtypes = [vp, vp, vp, vp, i32, vp, i32, vp, pt, vp, vp,
                                          C.POINTER(ba_segments), C.c_int, C.c_int, vp]
    lib.ba_final_attend_fused_paged.argtypes = [vp, vp, vp, vp, i32, vp, vp, pt, i32, vp, vp, vp,
                                                C.POINTER(ba_segments), C.c_int, C.c_int, vp]
    lib.ba_block_prefill_bwd.argtypes = [vp] + [vp] * 9 + [C.POINTER(ba_segments), C.c_int, C.c_int, vp]
    for name in EXPORTS:
        # without argtypes ctypes would pass addresses as 32-bit ints
        if getattr(lib, name).argtypes is None:
            raise RuntimeError(f"{name}: prototype not declared")
        if name not in ("ba_status_string", "ba_launch_count"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().ba_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != BA_OK:
        raise BaError(status, where)


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array / raw address / None."""
    if t is None or isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        if not t.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return t.data_ptr()
    return t.ctypes.data  # numpy (host arrays of lengths)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


# ---------------------------------------------------------------------------
# Same names as the C entry points
# ---------------------------------------------------------------------------
def ba_workspace_bytes(cfg: ba_config, max_blocks: int, max_q_rows: int) -> int:
    out = C.c_size_t(0)
    _check(load_library().ba_workspace_bytes(C.byref(cfg), max_blocks, max_q_rows, C.byref(out)),
           "ba_workspace_bytes")
    return out.value


def ba_create(cfg: ba_config, device: int, workspace_bytes: int) -> C.c_void_p:
    ctx = C.c_void_p()
    _check(load_library().ba_create(C.byref(ctx), C.byref(cfg), device, workspace_bytes), "ba_create")
    return ctx


def ba_destroy(ctx) -> None:
    _check(load_library().ba_destroy(ctx), "ba_destroy")


def ba_last_device_status(ctx) -> int:
    return load_library().ba_last_device_status(ctx)


def ba_launch_count(ctx) -> int:
    return int(load_library().ba_launch_count(ctx))


def ba_last_attend_shape(ctx) -> dict:
    """Layout of the last attention launch: CTAs, partial results per row, balanced tails and their key tiles."""
    out = (C.c_int32 * 4)()
    _check(load_library().ba_last_attend_shape(ctx, C.byref(out)), "ba_last_attend_shape")
    return {"ctas": out[0], "partials": out[1], "balanced_tails": out[2], "tail_tiles": out[3]}


def ba_plan_final_attend(n_sms: int, n_pairs: int, n_head_chunks: int, avg_key_tiles: int, key_tiles,
                         max_partials: int) -> dict:
    """The planning step of ba_final_attend (host arithmetic only)."""
    kt = (C.c_int32 * 3)(*[int(v) for v in key_tiles])
    out = (C.c_int32 * 3)()
    _check(load_library().ba_plan_final_attend(n_sms, n_pairs, n_head_chunks, avg_key_tiles, C.byref(kt), max_partials,
                                               C.byref(out)), "ba_plan_final_attend")
    return {"partials": out[0], "balanced_tails": out[1], "tail_tiles": out[2]}


def ba_segments_bytes(batch: int, n_blocks: int, n_tokens: int) -> int:
    out = C.c_size_t(0)
    _check(load_library().ba_segments_bytes(batch, n_blocks, n_tokens, C.byref(out)), "ba_segments_bytes")
    return out.value


def ba_segment(ctx, block_lens, seq_nblocks, batch, n_blocks, n_tokens, mode, table_buf, stream=None):
    """block_lens / seq_nblocks: int32 numpy arrays (host) or torch CUDA tensors.
    table_buf: torch uint8 CUDA tensor of at least ba_segments_bytes() bytes.  Returns ba_segments."""
    seg = ba_segments()
    _check(load_library().ba_segment(ctx, _ptr(block_lens), _ptr(seq_nblocks), batch, n_blocks, n_tokens,
                                     mode, _ptr(table_buf), table_buf.numel() * table_buf.element_size(),
                                     C.byref(seg), _stream_ptr(stream)), "ba_segment")
    return seg


def ba_reencode_k(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, stream=None):
    """cu / delta / src_off: device addresses (ints, e.g. seg.cache_cu) or torch int32 CUDA tensors."""
    _check(load_library().ba_reencode_k(ctx, _ptr(k_src), _ptr(src_off), n_src_rows, _ptr(k_dst),
                                        _ptr(cu), _ptr(delta), n_blocks, n_rows, _stream_ptr(stream)),
           "ba_reencode_k")


def ba_reencode_k_deferred(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, stream=None):
    """Queues the re-encoding; it runs in the background of the next attention call on this context."""
    _check(load_library().ba_reencode_k_deferred(ctx, _ptr(k_src), _ptr(src_off), n_src_rows, _ptr(k_dst),
                                                 _ptr(cu), _ptr(delta), n_blocks, n_rows, _stream_ptr(stream)),
           "ba_reencode_k_deferred")


def ba_flush(ctx, stream=None) -> None:
    _check(load_library().ba_flush(ctx, _stream_ptr(stream)), "ba_flush")


def ba_reencode_k_noalloc(cfg, device, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows,
                          status_word=None, stream=None):
    """Context-free re-encode that allocates nothing (see include/ba.h); arguments as ba_reencode_k."""
    _check(load_library().ba_reencode_k_noalloc(C.byref(cfg), device, _ptr(k_src), _ptr(src_off), n_src_rows,
                                                _ptr(k_dst), _ptr(cu), _ptr(delta), n_blocks, n_rows,
                                                _ptr(status_word), _stream_ptr(stream)),
           "ba_reencode_k_noalloc")


def ba_selftest_wait_expiry(ctx, stream=None) -> None:
    _check(load_library().ba_selftest_wait_expiry(ctx, _stream_ptr(stream)), "ba_selftest_wait_expiry")


def ba_block_prefill(ctx, q, k, v, o, lse, seg, mode, out_dtype, stream=None):
    _check(load_library().ba_block_prefill(ctx, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                           C.byref(seg), mode, out_dtype, _stream_ptr(stream)),
           "ba_block_prefill")


def ba_final_attend_fused(ctx, q_f, k_f, v_f, n_final_rows, k_src, v_src, n_src_rows, src_off,
                          n_cache_rows, o, lse, seg, mode, out_dtype, stream=None, k_out=None):
    """k_out: optional bf16 tensor [n_cache_rows, n_kv_heads, head_dim] that receives the re-encoded keys."""
    _check(load_library().ba_final_attend_fused(ctx, _ptr(q_f), _ptr(k_f), _ptr(v_f), n_final_rows,
                                                _ptr(k_src), _ptr(v_src), n_src_rows, _ptr(src_off),
                                                n_cache_rows, _ptr(k_out), _ptr(o), _ptr(lse), C.byref(seg), mode,
                                                out_dtype, _stream_ptr(stream)), "ba_final_attend_fused")


def ba_final_attend(ctx, q_f, k_f, v_f, n_final_rows, k_cache, v_cache, n_cache_rows, v_src_off,
                    n_v_rows, o, lse, seg, mode, out_dtype, stream=None):
    _check(load_library().ba_final_attend(ctx, _ptr(q_f), _ptr(k_f), _ptr(v_f), n_final_rows,
                                          _ptr(k_cache), _ptr(v_cache), n_cache_rows, _ptr(v_src_off),
                                          n_v_rows, _ptr(o), _ptr(lse), C.byref(seg), mode, out_dtype,
                                          _stream_ptr(stream)), "ba_final_attend")


def ba_reencode_k_paged(ctx, k_pool, pages, k_dst, cu, delta, n_blocks, n_rows, stream=None):
    _check(load_library().ba_reencode_k_paged(ctx, _ptr(k_pool), C.byref(pages), _ptr(k_dst), _ptr(cu), _ptr(delta),
                                              n_blocks, n_rows, _stream_ptr(stream)), "ba_reencode_k_paged")


def ba_final_attend_paged(ctx, q_f, k_f, v_f, n_final_rows, k_cache, n_cache_rows, v_pool, pages, o, lse, seg,
                          mode, out_dtype, stream=None):
    _check(load_library().ba_final_attend_paged(ctx, _ptr(q_f), _ptr(k_f), _ptr(v_f), n_final_rows, _ptr(k_cache),
                                                n_cache_rows, _ptr(v_pool), C.byref(pages), _ptr(o), _ptr(lse),
                                                C.byref(seg), mode, out_dtype, _stream_ptr(stream)),
           "ba_final_attend_paged")


def ba_final_attend_fused_paged(ctx, q_f, k_f, v_f, n_final_rows, k_pool, v_pool, pages, n_cache_rows, o, lse, seg,
                                mode, out_dtype, stream=None, k_out=None):
    _check(load_library().ba_final_attend_fused_paged(ctx, _ptr(q_f), _ptr(k_f), _ptr(v_f), n_final_rows,
                                                      _ptr(k_pool), _ptr(v_pool), C.byref(pages), n_cache_rows,
                                                      _ptr(k_out), _ptr(o), _ptr(lse), C.byref(seg), mode, out_dtype,
                                                      _stream_ptr(stream)), "ba_final_attend_fused_paged")


def ba_block_prefill_bwd(ctx, q, k, v, o, lse, d_o, dq, dk, dv, seg, mode, grad_dtype, stream=None):
    _check(load_library().ba_block_prefill_bwd(ctx, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o),
                                               _ptr(dq), _ptr(dk), _ptr(dv), C.byref(seg), mode, grad_dtype,
                                               _stream_ptr(stream)), "ba_block_prefill_bwd")
