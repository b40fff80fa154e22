"""ba_reencode_k_noalloc: the re-encode for callers that may not allocate.

Some users of this library cannot call cudaMalloc: an inference server that
gave all device memory to its own pool when it started, or a request path that
must not hit the device-wide synchronisation an allocation implies.  They cannot
create a context (its workspace is allocated), so this entry point keeps its
angle table in an array built into the library.  The test drives it through the
C ABI twice in a row, with different prompts, and requires the same bytes the
context-based ba_reencode_k produces (and a correct rounding of the fp64 oracle's
rotation): the second call must not see anything the first one left in the shared table.  It runs last so that a failure here cannot
hide results of the other tests.
"""
import numpy as np
import pytest
import torch

from oracle import block_attention as ob
from paper_2409_15355_b200 import binding as B
from paper_2409_15355_b200 import runtime as R
from paper_2409_15355_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _both(w, layout):
    c = R.Context.for_workload(w, rope_layout=layout)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    x = W.warm_inputs(w)
    if w.pool_lens is None:
        src, off = R.bits_to_device(x["k_cache"]), None
    else:
        src, off = R.bits_to_device(x["k_pool"]), torch.from_numpy(x["src_off"]).cuda()
    Tc = w.n_tokens - sum(w.final_lens())
    want = torch.zeros(Tc, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    got = torch.zeros_like(want)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ba_reencode_k(c.ctx, src, off, src.shape[0], want, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    B.ba_reencode_k_noalloc(c.cfg, 0, src, off, src.shape[0], got, seg.cache_cu, seg.cache_delta,
                            seg.n_cached_blocks, Tc, status)
    torch.cuda.synchronize()
    assert c.device_status() == B.BA_OK and int(status.item()) == 0
    assert torch.equal(got, want)
    assert not torch.equal(got, src[:Tc]) or w.pool_lens is not None
    # and against the oracle directly: every key a correct rounding of the fp64 rotation
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    src64 = W.bf16_bits_to_f64(x["k_cache"] if w.pool_lens is None else x["k_pool"])
    ref = ob.reencode_blocks(src64, None if w.pool_lens is None else x["src_off"], t["cache_cu"], t["cache_delta"],
                             w.rope_theta, ob.ROPE_HALF if layout == B.BA_ROPE_HALF else ob.ROPE_ADJACENT)
    g = W.bf16_bits_to_f64(R.device_to_bits(got))
    assert (np.abs(g - ref) <= np.abs(ref) * 2.0 ** -8 * 1.01 + 1e-6).all()
    r = W.bf16_bits_to_f64(W.f32_to_bf16_bits(ref.astype(np.float32)))
    assert (g == r).mean() >= 0.995
    c.close()
    return seg.n_cached_blocks


def test_noalloc_matches_reencode_on_two_calls_in_a_row():
    n1 = _both(W.config2(), B.BA_ROPE_ADJACENT)
    # second call: other prompt, other deltas, fewer blocks than the table now holds, other pairing
    n2 = _both(W.config5(3, 40, 5, 16), B.BA_ROPE_HALF)
    assert n1 != n2
    _both(W.config1(), B.BA_ROPE_ADJACENT)


def test_noalloc_rejects_oversize_and_reports_bad_rows():
    w = W.config1()
    cfg = B.ba_config(w.n_q_heads, w.n_kv_heads, w.head_dim, 0, w.rope_theta, 0.0, 0)
    k = torch.zeros(256, 2, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(k)
    cu = torch.tensor([0, 64, 128, 192, 256], dtype=torch.int32, device="cuda")
    delta = torch.tensor([0, 64, 128, 192], dtype=torch.int32, device="cuda")
    with pytest.raises(B.BaError) as e:
        B.ba_reencode_k_noalloc(cfg, 0, k, None, 256, out, cu, delta, B.BA_NOALLOC_MAX_BLOCKS + 1, 256)
    assert e.value.status == B.BA_ERR_WORKSPACE
    off = torch.tensor([0, 64, 128, 250], dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ba_reencode_k_noalloc(cfg, 0, k, off, 256, out, cu, delta, 4, 256, status)
    B.ba_reencode_k_noalloc(cfg, 0, k, off, 256, out, cu, delta, 4, 256, None)   # silent variant must not fault
    torch.cuda.synchronize()
    assert int(status.item()) == B.BA_ERR_INVALID_ARG
