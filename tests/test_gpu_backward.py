"""Backward pass of attention under the Block-attention mask (Section 2.4) against the fp64 oracle.

Tolerance.  The kernels recompute P from the stored log-sum-exp and round P and dS to bf16 before the
tensor-core products (relative rounding error 2^-9 each), inputs are bf16 and sums are fp32: gradients
written as fp32 are required to agree with the oracle to a relative Frobenius error of 1e-2 per tensor
and every element to within 2e-2 of the tensor's largest magnitude; bf16 gradients add their own
rounding (same bounds).  The forward output and log-sum-exp handed to the backward call are the CUDA
forward's own, as in training.
"""
import numpy as np
import pytest
import torch

from oracle import block_attention as ob
from paper_2409_15355_b200 import binding as B
from paper_2409_15355_b200 import runtime as R
from paper_2409_15355_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_forward_backward(w, mode, grad_dtype=B.BA_OUT_F32, seed_extra=0):
    c = R.Context.for_workload(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, mode)
    qb, kb, vb = W.prefill_inputs(w)
    gb = W.normal_bf16(w.seed * 1000 + 77 + seed_extra, (w.n_tokens, w.n_q_heads, w.head_dim))
    q, k, v, g = (R.bits_to_device(x) for x in (qb, kb, vb, gb))
    T = w.n_tokens
    o = torch.empty(T, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(T, w.n_q_heads, dtype=torch.float32, device="cuda")
    B.ba_block_prefill(c.ctx, q, k, v, o, lse, seg, mode, B.BA_OUT_BF16)
    dt = torch.float32 if grad_dtype == B.BA_OUT_F32 else torch.bfloat16
    dq = torch.full((T, w.n_q_heads, w.head_dim), float("nan"), dtype=dt, device="cuda")
    dk = torch.full((T, w.n_kv_heads, w.head_dim), float("nan"), dtype=dt, device="cuda")
    dv = torch.full_like(dk, float("nan"))
    B.ba_block_prefill_bwd(c.ctx, q, k, v, o, lse, g, dq, dk, dv, seg, mode, grad_dtype)
    assert c.device_status() == B.BA_OK
    c.close()
    f64 = W.bf16_bits_to_f64
    return (dq.float().cpu().numpy(), dk.float().cpu().numpy(), dv.float().cpu().numpy(),
            f64(qb), f64(kb), f64(vb), f64(gb))


def check_grad(name, got, ref, rel=1e-2, elem=2e-2):
    got = np.asarray(got, dtype=np.float64)
    assert np.isfinite(got).all(), name
    if np.abs(ref).max() < 1e-9:        # an identically zero gradient (a row that sees one key): fp32 cancellation noise only
        assert np.abs(got).max() <= 1e-5, f"{name}: {np.abs(got).max()} where the gradient vanishes"
        return
    fro = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert fro <= rel, f"{name}: relative Frobenius {fro}"
    assert np.abs(got - ref).max() <= elem * np.abs(ref).max(), f"{name}: max-abs {np.abs(got - ref).max()} of {np.abs(ref).max()}"


BWD_CASES = [W.config1(), W.config2(), W.random_ragged(61, 3, 5, 300, 4, 2, 64), W.random_ragged(62, 2, 4, 300, 8, 2, 128),
             W.random_ragged(63, 3, 4, 200, 8, 1, 128), W.random_ragged(64, 3, 4, 200, 6, 2, 64),
             W.Workload("one_token", 4, 2, 64, 1e4, [1], [1], seed=65),
             W.Workload("single_block", 4, 4, 128, 1e4, [333], [1], seed=66)]


@pytest.mark.parametrize("w", BWD_CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("mode", [B.BA_MODE_BLOCK, B.BA_MODE_FULL])
def test_backward_parity(w, mode):
    dq, dk, dv, q, k, v, g = run_forward_backward(w, mode)
    rq, rk, rv = ob.block_prefill_backward(q, k, v, g, w.block_lens, w.seq_nblocks, mode)
    check_grad("dq", dq, rq); check_grad("dk", dk, rk); check_grad("dv", dv, rv)


def test_backward_bf16_gradients_and_bit_stability():
    w = W.config2()
    a = run_forward_backward(w, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    b = run_forward_backward(w, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    rq, rk, rv = ob.block_prefill_backward(a[3], a[4], a[5], a[6], w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    check_grad("dq", a[0], rq); check_grad("dk", a[1], rk); check_grad("dv", a[2], rv)
    for x, y in zip(a[:3], b[:3]):
        assert np.array_equal(x, y)                      # no atomics: the same bits every run


def test_backward_llama_shape_two_ragged_sequences():
    rng = np.random.default_rng(71)
    lens, nbs = [], []
    for _ in range(2):
        l = W._ragged_to_total(rng, 2048, 64, 512)
        lens += l; nbs.append(len(l))
    w = W.Workload("bwd_llama_2x2048", 32, 8, 128, 5e5, lens, nbs, seed=71)
    dq, dk, dv, q, k, v, g = run_forward_backward(w, B.BA_MODE_BLOCK)
    rq, rk, rv = ob.block_prefill_backward(q, k, v, g, w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    check_grad("dq", dq, rq); check_grad("dk", dk, rk); check_grad("dv", dv, rv)


def test_backward_cold_batch_full_size_sampled_rows_and_invariants():
    """The cold ragged workload (8 x 16384 tokens) at full size: dQ of sampled rows against the oracle
    (a row's dQ needs only that row's softmax), and two identities that hold for any input: the rows of
    P sum to one, so summing dV over the keys of a sequence gives the sum of dO over its queries (per KV
    group); the rows of dS sum to zero, so dK sums to zero over the keys of a sequence."""
    w = W.config4()
    dq, dk, dv, q, k, v, g = run_forward_backward(w, B.BA_MODE_BLOCK)
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    rng = np.random.default_rng(4)
    rows = np.unique(np.concatenate([rng.integers(0, w.n_tokens, 96), t["cu_block"][:-1], t["cu_block"][1:] - 1]))
    cu_seq = t["cu_seq"]
    G = w.n_q_heads // w.n_kv_heads
    for s in range(w.batch):
        c0, c1 = int(cu_seq[s]), int(cu_seq[s + 1])
        sel = rows[(rows >= c0) & (rows < c1)]
        nb0 = sum(w.seq_nblocks[:s])
        lens = w.block_lens[nb0:nb0 + w.seq_nblocks[s]]
        m = ob.mask_rows(lens, [len(lens)], ob.MODE_BLOCK, sel - c0)
        rq, _, _ = ob.attention_rows_backward(q[sel], k[c0:c1], v[c0:c1], m, g[sel])
        check_grad(f"dq rows of sequence {s}", dq[sel], rq)
        want_dv = g[c0:c1].reshape(c1 - c0, w.n_kv_heads, G, w.head_dim).sum(axis=(0, 2))
        got_dv = dv[c0:c1].astype(np.float64).sum(axis=0)
        assert np.abs(got_dv - want_dv).max() <= 2e-2 * np.abs(want_dv).max() + 0.5
        got_dk = dk[c0:c1].astype(np.float64).sum(axis=0)
        assert np.abs(got_dk).max() <= 2e-3 * np.abs(dk[c0:c1]).sum(axis=0).max() + 0.05


def test_backward_rejects_missing_arguments():
    w = W.config1()
    c = R.Context.for_workload(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    q = torch.zeros(288, 4, 64, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(288, 2, 64, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(288, 4, dtype=torch.float32, device="cuda")
    with pytest.raises(B.BaError) as e:
        B.ba_block_prefill_bwd(c.ctx, q, kv, kv, q, None, q, q, kv, kv, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    assert e.value.status == B.BA_ERR_INVALID_ARG
    with pytest.raises(B.BaError):
        B.ba_block_prefill_bwd(c.ctx, q, kv, kv, q, lse, q, q, kv, kv, seg, B.BA_MODE_FULL, B.BA_OUT_BF16)
    small = B.ba_create(c.cfg, 0, 64 * 1024 + 1024)
    tb = torch.empty(B.ba_segments_bytes(1, 5, 288), dtype=torch.uint8, device="cuda")
    seg2 = B.ba_segment(small, np.asarray(w.block_lens, dtype=np.int32), np.asarray([5], dtype=np.int32), 1, 5, 288,
                        B.BA_MODE_BLOCK, tb)
    with pytest.raises(B.BaError) as e:
        B.ba_block_prefill_bwd(small, q, kv, kv, q, lse, q, q, kv, kv, seg2, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    assert e.value.status == B.BA_ERR_WORKSPACE
    B.ba_destroy(small)
    c.close()
