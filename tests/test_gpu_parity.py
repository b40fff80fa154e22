"""Parity of the CUDA path (through the C ABI) with the fp64 oracle on the same
seeded inputs.

Tolerances.  Integer tables: bit-exact.  Attention outputs written as fp32
(bf16 inputs, fp32 accumulation): max-abs <= 1e-2 and mean-abs <= 1e-3 against
the fp64 oracle, plus a relative Frobenius error <= 5e-3 and log-sum-exp within
2e-3 (the absolute bounds alone are loose once thousands of keys are averaged).
Outputs stored as bf16 are compared with the oracle rounded to bf16 under the
same absolute bounds, except that a difference of one bf16 ulp is accepted where
the ulp itself exceeds 1e-2 (|x| >= 2); their relative Frobenius error is taken
against the unrounded oracle and must also stay within 5e-3 (the store adds an
rms relative error of about 2^-8 / sqrt(3) = 2.3e-3 in quadrature to the
arithmetic's own; against a rounded reference an arithmetic error e far below one
ulp u would instead show up as sqrt(e u), which measures the grid, not the
kernel).  Re-encoded keys are bf16 by contract: each must lie
within half a bf16 ulp (plus 1e-6 of fp32 noise: a rotation can cancel to a tiny value) of the fp64 value, i.e. be a correct
rounding of it, and within one ulp of the oracle's own rounding.
"""
import numpy as np
import pytest
import torch

from oracle import block_attention as ob
from paper_2409_15355_b200 import binding as B
from paper_2409_15355_b200 import runtime as R
from paper_2409_15355_b200 import workloads as W

pytestmark = pytest.mark.gpu

TABLE_KEYS = ["cu_seq", "cu_cache_seq", "cu_final_seq", "cu_block", "block_delta", "block_seq",
              "block_kv_begin", "block_part_off", "block_is_final", "cache_block", "cache_cu",
              "cache_delta", "tok_block", "tok_pos", "tok_pos_local"]


def check_attention(o_gpu, o_ref, lse_gpu=None, lse_ref=None, rel=5e-3, bf16_store=False):
    """o_ref: the fp64 oracle, unrounded.  bf16_store: o_gpu was stored as bf16."""
    o_gpu = np.asarray(o_gpu, dtype=np.float64)
    assert np.isfinite(o_gpu).all()
    if bf16_store:
        # a bf16 store may land on the neighbouring bf16 value: one ulp, which exceeds 1e-2 once |x| >= 2
        r = round_bf16(o_ref)
        d = np.abs(o_gpu - r)
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(r), 1e-30))) - 7)
        assert (d <= np.maximum(1e-2, ulp)).all(), f"max-abs {d.max()}"
    else:
        d = np.abs(o_gpu - o_ref)
        assert d.max() <= 1e-2, f"max-abs {d.max()}"
    assert d.mean() <= 1e-3, f"mean-abs {d.mean()}"
    fro = np.linalg.norm(o_gpu - o_ref) / np.linalg.norm(o_ref)
    assert fro <= rel, f"relative Frobenius {fro}"
    if lse_gpu is not None:
        dl = np.abs(np.asarray(lse_gpu, dtype=np.float64) - lse_ref).max()
        assert dl <= 2e-3, f"lse {dl}"


def round_bf16(x64):
    return W.bf16_bits_to_f64(W.f32_to_bf16_bits(np.asarray(x64, dtype=np.float32)))


def check_reencoded(k_gpu_bits, k_ref64):
    g = W.bf16_bits_to_f64(k_gpu_bits)
    # a correct rounding of the fp64 value: within half a bf16 ulp (at most 2^-8 relative) + fp32 noise
    assert (np.abs(g - k_ref64) <= np.abs(k_ref64) * (2.0 ** -8) * 1.01 + 1e-6).all()
    r = round_bf16(k_ref64)
    d = np.abs(g - r)
    assert d.mean() <= 1e-3
    assert (d <= np.abs(r) * 2.0 ** -7 + 1e-6).all()         # at most one ulp from the oracle's rounding
    assert (g == r).mean() >= 0.995


def ctx_for(w, **kw):
    return R.Context.for_workload(w, **kw)


def dev(bits):
    return R.bits_to_device(bits)


# --------------------------------------------------------------------------- tables
def table_cases():
    return [W.config1(), W.config2(), W.config3(1), W.config4(), W.config5(),
            W.random_ragged(11, 5, 7, 300, 4, 2, 64), W.random_ragged(12, 40, 3, 50, 4, 2, 64),
            W.Workload("one_token", 4, 2, 64, 1e4, [1], [1], seed=1),
            W.Workload("many_seqs", 4, 2, 64, 1e4, [1] * 3000, [1] * 3000, seed=2),
            W.Workload("many_blocks", 4, 2, 64, 1e4, [3, 1, 2] * 1000, [3000], seed=3)]


@pytest.mark.parametrize("w", table_cases(), ids=lambda w: w.name)
@pytest.mark.parametrize("mode", [B.BA_MODE_BLOCK, B.BA_MODE_FULL])
def test_tables_bit_exact(w, mode):
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, mode)
    got = R.read_tables(seg, buf)
    assert c.device_status() == B.BA_OK
    ref = ob.segment_tables(w.block_lens, w.seq_nblocks, mode)
    for k in TABLE_KEYS:
        assert got[k].tolist() == ref[k].tolist(), k
    assert got["totals"][0] == ref["n_cached_tokens"] and got["totals"][1] == ref["n_final_tokens"]
    # host-side counts that size and balance the attention launches: work items, and the 128-key tiles the
    # items of the final blocks see (cached keys in one run per sequence / a fresh tile per cached block)
    tt = seg.q_tile_tokens
    assert seg.n_prompt_items == sum(-(-n // tt) for n in w.block_lens)
    packed, walked = [], []
    for cached, fin in zip(w.cached_lens_per_seq(), w.final_lens()):
        for r0 in range(0, fin, tt):
            own = -(-min(fin, r0 + tt) // 128)
            packed.append(-(-sum(cached) // 128) + own)
            walked.append(sum(-(-n // 128) for n in cached) + own)
    assert seg.n_final_items == len(packed)
    assert list(seg.final_key_tiles) == [sum(packed), min(packed), max(packed), sum(walked), min(walked), max(walked)]
    c.close()


def test_tables_from_device_lengths_and_bad_lengths():
    w = W.config2()
    c = ctx_for(w)
    lens = torch.tensor(w.block_lens, dtype=torch.int32, device="cuda")
    nb = torch.tensor(w.seq_nblocks, dtype=torch.int32, device="cuda")
    seg, buf = c.segment(lens, nb, B.BA_MODE_BLOCK, n_tokens=w.n_tokens)
    got = R.read_tables(seg, buf)
    ref = ob.segment_tables(w.block_lens, w.seq_nblocks)
    for k in TABLE_KEYS:
        assert got[k].tolist() == ref[k].tolist(), k
    assert c.device_status() == B.BA_OK
    # device-side lengths that do not add up: reported by the status word, nothing faults
    seg, buf = c.segment(lens, nb, B.BA_MODE_BLOCK, n_tokens=w.n_tokens + 5)
    assert c.device_status() == B.BA_ERR_INVALID_ARG
    assert c.device_status() == B.BA_OK          # cleared by the read
    bad = lens.clone(); bad[3] = 0
    seg, buf = c.segment(bad, nb, B.BA_MODE_BLOCK, n_tokens=w.n_tokens)
    assert c.device_status() == B.BA_ERR_INVALID_ARG
    # tables marked invalid: attention over them does nothing and does not fault
    q = torch.zeros(w.n_tokens, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(w.n_tokens, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    o = torch.full_like(q, 7.0)
    B.ba_block_prefill(c.ctx, q, kv, kv, o, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    torch.cuda.synchronize()
    assert (o == 7.0).all()
    # host-side lengths are rejected before any launch
    with pytest.raises(B.BaError) as e:
        c.segment([3, 0, 2], [3], B.BA_MODE_BLOCK, n_tokens=5)
    assert e.value.status == B.BA_ERR_INVALID_ARG
    with pytest.raises(B.BaError):
        c.segment([3, 1, 2], [2], B.BA_MODE_BLOCK)
    c.close()


# --------------------------------------------------------------------------- re-encode
def reencode_case(w, layout=B.BA_ROPE_ADJACENT, layer=0):
    c = ctx_for(w, rope_layout=layout)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    x = W.warm_inputs(w, layer)
    Tc = t["n_cached_tokens"]
    if w.pool_lens is None:
        src, off, off_np = dev(x["k_cache"]), None, None
        src_np = x["k_cache"]
    else:
        src, off_np = dev(x["k_pool"]), x["src_off"]
        off = torch.from_numpy(off_np).cuda()
        src_np = x["k_pool"]
    dst = torch.empty(Tc, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    B.ba_reencode_k(c.ctx, src, off, src.shape[0], dst, seg.cache_cu, seg.cache_delta,
                    seg.n_cached_blocks, Tc)
    assert c.device_status() == B.BA_OK
    ref = ob.reencode_blocks(W.bf16_bits_to_f64(src_np), off_np, t["cache_cu"], t["cache_delta"],
                             w.rope_theta, layout)
    return c, seg, buf, src, dst, ref, t


@pytest.mark.parametrize("w", [W.config1(), W.config2(), W.config5(4, 64, 6, 32), W.config3(1)],
                         ids=lambda w: w.name)
def test_reencode_parity(w):
    c, seg, buf, src, dst, ref, t = reencode_case(w)
    check_reencoded(R.device_to_bits(dst), ref)
    # the block with delta 0 is copied bit-exactly
    n0 = int(t["cache_cu"][1])
    if w.pool_lens is None:
        assert torch.equal(dst[:n0], src[:n0])
    c.close()


def test_reencode_half_layout_in_place_and_inverse():
    w = W.config2()
    c, seg, buf, src, dst, ref, t = reencode_case(w, layout=B.BA_ROPE_HALF)
    check_reencoded(R.device_to_bits(dst), ref)
    Tc = t["n_cached_tokens"]
    # in place
    inplace = src.clone()
    B.ba_reencode_k(c.ctx, inplace, None, Tc, inplace, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    assert torch.equal(inplace, dst)
    # negative deltas (Eq. 2: back to position zero) undo the re-encoding up to bf16 rounding
    neg = torch.from_numpy(-t["cache_delta"]).cuda()
    back = torch.empty_like(dst)
    B.ba_reencode_k(c.ctx, dst, None, Tc, back, seg.cache_cu, neg, seg.n_cached_blocks, Tc)
    ref_back = ob.reencode_blocks(W.bf16_bits_to_f64(R.device_to_bits(dst)), None, t["cache_cu"],
                                  -t["cache_delta"], w.rope_theta, ob.ROPE_HALF)
    check_reencoded(R.device_to_bits(back), ref_back)
    assert c.device_status() == B.BA_OK
    c.close()


def test_reencode_errors_do_not_fault():
    w = W.config1()
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    k = torch.zeros(256, 2, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(k)
    off = torch.tensor([0, 64, 128, 250], dtype=torch.int32, device="cuda")   # last block runs off the source
    B.ba_reencode_k(c.ctx, k, off, 256, out, seg.cache_cu, seg.cache_delta, 4, 256)
    assert c.device_status() == B.BA_ERR_INVALID_ARG
    with pytest.raises(B.BaError) as e:
        B.ba_reencode_k(c.ctx, k, off, 256, k, seg.cache_cu, seg.cache_delta, 4, 256)   # gather in place
    assert e.value.status == B.BA_ERR_INVALID_ARG
    with pytest.raises(B.BaError):
        B.ba_reencode_k(c.ctx, k.view(-1)[1:], None, 255, out, seg.cache_cu, seg.cache_delta, 4, 255)  # misaligned
    # a context created with a workspace too small for the call reports it instead of overrunning
    small = B.ba_create(c.cfg, 0, 1024)
    lens = np.ones(600, dtype=np.int32)
    tb = torch.empty(B.ba_segments_bytes(1, 600, 600), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.BaError) as e:
        B.ba_segment(small, lens, np.asarray([600], dtype=np.int32), 1, 600, 600, B.BA_MODE_BLOCK, tb)
    assert e.value.status == B.BA_ERR_WORKSPACE
    with pytest.raises(B.BaError) as e:
        B.ba_reencode_k(small, k, None, 256, out, seg.cache_cu, seg.cache_delta, 4, 256)   # 4 * 64 * 4 = 1024 > room
    assert e.value.status == B.BA_ERR_WORKSPACE
    B.ba_destroy(small)
    c.close()


# --------------------------------------------------------------------------- prefill
def run_prefill(w, mode, out_dtype=B.BA_OUT_F32, rows=None, layer=0):
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, mode)
    qb, kb, vb = W.prefill_inputs(w, layer)
    q, k, v = dev(qb), dev(kb), dev(vb)
    T = w.n_tokens
    o = torch.empty(T, w.n_q_heads, w.head_dim, device="cuda",
                    dtype=torch.float32 if out_dtype == B.BA_OUT_F32 else torch.bfloat16)
    lse = torch.empty(T, w.n_q_heads, dtype=torch.float32, device="cuda")
    B.ba_block_prefill(c.ctx, q, k, v, o, lse, seg, mode, out_dtype)
    assert c.device_status() == B.BA_OK
    if rows is None:
        rows = np.arange(T)
    o_ref, lse_ref = ob.block_prefill(W.bf16_bits_to_f64(qb), W.bf16_bits_to_f64(kb), W.bf16_bits_to_f64(vb),
                                      w.block_lens, w.seq_nblocks, mode, rows=rows)
    c.close()
    rt = torch.from_numpy(np.asarray(rows)).cuda()
    return o[rt].float().cpu().numpy(), lse[rt].cpu().numpy(), o_ref, lse_ref


PREFILL_CASES = [W.config1(), W.config2(), W.random_ragged(21, 3, 6, 300, 4, 2, 64),
                 W.random_ragged(22, 2, 5, 400, 8, 2, 128), W.random_ragged(23, 4, 4, 140, 4, 4, 128),
                 W.Workload("one_token", 4, 2, 64, 1e4, [1], [1], seed=5),
                 W.Workload("single_block", 8, 8, 128, 1e4, [333], [1], seed=6),
                 # enough work items for the persistent launch (several items per CTA, ragged)
                 W.random_ragged(24, 14, 8, 300, 8, 2, 128), W.random_ragged(25, 30, 6, 200, 4, 1, 64),
                 # eight query heads per KV head: two head chunks share every K/V tile
                 W.random_ragged(26, 3, 4, 300, 8, 1, 128),
                 # an odd group size: one head per query tile, 128 tokens per tile
                 W.random_ragged(27, 3, 4, 300, 6, 2, 64)]


@pytest.mark.parametrize("w", PREFILL_CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("mode", [B.BA_MODE_BLOCK, B.BA_MODE_FULL])
def test_prefill_parity(w, mode):
    o, lse, o_ref, lse_ref = run_prefill(w, mode)
    check_attention(o, o_ref, lse, lse_ref)


@pytest.mark.parametrize("mode", [B.BA_MODE_BLOCK, B.BA_MODE_FULL])
def test_prefill_running_maximum_that_keeps_growing(mode):
    """Keys whose magnitude grows along the sequence: the row maximum of the logits keeps rising from key
    tile to key tile and inside tiles, by far more than the factor the kernel lets its reference maximum
    lag behind, so every rescaling path of the online softmax runs many times."""
    w = W.Workload("growing_logits", 8, 2, 128, 1e4, [700, 300, 45], [2, 1], seed=55)
    qb, kb, vb = W.prefill_inputs(w)
    ramp = (1.0 + 60.0 * np.arange(w.n_tokens) / w.n_tokens).astype(np.float32)
    kb = W.f32_to_bf16_bits(W.bf16_bits_to_f32(kb) * ramp[:, None, None])
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, mode)
    o = torch.empty(w.n_tokens, w.n_q_heads, w.head_dim, device="cuda", dtype=torch.float32)
    lse = torch.empty(w.n_tokens, w.n_q_heads, dtype=torch.float32, device="cuda")
    B.ba_block_prefill(c.ctx, dev(qb), dev(kb), dev(vb), o, lse, seg, mode, B.BA_OUT_F32)
    assert c.device_status() == B.BA_OK
    o_ref, lse_ref = ob.block_prefill(W.bf16_bits_to_f64(qb), W.bf16_bits_to_f64(kb), W.bf16_bits_to_f64(vb),
                                      w.block_lens, w.seq_nblocks, mode)
    # logits reach the hundreds: the log-sum-exp is compared relative to its size, the outputs (convex
    # combinations of N(0,1) values) under the usual bounds
    og = o.cpu().numpy()
    assert np.isfinite(og).all()
    d = np.abs(og - o_ref)
    assert d.max() <= 2e-2 and d.mean() <= 1e-3, (d.max(), d.mean())
    assert np.linalg.norm(og - o_ref) / np.linalg.norm(o_ref) <= 5e-3
    assert (np.abs(lse.cpu().numpy() - lse_ref) <= 2e-3 + 1e-5 * np.abs(lse_ref)).all()
    c.close()


def test_prefill_bf16_output():
    o, lse, o_ref, lse_ref = run_prefill(W.config2(), B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    check_attention(o, o_ref, lse, lse_ref, bf16_store=True)


def sampled_rows(w, per_block=8, extra=128, seed=0, tile_tokens=64):
    """Rows the oracle is evaluated on at full size: the first and last rows of every block, seeded
    random rows, and per sequence two whole work items (two query tiles of `tile_tokens` / 2 tokens
    each, every head) from the interior -- one in the sequence's longest non-final block, one in its
    final block -- where the persistent launch interleaves items of different blocks."""
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    rows = []
    for b in range(w.n_blocks):
        lo, hi = int(t["cu_block"][b]), int(t["cu_block"][b + 1])
        rows += list(range(lo, min(hi, lo + per_block))) + list(range(max(lo, hi - per_block), hi))
    b0 = 0
    for nb in w.seq_nblocks:
        blocks = list(range(b0, b0 + nb))
        picks = [blocks[-1]]
        if nb > 1:
            picks.append(max(blocks[:-1], key=lambda b: w.block_lens[b]))
        for b in picks:
            lo, n = int(t["cu_block"][b]), w.block_lens[b]
            item = (n // tile_tokens) // 2                      # an item in the middle of the block
            rows += list(range(lo + item * tile_tokens, min(lo + n, lo + (item + 1) * tile_tokens)))
        b0 += nb
    rng = np.random.default_rng(seed)
    rows += [int(x) for x in rng.integers(0, w.n_tokens, size=extra)]
    return np.unique(np.asarray(rows))


def test_prefill_cold_batch_full_size_sampled_rows():
    # batch 8 x 16384 ragged cold prefill in one launch, the launch bench.py times (exact for the rows taken)
    w = W.config4()
    rows = sampled_rows(w, per_block=8, extra=128)
    o, lse, o_ref, lse_ref = run_prefill(w, B.BA_MODE_BLOCK, rows=rows)
    check_attention(o, o_ref, lse, lse_ref)


def test_prefill_full_causal_32k_sampled_rows():
    w = W.config3(1)
    rng = np.random.default_rng(3)
    # the first and the last work item, one that straddles the middle of the prompt, seeded rows
    rows = np.unique(np.concatenate([np.arange(0, 64), np.arange(32704, 32768), np.arange(16352, 16416),
                                     rng.integers(0, 32768, 64)]))
    o, lse, o_ref, lse_ref = run_prefill(w, B.BA_MODE_FULL, rows=rows)
    check_attention(o, o_ref, lse, lse_ref)


# --------------------------------------------------------------------------- warm path
def run_warm(w, mode, out_dtype=B.BA_OUT_F32, layer=0, v_from_pool=True, fused=False,
             layout=B.BA_ROPE_ADJACENT, shape_out=None):
    """ba_segment -> ba_reencode_k -> ba_final_attend (or ba_final_attend_fused on the keys as
    cached), against oracle re-encode + final attend.  The oracle attends its own unrounded fp64
    re-encoded keys."""
    c = ctx_for(w, rope_layout=layout)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, mode)
    t = ob.segment_tables(w.block_lens, w.seq_nblocks, mode)
    x = W.warm_inputs(w, layer)
    Tc, Tf = t["n_cached_tokens"], t["n_final_tokens"]
    q_f, k_f, v_f = dev(x["q_f"]), dev(x["k_f"]), dev(x["v_f"])
    k_re = torch.empty(Tc, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    if w.pool_lens is None:
        k_src, v_cache, off, off_np = dev(x["k_cache"]), dev(x["v_cache"]), None, None
        k_src_np, v_np = x["k_cache"], W.bf16_bits_to_f64(x["v_cache"])
        v_off, n_v = None, 0
    else:
        k_src, off_np = dev(x["k_pool"]), x["src_off"]
        off = torch.from_numpy(off_np).cuda()
        k_src_np = x["k_pool"]
        v_pool64 = W.bf16_bits_to_f64(x["v_pool"])
        v_np = np.concatenate([v_pool64[o_:o_ + (t["cache_cu"][i + 1] - t["cache_cu"][i])]
                               for i, o_ in enumerate(off_np)], axis=0)
        if v_from_pool:
            v_cache, v_off, n_v = dev(x["v_pool"]), off, x["v_pool"].shape[0]
        else:
            v_cache, v_off, n_v = dev(W.f32_to_bf16_bits(v_np.astype(np.float32))), None, 0
    o = torch.empty(Tf, w.n_q_heads, w.head_dim, device="cuda",
                    dtype=torch.float32 if out_dtype == B.BA_OUT_F32 else torch.bfloat16)
    lse = torch.empty(Tf, w.n_q_heads, dtype=torch.float32, device="cuda")
    if fused:
        # keys and values are addressed alike: both from the pool, or both in cache packing
        v_src = dev(x["v_pool"]) if w.pool_lens is not None else v_cache
        B.ba_final_attend_fused(c.ctx, q_f, k_f, v_f, Tf, k_src, v_src, k_src.shape[0], off, Tc, o, lse, seg,
                                mode, out_dtype)
    else:
        B.ba_reencode_k(c.ctx, k_src, off, k_src.shape[0], k_re, seg.cache_cu, seg.cache_delta,
                        seg.n_cached_blocks, Tc)
        B.ba_final_attend(c.ctx, q_f, k_f, v_f, Tf, k_re, v_cache, Tc, v_off, n_v, o, lse, seg, mode, out_dtype)
    assert c.device_status() == B.BA_OK
    if shape_out is not None:
        shape_out.append(c.last_attend_shape())
    k_ref = ob.reencode_blocks(W.bf16_bits_to_f64(k_src_np), off_np, t["cache_cu"], t["cache_delta"], w.rope_theta,
                               layout)
    o_ref, lse_ref = ob.final_attend(W.bf16_bits_to_f64(x["q_f"]), W.bf16_bits_to_f64(x["k_f"]),
                                     W.bf16_bits_to_f64(x["v_f"]), k_ref, v_np, w.block_lens, w.seq_nblocks, mode)
    c.close()
    return o.float().cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref


WARM_CASES = [W.config1(), W.config2(), W.random_ragged(31, 3, 5, 200, 4, 2, 64),
              W.Workload("no_cache", 4, 2, 64, 1e4, [50, 1, 130], [1, 1, 1], seed=7),
              W.config5(4, 64, 6, 32),
              # many requests: split keys and the persistent launch together
              W.random_ragged(32, 40, 4, 150, 8, 2, 128), W.config5(48, 64, 5, 40),
              # eight query heads per KV head (two head chunks per group); an odd group size (one head per tile)
              W.random_ragged(33, 3, 5, 200, 16, 2, 128), W.random_ragged(34, 3, 5, 200, 6, 2, 64)]


@pytest.mark.parametrize("w", WARM_CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("mode", [B.BA_MODE_BLOCK, B.BA_MODE_FULL])
def test_warm_path_parity(w, mode):
    o, lse, o_ref, lse_ref = run_warm(w, mode)
    check_attention(o, o_ref, lse, lse_ref)


def test_warm_path_pool_serving_full_size_and_mode_switch():
    w = W.config5()
    half = W.Workload("half", w.n_q_heads, w.n_kv_heads, w.head_dim, w.rope_theta,
                      w.block_lens[:21 * 8], w.seq_nblocks[:8], w.seed, pool_lens=w.pool_lens,
                      request_pool_idx=w.request_pool_idx[:8])
    ob_, lb, o_ref, lse_ref = run_warm(half, B.BA_MODE_BLOCK)
    check_attention(ob_, o_ref, lb, lse_ref)
    # final rows see the same keys under both masks: with the values in the same place the two
    # modes run the same tiles and agree to the last bit
    op_, lp, _, _ = run_warm(half, B.BA_MODE_BLOCK, v_from_pool=False)
    of_, lf, _, _ = run_warm(half, B.BA_MODE_FULL, v_from_pool=False)
    check_attention(op_, o_ref, lp, lse_ref)
    assert np.abs(of_ - op_).max() <= 1e-6 and np.abs(lf - lp).max() <= 1e-6


def test_pool_serving_as_stated_sixteen_requests_half_full_mode():
    """The pool-serving workload as it is stated: one pool, one draw of inputs for all 16 requests;
    requests 0-7 run under Block-attention tables, requests 8-15 under full-causal tables, both through
    ba_reencode_k (gather + rotation) and ba_final_attend with the values read from the pool in place.
    Every final row of every request is compared with the oracle."""
    w = W.config5()
    x = W.warm_inputs(w)
    c = ctx_for(w)
    k_pool, v_pool = dev(x["k_pool"]), dev(x["v_pool"])
    k64, v64 = W.bf16_bits_to_f64(x["k_pool"]), W.bf16_bits_to_f64(x["v_pool"])
    per = 21
    for lo, hi, mode in ((0, 8, B.BA_MODE_BLOCK), (8, 16, B.BA_MODE_FULL)):
        lens, nbs = w.block_lens[per * lo:per * hi], w.seq_nblocks[lo:hi]
        off_np = x["src_off"][20 * lo:20 * hi]
        f0, f1 = 128 * lo, 128 * hi
        seg, buf = c.segment(lens, nbs, mode)
        t = ob.segment_tables(lens, nbs, mode)
        Tc, Tf = t["n_cached_tokens"], t["n_final_tokens"]
        assert Tf == f1 - f0
        off = torch.from_numpy(np.ascontiguousarray(off_np)).cuda()
        q_f, k_f, v_f = dev(x["q_f"][f0:f1]), dev(x["k_f"][f0:f1]), dev(x["v_f"][f0:f1])
        k_re = torch.empty(Tc, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
        o = torch.empty(Tf, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda")
        lse = torch.empty(Tf, w.n_q_heads, dtype=torch.float32, device="cuda")
        B.ba_reencode_k(c.ctx, k_pool, off, k_pool.shape[0], k_re, seg.cache_cu, seg.cache_delta,
                        seg.n_cached_blocks, Tc)
        B.ba_final_attend(c.ctx, q_f, k_f, v_f, Tf, k_re, v_pool, Tc, off, v_pool.shape[0], o, lse, seg, mode,
                          B.BA_OUT_F32)
        assert c.device_status() == B.BA_OK
        k_ref = ob.reencode_blocks(k64, off_np, t["cache_cu"], t["cache_delta"], w.rope_theta)
        check_reencoded(R.device_to_bits(k_re), k_ref)
        v_np = np.concatenate([v64[o_:o_ + (t["cache_cu"][i + 1] - t["cache_cu"][i])] for i, o_ in enumerate(off_np)])
        o_ref, lse_ref = ob.final_attend(W.bf16_bits_to_f64(x["q_f"][f0:f1]), W.bf16_bits_to_f64(x["k_f"][f0:f1]),
                                         W.bf16_bits_to_f64(x["v_f"][f0:f1]), k_ref, v_np, lens, nbs, mode)
        check_attention(o.cpu().numpy(), o_ref, lse.cpu().numpy(), lse_ref)
    c.close()


def many_small_cached_blocks():
    """Appendix A's shape: a prompt of more than 300 small cached blocks (4-48 tokens each, drawn from
    a pool of 96 with repetition) and a short final block."""
    rng = np.random.default_rng(91)
    pool_lens = [int(v) for v in rng.integers(4, 49, size=96)]
    idx = [int(v) for v in rng.integers(0, 96, size=320)]
    lens = [pool_lens[i] for i in idx] + [40]
    return W.Workload("many_small_cached", 8, 2, 128, 5e5, lens, [321], seed=91, pool_lens=pool_lens,
                      request_pool_idx=[idx])


@pytest.mark.parametrize("fused", [False, True], ids=["reencode_then_attend", "fused"])
def test_final_block_over_many_small_cached_blocks(fused):
    """The final block attends 320 small cached blocks: with the values read from the pool the cached
    keys are walked block by block (every key tile belongs to one block and is mostly padding); the
    fused call prepares a query version per cached block.  Every final row against the oracle."""
    w = many_small_cached_blocks()
    o, lse, o_ref, lse_ref = run_warm(w, B.BA_MODE_BLOCK, fused=fused)
    check_attention(o, o_ref, lse, lse_ref)


def paged_case(w, page_rows, layer=0, layout=B.BA_ROPE_ADJACENT):
    """The cached keys and values of workload `w` scattered over paged pools (one page table for both)."""
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    x = W.warm_inputs(w, layer)
    cache_lens = [l for lens in w.cached_lens_per_seq() for l in lens]
    k_pool, page_cu, page_idx, n_pages = W.scatter_into_pages(x["k_cache"], cache_lens, page_rows, seed=w.seed + 5)
    v_pool, _, _, _ = W.scatter_into_pages(x["v_cache"], cache_lens, page_rows, seed=w.seed + 5)
    d_cu, d_idx = torch.from_numpy(page_cu).cuda(), torch.from_numpy(page_idx).cuda()
    pages = B.make_page_table(page_rows, n_pages, d_cu, d_idx)
    # the oracle reads the pools through the same table, by plain indexing
    rows = ob.paged_rows(cache_lens, page_rows, page_cu, page_idx)
    k64, v64 = W.bf16_bits_to_f64(k_pool[rows]), W.bf16_bits_to_f64(v_pool[rows])
    k_ref = ob.reencode_blocks(k64, None, t["cache_cu"], t["cache_delta"], w.rope_theta, layout)
    o_ref, lse_ref = ob.final_attend(W.bf16_bits_to_f64(x["q_f"]), W.bf16_bits_to_f64(x["k_f"]),
                                     W.bf16_bits_to_f64(x["v_f"]), k_ref, v64, w.block_lens, w.seq_nblocks)
    return t, x, dev(k_pool), dev(v_pool), pages, (d_cu, d_idx), k_ref, o_ref, lse_ref


def _balanced_cases():
    """Final blocks over long caches with fewer work items than SMs: the launch gives one CTA the tail of each
    item and lets the others share the key tiles in front (ragged cached blocks, ragged final blocks, two
    sequences of unequal length, two head chunks per KV group, head_dim 64)."""
    rng = np.random.default_rng(77)
    one = [int(v) for v in rng.integers(300, 900, 20)] + [700]
    two_a = [int(v) for v in rng.integers(200, 700, 20)] + [300]
    two_b = [int(v) for v in rng.integers(200, 700, 23)] + [330]
    d64 = [int(v) for v in rng.integers(500, 1500, 8)] + [1390]
    return [W.Workload("balanced_one_sequence", 32, 8, 128, 5e5, one, [21], seed=81),
            W.Workload("balanced_two_sequences", 32, 8, 128, 5e5, two_a + two_b, [21, 24], seed=82),
            W.Workload("balanced_head_dim_64_two_chunks", 16, 2, 64, 1e4, d64, [9], seed=83)]


PAGED_CASES = [(W.config1(), 16), (W.config2(), 16), (W.config2(), 64), (W.config2(), 128), (W.config2(), 256),
               (W.random_ragged(41, 3, 6, 300, 8, 2, 128), 32), (W.random_ragged(42, 5, 4, 200, 4, 2, 64), 16)]


def _paged_cases():
    # a long cache under few work items: paged values and keys in the balanced launch
    return PAGED_CASES + [(_balanced_cases()[0], 64)]


@pytest.mark.parametrize("w,page_rows", _paged_cases(), ids=lambda v: v.name if hasattr(v, "name") else f"p{v}")
def test_paged_cache_reencode_and_attend(w, page_rows):
    """Section 2.5 step 1 with a paged cache: cached keys gathered through the page table and re-encoded
    (ba_reencode_k_paged), values read from their pages in place by ba_final_attend_paged (one copy per
    page, a key tile never spans two pages); then both steps in one launch on the paged keys
    (ba_final_attend_fused_paged) with the re-encoded keys written back.  Pages are in a seeded order and
    the unused rows of last pages hold noise."""
    t, x, k_pool, v_pool, pages, keep, k_ref, o_ref, lse_ref = paged_case(w, page_rows)
    Tc, Tf = t["n_cached_tokens"], t["n_final_tokens"]
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    q_f, k_f, v_f = dev(x["q_f"]), dev(x["k_f"]), dev(x["v_f"])
    o = torch.empty(Tf, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda")
    lse = torch.empty(Tf, w.n_q_heads, dtype=torch.float32, device="cuda")
    if Tc > 0:
        k_re = torch.zeros(Tc, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
        B.ba_reencode_k_paged(c.ctx, k_pool, pages, k_re, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
        assert c.device_status() == B.BA_OK
        check_reencoded(R.device_to_bits(k_re), k_ref)
        # the same bytes as the contiguous call on the packed keys
        k_packed = torch.empty_like(k_re)
        B.ba_reencode_k(c.ctx, dev(x["k_cache"]), None, Tc, k_packed, seg.cache_cu, seg.cache_delta,
                        seg.n_cached_blocks, Tc)
        assert torch.equal(k_re, k_packed)
    else:
        k_re = None
    B.ba_final_attend_paged(c.ctx, q_f, k_f, v_f, Tf, k_re, Tc, v_pool, pages, o, lse, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    assert c.device_status() == B.BA_OK
    if w.name.startswith("balanced"):
        assert c.last_attend_shape()["balanced_tails"] > 0
    check_attention(o.cpu().numpy(), o_ref, lse.cpu().numpy(), lse_ref)
    o2 = torch.empty_like(o)
    k_out = torch.zeros_like(k_re) if Tc > 0 else None
    B.ba_final_attend_fused_paged(c.ctx, q_f, k_f, v_f, Tf, k_pool, v_pool, pages, Tc, o2, lse, seg, B.BA_MODE_BLOCK,
                                  B.BA_OUT_F32, k_out=k_out)
    assert c.device_status() == B.BA_OK
    check_attention(o2.cpu().numpy(), o_ref, lse.cpu().numpy(), lse_ref)
    if Tc > 0:
        assert torch.equal(k_out, k_re)
    c.close()


def test_paged_cache_bad_page_numbers_are_reported_and_bad_sizes_refused():
    w = W.config1()
    t, x, k_pool, v_pool, pages, (d_cu, d_idx), k_ref, o_ref, lse_ref = paged_case(w, 16)
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    k_re = torch.zeros(256, 2, 64, dtype=torch.bfloat16, device="cuda")
    bad_idx = d_idx.clone(); bad_idx[3] = 10 ** 6; bad_idx[5] = -2
    bad = B.make_page_table(16, pages.n_pages, d_cu, bad_idx)
    B.ba_reencode_k_paged(c.ctx, k_pool, bad, k_re, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, 256)
    assert c.device_status() == B.BA_ERR_INVALID_ARG
    assert not k_re[48:64].any() and not k_re[80:96].any()           # the rows of the bad pages were skipped
    for rows in (8, 24, 1 << 17):
        with pytest.raises(B.BaError) as e:
            B.ba_reencode_k_paged(c.ctx, k_pool, B.make_page_table(rows, 4, d_cu, d_idx), k_re, seg.cache_cu,
                                  seg.cache_delta, seg.n_cached_blocks, 256)
        assert e.value.status == B.BA_ERR_UNSUPPORTED
    c.close()


@pytest.mark.parametrize("w", _balanced_cases(), ids=lambda w: w.name)
@pytest.mark.parametrize("fused", [False, True], ids=["reencode_then_attend", "fused"])
def test_balanced_launch_parity(w, fused):
    shapes = []
    o, lse, o_ref, lse_ref = run_warm(w, B.BA_MODE_BLOCK, fused=fused, shape_out=shapes)
    assert shapes[-1]["balanced_tails"] > 0 and shapes[-1]["partials"] >= 2, shapes
    check_attention(o, o_ref, lse, lse_ref)
    if w.name == "balanced_two_sequences":
        # whichever CTA merges an item's partial results, the sum runs in the same order: the same bits every time
        for _ in range(3):
            o2, lse2, _, _ = run_warm(w, B.BA_MODE_BLOCK, fused=fused)
            assert np.array_equal(o, o2) and np.array_equal(lse, lse2)


def test_warm_path_32k_full_size():
    w = W.config3(1)
    o, lse, o_ref, lse_ref = run_warm(w, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    check_attention(o, o_ref, lse, lse_ref, bf16_store=True)
    o2, lse2, _, _ = run_warm(w, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    check_attention(o2, o_ref, lse2, lse_ref)


@pytest.mark.parametrize("w", WARM_CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("mode", [B.BA_MODE_BLOCK, B.BA_MODE_FULL])
def test_fused_warm_path_parity(w, mode):
    """Re-encoding applied to the query side inside the attention launch (keys as cached)."""
    o, lse, o_ref, lse_ref = run_warm(w, mode, fused=True)
    check_attention(o, o_ref, lse, lse_ref)


@pytest.mark.parametrize("w", [W.config1(), W.config2(), W.config5(4, 64, 6, 32)], ids=lambda w: w.name)
def test_fused_warm_path_half_layout(w):
    o, lse, o_ref, lse_ref = run_warm(w, B.BA_MODE_BLOCK, fused=True, layout=B.BA_ROPE_HALF)
    check_attention(o, o_ref, lse, lse_ref)


@pytest.mark.parametrize("w,layout", [(W.config1(), B.BA_ROPE_ADJACENT), (W.config2(), B.BA_ROPE_HALF),
                                      (W.config5(4, 64, 6, 32), B.BA_ROPE_ADJACENT), (W.config3(1), B.BA_ROPE_ADJACENT)],
                         ids=["tiny", "rag_half", "pool", "32k"])
def test_fused_call_writes_the_reencoded_keys_as_a_side_output(w, layout):
    """Section 2.5 steps 2-3 in one launch, with the re-encoded keys -- what later decode steps read --
    written back by the same launch: bit-identical to ba_reencode_k, a correct rounding of the oracle's
    rotation, and the attention output unchanged by the side job."""
    c, seg, buf, src, want, ref, t = reencode_case(w, layout=layout)      # `want`: ba_reencode_k
    x = W.warm_inputs(w)
    Tc, Tf = t["n_cached_tokens"], t["n_final_tokens"]
    off = torch.from_numpy(x["src_off"]).cuda() if w.pool_lens is not None else None
    v_src = dev(x["v_pool"] if w.pool_lens is not None else x["v_cache"])
    q_f, k_f, v_f = dev(x["q_f"]), dev(x["k_f"]), dev(x["v_f"])
    o_plain = torch.empty(Tf, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda")
    o_side = torch.empty_like(o_plain)
    k_out = torch.zeros_like(want)
    B.ba_final_attend_fused(c.ctx, q_f, k_f, v_f, Tf, src, v_src, src.shape[0], off, Tc, o_plain, None, seg,
                            B.BA_MODE_BLOCK, B.BA_OUT_F32)
    for _ in range(2):          # twice: the launch counters must be back at zero after the first launch
        k_out.zero_()
        B.ba_final_attend_fused(c.ctx, q_f, k_f, v_f, Tf, src, v_src, src.shape[0], off, Tc, o_side, None, seg,
                                B.BA_MODE_BLOCK, B.BA_OUT_F32, k_out=k_out)
        assert c.device_status() == B.BA_OK
        assert torch.equal(k_out, want)
        assert torch.equal(o_side, o_plain)
    check_reencoded(R.device_to_bits(k_out), ref)
    with pytest.raises(B.BaError) as e:          # in place: the attention reads the cached keys meanwhile
        B.ba_final_attend_fused(c.ctx, q_f, k_f, v_f, Tf, src, v_src, src.shape[0], off, Tc, o_side, None, seg,
                                B.BA_MODE_BLOCK, B.BA_OUT_F32, k_out=src)
    assert e.value.status == B.BA_ERR_INVALID_ARG
    c.close()


def test_fused_warm_path_32k_full_size_and_pool_serving():
    w = W.config3(1)
    o, lse, o_ref, lse_ref = run_warm(w, B.BA_MODE_BLOCK, fused=True)
    check_attention(o, o_ref, lse, lse_ref)
    w5 = W.config5()
    o, lse, o_ref, lse_ref = run_warm(w5, B.BA_MODE_BLOCK, fused=True)
    check_attention(o, o_ref, lse, lse_ref)


def test_incremental_block_update_many_small_blocks():
    """Section 2.1 and Appendix A (prompts of hundreds of small independent blocks): after an edit only
    the edited blocks are encoded again.  A non-final block sees only itself, so encoding it alone -- as
    a one-block sequence -- must reproduce its rows of the whole-prompt launch; checked on a prompt of
    320 small blocks, against the whole launch (bit-identical: same tiles) and against the oracle."""
    rng = np.random.default_rng(77)
    lens = [int(x) for x in rng.integers(4, 48, size=320)] + [40]
    w = W.Workload("many_small_blocks", 8, 2, 128, 5e5, lens, [len(lens)], seed=77)
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    qb, kb, vb = W.prefill_inputs(w)
    q, k, v = dev(qb), dev(kb), dev(vb)
    o = torch.empty(w.n_tokens, w.n_q_heads, w.head_dim, device="cuda", dtype=torch.float32)
    B.ba_block_prefill(c.ctx, q, k, v, o, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    cu = np.concatenate([[0], np.cumsum(lens)])
    edited = [3, 57, 58, 200, 319]
    rows = np.concatenate([np.arange(cu[b], cu[b + 1]) for b in edited])
    rt = torch.from_numpy(rows).cuda()
    # the edited blocks alone: each is a sequence of one block (its final block = causal inside itself)
    sub_lens = [lens[b] for b in edited]
    seg2, buf2 = c.segment(sub_lens, [1] * len(edited), B.BA_MODE_BLOCK)
    q2, k2, v2 = q[rt].contiguous(), k[rt].contiguous(), v[rt].contiguous()
    o2 = torch.empty(len(rows), w.n_q_heads, w.head_dim, device="cuda", dtype=torch.float32)
    B.ba_block_prefill(c.ctx, q2, k2, v2, o2, None, seg2, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    assert c.device_status() == B.BA_OK
    assert torch.equal(o2, o[rt])
    o_ref, _ = ob.block_prefill(W.bf16_bits_to_f64(qb), W.bf16_bits_to_f64(kb), W.bf16_bits_to_f64(vb),
                                w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK, rows=rows)
    check_attention(o2.cpu().numpy(), o_ref)
    c.close()


def test_cache_fill_and_no_position_variant():
    """Section 2.3: after a cold prefill the keys of a block are put into the cache at positions 0..L-1
    (Eq. 2: rotation by minus the block's start), and re-encoding them later to the same start gives
    the prompt keys back up to bf16 rounding.  Delta 0 everywhere (the ablation without position
    re-encoding, Section 3.3) leaves the keys bit-identical."""
    w = W.config2()
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    x = W.warm_inputs(w)
    Tc = t["n_cached_tokens"]
    k_prompt = dev(x["k_cache"])                       # taken as keys at prompt positions
    neg = torch.from_numpy(-t["cache_delta"]).cuda()
    k_cached = torch.empty_like(k_prompt)
    B.ba_reencode_k(c.ctx, k_prompt, None, Tc, k_cached, seg.cache_cu, neg, seg.n_cached_blocks, Tc)
    ref = ob.reencode_blocks(W.bf16_bits_to_f64(x["k_cache"]), None, t["cache_cu"], -t["cache_delta"], w.rope_theta)
    check_reencoded(R.device_to_bits(k_cached), ref)
    zero = torch.zeros_like(neg)
    same = torch.empty_like(k_prompt)
    B.ba_reencode_k(c.ctx, k_prompt, None, Tc, same, seg.cache_cu, zero, seg.n_cached_blocks, Tc)
    assert torch.equal(same, k_prompt)
    assert c.device_status() == B.BA_OK
    c.close()


def test_attention_rejects_mode_mismatch_and_null():
    w = W.config1()
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    q = torch.zeros(288, 4, 64, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(288, 2, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.BaError) as e:
        B.ba_block_prefill(c.ctx, q, kv, kv, q, None, seg, B.BA_MODE_FULL, B.BA_OUT_BF16)
    assert e.value.status == B.BA_ERR_INVALID_ARG
    with pytest.raises(B.BaError):
        B.ba_block_prefill(c.ctx, q, None, kv, q, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    with pytest.raises(B.BaError):
        B.ba_final_attend(c.ctx, q, kv, kv, 32, None, None, 256, None, 0, q, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
    c.close()


def test_runs_are_bit_stable():
    w = W.config2()
    a = run_warm(w, B.BA_MODE_BLOCK)[0]
    b = run_warm(w, B.BA_MODE_BLOCK)[0]
    assert (a == b).all()


def test_bounded_wait_expires_into_a_status_and_the_device_stays_usable():
    w = W.config1()
    c = ctx_for(w)
    B.ba_selftest_wait_expiry(c.ctx)
    assert c.device_status() == B.BA_ERR_TIMEOUT       # the wait gave up; nothing hung, nothing faulted
    assert c.device_status() == B.BA_OK
    c.close()
    o, lse, o_ref, lse_ref = run_prefill(w, B.BA_MODE_BLOCK)   # same process, same device: still works
    check_attention(o, o_ref, lse, lse_ref)


@pytest.mark.parametrize("w,layout", [(W.config2(), B.BA_ROPE_ADJACENT), (W.config1(), B.BA_ROPE_HALF),
                                      (W.config5(4, 64, 6, 32), B.BA_ROPE_ADJACENT)], ids=["rag", "tiny_half", "pool"])
def test_deferred_reencode_rides_along_with_attention(w, layout):
    """A queued re-encoding job is carried out by the next attention launch (or by ba_flush) and
    gives the same bytes as the immediate call; the attention results are unaffected."""
    c, seg, buf, src, want, ref, t = reencode_case(w, layout=layout)      # `want`: immediate ba_reencode_k
    off = torch.from_numpy(W.warm_inputs(w)["src_off"]).cuda() if w.pool_lens is not None else None
    Tc = t["n_cached_tokens"]
    qb, kb, vb = W.prefill_inputs(w)
    q, k, v = dev(qb), dev(kb), dev(vb)
    o_plain = torch.empty(w.n_tokens, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda")
    o_with = torch.empty_like(o_plain)
    B.ba_block_prefill(c.ctx, q, k, v, o_plain, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    got = torch.zeros_like(want)
    n0 = c.launches()
    own_delta = torch.from_numpy(t["cache_delta"]).cuda()  # not the tables' array: the call builds its own angle table
    B.ba_reencode_k_deferred(c.ctx, src, off, src.shape[0], got, seg.cache_cu, own_delta, seg.n_cached_blocks, Tc)
    assert c.launches() == n0 + 1                       # only the angle table so far
    torch.cuda.synchronize()
    assert not got.any()                                # nothing written yet
    B.ba_block_prefill(c.ctx, q, k, v, o_with, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    torch.cuda.synchronize()
    assert c.device_status() == B.BA_OK
    assert torch.equal(got, want)
    assert torch.equal(o_with, o_plain)
    # ba_flush runs a queued job on its own; a second flush is a no-op
    got2 = torch.zeros_like(want)
    n2 = c.launches()
    B.ba_reencode_k_deferred(c.ctx, src, off, src.shape[0], got2, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    assert c.launches() == n2                           # with the tables' own deltas the table ba_segment built is reused
    B.ba_flush(c.ctx)
    n1 = c.launches()
    B.ba_flush(c.ctx)
    assert c.launches() == n1
    torch.cuda.synchronize()
    assert torch.equal(got2, want)
    # an immediate call while a job is queued uses its own table; queuing twice runs the first job
    got3, got4, got5 = torch.zeros_like(want), torch.zeros_like(want), torch.zeros_like(want)
    B.ba_reencode_k_deferred(c.ctx, src, off, src.shape[0], got3, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    B.ba_reencode_k(c.ctx, src, off, src.shape[0], got4, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    B.ba_reencode_k_deferred(c.ctx, src, off, src.shape[0], got5, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    c.close()                                           # destroying the context runs what is still queued
    torch.cuda.synchronize()
    assert torch.equal(got3, want) and torch.equal(got4, want) and torch.equal(got5, want)


def test_final_rows_beyond_the_output_tensor_are_reported_not_written():
    """Tables that describe more final rows than the tensors passed to ba_final_attend hold: the surplus
    rows are not stored (a canary behind the claimed end stays intact) and the status word says so."""
    w = W.config1()
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)     # 256 cached + 32 final rows
    x = W.warm_inputs(w)
    q_f, k_f, v_f = dev(x["q_f"]), dev(x["k_f"]), dev(x["v_f"])
    kc = torch.zeros(272, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    kc[:256] = dev(x["k_cache"]); vc = kc.clone()
    o = torch.full((32 + 8, w.n_q_heads, w.head_dim), 7.0, dtype=torch.float32, device="cuda")
    lse = torch.full((32 + 8, w.n_q_heads), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(B.BaError) as e:      # sizes that do not add up to the tables' rows: refused on the host
        B.ba_final_attend(c.ctx, q_f, k_f, v_f, 16, kc, vc, 256, None, 0, o, lse, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    assert e.value.status == B.BA_ERR_SHAPE
    # sizes that add up but split the rows differently from the tables: 16 final rows claimed, the tables say 32
    B.ba_final_attend(c.ctx, q_f, k_f, v_f, 16, kc, vc, 272, None, 0, o, lse, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    assert c.device_status() == B.BA_ERR_SHAPE
    assert (o[16:] == 7.0).all() and (lse[16:] == 7.0).all()
    assert c.device_status() == B.BA_OK
    c.close()


def test_deferred_table_and_split_partials_share_an_exactly_sized_workspace():
    """A context whose workspace is exactly what ba_workspace_bytes asks for: a queued re-encoding job
    with its own angle table rides along with a final-attend launch that splits its keys.  The partial
    results and the table must not overlap: both outputs equal those of the immediate calls."""
    w = W.config2()
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    Tc, Tf = t["n_cached_tokens"], t["n_final_tokens"]
    cfg = B.ba_config(w.n_q_heads, w.n_kv_heads, w.head_dim, B.BA_ROPE_ADJACENT, w.rope_theta, 0.0, 0)
    ctx = B.ba_create(cfg, 0, B.ba_workspace_bytes(cfg, w.n_blocks, Tf))
    tb = torch.empty(B.ba_segments_bytes(1, w.n_blocks, w.n_tokens), dtype=torch.uint8, device="cuda")
    lens, nb = np.asarray(w.block_lens, dtype=np.int32), np.asarray(w.seq_nblocks, dtype=np.int32)
    seg = B.ba_segment(ctx, lens, nb, 1, w.n_blocks, w.n_tokens, B.BA_MODE_BLOCK, tb)
    x = W.warm_inputs(w)
    q_f, k_f, v_f, kc, vc = (dev(x[k]) for k in ("q_f", "k_f", "v_f", "k_cache", "v_cache"))
    own_delta = torch.from_numpy(t["cache_delta"]).cuda()       # not the tables' array: the call builds its own table
    k_re = torch.empty_like(kc)
    B.ba_reencode_k(ctx, kc, None, Tc, k_re, seg.cache_cu, own_delta, seg.n_cached_blocks, Tc)
    o_want = torch.empty(Tf, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda")
    B.ba_final_attend(ctx, q_f, k_f, v_f, Tf, k_re, vc, Tc, None, 0, o_want, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    other = dev(W.warm_inputs(w, layer=1)["k_cache"])            # the next layer's cached keys
    want2 = torch.empty_like(other)
    B.ba_reencode_k(ctx, other, None, Tc, want2, seg.cache_cu, own_delta, seg.n_cached_blocks, Tc)
    got2 = torch.zeros_like(other)
    o_got = torch.empty_like(o_want)
    B.ba_reencode_k_deferred(ctx, other, None, Tc, got2, seg.cache_cu, own_delta, seg.n_cached_blocks, Tc)
    B.ba_final_attend(ctx, q_f, k_f, v_f, Tf, k_re, vc, Tc, None, 0, o_got, None, seg, B.BA_MODE_BLOCK, B.BA_OUT_F32)
    torch.cuda.synchronize()
    assert B.ba_last_device_status(ctx) == B.BA_OK
    assert torch.equal(got2, want2)
    # (the table takes room from the partial results, so the launch may use one split fewer than before:
    # same result up to the order of the fp32 sums)
    assert (o_got - o_want).abs().max().item() <= 1e-3
    o_ref, _ = ob.final_attend(W.bf16_bits_to_f64(x["q_f"]), W.bf16_bits_to_f64(x["k_f"]), W.bf16_bits_to_f64(x["v_f"]),
                               ob.reencode_blocks(W.bf16_bits_to_f64(x["k_cache"]), None, t["cache_cu"], t["cache_delta"],
                                                  w.rope_theta),
                               W.bf16_bits_to_f64(x["v_cache"]), w.block_lens, w.seq_nblocks)
    check_attention(o_got.cpu().numpy(), o_ref)
    B.ba_destroy(ctx)


def test_rotation_table_of_overwritten_tables_is_not_reused():
    """ba_reencode_k reuses the rotation table stored with the tables of the context's last ba_segment.
    When another context has rebuilt tables in the same buffer since (other lengths, other base), that
    table is foreign: the call must report it and rotate nothing."""
    w = W.config2()
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    x = W.warm_inputs(w)
    Tc = w.n_tokens - 64
    kc = dev(x["k_cache"])
    good = torch.zeros_like(kc)
    B.ba_reencode_k(c.ctx, kc, None, Tc, good, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    assert c.device_status() == B.BA_OK and good.any()
    other = R.Context(w.n_q_heads, w.n_kv_heads, w.head_dim, 1e4)          # another base
    lens2 = list(reversed(w.block_lens[:-1])) + [64]
    B.ba_segment(other.ctx, np.asarray(lens2, dtype=np.int32), np.asarray([11], dtype=np.int32), 1, 11, w.n_tokens,
                 B.BA_MODE_BLOCK, buf)
    out = torch.zeros_like(kc)
    B.ba_reencode_k(c.ctx, kc, None, Tc, out, seg.cache_cu, seg.cache_delta, seg.n_cached_blocks, Tc)
    assert c.device_status() == B.BA_ERR_INVALID_ARG
    assert not out.any()
    other.close()
    c.close()


def test_reencode_on_a_second_stream_beside_the_attention_gives_the_same_bits():
    """The serving loop the benchmark times: layer l+1 is re-encoded on a second stream (same context, the
    tables' own deltas: no workspace involved) while layer l attends on the first, with events in between.
    Outputs and re-encoded keys of every layer must be bit-identical to running everything on one stream."""
    w = W.config2()
    L = 6
    c = ctx_for(w)
    seg, buf = c.segment(w.block_lens, w.seq_nblocks, B.BA_MODE_BLOCK)
    t = ob.segment_tables(w.block_lens, w.seq_nblocks)
    Tc, Tf = t["n_cached_tokens"], t["n_final_tokens"]
    xs = [{k: dev(v) for k, v in W.warm_inputs(w, l).items()} for l in range(L)]
    def run(overlap):
        k_re = [torch.zeros(Tc, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda") for _ in range(L)]
        o = [torch.zeros(Tf, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device="cuda") for _ in range(L)]
        main = torch.cuda.Stream(priority=-1)
        side = torch.cuda.Stream(priority=0) if overlap else main
        start = torch.cuda.Event(); start.record(torch.cuda.current_stream())
        main.wait_event(start); side.wait_event(start)
        ev_re, ev_att = [], []
        def attend(l):
            main.wait_event(ev_re[l])
            B.ba_final_attend(c.ctx, xs[l]["q_f"], xs[l]["k_f"], xs[l]["v_f"], Tf, k_re[l], xs[l]["v_cache"], Tc, None, 0,
                              o[l], None, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16, stream=main)
            e = torch.cuda.Event(); e.record(main); ev_att.append(e)
        for l in range(L):
            if l >= 2:
                side.wait_event(ev_att[l - 2])
            B.ba_reencode_k(c.ctx, xs[l]["k_cache"], None, Tc, k_re[l], seg.cache_cu, seg.cache_delta,
                            seg.n_cached_blocks, Tc, stream=side)
            e = torch.cuda.Event(); e.record(side); ev_re.append(e)
            if l >= 1:
                attend(l - 1)
        attend(L - 1)
        torch.cuda.synchronize()
        return k_re, o
    k1, o1 = run(False)
    for _ in range(3):
        k2, o2 = run(True)
        for l in range(L):
            assert torch.equal(k1[l], k2[l]) and torch.equal(o1[l], o2[l]), l
    assert c.device_status() == B.BA_OK
    o_ref, _ = ob.final_attend(*(W.bf16_bits_to_f64(W.warm_inputs(w, 3)[k]) for k in ("q_f", "k_f", "v_f")),
                               ob.reencode_blocks(W.bf16_bits_to_f64(W.warm_inputs(w, 3)["k_cache"]), None, t["cache_cu"],
                                                  t["cache_delta"], w.rope_theta),
                               W.bf16_bits_to_f64(W.warm_inputs(w, 3)["v_cache"]), w.block_lens, w.seq_nblocks)
    check_attention(o1[3].float().cpu().numpy(), o_ref, bf16_store=True)
    c.close()
