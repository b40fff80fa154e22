"""Pins of the CPU oracle against what the paper and the mathematics fix.

The paper prints no numeric worked example of the path, so the oracle is tied
down by: brute force written as explicit per-pair loops (independent of the
oracle's vectorised code), closed forms (zero queries give prefix means,
constant values pass through), the invariants Section 2.3 states (Eq. 2 undoes
Eq. 1; zero-then-rotate equals one rotation by the difference; caching at
position zero is legal because RoPE scores depend on position differences), the
mask rules of Sections 1, 2.1 and 2.4 (one block is full causal attention; a
non-final block equals attention over that block alone; final rows are the same
in both modes), a library routine for the full-causal special case, and the
FLOPs figures of Table 3.
"""
import cmath
import math
import os

import numpy as np
import pytest

from oracle import block_attention as ob

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rnd(seed, *shape):
    return np.random.default_rng(seed).standard_normal(shape)


# --------------------------------------------------------------------------- brute force
def brute_attention(q, k, v, seqs, mode):
    """seqs: list of lists of block lengths.  Pure loops; the mask rule is
    spelled out per (i, j) pair from Sections 1 / 2.1 / 2.4."""
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    o = np.zeros((T, Hq, d))
    lse = np.zeros((T, Hq))
    tok = []  # (sequence, block-in-sequence, is_final)
    for s, lens in enumerate(seqs):
        for bi, L in enumerate(lens):
            tok += [(s, bi, bi == len(lens) - 1)] * L
    for i in range(T):
        si, bi, fin = tok[i]
        allowed = []
        for j in range(i + 1):
            sj, bj, _ = tok[j]
            if sj != si:
                continue
            if mode == ob.MODE_FULL or bj == bi or fin:
                allowed.append(j)
        for h in range(Hq):
            g = h // G
            sc = [sum(q[i, h, c] * k[j, g, c] for c in range(d)) / math.sqrt(d) for j in allowed]
            mx = max(sc)
            w = [math.exp(x - mx) for x in sc]
            z = sum(w)
            for c in range(d):
                o[i, h, c] = sum(wj * v[j, g, c] for wj, j in zip(w, allowed)) / z
            lse[i, h] = mx + math.log(z)
    return o, lse


@pytest.mark.parametrize("mode", [ob.MODE_BLOCK, ob.MODE_FULL])
@pytest.mark.parametrize("seqs", [[[2, 3, 1]], [[1, 1], [3, 2, 2]], [[4]], [[1], [1, 1, 1]]])
def test_brute_force_tiny(seqs, mode):
    lens = [l for s in seqs for l in s]
    nb = [len(s) for s in seqs]
    T = sum(lens)
    q, k, v = rnd(1, T, 4, 4), rnd(2, T, 2, 4), rnd(3, T, 2, 4)
    o, lse = ob.block_prefill(q, k, v, lens, nb, mode)
    o_ref, lse_ref = brute_attention(q, k, v, seqs, mode)
    np.testing.assert_allclose(o, o_ref, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref, atol=1e-12)


def test_brute_force_final_attend():
    seqs = [[2, 3, 2], [1, 2]]
    lens = [l for s in seqs for l in s]
    nb = [len(s) for s in seqs]
    T = sum(lens)
    q, k, v = rnd(4, T, 4, 4), rnd(5, T, 2, 4), rnd(6, T, 2, 4)
    t = ob.segment_tables(lens, nb)
    fin = t["block_is_final"][t["tok_block"]].astype(bool)
    o_ref, lse_ref = brute_attention(q, k, v, seqs, ob.MODE_BLOCK)
    o, lse = ob.final_attend(q[fin], k[fin], v[fin], k[~fin], v[~fin], lens, nb)
    np.testing.assert_allclose(o, o_ref[fin], atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref[fin], atol=1e-12)


# --------------------------------------------------------------------------- tables
def test_tables_hand_example():
    # two sequences: [2,3,1] and [1,2]; written out by hand
    t = ob.segment_tables([2, 3, 1, 1, 2], [3, 2], ob.MODE_BLOCK)
    assert t["cu_seq"].tolist() == [0, 6, 9]
    assert t["cu_block"].tolist() == [0, 2, 5, 6, 7, 9]
    assert t["tok_block"].tolist() == [0, 0, 1, 1, 1, 2, 3, 4, 4]
    assert t["tok_pos"].tolist() == [0, 1, 2, 3, 4, 5, 0, 1, 2]
    assert t["tok_pos_local"].tolist() == [0, 1, 0, 1, 2, 0, 0, 0, 1]
    assert t["block_delta"].tolist() == [0, 2, 5, 0, 1]
    assert t["block_is_final"].tolist() == [0, 0, 1, 0, 1]
    assert t["block_seq"].tolist() == [0, 0, 0, 1, 1]
    assert t["block_kv_begin"].tolist() == [0, 2, 0, 6, 6]
    assert t["block_part_off"].tolist() == [0, 2, 0, 5, 1]
    assert t["cu_cache_seq"].tolist() == [0, 5, 6]
    assert t["cu_final_seq"].tolist() == [0, 1, 3]
    assert t["cache_block"].tolist() == [0, 1, 3]
    assert t["cache_cu"].tolist() == [0, 2, 5, 6]
    assert t["cache_delta"].tolist() == [0, 2, 0]
    f = ob.segment_tables([2, 3, 1, 1, 2], [3, 2], ob.MODE_FULL)
    assert f["block_kv_begin"].tolist() == [0, 0, 0, 6, 6]
    for key in ("cu_block", "tok_pos", "block_delta", "block_is_final", "cache_cu"):
        assert f[key].tolist() == t[key].tolist()


def test_tables_tiny_config_offsets():
    # 4 cached blocks of 64 are re-encoded to offsets 0,64,128,192; the final block
    # of 32 sits at positions 256..287
    t = ob.segment_tables([64, 64, 64, 64, 32], [5])
    assert t["cache_delta"].tolist() == [0, 64, 128, 192]
    assert t["tok_pos"][256:].tolist() == list(range(256, 288))
    assert t["block_is_final"].tolist() == [0, 0, 0, 0, 1]


def test_tables_match_mask():
    lens, nb = [3, 1, 4, 2, 2, 5, 1], [3, 1, 3]
    for mode in (ob.MODE_BLOCK, ob.MODE_FULL):
        t = ob.segment_tables(lens, nb, mode)
        m = ob.dense_mask(lens, nb, mode)
        T = sum(lens)
        for i in range(T):
            lo = t["block_kv_begin"][t["tok_block"][i]]
            expect = np.zeros(T, bool)
            expect[lo:i + 1] = True
            assert (m[i] == expect).all()
        assert int(m.sum()) == ob.allowed_pairs(lens, nb, mode)


def test_tables_reject_bad_input():
    with pytest.raises(ValueError):
        ob.segment_tables([3, 0], [2])
    with pytest.raises(ValueError):
        ob.segment_tables([3, 1], [3])


# --------------------------------------------------------------------------- RoPE
def test_rope_is_complex_multiplication():
    # RoPE's closed form: pair m as a complex number is multiplied by exp(i p theta_m)
    d, base = 8, 10000.0
    x = rnd(7, 5, d)
    pos = np.array([0, 1, 7, 100, 32767])
    y = ob.rotate(x, pos[:, None][:, 0], base, ob.ROPE_ADJACENT)
    for r in range(5):
        for m in range(d // 2):
            z = complex(x[r, 2 * m], x[r, 2 * m + 1]) * cmath.exp(1j * pos[r] * base ** (-2.0 * m / d))
            assert abs(y[r, 2 * m] - z.real) < 1e-9 and abs(y[r, 2 * m + 1] - z.imag) < 1e-9
    yh = ob.rotate(x, pos, base, ob.ROPE_HALF)
    for r in range(5):
        for m in range(d // 2):
            z = complex(x[r, m], x[r, m + d // 2]) * cmath.exp(1j * pos[r] * base ** (-2.0 * m / d))
            assert abs(yh[r, m] - z.real) < 1e-9 and abs(yh[r, m + d // 2] - z.imag) < 1e-9


def test_rope_matrix_is_eq1_and_rotate_applies_it():
    d, base = 6, 100.0
    R = ob.rope_matrix(3, d, base)
    th = [base ** (-2.0 * m / d) for m in range(3)]
    expect = np.zeros((d, d))
    for m in range(3):
        c, s = math.cos(3 * th[m]), math.sin(3 * th[m])
        expect[2 * m, 2 * m], expect[2 * m, 2 * m + 1] = c, -s
        expect[2 * m + 1, 2 * m], expect[2 * m + 1, 2 * m + 1] = s, c
    np.testing.assert_allclose(R, expect, atol=1e-15)
    x = rnd(8, 4, d)
    np.testing.assert_allclose(ob.rotate(x, np.full(4, 3.0), base), x @ R.T, atol=1e-14)
    # Eq. 2's matrix is the transpose of Eq. 1's and undoes it
    np.testing.assert_allclose(ob.rotate(x, np.full(4, 3.0), base, inverse=True), x @ R, atol=1e-14)
    np.testing.assert_allclose(R.T @ R, np.eye(d), atol=1e-14)


@pytest.mark.parametrize("layout", [ob.ROPE_ADJACENT, ob.ROPE_HALF])
def test_reencode_equals_rope_at_new_position(layout):
    # keys rotated at 0..L-1 then re-encoded by p equal keys rotated at p..p+L-1
    L, H, d, base, p = 9, 2, 16, 500000.0, 1234
    raw = rnd(9, L, H, d)
    t = np.arange(L, dtype=float)[:, None]
    cached = ob.rotate(raw, t, base, layout)
    direct = ob.rotate(raw, t + p, base, layout)
    np.testing.assert_allclose(ob.reencode_literal(cached, p, base, layout), direct, atol=1e-10)
    np.testing.assert_allclose(ob.reencode_delta(cached, p, base, layout), direct, atol=1e-10)
    # delta zero is the identity; negative delta is Eq. 2 (back towards zero)
    np.testing.assert_allclose(ob.reencode_literal(cached, 0, base, layout), cached, atol=1e-13)
    assert (ob.reencode_delta(cached, 0, base, layout) == cached).all()
    np.testing.assert_allclose(ob.reencode_delta(direct, -p, base, layout), cached, atol=1e-10)
    # rotations keep each pair's norm
    ix, iy = ob.rope_pairs(d, layout)
    n0 = cached[..., ix] ** 2 + cached[..., iy] ** 2
    n1 = ob.reencode_literal(cached, p, base, layout)
    np.testing.assert_allclose(n1[..., ix] ** 2 + n1[..., iy] ** 2, n0, rtol=1e-12)


def test_reencode_blocks_gather_and_offsets():
    H, d, base = 2, 8, 10000.0
    pool = rnd(10, 20, H, d)
    cache_cu, cache_delta, src_off = [0, 3, 8], [0, 3], [12, 2]
    out = ob.reencode_blocks(pool, src_off, cache_cu, cache_delta, base)
    np.testing.assert_allclose(out[0:3], pool[12:15], atol=1e-13)
    np.testing.assert_allclose(out[3:8], ob.reencode_delta(pool[2:7], 3, base), atol=1e-12)
    packed = ob.reencode_blocks(pool[:8], None, cache_cu, cache_delta, base)
    np.testing.assert_allclose(packed[3:8], ob.reencode_delta(pool[3:8], 3, base), atol=1e-12)


def test_layout_flag_is_a_permutation():
    # adjacent vs half-split pairing with correspondingly permuted q, k gives identical scores
    d, base = 8, 10000.0
    q, k = rnd(11, 3, d), rnd(12, 3, d)
    perm = np.concatenate([np.arange(0, d, 2), np.arange(1, d, 2)])  # adjacent -> half
    pos = np.array([5.0, 17.0, 40.0])
    qa, ka = ob.rotate(q, pos, base, ob.ROPE_ADJACENT), ob.rotate(k, pos, base, ob.ROPE_ADJACENT)
    qh, kh = ob.rotate(q[:, perm], pos, base, ob.ROPE_HALF), ob.rotate(k[:, perm], pos, base, ob.ROPE_HALF)
    np.testing.assert_allclose(qa @ ka.T, qh @ kh.T, atol=1e-12)
    np.testing.assert_allclose(qa[:, perm], qh, atol=1e-13)


# --------------------------------------------------------------------------- mask rules
def test_single_block_is_full_causal_and_matches_library():
    import torch
    T, Hq, Hkv, d = 37, 4, 2, 16
    q, k, v = rnd(13, T, Hq, d), rnd(14, T, Hkv, d), rnd(15, T, Hkv, d)
    ob_block, lse_b = ob.block_prefill(q, k, v, [T], [1], ob.MODE_BLOCK)
    ob_full, lse_f = ob.block_prefill(q, k, v, [T], [1], ob.MODE_FULL)
    assert (ob_block == ob_full).all() and (lse_b == lse_f).all()
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    tv = torch.from_numpy(v).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    np.testing.assert_allclose(ob_full, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)
    # full mode on several blocks is also plain causal attention over the sequence
    o2, _ = ob.block_prefill(q, k, v, [10, 20, 7], [3], ob.MODE_FULL)
    np.testing.assert_allclose(o2, ob_full, atol=1e-13)


def test_nonfinal_block_equals_attention_over_that_block_alone():
    lens, nb = [5, 9, 3, 4, 6], [3, 2]
    T = sum(lens)
    q, k, v = rnd(16, T, 4, 8), rnd(17, T, 2, 8), rnd(18, T, 2, 8)
    o, lse = ob.block_prefill(q, k, v, lens, nb, ob.MODE_BLOCK)
    t = ob.segment_tables(lens, nb)
    for b in range(len(lens)):
        if t["block_is_final"][b]:
            continue
        lo, hi = t["cu_block"][b], t["cu_block"][b + 1]
        o1, l1 = ob.block_prefill(q[lo:hi], k[lo:hi], v[lo:hi], [hi - lo], [1], ob.MODE_FULL)
        np.testing.assert_allclose(o[lo:hi], o1, atol=1e-13)
        np.testing.assert_allclose(lse[lo:hi], l1, atol=1e-13)


def test_final_rows_same_in_both_modes_and_final_attend_agrees():
    lens, nb = [5, 9, 3, 4, 6], [3, 2]
    T = sum(lens)
    q, k, v = rnd(19, T, 4, 8), rnd(20, T, 2, 8), rnd(21, T, 2, 8)
    ob_, _ = ob.block_prefill(q, k, v, lens, nb, ob.MODE_BLOCK)
    of_, _ = ob.block_prefill(q, k, v, lens, nb, ob.MODE_FULL)
    t = ob.segment_tables(lens, nb)
    fin = t["block_is_final"][t["tok_block"]].astype(bool)
    np.testing.assert_allclose(ob_[fin], of_[fin], atol=1e-13)
    assert np.abs(ob_[~fin] - of_[~fin]).max() > 1e-3      # and the other rows do differ
    for mode in (ob.MODE_BLOCK, ob.MODE_FULL):
        o, _ = ob.final_attend(q[fin], k[fin], v[fin], k[~fin], v[~fin], lens, nb, mode)
        np.testing.assert_allclose(o, of_[fin], atol=1e-13)


def test_zero_queries_give_prefix_means():
    lens, nb = [3, 4, 2], [3]
    T = sum(lens)
    v = rnd(22, T, 2, 4)
    q, k = np.zeros((T, 4, 4)), rnd(23, T, 2, 4)
    o, lse = ob.block_prefill(q, k, v, lens, nb, ob.MODE_BLOCK)
    starts = [0, 0, 0, 3, 3, 3, 3, 0, 0]     # non-final rows: own block; final rows: everything
    for i in range(T):
        for h in range(4):
            np.testing.assert_allclose(o[i, h], v[starts[i]:i + 1, h // 2].mean(axis=0), atol=1e-14)
            assert abs(lse[i, h] - math.log(i + 1 - starts[i])) < 1e-14


def test_constant_values_pass_through_and_split_kv_combines():
    T = 23
    q, k = rnd(24, T, 2, 8), rnd(25, T, 1, 8)
    v = np.tile(rnd(26, 1, 1, 8), (T, 1, 1))
    o, _ = ob.block_prefill(q, k, v, [T], [1], ob.MODE_FULL)
    np.testing.assert_allclose(o, np.broadcast_to(v[:1], o.shape), atol=1e-14)
    # splitting the keys and merging partial results by their log-sum-exp is exact
    v = rnd(27, T, 1, 8)
    row = q[-1:]
    full_mask = np.ones((1, T), bool)
    o_all, l_all = ob.attention_rows(row, k, v, full_mask)
    o_a, l_a = ob.attention_rows(row, k[:9], v[:9], full_mask[:, :9])
    o_b, l_b = ob.attention_rows(row, k[9:], v[9:], full_mask[:, 9:])
    l = np.logaddexp(l_a, l_b)
    merged = o_a * np.exp(l_a - l)[..., None] + o_b * np.exp(l_b - l)[..., None]
    np.testing.assert_allclose(merged, o_all, atol=1e-13)
    np.testing.assert_allclose(l, l_all, atol=1e-13)


def test_caching_at_position_zero_is_legal():
    # block-local outputs do not change when q, k of a block are encoded at the block's
    # prompt positions instead of its local positions (RoPE scores depend on differences)
    L, d, base, p = 11, 16, 10000.0, 300
    raw_q, raw_k, v = rnd(28, L, 2, d), rnd(29, L, 1, d), rnd(30, L, 1, d)
    t = np.arange(L, dtype=float)[:, None]
    o_local, _ = ob.block_prefill(ob.rotate(raw_q, t, base), ob.rotate(raw_k, t, base), v, [L], [1], 0)
    o_prompt, _ = ob.block_prefill(ob.rotate(raw_q, t + p, base), ob.rotate(raw_k, t + p, base), v, [L], [1], 0)
    np.testing.assert_allclose(o_local, o_prompt, atol=1e-10)


def test_warm_path_equals_prefill_with_direct_rope():
    # fetch cached K (positions 0..L-1) -> re-encode -> final attend  ==  final rows of a
    # prefill whose K was rotated at prompt positions from the start
    lens, nb, d, base = [4, 6, 3], [3], 8, 10000.0
    T = sum(lens)
    raw_k, v, q = rnd(31, T, 1, d), rnd(32, T, 1, d), rnd(33, T, 2, d)
    t = ob.segment_tables(lens, nb)
    k_prompt = ob.rotate(raw_k, t["tok_pos"][:, None].astype(float), base)
    k_cache = ob.rotate(raw_k, t["tok_pos_local"][:, None].astype(float), base)
    fin = t["block_is_final"][t["tok_block"]].astype(bool)
    k_re = ob.reencode_blocks(k_cache[~fin], None, t["cache_cu"], t["cache_delta"], base)
    np.testing.assert_allclose(k_re, k_prompt[~fin], atol=1e-12)
    o_warm, _ = ob.final_attend(q[fin], k_prompt[fin], v[fin], k_re, v[~fin], lens, nb)
    o_cold, _ = ob.block_prefill(q, k_prompt, v, lens, nb, ob.MODE_BLOCK)
    np.testing.assert_allclose(o_warm, o_cold[fin], atol=1e-12)


def test_reencoding_may_be_applied_to_the_query_side():
    # Eq. 3 after Eq. 2 is one rotation R(delta) of the cached key; rotations are orthogonal, so
    # q . (R(delta) k) = (R(-delta) q) . k: the logits of a cached block against the re-encoded keys
    # equal those of the counter-rotated queries against the keys as cached (both RoPE layouts).
    d, base = 8, 10000.0
    for layout in (ob.ROPE_ADJACENT, ob.ROPE_HALF):
        q, k = rnd(41, 5, 2, d), rnd(42, 7, 2, d)
        for delta in (0, 3, 250, 31000):
            k_re = ob.reencode_delta(k, delta, base, layout)
            q_rot = ob.rotate(q, np.full((5, 1), float(delta)), base, layout, inverse=True)
            lhs = np.einsum("ihd,jhd->hij", q, k_re)
            rhs = np.einsum("ihd,jhd->hij", q_rot, k)
            np.testing.assert_allclose(lhs, rhs, atol=1e-10)


# --------------------------------------------------------------------------- Table 3
def test_table3_flops_exclude_attention_scores():
    # FLOPs-TFT = 2 * (about 7.5e9 parameters) * (tokens encoded): 50 tokens under
    # Block-attention at every length, the whole prompt under full attention.
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table3_flops.txt")) if l[0] != "#"]
    per_token = float(rows[0][2]) / 50
    assert abs(per_token / 2 - 7.5e9) / 7.5e9 < 0.01
    for r in rows:
        n, vanilla, block = int(r[0]), float(r[1]), float(r[2])
        assert block == 7.5e11
        assert abs(vanilla - per_token * n) / vanilla < 0.03


# --------------------------------------------------------------------------- planted mistakes
def _fails(fn, *args):
    try:
        fn(*args)
    except AssertionError:
        return True
    return False


def test_pins_catch_planted_mistakes(monkeypatch):
    """Mistakes are planted in the oracle (never in the CUDA path) and each must
    trip at least one pin above."""
    seqs = [[1, 1], [3, 2, 2]]
    # wrong rotation sign
    good_rotate = ob.rotate
    monkeypatch.setattr(ob, "rotate", lambda x, p, b, layout=0, inverse=False:
                        good_rotate(x, p, b, layout, not inverse))
    assert _fails(test_rope_is_complex_multiplication)
    monkeypatch.setattr(ob, "rotate", good_rotate)
    # wrong frequency exponent (dropped factor two)
    good_theta = ob.rope_theta
    monkeypatch.setattr(ob, "rope_theta", lambda d, base: np.float64(base) ** (-np.arange(d // 2) / d))
    assert _fails(test_rope_is_complex_multiplication)
    monkeypatch.setattr(ob, "rope_theta", good_theta)
    # wrong grouped-query head mapping
    good_rows = ob.attention_rows

    def bad_gqa(q_rows, k, v, mask, scale=None):
        Hq, Hkv = q_rows.shape[1], k.shape[1]
        perm = [(h % Hkv) for h in range(Hq)]
        return good_rows(q_rows, k[:, perm], v[:, perm], mask, scale)
    monkeypatch.setattr(ob, "attention_rows", bad_gqa)
    assert _fails(test_brute_force_tiny, seqs, ob.MODE_BLOCK)
    # missing softmax scale
    monkeypatch.setattr(ob, "attention_rows", lambda q, k, v, m, scale=None: good_rows(q, k, v, m, 1.0))
    assert _fails(test_brute_force_tiny, seqs, ob.MODE_BLOCK)
    monkeypatch.setattr(ob, "attention_rows", good_rows)
    # final block forgets the earlier blocks
    good_mask = ob.mask_rows

    def bad_mask(block_lens, seq_nblocks, mode, rows, cols=None):
        m = good_mask(block_lens, seq_nblocks, ob.MODE_FULL, rows, cols)
        blk = np.repeat(np.arange(len(block_lens)), block_lens)
        c0, c1 = (0, len(blk)) if cols is None else cols
        return m & (blk[None, c0:c1] == blk[np.asarray(rows)][:, None]) if mode == ob.MODE_BLOCK else m
    monkeypatch.setattr(ob, "mask_rows", bad_mask)
    assert _fails(test_brute_force_tiny, seqs, ob.MODE_BLOCK)
    assert _fails(test_zero_queries_give_prefix_means)
    monkeypatch.setattr(ob, "mask_rows", good_mask)
    # delta taken from the wrong block
    good_tables = ob.segment_tables

    def bad_tables(block_lens, seq_nblocks, mode=0):
        t = good_tables(block_lens, seq_nblocks, mode)
        t["cache_delta"] = np.roll(t["cache_delta"], 1)
        return t
    monkeypatch.setattr(ob, "segment_tables", bad_tables)
    assert _fails(test_warm_path_equals_prefill_with_direct_rope)
    assert _fails(test_tables_hand_example)


def test_paged_rows_gather_reproduces_the_contiguous_cache():
    """A paged pool is an indexing scheme only: gathering the rows the page table names gives back the
    packed cache, whatever the page size and page order; checked against a hand-written table and
    against per-row brute force."""
    from paper_2409_15355_b200 import workloads as W
    # hand-written: blocks of 5 and 3 rows, pages of 4 rows; block 0 -> pages 2, 0; block 1 -> page 3
    rows = ob.paged_rows([5, 3], 4, [0, 2, 3], [2, 0, 3])
    assert rows.tolist() == [8, 9, 10, 11, 0, 12, 13, 14]
    lens = [37, 1, 16, 130, 64]
    packed = W.normal_bf16(3, (sum(lens), 2, 8))
    for page_rows in (16, 32, 128):
        pool, page_cu, page_idx, n_pages = W.scatter_into_pages(packed, lens, page_rows, seed=9)
        assert pool.shape[0] == n_pages * page_rows and len(set(page_idx.tolist())) == len(page_idx)
        got = pool[ob.paged_rows(lens, page_rows, page_cu, page_idx)]
        assert np.array_equal(got, packed)
        # brute force, row by row
        r = 0
        for c, L in enumerate(lens):
            for t in range(L):
                g = page_idx[page_cu[c] + t // page_rows]
                assert np.array_equal(pool[g * page_rows + t % page_rows], packed[r])
                r += 1


# --------------------------------------------------------------------------- backward pass
def _tiny_backward_case(seed=0, lens=(3, 2, 2), nbs=(2, 1), Hq=4, Hkv=2, d=4):
    rng = np.random.default_rng(seed)
    T = sum(lens)
    q, g = rng.standard_normal((T, Hq, d)), rng.standard_normal((T, Hq, d))
    k, v = rng.standard_normal((T, Hkv, d)), rng.standard_normal((T, Hkv, d))
    return list(lens), list(nbs), q, k, v, g


@pytest.mark.parametrize("mode", [ob.MODE_BLOCK, ob.MODE_FULL])
def test_backward_matches_central_finite_differences(mode):
    """dQ, dK, dV against (L(x + e) - L(x - e)) / 2e of L = sum(dO * O), element by element, on a tiny
    two-sequence layout with grouped heads: a dropped term, a wrong sign, a missing scale or a wrong
    head-to-group map each change some entry by far more than the 1e-6 allowed."""
    lens, nbs, q, k, v, g = _tiny_backward_case()
    dq, dk, dv = ob.block_prefill_backward(q, k, v, g, lens, nbs, mode)
    loss = lambda q_, k_, v_: float((ob.block_prefill(q_, k_, v_, lens, nbs, mode)[0] * g).sum())
    eps = 1e-6
    for name, x, dx in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        num = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps; xm[idx] -= eps
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            num[idx] = (loss(*args_p) - loss(*args_m)) / (2 * eps)
        assert np.abs(num - dx).max() <= 1e-6, (name, np.abs(num - dx).max())


def test_backward_single_block_matches_library_autograd():
    """One block is ordinary causal attention: gradients equal those torch's autograd gives for its
    scaled-dot-product attention in fp64 (grouped heads expanded for the library call)."""
    import torch
    rng = np.random.default_rng(5)
    L, Hq, Hkv, d = 9, 4, 2, 8
    q, g = rng.standard_normal((L, Hq, d)), rng.standard_normal((L, Hq, d))
    k, v = rng.standard_normal((L, Hkv, d)), rng.standard_normal((L, Hkv, d))
    for mode in (ob.MODE_BLOCK, ob.MODE_FULL):
        dq, dk, dv = ob.block_prefill_backward(q, k, v, g, [L], [1], mode)
        tq = torch.tensor(q.transpose(1, 0, 2), requires_grad=True)
        tk = torch.tensor(k.transpose(1, 0, 2), requires_grad=True)
        tv = torch.tensor(v.transpose(1, 0, 2), requires_grad=True)
        o = torch.nn.functional.scaled_dot_product_attention(tq, tk.repeat_interleave(Hq // Hkv, 0),
                                                             tv.repeat_interleave(Hq // Hkv, 0), is_causal=True)
        (o * torch.tensor(g.transpose(1, 0, 2))).sum().backward()
        assert np.abs(tq.grad.numpy().transpose(1, 0, 2) - dq).max() <= 1e-10
        assert np.abs(tk.grad.numpy().transpose(1, 0, 2) - dk).max() <= 1e-10
        assert np.abs(tv.grad.numpy().transpose(1, 0, 2) - dv).max() <= 1e-10


def test_backward_of_a_nonfinal_block_stays_inside_it():
    """Rows of a non-final block see only their own block, so a loss on those rows alone gives no
    gradient to keys and values outside the block (nor to other queries) and equals the gradient of
    attention over that block taken alone; in full mode the same loss does reach the earlier blocks."""
    lens, nbs, q, k, v, g = _tiny_backward_case(seed=3, lens=(4, 3, 5), nbs=(3,), Hq=2, Hkv=1, d=4)
    gm = np.zeros_like(g); gm[4:7] = g[4:7]                       # block 1 (rows 4..6), non-final
    dq, dk, dv = ob.block_prefill_backward(q, k, v, gm, lens, nbs, ob.MODE_BLOCK)
    outside = np.r_[0:4, 7:12]
    assert not dq[outside].any() and not dk[outside].any() and not dv[outside].any()
    aq, ak, av = ob.block_prefill_backward(q[4:7], k[4:7], v[4:7], g[4:7], [3], [1], ob.MODE_BLOCK)
    assert np.abs(dq[4:7] - aq).max() <= 1e-14 and np.abs(dk[4:7] - ak).max() <= 1e-14 and np.abs(dv[4:7] - av).max() <= 1e-14
    fq, fk, fv = ob.block_prefill_backward(q, k, v, gm, lens, nbs, ob.MODE_FULL)
    assert fk[0:4].any() and fv[0:4].any()
    # a loss on the final block reaches every earlier block in both modes
    gf = np.zeros_like(g); gf[7:] = g[7:]
    _, dk2, dv2 = ob.block_prefill_backward(q, k, v, gf, lens, nbs, ob.MODE_BLOCK)
    assert dk2[0:4].any() and dv2[4:7].any()


def test_backward_pins_catch_planted_mistakes(monkeypatch):
    good = ob.attention_rows_backward

    def no_jacobian_term(q_rows, k, v, mask, d_o, scale=None):     # dS = P * dP: the row term of the softmax Jacobian dropped
        n, Hq, d = q_rows.shape
        G = Hq // k.shape[1]
        sc = 1.0 / np.sqrt(d) if scale is None else scale
        dq, dk, dv = np.zeros_like(q_rows), np.zeros_like(k), np.zeros_like(v)
        for h in range(Hq):
            g = h // G
            s = (q_rows[:, h] @ k[:, g].T) * sc + np.where(mask, 0.0, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True)); p /= p.sum(axis=1, keepdims=True)
            dv[:, g] += p.T @ d_o[:, h]
            ds = p * (d_o[:, h] @ v[:, g].T)
            dq[:, h] = (ds @ k[:, g]) * sc
            dk[:, g] += (ds.T @ q_rows[:, h]) * sc
        return dq, dk, dv
    monkeypatch.setattr(ob, "attention_rows_backward", no_jacobian_term)
    assert _fails(test_backward_matches_central_finite_differences, ob.MODE_BLOCK)
    monkeypatch.setattr(ob, "attention_rows_backward", lambda q, k, v, m, g, scale=None: good(q, k, v, m, g, 1.0))
    assert _fails(test_backward_matches_central_finite_differences, ob.MODE_BLOCK)
    assert _fails(test_backward_single_block_matches_library_autograd)

    def swapped_groups(q_rows, k, v, mask, d_o, scale=None):
        dq, dk, dv = good(q_rows, k, v, mask, d_o, scale)
        return dq, dk[:, ::-1], dv
    monkeypatch.setattr(ob, "attention_rows_backward", swapped_groups)
    assert _fails(test_backward_matches_central_finite_differences, ob.MODE_FULL)
