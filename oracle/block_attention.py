"""CPU oracle for the Block-attention prefilling hot path (arXiv 2409.15355).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, fp64 restatement of what
the paper defines; it exists so that the CUDA library can be checked against
something written independently of it.  Only the test-suite, the smoke check
and the CPU-baseline leg of the benchmark may import it.  It shares no code,
tables or constants with the CUDA path and never imports it.

What is computed, and where the paper defines it:

* segment tables      -- Section 2.2 (one passage = one block, the user query
                         is the final block) and Section 2.5 (a block's new
                         positions follow from its place in the prompt).
* the attention mask  -- Section 1 / Section 2.1 / Section 2.4: a token of a
                         non-final block attends only inside its own block; a
                         token of the final block attends every earlier token;
                         the base mask is the usual lower-triangular one.
* RoPE re-encoding    -- Section 2.3, Eq. 1 (rotation to position i), Eq. 2
                         (inverse rotation, back to position zero), Eq. 3
                         (rotation to the new position).
* backward pass       -- Section 2.4 (block fine-tune): gradients of that attention
                         under the same mask, by the softmax Jacobian.
* attention           -- plain softmax(Q K^T / sqrt(d)) V under that mask, with
                         grouped-query heads (query head h reads KV head
                         floor(h / G)).  The paper keeps the model's attention
                         and only changes the mask, so this is the definition.

Readings of points the paper leaves open are listed where they are used.
All functions have at least one pin in tests/test_oracle_pins.py (brute force
on tiny inputs, closed forms, invariants, or a library routine for a special
case); none is "parity unpinned" except the numeric values of attention on
random inputs, for which the paper prints no worked example.
"""
from __future__ import annotations

import numpy as np

MODE_BLOCK = 0
MODE_FULL = 1
ROPE_ADJACENT = 0   # Eq. 1 pairs coordinates (2m, 2m+1)
ROPE_HALF = 1       # pairs (m, m + d/2), the other common convention


# ---------------------------------------------------------------------------
# Segment tables (Section 2.2, Section 2.5)
# ---------------------------------------------------------------------------
def segment_tables(block_lens, seq_nblocks, mode=MODE_BLOCK):
    """Offsets, positions and visibility ranges from block lengths.

    Blocks are listed in prompt order; sequence s owns seq_nblocks[s]
    consecutive blocks and its last block is the final block (Section 2.2).
    A token's prompt position counts tokens from the start of its sequence,
    exactly as under full attention (Section 2.5: positions follow the block's
    place in the input).  A cached block holds positions 0..L-1 (Section 2.3:
    the first token of each cached block is standardised to zero), so the
    re-encoding delta of a block is the prompt position of its first token.

    block_kv_begin[b] is the first key row (in the packed prompt) that rows of
    block b may see: the block's own start for a non-final block in block mode,
    the sequence start for a final block and for every block in full mode.
    """
    block_lens = [int(x) for x in block_lens]
    seq_nblocks = [int(x) for x in seq_nblocks]
    if any(l < 1 for l in block_lens) or any(n < 1 for n in seq_nblocks):
        raise ValueError("block lengths and block counts must be >= 1")
    if sum(seq_nblocks) != len(block_lens):
        raise ValueError("seq_nblocks does not add up to the number of blocks")
    B, batch, T = len(block_lens), len(seq_nblocks), sum(block_lens)
    cu_seq = [0]
    cu_block = [0]
    cu_cache_seq = [0]
    cu_final_seq = [0]
    tok_block, tok_pos, tok_pos_local = [], [], []
    block_delta, block_is_final, block_seq = [], [], []
    block_kv_begin, block_part_off = [], []
    cache_block, cache_cu, cache_delta = [], [0], []
    b = 0
    n_cache = 0
    n_final = 0
    for s in range(batch):
        pos = 0
        seq_start = cu_block[-1]
        for j in range(seq_nblocks[s]):
            L = block_lens[b]
            final = (j == seq_nblocks[s] - 1)
            start = cu_block[-1]
            block_delta.append(pos)
            block_is_final.append(1 if final else 0)
            block_seq.append(s)
            if mode == MODE_FULL or final:
                block_kv_begin.append(seq_start)
            else:
                block_kv_begin.append(start)
            if final:
                block_part_off.append(n_final)
                n_final += L
            else:
                block_part_off.append(n_cache)
                cache_block.append(b)
                cache_delta.append(pos)
                n_cache += L
                cache_cu.append(n_cache)
            for t in range(L):
                tok_block.append(b)
                tok_pos.append(pos + t)
                tok_pos_local.append(t)
            pos += L
            cu_block.append(start + L)
            b += 1
        cu_seq.append(cu_block[-1])
        cu_cache_seq.append(n_cache)
        cu_final_seq.append(n_final)
    i32 = lambda a: np.asarray(a, dtype=np.int32)
    return dict(
        batch=batch, n_blocks=B, n_tokens=T, n_cached_blocks=len(cache_block),
        n_cached_tokens=n_cache, n_final_tokens=n_final, mode=mode,
        cu_seq=i32(cu_seq), cu_cache_seq=i32(cu_cache_seq), cu_final_seq=i32(cu_final_seq),
        cu_block=i32(cu_block), block_delta=i32(block_delta), block_seq=i32(block_seq),
        block_kv_begin=i32(block_kv_begin), block_part_off=i32(block_part_off),
        block_is_final=np.asarray(block_is_final, dtype=np.uint8),
        tok_block=i32(tok_block), tok_pos=i32(tok_pos), tok_pos_local=i32(tok_pos_local),
        cache_block=i32(cache_block), cache_cu=i32(cache_cu), cache_delta=i32(cache_delta),
    )


# ---------------------------------------------------------------------------
# The explicit mask (Section 1, Section 2.1, Section 2.4)
# ---------------------------------------------------------------------------
def mask_rows(block_lens, seq_nblocks, mode, rows, cols=None):
    """Rows `rows` of the dense 0/1 mask over the packed batch, as bool [n, T].

    M[i, j] = 1 iff j is in the same sequence as i, j <= i, and either the
    mode is full attention, or block(j) == block(i), or block(i) is its
    sequence's final block.  Written from the block lists directly (not from
    block_kv_begin) so that the tables and the mask pin one another.
    `cols` = (c0, c1) restricts the result to key columns c0..c1-1.
    """
    block_lens = [int(x) for x in block_lens]
    T = sum(block_lens)
    blk = np.repeat(np.arange(len(block_lens)), block_lens)
    seq_of_block = np.repeat(np.arange(len(seq_nblocks)), seq_nblocks)
    seq = seq_of_block[blk]
    last_block_of_seq = np.cumsum(seq_nblocks) - 1
    is_final_tok = (blk == last_block_of_seq[seq])
    rows = np.asarray(rows, dtype=np.int64)
    c0, c1 = (0, T) if cols is None else cols
    j = np.arange(c0, c1)[None, :]
    i = rows[:, None]
    m = (seq[None, c0:c1] == seq[rows][:, None]) & (j <= i)
    if mode == MODE_BLOCK:
        m &= (blk[None, c0:c1] == blk[rows][:, None]) | is_final_tok[rows][:, None]
    return m


def dense_mask(block_lens, seq_nblocks, mode):
    return mask_rows(block_lens, seq_nblocks, mode, np.arange(sum(int(x) for x in block_lens)))


# ---------------------------------------------------------------------------
# RoPE (Section 2.3, Eq. 1-3)
# ---------------------------------------------------------------------------
def rope_theta(head_dim, base):
    """theta_m = base^(-2m/d), m = 0..d/2-1.  The paper uses theta_m without
    defining it; this is RoPE's standard definition (the paper cites RoPE)."""
    m = np.arange(head_dim // 2, dtype=np.float64)
    return np.float64(base) ** (-2.0 * m / head_dim)


def rope_pairs(head_dim, layout):
    """Coordinates (x, y) of rotary pair m.  Eq. 1 writes the rotation as 2x2
    diagonal blocks, i.e. pair m = coordinates (2m, 2m+1); the half-split
    pairing (m, m + d/2) is the same map on permuted coordinates."""
    m = np.arange(head_dim // 2)
    if layout == ROPE_ADJACENT:
        return 2 * m, 2 * m + 1
    if layout == ROPE_HALF:
        return m, m + head_dim // 2
    raise ValueError("unknown RoPE layout")


def rope_matrix(p, head_dim, base, layout=ROPE_ADJACENT):
    """The d x d matrix of Eq. 1 for position p: 2x2 blocks
    [[cos p*theta_m, -sin p*theta_m], [sin p*theta_m, cos p*theta_m]].
    (The printed off-diagonal entries lost their subscripts; each 2x2 block
    uses one theta_m, as the last block of the printed matrix shows.)"""
    th = rope_theta(head_dim, base) * np.float64(p)
    ix, iy = rope_pairs(head_dim, layout)
    R = np.zeros((head_dim, head_dim), dtype=np.float64)
    R[ix, ix] = np.cos(th)
    R[ix, iy] = -np.sin(th)
    R[iy, ix] = np.sin(th)
    R[iy, iy] = np.cos(th)
    return R


def rotate(x, pos, base, layout=ROPE_ADJACENT, inverse=False):
    """Apply Eq. 1's matrix R(pos) (or its transpose, Eq. 2, when inverse) to
    the last axis of x.  `pos` broadcasts against x.shape[:-1]."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    ang = np.asarray(pos, dtype=np.float64)[..., None] * rope_theta(d, base)
    c, s = np.cos(ang), np.sin(ang)
    if inverse:
        s = -s
    ix, iy = rope_pairs(d, layout)
    out = np.empty_like(x)
    out[..., ix] = x[..., ix] * c - x[..., iy] * s
    out[..., iy] = x[..., ix] * s + x[..., iy] * c
    return out


def reencode_literal(k_cached, delta, base, layout=ROPE_ADJACENT):
    """Section 2.3 exactly as stated: a cached block [L, H, d] holds positions
    t = 0..L-1.  Step 2 (Eq. 2) takes every token back to position zero with
    the transposed matrix; step 3 (Eq. 3) rotates it to its new position
    delta + t.  (The prose names the directions the other way round; the
    printed matrices decide.)"""
    k_cached = np.asarray(k_cached, dtype=np.float64)
    t = np.arange(k_cached.shape[0], dtype=np.float64)[:, None]
    k_zero = rotate(k_cached, t, base, layout, inverse=True)         # Eq. 2
    return rotate(k_zero, t + np.float64(delta), base, layout)        # Eq. 3


def reencode_delta(k_cached, delta, base, layout=ROPE_ADJACENT):
    """The single rotation by the position difference that Section 2.3 says is
    equivalent ("why not rotate by (i_delta - i) theta directly")."""
    k_cached = np.asarray(k_cached, dtype=np.float64)
    return rotate(k_cached, np.full(k_cached.shape[:1] + (1,), float(delta)), base, layout)


def paged_rows(cache_lens, page_rows, page_cu, page_idx):
    """Pool row of every cached row when the cache is a pool of fixed-size pages (Section 2.3: what the
    cache holds; Section 2.5 step 1: the look-up).  Cached block c owns the pages
    page_idx[page_cu[c]] .. page_idx[page_cu[c+1] - 1], in order; its row t is row t mod page_rows of its
    page number t div page_rows.  Plain loops; the result indexes the pool tensor."""
    rows = []
    for c, L in enumerate(cache_lens):
        for t in range(int(L)):
            page = int(page_idx[int(page_cu[c]) + t // page_rows])
            rows.append(page * page_rows + t % page_rows)
    return np.asarray(rows, dtype=np.int64)


def reencode_blocks(k_src, src_off, cache_cu, cache_delta, base, layout=ROPE_ADJACENT):
    """Re-encode every cached block (Section 2.5, step 2).  Block c occupies
    rows cache_cu[c]..cache_cu[c+1] of the result; its source rows start at
    src_off[c] in k_src (a pool) or at cache_cu[c] when src_off is None.
    Returns fp64 [T_c, H, d] computed by the literal two-step route; the
    one-step route must agree (asserted)."""
    k_src = np.asarray(k_src, dtype=np.float64)
    n = len(cache_delta)
    out = np.empty((int(cache_cu[n]),) + k_src.shape[1:], dtype=np.float64)
    for c in range(n):
        lo, hi = int(cache_cu[c]), int(cache_cu[c + 1])
        s0 = lo if src_off is None else int(src_off[c])
        blk = k_src[s0:s0 + (hi - lo)]
        lit = reencode_literal(blk, int(cache_delta[c]), base, layout)
        one = reencode_delta(blk, int(cache_delta[c]), base, layout)
        if lit.size and np.max(np.abs(lit - one)) > 1e-9 * max(1.0, np.max(np.abs(blk))):
            raise AssertionError("two-step and one-step re-encoding disagree")
        out[lo:hi] = lit
    return out


# ---------------------------------------------------------------------------
# Attention under a mask
# ---------------------------------------------------------------------------
def attention_rows(q_rows, k, v, mask, scale=None):
    """softmax(q k^T * scale + log mask) v for the given query rows.

    q_rows [n, Hq, d]; k, v [T, Hkv, d]; mask bool [n, T].  Query head h reads
    KV head h // (Hq // Hkv).  scale defaults to 1/sqrt(d).  Returns
    o [n, Hq, d] and lse [n, Hq] (natural log of the softmax denominator,
    including the subtracted maximum).  Every row must see at least one key
    (always true for this mask: a token sees itself)."""
    q_rows = np.asarray(q_rows, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n, Hq, d = q_rows.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(np.float64(d))
    o = np.empty((n, Hq, d), dtype=np.float64)
    lse = np.empty((n, Hq), dtype=np.float64)
    neg = np.where(mask, 0.0, -np.inf)
    for h in range(Hq):
        g = h // G
        s = (q_rows[:, h, :] @ k[:, g, :].T) * scale + neg
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        l = p.sum(axis=1, keepdims=True)
        o[:, h, :] = (p @ v[:, g, :]) / l
        lse[:, h] = (m + np.log(l))[:, 0]
    return o, lse


def block_prefill(q, k, v, block_lens, seq_nblocks, mode, rows=None, scale=None):
    """Attention of the packed ragged batch under the Block-attention mask
    (or the full causal mask).  `rows` selects query rows (default all); rows
    are independent, so a subset is exact for the rows it contains."""
    T = sum(int(x) for x in block_lens)
    if rows is None:
        rows = np.arange(T)
    rows = np.asarray(rows, dtype=np.int64)
    o = np.empty((len(rows),) + tuple(np.shape(q)[1:]), dtype=np.float64)
    lse = np.empty((len(rows), np.shape(q)[1]), dtype=np.float64)
    # rows are handled sequence by sequence: keys of other sequences are masked for
    # every row, so only the sequence's own key columns are materialised
    cu_seq = np.concatenate([[0], np.cumsum([sum(int(x) for x in block_lens[a:b]) for a, b in zip(
        np.concatenate([[0], np.cumsum(seq_nblocks)[:-1]]), np.cumsum(seq_nblocks))])])
    seq_of_row = np.searchsorted(cu_seq, rows, side="right") - 1
    step = 1024
    qf, kf, vf = np.asarray(q), np.asarray(k), np.asarray(v)
    for s in np.unique(seq_of_row):
        sel = np.flatnonzero(seq_of_row == s)
        c0, c1 = int(cu_seq[s]), int(cu_seq[s + 1])
        for lo in range(0, len(sel), step):
            idx = sel[lo:lo + step]
            r = rows[idx]
            m = mask_rows(block_lens, seq_nblocks, mode, r, cols=(c0, c1))
            o[idx], lse[idx] = attention_rows(qf[r], kf[c0:c1], vf[c0:c1], m, scale)
    return o, lse


def final_attend(q_f, k_f, v_f, k_cache_reencoded, v_cache, block_lens, seq_nblocks,
                 mode=MODE_BLOCK, scale=None):
    """Section 2.5, step 3: each request's final block attends its re-encoded
    cached blocks plus itself.  Inputs are packed over the batch: cached rows
    of request s are cu_cache_seq[s]..cu_cache_seq[s+1] of k_cache_reencoded /
    v_cache, final rows are cu_final_seq[s]..cu_final_seq[s+1] of q_f/k_f/v_f.
    The result is, by definition, the final-block rows of masked attention over
    the concatenation [cached blocks in prompt order ; final block]."""
    t = segment_tables(block_lens, seq_nblocks, mode)
    Hq, d = np.shape(q_f)[1], np.shape(q_f)[2]
    o = np.empty((t["n_final_tokens"], Hq, d), dtype=np.float64)
    lse = np.empty((t["n_final_tokens"], Hq), dtype=np.float64)
    b0 = 0
    for s in range(t["batch"]):
        nb = int(seq_nblocks[s])
        lens = [int(x) for x in block_lens[b0:b0 + nb]]
        c0, c1 = int(t["cu_cache_seq"][s]), int(t["cu_cache_seq"][s + 1])
        f0, f1 = int(t["cu_final_seq"][s]), int(t["cu_final_seq"][s + 1])
        k_all = np.concatenate([np.asarray(k_cache_reencoded, dtype=np.float64)[c0:c1],
                                np.asarray(k_f, dtype=np.float64)[f0:f1]], axis=0)
        v_all = np.concatenate([np.asarray(v_cache, dtype=np.float64)[c0:c1],
                                np.asarray(v_f, dtype=np.float64)[f0:f1]], axis=0)
        n = k_all.shape[0]
        rows = np.arange(n - (f1 - f0), n)
        m = mask_rows(lens, [nb], mode, rows)
        o[f0:f1], lse[f0:f1] = attention_rows(np.asarray(q_f, dtype=np.float64)[f0:f1],
                                              k_all, v_all, m, scale)
        b0 += nb
    return o, lse


# ---------------------------------------------------------------------------
# Backward pass under the same mask (Section 2.4: block fine-tuning trains the model with
# the Block-attention mask in place of the lower-triangular one, so gradients flow through
# exactly the masked softmax attention defined above)
# ---------------------------------------------------------------------------
def attention_rows_backward(q_rows, k, v, mask, d_o, scale=None):
    """Gradients of  L = sum(d_o * O)  for the rows computed by attention_rows.

    With P the row-wise softmax of the masked scaled scores S (P = 0 where the mask forbids)
    and O = P V:   dV = P^T dO;   dP = dO V^T;   dS = P * (dP - rowsum(P * dP))   (the softmax
    Jacobian applied to dP);   dQ = scale * dS K;   dK = scale * dS^T Q.  Query head h reads KV
    head floor(h / G), so dK and dV collect the contributions of the G heads of their group.
    Returns dq [n, Hq, d] and dk, dv [T, Hkv, d] (the contributions of these rows only)."""
    q_rows = np.asarray(q_rows, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    d_o = np.asarray(d_o, dtype=np.float64)
    n, Hq, d = q_rows.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(np.float64(d))
    dq = np.zeros_like(q_rows)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    neg = np.where(mask, 0.0, -np.inf)
    for h in range(Hq):
        g = h // G
        s = (q_rows[:, h, :] @ k[:, g, :].T) * scale + neg
        p = np.exp(s - s.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        dv[:, g, :] += p.T @ d_o[:, h, :]
        dp = d_o[:, h, :] @ v[:, g, :].T
        ds = p * (dp - (p * dp).sum(axis=1, keepdims=True))
        dq[:, h, :] = (ds @ k[:, g, :]) * scale
        dk[:, g, :] += (ds.T @ q_rows[:, h, :]) * scale
    return dq, dk, dv


def block_prefill_backward(q, k, v, d_o, block_lens, seq_nblocks, mode, scale=None):
    """dQ, dK, dV of block_prefill over the whole packed batch, sequence by sequence (keys of other
    sequences are masked for every row, so they receive no gradient)."""
    qf, kf, vf, gf = (np.asarray(x, dtype=np.float64) for x in (q, k, v, d_o))
    dq, dk, dv = np.zeros_like(qf), np.zeros_like(kf), np.zeros_like(vf)
    b0, row0 = 0, 0
    for nb in seq_nblocks:
        lens = [int(x) for x in block_lens[b0:b0 + nb]]
        n = sum(lens)
        rows = np.arange(n)
        m = mask_rows(lens, [nb], mode, rows)
        sl = slice(row0, row0 + n)
        a, b, c = attention_rows_backward(qf[sl], kf[sl], vf[sl], m, gf[sl], scale)
        dq[sl], dk[sl], dv[sl] = a, b, c
        b0 += nb
        row0 += n
    return dq, dk, dv


def allowed_pairs(block_lens, seq_nblocks, mode):
    """Number of (query, key) pairs the mask allows, per query head (closed form)."""
    total, b0 = 0, 0
    for nb in seq_nblocks:
        lens = [int(x) for x in block_lens[b0:b0 + nb]]
        if mode == MODE_FULL:
            n = sum(lens)
            total += n * (n + 1) // 2
        else:
            for L in lens[:-1]:
                total += L * (L + 1) // 2
            Lf, n = lens[-1], sum(lens)
            total += Lf * (n - Lf) + Lf * (Lf + 1) // 2
        b0 += nb
    return total
