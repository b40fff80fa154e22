"""Host-side logic that needs no GPU: workload generators, bf16 conversion, and
the replica aggregation of bench.py under a 2-rank gloo group."""
import os
import subprocess
import sys

import numpy as np

from oracle import block_attention as ob
from paper_2409_15355_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, -2.5, 1.00390625, 1.01171875, 3.1415927, 1e-20, 65504.0], dtype=np.float32)
    b = W.f32_to_bf16_bits(x)
    y = W.bf16_bits_to_f32(b)
    assert y[0] == 1.0 and y[1] == -2.5
    assert y[2] == 1.0            # 1 + 2^-8 is a tie: rounds to even (1.0)
    assert y[3] == 1.015625       # 1 + 3*2^-8 is a tie: rounds to even (1 + 2^-6)
    assert np.all(np.abs(y - x) <= np.abs(x) * 2.0 ** -8)
    import torch
    assert np.array_equal(torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16), b)
    assert np.array_equal(W.f32_to_bf16_bits(y), b)


def test_workload_shapes():
    w1, w2, w3, w4, w5 = W.config1(), W.config2(), W.config3(), W.config4(), W.config5()
    assert w1.n_tokens == 288 and w1.final_lens() == [32]
    assert len(w2.block_lens) == 11 and all(128 <= l <= 384 for l in w2.block_lens[:10]) and w2.block_lens[-1] == 64
    assert w3.n_tokens == 32768 and w3.final_lens() == [768] and w3.n_layers == 32
    assert w4.batch == 8 and w4.n_tokens == 8 * 16384
    b = 0
    for nb in w4.seq_nblocks:
        lens = w4.block_lens[b:b + nb]
        assert sum(lens) == 16384 and all(64 <= l <= 2048 for l in lens[:-1]) and 1 <= lens[-1] <= 2048
        b += nb
    assert w5.batch == 16 and len(w5.pool_lens) == 512 and all(50 <= l <= 500 for l in w5.pool_lens)
    assert all(len(r) == 20 for r in w5.request_pool_idx) and w5.final_lens() == [128] * 16
    # deterministic
    assert W.config4().block_lens == w4.block_lens and W.config5().request_pool_idx == w5.request_pool_idx
    assert np.array_equal(W.normal_bf16(5, (3, 4)), W.normal_bf16(5, (3, 4)))
    # algorithmic pair counts used by the roofline arithmetic
    assert ob.allowed_pairs(w3.block_lens, w3.seq_nblocks, ob.MODE_BLOCK) - 32 * (1000 * 1001 // 2) == 768 * 32000 + 768 * 769 // 2
    x = W.warm_inputs(W.config5(2, 8, 3, 4))
    assert x["src_off"].shape == (6,) and x["q_f"].shape == (8, 32, 128)


_RANK_SCRIPT = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
ms, us = bench.aggregate(10.0 + 5.0 * rank, 32.0)
assert ms == 15.0, ms
assert abs(us - 15.0e3 / 64.0) < 1e-9, us
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_replica_aggregation_two_ranks_gloo(tmp_path):
    port = 29500 + os.getpid() % 2000
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
        assert "ok" in o


def _pieces_of_a_balanced_launch(sizes, n_chunks, n_sms, tail, n_partials):
    """Which key tiles of which (chunk, item) every CTA of a balanced launch takes and into which slot of the
    partial results it writes them, from the launch's definition: the first len(sizes) * n_chunks CTAs take
    the last `tail` tiles of one item each (slot 0); the tiles in front of those, laid end to end over all
    (chunk, item), are cut into equal runs for the remaining CTAs; a piece's slot is 1 + the number of CTAs
    since the one that holds the first front tile of its item."""
    n_main = len(sizes) * n_chunks
    n_front = n_sms - n_main
    front = [max(0, n - tail) for n in sizes]
    cover = {}
    for c in range(n_chunks):
        for i, n in enumerate(sizes):
            for t in range(front[i], n):
                cover.setdefault((c, i, t), []).append(0)
    line = [(c, i, t) for c in range(n_chunks) for i in range(len(sizes)) for t in range(front[i])]
    total = len(line)
    owner_of = lambda pos: next(j for j in range(n_front) if total * j // n_front <= pos < total * (j + 1) // n_front)
    first_pos, pieces_per_cta = {}, [set() for _ in range(n_front)]
    for pos, (c, i, t) in enumerate(line):
        first_pos.setdefault((c, i), pos)
    for (c, i), g0 in first_pos.items():
        # the closed form the kernel uses for the CTA that holds position g0
        assert owner_of(g0) == ((g0 + 1) * n_front - 1) // total
    for pos, (c, i, t) in enumerate(line):
        j = owner_of(pos)
        slot = 1 + j - owner_of(first_pos[(c, i)])
        assert slot < n_partials
        cover.setdefault((c, i, t), []).append(slot)
        pieces_per_cta[j].add((c, i))
    return cover, pieces_per_cta, total


def test_balanced_launch_plan_covers_every_tile_once_within_its_slots():
    """ba_plan_final_attend (the planning step of ba_final_attend, host arithmetic): the metric's workload gets
    the balanced launch; whenever a plan is balanced, every key tile of every item is taken exactly once, no
    piece needs a slot beyond the planned number of partial results, and no CTA has more than a few tiles more
    than an even share."""
    from paper_2409_15355_b200 import binding as B
    sizes32k = [250 + -(-min(768, r0 + 64) // 128) for r0 in range(0, 768, 64)]
    plan = B.ba_plan_final_attend(148, 12, 8, -(-sum(sizes32k) // 12), [sum(sizes32k), min(sizes32k), max(sizes32k)], 6)
    assert plan == {"partials": 3, "balanced_tails": 96, "tail_tiles": 167}
    # item sizes unknown, no room for partial results, more items than SMs: no balanced launch
    assert B.ba_plan_final_attend(148, 12, 8, 254, [0, 0, 0], 6)["balanced_tails"] == 0
    assert B.ba_plan_final_attend(148, 12, 8, 254, [sum(sizes32k), 251, 256], 0) == \
        {"partials": 1, "balanced_tails": 0, "tail_tiles": 0}
    assert B.ba_plan_final_attend(148, 40, 8, 254, [40 * 254, 254, 254], 6)["balanced_tails"] == 0
    rng = np.random.default_rng(5)
    n_balanced = 0
    for _ in range(300):
        n_sms = int(rng.choice([108, 132, 148]))
        n_chunks = int(rng.choice([1, 2, 4, 8]))
        n_pairs = int(rng.integers(1, max(2, n_sms // n_chunks)))
        base = int(rng.integers(4, 300))
        sizes = [base + int(v) for v in rng.integers(0, max(1, base // 3), n_pairs)]
        cap = int(rng.integers(2, 33))
        plan = B.ba_plan_final_attend(n_sms, n_pairs, n_chunks, -(-sum(sizes) // n_pairs),
                                      [sum(sizes), min(sizes), max(sizes)], cap)
        assert 1 <= plan["partials"] <= max(cap, 1)
        if not plan["balanced_tails"]:
            continue
        n_balanced += 1
        tail = plan["tail_tiles"]
        assert plan["balanced_tails"] == n_pairs * n_chunks < n_sms and 1 <= tail <= min(sizes)
        cover, pieces, total_front = _pieces_of_a_balanced_launch(sizes, n_chunks, n_sms, tail, plan["partials"])
        assert len(cover) == n_chunks * sum(sizes) and all(len(v) == 1 for v in cover.values())
        share = -(-n_chunks * sum(sizes) // n_sms)
        n_front = n_sms - n_pairs * n_chunks
        assert tail <= share + 8 and -(-total_front // n_front) <= tail + 3
    assert n_balanced >= 20
