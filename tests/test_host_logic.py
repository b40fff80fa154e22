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
