#!/usr/bin/env python
"""Benchmark of the Block-attention warm path at 32K context.

One step = one pass of the hot path over a 32768-token prompt (32 cached
passages of 1000 tokens + a 768-token final block, Llama-3-8B attention shape):
ba_segment once, then for each of 32 layers ba_reencode_k (cached K to prompt
positions) and ba_final_attend (final block over re-encoded cache + itself),
every layer with its own seeded K/V/Q.  The metric is microseconds per layer.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line.  With N > 1 (torchrun) every rank runs an independent
replica of the same job (the path has no exchange step); the reported value is
the time per layer-job over all replicas.  --impl reference times the fp64 CPU
oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "final-block attend+reencode us/layer at 32K ctx"
UNIT = "us/layer"


def attend_dram_traffic():
    """DRAM bytes (read + write) of one attention launch of this workload, as counted by the profiler.
    The figure sits in a small text file next to the profiler summaries together with a digest of the
    kernel sources it was taken from; once the sources differ from that digest the figure is stale and
    None is reported instead."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "attend_dram_traffic.txt")
    if not os.path.exists(path):
        return None
    kv = {}
    for line in open(path):
        if ":" in line and not line.lstrip().startswith("#"):
            k, v = line.split(":", 1)
            kv[k.strip()] = v.strip()
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2409_15355_b200", "csrc")
    for name in ("ba_attend_sm100.cu", "ba_sm100.cuh"):
        with open(os.path.join(csrc, name), "rb") as fh:
            h.update(fh.read())
    if kv.get("sources_sha256") != h.hexdigest():
        return None
    try:
        return float(kv["dram_bytes_per_launch"])
    except (KeyError, ValueError):
        return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20", "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- distributed plumbing
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, device=None) -> float:
    """Max of a host scalar over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate(ms_local: float, layer_jobs_local: float, device=None):
    """Replica aggregation: the job takes as long as its slowest rank; the work
    done is the sum over ranks.  Returns (ms, us per layer-job over all ranks)."""
    ms = max_over_ranks(ms_local, device)
    jobs = sum_over_ranks(layer_jobs_local, device)
    return ms, ms * 1e3 / jobs


# --------------------------------------------------------------------------- the oracle legs
class OracleSampler:
    """The fp64 oracle on one layer of the workload, timed on a bounded sample: re-encode of the
    first `n_blocks` cached blocks and final attend of the first `n_rows` rows of the final block,
    each scaled linearly to the whole layer (rows and blocks are independent, so a subset is
    exact for what it covers).  Inputs are generated and widened to fp64 once, outside the timing."""

    def __init__(self, w, layer: int = 0):
        from oracle import block_attention as ob
        from paper_2409_15355_b200 import workloads as W
        self.ob, self.w = ob, w
        x = W.warm_inputs(w, layer)
        self.t = ob.segment_tables(w.block_lens, w.seq_nblocks)
        self.Lf = w.final_lens()[0]
        f64 = W.bf16_bits_to_f64
        self.kc, self.vc = f64(x["k_cache"]), f64(x["v_cache"])
        self.qf, self.kf, self.vf = f64(x["q_f"]), f64(x["k_f"]), f64(x["v_f"])
        self.k_re = ob.reencode_blocks(self.kc, None, self.t["cache_cu"], self.t["cache_delta"], w.rope_theta)

    def sample(self, n_rows: int, n_blocks: int):
        """Returns (microseconds per layer, seconds actually spent)."""
        ob, t, w = self.ob, self.t, self.w
        nb_all = len(t["cache_delta"])
        n_blocks = max(1, min(n_blocks, nb_all))
        n_rows = max(1, min(n_rows, self.Lf))
        t0 = time.perf_counter()
        ob.reencode_blocks(self.kc, None, t["cache_cu"][:n_blocks + 1], t["cache_delta"][:n_blocks], w.rope_theta)
        t1 = time.perf_counter()
        k_all = np.concatenate([self.k_re, self.kf]); v_all = np.concatenate([self.vc, self.vf])
        rows = np.arange(t["n_cached_tokens"], t["n_cached_tokens"] + n_rows)
        m = ob.mask_rows(w.block_lens, w.seq_nblocks, ob.MODE_BLOCK, rows)
        ob.attention_rows(self.qf[:n_rows], k_all, v_all, m)
        t2 = time.perf_counter()
        us = ((t1 - t0) * (nb_all / n_blocks) + (t2 - t1) * (self.Lf / n_rows)) * 1e6
        return us, t2 - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The oracle as it stands, on host cores.  Every step is a bounded sample of one layer,
    sized from the first warm-up so that the whole run stays within about two minutes."""
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    from paper_2409_15355_b200 import workloads as W
    smp = OracleSampler(W.config3(1))
    _, sec = smp.sample(4, 1)                          # calibration: 4 rows, 1 block
    budget = 110.0 / max(1, args.steps + args.warmup)  # seconds per step
    scale = max(1.0, min(24.0, 0.8 * budget / max(sec, 1e-3)))
    rows, blocks = int(4 * scale), int(max(1, min(32, scale)))
    for _ in range(args.warmup):
        smp.sample(rows, blocks)
    vals = []
    t0 = time.perf_counter()
    for _ in range(args.steps):
        vals.append(smp.sample(rows, blocks)[0])
    wall = time.perf_counter() - t0
    v = statistics.mean(vals) if vals else float("nan")
    sample = (f"per step: one layer; re-encode of {blocks}/32 cached blocks scaled x{32 / blocks:.1f} + final attend "
              f"of {rows}/768 final rows (all 32 heads) scaled x{768 / rows:.1f}")
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": wall * 1e3 / max(args.steps, 1),
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def workload_config():
    return {"workload": "cfg3_32k: 32 cached blocks x 1000 tokens + 768-token final block, "
                        "32 q heads / 8 kv heads / head_dim 128, 32 layers with independent seeded K/V/Q",
            "layers": 32, "context": 32768, "final_block": 768, "mode": "block",
            "l2": "inputs larger than L2 (131 MB of K/V per layer, distinct buffers per layer)"}


# --------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2409_15355_b200 import binding as B
    from paper_2409_15355_b200 import runtime as R
    from paper_2409_15355_b200 import workloads as W

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    L = args.layers
    w = W.config3(L)
    Tc, Tf = 32000, 768
    ctx = R.Context.for_workload(w, device=local_rank)
    pin = lambda bits: R.bits_to_tensor(bits).pin_memory()
    host = []
    for l in range(L):
        x = W.warm_inputs(w, l)
        host.append({k: pin(v) for k, v in x.items()})
    names = ("q_f", "k_f", "v_f", "k_cache", "v_cache")
    d_in = [{k: h[k].to(dev) for k in names} for h in host]
    k_re = [torch.empty(Tc, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device=dev) for _ in range(L)]
    o = [torch.empty(Tf, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev) for _ in range(L)]
    o_host = [torch.empty(Tf, w.n_q_heads, w.head_dim, dtype=torch.bfloat16).pin_memory() for _ in range(L)]
    lens = np.asarray(w.block_lens, dtype=np.int32)
    nb = np.asarray(w.seq_nblocks, dtype=np.int32)
    nbytes = B.ba_segments_bytes(1, len(lens), w.n_tokens)
    tbuf = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    # --overlap: the re-encoding of layer l+1 runs on a second, lower-priority stream while layer l attends.
    # The attention launch leaves a few SMs idle in its last wave (288 CTAs on 148 SMs) and cannot share an
    # SM with anything else; the bandwidth-bound re-encode fills those gaps instead of waiting its turn.
    re_stream = torch.cuda.Stream(device=dev, priority=0) if args.overlap else None
    if args.overlap:
        main_stream = torch.cuda.Stream(device=dev, priority=-1)
        torch.cuda.set_stream(main_stream)
        stream = main_stream

    att_events = []
    re_events = []

    def step_overlap(inputs, record=False, ready=None, done=None):
        seg = B.ba_segment(ctx.ctx, lens, nb, 1, len(lens), w.n_tokens, B.BA_MODE_BLOCK, tbuf)
        ev_seg = torch.cuda.Event(); ev_seg.record(stream)
        re_stream.wait_event(ev_seg)          # tables ready; the previous step no longer reads k_re
        ev_re, ev_att = [], []
        for l in range(L):
            x = inputs[l]
            if l >= 2:
                re_stream.wait_event(ev_att[l - 2])     # stay one layer ahead of the attention, not more
            if ready is not None:
                re_stream.wait_event(ready[l])          # this layer's inputs have arrived from the host
            B.ba_reencode_k(ctx.ctx, x["k_cache"], None, Tc, k_re[l], seg.cache_cu, seg.cache_delta,
                            seg.n_cached_blocks, Tc, stream=re_stream)
            e = torch.cuda.Event(); e.record(re_stream); ev_re.append(e)
            if l >= 1:
                issue_attend(inputs, l - 1, seg, ev_re, ev_att, record)
        issue_attend(inputs, L - 1, seg, ev_re, ev_att, record)
        if done is not None:
            done.extend(ev_att)

    def issue_attend(inputs, l, seg, ev_re, ev_att, record):
        x = inputs[l]
        stream.wait_event(ev_re[l])                     # (the re-encode stream waited for the layer's inputs)
        record = record and (l % 4 == 2 or L < 4)     # a sample of the launches: event records are stream work too
        if record:
            e0 = torch.cuda.Event(enable_timing=True); e0.record(stream)
        B.ba_final_attend(ctx.ctx, x["q_f"], x["k_f"], x["v_f"], Tf, k_re[l], x["v_cache"], Tc, None, 0,
                          o[l], None, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
        e1 = torch.cuda.Event(enable_timing=record); e1.record(stream)
        ev_att.append(e1)
        if record:
            att_events.append((e0, e1))

    def step(inputs, record=False, ready=None, done=None):
        if args.overlap:
            return step_overlap(inputs, record, ready, done)
        if ready is not None:
            stream.wait_event(ready[-1])                # single-stream order: all inputs first
        seg = B.ba_segment(ctx.ctx, lens, nb, 1, len(lens), w.n_tokens, B.BA_MODE_BLOCK, tbuf)
        # Layer l+1 is re-encoded before layer l attends (the cached keys of all layers are known up
        # front); with --deferred that re-encoding is queued and runs inside layer l's attention launch.
        B.ba_reencode_k(ctx.ctx, inputs[0]["k_cache"], None, Tc, k_re[0], seg.cache_cu, seg.cache_delta,
                        seg.n_cached_blocks, Tc)
        for l in range(L):
            x = inputs[l]
            if l + 1 < L and args.deferred:
                B.ba_reencode_k_deferred(ctx.ctx, inputs[l + 1]["k_cache"], None, Tc, k_re[l + 1], seg.cache_cu,
                                         seg.cache_delta, seg.n_cached_blocks, Tc)
            elif l + 1 < L:
                rec_re = record and l % 4 == 0          # a sample of the launches: event records are stream work too
                if rec_re:
                    r0 = torch.cuda.Event(enable_timing=True); r0.record(stream)
                B.ba_reencode_k(ctx.ctx, inputs[l + 1]["k_cache"], None, Tc, k_re[l + 1], seg.cache_cu,
                                seg.cache_delta, seg.n_cached_blocks, Tc)
                if rec_re:
                    r1 = torch.cuda.Event(enable_timing=True); r1.record(stream)
                    re_events.append((r0, r1))
            rec_att = record and (l % 4 == 2 or L < 4)
            if rec_att:
                e0 = torch.cuda.Event(enable_timing=True); e0.record(stream)
            B.ba_final_attend(ctx.ctx, x["q_f"], x["k_f"], x["v_f"], Tf, k_re[l], x["v_cache"], Tc, None, 0,
                              o[l], None, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
            if rec_att:
                e1 = torch.cuda.Event(enable_timing=True); e1.record(stream)
                att_events.append((e0, e1))
            if done is not None:
                e = torch.cuda.Event(); e.record(stream); done.append(e)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(d_in)
    barrier()
    launches0 = ctx.launches()
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step(d_in, record=True)
    ev1.record(stream)
    barrier()
    ms_local = ev0.elapsed_time(ev1) / args.steps
    clocks = sampler.stop()
    launches = ctx.launches() - launches0
    attend_launch = ctx.last_attend_shape()      # how the library laid out the attention launches just timed
    assert ctx.device_status() == B.BA_OK
    ms, us_per_layer = aggregate(ms_local, float(L), dev)

    att_ms = statistics.mean(a.elapsed_time(b) for a, b in att_events)
    re_ms = statistics.mean(a.elapsed_time(b) for a, b in re_events) if re_events else None
    re_how = "every fourth launch inside the timed region"
    if re_ms is None and not args.deferred:
        # the launches of the timed region ran beside the attention on their own stream: time the kernel
        # alone instead, over the layers' buffers (65.5 MB read + 65.5 MB written each, nothing stays in L2)
        seg = B.ba_segment(ctx.ctx, lens, nb, 1, len(lens), w.n_tokens, B.BA_MODE_BLOCK, tbuf)
        for rep in range(2):
            if rep == 1:
                ev0.record(stream)
            for l in range(L):
                B.ba_reencode_k(ctx.ctx, d_in[l]["k_cache"], None, Tc, k_re[l], seg.cache_cu, seg.cache_delta,
                                seg.n_cached_blocks, Tc)
        ev1.record(stream)
        barrier()
        re_ms = ev0.elapsed_time(ev1) / L
        re_how = "alone, back to back over the layers' buffers, after the timed region"

    # ---- end to end: host buffers in, host result out, copies inside the timed region
    e2e_steps = max(1, min(args.steps, 3))
    h2d = sum(h[k].numel() * 2 for h in host for k in names)
    d2h = sum(t.numel() * 2 for t in o_host)
    stage = [{k: torch.empty_like(d_in[l][k]) for k in names} for l in range(L)]

    # copies run on streams of their own: layer l+1 arrives while layer l is worked on, results leave as
    # soon as their layer is done (PCIe is full duplex); everything is inside the timed region
    h2d_stream, d2h_stream = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def e2e_step():
        h2d_stream.wait_stream(stream)                  # the previous step has consumed the staging buffers
        ready, done = [], []
        with torch.cuda.stream(h2d_stream):
            for l in range(L):
                for k in names:
                    stage[l][k].copy_(host[l][k], non_blocking=True)
                e = torch.cuda.Event(); e.record(h2d_stream); ready.append(e)
        step(stage, ready=ready, done=done)
        with torch.cuda.stream(d2h_stream):
            for l in range(L):
                d2h_stream.wait_event(done[l])
                o_host[l].copy_(o[l], non_blocking=True)
        stream.wait_stream(d2h_stream)                  # the step ends when its last result is on the host

    e2e_step()
    barrier()
    ev0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record(stream)
    barrier()
    _, e2e_us = aggregate(ev0.elapsed_time(ev1) / e2e_steps, float(L), dev)

    # ---- secondary number: cold block-diagonal prefill (batch 8 x 16384 ragged blocks), one launch
    prefill = None
    if rank == 0 and not args.no_prefill:
        from oracle import block_attention as ob     # closed-form pair count only (no oracle compute)
        w4 = W.config4()
        ctx4 = R.Context.for_workload(w4, device=local_rank)
        seg4, buf4 = ctx4.segment(w4.block_lens, w4.seq_nblocks, B.BA_MODE_BLOCK)
        q4, k4, v4 = (R.bits_to_tensor(b).to(dev) for b in W.prefill_inputs(w4))   # the tensors the parity test checks
        o4 = torch.empty_like(q4)
        for _ in range(3):
            B.ba_block_prefill(ctx4.ctx, q4, k4, v4, o4, None, seg4, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
        torch.cuda.synchronize()
        reps = 10
        ev0.record(stream)
        for _ in range(reps):
            B.ba_block_prefill(ctx4.ctx, q4, k4, v4, o4, None, seg4, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
        ev1.record(stream)
        torch.cuda.synchronize()
        ms4 = ev0.elapsed_time(ev1) / reps
        pairs4 = ob.allowed_pairs(w4.block_lens, w4.seq_nblocks, ob.MODE_BLOCK)
        fl4 = 4.0 * w4.head_dim * w4.n_q_heads * pairs4
        prefill = {"workload": "cfg4: batch 8 x 16384 tokens, ragged blocks U[64,2048], one ba_block_prefill launch",
                   "ms": ms4, "algorithmic_flops": fl4, "tflops": fl4 / ms4 / 1e9, "allowed_pairs_per_head": pairs4,
                   "inputs": "seeded N(0,1) bf16 (workloads.prefill_inputs)"}
        assert ctx4.device_status() == B.BA_OK
        # the backward pass of the same launch (block fine-tuning): forward with log-sum-exp, then gradients
        lse4 = torch.empty(w4.n_tokens, w4.n_q_heads, dtype=torch.float32, device=dev)
        B.ba_block_prefill(ctx4.ctx, q4, k4, v4, o4, lse4, seg4, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
        g4 = R.bits_to_tensor(W.normal_bf16(4004077, tuple(q4.shape))).to(dev)
        dq4, dk4, dv4 = torch.empty_like(q4), torch.empty_like(k4), torch.empty_like(v4)
        for _ in range(2):
            B.ba_block_prefill_bwd(ctx4.ctx, q4, k4, v4, o4, lse4, g4, dq4, dk4, dv4, seg4, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
        torch.cuda.synchronize()
        ev0.record(stream)
        for _ in range(5):
            B.ba_block_prefill_bwd(ctx4.ctx, q4, k4, v4, o4, lse4, g4, dq4, dk4, dv4, seg4, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
        ev1.record(stream)
        torch.cuda.synchronize()
        msb = ev0.elapsed_time(ev1) / 5
        prefill["backward"] = {"workload": "gradients of the same launch (ba_block_prefill_bwd, bf16 gradients)", "ms": msb,
                               "algorithmic_flops": 2.5 * fl4, "tflops": 2.5 * fl4 / msb / 1e9,
                               "note": "five products per allowed pair (S, dP, dV, dK, dQ); the two kernels execute "
                                       "seven (S and dP are formed in both)"}
        assert ctx4.device_status() == B.BA_OK
        ctx4.close()
        del q4, k4, v4, o4, g4, dq4, dk4, dv4, lse4
        # the 32K prompt of the metric's workload encoded cold, under the full causal mask and under the
        # Block-attention mask (same tensors, one launch each): the paper's FLOPs / latency comparison
        T3 = w.n_tokens
        q3, k3, v3 = (R.bits_to_tensor(b).to(dev) for b in W.prefill_inputs(w))
        o3 = torch.empty_like(q3)
        p32 = {"workload": "cfg3 prompt (32 x 1000 + 768 tokens) encoded cold, one ba_block_prefill launch per mode"}
        for name, mode, omode in (("full_causal", B.BA_MODE_FULL, ob.MODE_FULL), ("block", B.BA_MODE_BLOCK, ob.MODE_BLOCK)):
            seg3 = B.ba_segment(ctx.ctx, lens, nb, 1, len(lens), T3, mode, tbuf)
            for _ in range(2):
                B.ba_block_prefill(ctx.ctx, q3, k3, v3, o3, None, seg3, mode, B.BA_OUT_BF16)
            torch.cuda.synchronize()
            ev0.record(stream)
            for _ in range(5):
                B.ba_block_prefill(ctx.ctx, q3, k3, v3, o3, None, seg3, mode, B.BA_OUT_BF16)
            ev1.record(stream)
            torch.cuda.synchronize()
            ms3 = ev0.elapsed_time(ev1) / 5
            fl3 = 4.0 * w.head_dim * w.n_q_heads * ob.allowed_pairs(w.block_lens, w.seq_nblocks, omode)
            p32[name] = {"ms": ms3, "algorithmic_flops": fl3, "tflops": fl3 / ms3 / 1e9}
        prefill["prompt_32k"] = p32
        assert ctx.device_status() == B.BA_OK
        del q3, k3, v3, o3

    # ---- secondary number: the fused warm path (keys as cached, queries counter-rotated per block in
    # the attention launch, no re-encoding pass) on the same 32-layer workload, and both paths with a
    # short final block, where the query side is small and the fused path is the faster one
    fused = None
    if rank == 0 and not args.no_fused:
        def fused_step(inputs, side_output):
            seg = B.ba_segment(ctx.ctx, lens, nb, 1, len(lens), w.n_tokens, B.BA_MODE_BLOCK, tbuf)
            for l in range(L):
                x = inputs[l]
                B.ba_final_attend_fused(ctx.ctx, x["q_f"], x["k_f"], x["v_f"], Tf, x["k_cache"], x["v_cache"], Tc,
                                        None, Tc, o[l], None, seg, B.BA_MODE_BLOCK, B.BA_OUT_BF16,
                                        k_out=k_re[l] if side_output else None)
        reps = max(1, min(args.steps, 20))
        fused = {"workload": "the metric's workload through ba_final_attend_fused (no ba_reencode_k pass)"}
        for key, side in (("us_per_layer", False), ("us_per_layer_with_k_out", True)):
            for _ in range(3):
                fused_step(d_in, side)
            torch.cuda.synchronize()
            ev0.record(stream)
            for _ in range(reps):
                fused_step(d_in, side)
            ev1.record(stream)
            torch.cuda.synchronize()
            fused[key] = ev0.elapsed_time(ev1) * 1e3 / reps / L
        fused["k_out"] = "re-encoded keys written back by the same call: the re-encoding kernel runs on the context's side stream beside the attention launch (65.5 MB per layer)"
        # short final block: 32 x 1000 cached + 64 final tokens, one layer's tensors reused over 4 buffers
        Ts = 64
        lens_s = np.asarray([1000] * 32 + [Ts], dtype=np.int32)
        seg_s = B.ba_segment(ctx.ctx, lens_s, nb, 1, len(lens_s), int(lens_s.sum()), B.BA_MODE_BLOCK, tbuf)
        nl = min(L, 4)
        def short_step(use_fused):
            for l in range(nl):
                x = d_in[l]
                if use_fused:
                    B.ba_final_attend_fused(ctx.ctx, x["q_f"][:Ts], x["k_f"][:Ts], x["v_f"][:Ts], Ts, x["k_cache"],
                                            x["v_cache"], Tc, None, Tc, o[l][:Ts], None, seg_s, B.BA_MODE_BLOCK,
                                            B.BA_OUT_BF16)
                else:
                    B.ba_reencode_k(ctx.ctx, x["k_cache"], None, Tc, k_re[l], seg_s.cache_cu, seg_s.cache_delta,
                                    seg_s.n_cached_blocks, Tc)
                    B.ba_final_attend(ctx.ctx, x["q_f"][:Ts], x["k_f"][:Ts], x["v_f"][:Ts], Ts, k_re[l], x["v_cache"],
                                      Tc, None, 0, o[l][:Ts], None, seg_s, B.BA_MODE_BLOCK, B.BA_OUT_BF16)
        short = {}
        for name, uf in (("unfused_us_per_layer", False), ("fused_us_per_layer", True)):
            for _ in range(3):
                short_step(uf)
            torch.cuda.synchronize()
            ev0.record(stream)
            for _ in range(10):
                short_step(uf)
            ev1.record(stream)
            torch.cuda.synchronize()
            short[name] = ev0.elapsed_time(ev1) * 1e3 / 10 / nl
        fused["short_final_block"] = dict(final_block=Ts, cached="32 x 1000", **short)
        assert ctx.device_status() == B.BA_OK

    if rank == 0:
        peaks = load_peaks()
        cfg_extra = {}
        if args.deferred:
            cfg_extra["reencode"] = "queued, in the background of the previous layer's attention launch"
        if args.overlap:
            cfg_extra["reencode"] = ("on a second, lower-priority stream: layer l+1 is re-encoded while layer l "
                                     "attends (both inside the timed region)")
        pairs = Tf * Tc + Tf * (Tf + 1) // 2
        flops = 4.0 * w.head_dim * w.n_q_heads * pairs
        achieved = flops / (att_ms * 1e-3) / 1e12
        burst, sustained = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
        # the dominant kernel, against the measured burst peak of a dense bf16 product
        roofline = {"bound": "tensor", "kernel": "ba_final_attend", "achieved": achieved, "peak": burst,
                    "unit": "TFLOP/s", "frac": achieved / burst, "traffic": attend_dram_traffic(),
                    "peak_source": f"{peaks['source']} bf16 burst (cuBLAS 8192^3, best of 10)",
                    "frac_of_sustained": achieved / sustained if sustained else None,
                    "peak_sustained": sustained,
                    "attend_us_per_launch": att_ms * 1e3, "attend_launch": attend_launch,
                    "algorithmic_flops_per_launch": flops}
        # the metric itself: re-encode + attend of one layer against max(FLOPs / tensor peak, bytes / HBM peak)
        att_bytes = (2.0 * Tc * w.n_kv_heads + 2.0 * Tf * w.n_kv_heads + 2.0 * Tf * w.n_q_heads) * w.head_dim * 2
        re_bytes = 2.0 * Tc * w.n_kv_heads * w.head_dim * 2        # cached K read once + re-encoded K written once
        floor_us = max(flops / (burst * 1e12), (att_bytes + re_bytes) / (peaks["hbm_gbs"] * 1e9)) * 1e6
        metric_roofline = {"what": "ba_reencode_k + ba_final_attend per layer", "floor_us": floor_us,
                           "floor": "max(algorithmic FLOPs / bf16 burst peak, algorithmic bytes / copy bandwidth)",
                           "algorithmic_flops": flops, "algorithmic_bytes": att_bytes + re_bytes,
                           "value_us": us_per_layer, "frac": floor_us / us_per_layer, "target_frac": 0.60,
                           "target_met": bool(floor_us / us_per_layer >= 0.60),
                           "sm_mhz_median": clocks.get("sm_mhz"),
                           "us_times_mhz": us_per_layer * clocks["sm_mhz"] if clocks.get("sm_mhz") else None}
        t0 = time.perf_counter()
        cpu_rows = 96
        cpu_us, _ = OracleSampler(W.config3(1)).sample(cpu_rows, 32)
        cpu = {"value": cpu_us, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"one layer: re-encode of 32000 cached rows + final attend of {cpu_rows}/768 final rows, "
                         f"attend scaled x{768 // cpu_rows}; {time.perf_counter() - t0:.1f} s of CPU work"}
        line = {"metric": METRIC, "value": us_per_layer, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(),
                "clocks": clocks,
                "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "steps": e2e_steps},
                "gpu_launches": launches, "roofline": roofline, "metric_roofline": metric_roofline,
                "cpu_baseline": cpu}
        if re_ms is not None:
            line["reencode"] = {"bound": "hbm", "kernel": "ba_reencode_k", "us_per_launch": re_ms * 1e3,
                                "timed": re_how,
                                "algorithmic_bytes_per_launch": re_bytes, "achieved": re_bytes / (re_ms * 1e-3) / 1e9,
                                "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                "frac": re_bytes / (re_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                "peak_source": f"{peaks['source']} copy bandwidth"}
        if fused is not None:
            line["fused_warm_path"] = fused
        if prefill is not None:
            prefill["frac_of_bf16_burst"] = prefill["tflops"] / peaks["bf16_tflops"]
            line["block_prefill"] = prefill
        line["config"].update(cfg_extra)
        if L != 32:
            line["config"]["layers"] = L
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=32, help="layers per step (32 = the metric's workload)")
    ap.add_argument("--no-prefill", action="store_true", help="skip the secondary cold-prefill measurement")
    ap.add_argument("--no-fused", action="store_true", help="skip the secondary fused-warm-path measurement")
    ap.add_argument("--no-overlap", dest="overlap", action="store_false",
                    help="issue re-encode and attend of every layer on one stream (default: layer l+1 is "
                         "re-encoded on a second stream while layer l attends)")
    ap.add_argument("--deferred", action="store_true",
                    help="queue each layer's re-encoding so that it runs in the background of the previous layer's "
                         "attention launch (ba_reencode_k_deferred) instead of as a stand-alone launch")
    args = ap.parse_args()
    if args.deferred:
        args.overlap = False
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
