#!/usr/bin/env python
"""Benchmark of the router-selective decode step (decode tokens/s and step latency at the
Llama-3-8B shape, with the achieved fraction of the HBM roofline).

    python bench.py --gpus N --steps K --warmup W            # the CUDA library (N > 1: N independent replicas,
                                                             # started here, one process per GPU, or by torchrun)
    python bench.py --impl reference --steps K --warmup W    # the host oracle, bounded sample

One step = one routed decode step of the whole batch (embedding, every layer for the rows
that keep it, final norm, lm_head, greedy token).  Routing and the per-layer row plan are
done once per batch, before the timed steps, and reported separately.  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import first_inputs as fi  # noqa: E402

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"

WORKLOADS = {
    # name: (shape, B, prompt lo, prompt hi, default steps, mask recipe)
    "cfg1_1b_b1": dict(shape="1b", B=1, lo=512, hi=512, steps=256, mask=("fraction", 0.25, 0.25)),
    "cfg2_8b_b32": dict(shape="8b", B=32, lo=128, hi=2048, steps=128, mask=("fraction", 0.10, 0.40)),
    "cfg3_8b_b256": dict(shape="8b", B=256, lo=1024, hi=4096, steps=64, mask=("bernoulli", 0.7)),
    # small-cache cases for profiler captures of the projections at a given row count (not benchmark lines)
    "prof_8b_b192": dict(shape="8b", B=192, lo=64, hi=128, steps=8, mask=("dense",)),
    "prof_8b_b64": dict(shape="8b", B=64, lo=64, hi=128, steps=8, mask=("dense",)),
    # the paper's second model shape (Llama-3.2-3B: 28 layers, 24 query / 8 KV heads), config-2-like batch
    "llama3b_b32": dict(shape="3b", B=32, lo=128, hi=2048, steps=128, mask=("fraction", 0.10, 0.40)),
    "cfg4_8b_b64": dict(shape="8b", B=64, lo=1024, hi=1024, steps=128, mask=("aligned", 0.25)),
}
SHAPES = {"1b": fi.LLAMA_1B, "8b": fi.LLAMA_8B, "3b": fi.LLAMA_3B}


def make_mask(recipe, B, L, seed):
    kind = recipe[0]
    if kind == "fraction":
        return fi.mask_skip_fraction(B, L, recipe[1], recipe[2], seed)
    if kind == "bernoulli":
        return fi.mask_bernoulli(B, L, recipe[1], seed)
    if kind == "aligned":
        return fi.mask_aligned(B, L, recipe[1])
    if kind == "independent":
        return fi.mask_independent(B, L, recipe[1], seed)
    if kind == "unified":
        return fi.mask_unified(B, L, int(recipe[1]))
    if kind == "random":
        return fi.mask_random_shared(B, L, recipe[1], 2000)  # one draw for the whole job, every rank the same
    if kind == "dense":
        return np.ones((B, L), np.uint8)
    raise ValueError(kind)


def byte_model(shape, mask, lens, kv_elem=2, w_elem=2):
    """Roofline bytes of one step: weights of layers with any active row + KV of active rows
    (strict), and the same plus lm_head, embedding rows, KV appends and the logits (full)."""
    B, L = mask.shape
    cnt = mask.sum(0)
    w_layer = shape.layer_params() * w_elem
    kv_tok = 2 * shape.kv_dim * kv_elem
    weights = int((cnt > 0).sum()) * w_layer
    kv = int(sum(kv_tok * (int(lens[b]) + 1) for b in range(B) for l in range(L) if mask[b, l]))
    strict = weights + kv
    full = strict + shape.vocab * shape.d_model * w_elem + B * shape.d_model * w_elem + int(cnt.sum()) * kv_tok \
        + B * shape.vocab * 4
    return dict(strict=strict, full=full, weights=weights, kv=kv, lm_head=shape.vocab * shape.d_model * w_elem)


def max_over_ranks(ms, dist, device):
    """Slowest rank's time (replicas run independently; the job is as slow as its slowest GPU)."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(world, batch_per_rank, steps, ms_max):
    """Whole-job throughput of `world` replicas, each decoding `batch_per_rank` sequences for `steps` steps."""
    return world * batch_per_rank * steps / (ms_max / 1e3)


def physical_gpu_index(local):
    """nvidia-smi's index of CUDA device `local` of this process (CUDA_VISIBLE_DEVICES may renumber)."""
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")
    if local < len(vis) and vis[local].strip().isdigit():
        return int(vis[local])
    return local


class ClockSampler:
    """nvidia-smi sampled every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.t.start()
        except OSError:
            self.proc = None
        return self

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.25)
            self.proc.terminate()
            self.t.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------- oracle arm
class OracleSample:
    """A bounded sample of the workload for the host oracle: `rows` sequences of the batch (their real cache
    lengths, stand-in cache contents), `layers` decoder layers of the same width, plus final norm + lm_head.
    step() times one decode step of the sample and extrapolates to the whole step by the mask's kept
    (row, layer) count."""

    def __init__(self, shape, mask, lens, seed, rows=4, layers=2):
        import oracle
        from oracle.workload import oracle_model, stand_in_cache
        self.oracle = oracle
        self.B, self.L = mask.shape
        self.rows, self.layers = min(rows, self.B), layers
        self.kept = int(mask.sum())
        sub = fi.ModelShape(layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn_dim,
                            shape.vocab, shape.rope_base, shape.rms_eps)
        self.om = oracle_model(sub, fi.make_weights(sub, seed, True))
        sel = np.linspace(0, self.B - 1, self.rows).astype(int)
        l_sel = [int(lens[b]) for b in sel]
        self.caps = [n + 2 for n in l_sel]
        self.okv = stand_in_cache(sub, l_sel, self.caps, seed, True)
        self.len0, self.pos0 = self.okv.len.copy(), self.okv.pos.copy()
        self.toks = fi.tokens(sub, self.rows, seed, "oracle_tokens")

    def step(self):
        rows, layers, oracle = self.rows, self.layers, self.oracle
        self.okv.len[:], self.okv.pos[:] = self.len0, self.pos0  # every timed step sees the same cache lengths
        t0 = time.perf_counter()
        oracle.decode_step(self.om, self.toks, np.zeros((rows, layers), np.uint8), self.okv)
        t_head = (time.perf_counter() - t0) / rows
        self.okv.pos[:] = self.pos0
        t0 = time.perf_counter()
        oracle.decode_step(self.om, self.toks, np.ones((rows, layers), np.uint8), self.okv)
        t_all = time.perf_counter() - t0
        t_layer = max(t_all - t_head * rows, 0.0) / (rows * layers)
        step_s = self.kept * t_layer + self.B * t_head
        cores = len(os.sched_getaffinity(0))
        return dict(value=self.B / step_s, unit=UNIT, cores=cores, kind="oracle",
                    sample=f"{rows} of {self.B} sequences x {layers} of {self.L} layers + lm_head, 1 step, bf16-valued "
                           f"weights; {t_layer * 1e3:.1f} ms per (sequence, kept layer), {t_head * 1e3:.1f} ms per "
                           f"sequence for norm+lm_head; extrapolated to {self.kept} kept (sequence, layer) pairs",
                    ms_per_step=step_s * 1e3)


def oracle_sample(shape, mask, lens, seed, rows=4, layers=2):
    return OracleSample(shape, mask, lens, seed, rows, layers).step()


def run_reference(args, wl, shape, mask, lens):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = OracleSample(shape, mask, lens, 100, rows=min(mask.shape[0], 8), layers=2)  # built once, stepped K times
    vals = []
    for i in range(args.warmup + args.steps):
        r = sample.step()
        if i >= args.warmup:
            vals.append(r)
    ms = float(np.mean([v["ms_per_step"] for v in vals]))
    value = mask.shape[0] / (ms / 1e3)
    cb = dict(vals[-1])
    cb["value"] = value
    cb.pop("ms_per_step")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": args.workload, "shape": wl["shape"], "batch_per_gpu": int(mask.shape[0]),
                      "prompt_lengths": [int(lens.min()), int(lens.max())], "mask": list(wl["mask"]),
                      "skip_fraction": float(1 - mask.mean()),
                      "note": "host oracle on a bounded sample of this workload, extrapolated"},
           "cpu_baseline": cb,
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def prefill_leg(torch, FirstContext, shape, weights, kv, lens, caps, dev, peaks, max_tokens=40000, opts=()):
    """The prompt phase that precedes the timed decode steps, on this workload's prompts (the first sequences of
    the batch up to `max_tokens` prompt tokens): one first_prefill call with routers, timed with CUDA events.
    Reported beside the decode metric, not part of it; it overwrites the stand-in caches, so it runs last."""
    s, L = shape, shape.n_layers
    nb = int(max(1, np.searchsorted(np.cumsum(lens), max_tokens, side="right")))
    pl = lens[:nb]
    total = int(pl.sum())
    ctx = FirstContext(shape, 1, max(256, nb), int(caps.max()), weights)
    for o in opts:
        name, val = o.split("=")
        ctx.set_option(name, int(val))
    cu = np.concatenate([[0], np.cumsum(pl)]).astype(np.int32)
    toks = torch.from_numpy(fi.tokens(shape, total, 11)).to(dev)
    g = torch.Generator(device=dev)
    g.manual_seed(99)
    rw = 0.02 * torch.randn((L, s.d_model), device=dev, generator=g)
    mask = torch.zeros((nb, L), dtype=torch.uint8, device=dev)
    nxt = torch.empty((nb,), dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    ctx.prefill(toks[:int(cu[1])], cu[:2], kv, rw, None, 0.5, 0, mask[:1], None, None, nxt[:1])  # warm-up: one prompt
    torch.cuda.synchronize()
    l0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    ctx.prefill(toks, cu, kv, rw, None, 0.5, 0, mask, None, None, nxt)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    flags = ctx.device_flags()
    if flags:
        raise RuntimeError(f"device flags set during the prefill leg: {flags}")
    proj = 2.0 * s.layer_params() * L * total + 2.0 * s.vocab * s.d_model * nb
    attn = float(sum(2.0 * int(n) * int(n) * s.head_dim * s.n_q_heads * L for n in pl))
    tf = (proj + attn) / ms / 1e9
    pk = float(peaks.get("bf16_tflops_sustained", 1400.0))
    out = {"sequences": nb, "prompt_tokens": total, "ms": ms, "tokens_per_s": total / ms * 1e3,
           "model_tflops": tf, "frac_of_bf16_sustained_peak": tf / pk, "gpu_launches": int(ctx.launch_count() - l0),
           "chunk_rows": 256, "kept_fraction_routed": float(mask.float().mean().item()),
           "note": "prompt tokens as rows of the decode-step kernels, 256 per chunk; weights streamed once per chunk"}
    if not any(o.startswith("prefill_lo=") for o in opts):
        # for information: the same call with the projections on the bfloat16 hi half of the activations alone
        # (plain bf16 activations: half the tensor work; outside this library's parity bar, so not the default)
        ctx.set_option("prefill_lo", 0)
        e0.record(stream)
        ctx.prefill(toks, cu, kv, rw, None, 0.5, 0, mask, None, None, nxt)
        e1.record(stream)
        torch.cuda.synchronize()
        ctx.set_option("prefill_lo", 1)
        ms2 = e0.elapsed_time(e1)
        out["bf16_activations_for_information"] = {
            "ms": ms2, "tokens_per_s": total / ms2 * 1e3, "frac_of_bf16_sustained_peak": (proj + attn) / ms2 / 1e9 / pk,
            "option": "prefill_lo=0",
            "note": "first-token logits 2.3e-2 of the logit range off the oracle at the 8B shape (bar 2e-2): not the default"}
    return out


def join_leg(torch, job, mask, lens, room, changes=8):
    """Cost of a batch change between steps: the job's batch decodes through a slab pool laid over the same cache
    tensors (slabs only for kept (sequence, layer) pairs); then, `changes` times, one sequence leaves, another
    (same prompt length, another mask row) joins, the plan is rebuilt from the host masks, and the next step runs.
    Host time of leave + join + commit, and the device time of the first step after the change against a steady
    step (a change that moves a layer's row count into another bucket of 16 records a new step graph)."""
    from paper_2410_12513_b200 import FirstPool
    ctx, B, L = job.ctx, job.B, job.L
    pool = FirstPool(ctx, B, job.kk, job.vv)
    caps = [int(n) + room + 1 for n in lens]
    slots = [pool.join(mask[b], caps[b], None, 0, int(lens[b])) for b in range(B)]
    pool.commit()
    stream = job.stream

    def step_ms(n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        a, b = job.tok_a, job.tok_b
        for _ in range(n):
            ctx.decode_step(a, pool.kv, None, b)
            a, b = b, a
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    job.tok_a.copy_(job.tok0)
    step_ms(3)
    steady = step_ms(8)
    held0 = pool.stats()[0].sum()
    rng = np.random.default_rng(11)
    host_us, first_ms = [], []
    g0 = ctx.graph_count()
    for i in range(changes):
        b = int(rng.integers(0, B))
        row = mask[int(rng.integers(0, B))]
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        pool.leave(slots[b])
        slots[b] = pool.join(row, caps[b], None, 0, int(lens[b]))
        pool.commit()
        host_us.append((time.perf_counter() - t0) * 1e6)
        first_ms.append(step_ms(1))
        step_ms(2)
    flags = ctx.device_flags()
    rec = {"steady_ms_per_step_through_pool": steady, "host_us_leave_join_commit_median": float(np.median(host_us)),
           "first_step_after_change_ms_median": float(np.median(first_ms)),
           "first_step_after_change_ms_max": float(np.max(first_ms)), "changes": changes,
           "step_graphs_recorded_during_changes": int(ctx.graph_count() - g0),
           "kv_rows_held": int(held0), "kv_rows_if_every_layer_had_a_slab": int(sum(caps)) * L, "device_flags": int(flags),
           "note": "no call of a change waits for the stream; rows held = sum over kept (sequence, layer) slabs"}
    pool.close()
    return rec


# ----------------------------------------------------------------------------- replicas (N > 1)
def init_replica():
    """(rank, world, local device index, dist module or None, device for the max-over-ranks tensor).
    Sequences are independent, so N GPUs run N independent replicas: the only communication is the
    barrier around the timed region and the max over ranks of the device time (NCCL under torchrun,
    gloo when bench.py starts the replicas itself)."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world == 1:
        return rank, world, local, None, None
    import torch.distributed as dist
    backend = os.environ.get("FIRST_BENCH_BACKEND", "nccl")
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        return rank, world, local, dist, torch.device("cuda", local)
    dist.init_process_group("gloo")
    return rank, world, local, dist, torch.device("cpu")


def free_port():
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_replicas(n, argv, script=None, backend="gloo", timeout=3600):
    """Start n copies of `script argv` (default: this file), replica i on GPU i alone (CUDA_VISIBLE_DEVICES=i,
    LOCAL_RANK 0), joined by a 127.0.0.1 rendezvous.  Rank 0's standard output is passed through; the return
    value is the largest exit code."""
    script = [str(Path(__file__).resolve())] if script is None else list(script)
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE=str(n), LOCAL_RANK="0", LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES=str(r),
                   FIRST_BENCH_BACKEND=backend)
        procs.append(subprocess.Popen([sys.executable, *script, *argv], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    t_end = time.time() + timeout
    for pr in procs:
        try:
            rc = max(rc, abs(pr.wait(timeout=max(1.0, t_end - time.time()))))
        except subprocess.TimeoutExpired:
            pr.kill()  # this replica's own process, by handle
            rc = max(rc, 124)
    return rc


# ----------------------------------------------------------------------------- CUDA arm
def make_weights_dev(torch, s, dev, g):
    def rnd(shp, std):
        t = torch.empty(shp, dtype=torch.bfloat16, device=dev)
        t.normal_(0.0, std, generator=g)
        return t

    def gain():
        return torch.ones(s.d_model, device=dev) + 0.02 * torch.randn(s.d_model, device=dev, generator=g)

    w = {"embed": rnd((s.vocab, s.d_model), 0.02), "lm_head": rnd((s.vocab, s.d_model), 0.02), "final_norm": gain()}
    for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down"):
        w[k] = []
    for _ in range(s.n_layers):
        w["attn_norm"].append(gain())
        w["ffn_norm"].append(gain())
        w["wqkv"].append(rnd((s.q_dim + 2 * s.kv_dim, s.d_model), 0.02))
        w["wo"].append(rnd((s.d_model, s.q_dim), 0.02))
        w["w_gate_up"].append(rnd((2 * s.ffn_dim, s.d_model), 0.02))
        w["w_down"].append(rnd((s.d_model, s.ffn_dim), 0.02))
    return w


class Job:
    """One workload resident on one GPU: weights, stand-in caches of `lens` tokens with room for `room`
    more, a context, and the timed loops over it."""

    def __init__(self, torch, shape, weights, lens, room, dev, rank, dist, dist_dev, opts=()):
        from paper_2410_12513_b200 import FirstContext, KVCache
        self.torch, self.shape, self.lens, self.dev, self.dist, self.dist_dev = torch, shape, lens, dev, dist, dist_dev
        s, L, B = shape, shape.n_layers, len(lens)
        self.B, self.L = B, L
        g = torch.Generator(device=dev)
        g.manual_seed(4321 + rank)
        caps = (lens + room + 1).astype(np.int32)
        off = np.concatenate([[0], np.cumsum(caps[:-1], dtype=np.int64)]).astype(np.int64)
        tot = int(caps.sum())
        self.caps = caps

        def rnd(shp):
            t = torch.empty(shp, dtype=torch.bfloat16, device=dev)
            t.normal_(0.0, 1.0, generator=g)
            return t

        self.kk = [rnd((s.n_kv_heads, tot, s.head_dim)) for _ in range(L)]
        self.vv = [rnd((s.n_kv_heads, tot, s.head_dim)) for _ in range(L)]
        self.len0 = torch.from_numpy(np.broadcast_to(lens.astype(np.int32), (L, B)).copy()).to(dev)
        self.pos0 = torch.from_numpy(lens.astype(np.int32)).to(dev)
        self.len_t, self.pos_t = self.len0.clone(), self.pos0.clone()
        self.kv = KVCache(self.kk, self.vv, torch.from_numpy(off).to(dev), torch.from_numpy(caps).to(dev),
                          self.len_t, self.pos_t)
        self.ctx = FirstContext(shape, 1, B, int(caps.max()), weights)
        for o in opts:
            name, val = o.split("=")
            self.ctx.set_option(name, int(val))
        self.tok0 = torch.from_numpy(fi.tokens(shape, B, 7 + rank)).to(dev)
        self.tok_a, self.tok_b = self.tok0.clone(), self.tok0.clone()
        self.stream = torch.cuda.current_stream()

    def close(self):
        self.ctx.close()
        self.kk = self.vv = self.kv = None
        self.torch.cuda.empty_cache()

    def reset(self):
        self.len_t.copy_(self.len0)
        self.pos_t.copy_(self.pos0)
        self.tok_a.copy_(self.tok0)

    def steps(self, n):
        a, b = self.tok_a, self.tok_b
        for _ in range(n):
            self.ctx.decode_step(a, self.kv, None, b)
            a, b = b, a

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            self.torch.cuda.synchronize()

    def timed(self, mask, K, W):
        """W untimed + exactly K timed steps under `mask` (numpy [B][L]); -> (ms of the K steps, max over
        ranks; launches)."""
        torch = self.torch
        self.ctx.set_mask(torch.from_numpy(np.ascontiguousarray(mask)).to(self.dev))
        self.reset()
        self.steps(W)
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = self.ctx.launch_count()
        e0.record(self.stream)
        self.steps(K)
        e1.record(self.stream)
        self.barrier()
        ms = max_over_ranks(e0.elapsed_time(e1), self.dist, self.dist_dev)
        return ms, self.ctx.launch_count() - l0

    def step_percentiles(self, mask, n=48, W=5):
        """Per-step latency: an event after every step of an untimed run (the events add nothing to a step that is one
        graph launch); p10 / p50 / p90 in ms."""
        torch = self.torch
        self.ctx.set_mask(torch.from_numpy(np.ascontiguousarray(mask)).to(self.dev))
        self.reset()
        self.steps(W)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        a, b = self.tok_a, self.tok_b
        ev[0].record(self.stream)
        for i in range(n):
            self.ctx.decode_step(a, self.kv, None, b)
            a, b = b, a
            ev[i + 1].record(self.stream)
        torch.cuda.synchronize()
        t = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(n)])
        return {"p10": float(np.percentile(t, 10)), "p50": float(np.percentile(t, 50)), "p90": float(np.percentile(t, 90)),
                "steps": n}

    def in_step_ms(self, mask, n=8):
        """Where a step's time goes while it runs the way it is timed (one graph, dependent launches overlapping):
        every launch stamps first-CTA start / last-warp end; per class, the time from the previous launch's end to
        this launch's end, summed -- the classes add up to the step.  Mean over n steps, ms."""
        torch = self.torch
        self.ctx.set_mask(torch.from_numpy(np.ascontiguousarray(mask)).to(self.dev))
        self.ctx.set_option("stamp", 1)
        self.reset()
        self.steps(3)
        excl, span, cnt = {}, {}, {}
        total = 0.0
        for _ in range(n):
            self.steps(1)
            tr = self.ctx.step_trace()
            prev_end = tr[0][1]
            for name, t0, t1 in tr:
                excl[name] = excl.get(name, 0.0) + max(0, t1 - prev_end) / 1e6
                span[name] = span.get(name, 0.0) + (t1 - t0) / 1e6
                cnt[name] = cnt.get(name, 0) + 1
                prev_end = max(prev_end, t1)
            total += (prev_end - tr[0][1]) / 1e6
        self.ctx.set_option("stamp", 0)
        return ({k: v / n for k, v in excl.items()}, {k: v / n for k, v in span.items()},
                {k: v // n for k, v in cnt.items()}, total / n)


def fractions(bm, ms_step, peak):
    return {"bytes_strict": bm["strict"], "bytes_full": bm["full"],
            "frac_strict_of_measured": bm["strict"] / (ms_step * 1e6) / peak,
            "frac_full_of_measured": bm["full"] / (ms_step * 1e6) / peak,
            "frac_strict_of_8TBps": bm["strict"] / (ms_step * 1e6) / 8000.0,
            "floor_ms_strict_measured_peak": bm["strict"] / peak / 1e6}


def sub_record(torch, name, weights_for, dev, rank, dist, dist_dev, peak, opts, K, W, sweep=False):
    """A compact record of another workload of the benchmark set, measured the same way (W + exactly K steps,
    CUDA events): routed and all-keep step time, bytes and roofline fractions; for the sweep config the six
    skip fractions with aligned and independent masks."""
    wl = WORKLOADS[name]
    shape = SHAPES[wl["shape"]]
    B, L = wl["B"], shape.n_layers
    lens = fi.prompt_lengths(B, wl["lo"], wl["hi"], 1000 + rank)
    mask = make_mask(wl["mask"], B, L, 2000 + rank)
    job = Job(torch, shape, weights_for(wl["shape"]), lens, W + K, dev, rank, dist, dist_dev, opts)
    mid = lens + W + K // 2
    try:
        ms, launches = job.timed(mask, K, W)
        dense_ms, _ = job.timed(np.ones_like(mask), K, W)
        bm, bmd = byte_model(shape, mask, mid), byte_model(shape, np.ones_like(mask), mid)
        rec = {"workload": name, "shape": wl["shape"], "batch": B, "prompt_lengths": [int(lens.min()), int(lens.max())],
               "mask": list(wl["mask"]), "skip_fraction": float(1 - mask.mean()), "steps": K, "warmup": W,
               "ms_per_step": ms / K, "tokens_per_s": job_tokens_per_s(1 if dist is None else dist.get_world_size(), B, K, ms),
               "gpu_launches_per_step": launches / K, **fractions(bm, ms / K, peak),
               "dense": {"ms_per_step": dense_ms / K, "bytes_strict": bmd["strict"],
                         "latency_ratio_routed_over_dense": ms / dense_ms,
                         "bytes_ratio_routed_over_dense": bm["full"] / bmd["full"]}}
        if sweep:
            rows = []
            for frac in (0.0, 0.1, 0.2, 0.3, 0.4, 0.5):
                row = {"skip": frac}
                for kind in ("aligned", "independent"):
                    mk = fi.mask_aligned(B, L, frac) if kind == "aligned" else fi.mask_independent(B, L, frac, 3000 + rank)
                    t, _ = job.timed(mk, K, W)
                    b_ = byte_model(shape, mk, mid)
                    row[kind] = {"ms_per_step": t / K, "bytes_strict": b_["strict"],
                                 "frac_strict_of_measured": b_["strict"] / (t / K * 1e6) / peak,
                                 "latency_over_all_keep": (t / K) / (dense_ms / K)}
                rows.append(row)
            rec["skip_sweep"] = rows
        if job.ctx.device_flags():
            raise RuntimeError(f"device flags set during sub-record {name}")
        return rec
    finally:
        job.close()


def run_cuda(args, wl, shape, mask, lens):
    import torch
    from paper_2410_12513_b200 import FirstContext

    rank, world, local, dist, dist_dev = init_replica()
    dev = torch.device("cuda", local)
    B, L, K, W = mask.shape[0], shape.n_layers, args.steps, args.warmup
    g = torch.Generator(device=dev)
    g.manual_seed(1234 + rank)
    s = shape
    w_cache = {}

    def weights_for(shape_key):
        if shape_key not in w_cache:
            w_cache.clear()  # one model resident at a time
            torch.cuda.empty_cache()
            w_cache[shape_key] = make_weights_dev(torch, shape if shape_key == wl["shape"] else SHAPES[shape_key], dev, g)
        return w_cache[shape_key]

    weights = weights_for(wl["shape"])
    job = Job(torch, shape, weights, lens, W + K, dev, rank, dist, dist_dev, args.opt)
    ctx, kv, caps, stream = job.ctx, job.kv, job.caps, job.stream
    peaks = {}
    try:
        peaks = json.loads((ROOT / "MEASURED_PEAKS.json").read_text())
    except Exception:
        pass
    peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured (MEASURED_PEAKS.json hbm_gbs)" if "hbm_gbs" in peaks else "fallback 6650 GB/s"

    if args.prefill_only:
        if rank == 0:
            print(json.dumps({"prefill_only": True, "layers": L, "options": args.opt,
                              "prefill": prefill_leg(torch, FirstContext, shape, weights, kv, lens, caps, dev, peaks, opts=args.opt),
                              "note": "profiling case, not a benchmark value"}))
        return

    # ---- routing + plan, once per batch (reported, not part of the step)
    route = None
    if rank == 0 and not args.no_route and not args.quick:
        n_tok = int(lens.sum())
        hid = torch.empty((n_tok, s.d_model), dtype=torch.bfloat16, device=dev)
        hid.normal_(0.0, 1.0, generator=g)
        cu = torch.from_numpy(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)).to(dev)
        rw = 0.02 * torch.randn(s.d_model, device=dev, generator=g)
        rmask = torch.zeros((B, L), dtype=torch.uint8, device=dev)
        for _ in range(3):
            ctx.prefill_route(0, hid, cu, rw, None, 0.5, 0, rmask)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        reps = 10
        for i in range(reps):
            ctx.prefill_route(i % L, hid, cu, rw, None, 0.5, 0, rmask)
        e1.record(stream)
        torch.cuda.synchronize()
        rms = e0.elapsed_time(e1) / reps
        route = {"ms_per_layer": rms, "hidden_bytes": n_tok * s.d_model * 2, "router_mode": "mean of per-token sigmoids",
                 "GBps": n_tok * s.d_model * 2 / rms / 1e6, "tokens": n_tok}
        del hid

    sampler = ClockSampler(physical_gpu_index(local))
    with sampler:
        ms_total, launches = job.timed(mask, K, W)
    clocks = sampler.summary()
    ms_step = ms_total / K
    value = job_tokens_per_s(world, B, K, ms_total)

    if args.quick:
        if rank == 0:
            print(json.dumps({"quick": True, "ms_per_step": ms_step, "value": value, "layers": L,
                              "gpu_launches": int(launches), "note": "profiling case, not a benchmark value"}))
        return
    dense_ms, dense_launches = job.timed(np.ones_like(mask), K, W)
    dense_ms /= K
    repeat_ms, _ = job.timed(mask, K, W)  # the routed run once more, after the dense one (order effects show here)
    repeat_ms /= K

    # Step latency against the skip rate, on this workload's batch and caches: a short version (three rates, both
    # mask structures); the six rates on this workload with --sweep (the sweep config itself is a sub-record).
    sweep = []
    for frac in ((0.0, 0.1, 0.2, 0.3, 0.4, 0.5) if args.sweep else (0.0, 0.25, 0.5)):
        row = {"skip": frac}
        for kind in ("aligned", "independent"):
            mk = fi.mask_aligned(B, L, frac) if kind == "aligned" else fi.mask_independent(B, L, frac, 3000 + rank)
            ms, _ = job.timed(mk, K, W)
            bmk = byte_model(shape, mk, lens + W + K // 2)
            row[kind] = {"ms_per_step": ms / K, "bytes_strict": bmk["strict"]}
        sweep.append(row)

    # ---- end to end through the public call with host buffers
    ctx.set_mask(torch.from_numpy(mask).to(dev))
    job.reset()
    tok_a, tok_b = job.tok_a, job.tok_b
    h_tok = torch.from_numpy(fi.tokens(shape, B, 7 + rank)).pin_memory()
    h_next = torch.empty(B, dtype=torch.int32).pin_memory()

    def e2e_steps(n):
        for _ in range(n):
            tok_a.copy_(h_tok, non_blocking=True)
            ctx.decode_step(tok_a, kv, None, tok_b)
            h_next.copy_(tok_b, non_blocking=True)
            stream.synchronize()
            h_tok.copy_(h_next)

    e2e_steps(W)
    job.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    e2e_steps(K)
    e1.record(stream)
    job.barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, dist_dev)
    e2e = {"value": job_tokens_per_s(world, B, K, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": B * 4,
           "d2h_bytes_per_step": B * 4, "ms_per_step": e2e_ms / K}

    pct = job.step_percentiles(mask, n=min(48, K), W=W)
    # ---- where the step's time goes: in-step stamps (nothing serialised), then event pairs (serialised)
    excl_ms, span_ms, cls_launches, traced_step_ms = job.in_step_ms(mask)
    ctx.set_mask(torch.from_numpy(mask).to(dev))
    job.reset()
    job.steps(2)
    torch.cuda.synchronize()
    kp = min(K, 16)
    ctx.profile(True)
    job.steps(kp)
    prof = ctx.profile_read()
    ctx.profile(False)
    flags = ctx.device_flags()
    if flags:
        raise RuntimeError(f"device flags set during the benchmark: {flags}")

    mid_lens = lens + W + K // 2
    bm = byte_model(shape, mask, mid_lens)
    bm_dense = byte_model(shape, np.ones_like(mask), mid_lens)
    cls_ms = {k: v[0] / kp for k, v in prof.items() if v[1]}
    cnt = mask.sum(0)
    proj_bytes = bm["weights"] + bm["lm_head"]
    alg = {"gemv_rows": proj_bytes, "gemm_tc": proj_bytes, "attn_split": bm["kv"]}
    if cls_ms.get("gemv_rows") and cls_ms.get("gemm_tc"):
        alg = {"attn_split": bm["kv"]}  # projections split over two classes: attribute by class below
    dom = max(excl_ms, key=excl_ms.get)
    traffic = None
    try:  # DRAM bytes of the projection launches from the committed ncu capture, if the kernel is unchanged since
        import hashlib
        tj = json.loads((ROOT / "profiles" / "traffic_gemm_tc_cfg2.json").read_text())
        cur = hashlib.sha256((ROOT / tj["source"]).read_bytes()).hexdigest()[:16]
        if dom == "gemm_tc" and cur == tj["source_sha256_16"] and wl["shape"] == "8b":
            bl = tj["bytes_per_launch"]
            traffic = int((cnt > 0).sum()) * (bl["qkv"] + bl["o"] + bl["gate_up"] + bl["down"]) + bl["lm_head"]
    except Exception:
        traffic = None
    roof = {"bound": "hbm", "kernel": dom, "unit": "GB/s", "peak": peak, "peak_kind": peak_kind, "traffic": traffic,
            "traffic_note": "per step, scaled from the 2-layer ncu capture in profiles/ (per launch x launches)" if traffic else None,
            "ms_per_step": excl_ms[dom], "share_of_step": excl_ms[dom] / max(traced_step_ms, 1e-9),
            "launches_per_step": cls_launches.get(dom),
            "timing": "in-step: every launch stamps its first CTA's start and last warp's end (global ns timer) while the "
                      "step runs as timed (one CUDA graph, dependent launches overlapping); a class's time is the sum, over "
                      "its launches, of (this launch's end - previous launch's end), so the classes add up to the step",
            "ms_per_step_event_pairs": cls_ms.get(dom),
            "event_pairs_note": "CUDA event pair around every launch (serialises the step: an upper bound on the class's time)"}
    if dom in alg:
        roof["achieved"] = alg[dom] / excl_ms[dom] / 1e6
        roof["frac"] = roof["achieved"] / peak
        roof["algorithmic_bytes_per_step"] = alg[dom]
    else:
        roof["achieved"] = None
        roof["frac"] = None
    in_step = {k: {"ms": excl_ms[k], "span_ms": span_ms[k], "launches": cls_launches[k],
                   **({"GBps": alg[k] / excl_ms[k] / 1e6, "frac_of_measured": alg[k] / excl_ms[k] / 1e6 / peak}
                      if k in alg and excl_ms[k] > 0 else {})} for k in excl_ms}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
           "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "bf16", "data": "synthetic",
           "config": {"workload": args.workload, "shape": wl["shape"], "batch_per_gpu": B,
                      "prompt_lengths": [int(lens.min()), int(lens.max())], "mask": list(wl["mask"]),
                      "skip_fraction": float(1 - mask.mean()), "l2": "inputs larger than L2 (weights + KV >> 126 MB)",
                      "parallelism": "replicas" if world > 1 else "single",
                      **({"options": args.opt} if args.opt else {}),
                      **({"layers": L, "note": "reduced layer count: not a benchmark value"} if args.layers else {})},
           "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
           "roofline": roof,
           "step_roofline": fractions(bm, ms_step, peak),
           "dense": {"ms_per_step": dense_ms, "gpu_launches": int(dense_launches), "bytes_strict": bm_dense["strict"],
                     "latency_ratio_routed_over_dense": ms_step / dense_ms,
                     "bytes_ratio_routed_over_dense": bm["full"] / bm_dense["full"]},
           "ms_per_step_repeat": repeat_ms, "step_latency_ms": pct, "skip_sweep": sweep,
           "kernel_ms_in_step": in_step, "traced_step_ms": traced_step_ms,
           "kernel_ms_per_step_event_pairs": cls_ms, "route": route}
    if not args.no_join and rank == 0:
        out["batch_change"] = join_leg(torch, job, mask, lens, W + K)
    if not args.no_prefill and rank == 0:
        out["prefill"] = prefill_leg(torch, FirstContext, shape, weights, kv, lens, caps, dev, peaks, opts=args.opt)
    job.close()
    if not args.no_sub and not args.layers and not args.opt and args.workload == "cfg2_8b_b32":
        # the other workloads of the benchmark set, each measured the same way (every rank runs them: replicas)
        subs = {}
        for name, k_sub, sweep_sub in (("cfg4_8b_b64", 32, True), ("cfg3_8b_b256", 32, False), ("cfg1_1b_b1", 128, False)):
            try:
                subs[name] = sub_record(torch, name, weights_for, dev, rank, dist, dist_dev, peak, args.opt, k_sub, 5, sweep_sub)
            except Exception as e:  # a sub-record never takes the main line down
                subs[name] = {"error": f"{type(e).__name__}: {e}"[:300]}
        out["workloads"] = subs
    if rank == 0:
        if not args.no_cpu_baseline:
            out["cpu_baseline"] = oracle_sample(shape, mask, lens, 5, rows=min(B, 32), layers=4)
            out["cpu_baseline"].pop("ms_per_step", None)
        print(json.dumps(out))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg2_8b_b32", choices=sorted(WORKLOADS))
    ap.add_argument("--mask", default=None, help="override: dense | aligned:F | independent:F | fraction:LO:HI | bernoulli:P | unified:EVERY | random:F")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-route", action="store_true")
    ap.add_argument("--no-prefill", action="store_true", help="skip the prompt-phase leg (first_prefill on this workload's prompts)")
    ap.add_argument("--prefill-only", action="store_true",
                    help="only the prompt-phase leg (for profiler captures with --layers; not a benchmark line)")
    ap.add_argument("--opt", action="append", default=[], help="library option name=value (A/B runs)")
    ap.add_argument("--layers", type=int, default=None,
                    help="reduced layer count: a small case for profiler captures, never a benchmark value")
    ap.add_argument("--sweep", action="store_true",
                    help="time six skip fractions 0..50 %% (aligned and independent masks) on this workload instead of three")
    ap.add_argument("--no-join", action="store_true", help="skip the batch-change leg (slab pool: leave + join + plan rebuild)")
    ap.add_argument("--no-sub", action="store_true", help="skip the sub-records of the other benchmark workloads")
    ap.add_argument("--quick", action="store_true",
                    help="only the main timed loop (for profiler captures): no dense/e2e/per-kernel legs")
    args = ap.parse_args()
    wl = dict(WORKLOADS[args.workload])
    if args.mask:
        parts = args.mask.split(":")
        wl["mask"] = tuple([parts[0]] + [float(x) for x in parts[1:]])
    if args.steps is None:
        args.steps = 64 if args.impl == "cuda" else 2
    if args.impl == "cuda" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under torchrun: start the N replicas here, one process per GPU
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))
    if args.impl == "cuda" and not args.quick:
        args.warmup = max(args.warmup, 3)
    shape = SHAPES[wl["shape"]]
    if args.layers:
        d = shape.asdict()
        d["n_layers"] = args.layers
        shape = fi.ModelShape(**d)
    rank = int(os.environ.get("RANK", "0"))
    lens = fi.prompt_lengths(wl["B"], wl["lo"], wl["hi"], 1000 + rank)
    mask = make_mask(wl["mask"], wl["B"], shape.n_layers, 2000 + rank)
    if args.impl == "reference":
        run_reference(args, wl, shape, mask, lens)
    else:
        run_cuda(args, wl, shape, mask, lens)


if __name__ == "__main__":
    main()
