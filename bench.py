#!/usr/bin/env python
"""Benchmark of the action-expert denoising loop on B200.

One "step" = one whole action chunk: one call of the hot path (embedding, all layers, head and
Euler update for every integration step) over one batch of synthetic input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2|C3|C4|C5b1|...] [--impl reference]

Prints ONE JSON line.  ``value`` is measured with the inputs resident in device memory and CUDA
events on the launching stream; ``e2e`` goes through the host-buffer entry point (pinned host
inputs, host<->device copies inside the timed region).  ``--impl reference`` times the float64 CPU
oracle on the host cores instead.  Under torchrun every rank runs an independent replica (the
path shards by request, no collective); rank 0 reports the maximum time over ranks.

Workloads: C2 (pi0-shaped, bf16, batch 1: the headline), C2m (C2 with the block-causal mask), C3 (pi0.5-shaped), C4
(batch 64, ragged prefixes), C5b1 / b8 / b64 / b256 (e4m3 weights), C6b8 / b64 / b256 (e4m3 weights and per-token e4m3
activations: W8A8), C7b1 (int4 weights), G1 (a GR00T-shaped feature-handoff head: K / V projections of the features,
then four steps on a 40 x 132 chunk).  A run without --workload reports C2 on the line and the others in ``workloads``.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_03682_b200 import synth  # noqa: E402

METRIC = "ms per action chunk (batch 1, 10 steps)"
METRIC_BATCHED = "chunks/sec at batch %d"
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures
# summarised under profiles/ (bench.py cannot run ncu itself)
NCU_TRAFFIC = {"C2": (180 * 37.41e6 + 10 * 2.8e6, "profiles/cluster_loop_c2_c5_batch1.md"),
               "C5b1": (180 * 20.39e6 + 10 * 2.8e6, "profiles/cluster_loop_c2_c5_batch1.md"),
               "C7b1": (180 * 11.70e6 + 10 * 2.8e6, "profiles/cluster_loop_c2_c5_batch1.md")}
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1590.0


# ------------------------------------------------------------------------------------------------
# workloads
# ------------------------------------------------------------------------------------------------
def workload(name: str):
    """(cfg, cfg_id, batch, prefix lengths, n_steps)"""
    if name == "C1":
        return synth.tiny_config(), 1, 1, [64], 4
    if name == "C2":
        return synth.pi0_config(), 2, 1, [816], 10
    if name == "C2m":   # C2 with the block-causal suffix mask (state token cached once per call)
        return synth.pi0_config().with_(suffix_block_causal=True), 2, 1, [816], 10
    if name == "C3":
        return synth.pi05_config(), 3, 1, [968], 10
    if name == "C4":
        lens = synth.make_ragged_lengths(4, 64, 600, 968)
        return synth.pi0_config(max_batch=64), 4, 64, [int(x) for x in lens], 10
    if name.startswith("C5b"):
        b = int(name[3:])
        return synth.pi0_config(max_batch=b, dtype="w8e4m3", max_prefix_len=816), 5, b, [816] * b, 10
    if name.startswith("C7b"):   # the C5 expert with 4-bit integer weights (W4A16)
        b = int(name[3:])
        return synth.pi0_config(max_batch=b, dtype="w4a16", max_prefix_len=816), 5, b, [816] * b, 10
    if name.startswith("C6b"):   # the C5 expert in the W8A8 mode: per-token e4m3 activations, FP8 tensor path
        b = int(name[3:])
        return synth.pi0_config(max_batch=b, dtype="w8a8e4m3", max_prefix_len=816), 5, b, [816] * b, 10
    raise SystemExit(f"unknown workload {name}")


def algorithmic_cost(cfg, lens, n_steps):
    """Bytes that must cross HBM and FLOPs per chunk: every big weight once per Euler step, each
    request's prefix KV once per layer per step; activations and tables are cache resident."""
    D, F, L, S = cfg.width, cfg.mlp_dim, cfg.n_layers, cfg.suffix_len
    wbytes = 0.5 if cfg.dtype == "w4a16" else (1 if cfg.dtype in ("w8e4m3", "w8a8e4m3") else (4 if cfg.dtype == "f32" else 2))
    ebytes = 4 if cfg.dtype == "f32" else 2
    nqkv = cfg.q_dim + 2 * cfg.kv_dim
    per_layer_params = D * nqkv + cfg.q_dim * D + 2 * D * F + F * D
    embed_params = D * D + (cfg.action_dim * D) + D * cfg.action_dim if cfg.cond == "pi0" else 2 * cfg.action_dim * D
    B = len(lens)
    kv_bytes = sum(lens) * L * 2 * cfg.kv_dim * ebytes
    bytes_step = L * per_layer_params * wbytes + embed_params * ebytes + kv_bytes
    lin_flops = 2 * B * S * L * per_layer_params + (2 * B * cfg.horizon * D * D if cfg.cond == "pi0" else 0)
    attn_flops = sum(4 * S * (p + S) * cfg.n_q_heads * cfg.head_dim for p in lens) * L
    return bytes_step * n_steps, (lin_flops + attn_flops) * n_steps


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS, bf16_tflops_sustained=1400.0,
                source="fallback")


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])), mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # samples under load: the upper half of the observed clocks (idle samples precede the run)
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# oracle timing (CPU baseline and the reference arm)
# ------------------------------------------------------------------------------------------------
def time_oracle(cfg, cfg_id, lens, n_steps, budget_s: float, repeats: int = 1, warm: int = 0):
    """Times the float64 oracle as it stands on a bounded sample: one request, ``sample_steps`` of
    the ``n_steps`` Euler steps (all steps cost the same), scaled to a whole batch of chunks."""
    from oracle import expert_oracle as O

    W = O.Weights(synth.make_weights(cfg, cfg_id))
    P = lens[0]
    kv = O.to_f64(synth.make_prefix_kv(cfg, cfg_id, P, 0))
    state = synth.make_state(cfg, cfg_id, 0) if cfg.has_state_token else None
    st = None if state is None else O.to_f64(state)
    x = O.to_f64(synth.make_noise(cfg, cfg_id, 0))
    t0 = time.perf_counter()
    O.velocity(cfg, W, kv, P, st, x, 1.0)
    one = time.perf_counter() - t0
    per_call = budget_s / max(1, repeats + warm)
    sample_steps = int(max(1, min(n_steps, per_call // max(one, 1e-9))))
    times = []
    for i in range(warm + repeats):
        t0 = time.perf_counter()
        xx = x
        for k in range(sample_steps):
            xx = xx + (-1.0 / n_steps) * O.velocity(cfg, W, kv, P, st, xx, 1.0 - k / n_steps)
        if i >= warm:
            times.append(time.perf_counter() - t0)
    scale = (n_steps / sample_steps) * len(lens)
    ms_per_batch = float(np.mean(times)) * 1e3 * scale
    sample = (f"1 of {len(lens)} request(s) (prefix {P}), {sample_steps} of {n_steps} Euler steps, "
              f"scaled x{scale:g}; {repeats} timed repeat(s)")
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count()
    return ms_per_batch, sample, cores


# ------------------------------------------------------------------------------------------------
# one workload on the CUDA path
# ------------------------------------------------------------------------------------------------
def percentiles(ms):
    a = np.sort(np.asarray(ms, dtype=np.float64))
    return {"mean": float(a.mean()), "p50": float(np.percentile(a, 50)), "p99": float(np.percentile(a, 99)),
            "min": float(a[0]), "max": float(a[-1])}


def roofline_of(name, cfg, lens, n_steps, batch, ms_per_step, peaks):
    alg_bytes, alg_flops = algorithmic_cost(cfg, lens, n_steps)
    secs = ms_per_step / 1e3
    if batch < 8:
        achieved = alg_bytes / secs / 1e9
        traffic = NCU_TRAFFIC.get(name, (None, None))
        return {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": traffic[0], "traffic_source": traffic[1],
                "kernel": "whole captured loop (one graph launch = one chunk: all Euler steps and layers)",
                "peak_source": f"{peaks['source']} copy bandwidth", "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": alg_bytes}
    achieved = alg_flops / secs / 1e12
    if cfg.dtype == "w8a8e4m3":
        # the linear layers (5/6 of the FLOPs) run on the FP8 tensor path: measured bf16 rate x the nominal FP8 : bf16
        # ratio of 2; attention stays bf16, so this peak is an upper bound of what the loop can reach
        pk = 2.0 * peaks["bf16_tflops_sustained"]
        return {"bound": "tensor", "achieved": achieved, "peak": pk, "unit": "TFLOP/s", "frac": achieved / pk, "traffic": None,
                "kernel": "whole captured loop (one graph launch = one batch of chunks)",
                "peak_source": f"2 x {peaks['source']} sustained bf16 GEMM (nominal FP8 : bf16 ratio)",
                "frac_of_bf16_sustained": achieved / peaks["bf16_tflops_sustained"],
                "frac_of_nominal": achieved / (2.0 * NOMINAL_BF16_TFLOPS), "algorithmic_flops_per_launch": alg_flops}
    return {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
            "frac": achieved / peaks["bf16_tflops_sustained"], "traffic": None,
            "kernel": "whole captured loop (one graph launch = one batch of chunks)",
            "peak_source": f"{peaks['source']} sustained bf16 GEMM (the loop runs for tens of ms under the power cap)",
            "frac_of_burst": achieved / peaks["bf16_tflops"], "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS,
            "algorithmic_flops_per_launch": alg_flops}


class Inputs:
    """Host-side synthetic inputs of one workload; requests are generated once and shared by the batch sizes of a
    sweep (request b has the same seed whatever the batch)."""

    def __init__(self, cfg, cfg_id, lens):
        import torch

        self.kvs = [synth.make_prefix_kv(cfg, cfg_id, int(p), b) for b, p in enumerate(lens)]
        self.states = ([synth.make_state(cfg, cfg_id, b) for b in range(len(lens))] if cfg.has_state_token else None)
        self.noise = [synth.make_noise(cfg, cfg_id, b) for b in range(len(lens))]
        self.torch = torch

    def batch(self, n):
        torch = self.torch
        kv_h, cu = synth.pack_prefix_kv(self.kvs[:n])
        states = None if self.states is None else torch.stack(self.states[:n])
        return kv_h, torch.from_numpy(cu), states, torch.stack(self.noise[:n])


def run_workload(name, ex, cfg, lens, n_steps, inputs, K, Wm, world, rank, local_rank, e2e=True, sample_clocks=False):
    """Times one workload on an existing handle: K calls bracketed by one event pair (``ms_per_step``), one event pair
    per call as well (mean / p50 / p99 / min), then the same through the host-buffer entry point."""
    import torch

    from paper_2608_03682_b200 import replicas

    batch = len(lens)
    batched = batch > 1
    kv_h, cu_h, states_h, noise_h = inputs.batch(batch)
    kv_d, noise_d, cu_d = kv_h.cuda(), noise_h.cuda(), cu_h.cuda()
    states_d = None if states_h is None else states_h.cuda()
    out_d = torch.empty_like(noise_d)
    stream = torch.cuda.current_stream()

    def call_device():
        if batched:
            ex.denoise_batched(kv_d, cu_d, states_d, noise_d, n_steps, out=out_d, stream=stream)
        else:
            ex.denoise(kv_d, lens[0], None if states_d is None else states_d[0], noise_d[0], n_steps, out=out_d[0],
                       stream=stream)

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()

    def timed(fn, iters):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
        barrier()
        ev[0].record(stream)
        for i in range(iters):
            fn()
            ev[i + 1].record(stream)
        barrier()
        total = replicas.max_over_ranks(ev[0].elapsed_time(ev[iters]), device="cuda")
        return total, [ev[i].elapsed_time(ev[i + 1]) for i in range(iters)]

    for _ in range(Wm):
        call_device()
    torch.cuda.synchronize()
    status = ex.poll_status()
    if status != 0:
        raise SystemExit(f"{name}: device status {status} after warm-up")
    sampler = ClockSampler(local_rank) if (sample_clocks and rank == 0) else None
    total_ms, per_call = timed(call_device, K)
    clocks = sampler.stop() if sampler else None
    ms_per_step = total_ms / K
    res = {"ms_per_step": ms_per_step, "per_call_ms": percentiles(per_call), "chunks_per_s": world * batch / (ms_per_step / 1e3),
           "clocks": clocks, "launches_per_step": int(ex.launches_per_call(batch, n_steps)), "batch": batch}
    ok = bool(torch.isfinite(out_d).all().item())
    if e2e:
        pin = lambda t: None if t is None else t.pin_memory()
        kv_p, noise_p, states_p, cu_p = pin(kv_h), pin(noise_h), pin(states_h), pin(cu_h)
        out_p = torch.empty_like(noise_h).pin_memory()

        def call_host():
            if batched:
                ex.denoise_batched_host(kv_p, cu_p, states_p, noise_p, n_steps, out_p, stream=stream)
            else:
                ex.denoise_host(kv_p, lens[0], None if states_p is None else states_p[0], noise_p[0], n_steps, out_p[0],
                                stream=stream)

        for _ in range(3):
            call_host()
        e2e_total, _ = timed(call_host, K)
        e2e_ms = e2e_total / K
        h2d = kv_h.numel() * kv_h.element_size() + noise_h.numel() * 4 + (0 if states_h is None else states_h.numel() * 4)
        if batched:
            h2d += cu_h.numel() * 4
        res["e2e"] = {"ms_per_step": e2e_ms, "chunks_per_s": world * batch / (e2e_ms / 1e3), "h2d_bytes_per_step": int(h2d),
                      "d2h_bytes_per_step": int(noise_h.numel() * 4)}
        ok = ok and bool(torch.isfinite(out_p).all().item())
    status = ex.poll_status()
    if status != 0:
        raise SystemExit(f"{name}: device status {status} after the timed region")
    res["finite"] = ok
    del kv_d, noise_d, cu_d, states_d, out_d
    return res


def free_port():
    import socket

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def respawn_replicas(n: int) -> int:
    """``--gpus N`` outside torchrun: start N replica processes of this script (one per GPU, rendezvous on the loopback
    address) and hand their output through.  Rank 0 of the children prints the JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=None,
                    help="time one workload only (C1, C2, C3, C4, C5b1, C5b8, C5b64, C5b256, C6b8 ... C6b256: W8A8); default: C2 as the headline "
                         "plus every other configuration of the metric in the line's `workloads` map")
    ap.add_argument("--impl", default="phyai", choices=["phyai", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--opt", action="append", default=[], metavar="KEY=VALUE",
                    help="library option set on the handle before timing (phyai_set_option), may repeat")
    args = ap.parse_args()
    K, Wm = args.steps, max(args.warmup, 3)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(respawn_replicas(args.gpus))

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    head = args.workload or "C2"
    cfg, cfg_id, batch, lens, n_steps = workload(head)
    batched = batch > 1
    metric = (METRIC_BATCHED % batch) if batched else METRIC
    unit = "chunks/s" if batched else "ms"

    def describe(name, cfg, batch, lens, n_steps):
        return (f"{name}: {cfg.cond}-shaped expert, {cfg.dtype}, batch {batch}, prefix {min(lens)}..{max(lens)}, "
                f"{cfg.suffix_len} suffix tokens, {n_steps} Euler steps")

    config = {"workload": describe(head, cfg, batch, lens, n_steps), "batch": batch, "n_steps": n_steps, "replicas": world,
              "l2": "inputs larger than L2 (weights streamed per step exceed 126 MB); no flush"}

    # -------------------------------------------------------------------------- reference arm
    if args.impl == "reference":
        if rank != 0:
            return
        ms, sample, cores = time_oracle(cfg, cfg_id, lens, n_steps, budget_s=120.0, repeats=K, warm=min(Wm, 1))
        value = batch / (ms / 1e3) if batched else ms
        line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": K,
                "warmup": Wm, "ms_per_step": ms, "higher_is_better": batched, "scaling": "weak", "vs_baseline": None,
                "dtype": "f64", "data": "synthetic", "config": config,
                "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    # -------------------------------------------------------------------------- CUDA arm
    import torch

    from paper_2608_03682_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = measured_peaks()

    def make_expert(cfg, cfg_id):
        W = synth.make_weights(cfg, cfg_id)
        ex = binding.Expert(cfg, binding.weights_to_device(W))
        del W
        if args.no_graph:
            ex.set_option("use_graph", 0)
        for kv_ in args.opt:
            key, _, val = kv_.partition("=")
            ex.set_option(key, int(val))
        return ex

    ex = make_expert(cfg, cfg_id)
    inputs = Inputs(cfg, cfg_id, lens)
    res = run_workload(head, ex, cfg, lens, n_steps, inputs, K, Wm, world, rank, local_rank, sample_clocks=True)
    ex.close()
    del inputs
    torch.cuda.empty_cache()

    # every other configuration the metric names, on fewer calls: batch 64 (C4), the adaRMS expert (C3), the e4m3 sweep
    others = {}
    if args.workload is None and world == 1:
        Ko, Wo = min(K, 10), 3
        for name in ("C3", "C4"):
            c2, id2, b2, l2, n2 = workload(name)
            e2 = make_expert(c2, id2)
            r2 = run_workload(name, e2, c2, l2, n2, Inputs(c2, id2, l2), Ko, Wo, world, rank, local_rank)
            e2.close()
            torch.cuda.empty_cache()
            r2["workload"], r2["steps"], r2["warmup"] = describe(name, c2, b2, l2, n2), Ko, Wo
            r2["roofline"] = roofline_of(name, c2, l2, n2, b2, r2["ms_per_step"], peaks)
            others[name] = r2
        # the block-causal variant of C2, and the same handle with the state token cached once per call
        cm, idm, bm, lm, nm = workload("C2m")
        em = make_expert(cm, idm)
        inm = Inputs(cm, idm, lm)
        rm = run_workload("C2m", em, cm, lm, nm, inm, Ko, Wo, world, rank, local_rank, e2e=False)
        em.set_option("use_state_cache", 1)
        rm["ms_per_step_with_state_cache"] = run_workload("C2m", em, cm, lm, nm, inm, Ko, Wo, world, rank, local_rank,
                                                             e2e=False)["ms_per_step"]
        em.close()
        rm["workload"], rm["steps"], rm["warmup"] = describe("C2m", cm, bm, lm, nm) + ", block-causal suffix mask", Ko, Wo
        rm["roofline"] = roofline_of("C2m", cm, lm, nm, bm, rm["ms_per_step"], peaks)
        others["C2m"] = rm
        c5, id5, _, l5, n5 = workload("C5b256")
        e5 = make_expert(c5, id5)                       # one handle (max_batch 256) serves the whole sweep
        in5 = Inputs(c5, id5, l5)
        for b5 in (1, 8, 64, 256):
            name = f"C5b{b5}"
            r5 = run_workload(name, e5, c5, l5[:b5], n5, in5, Ko if b5 < 256 else min(Ko, 5), Wo, world, rank, local_rank,
                              e2e=(b5 <= 64))
            if b5 == 1:   # the single-tile path streams the e4m3 bytes; for comparison: the bf16 images made at create
                e5.set_option("use_w8_inkernel", 0)
                r5["ms_per_step_bf16_images"] = run_workload(name, e5, c5, l5[:b5], n5, in5, Ko, Wo, world, rank, local_rank,
                                                             e2e=False)["ms_per_step"]
                e5.set_option("use_w8_inkernel", 1)
            r5["workload"], r5["steps"], r5["warmup"] = describe(name, c5, b5, l5[:b5], n5), Ko, Wo
            r5["roofline"] = roofline_of(name, c5, l5[:b5], n5, b5, r5["ms_per_step"], peaks)
            others[name] = r5
        e5.close()
        torch.cuda.empty_cache()
        # the same expert and requests in the W8A8 mode (FP8 tensor path)
        c6, id6, _, l6, n6 = workload("C6b256")
        e6 = make_expert(c6, id6)
        for b6 in (8, 64, 256):
            name = f"C6b{b6}"
            r6 = run_workload(name, e6, c6, l6[:b6], n6, in5, Ko if b6 < 256 else min(Ko, 5), Wo, world, rank, local_rank,
                              e2e=False)
            r6["workload"], r6["steps"], r6["warmup"] = describe(name, c6, b6, l6[:b6], n6), Ko, Wo
            r6["roofline"] = roofline_of(name, c6, l6[:b6], n6, b6, r6["ms_per_step"], peaks)
            others[name] = r6
        e6.close()
        del in5
        torch.cuda.empty_cache()
        # the same expert with 4-bit integer weights at batch 1: the cluster path streams half a byte per weight
        c7, id7, _, l7, n7 = workload("C7b1")
        e7 = make_expert(c7, id7)
        in7 = Inputs(c7, id7, l7)
        r7 = run_workload("C7b1", e7, c7, l7, n7, in7, Ko, Wo, world, rank, local_rank, e2e=False)
        e7.set_option("use_w8_inkernel", 0)
        r7["ms_per_step_bf16_images"] = run_workload("C7b1", e7, c7, l7, n7, in7, Ko, Wo, world, rank, local_rank,
                                                     e2e=False)["ms_per_step"]
        r7["workload"], r7["steps"], r7["warmup"] = describe("C7b1", c7, 1, l7, n7), Ko, Wo
        r7["roofline"] = roofline_of("C7b1", c7, l7, n7, 1, r7["ms_per_step"], peaks)
        others["C7b1"] = r7
        e7.close()
        del in7
        torch.cuda.empty_cache()
        # a feature-handoff head of the shape the paper's GR00T profile names (40 x 132 chunk, four steps): the
        # request-local K / V projections of the features, then the loop on the projected prefix
        from paper_2608_03682_b200 import binding as _b
        cg = synth.groot_like_config()
        eg = make_expert(cg, 6)
        feat_dim, n_feat = 2048, 640
        feats = synth.make_features(6, n_feat, feat_dim).cuda()
        wk, wv = synth.make_kv_projections(cg, 6, feat_dim)
        wk, wv = [w.cuda() for w in wk], [w.cuda() for w in wv]
        proj = _b.KvProjector(wk, wv, cg.n_kv_heads, cg.head_dim, max_tokens=n_feat)
        kvg = proj.run(feats)
        for _ in range(3):
            proj.run(feats, out=kvg)
        torch.cuda.synchronize()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record()
        for _ in range(10):
            proj.run(feats, out=kvg)
        p1.record()
        torch.cuda.synchronize()
        proj_ms = p0.elapsed_time(p1) / 10
        proj.close()
        st_g, nz_g = synth.make_state(cg, 6).cuda(), synth.make_noise(cg, 6).cuda()
        out_g = torch.empty_like(nz_g)
        for _ in range(Wo):
            eg.denoise(kvg, n_feat, st_g, nz_g, 4, out=out_g)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(Ko):
            eg.denoise(kvg, n_feat, st_g, nz_g, 4, out=out_g)
        e1.record()
        torch.cuda.synchronize()
        others["G1"] = {"workload": "G1: feature-handoff head (GR00T-shaped: 16 layers, width 1024, 8 / 2 heads of 128, 41 suffix "
                                    f"tokens, action 40 x 132), bf16, batch 1, {n_feat} feature tokens of {feat_dim}, 4 Euler steps",
                        "ms_per_step": e0.elapsed_time(e1) / Ko, "kv_projection_ms": proj_ms,
                        "kv_projection_note": "once per request: feature rows -> per-layer K / V (projector handle, CUDA events)",
                        "launches_per_step": int(eg.launches_per_call(1, 4)), "steps": Ko, "warmup": Wo,
                        "finite": bool(torch.isfinite(out_g).all().item()) and eg.poll_status() == 0,
                        "roofline": roofline_of("G1", cg, [n_feat], 4, 1, e0.elapsed_time(e1) / Ko, peaks)}
        eg.close()
        torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = res["ms_per_step"]
    roofline = roofline_of(head, cfg, lens, n_steps, batch, ms_per_step, peaks)
    value = res["chunks_per_s"] if batched else ms_per_step
    e2e_value = res["e2e"]["chunks_per_s"] if batched else res["e2e"]["ms_per_step"]
    launches = res["launches_per_step"]
    line = {"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_per_step, "per_call_ms": res["per_call_ms"], "higher_is_better": batched, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if cfg.dtype != "f32" else "f32", "data": "synthetic", "config": config,
            "chunks_per_s": res["chunks_per_s"], "clocks": res["clocks"],
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": res["e2e"]["h2d_bytes_per_step"],
                    "d2h_bytes_per_step": res["e2e"]["d2h_bytes_per_step"], "ms_per_step": res["e2e"]["ms_per_step"]},
            "gpu_launches": int(launches * K), "launches_per_step": int(launches), "finite": res["finite"],
            "roofline": roofline}
    if others:
        line["workloads"] = others
        if "C4" in others:
            line["chunks_per_s_batch64"] = others["C4"]["chunks_per_s"]
            line["tensor_frac_batch64"] = others["C4"]["roofline"]["frac"]

    if not args.no_cpu_baseline and world == 1:
        ms, sample, cores = time_oracle(cfg, cfg_id, lens, n_steps, budget_s=15.0, repeats=1)
        line["cpu_baseline"] = {"value": batch / (ms / 1e3) if batched else ms, "unit": unit, "cores": cores,
                                "kind": "oracle", "sample": sample}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
