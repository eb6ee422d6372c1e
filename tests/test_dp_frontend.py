"""Data-parallel front-end on CPU: the batching window and scatter plan of the C-ABI batcher (host code, no GPU
needed), and the scatter / pad / gather path with two gloo ranks whose worker is the float64 oracle."""
import os
import threading
import time

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth


def test_batch_is_due_when_full_or_when_the_oldest_request_has_waited_the_window():
    with binding.Batcher(max_batch=4, n_workers=2, local_batch=2, window_ms=60.0) as b:
        t0 = time.perf_counter()
        assert b.next(timeout_ms=20.0) == [] and time.perf_counter() - t0 >= 0.015        # nothing pending: times out
        for i in range(3):
            b.submit(100 + i)
        t0 = time.perf_counter()
        got = b.next(timeout_ms=1000.0)
        waited = time.perf_counter() - t0
        assert got == [100, 101, 102] and 0.04 <= waited < 0.5                            # window, not timeout
        for i in range(6):
            b.submit(i)
        t0 = time.perf_counter()
        assert b.next(timeout_ms=1000.0) == [0, 1, 2, 3] and time.perf_counter() - t0 < 0.03   # full: at once
        assert b.pending() == 2
        assert b.next(timeout_ms=1000.0) == [4, 5]


def test_a_late_submit_from_another_thread_joins_the_open_window():
    with binding.Batcher(max_batch=8, n_workers=2, local_batch=4, window_ms=80.0) as b:
        b.submit(1)
        threading.Timer(0.02, lambda: b.submit(2)).start()
        assert b.next(timeout_ms=1000.0) == [1, 2]


def test_plan_fills_workers_in_order_and_marks_padding():
    with binding.Batcher(max_batch=32, n_workers=8, local_batch=4, window_ms=20.0) as b:
        slots, active = b.plan(32)
        assert active == 8 and slots[0] == [0, 1, 2, 3] and slots[7] == [28, 29, 30, 31]
        slots, active = b.plan(6)
        assert active == 2 and slots[0] == [0, 1, 2, 3] and slots[1] == [4, 5, -1, -1] and slots[2] == [-1] * 4
        slots, active = b.plan(0)
        assert active == 0 and all(s == [-1] * 4 for s in slots)
        with pytest.raises(binding.PhyaiError):
            b.plan(33)
    with pytest.raises(binding.PhyaiError):
        binding.Batcher(max_batch=9, n_workers=2, local_batch=4, window_ms=1.0)               # 2 x 4 < 9


def _requests(cfg, n):
    return [dict(prefix_kv=synth.make_prefix_kv(cfg, 1, 5 + 3 * i, i), state=synth.make_state(cfg, 1, i),
                 noise=synth.make_noise(cfg, 1, i), n_steps=2) for i in range(n)]


def _oracle_worker(cfg, W):
    def run(local):
        out = []
        for r in local:
            if r is None:
                out.append(np.zeros((cfg.horizon, cfg.action_dim)))     # the padded slot still produces a row
            else:
                out.append(O.denoise(cfg, W, r["prefix_kv"], r["prefix_kv"].shape[2], r["state"], r["noise"], r["n_steps"]))
        return out
    return run


def _rank_main(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_03682_b200.frontend import DPFrontend
    cfg = synth.tiny_config()
    W = O.Weights(synth.make_weights(cfg, 1))
    fe = DPFrontend(_oracle_worker(cfg, W), local_batch=2, window_ms=10.0)
    results = {}
    if rank == 0:
        reqs = _requests(cfg, 5)
        ids = [fe.submit(r) for r in reqs]
    for _ in range(2):                      # 5 requests, 2 workers x 2 slots: a full batch of 4, then 1 + 3 padding
        out = fe.serve_round(timeout_ms=500.0)
        if rank == 0:
            results.update(out)
    assert fe.serve_round(stop=True) is None
    if rank == 0:
        assert sorted(results) == ids
        for rid, r in zip(ids, reqs):
            ref = O.denoise(cfg, W, r["prefix_kv"], r["prefix_kv"].shape[2], r["state"], r["noise"], 2)
            assert np.array_equal(results[rid], ref)
        ret.put("ok")
    fe.close()
    dist.destroy_process_group()


def test_two_ranks_scatter_pad_gather_and_every_request_gets_its_own_answer():
    ctx = mp.get_context("spawn")
    ret = ctx.SimpleQueue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, 29741, ret)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    assert ret.get() == "ok"
