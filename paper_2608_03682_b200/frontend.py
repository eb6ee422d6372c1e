"""Data-parallel serving front-end (paper, Sec. "Parallel Execution" and the appendix on eight-GPU serving).

Requests are independent, so N GPUs are N replicas of the single-GPU path that exchange no state while they
compute.  What the front-end adds sits around the loop: rank 0 collects pending requests in a batching window
(``binding.Batcher``: at most ``max_batch``, at most ``window_ms`` after the oldest arrived), gives every worker a
fixed local batch -- the shape its CUDA graph was captured for --, pads the local inputs to that shape, and drops the
padded outputs after the gather.  The only communication is that scatter and gather (``torch.distributed`` object
collectives: NCCL-backed groups on GPUs, gloo on CPU); nothing crosses ranks inside the denoising loop.

A worker is any callable ``worker(requests) -> list of [H, A] arrays`` over ``local_batch`` entries, ``None`` marking
padding.  ``ExpertWorker`` runs them through ``phyai_denoise_batched``.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional

import numpy as np
import torch
import torch.distributed as dist


class ExpertWorker:
    """Runs a fixed-shape local batch on one GPU.  A request is a dict with ``prefix_kv`` ``[L, 2, P, Hkv, dh]``,
    ``state`` ``[Ds]`` or None, ``noise`` ``[H, A]`` (host tensors) and ``n_steps``; padding entries become requests
    with an empty prefix and zero inputs, so the batch (and with it the captured graph) keeps its shape."""

    def __init__(self, expert, cfg, n_steps: int, device="cuda"):
        self.ex, self.cfg, self.n_steps, self.device = expert, cfg, n_steps, device
        self.stream = None      # created on first use (CUDA only)

    def launch(self, requests: List[Optional[dict]]):
        """Enqueue one local batch on the worker's own stream and return at once (the paper's RTC schedule prepares the
        next action chunk while the current one is being executed: a caller launches the next request here and
        collects it when the controller is ready for the hand-over).  One batch in flight per worker."""
        cfg = self.cfg
        if self.stream is None:
            self.stream = torch.cuda.Stream(device=self.device)
        kv_dtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        empty = torch.zeros(cfg.n_layers, 2, 0, cfg.n_kv_heads, cfg.head_dim, dtype=kv_dtype)
        kvs = [empty if r is None else r["prefix_kv"] for r in requests]
        cu = np.zeros(len(requests) + 1, dtype=np.int32)
        cu[1:] = np.cumsum([kv.shape[2] for kv in kvs])
        packed = torch.cat(kvs, dim=2).contiguous()
        if packed.shape[2] == 0:                       # an all-padding batch still needs a valid (non-null) buffer
            packed = torch.zeros(cfg.n_layers, 2, 1, cfg.n_kv_heads, cfg.head_dim, dtype=kv_dtype)
        noise = torch.stack([torch.zeros(cfg.horizon, cfg.action_dim) if r is None else r["noise"] for r in requests])
        states = None
        if cfg.has_state_token:
            states = torch.stack([torch.zeros(cfg.state_dim) if r is None else r["state"] for r in requests])
        host = [packed.pin_memory(), torch.from_numpy(cu).pin_memory(), None if states is None else states.pin_memory(),
                noise.pin_memory()]
        with torch.cuda.stream(self.stream):
            dev = [None if t is None else t.to(self.device, non_blocking=True) for t in host]
            out = self.ex.denoise_batched(dev[0], dev[1], dev[2], dev[3], self.n_steps, stream=self.stream)
            done = torch.cuda.Event()
            done.record(self.stream)
        return {"out": out, "done": done, "keep": (host, dev)}

    def collect(self, pending) -> List[np.ndarray]:
        """Wait for a launched batch and return its action chunks."""
        pending["done"].synchronize()
        status = self.ex.poll_status()
        if status != 0:
            raise RuntimeError(f"device status {status}")
        return [o.cpu().numpy() for o in pending["out"]]

    def __call__(self, requests: List[Optional[dict]]) -> List[np.ndarray]:
        return self.collect(self.launch(requests))


class DPFrontend:
    """One instance per rank.  Rank 0 owns the batcher and the request table; every rank calls ``serve_round`` in
    lock step (rank 0 decides when a batch is due and what it contains)."""

    def __init__(self, worker: Callable[[List[Optional[dict]]], List[np.ndarray]], local_batch: int,
                 window_ms: float = 20.0, max_batch: Optional[int] = None, group=None):
        self.worker, self.local_batch, self.group = worker, local_batch, group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.batcher = None
        self.requests: Dict[int, dict] = {}
        self._next_id = 0
        if self.rank == 0:
            from . import binding
            self.batcher = binding.Batcher(max_batch or self.world * local_batch, self.world, local_batch, window_ms)

    # ---- rank 0, any thread ----
    def submit(self, request: dict) -> int:
        rid = self._next_id
        self._next_id += 1
        self.requests[rid] = request
        self.batcher.submit(rid)
        return rid

    # ---- every rank ----
    def serve_round(self, timeout_ms: float = 100.0, stop: bool = False) -> Optional[Dict[int, np.ndarray]]:
        """One batch: rank 0 takes what is due, scatters the padded local batches, every rank runs its worker, rank 0
        gathers and returns {request id: actions} (other ranks return {}).  Returns None on every rank when rank 0
        passes ``stop`` (shutdown)."""
        payload: List[object] = [None] * self.world
        ids: List[int] = []
        if self.rank == 0:
            if stop:
                payload = ["stop"] * self.world
            else:
                ids = self.batcher.next(timeout_ms)
                slots, _ = self.batcher.plan(len(ids))
                payload = [[None if s < 0 else self.requests[ids[s]] for s in slots[w]] for w in range(self.world)]
        mine = [None]
        if self.world > 1:
            dist.scatter_object_list(mine, payload if self.rank == 0 else None, src=0, group=self.group)
        else:
            mine[0] = payload[0]
        if mine[0] == "stop":
            return None
        local = mine[0]
        # a worker whose whole local batch is padding has nothing to compute
        result = [None] * len(local) if all(r is None for r in local) else self.worker(local)
        gathered: List[object] = [None] * self.world
        if self.world > 1:
            dist.gather_object(result, gathered if self.rank == 0 else None, dst=0, group=self.group)
        else:
            gathered[0] = result
        if self.rank != 0:
            return {}
        out: Dict[int, np.ndarray] = {}
        for i, rid in enumerate(ids):               # request i sits at worker i // local_batch, slot i % local_batch
            out[rid] = gathered[i // self.local_batch][i % self.local_batch]
            del self.requests[rid]
        return out

    def close(self):
        if self.batcher is not None:
            self.batcher.close()
