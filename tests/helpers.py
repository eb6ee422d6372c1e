"""Shared helpers of the GPU parity tests: run the CUDA library and the oracle on the same inputs."""
import numpy as np
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth

BAR = {"f32": 1e-4, "bf16": 2e-2, "w8e4m3": 2e-2, "w4a16": 2e-2}   # max relative error on the final action chunk


def gpu_single(cfg, W, kv, P, state, noise, n_steps, engine="auto", use_graph=True, expert=None):
    """One request through phyai_denoise; returns the [H,A] result as float64 numpy."""
    ex = expert or binding.Expert(cfg, binding.weights_to_device(W), engine=engine)
    try:
        if not use_graph:
            ex.set_option("use_graph", 0)
        out = ex.denoise(kv.cuda(), P, None if state is None else state.cuda(), noise.cuda(), n_steps)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        return out.double().cpu().numpy()
    finally:
        if expert is None:
            ex.close()


def small_bf16_config(cond="pi0", **kw):
    """A reduced expert whose dimensions still satisfy the tensor path's tiling (multiples of 128)
    and span several tiles: 3 layers, width 256, MLP 512, 2 query heads of 128."""
    base = dict(n_layers=3, width=256, mlp_dim=512, n_q_heads=2, n_kv_heads=1, head_dim=128, state_dim=6,
                action_dim=5, horizon=13, has_state_token=(cond == "pi0"), max_prefix_len=200, max_batch=1,
                cond=cond, dtype="bf16")
    base.update(kw)
    return synth.ExpertConfig(**base)


def rel_err(got, ref):
    return O.max_rel_err(got, ref)


def elem_rel_err(got, ref):
    """Element-wise relative error with a floor on the denominator, max over the chunk:
    |got - ref| / max(|ref|, 1e-3 * ||ref||_inf).  Reported beside the gated metric, not gated itself: some of the
    1600 outputs of a chunk are ~1e-3 in magnitude, where even exact fp32 arithmetic cannot give 1e-4 element-wise."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    floor = 1e-3 * np.max(np.abs(ref))
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), floor)))


def w8a8_bar(cfg, W, kv, P, state, noise, n_steps, ref_w8a8):
    """Tolerance of a whole-network W8A8 comparison.  The activation quantizer is a step function with steps of
    1/16 .. 1/8 of an element: the bf16-level differences between the device's activations and the oracle's move a few
    per cent of the elements across a step, and each such element then differs by a whole step -- noise of the same
    kind, and nearly the same size, as the quantization noise of the mode itself.  That size is measured on the
    case at hand as the distance d_q between the oracle's W8A8 and W8A16 results; the device result must lie within
    2.5 d_q of the W8A8 oracle (and within 15 % in any case).  The arithmetic of the mode itself -- codes, scales,
    FP8 product -- is checked exactly in test_gpu_w8a8.py."""
    import dataclasses
    cfg16 = dataclasses.replace(cfg, dtype="w8e4m3")
    d_q = O.max_rel_err(O.denoise(cfg16, W, kv, P, state, noise, n_steps), ref_w8a8)
    return min(0.15, 2.5 * d_q), d_q
