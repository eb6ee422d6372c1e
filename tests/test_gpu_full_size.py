"""Parity at the benchmark's full sizes, in the launch configuration bench.py times, on sampled
requests the oracle can compute one by one: the ragged batch-64 workload and the e4m3-weight sweep."""
import numpy as np
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth
from tests.helpers import BAR, elem_rel_err, rel_err, w8a8_bar

pytestmark = pytest.mark.gpu


def _run_batched(cfg, cfg_id, W, lens, n_steps, check):
    kvs = [synth.make_prefix_kv(cfg, cfg_id, int(p), b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    B = len(lens)
    states = torch.stack([synth.make_state(cfg, cfg_id, b) for b in range(B)])
    noise = torch.stack([synth.make_noise(cfg, cfg_id, b) for b in range(B)])
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        out = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), n_steps)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        out = out.double().cpu().numpy()
    assert np.isfinite(out).all()
    Wf = O.Weights(W)
    errs = {}
    for b in check:
        ref = O.denoise(cfg, Wf, kvs[b], int(lens[b]), states[b], noise[b], n_steps)
        errs[b] = rel_err(out[b], ref)
        print(f"request {b}: max rel err {errs[b]:.2e}, element-wise (floored) {elem_rel_err(out[b], ref):.2e}")
    return errs


def test_batch64_ragged_rollout_matches_oracle_on_sampled_requests():
    cfg = synth.pi0_config(max_batch=64)
    lens = synth.make_ragged_lengths(4, 64, 600, 968)
    order = np.argsort(lens)
    check = sorted({0, 63, int(order[0]), int(order[-1])})
    errs = _run_batched(cfg, 4, synth.make_weights(cfg, 4), lens, 10, check)
    print("C4 max rel err per sampled request:", {b: f"{e:.2e}" for b, e in errs.items()})
    assert max(errs.values()) <= BAR["bf16"], errs


@pytest.mark.parametrize("batch", [1, 8, 64, 256])
def test_e4m3_weight_expert_matches_oracle(batch):
    """Every batch size of the e4m3-weight sweep: 1 (cluster split-K kernels), 8 (general kernel, 128-token tiles,
    split-K with per-channel scales), 64 and 256 (192 / 256-token tiles, rotary epilogue with scales, tcgen05
    attention); up to three sampled requests per batch against the oracle."""
    cfg = synth.pi0_config(max_batch=batch, dtype="w8e4m3", max_prefix_len=816)
    W = synth.make_weights(cfg, 5)
    check = [0] if batch == 1 else ([0, batch - 1] if batch == 8 else [0, batch // 2, batch - 1])
    errs = _run_batched(cfg, 5, W, [816] * batch, 10, check)
    print(f"C5 batch {batch} max rel err:", {b: f"{e:.2e}" for b, e in errs.items()})
    assert max(errs.values()) <= BAR["w8e4m3"], errs


@pytest.mark.parametrize("batch", [1, 8, 64])
def test_w8a8_expert_matches_oracle(batch):
    """The pi0-shaped expert with e4m3 weights and per-token e4m3 activations (FP8 tensor path) against the oracle's
    W8A8 mode on sampled requests, within the tolerance that the mode's own quantization noise sets (see w8a8_bar)."""
    cfg = synth.pi0_config(max_batch=batch, dtype="w8a8e4m3", max_prefix_len=816)
    W = synth.make_weights(cfg, 5)
    check = [0] if batch == 1 else [0, batch - 1]
    errs = _run_batched(cfg, 5, W, [816] * batch, 10, check)
    Wf = O.Weights(W)
    for b in check:
        kv, st, nz = synth.make_prefix_kv(cfg, 5, 816, b), synth.make_state(cfg, 5, b), synth.make_noise(cfg, 5, b)
        ref = O.denoise(cfg, Wf, kv, 816, st, nz, 10)
        bar, d_q = w8a8_bar(cfg, Wf, kv, 816, st, nz, 10, ref)
        print(f"W8A8 batch {batch} request {b}: max rel err {errs[b]:.2e}, quantization noise of the mode {d_q:.2e}, bar {bar:.2e}")
        assert errs[b] <= bar, (b, errs[b], bar)


@pytest.mark.parametrize("batch", [1, 64])
def test_w4a16_expert_matches_oracle(batch):
    """The pi0-shaped expert with 4-bit integer weights against the oracle on sampled requests."""
    cfg = synth.pi0_config(max_batch=batch, dtype="w4a16", max_prefix_len=816)
    W = synth.make_weights(cfg, 5)
    check = [0] if batch == 1 else [0, batch - 1]
    errs = _run_batched(cfg, 5, W, [816] * batch, 10, check)
    print(f"W4A16 batch {batch} max rel err:", {b: f"{e:.2e}" for b, e in errs.items()})
    assert max(errs.values()) <= BAR["w4a16"], errs
