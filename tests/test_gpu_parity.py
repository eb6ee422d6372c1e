"""GPU parity: the CUDA library (through the C ABI) against the float64 oracle on the same seeded
inputs.  Bars: max relative error on the final action chunk <= 1e-4 (fp32), <= 2e-2 (bf16 / e4m3)."""
import numpy as np
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth
from tests.helpers import BAR, gpu_single, rel_err, small_bf16_config

pytestmark = pytest.mark.gpu


def _inputs(cfg, cfg_id, P, request=0):
    kv = synth.make_prefix_kv(cfg, cfg_id, P, request)
    state = synth.make_state(cfg, cfg_id, request) if cfg.has_state_token else None
    noise = synth.make_noise(cfg, cfg_id, request)
    return kv, state, noise


# ------------------------------------------------------------------------------------------ C1
@pytest.mark.parametrize("use_graph", [True, False])
def test_tiny_fp32_config_matches_oracle(use_graph):
    cfg = synth.tiny_config()
    W = synth.make_weights(cfg, 1)
    kv, state, noise = _inputs(cfg, 1, 64)
    ref = O.denoise(cfg, W, kv, 64, state, noise, 4)
    got = gpu_single(cfg, W, kv, 64, state, noise, 4, use_graph=use_graph)
    assert rel_err(got, ref) <= BAR["f32"], rel_err(got, ref)


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
@pytest.mark.parametrize("opts", [dict(), dict(rope_theta=0.0), dict(gelu_exact=True),
                                  dict(suffix_block_causal=True)])
def test_fp32_variants_match_oracle(cond, opts):
    cfg = synth.ExpertConfig(n_layers=2, width=96, mlp_dim=160, n_q_heads=4, n_kv_heads=2, head_dim=24, state_dim=5,
                             action_dim=7, horizon=9, has_state_token=True, max_prefix_len=40, cond=cond,
                             dtype="f32", **opts)
    W = synth.make_weights(cfg, 11, std=0.08)
    for P in (0, 1, 37):
        kv, state, noise = _inputs(cfg, 11, P)
        ref = O.denoise(cfg, W, kv, P, state, noise, 3)
        got = gpu_single(cfg, W, kv, P, state, noise, 3)
        assert rel_err(got, ref) <= BAR["f32"], (P, rel_err(got, ref))


# ------------------------------------------------------------------------------------------ bf16, reduced
@pytest.mark.parametrize("cond", ["pi0", "pi05"])
@pytest.mark.parametrize("engine", ["simt", "auto"])
def test_small_bf16_expert_matches_oracle(cond, engine):
    cfg = small_bf16_config(cond)
    W = synth.make_weights(cfg, 12, std=0.05)
    for P in (0, 77, 200):
        kv, state, noise = _inputs(cfg, 12, P)
        ref = O.denoise(cfg, W, kv, P, state, noise, 4)
        got = gpu_single(cfg, W, kv, P, state, noise, 4, engine=engine)
        bar = BAR["f32"] if engine == "simt" else BAR["bf16"]
        assert rel_err(got, ref) <= bar, (P, rel_err(got, ref))


# ------------------------------------------------------------------------------------------ C2 / C3
@pytest.mark.parametrize("name", ["C2", "C3"])
def test_pi_shaped_bf16_batch1_matches_oracle(name):
    wl = synth.WORKLOADS[name]
    cfg = synth.pi0_config() if name == "C2" else synth.pi05_config()
    W = synth.make_weights(cfg, wl["cfg_id"])
    kv, state, noise = _inputs(cfg, wl["cfg_id"], wl["prefix"])
    ref = O.denoise(cfg, W, kv, wl["prefix"], state, noise, wl["n_steps"])
    got = gpu_single(cfg, W, kv, wl["prefix"], state, noise, wl["n_steps"])
    err = rel_err(got, ref)
    print(f"{name}: max rel err {err:.3e}, ||ref||inf {np.abs(ref).max():.3f}")
    assert err <= BAR["bf16"], err
