"""The oracle's invariants checked THROUGH the GPU library (C ABI), plus boundary behaviour:
zero / constant velocity head, NaN beyond prefix_len, prefix permutation, aliasing, handle reuse,
run-to-run determinism, argument errors."""
import numpy as np
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth
from tests.helpers import BAR, rel_err, small_bf16_config

pytestmark = pytest.mark.gpu


def fp32_cfg(**kw):
    base = dict(n_layers=2, width=96, mlp_dim=160, n_q_heads=4, n_kv_heads=2, head_dim=24, state_dim=5, action_dim=7,
                horizon=9, has_state_token=True, max_prefix_len=40, cond="pi0", dtype="f32")
    base.update(kw)
    return synth.ExpertConfig(**base)


def inputs(cfg, cfg_id, P, kv_tokens=None):
    kv = synth.make_prefix_kv(cfg, cfg_id, kv_tokens or P)
    state = synth.make_state(cfg, cfg_id) if cfg.has_state_token else None
    return kv, state, synth.make_noise(cfg, cfg_id)


def run(ex, kv, P, state, noise, n, out=None):
    o = ex.denoise(kv.cuda(), P, None if state is None else state.cuda(), noise.cuda(), n, out=out)
    torch.cuda.synchronize()
    assert ex.poll_status() == 0
    return o


CONFIGS = [("fp32", lambda: fp32_cfg(), 21, 0.08), ("bf16-pi0", lambda: small_bf16_config("pi0"), 22, 0.05),
           ("bf16-pi05", lambda: small_bf16_config("pi05"), 23, 0.05)]


@pytest.mark.parametrize("name,make,cfg_id,std", CONFIGS)
def test_zero_velocity_head_returns_the_noise_bit_exactly(name, make, cfg_id, std):
    cfg = make()
    W = synth.make_weights(cfg, cfg_id, std=std)
    W["action_out_w"] = torch.zeros_like(W["action_out_w"])
    W["action_out_b"] = torch.zeros_like(W["action_out_b"])
    kv, state, noise = inputs(cfg, cfg_id, 30)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        out = run(ex, kv, 30, state, noise, 4)
    assert torch.equal(out.cpu(), noise)


@pytest.mark.parametrize("name,make,cfg_id,std", CONFIGS)
def test_constant_velocity_head_gives_x0_minus_c(name, make, cfg_id, std):
    cfg = make()
    W = synth.make_weights(cfg, cfg_id, std=std)
    W["action_out_w"] = torch.zeros_like(W["action_out_w"])
    c = W["action_out_b"].float()
    kv, state, noise = inputs(cfg, cfg_id, 30)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        out = run(ex, kv, 30, state, noise, 5)
    np.testing.assert_allclose(out.cpu().numpy(), (noise - c[None, :]).numpy(), rtol=0, atol=2e-6)


@pytest.mark.parametrize("name,make,cfg_id,std", CONFIGS)
def test_rows_beyond_prefix_len_are_never_read(name, make, cfg_id, std):
    cfg = make()
    W = synth.make_weights(cfg, cfg_id, std=std)
    P = 27
    kv, state, noise = inputs(cfg, cfg_id, P, kv_tokens=P + 9)
    poisoned = kv.clone()
    poisoned[:, :, P:] = float("nan")
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        a = run(ex, kv, P, state, noise, 3).clone()
        b = run(ex, poisoned, P, state, noise, 3).clone()
    assert torch.isfinite(b).all() and torch.equal(a, b)


@pytest.mark.parametrize("name,make,cfg_id,std", CONFIGS)
def test_permuting_prefix_tokens_with_their_kv_changes_nothing_beyond_rounding(name, make, cfg_id, std):
    cfg = make()
    W = synth.make_weights(cfg, cfg_id, std=std)
    P = 33
    kv, state, noise = inputs(cfg, cfg_id, P)
    perm = torch.from_numpy(np.random.default_rng(5).permutation(P))
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        a = run(ex, kv, P, state, noise, 3).double().cpu().numpy()
        b = run(ex, kv[:, :, perm].contiguous(), P, state, noise, 3).double().cpu().numpy()
    # only the summation order inside the softmax / PV changes
    assert rel_err(b, a) <= (1e-5 if cfg.dtype == "f32" else 5e-3)


def test_out_actions_may_alias_noise_and_handles_are_reusable():
    cfg = small_bf16_config("pi0")
    W = synth.make_weights(cfg, 24, std=0.05)
    kv, state, noise = inputs(cfg, 24, 180)
    Wd = binding.weights_to_device(W)
    with binding.Expert(cfg, Wd) as ex:
        ref = run(ex, kv, 150, state, noise, 4).clone()
        x = noise.cuda().clone()
        ex.denoise(kv.cuda(), 150, state.cuda(), x, 4, out=x)     # in place
        torch.cuda.synchronize()
        assert torch.equal(x, ref)
        # other prefix lengths and step counts on the same handle, then the first one again
        other = run(ex, kv, 77, state, noise, 2).clone()
        again = run(ex, kv, 150, state, noise, 4).clone()
        assert torch.equal(again, ref) and not torch.equal(other, ref)
    with binding.Expert(cfg, Wd) as fresh:
        assert torch.equal(run(fresh, kv, 77, state, noise, 2), other)
    r = O.denoise(cfg, W, kv, 77, state, noise, 2)
    assert rel_err(other.double().cpu().numpy(), r) <= BAR["bf16"]


def test_graph_replay_and_direct_launch_give_identical_results():
    cfg = small_bf16_config("pi05")
    W = synth.make_weights(cfg, 25, std=0.05)
    kv, state, noise = inputs(cfg, 25, 99)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        a = run(ex, kv, 99, state, noise, 3).clone()
        a2 = run(ex, kv, 99, state, noise, 3).clone()
        ex.set_option("use_graph", 0)
        b = run(ex, kv, 99, state, noise, 3).clone()
    assert torch.equal(a, a2) and torch.equal(a, b)


def test_argument_errors_are_status_codes():
    cfg = small_bf16_config("pi0")
    W = synth.make_weights(cfg, 26, std=0.05)
    kv, state, noise = inputs(cfg, 26, 50)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        with pytest.raises(binding.PhyaiError) as e:
            ex.denoise(kv.cuda(), 51, state.cuda(), noise.cuda(), 2)          # prefix_len > kv_tokens
        assert e.value.status == binding.ERR_INVALID_ARG
        with pytest.raises(binding.PhyaiError) as e:
            ex.denoise(kv.cuda(), 50, state.cuda(), noise.cuda(), 0)          # n_steps == 0
        assert e.value.status == binding.ERR_INVALID_ARG
        with pytest.raises(binding.PhyaiError) as e:
            ex.denoise(kv.cuda(), 50, None, noise.cuda(), 2)                  # state missing
        assert e.value.status == binding.ERR_INVALID_ARG
        big = synth.make_prefix_kv(cfg, 26, cfg.max_prefix_len + 8)
        with pytest.raises(binding.PhyaiError) as e:
            ex.denoise(big.cuda(), cfg.max_prefix_len + 1, state.cuda(), noise.cuda(), 2)
        assert e.value.status == binding.ERR_INVALID_ARG
        with pytest.raises(binding.PhyaiError):
            ex.set_option("no_such_option", 1)
        out = ex.denoise(kv.cuda(), 50, state.cuda(), noise.cuda(), 2)         # the handle still works
        torch.cuda.synchronize()
        assert ex.poll_status() == 0 and bool(torch.isfinite(out).all())


def test_host_buffer_entry_points_match_the_device_ones():
    cfg = small_bf16_config("pi0", max_batch=3)
    W = synth.make_weights(cfg, 27, std=0.05)
    lens = [90, 0, 200]
    kvs = [synth.make_prefix_kv(cfg, 27, p, b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 27, b) for b in range(3)])
    noise = torch.stack([synth.make_noise(cfg, 27, b) for b in range(3)])
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        dev = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), 3).cpu()
        host_out = torch.empty_like(noise).pin_memory()
        ex.denoise_batched_host(packed.pin_memory(), torch.from_numpy(cu).pin_memory(), states.pin_memory(),
                                noise.pin_memory(), 3, host_out)
        torch.cuda.synchronize()
        assert torch.equal(host_out, dev)
        single = torch.empty_like(noise[2]).pin_memory()
        ex.denoise_host(kvs[2].pin_memory(), 200, states[2].pin_memory(), noise[2].pin_memory(), 3, single)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        assert rel_err(single.double().numpy(), dev[2].double().numpy()) <= BAR["bf16"]


def test_timer_stamps_of_the_tile_kernels_are_ordered_and_do_not_change_the_result():
    """Tracing aid at more than 1024 suffix tokens: with "trace_all_from" = i every CTA of launch i (a tile GEMM or the
    tcgen05 attention kernel) stamps one slot; the stamps of a slot are in order, the number of slots is the launch's
    grid, and a traced call returns the same action chunk as an untraced one (to the rounding of the atomic split-K
    adds)."""
    cfg = small_bf16_config("pi0", max_batch=90, max_prefix_len=96, head_dim=256, n_q_heads=4)
    W = synth.make_weights(cfg, 41, std=0.05)
    lens = [96 - (5 * b) % 60 for b in range(90)]
    kvs = [synth.make_prefix_kv(cfg, 41, p, b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 41, b) for b in range(90)])
    noise = torch.stack([synth.make_noise(cfg, 41, b) for b in range(90)])
    args = (packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), 2)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        plain = ex.denoise_batched(*args).double().cpu().numpy()
        ex.set_option("trace", 1)
        traced_launches = 0
        for launch in range(1, 12):
            ex.set_option("trace_all_from", launch)
            out = ex.denoise_batched(*args).double().cpu().numpy()
            assert ex.poll_status() == 0
            assert rel_err(out, plain) <= BAR["bf16"]
            tr = ex.read_trace().astype(np.int64)
            r = tr[tr[:, 0] != 0]
            if len(r) == 0:
                continue
            traced_launches += 1
            assert len(r) <= 148 * 4
            attention = r[:, 10].max() == 1
            order = (0, 1, 2, 3, 4, 5, 6, 8) if attention else (0, 1, 2, 3, 4)
            for a, b in zip(order[:-1], order[1:]):
                assert (r[:, b] >= r[:, a]).all(), (launch, a, b)
            assert (r[:, 8] >= r[:, 6]).all() and (r[:, 6] >= r[:, 5]).all()
            assert (r[:, 8] - r[:, 0]).max() < 1e9           # ns: a CTA lives microseconds, not seconds
        assert traced_launches >= 4                           # q|k|v, attention, O, gate/up, down of the first layer
