"""Pins for the float64 oracle: each test checks it against something other than itself - a
closed form, an invariant, a brute-force loop, a library routine or a hand computation - chosen
so that a dropped term, a wrong sign/index or a transposed operand fails at least one."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from oracle import expert_oracle as O
from paper_2608_03682_b200 import synth

torch.set_num_threads(4)


def small_cfg(cond="pi0", D=16, dh=4, Hq=2, Hkv=1, Fm=32, L=2, H=3, ns=True, A=3, Ds=5, P=6, rope=10000.0,
              gelu_exact=False, heads=None):
    if heads is not None:
        Hq, Hkv = heads
    if cond == "pi05":
        ns = False
    return synth.ExpertConfig(n_layers=L, width=D, mlp_dim=Fm, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=dh,
                              state_dim=Ds, action_dim=A, horizon=H, has_state_token=ns, max_prefix_len=max(P, 1),
                              cond=cond, dtype="f32", rope_theta=rope, gelu_exact=gelu_exact)


def rand_inputs(cfg, P, seed=0, std=0.3):
    rng = np.random.default_rng(seed)
    W = {n: rng.standard_normal(s) * std for n, s in synth.weight_shapes(cfg)}
    kv = rng.standard_normal((cfg.n_layers, 2, P, cfg.n_kv_heads, cfg.head_dim))
    state = rng.standard_normal(cfg.state_dim) if cfg.has_state_token else None
    noise = rng.standard_normal((cfg.horizon, cfg.action_dim))
    return W, kv, state, noise


cfg_strategy = st.builds(
    small_cfg,
    cond=st.sampled_from(["pi0", "pi05"]), D=st.sampled_from([8, 16, 32]), dh=st.sampled_from([2, 4, 8]),
    heads=st.sampled_from([(1, 1), (2, 1), (2, 2), (4, 1), (4, 2)]),   # (query heads, kv heads): grouped-query maps a // G
    Fm=st.sampled_from([16, 32]), L=st.integers(1, 3),
    H=st.integers(1, 5), ns=st.booleans(), A=st.integers(1, 7), Ds=st.integers(1, 8), P=st.integers(0, 9),
    rope=st.sampled_from([0.0, 10000.0]), gelu_exact=st.booleans())
fast = settings(max_examples=12, deadline=None, suppress_health_check=list(HealthCheck))


# ------------------------------------------------------------------ loop / Euler update
@fast
@given(cfg=cfg_strategy, n=st.integers(1, 4))
def test_zero_velocity_head_returns_noise_bit_exactly(cfg, n):
    P = cfg.max_prefix_len if cfg.max_prefix_len > 1 else 0
    W, kv, state, noise = rand_inputs(cfg, P, 1)
    W["action_out_w"] = np.zeros_like(W["action_out_w"])
    W["action_out_b"] = np.zeros_like(W["action_out_b"])
    out = O.denoise(cfg, W, kv, P, state, noise, n)
    assert np.array_equal(out, noise)


@fast
@given(cfg=cfg_strategy, n=st.integers(1, 4))
def test_constant_velocity_head_closed_form(cfg, n):
    """W_out = 0, b_out = c  =>  x_n = x_0 + c * sum(dt) = x_0 - c."""
    P = 4
    W, kv, state, noise = rand_inputs(cfg, P, 2)
    W["action_out_w"] = np.zeros_like(W["action_out_w"])
    c = W["action_out_b"]
    out = O.denoise(cfg, W, kv, P, state, noise, n)
    np.testing.assert_allclose(out, noise - c[None, :], rtol=0, atol=1e-13)


def test_time_grid_runs_from_one_towards_zero():
    dt, ts = O.time_grid(4)
    assert dt == -0.25 and ts == [1.0, 0.75, 0.5, 0.25]
    dt, ts = O.time_grid(10)
    assert abs(sum([dt] * 10) + 1.0) < 1e-15 and ts[0] == 1.0 and abs(ts[-1] - 0.1) < 1e-15


def test_single_step_is_one_forward_at_t_equal_one():
    cfg = small_cfg()
    W, kv, state, noise = rand_inputs(cfg, 6, 3)
    v = O.velocity(cfg, O.Weights(W), kv, 6, state, noise, 1.0)
    np.testing.assert_allclose(O.denoise(cfg, W, kv, 6, state, noise, 1), noise - v, rtol=0, atol=1e-15)


def test_two_steps_evaluate_velocity_at_start_of_each_step():
    cfg = small_cfg(cond="pi05")
    W, kv, state, noise = rand_inputs(cfg, 6, 4)
    Wv = O.Weights(W)
    x1 = noise - 0.5 * O.velocity(cfg, Wv, kv, 6, state, noise, 1.0)
    x2 = x1 - 0.5 * O.velocity(cfg, Wv, kv, 6, state, x1, 0.5)
    np.testing.assert_allclose(O.denoise(cfg, W, kv, 6, state, noise, 2), x2, rtol=0, atol=1e-15)


# ------------------------------------------------------------------ attention core
def brute_force_attention(q, kp, vp, ks, vs, mask, group):
    """Explicit loops over queries, heads and keys; no matmul, no vectorised softmax."""
    S, Hq, dh = q.shape
    P = kp.shape[0]
    out = np.zeros((S, Hq, dh))
    for i in range(S):
        for a in range(Hq):
            b = a // group
            keys, vals = [], []
            for j in range(P):
                keys.append(kp[j, b])
                vals.append(vp[j, b])
            for j in range(S):
                if mask[i][j]:
                    keys.append(ks[j, b])
                    vals.append(vs[j, b])
            logits = [sum(q[i, a, d] * k[d] for d in range(dh)) / math.sqrt(dh) for k in keys]
            mx = max(logits)
            w = [math.exp(z - mx) for z in logits]
            tot = sum(w)
            for d in range(dh):
                out[i, a, d] = sum(w[j] * vals[j][d] for j in range(len(w))) / tot
    return out


@pytest.mark.parametrize("S,Hq,Hkv,dh,P,block", [(3, 2, 1, 4, 5, False), (4, 4, 2, 2, 0, False),
                                                   (4, 2, 1, 4, 3, True), (1, 1, 1, 8, 7, False)])
def test_attention_matches_brute_force(S, Hq, Hkv, dh, P, block):
    rng = np.random.default_rng(S * 100 + P)
    q, ks, vs = rng.standard_normal((S, Hq, dh)), rng.standard_normal((S, Hkv, dh)), rng.standard_normal((S, Hkv, dh))
    kp, vp = rng.standard_normal((P, Hkv, dh)), rng.standard_normal((P, Hkv, dh))
    mask = np.ones((S, S), dtype=bool)
    if block:
        mask[0, 1:] = False
    got = O.attention(q, kp, vp, ks, vs, mask, Hq // Hkv)
    np.testing.assert_allclose(got, brute_force_attention(q, kp, vp, ks, vs, mask, Hq // Hkv), rtol=0, atol=1e-13)


def test_attention_matches_torch_sdpa_with_boolean_mask():
    rng = np.random.default_rng(11)
    S, Hq, Hkv, dh, P = 5, 4, 2, 8, 9
    q, ks, vs = rng.standard_normal((S, Hq, dh)), rng.standard_normal((S, Hkv, dh)), rng.standard_normal((S, Hkv, dh))
    kp, vp = rng.standard_normal((P, Hkv, dh)), rng.standard_normal((P, Hkv, dh))
    mask = rng.random((S, S)) > 0.3
    mask[np.arange(S), np.arange(S)] = True
    got = O.attention(q, kp, vp, ks, vs, mask, Hq // Hkv)
    k_all = torch.from_numpy(np.concatenate([kp, ks])).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
    v_all = torch.from_numpy(np.concatenate([vp, vs])).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
    full_mask = torch.from_numpy(np.concatenate([np.ones((S, P), dtype=bool), mask], axis=1))
    ref = F.scaled_dot_product_attention(torch.from_numpy(q).permute(1, 0, 2), k_all, v_all, attn_mask=full_mask)
    np.testing.assert_allclose(got, ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-13)


def test_zero_queries_give_plain_mean_of_visible_values():
    """q = 0 makes every logit equal, so the output is the mean over exactly P + S rows: catches an
    off-by-one in prefix_len."""
    rng = np.random.default_rng(5)
    S, Hkv, dh, P = 3, 1, 4, 6
    kp, vp = rng.standard_normal((P + 2, Hkv, dh)), rng.standard_normal((P + 2, Hkv, dh))
    ks, vs = rng.standard_normal((S, Hkv, dh)), rng.standard_normal((S, Hkv, dh))
    got = O.attention(np.zeros((S, 2, dh)), kp[:P], vp[:P], ks, vs, np.ones((S, S), bool), 2)
    mean = np.concatenate([vp[:P, 0], vs[:, 0]]).mean(axis=0)
    np.testing.assert_allclose(got, np.broadcast_to(mean, got.shape), rtol=0, atol=1e-14)


def test_whole_network_with_zero_wq_uses_exactly_prefix_len_rows():
    cfg = small_cfg(L=1)
    W, kv, state, noise = rand_inputs(cfg, 8, 6)
    W["wq.0"] = np.zeros_like(W["wq.0"])
    a = O.denoise(cfg, W, kv, 5, state, noise, 1)
    kv2 = kv.copy()
    kv2[:, 1, 4] += 1.0   # row 4 is inside prefix_len = 5: must matter
    b = O.denoise(cfg, W, kv2, 5, state, noise, 1)
    kv3 = kv.copy()
    kv3[:, :, 5] += 1.0   # row 5 is outside: must not
    c = O.denoise(cfg, W, kv3, 5, state, noise, 1)
    assert np.max(np.abs(a - b)) > 1e-6 and np.array_equal(a, c)


# ------------------------------------------------------------------ prefix handling
@fast
@given(cfg=cfg_strategy)
def test_rows_beyond_prefix_len_never_matter(cfg):
    P = 5
    W, kv, state, noise = rand_inputs(cfg, P + 3, 7)
    ref = O.denoise(cfg, W, kv[:, :, :P], P, state, noise, 2)
    poisoned = kv.copy()
    poisoned[:, :, P:] = np.nan
    assert np.array_equal(O.denoise(cfg, W, poisoned, P, state, noise, 2), ref)
    poisoned[:, :, P:] = 1e30
    assert np.array_equal(O.denoise(cfg, W, poisoned, P, state, noise, 2), ref)


@fast
@given(cfg=cfg_strategy)
def test_permuting_prefix_tokens_with_their_kv_changes_nothing(cfg):
    P = 7
    W, kv, state, noise = rand_inputs(cfg, P, 8)
    perm = np.random.default_rng(1).permutation(P)
    a = O.denoise(cfg, W, kv, P, state, noise, 2)
    b = O.denoise(cfg, W, kv[:, :, perm], P, state, noise, 2)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)


def test_empty_prefix_is_suffix_only_attention():
    cfg = small_cfg(L=1, rope=0.0)
    W, kv, state, noise = rand_inputs(cfg, 4, 9)
    a = O.denoise(cfg, W, kv[:, :, :0], 0, state, noise, 1)
    # huge negative-logit prefix rows are equivalent to no prefix: k = 0 rows get weight
    # exp(0 - max) which is not negligible, so instead compare with brute force directly
    assert a.shape == noise.shape and np.all(np.isfinite(a))
    q = np.random.default_rng(0).standard_normal((3, 2, 4))
    ks, vs = np.random.default_rng(1).standard_normal((2, 3, 1, 4))
    e = np.zeros((0, 1, 4))
    got = O.attention(q, e, e, ks, vs, np.ones((3, 3), bool), 2)
    np.testing.assert_allclose(got, brute_force_attention(q, e, e, ks, vs, np.ones((3, 3), bool), 2), atol=1e-14)


@fast
@given(cfg=cfg_strategy)
def test_batched_equals_single_and_ignores_neighbours(cfg):
    lens = [3, 0, 6]
    Ws, kvs, states, noises = None, [], [], []
    for b, P in enumerate(lens):
        W, kv, state, noise = rand_inputs(cfg, P, 20 + b)
        Ws = Ws or W
        kvs.append(kv), states.append(state), noises.append(noise)
    packed = np.concatenate(kvs, axis=2)
    cu = np.concatenate([[0], np.cumsum(lens)])
    st_ = states if cfg.has_state_token else None
    out = O.denoise_batched(cfg, Ws, packed, cu, st_, noises, 2)
    for b, P in enumerate(lens):
        assert np.array_equal(out[b], O.denoise(cfg, Ws, kvs[b], P, states[b], noises[b], 2))
    # change a neighbour's length: request 2 must not move
    kvs[0] = np.random.default_rng(3).standard_normal((cfg.n_layers, 2, 5, cfg.n_kv_heads, cfg.head_dim))
    packed2 = np.concatenate(kvs, axis=2)
    cu2 = np.concatenate([[0], np.cumsum([5, 0, 6])])
    out2 = O.denoise_batched(cfg, Ws, packed2, cu2, st_, noises, 2)
    assert np.array_equal(out2[2], out[2])


# ------------------------------------------------------------------ norms
def test_rmsnorm_matches_torch_rms_norm_with_one_plus_gamma():
    rng = np.random.default_rng(12)
    h, g = rng.standard_normal((5, 16)), rng.standard_normal(16) * 0.1
    ref = F.rms_norm(torch.from_numpy(h), (16,), weight=torch.from_numpy(1.0 + g), eps=1e-6).numpy()
    np.testing.assert_allclose(O.norm_plain(h, g, 1e-6), ref, rtol=0, atol=1e-14)


def test_rmsnorm_is_scale_invariant_without_eps_and_unit_rms():
    rng = np.random.default_rng(13)
    h = rng.standard_normal((4, 32))
    a, b = O.norm_plain(h, np.zeros(32), 0.0), O.norm_plain(7.5 * h, np.zeros(32), 0.0)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-14)
    np.testing.assert_allclose(np.mean(a * a, axis=1), 1.0, atol=1e-14)
    # eps sits inside the square root: for h = 0 rows the result is 0, for tiny rows r = eps^-1/2
    tiny = np.full((1, 32), 1e-12)
    np.testing.assert_allclose(O.norm_plain(tiny, np.zeros(32), 1e-6), tiny / math.sqrt(1e-24 + 1e-6), rtol=1e-12)


def test_adarms_order_is_scale_shift_gate():
    rng = np.random.default_rng(14)
    D = 8
    h, c = rng.standard_normal((3, D)), rng.standard_normal(D)
    w, b = rng.standard_normal((D, 3 * D)) * 0.1, rng.standard_normal(3 * D) * 0.1
    n, g = O.norm_ada(h, c, w, b, 1e-6)
    m = (torch.from_numpy(c) @ torch.from_numpy(w) + torch.from_numpy(b)).numpy()
    base = F.rms_norm(torch.from_numpy(h), (D,), eps=1e-6).numpy()
    np.testing.assert_allclose(n, base * (1.0 + m[:D]) + m[D:2 * D], rtol=0, atol=1e-14)
    np.testing.assert_allclose(g, m[2 * D:], rtol=0, atol=1e-15)


def test_adarms_with_zero_gates_makes_every_layer_the_identity():
    """W_mod = 0, b_mod = 0: scale = shift = gate = 0, so the residual stream stays the embedding
    and v = (h_embed r) W_out + b_out, recomputed here by hand."""
    cfg = small_cfg(cond="pi05", L=3)
    W, kv, state, noise = rand_inputs(cfg, 6, 15)
    for n_, s_ in synth.weight_shapes(cfg):
        if n_.startswith(("norm1", "norm2", "final_norm")):
            W[n_] = np.zeros(s_)
    h = noise @ W["action_in_w"] + W["action_in_b"]
    r = 1.0 / np.sqrt((h ** 2).mean(axis=1, keepdims=True) + cfg.rms_eps)
    v = (h * r) @ W["action_out_w"] + W["action_out_b"]
    np.testing.assert_allclose(O.denoise(cfg, W, kv, 6, None, noise, 1), noise - v, rtol=0, atol=1e-13)


# ------------------------------------------------------------------ activations, sinusoid, RoPE
def test_gelu_and_swish_match_library_and_spot_values():
    z = np.linspace(-6, 6, 101)
    zt = torch.from_numpy(z)
    np.testing.assert_allclose(O.gelu(z), F.gelu(zt, approximate="tanh").numpy(), rtol=0, atol=1e-15)
    np.testing.assert_allclose(O.gelu(z, exact=True), F.gelu(zt).numpy(), rtol=0, atol=1e-15)
    np.testing.assert_allclose(O.swish(z), F.silu(zt).numpy(), rtol=0, atol=1e-15)
    assert abs(O.gelu(np.array(1.0)) - 0.8411919906) < 1e-9
    assert abs(O.gelu(np.array(1.0), exact=True) - 0.8413447461) < 1e-9
    assert abs(O.swish(np.array(1.0)) - 0.7310585786) < 1e-9


def test_sinusoid_special_values():
    D = 64
    t0 = O.sinusoid(0.0, D, 4e-3, 4.0)
    assert np.all(t0[:D // 2] == 0.0) and np.all(t0[D // 2:] == 1.0)
    t1 = O.sinusoid(1.0, D, 4e-3, 4.0)
    # channel 0: period 4e-3 -> 250 full turns; last channel: period 4 -> a quarter turn
    assert abs(t1[0]) < 1e-9 and abs(t1[D // 2] - 1.0) < 1e-9
    assert abs(t1[D // 2 - 1] - 1.0) < 1e-12 and abs(t1[D - 1]) < 1e-12
    assert abs(O.sinusoid(0.9, D, 4e-3, 4.0)[D // 2 - 1] - 0.9876883406) < 1e-9
    # geometric spacing: middle channel of an odd-count grid has period sqrt(min*max)
    t = O.sinusoid(0.01, 6, 1e-2, 1.0)          # 3 channels: periods 0.01, 0.1, 1
    np.testing.assert_allclose(t[:3], np.sin(2 * math.pi * 0.01 / np.array([0.01, 0.1, 1.0])), atol=1e-12)


def test_rope_is_a_rotation_depending_only_on_relative_position():
    rng = np.random.default_rng(16)
    dh = 8
    q, k = rng.standard_normal((1, 1, dh)), rng.standard_normal((1, 1, dh))
    def dot(pq, pk):
        return float(np.sum(O.rope(q, np.array([pq]), 10000.0) * O.rope(k, np.array([pk]), 10000.0)))
    assert abs(dot(3, 7) - dot(103, 107)) < 1e-10
    assert abs(dot(3, 7) - dot(4, 7)) > 1e-6
    np.testing.assert_allclose(np.linalg.norm(O.rope(q, np.array([77]), 10000.0)), np.linalg.norm(q), rtol=1e-14)
    # explicit 2x2 rotations on the pairs (j, j + dh/2)
    pos, x = 5, q[0, 0]
    y = np.zeros(dh)
    for j in range(dh // 2):
        phi = pos * 10000.0 ** (-2.0 * j / dh)
        R = np.array([[math.cos(phi), -math.sin(phi)], [math.sin(phi), math.cos(phi)]])
        y[j], y[j + dh // 2] = R @ np.array([x[j], x[j + dh // 2]])
    np.testing.assert_allclose(O.rope(q, np.array([pos]), 10000.0)[0, 0], y, rtol=0, atol=1e-14)
    assert O.rope(q, np.array([9]), 0.0) is q
    np.testing.assert_array_equal(O.rope(q, np.array([0]), 10000.0), q)


def test_suffix_positions_follow_the_prefix():
    """Suffix token i sits at position prefix_len + i: with a single zero-length prefix versus a
    shifted position the logits between suffix tokens are unchanged (relative), but moving the
    prefix rows' count shifts positions consistently - checked through the permutation and
    tail tests; here: theta = 0 and theta > 0 differ, so RoPE is actually applied."""
    cfg = small_cfg(L=1)
    W, kv, state, noise = rand_inputs(cfg, 6, 17)
    a = O.denoise(cfg, W, kv, 6, state, noise, 1)
    b = O.denoise(cfg.with_(rope_theta=0.0), W, kv, 6, state, noise, 1)
    assert np.max(np.abs(a - b)) > 1e-8


# ------------------------------------------------------------------ embedding and head
def test_blocks_switched_off_leave_embedding_then_head_pi0():
    """W_o = 0 and W_down = 0 in every layer: residual stream = embedding; v by hand."""
    cfg = small_cfg(L=2)
    W, kv, state, noise = rand_inputs(cfg, 6, 18)
    for l in range(cfg.n_layers):
        W[f"wo.{l}"] = np.zeros_like(W[f"wo.{l}"])
        W[f"wdown.{l}"] = np.zeros_like(W[f"wdown.{l}"])
    t, D = 1.0, cfg.width
    half = D // 2
    period = cfg.time_min_period * (cfg.time_max_period / cfg.time_min_period) ** (np.arange(half) / (half - 1))
    tau = np.concatenate([np.sin(2 * math.pi * t / period), np.cos(2 * math.pi * t / period)])
    rows = []
    for i in range(cfg.horizon):
        e = noise[i] @ W["action_in_w"] + W["action_in_b"]
        z = e @ W["time_mlp1_w"][:D] + tau @ W["time_mlp1_w"][D:] + W["time_mlp1_b"]
        rows.append((z / (1 + np.exp(-z))) @ W["time_mlp2_w"] + W["time_mlp2_b"])
    h = np.stack(rows)                         # state token row is discarded by the head
    r = 1.0 / np.sqrt((h ** 2).mean(axis=1, keepdims=True) + cfg.rms_eps)
    v = (h * r * (1.0 + W["final_norm"])) @ W["action_out_w"] + W["action_out_b"]
    np.testing.assert_allclose(O.denoise(cfg, W, kv, 6, state, noise, 1), noise - v, rtol=0, atol=1e-13)


def test_state_token_reaches_the_actions_only_through_attention():
    cfg = small_cfg(L=1)
    W, kv, state, noise = rand_inputs(cfg, 6, 19)
    a = O.denoise(cfg, W, kv, 6, state, noise, 1)
    b = O.denoise(cfg, W, kv, 6, state + 1.0, noise, 1)
    assert np.max(np.abs(a - b)) > 1e-9
    W["wv.0"] = np.zeros_like(W["wv.0"])      # values from the suffix vanish -> but prefix V remains
    W["wk.0"] = np.zeros_like(W["wk.0"])      # and suffix keys no longer depend on the tokens
    a = O.denoise(cfg, W, kv, 6, state, noise, 1)
    b = O.denoise(cfg, W, kv, 6, state + 1.0, noise, 1)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-14)


# ------------------------------------------------------------------ independent transcription
def torch_transcription(cfg, W, kv, P, state, noise, n_steps):
    """A second derivation from the step list with a different structure: torch float64, all heads
    batched through scaled_dot_product_attention, library rms_norm / silu / gelu, time-embedding
    contribution split from the action contribution, RoPE via complex multiplication."""
    T = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in W.items()}
    kv = torch.from_numpy(np.asarray(kv, dtype=np.float64))
    x = torch.from_numpy(np.asarray(noise, dtype=np.float64)).clone()
    D, Hq, Hkv, dh = cfg.width, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    ns = 1 if cfg.has_state_token else 0
    S = cfg.horizon + ns
    ada = cfg.cond == "pi05"
    act = (lambda z: F.gelu(z)) if cfg.gelu_exact else (lambda z: F.gelu(z, approximate="tanh"))
    half = D // 2
    expo = torch.arange(half, dtype=torch.float64) / max(half - 1, 1)
    freq = 2 * math.pi / (cfg.time_min_period * (cfg.time_max_period / cfg.time_min_period) ** expo)

    def rot(z, pos):
        if cfg.rope_theta == 0:
            return z
        inv = cfg.rope_theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
        ang = torch.polar(torch.ones(S, dh // 2, dtype=torch.float64), pos[:, None] * inv[None, :])
        zc = torch.complex(z[..., : dh // 2], z[..., dh // 2:]) * ang[:, None, :]
        return torch.cat([zc.real, zc.imag], dim=-1)

    def norm(h, c, w, b):
        base = F.rms_norm(h, (D,), eps=cfg.rms_eps)
        if not ada:
            return base * (1 + w), 1.0
        sc, sh, g = (c @ w + b).split(D)
        return base * (1 + sc) + sh, g

    for k in range(n_steps):
        t = 1.0 - k / n_steps
        tau = torch.cat([torch.sin(freq * t), torch.cos(freq * t)])
        e = x @ T["action_in_w"] + T["action_in_b"]
        if ada:
            h = e
            c = F.silu(F.silu(tau @ T["time_mlp1_w"] + T["time_mlp1_b"]) @ T["time_mlp2_w"] + T["time_mlp2_b"])
        else:
            tb = tau @ T["time_mlp1_w"][D:] + T["time_mlp1_b"]
            h = F.silu(e @ T["time_mlp1_w"][:D] + tb) @ T["time_mlp2_w"] + T["time_mlp2_b"]
            c = None
        if ns:
            h = torch.cat([(torch.from_numpy(state) @ T["state_w"] + T["state_b"])[None], h])
        pos = torch.arange(P, P + S, dtype=torch.float64)
        for l in range(cfg.n_layers):
            n1, g1 = norm(h, c, T[f"norm1.{l}"], T.get(f"norm1_b.{l}"))
            wqkv = torch.cat([T[f"wq.{l}"], T[f"wk.{l}"], T[f"wv.{l}"]], dim=1)
            q, ks, vs = (n1 @ wqkv).split([Hq * dh, Hkv * dh, Hkv * dh], dim=1)
            q, ks = rot(q.view(S, Hq, dh), pos), rot(ks.view(S, Hkv, dh), pos)
            K = torch.cat([kv[l, 0, :P], ks]).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
            V = torch.cat([kv[l, 1, :P], vs.view(S, Hkv, dh)]).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
            o = F.scaled_dot_product_attention(q.transpose(0, 1), K, V).transpose(0, 1).reshape(S, Hq * dh)
            h = h + g1 * (o @ T[f"wo.{l}"])
            n2, g2 = norm(h, c, T[f"norm2.{l}"], T.get(f"norm2_b.{l}"))
            gu = n2 @ torch.cat([T[f"wgate.{l}"], T[f"wup.{l}"]], dim=1)
            h = h + g2 * ((act(gu[:, : cfg.mlp_dim]) * gu[:, cfg.mlp_dim:]) @ T[f"wdown.{l}"])
        nf, _ = norm(h, c, T["final_norm"], T.get("final_norm_b"))
        x = x - (nf[ns:] @ T["action_out_w"] + T["action_out_b"]) / n_steps
    return x.numpy()


@fast
@given(cfg=cfg_strategy, n=st.integers(1, 3))
def test_oracle_agrees_with_independent_torch_transcription(cfg, n):
    P = cfg.max_prefix_len if cfg.max_prefix_len > 1 else 0
    W, kv, state, noise = rand_inputs(cfg, P, 30)
    a = O.denoise(cfg, W, kv, P, state, noise, n)
    b = torch_transcription(cfg, W, kv, P, state, noise, n)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-11)


def test_tiny_config_agrees_with_transcription_and_golden_file():
    """C1 (the tiny fp32 configuration) through both derivations, and against the stored output
    written by tests/golden/make_golden.py (which calls only the oracle)."""
    import os
    cfg = synth.tiny_config()
    W = synth.make_weights(cfg, 1)
    kv, state, noise = synth.make_prefix_kv(cfg, 1, 64), synth.make_state(cfg, 1), synth.make_noise(cfg, 1)
    a = O.denoise(cfg, W, kv, 64, state, noise, 4)
    Wn = {k: v.double().numpy() for k, v in W.items()}
    b = torch_transcription(cfg, Wn, kv.double().numpy(), 64, state.double().numpy(), noise.double().numpy(), 4)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-11)
    gold = np.loadtxt(os.path.join(os.path.dirname(__file__), "golden", "c1_actions.txt"))
    np.testing.assert_allclose(a, gold, rtol=0, atol=1e-12)


# ------------------------------------------------------------------ e4m3 storage
def test_e4m3_decode_exhaustive_against_ml_dtypes():
    import ml_dtypes
    codes = np.arange(256, dtype=np.uint8)
    ref = codes.view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    got = O.decode_e4m3(codes)
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok], ref[ok])
    assert got[0x7E] == 448.0 and got[0xFE] == -448.0 and got[0x01] == 2.0 ** -9


def test_column_quantizer_is_round_to_nearest_even_and_saturating():
    import ml_dtypes
    rng = np.random.default_rng(21)
    w = torch.from_numpy(rng.standard_normal((64, 8)).astype(np.float32) * 0.02)
    w[:, 3] = 0.0
    codes, scales = synth.quantize_e4m3_columns(w)
    assert scales[3] == 1.0 and torch.all(codes[:, 3] == 0)
    ref = (w.numpy() / scales.numpy()[None, :]).astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    assert np.array_equal(codes.numpy(), ref)
    dec = O.to_f64((codes, scales))
    assert not np.isnan(dec).any()
    assert np.max(np.abs(dec).max(axis=0)[[0, 1, 2, 4]] / (448.0 * scales.numpy()[[0, 1, 2, 4]])) == pytest.approx(1.0, abs=1e-6)
    assert np.max(np.abs(dec - w.numpy().astype(np.float64))) <= 0.0625 * np.abs(w.numpy()).max()
    # ties to even at a midpoint: 1.0625 lies halfway between 1.0 and 1.125
    mid = torch.tensor([[448.0, 448.0], [1.0625, 1.1875]])
    c, s = synth.quantize_e4m3_columns(mid)
    assert O.decode_e4m3(c.numpy())[1].tolist() == [1.0, 1.25]
