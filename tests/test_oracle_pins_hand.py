"""Hand-built pins for the parts of the oracle that only a second transcription covered before:
the block-causal suffix mask, the suffix positions prefix_len + i, the grouped-query head map
through the whole network, and the pi0.5 conditioning vector.  Everything the oracle is compared
with here is written out with scalar loops, explicit 2x2 rotations and an explicit head table."""
import math

import numpy as np

from oracle import expert_oracle as O
from paper_2608_03682_b200 import synth

KV_HEAD_OF = {0: 0, 1: 0, 2: 1, 3: 1}   # 4 query heads on 2 kv heads: contiguous groups (reading R12)


def cfg_of(**kw):
    base = dict(n_layers=2, width=8, mlp_dim=16, n_q_heads=4, n_kv_heads=2, head_dim=4, state_dim=3, action_dim=2,
                horizon=3, has_state_token=True, max_prefix_len=8, cond="pi0", dtype="f32")
    base.update(kw)
    return synth.ExpertConfig(**base)


def draw(cfg, P, seed):
    rng = np.random.default_rng(seed)
    W = {n: rng.standard_normal(s) * 0.4 for n, s in synth.weight_shapes(cfg)}
    kv = rng.standard_normal((cfg.n_layers, 2, P, cfg.n_kv_heads, cfg.head_dim))
    state = rng.standard_normal(cfg.state_dim)
    noise = rng.standard_normal((cfg.horizon, cfg.action_dim))
    return W, kv, state, noise


def rotate_by_hand(x, pos, theta):
    """x[dh] -> pairs (j, j + dh/2) turned by the angle pos * theta^(-2j/dh), as 2x2 matrices."""
    dh = len(x)
    y = np.zeros(dh)
    for j in range(dh // 2):
        phi = pos * theta ** (-2.0 * j / dh)
        R = np.array([[math.cos(phi), -math.sin(phi)], [math.sin(phi), math.cos(phi)]])
        y[j], y[j + dh // 2] = R @ np.array([x[j], x[j + dh // 2]])
    return y


def rms_gain_by_hand(row, gamma, eps):
    ms = sum(v * v for v in row) / len(row)
    return np.array([v / math.sqrt(ms + eps) * (1.0 + g) for v, g in zip(row, gamma)])


def gelu_tanh_scalar(z):
    return 0.5 * z * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))


def softmax_mix_by_hand(q, keys, vals, dh):
    logits = [sum(q[d] * k[d] for d in range(dh)) / math.sqrt(dh) for k in keys]
    mx = max(logits)
    w = [math.exp(z - mx) for z in logits]
    tot = sum(w)
    return np.array([sum(w[j] * vals[j][d] for j in range(len(w))) / tot for d in range(dh)])


def tokens_through_layers_by_hand(cfg, W, kv, P, h_rows, first_pos, visible):
    """Rows h_rows[i] (at positions first_pos + i) through all layers; row i attends the P prefix rows
    and the suffix rows listed in visible[i].  Returns the final rows and, per layer, the rotated keys
    and the values of every row: [(k[i][kv head], v[i][kv head]), ...]."""
    Hq, Hkv, dh, D = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.width
    h = [np.array(r, dtype=float) for r in h_rows]
    per_layer = []
    for l in range(cfg.n_layers):
        n1 = [rms_gain_by_hand(r, W[f"norm1.{l}"], cfg.rms_eps) for r in h]
        q = [[rotate_by_hand((n @ W[f"wq.{l}"])[a * dh:(a + 1) * dh], first_pos + i, cfg.rope_theta) for a in range(Hq)]
             for i, n in enumerate(n1)]
        k = [[rotate_by_hand((n @ W[f"wk.{l}"])[b * dh:(b + 1) * dh], first_pos + i, cfg.rope_theta) for b in range(Hkv)]
             for i, n in enumerate(n1)]
        v = [[(n @ W[f"wv.{l}"])[b * dh:(b + 1) * dh] for b in range(Hkv)] for n in n1]
        per_layer.append((k, v))
        new_h = []
        for i in range(len(h)):
            o = np.zeros(Hq * dh)
            for a in range(Hq):
                b = KV_HEAD_OF[a] if Hkv == 2 else 0
                keys = [kv[l, 0, j, b] for j in range(P)] + [k[j][b] for j in visible[i]]
                vals = [kv[l, 1, j, b] for j in range(P)] + [v[j][b] for j in visible[i]]
                o[a * dh:(a + 1) * dh] = softmax_mix_by_hand(q[i][a], keys, vals, dh)
            hi = h[i] + o @ W[f"wo.{l}"]
            n2 = rms_gain_by_hand(hi, W[f"norm2.{l}"], cfg.rms_eps)
            g, u = n2 @ W[f"wgate.{l}"], n2 @ W[f"wup.{l}"]
            m = np.array([gelu_tanh_scalar(gz) * uz for gz, uz in zip(g, u)])
            new_h.append(hi + m @ W[f"wdown.{l}"])
        h = new_h
    return h, per_layer


def pi0_action_rows_by_hand(cfg, W, x, t):
    D, half = cfg.width, cfg.width // 2
    tau = np.zeros(D)
    for j in range(half):
        period = cfg.time_min_period * (cfg.time_max_period / cfg.time_min_period) ** (j / (half - 1))
        tau[j], tau[half + j] = math.sin(2 * math.pi * t / period), math.cos(2 * math.pi * t / period)
    rows = []
    for i in range(cfg.horizon):
        e = x[i] @ W["action_in_w"] + W["action_in_b"]
        z = np.concatenate([e, tau]) @ W["time_mlp1_w"] + W["time_mlp1_b"]
        rows.append(np.array([zz / (1.0 + math.exp(-zz)) for zz in z]) @ W["time_mlp2_w"] + W["time_mlp2_b"])
    return rows


def head_by_hand(cfg, W, rows):
    out = []
    for r in rows:
        out.append(rms_gain_by_hand(r, W["final_norm"], cfg.rms_eps) @ W["action_out_w"] + W["action_out_b"])
    return np.stack(out)


# ------------------------------------------------------------------ block-causal suffix mask
def test_block_causal_visibility_written_out():
    cfg = cfg_of(suffix_block_causal=True)
    expect = np.array([[1, 0, 0, 0],      # the state token sees, of the suffix, only itself
                       [1, 1, 1, 1],      # action tokens see the state token and every action token
                       [1, 1, 1, 1],
                       [1, 1, 1, 1]], dtype=bool)
    assert np.array_equal(O.suffix_visibility(cfg), expect)
    assert O.suffix_visibility(cfg.with_(suffix_block_causal=False)).all()
    # without a state token the flag has nothing to act on
    assert O.suffix_visibility(cfg.with_(has_state_token=False)).all()


def test_block_causal_forward_by_hand_one_step():
    """The whole velocity with the mask, against scalar loops in which row 0's key list is written out as
    prefix + its own key and the other rows' as prefix + all four suffix keys."""
    cfg = cfg_of(suffix_block_causal=True)
    P = 5
    W, kv, state, noise = draw(cfg, P, 41)
    rows = [state @ W["state_w"] + W["state_b"]] + pi0_action_rows_by_hand(cfg, W, noise, 1.0)
    visible = [[0], [0, 1, 2, 3], [0, 1, 2, 3], [0, 1, 2, 3]]
    h, _ = tokens_through_layers_by_hand(cfg, W, kv, P, rows, P, visible)
    v = head_by_hand(cfg, W, h[1:])
    np.testing.assert_allclose(O.velocity(cfg, O.Weights(W), kv, P, state, noise, 1.0), v, rtol=0, atol=1e-12)
    # and the unmasked network differs: the mask is not a no-op
    v_full = O.velocity(cfg.with_(suffix_block_causal=False), O.Weights(W), kv, P, state, noise, 1.0)
    assert np.max(np.abs(v_full - v)) > 1e-6


def test_block_causal_state_token_is_step_invariant_and_acts_like_a_cached_prefix_row():
    """Under the block-causal mask the state token sees the prefix and itself only, so its hidden states,
    rotated key and value of every layer depend neither on x nor on t.  They are computed here once, by
    hand, from the state alone; appended to the prefix as row P they must reproduce the masked network's
    output with a state-token-free expert (action token i then sits at (P + 1) + i = P + (1 + i): the
    suffix positions continue the prefix without a gap)."""
    cfg = cfg_of(suffix_block_causal=True)
    P, n = 5, 3
    W, kv, state, noise = draw(cfg, P, 42)
    _, per_layer = tokens_through_layers_by_hand(cfg, W, kv, P, [state @ W["state_w"] + W["state_b"]], P, [[0]])
    kv_ext = np.zeros((cfg.n_layers, 2, P + 1, cfg.n_kv_heads, cfg.head_dim))
    kv_ext[:, :, :P] = kv
    for l, (k, v) in enumerate(per_layer):
        for b in range(cfg.n_kv_heads):
            kv_ext[l, 0, P, b], kv_ext[l, 1, P, b] = k[0][b], v[0][b]
    cfg_ns = cfg.with_(has_state_token=False, suffix_block_causal=False, max_prefix_len=P + 1)
    W_ns = {k_: v_ for k_, v_ in W.items() if not k_.startswith("state_")}
    a = O.denoise(cfg, W, kv, P, state, noise, n)
    b = O.denoise(cfg_ns, W_ns, kv_ext, P + 1, None, noise, n)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)
    # the bidirectional network is NOT reproduced by that cached row (its state token reads the actions)
    c = O.denoise(cfg.with_(suffix_block_causal=False), W, kv, P, state, noise, n)
    assert np.max(np.abs(c - b)) > 1e-6


# ------------------------------------------------------------------ suffix positions and the head map
def test_forward_by_hand_pins_suffix_positions_and_the_grouped_query_map():
    """Two layers, four query heads on two kv heads, rotary on, default (bidirectional) mask: the logit of
    suffix row i against prefix row j is <R(P + i) q, K_j> with K_j used as stored, and against suffix row
    j' it is <R(P + i) q, R(P + j') k>, all rotations explicit 2x2 matrices."""
    cfg = cfg_of()
    P = 6
    W, kv, state, noise = draw(cfg, P, 43)
    rows = [state @ W["state_w"] + W["state_b"]] + pi0_action_rows_by_hand(cfg, W, noise, 0.7)
    everything = [[0, 1, 2, 3]] * 4
    h, _ = tokens_through_layers_by_hand(cfg, W, kv, P, rows, P, everything)
    v = head_by_hand(cfg, W, h[1:])
    np.testing.assert_allclose(O.velocity(cfg, O.Weights(W), kv, P, state, noise, 0.7), v, rtol=0, atol=1e-12)
    # a different first position, or the interleaved head map, gives a different answer (the pin can fail)
    h_bad, _ = tokens_through_layers_by_hand(cfg, W, kv, P, rows, P + 1, everything)
    assert np.max(np.abs(head_by_hand(cfg, W, h_bad[1:]) - v)) > 1e-6
    saved = dict(KV_HEAD_OF)
    try:
        KV_HEAD_OF.update({0: 0, 1: 1, 2: 0, 3: 1})
        h_il, _ = tokens_through_layers_by_hand(cfg, W, kv, P, rows, P, everything)
    finally:
        KV_HEAD_OF.update(saved)
    assert np.max(np.abs(head_by_hand(cfg, W, h_il[1:]) - v)) > 1e-6


def test_one_prefix_key_one_query_logit_by_hand():
    """One layer, one head, one suffix token, one prefix row whose key was rotated by hand at position p0:
    with W_v = 0 the suffix value vanishes, so o = w_prefix * V_0 where w_prefix is the softmax weight of
    the logit <R(P) q, R(p0) k_raw> against <R(P) q, R(P) k_s>.  P = 1 here, p0 is free."""
    cfg = cfg_of(n_layers=1, n_q_heads=1, n_kv_heads=1, horizon=1, has_state_token=False)
    rng = np.random.default_rng(44)
    W = {n: rng.standard_normal(s) * 0.4 for n, s in synth.weight_shapes(cfg)}
    W["wv.0"] = np.zeros_like(W["wv.0"])
    x = rng.standard_normal((1, cfg.action_dim))
    k_raw, v0, p0 = rng.standard_normal(cfg.head_dim), rng.standard_normal(cfg.head_dim), 0
    kv = np.zeros((1, 2, 1, 1, cfg.head_dim))
    kv[0, 0, 0, 0], kv[0, 1, 0, 0] = rotate_by_hand(k_raw, p0, cfg.rope_theta), v0
    row = pi0_action_rows_by_hand(cfg, W, x, 1.0)[0]
    n1 = rms_gain_by_hand(row, W["norm1.0"], cfg.rms_eps)
    q = rotate_by_hand(n1 @ W["wq.0"], 1, cfg.rope_theta)          # suffix position = prefix_len + 0 = 1
    ks = rotate_by_hand(n1 @ W["wk.0"], 1, cfg.rope_theta)
    lp = float(q @ rotate_by_hand(k_raw, p0, cfg.rope_theta)) / math.sqrt(cfg.head_dim)
    ls = float(q @ ks) / math.sqrt(cfg.head_dim)
    w_prefix = math.exp(lp) / (math.exp(lp) + math.exp(ls))
    h = row + (w_prefix * v0) @ W["wo.0"]
    n2 = rms_gain_by_hand(h, W["norm2.0"], cfg.rms_eps)
    m = np.array([gelu_tanh_scalar(g) * u for g, u in zip(n2 @ W["wgate.0"], n2 @ W["wup.0"])])
    h = h + m @ W["wdown.0"]
    v = head_by_hand(cfg, W, [h])
    np.testing.assert_allclose(O.velocity(cfg, O.Weights(W), kv, 1, None, x, 1.0), v, rtol=0, atol=1e-13)


# ------------------------------------------------------------------ pi0.5 conditioning vector
def test_pi05_conditioning_vector_by_hand_width_two():
    """width 2: tau = (sin, cos)(2 pi t / p_min); c = swish(swish(tau W1 + b1) W2 + b2) in scalars.  All layer
    modulations are zero (every layer is the identity), the final site has W_mod != 0, so
    v = (h r (1 + c W_scale + b_scale) + c W_shift + b_shift) W_out + b_out depends on c alone."""
    cfg = synth.ExpertConfig(n_layers=1, width=2, mlp_dim=4, n_q_heads=1, n_kv_heads=1, head_dim=2, state_dim=1,
                             action_dim=2, horizon=2, has_state_token=False, max_prefix_len=3, cond="pi05", dtype="f32")
    rng = np.random.default_rng(45)
    W = {n: rng.standard_normal(s) * 0.5 for n, s in synth.weight_shapes(cfg)}
    for name in ("norm1.0", "norm1_b.0", "norm2.0", "norm2_b.0"):
        W[name] = np.zeros_like(W[name])
    kv = rng.standard_normal((1, 2, 3, 1, 2))
    x = rng.standard_normal((2, 2))
    t = 0.3
    sw = lambda z: z / (1.0 + math.exp(-z))
    arg = 2.0 * math.pi * t / cfg.time_min_period          # a single channel: its period is the minimum
    tau = [math.sin(arg), math.cos(arg)]
    W1, b1, W2, b2 = W["time_mlp1_w"], W["time_mlp1_b"], W["time_mlp2_w"], W["time_mlp2_b"]
    a = [sw(tau[0] * W1[0][n] + tau[1] * W1[1][n] + b1[n]) for n in range(2)]
    c = [sw(a[0] * W2[0][n] + a[1] * W2[1][n] + b2[n]) for n in range(2)]
    Wm, bm = W["final_norm"], W["final_norm_b"]            # [2, 6], [6]: (scale | shift | gate)
    mod = [c[0] * Wm[0][n] + c[1] * Wm[1][n] + bm[n] for n in range(6)]
    v = np.zeros((2, 2))
    for i in range(2):
        h = [x[i][0] * W["action_in_w"][0][n] + x[i][1] * W["action_in_w"][1][n] + W["action_in_b"][n] for n in range(2)]
        r = 1.0 / math.sqrt((h[0] ** 2 + h[1] ** 2) / 2.0 + cfg.rms_eps)
        nf = [h[n] * r * (1.0 + mod[n]) + mod[2 + n] for n in range(2)]
        for aa in range(2):
            v[i][aa] = nf[0] * W["action_out_w"][0][aa] + nf[1] * W["action_out_w"][1][aa] + W["action_out_b"][aa]
    np.testing.assert_allclose(O.velocity(cfg, O.Weights(W), kv, 3, None, x, t), v, rtol=0, atol=1e-13)
