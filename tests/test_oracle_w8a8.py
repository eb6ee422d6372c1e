"""Pins of the oracle's W8A8 pieces (quantization paragraph: round-to-nearest e4m3): the rounding
function against an independent library cast and against values fixed by the format itself, the
per-token scale rule by hand, and the quantized projection on inputs where it must reduce to the
plain product."""
import numpy as np
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import synth


def all_finite_e4m3():
    codes = np.arange(256, dtype=np.uint8)
    vals = O.decode_e4m3(codes)
    return vals[np.isfinite(vals)]


def test_every_e4m3_value_is_a_fixed_point_of_the_rounding():
    v = all_finite_e4m3()
    assert np.array_equal(O.round_e4m3(v), v)


def test_rounding_agrees_with_the_library_cast_on_a_dense_sweep():
    # torch's float8_e4m3fn cast is round-to-nearest-even; it has no saturation (values beyond 464 become NaN), so
    # the sweep stays inside the finite range and saturation is pinned separately below
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.uniform(-448, 448, 20000), rng.uniform(-1, 1, 20000), rng.uniform(-0.02, 0.02, 20000),
                        np.linspace(-447.9, 447.9, 9973)]).astype(np.float32)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(O.round_e4m3(x.astype(np.float64)), lib)


def test_ties_go_to_the_even_mantissa_and_large_values_saturate():
    # neighbours 1.0 (m = 0) and 1.125 (m = 1): the midpoint goes to 1.0; 1.125 and 1.25 (m = 2): midpoint to 1.25
    assert O.round_e4m3(np.array([1.0625]))[0] == 1.0
    assert O.round_e4m3(np.array([1.1875]))[0] == 1.25
    # subnormal grid: step 2^-9; 1.5 steps -> 2 steps (even), 0.5 step -> 0
    assert O.round_e4m3(np.array([1.5 * 2.0 ** -9]))[0] == 2.0 ** -8
    assert O.round_e4m3(np.array([0.5 * 2.0 ** -9]))[0] == 0.0
    assert O.round_e4m3(np.array([-0.5 * 2.0 ** -9]))[0] == 0.0
    # binade boundary: 15.5 is halfway between 15 (m = 7) and 16 (next binade, m = 0) -> 16
    assert O.round_e4m3(np.array([15.5]))[0] == 16.0
    # the largest finite value is 448; everything beyond saturates
    assert np.array_equal(O.round_e4m3(np.array([448.0, 460.0, 1e9, -1e9])), np.array([448.0, 448.0, 448.0, -448.0]))


def test_bf16_rounding_agrees_with_the_library_cast():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.standard_normal(50000) * np.exp(rng.uniform(-20, 20, 50000)),
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8), 0.0, 2.0 ** -130])]).astype(np.float32)
    lib = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.round_bf16(x), lib)
    # ties to even by hand: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> 1; 1 + 3 * 2^-8 -> 1 + 2^-6
    assert O.round_bf16(np.float32(1.0 + 2.0 ** -8)) == np.float32(1.0)
    assert O.round_bf16(np.float32(1.0 + 3 * 2.0 ** -8)) == np.float32(1.0 + 2.0 ** -6)


def test_row_scale_rule_by_hand():
    x = np.array([[0.5, -3.5, 1.0, 0.0], [0.0, 0.0, 0.0, 0.0], [448.0, 1.0, -2.0, 3.0]])
    q, s = O.quantize_rows_e4m3(x)
    assert np.allclose(s[:, 0], [3.5 / 448.0, 1.0, 1.0], rtol=1e-7)
    # row 0: x / s = (64, -448, 128, 0): all on the grid
    assert np.array_equal(q[0], [64.0, -448.0, 128.0, 0.0])
    assert np.array_equal(q[1], [0.0, 0.0, 0.0, 0.0])
    assert np.array_equal(q[2], [448.0, 1.0, -2.0, 3.0])


def test_quantized_projection_is_the_plain_product_for_rows_on_the_grid():
    # rows whose elements are (e4m3 value) x (row maximum / 448) quantize without error
    rng = np.random.default_rng(3)
    grid = all_finite_e4m3()
    q = rng.choice(grid, size=(5, 64))
    q[:, 0] = 448.0                                   # the row maximum maps to 448
    scale = np.array([[1.0], [0.25], [2.0 ** -7], [8.0], [0.5]])
    x = q * scale
    w = rng.standard_normal((64, 9))

    class Cfg:
        dtype = "w8a8e4m3"

    assert np.allclose(O.project(Cfg, x, w), x @ w, rtol=1e-12, atol=0)

    class Plain:
        dtype = "bf16"

    y = rng.standard_normal((5, 64))
    assert np.array_equal(O.project(Plain, y, w), y @ w)


def test_quantization_error_of_a_projection_is_within_the_format_bound():
    # |x - s q| <= s * (half a grid step at q) <= |x| / 16 + s 2^-10 elementwise
    rng = np.random.default_rng(5)
    x = rng.standard_normal((7, 256)) * np.exp(rng.standard_normal((7, 1)))
    q, s = O.quantize_rows_e4m3(x)
    xb = O.round_bf16(x.astype(np.float32)).astype(np.float64)
    err = np.abs(xb - q * s)
    assert np.all(err <= np.abs(xb) / 16.0 + s * 2.0 ** -10 + 1e-12)


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
def test_w8a8_network_stays_close_to_the_w8a16_network(cond):
    # the activation quantization perturbs every projection by a few per cent of noise with random sign: the chunk
    # moves, but by far less than its size; and the two modes differ (the quantization is really applied)
    cfg8 = synth.ExpertConfig(n_layers=2, width=64, mlp_dim=128, n_q_heads=2, n_kv_heads=1, head_dim=32, state_dim=4,
                              action_dim=4, horizon=6, has_state_token=(cond == "pi0"), max_prefix_len=16, max_batch=1,
                              cond=cond, dtype="w8a8e4m3")
    cfg16 = synth.ExpertConfig(**{**cfg8.__dict__, "dtype": "w8e4m3"})
    W = synth.make_weights(cfg8, 31, std=0.2)
    kv = synth.make_prefix_kv(cfg8, 31, 9)
    state = synth.make_state(cfg8, 31) if cfg8.has_state_token else None
    noise = synth.make_noise(cfg8, 31)
    a = O.denoise(cfg8, W, kv, 9, state, noise, 3)
    b = O.denoise(cfg16, W, kv, 9, state, noise, 3)
    d = O.max_rel_err(a, b)
    assert 0.0 < d < 0.2, d


# ------------------------------------------------------------------------------------------------ W4A16 storage
def test_int4_decode_every_code_and_the_nibble_order_by_hand():
    # byte 0x1F: low nibble 15 -> +7 (even channel), high nibble 1 -> -7 (odd channel); 0x80: (0 -> -8, 8 -> 0)
    packed = np.array([[0x1F, 0x80], [0x98, 0x07]], dtype=np.uint8)
    assert np.array_equal(O.decode_int4(packed), [[7.0, -7.0, -8.0, 0.0], [0.0, 1.0, -1.0, -8.0]])
    allc = np.array([[(hi << 4) | lo for lo in range(16)] for hi in range(16)], dtype=np.uint8)
    dec = O.decode_int4(allc)
    assert np.array_equal(dec[:, 0::2], np.tile(np.arange(16) - 8.0, (16, 1)))
    assert np.array_equal(dec[:, 1::2], np.tile((np.arange(16) - 8.0)[:, None], (1, 16)))


def test_int4_column_quantizer_is_round_to_nearest_within_half_a_step():
    rng = np.random.default_rng(9)
    w = torch.from_numpy(rng.standard_normal((64, 10)).astype(np.float32))
    w[:, 3] = 0.0                                                   # an all-zero column: scale 1, codes 8
    w[0, 4], w[1, 4], w[2, 4], w[3, 4] = 7.0, 0.5, 1.5, -7.6        # column maximum 7.6... see below
    packed, scales, tag = synth.quantize_int4_columns(w)
    assert tag == "int4" and packed.shape == (64, 5) and packed.dtype == torch.uint8
    deq = O.to_f64((packed, scales, tag))
    s = scales.double().numpy()
    assert s[3] == 1.0 and np.all(deq[:, 3] == 0.0)
    assert np.allclose(s, np.maximum(w.abs().amax(dim=0).double().numpy(), 0) / 7.0 + (s == 1.0) * 1.0, rtol=1e-6)
    assert np.all(np.abs(deq - w.double().numpy()) <= s[None, :] / 2 * (1 + 1e-6))
    ints = deq / s[None, :]
    assert np.all(np.abs(ints - np.rint(ints)) < 1e-9) and ints.min() >= -8 and ints.max() <= 7
    # ties go to the even integer: with scale 1 (column maximum 7) 0.5 -> 0, 1.5 -> 2, 2.5 -> 2, -0.5 -> 0
    t = torch.tensor([[7.0], [0.5], [1.5], [2.5], [-0.5], [-7.0]])
    t = torch.cat([t, torch.zeros_like(t)], dim=1)
    p2, s2, _ = synth.quantize_int4_columns(t)
    assert np.array_equal(O.to_f64((p2, s2, "int4"))[:, 0], [7.0, 0.0, 2.0, 2.0, 0.0, -7.0])
