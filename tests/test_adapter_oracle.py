"""Pins of the adapter oracle (KV-layout writer, action post-processing) against hand-written values."""
import numpy as np

from oracle import adapter_oracle as A


def test_pack_prefix_kv_hand_written_ragged_example():
    # one layer, two requests of lengths 2 and 1, p_max = 3, one kv head of dimension 2; K holds 10s, V holds 20s
    k = np.array([[[[[10, 11]], [[12, 13]], [[-1, -1]]],          # request 0: rows 0, 1 real, row 2 padding
                   [[[14, 15]], [[-2, -2]], [[-3, -3]]]]])        # request 1: row 0 real
    v = k + 10 * (k > 0)
    out, cu = A.pack_prefix_kv(k, v, [2, 1])
    assert cu.tolist() == [0, 2, 3]
    assert out.shape == (1, 2, 3, 1, 2)
    assert out[0, 0, :, 0].tolist() == [[10, 11], [12, 13], [14, 15]]
    assert out[0, 1, :, 0].tolist() == [[20, 21], [22, 23], [24, 25]]


def test_pack_prefix_kv_handles_empty_requests_and_several_layers():
    rng = np.random.default_rng(0)
    k, v = rng.integers(0, 1000, (3, 4, 5, 2, 2)), rng.integers(0, 1000, (3, 4, 5, 2, 2))
    lens = [0, 5, 0, 3]
    out, cu = A.pack_prefix_kv(k, v, lens)
    assert cu.tolist() == [0, 0, 5, 5, 8]
    for l in range(3):
        assert np.array_equal(out[l, 0, 0:5], k[l, 1, :5]) and np.array_equal(out[l, 1, 5:8], v[l, 3, :3])


def test_postprocess_quantile_map_endpoints_midpoint_saturation_and_slice():
    q01, q99 = np.array([-2.0, 0.0, 10.0]), np.array([2.0, 1.0, 30.0])
    x = np.array([[[-1.0, -1.0, -1.0], [1.0, 1.0, 1.0], [0.0, 0.0, 0.0], [1.5, -7.0, 0.5]]])
    y = A.postprocess_actions(x, q01, q99)
    assert y[0, 0].tolist() == [-2.0, 0.0, 10.0]          # x = -1 -> q01
    assert y[0, 1].tolist() == [2.0, 1.0, 30.0]           # x = +1 -> q99
    assert y[0, 2].tolist() == [0.0, 0.5, 20.0]           # x = 0 -> midpoint
    assert y[0, 3].tolist() == [2.0, 0.0, 25.0]           # clipped to [-1, 1] first
    assert A.postprocess_actions(x, q01, q99, clip=None)[0, 3].tolist() == [3.0, -3.0, 25.0]
    z = A.postprocess_actions(x, q01, q99, out_horizon=2, out_dim=2)
    assert z.shape == (1, 2, 2) and z[0, 1].tolist() == [2.0, 1.0]
    assert A.postprocess_actions(x, None, None, clip=None)[0, 3].tolist() == [1.5, -7.0, 0.5]


def test_feature_projection_by_hand_and_with_one_hot_weights():
    # two tokens, three feature channels, one kv head of two channels, two layers, small integers
    F = np.array([[1.0, 2.0, 3.0], [0.0, -1.0, 4.0]])
    wk = [np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]]), np.array([[2.0, 0.0], [0.0, 0.0], [0.0, -1.0]])]
    wv = [np.array([[0.0, 1.0], [1.0, 0.0], [0.0, 0.0]]), np.array([[1.0, 1.0], [1.0, 1.0], [1.0, 1.0]])]
    out = A.project_features_kv(F, wk, wv, 1, 2)
    assert out.shape == (2, 2, 2, 1, 2)
    assert np.array_equal(out[0, 0, :, 0], [[4.0, 5.0], [4.0, 3.0]])      # K, layer 0: (f0 + f2, f1 + f2)
    assert np.array_equal(out[0, 1, :, 0], [[2.0, 1.0], [-1.0, 0.0]])     # V, layer 0: (f1, f0)
    assert np.array_equal(out[1, 0, :, 0], [[2.0, -3.0], [0.0, -4.0]])    # K, layer 1: (2 f0, -f2)
    assert np.array_equal(out[1, 1, :, 0], [[6.0, 6.0], [3.0, 3.0]])      # V, layer 1: sums
    # one-hot weights select feature columns, head-major then channel
    rng = np.random.default_rng(0)
    F = rng.standard_normal((5, 8))
    sel = np.zeros((8, 4))
    for c, f in enumerate([7, 0, 3, 3]):
        sel[f, c] = 1.0
    out = A.project_features_kv(F, [sel], [sel[:, ::-1]], 2, 2)
    assert np.array_equal(out[0, 0].reshape(5, 4), F[:, [7, 0, 3, 3]])
    assert np.array_equal(out[0, 1].reshape(5, 4), F[:, [3, 3, 0, 7]])
