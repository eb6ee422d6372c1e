"""The W8A8 arithmetic checked where it can be checked exactly: the quantization kernel and the FP8 GEMM of the loop,
through the stand-alone projection entry point, against the oracle's quantizer and its float64 product on the same
stored activations.  Codes and scales must agree exactly; the product to fp32 summation error."""
import numpy as np
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _case(seed, M, K, N, spread):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K)).astype(np.float32) * np.exp(rng.uniform(-spread, spread, (M, 1))).astype(np.float32)
    x[0, :] = 0.0 if M > 3 else x[0, :]                       # an all-zero row: scale 1, codes 0
    xb = torch.from_numpy(x).to(torch.bfloat16)
    master = torch.from_numpy(rng.standard_normal((K, N)).astype(np.float32) * 0.05)
    codes, scales = synth.quantize_e4m3_columns(master)
    return xb, codes, scales


@pytest.mark.parametrize("M,K,N", [(1, 128, 128), (51, 1024, 2560), (3, 256, 384), (200, 2048, 1024), (408, 4096, 1024),
                                   (1300, 1024, 512)])
def test_projection_codes_scales_and_product_match_the_oracle(M, K, N):
    xb, codes, scales = _case(M * 7 + K, M, K, N, 3.0)
    y, qc, qs = binding.w8a8_project(xb.cuda(), codes.cuda(), scales.cuda(), return_codes=True)
    torch.cuda.synchronize()
    q_ref, s_ref = O.quantize_rows_e4m3(xb.to(torch.float32).numpy())
    # scales: the same float32 division; codes: the same decision on the same inputs -> exact
    assert np.array_equal(qs.cpu().numpy(), s_ref[:, 0].astype(np.float32))
    assert np.array_equal(O.decode_e4m3(qc.cpu().numpy()), q_ref)
    w = O.to_f64((codes, scales))
    ref = (q_ref @ w) * s_ref
    got = y.double().cpu().numpy()
    scale = np.max(np.abs(ref), axis=1, keepdims=True) + 1e-300
    assert np.max(np.abs(got - ref) / scale) <= 2e-6, float(np.max(np.abs(got - ref) / scale))


def test_values_that_sit_on_rounding_ties_and_beyond_the_range():
    # a row whose maximum maps to 448 and whose other elements sit exactly on midpoints of the e4m3 grid
    K, N = 128, 128
    grid_mid = np.array([1.0625, 1.1875, 15.5, 0.5 * 2.0 ** -9, 1.5 * 2.0 ** -9, 240.0 + 8.0, 416.0 + 16.0], dtype=np.float64)
    row = np.zeros(K)
    row[0] = 448.0
    row[1:1 + len(grid_mid)] = grid_mid
    row[20:27] = -grid_mid
    x = torch.from_numpy(np.stack([row, row * 0.25]).astype(np.float32)).to(torch.bfloat16)
    assert np.array_equal(x.to(torch.float64).numpy()[0], row)       # all representable in bf16
    codes = torch.zeros(K, N, dtype=torch.uint8)
    codes[:, 0] = 0x38                                                # value 1.0 in column 0: y[:, 0] = s * sum of codes
    scales = torch.ones(N)
    y, qc, qs = binding.w8a8_project(x.cuda(), codes.cuda(), scales.cuda(), return_codes=True)
    q_ref, s_ref = O.quantize_rows_e4m3(x.to(torch.float32).numpy())
    assert np.array_equal(O.decode_e4m3(qc.cpu().numpy()), q_ref)
    assert np.array_equal(qs.cpu().numpy(), s_ref[:, 0].astype(np.float32))
    assert np.allclose(y[:, 0].double().cpu().numpy(), (q_ref.sum(axis=1) * s_ref[:, 0]), rtol=1e-6)


def test_bad_arguments_are_refused():
    x = torch.zeros(4, 100, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.PhyaiError):
        binding.w8a8_project(x, torch.zeros(100, 128, dtype=torch.uint8, device="cuda"), torch.ones(128, device="cuda"))
