"""The stand-alone attention operator (phyai_suffix_attention) against the oracle's attention on
random inputs: ragged prefixes, several key tiles, split and unsplit key ranges, RoPE on/off."""
import numpy as np
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding

pytestmark = pytest.mark.gpu


def make_case(seed, Hq, Hkv, dh, S, lens, L=2, layer=1, theta=10000.0):
    rng = np.random.default_rng(seed)
    B = len(lens)
    qkv = torch.from_numpy(rng.standard_normal((B * S, (Hq + 2 * Hkv) * dh)).astype(np.float32))
    T = int(sum(lens)) + 3                      # a few never-read rows at the end
    kv = torch.from_numpy(rng.standard_normal((L, 2, T, Hkv, dh)).astype(np.float32)).to(torch.bfloat16)
    kv[:, :, int(sum(lens)):] = float("nan")    # must never be read
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    rope = None
    if theta:
        pos = np.arange(max(lens) + S, dtype=np.float64)[:, None]
        ang = pos * theta ** (-2.0 * np.arange(dh // 2, dtype=np.float64) / dh)[None, :]
        rope = torch.from_numpy(np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32))
    return qkv, kv, cu, rope


def oracle_attention(qkv, kv, cu, Hq, Hkv, dh, S, layer, theta, block_causal=False):
    outs = []
    q64, kv64 = qkv.double().numpy(), kv.double().numpy()
    for b in range(len(cu) - 1):
        lo, hi = int(cu[b]), int(cu[b + 1])
        rows = q64[b * S:(b + 1) * S]
        q = rows[:, :Hq * dh].reshape(S, Hq, dh)
        k = rows[:, Hq * dh:(Hq + Hkv) * dh].reshape(S, Hkv, dh)
        v = rows[:, (Hq + Hkv) * dh:].reshape(S, Hkv, dh)
        pos = (hi - lo) + np.arange(S)
        q, k = O.rope(q, pos, theta), O.rope(k, pos, theta)
        mask = np.ones((S, S), dtype=bool)
        if block_causal:
            mask[0, 1:] = False
        outs.append(O.attention(q, kv64[layer, 0, lo:hi], kv64[layer, 1, lo:hi], k, v, mask, Hq // Hkv).reshape(S, Hq * dh))
    return np.concatenate(outs)


@pytest.mark.parametrize("Hq,Hkv,dh,S,lens,splits,theta,causal", [
    (8, 1, 256, 51, [816], 0, 10000.0, False),          # the pi0-shaped batch-1 case (16-way split)
    (8, 1, 256, 51, [968, 600, 0, 65], 1, 10000.0, False),
    (4, 2, 128, 14, [200, 1, 63, 64, 129], 3, 10000.0, True),
    (2, 1, 64, 64, [100, 7], 2, 0.0, False),
])
def test_attention_operator_matches_oracle(Hq, Hkv, dh, S, lens, splits, theta, causal):
    qkv, kv, cu, rope = make_case(7, Hq, Hkv, dh, S, lens, theta=theta)
    desc = binding.attention_desc(Hq, Hkv, dh, S, n_layers=2, layer=1, block_causal=causal, num_splits=splits)
    out, status = binding.suffix_attention(desc, qkv.cuda(), kv.cuda(), torch.from_numpy(cu).cuda(),
                                           None if rope is None else rope.cuda())
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle_attention(qkv, kv, cu, Hq, Hkv, dh, S, 1, theta, causal)
    got = out.double().cpu().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err <= 2e-2, err


def test_attention_operator_rejects_bad_arguments():
    qkv, kv, cu, rope = make_case(8, 2, 1, 64, 8, [10])
    desc = binding.attention_desc(2, 1, 96, 8, n_layers=2, layer=0)
    with pytest.raises(binding.PhyaiError) as e:
        binding.suffix_attention(desc, qkv.cuda(), kv.cuda(), torch.from_numpy(cu).cuda(), None)
    assert e.value.status == binding.ERR_UNSUPPORTED
    desc = binding.attention_desc(2, 1, 64, 8, n_layers=2, layer=2)
    with pytest.raises(binding.PhyaiError) as e:
        binding.suffix_attention(desc, qkv.cuda(), kv.cuda(), torch.from_numpy(cu).cuda(), None)
    assert e.value.status == binding.ERR_INVALID_ARG
