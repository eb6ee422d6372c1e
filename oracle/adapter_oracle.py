"""CPU oracle of the adapter-side steps either side of the denoising loop.

TEST INFRASTRUCTURE ONLY (see expert_oracle.py): nothing in the product path may import this file.

What it computes (paper, Sec. "Architecture": the model adapter owns cache layout and action conversion; appendices
on the pi0 / pi0.5 reproductions: actions are clipped to [-1, 1] and un-normalised with the checkpoint's q01 / q99
quantile statistics, the controller uses a slice of the chunk):

* ``pack_prefix_kv``: padded per-layer K / V ``[L, B, p_max, Hkv, dh]`` and per-request lengths -> the library's
  ragged layout ``[L, 2, total, Hkv, dh]`` (requests concatenated along the token axis, no padding rows) and the
  exclusive prefix sum of the lengths.  A gather: exact for any element type.
* ``postprocess_actions``: ``(clip(x, lo, hi) + 1) / 2 * (q99 - q01) + q01`` on the first ``out_horizon`` steps and
  ``out_dim`` action dimensions, float64.  Reading: the clip acts in normalised space, before un-normalisation.

* ``project_features_kv``: the request-local K / V projections of a feature-handoff head (results section, phase
  list of the GR00T profile: the action head contains "request-local cross-attention K/V projections"; the paper gives
  no equations -- reading: per layer ``K_l = F Wk_l``, ``V_l = F Wv_l`` of the fixed vision-language features ``F``,
  computed once per request, no rotary embedding on features) -> ``[L, 2, P, Hkv, dh]``, float64 matmul.

Pins (tests/test_adapter_oracle.py): a hand-written ragged example with distinct integers; endpoints and midpoint of
the quantile map (x = -1 -> q01, x = +1 -> q99, x = 0 -> the mean of the two), saturation outside [-1, 1], the slice;
the projection with one-hot weights (a column selection), with small integers by hand, and its layer / plane order.
"""
from __future__ import annotations

import numpy as np


def pack_prefix_kv(k: np.ndarray, v: np.ndarray, lens) -> tuple:
    """k, v ``[L, B, p_max, Hkv, dh]``; lens ``[B]``.  Returns (packed ``[L, 2, sum(lens), Hkv, dh]``, cu ``[B+1]``)."""
    L, B, p_max, Hkv, dh = k.shape
    lens = [int(n) for n in lens]
    cu = np.zeros(B + 1, dtype=np.int32)
    for b in range(B):
        cu[b + 1] = cu[b] + lens[b]
    out = np.zeros((L, 2, int(cu[B]), Hkv, dh), dtype=k.dtype)
    for l in range(L):
        for b in range(B):
            for p in range(lens[b]):
                out[l, 0, cu[b] + p] = k[l, b, p]
                out[l, 1, cu[b] + p] = v[l, b, p]
    return out, cu


def postprocess_actions(x, q01, q99, clip=(-1.0, 1.0), out_horizon=None, out_dim=None) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    B, H, A = x.shape
    out_horizon, out_dim = out_horizon or H, out_dim or A
    y = x[:, :out_horizon, :out_dim]
    if clip is not None and clip[0] < clip[1]:
        y = np.minimum(np.maximum(y, clip[0]), clip[1])
    lo = -np.ones(out_dim) if q01 is None else np.asarray(q01, dtype=np.float64)[:out_dim]
    hi = np.ones(out_dim) if q99 is None else np.asarray(q99, dtype=np.float64)[:out_dim]
    return (y + 1.0) / 2.0 * (hi - lo) + lo


def project_features_kv(features, wk, wv, n_kv_heads: int, head_dim: int) -> np.ndarray:
    """features ``[P, Dv]``; wk, wv: per-layer lists of ``[Dv, Hkv * dh]``.  Returns ``[L, 2, P, Hkv, dh]`` float64."""
    F = np.asarray(features, dtype=np.float64)
    L = len(wk)
    out = np.zeros((L, 2, F.shape[0], n_kv_heads, head_dim), dtype=np.float64)
    for l in range(L):
        out[l, 0] = (F @ np.asarray(wk[l], dtype=np.float64)).reshape(F.shape[0], n_kv_heads, head_dim)
        out[l, 1] = (F @ np.asarray(wv[l], dtype=np.float64)).reshape(F.shape[0], n_kv_heads, head_dim)
    return out
