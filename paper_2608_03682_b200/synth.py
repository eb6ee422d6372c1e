"""Seeded synthetic inputs for the action-expert denoising loop.

This module only *describes shapes* and *draws random numbers*.  It contains none of the
method's arithmetic (no norm, attention, embedding or solver code), so both the CPU oracle's
tests and the CUDA path's tests can take their inputs from here without sharing any
computation.  The only numeric transformations are storage casts done by library routines:
round-to-nearest-even float32 -> bfloat16, float32 -> float8_e4m3fn (PyTorch casts) and float32 -> 4-bit integers
(``torch.round`` and a clamp) with one scale per output channel.

Shapes follow the paper's pi0 / pi0.5 serving workloads (three camera views, a 50-action
chunk, ten Euler steps, bf16; Sec. "Results", batch sweep) with random-initialised weights:
no checkpoint, dataset or simulator is involved.

Recipe: ``numpy.random.Generator(PCG64(SeedSequence([cfg_id, stream_id, ...])))``, float32
draws; streams: 0 = weights, 1 = prefix KV, 2 = state, 3 = noise, 4 = ragged lengths.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Tuple

import numpy as np
import torch

STREAM_WEIGHTS, STREAM_KV, STREAM_STATE, STREAM_NOISE, STREAM_LENS = 0, 1, 2, 3, 4

#: names of the seven large per-layer matrices (the ones the W8A16 mode stores as e4m3)
BIG_MATS = ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown")


@dataclass(frozen=True)
class ExpertConfig:
    """Shape/hyper-parameter description of one action expert (mirrors ``phyai_expert_config_t``)."""

    n_layers: int
    width: int
    mlp_dim: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    state_dim: int
    action_dim: int
    horizon: int
    has_state_token: bool
    max_prefix_len: int
    max_batch: int = 1
    cond: str = "pi0"            # "pi0": time concatenated into the action MLP; "pi05": adaRMSNorm
    dtype: str = "bf16"          # "f32" | "bf16" | "w8e4m3" | "w8a8e4m3" | "w4a16" (storage of weights and prefix KV; the last
                                 # "w8a8e4m3" also names the arithmetic of the seven large projections: e4m3 x e4m3)
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0  # 0 disables RoPE
    time_min_period: float = 4e-3
    time_max_period: float = 4.0
    gelu_exact: bool = False
    suffix_block_causal: bool = False

    def __post_init__(self):
        # The C ABI carries these four as float32; store the float32-representable value so that
        # every consumer of the configuration sees exactly the same number.
        for name in ("rms_eps", "rope_theta", "time_min_period", "time_max_period"):
            object.__setattr__(self, name, float(np.float32(getattr(self, name))))

    @property
    def suffix_len(self) -> int:
        return self.horizon + (1 if self.has_state_token else 0)

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def with_(self, **kw) -> "ExpertConfig":
        return replace(self, **kw)


# ----------------------------------------------------------------------------------------------
# Named workloads (the five configurations of the benchmark definition)
# ----------------------------------------------------------------------------------------------
def tiny_config() -> ExpertConfig:
    """C1: tiny fp32 expert, batch 1."""
    return ExpertConfig(n_layers=2, width=256, mlp_dim=1024, n_q_heads=4, n_kv_heads=1, head_dim=64,
                        state_dim=8, action_dim=7, horizon=16, has_state_token=True,
                        max_prefix_len=64, max_batch=1, cond="pi0", dtype="f32")


def pi0_config(max_batch: int = 1, dtype: str = "bf16", max_prefix_len: int = 968) -> ExpertConfig:
    """C2 / C4 / C5: pi0-shaped expert."""
    return ExpertConfig(n_layers=18, width=1024, mlp_dim=4096, n_q_heads=8, n_kv_heads=1, head_dim=256,
                        state_dim=32, action_dim=32, horizon=50, has_state_token=True,
                        max_prefix_len=max_prefix_len, max_batch=max_batch, cond="pi0", dtype=dtype)


def pi05_config(max_batch: int = 1, dtype: str = "bf16", max_prefix_len: int = 968) -> ExpertConfig:
    """C3: pi0.5-shaped expert (adaRMSNorm conditioning, no state token)."""
    return ExpertConfig(n_layers=18, width=1024, mlp_dim=4096, n_q_heads=8, n_kv_heads=1, head_dim=256,
                        state_dim=32, action_dim=32, horizon=50, has_state_token=False,
                        max_prefix_len=max_prefix_len, max_batch=max_batch, cond="pi05", dtype=dtype)


WORKLOADS = {
    # name: (cfg_id, config factory, prefix length(s), n_steps, batch)
    "C1": dict(cfg_id=1, prefix=64, n_steps=4, batch=1),
    "C2": dict(cfg_id=2, prefix=816, n_steps=10, batch=1),
    "C3": dict(cfg_id=3, prefix=968, n_steps=10, batch=1),
    "C4": dict(cfg_id=4, prefix=(600, 968), n_steps=10, batch=64),
    "C5": dict(cfg_id=5, prefix=816, n_steps=10, batch=(1, 8, 64, 256)),
}


# ----------------------------------------------------------------------------------------------
# Random draws
# ----------------------------------------------------------------------------------------------
def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(key))))


def _normal(rng: np.random.Generator, shape, std: float) -> torch.Tensor:
    a = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return torch.from_numpy(a)


def _store(t: torch.Tensor, dtype: str) -> torch.Tensor:
    """Cast float32 master values to the storage type of activations-side tensors."""
    if dtype == "f32":
        return t
    return t.to(torch.bfloat16)  # round-to-nearest-even


def weight_shapes(cfg: ExpertConfig) -> List[Tuple[str, Tuple[int, ...]]]:
    """(name, shape) of every weight tensor, in the fixed order in which they are drawn.

    Matrices are ``[in, out]`` row-major; per-layer names carry a ``.{layer}`` suffix."""
    D, F, A = cfg.width, cfg.mlp_dim, cfg.action_dim
    ada = cfg.cond == "pi05"
    out: List[Tuple[str, Tuple[int, ...]]] = []
    if cfg.has_state_token:
        out += [("state_w", (cfg.state_dim, D)), ("state_b", (D,))]
    out += [("action_in_w", (A, D)), ("action_in_b", (D,))]
    out += [("time_mlp1_w", (D if ada else 2 * D, D)), ("time_mlp1_b", (D,)),
            ("time_mlp2_w", (D, D)), ("time_mlp2_b", (D,))]
    out += [("action_out_w", (D, A)), ("action_out_b", (A,))]
    if ada:
        out += [("final_norm", (D, 3 * D)), ("final_norm_b", (3 * D,))]
    else:
        out += [("final_norm", (D,))]
    for l in range(cfg.n_layers):
        out += [(f"wq.{l}", (D, cfg.q_dim)), (f"wk.{l}", (D, cfg.kv_dim)), (f"wv.{l}", (D, cfg.kv_dim)),
                (f"wo.{l}", (cfg.q_dim, D)), (f"wgate.{l}", (D, F)), (f"wup.{l}", (D, F)),
                (f"wdown.{l}", (F, D))]
        for site in ("norm1", "norm2"):
            if ada:
                out += [(f"{site}.{l}", (D, 3 * D)), (f"{site}_b.{l}", (3 * D,))]
            else:
                out += [(f"{site}.{l}", (D,))]
    return out


def quantize_e4m3_columns(w: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """Round-to-nearest per-output-channel e4m3 storage of a float32 ``[in, out]`` matrix.

    Returns (codes as uint8 ``[in, out]``, float32 scales ``[out]``); ``scale = max|column|/448``
    (1 for an all-zero column).  The rounding itself is PyTorch's float8_e4m3fn cast."""
    amax = w.abs().amax(dim=0)
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax)).to(torch.float32)
    q = (w / scale).clamp_(-448.0, 448.0).to(torch.float8_e4m3fn)
    return q.view(torch.uint8).contiguous(), scale.contiguous()


def quantize_int4_columns(w: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor, str]:
    """Round-to-nearest per-output-channel symmetric int4 storage of a float32 ``[in, out]`` matrix (``out`` even).

    Returns (packed uint8 ``[in, out / 2]``, float32 scales ``[out]``, the tag ``"int4"``): ``scale = max|column| / 7``
    (1 for an all-zero column), integer ``q = clamp(round_half_even(w / scale), -8, 7)``, stored as the code ``q + 8``;
    a byte holds two neighbouring output channels of one input row, the even channel in the low nibble."""
    amax = w.abs().amax(dim=0)
    scale = torch.where(amax > 0, amax / 7.0, torch.ones_like(amax)).to(torch.float32)
    q = torch.round(w / scale).clamp_(-8, 7).to(torch.int16) + 8          # torch.round: half to even
    packed = (q[:, 0::2] | (q[:, 1::2] << 4)).to(torch.uint8)
    return packed.contiguous(), scale.contiguous(), "int4"


def make_weights(cfg: ExpertConfig, cfg_id: int, std: float = 0.02) -> Dict[str, object]:
    """All weights of one expert, ~N(0, std) in float32, cast to the configuration's storage.

    For ``dtype == "w8e4m3"`` / ``"w8a8e4m3"`` the seven large per-layer matrices become ``(codes, scales)``
    tuples and everything else is bfloat16."""
    rng = _rng(cfg_id, STREAM_WEIGHTS)
    W: Dict[str, object] = {}
    for name, shape in weight_shapes(cfg):
        master = _normal(rng, shape, std)
        base = name.split(".")[0]
        if cfg.dtype in ("w8e4m3", "w8a8e4m3") and base in BIG_MATS:
            W[name] = quantize_e4m3_columns(master)
        elif cfg.dtype == "w4a16" and base in BIG_MATS:
            W[name] = quantize_int4_columns(master)
        else:
            W[name] = _store(master, "f32" if cfg.dtype == "f32" else "bf16")
    return W


def make_prefix_kv(cfg: ExpertConfig, cfg_id: int, prefix_len: int, request: int = 0) -> torch.Tensor:
    """Prefix K/V of one request, ``[L, 2, P, Hkv, dh]`` ~N(0,1), K taken as already rotated."""
    rng = _rng(cfg_id, STREAM_KV, request)
    kv = _normal(rng, (cfg.n_layers, 2, prefix_len, cfg.n_kv_heads, cfg.head_dim), 1.0)
    return _store(kv, "f32" if cfg.dtype == "f32" else "bf16")


def make_state(cfg: ExpertConfig, cfg_id: int, request: int = 0) -> torch.Tensor:
    return _normal(_rng(cfg_id, STREAM_STATE, request), (cfg.state_dim,), 1.0)


def make_noise(cfg: ExpertConfig, cfg_id: int, request: int = 0) -> torch.Tensor:
    return _normal(_rng(cfg_id, STREAM_NOISE, request), (cfg.horizon, cfg.action_dim), 1.0)


STREAM_FEATURES, STREAM_KV_PROJ = 6, 7


def make_features(cfg_id: int, tokens: int, feat_dim: int, request: int = 0) -> torch.Tensor:
    """Vision-language feature rows of one request for a feature-handoff head, ``[tokens, feat_dim]`` ~N(0,1), bf16."""
    return _normal(_rng(cfg_id, STREAM_FEATURES, request), (tokens, feat_dim), 1.0).to(torch.bfloat16)


def make_kv_projections(cfg: ExpertConfig, cfg_id: int, feat_dim: int):
    """Per-layer request-local K / V projection matrices ``[feat_dim, Hkv * dh]`` ~N(0, feat_dim^-1/2), bf16: the
    projected keys and values then have unit scale like the synthetic prefix KV of the other workloads."""
    rng = _rng(cfg_id, STREAM_KV_PROJ)
    std = float(feat_dim) ** -0.5
    wk = [_normal(rng, (feat_dim, cfg.kv_dim), std).to(torch.bfloat16) for _ in range(cfg.n_layers)]
    wv = [_normal(rng, (feat_dim, cfg.kv_dim), std).to(torch.bfloat16) for _ in range(cfg.n_layers)]
    return wk, wv


def groot_like_config(max_batch: int = 1, n_layers: int = 16, max_prefix_len: int = 640) -> ExpertConfig:
    """A feature-handoff action head of the shape the paper's GR00T profile names (action chunk 40 x 132, four
    flow-matching steps); the paper gives no widths for it, so the transformer dimensions are this repository's
    choice: width 1024, MLP 4096, 8 query heads on 2 kv heads of 128, no rotary embedding on the feature keys."""
    return ExpertConfig(n_layers=n_layers, width=1024, mlp_dim=4096, n_q_heads=8, n_kv_heads=2, head_dim=128, state_dim=64,
                        action_dim=132, horizon=40, has_state_token=True, max_prefix_len=max_prefix_len, max_batch=max_batch,
                        cond="pi0", dtype="bf16", rope_theta=0.0)


def make_ragged_lengths(cfg_id: int, batch: int, lo: int, hi: int) -> np.ndarray:
    """``batch`` prefix lengths, integers uniform on [lo, hi] inclusive."""
    return _rng(cfg_id, STREAM_LENS).integers(lo, hi + 1, size=batch).astype(np.int32)


def pack_prefix_kv(kvs: List[torch.Tensor]) -> Tuple[torch.Tensor, np.ndarray]:
    """Concatenate per-request ``[L,2,P_b,Hkv,dh]`` tensors along the token axis (no padding rows).

    Returns the packed ``[L,2,P_total,Hkv,dh]`` tensor and ``cu_prefix_lens`` (int32, ``[B+1]``)."""
    lens = np.array([kv.shape[2] for kv in kvs], dtype=np.int64)
    cu = np.zeros(len(kvs) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return torch.cat(kvs, dim=2).contiguous(), cu
