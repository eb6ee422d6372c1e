"""Float64 CPU oracle of the flow-matching action-expert denoising loop.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA library is
checked against.  Nothing in the product path may import it; it shares no code with the CUDA
path and imports nothing from the package.  Only tests, the smoke check and the benchmark's
CPU-baseline leg call it.

What it computes (paper, Sec. "Optimization Methods": graph replay paragraph - the
vision-language prefix is fixed over ten Euler steps, its KV tensors are retained, the
sinusoidal timestep table and each layer's AdaRMS modulation table depend only on the step;
kernel-fusion paragraph - AdaRMSNorm, residual-add + RMSNorm, one GEMM for Q,K,V, one for MLP
gate and up, GeGLU fused with its multiply; operator-selection paragraph - a 50-token query
against a longer prefix with head dimension 256; quantization paragraph - offline
round-to-nearest weights).  The paper gives no equations for the expert itself; the readings
taken where it is silent are listed in the design notes and marked "reading" below.

The method has no shortcut result: the GPU computes the same iteration, only faster.  So this
is the iteration written out in the paper's order, in float64, on exactly the stored input
values (bf16 / e4m3 inputs convert to float64 exactly).  Library primitives used as steps:
``numpy.matmul``, ``numpy.exp/sin/cos/tanh``.

Pins (tests/test_oracle_*.py): zero velocity head returns the noise bit-exactly; constant head
closed form; brute-force attention in pure-Python loops; torch float64 library routines for
rms_norm / gelu / silu / scaled_dot_product_attention; prefix permutation; NaN tail beyond
prefix_len; sinusoid special values; RoPE relative-position property; hand-computed network
with identity blocks; exhaustive e4m3 decode against ml_dtypes; e4m3 rounding against torch's
float8_e4m3fn cast, all codes as fixed points, ties and saturation by hand; the W8A8 projection on
inputs that are already on the e4m3 grid.
Whole-network values: **parity unpinned** by any number printed in the paper (it prints none);
they are covered by the composition of the pins above and by a second, differently structured
transcription in the tests.
"""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------------------------
# storage decoding (exact)
# ----------------------------------------------------------------------------------------------
def decode_e4m3(codes: np.ndarray) -> np.ndarray:
    """OCP e4m3 "fn" byte -> float64: 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinities,
    S.1111.111 is NaN, exponent field 0 is subnormal (quantization paragraph; format: reading)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where((c >> 7) & 1, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    normal = (1.0 + m / 8.0) * np.exp2((e - 7).astype(F64))
    sub = (m / 8.0) * 2.0 ** (-6)
    val = np.where(e == 0, sub, normal)
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return (sign * val).astype(F64)


def decode_int4(packed) -> np.ndarray:
    """W4A16 storage (quantization paragraph: W4A16, round-to-nearest; the format is a reading): a byte holds the
    codes of two neighbouring output channels of one input row, the even channel in the low nibble; a code c in 0..15
    stands for the integer c - 8.  ``[in, out / 2]`` bytes -> ``[in, out]`` float64 integers in [-8, 7]."""
    b = packed.numpy() if hasattr(packed, "numpy") else np.asarray(packed)
    b = b.astype(np.int64)
    out = np.empty((b.shape[0], 2 * b.shape[1]), dtype=F64)
    out[:, 0::2] = (b & 15) - 8
    out[:, 1::2] = (b >> 4) - 8
    return out


def to_f64(t) -> np.ndarray:
    """Stored tensor -> float64 array, exactly.  Accepts numpy arrays, torch tensors (f32/bf16)
    and ``(codes_uint8[in,out], scales_f32[out])`` pairs of the W8A16 / W8A8 modes (and ``(packed, scales, "int4")``
    triples of the W4A16 mode), which decode to
    ``decode(code) * scale`` per output channel (column)."""
    if isinstance(t, tuple) and len(t) == 3 and t[2] == "int4":
        return decode_int4(t[0]) * to_f64(t[1])[None, :]
    if isinstance(t, tuple):
        codes, scales = t
        codes = codes.numpy() if hasattr(codes, "numpy") else np.asarray(codes)
        return decode_e4m3(codes) * to_f64(scales)[None, :]
    if isinstance(t, np.ndarray):
        return t.astype(F64)
    import torch  # storage container only

    return t.detach().to(torch.float64).cpu().numpy()


def round_e4m3(y: np.ndarray) -> np.ndarray:
    """Nearest OCP e4m3 "fn" value of every element, ties to the even mantissa, saturating at the
    largest finite value 448 (the format has no infinities): the round-to-nearest of the quantization
    paragraph applied to a value that is already divided by its scale.  Normal numbers 2^e (1 + m/8),
    e in [-6, 8]; below 2^-6 the grid is uniform with step 2^-9 (subnormals)."""
    y = np.asarray(y, dtype=F64)
    a = np.minimum(np.abs(y), 448.0)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.clip(e, -6.0, 8.0)
    step = np.exp2(e - 3.0)                      # spacing of the grid in the binade of a
    q = np.rint(a / step) * step                 # numpy.rint rounds halves to even
    return np.sign(y) * np.minimum(q, 448.0)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bfloat16 (ties to even), returned as float32: the upper 16 bits of the float32 pattern after
    adding half an ulp (0x7FFF plus the lowest kept bit)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000).astype(np.uint32)
    return r.view(np.float32)


def quantize_rows_e4m3(x: np.ndarray):
    """W8A8 activation quantization (quantization paragraph: the paper lists W8A8 among its
    round-to-nearest modes; granularity and scale rule are a reading).  The activation that enters a
    projection is a bfloat16 tensor, as in the W8A16 mode; every row (token) of it gets the scale
    s = max|x| / 448 (1 for an all-zero row) and its elements become round_e4m3(x / s).  The decision is
    taken the way the device takes it: on the bfloat16 rounding of x, with scale and quotient in float32.
    Returns (codes' values as float64, scales as float64): the projection then computes (values @ Wq) * s."""
    xb = round_bf16(np.asarray(x, dtype=np.float32))
    amax = np.max(np.abs(xb), axis=-1, keepdims=True)
    s = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    y = (xb / s).astype(np.float32)
    return round_e4m3(y.astype(F64)), s.astype(F64)


def project(cfg, x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """x @ w for one of the seven large per-layer matrices; in the W8A8 mode through the per-token
    e4m3 quantization of x (the weights are already the decoded e4m3 values times their scales)."""
    if getattr(cfg, "dtype", "") == "w8a8e4m3":
        q, s = quantize_rows_e4m3(x)
        return (q @ w) * s
    return x @ w


# ----------------------------------------------------------------------------------------------
# elementary functions
# ----------------------------------------------------------------------------------------------
def swish(z: np.ndarray) -> np.ndarray:
    """swish(z) = z / (1 + exp(-z))."""
    return z / (1.0 + np.exp(-z))


def gelu(z: np.ndarray, exact: bool = False) -> np.ndarray:
    """GELU of the GeGLU MLP (kernel-fusion paragraph).  Reading: tanh form
    0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3))); ``exact`` selects 0.5 z (1 + erf(z/sqrt 2))."""
    if exact:
        erf = np.vectorize(math.erf, otypes=[F64])
        return 0.5 * z * (1.0 + erf(z / math.sqrt(2.0)))
    return 0.5 * z * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))


def time_grid(n_steps: int):
    """Explicit Euler from t = 1 to t = 0: dt = -1/n, t_k = 1 - k/n computed directly."""
    dt = -1.0 / n_steps
    return dt, [1.0 - k / n_steps for k in range(n_steps)]


def sinusoid(t: float, width: int, min_period: float, max_period: float) -> np.ndarray:
    """Sinusoidal timestep embedding tau in R^width (graph-replay paragraph: "sinusoidal
    timestep table").  Reading: periods geometric from min to max over width/2 channels,
    [sin | cos], argument 2 pi t / period."""
    half = width // 2
    j = np.arange(half, dtype=F64)
    frac = j / (half - 1) if half > 1 else np.zeros(half)
    period = min_period * (max_period / min_period) ** frac
    arg = 2.0 * math.pi * t / period
    return np.concatenate([np.sin(arg), np.cos(arg)])


def rms_rows(h: np.ndarray, eps: float) -> np.ndarray:
    """r_i = 1 / sqrt(mean_d h[i,d]^2 + eps)."""
    return 1.0 / np.sqrt(np.mean(h * h, axis=-1, keepdims=True) + eps)


def norm_plain(h: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """RMSNorm with gain (1 + gamma) (reading: Gemma convention)."""
    return h * rms_rows(h, eps) * (1.0 + gamma)


def norm_ada(h: np.ndarray, c: np.ndarray, w_mod: np.ndarray, b_mod: np.ndarray, eps: float):
    """AdaRMSNorm: m = c W_mod + b_mod in R^{3D} = (scale | shift | gate);
    n = h r (1 + scale) + shift.  Returns (n, gate)."""
    D = h.shape[-1]
    m = c @ w_mod + b_mod
    sc, sh, g = m[0:D], m[D:2 * D], m[2 * D:3 * D]
    return h * rms_rows(h, eps) * (1.0 + sc) + sh, g


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding on ``x[token, head, dh]`` at integer positions ``pos[token]``; pairs
    (j, j + dh/2), angle pos * theta^(-2j/dh).  theta == 0 means no rotation (reading)."""
    if theta == 0.0:
        return x
    dh = x.shape[-1]
    half = dh // 2
    j = np.arange(half, dtype=F64)
    inv = theta ** (-2.0 * j / dh)
    phi = pos.astype(F64)[:, None] * inv[None, :]
    cos, sin = np.cos(phi)[:, None, :], np.sin(phi)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * cos - b * sin, b * cos + a * sin], axis=-1)


def suffix_visibility(cfg) -> np.ndarray:
    """mask[i][j]: may suffix query i see suffix key j.  Default: everything (bidirectional,
    state token included).  ``suffix_block_causal``: the state token forms its own earlier
    block - it sees only itself, action tokens see everything."""
    S = cfg.horizon + (1 if cfg.has_state_token else 0)
    mask = np.ones((S, S), dtype=bool)
    if getattr(cfg, "suffix_block_causal", False) and cfg.has_state_token:
        mask[0, 1:] = False
    return mask


def attention(q, k_prefix, v_prefix, k_suffix, v_suffix, mask, group: int) -> np.ndarray:
    """Suffix queries over prefix keys (all visible) and suffix keys (visible where mask), one
    softmax over the union, scale dh^-1/2; query head a reads kv head a // group.

    q [S,Hq,dh]; k_prefix,v_prefix [P,Hkv,dh]; k_suffix,v_suffix [S,Hkv,dh]; returns [S,Hq,dh]."""
    S, Hq, dh = q.shape
    P = k_prefix.shape[0]
    out = np.zeros((S, Hq, dh), dtype=F64)
    inv_sqrt = 1.0 / math.sqrt(dh)
    for a in range(Hq):
        b = a // group
        logits_p = (q[:, a, :] @ k_prefix[:P, b, :].T) * inv_sqrt          # [S,P]
        logits_s = (q[:, a, :] @ k_suffix[:, b, :].T) * inv_sqrt           # [S,S]
        logits_s = np.where(mask, logits_s, -np.inf)
        logits = np.concatenate([logits_p, logits_s], axis=1)
        logits = logits - logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, a, :] = p[:, :P] @ v_prefix[:P, b, :] + p[:, P:] @ v_suffix[:, b, :]
    return out


# ----------------------------------------------------------------------------------------------
# the loop
# ----------------------------------------------------------------------------------------------
class Weights:
    """Float64 view of a weight dictionary (names as in the C-ABI weight struct, per-layer
    tensors suffixed ``.{layer}``)."""

    def __init__(self, W: Dict[str, object]):
        self._w = {k: to_f64(v) for k, v in W.items()}

    def __getitem__(self, name: str) -> np.ndarray:
        return self._w[name]

    def layer(self, name: str, l: int) -> np.ndarray:
        return self._w[f"{name}.{l}"]


def embed_suffix(cfg, W: Weights, x: np.ndarray, state: Optional[np.ndarray], tau: np.ndarray):
    """Suffix tokens h in R^{S x D} and (pi0.5 only) the conditioning vector c.

    pi0: h[0] = state Ws + bs; e_i = x_i Wa + ba; h[1+i] = swish([e_i ; tau] W1 + b1) W2 + b2.
    pi0.5: h[i] = x_i Wa + ba; c = swish(swish(tau W1 + b1) W2 + b2)."""
    e = x @ W["action_in_w"] + W["action_in_b"]
    if cfg.cond == "pi0":
        cat = np.concatenate([e, np.broadcast_to(tau, e.shape)], axis=1)
        tok = swish(cat @ W["time_mlp1_w"] + W["time_mlp1_b"]) @ W["time_mlp2_w"] + W["time_mlp2_b"]
        cvec = None
    else:
        tok = e
        cvec = swish(swish(tau @ W["time_mlp1_w"] + W["time_mlp1_b"]) @ W["time_mlp2_w"] + W["time_mlp2_b"])
    if cfg.has_state_token:
        s_tok = state @ W["state_w"] + W["state_b"]
        tok = np.concatenate([s_tok[None, :], tok], axis=0)
    return tok, cvec


def velocity(cfg, W: Weights, prefix_kv: np.ndarray, prefix_len: int, state, x: np.ndarray,
             t: float, mask: Optional[np.ndarray] = None) -> np.ndarray:
    """v(x, t): one forward of the action expert over the suffix tokens."""
    D, Hq, Hkv, dh = cfg.width, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    ns = 1 if cfg.has_state_token else 0
    S = cfg.horizon + ns
    P = int(prefix_len)
    ada = cfg.cond == "pi05"
    if mask is None:
        mask = suffix_visibility(cfg)

    tau = sinusoid(t, D, cfg.time_min_period, cfg.time_max_period)
    h, c = embed_suffix(cfg, W, x, state, tau)
    pos = P + np.arange(S)

    for l in range(cfg.n_layers):
        # norm -> fused QKV
        if ada:
            n1, g1 = norm_ada(h, c, W.layer("norm1", l), W.layer("norm1_b", l), cfg.rms_eps)
        else:
            n1, g1 = norm_plain(h, W.layer("norm1", l), cfg.rms_eps), 1.0
        q = project(cfg, n1, W.layer("wq", l)).reshape(S, Hq, dh)
        ks = project(cfg, n1, W.layer("wk", l)).reshape(S, Hkv, dh)
        vs = project(cfg, n1, W.layer("wv", l)).reshape(S, Hkv, dh)
        q = rope(q, pos, cfg.rope_theta)
        ks = rope(ks, pos, cfg.rope_theta)
        # attention over prefix (as given, K already rotated) and suffix
        o = attention(q, prefix_kv[l, 0, :P], prefix_kv[l, 1, :P], ks, vs, mask, Hq // Hkv)
        h = h + g1 * project(cfg, o.reshape(S, Hq * dh), W.layer("wo", l))
        # norm -> gate/up -> GeGLU -> down
        if ada:
            n2, g2 = norm_ada(h, c, W.layer("norm2", l), W.layer("norm2_b", l), cfg.rms_eps)
        else:
            n2, g2 = norm_plain(h, W.layer("norm2", l), cfg.rms_eps), 1.0
        m = gelu(project(cfg, n2, W.layer("wgate", l)), cfg.gelu_exact) * project(cfg, n2, W.layer("wup", l))
        h = h + g2 * project(cfg, m, W.layer("wdown", l))

    if ada:
        nf, _ = norm_ada(h, c, W["final_norm"], W["final_norm_b"], cfg.rms_eps)
    else:
        nf = norm_plain(h, W["final_norm"], cfg.rms_eps)
    return nf[ns:] @ W["action_out_w"] + W["action_out_b"]


def denoise(cfg, weights, prefix_kv, prefix_len: int, state, noise, n_steps: int,
            mask: Optional[np.ndarray] = None) -> np.ndarray:
    """x <- x + dt v(x, t_k) for k = 0..n-1, from x = noise at t = 1; returns x at t = 0.

    ``weights``: dict of stored tensors or a ``Weights``; ``prefix_kv`` [L,2,>=P,Hkv,dh];
    ``state`` [Ds] or None; ``noise`` [H,A]."""
    W = weights if isinstance(weights, Weights) else Weights(weights)
    kv = to_f64(prefix_kv)
    st = None if state is None else to_f64(state)
    x = to_f64(noise).copy()
    dt, ts = time_grid(n_steps)
    for t in ts:
        v = velocity(cfg, W, kv, prefix_len, st, x, t, mask)
        x = x + dt * v
    return x


def denoise_batched(cfg, weights, prefix_kv_packed, cu_prefix_lens, states, noise, n_steps: int):
    """Batched = the same loop independently per request; ``prefix_kv_packed`` is
    [L,2,P_total,Hkv,dh] with request b occupying rows cu[b]:cu[b+1]."""
    W = weights if isinstance(weights, Weights) else Weights(weights)
    outs = []
    for b in range(len(cu_prefix_lens) - 1):
        lo, hi = int(cu_prefix_lens[b]), int(cu_prefix_lens[b + 1])
        st = None if states is None else states[b]
        outs.append(denoise(cfg, W, prefix_kv_packed[:, :, lo:hi], hi - lo, st, noise[b], n_steps))
    return np.stack(outs)


def max_rel_err(got, ref) -> float:
    """Error metric of the parity bar: ||got - ref||_inf / ||ref||_inf over one action chunk."""
    got = np.asarray(got, dtype=F64)
    ref = np.asarray(ref, dtype=F64)
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))
