"""Thin ctypes binding of the C-ABI library (``include/phyai.h``): argument marshalling only.

Every step of the denoising loop runs inside the CUDA library; PyTorch is used here for device
memory and streams.  There is no CPU fallback: loading fails loudly when ``libphyai.so`` has not
been built, and every compute call fails without a CUDA device.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libphyai.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_OOM, ERR_CUDA, ERR_TIMEOUT = range(6)
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "OOM", 4: "CUDA", 5: "TIMEOUT"}
DTYPES = {"f32": 0, "bf16": 1, "w8e4m3": 2, "w8a8e4m3": 3, "w4a16": 4}
CONDS = {"pi0": 0, "pi05": 1}
ENGINES = {"auto": 0, "simt": 1}
BIG = ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown")

#: every symbol the header declares
EXPORTS = ("phyai_expert_create", "phyai_expert_destroy", "phyai_prefix_kv_bytes", "phyai_denoise",
           "phyai_denoise_batched", "phyai_denoise_host", "phyai_denoise_batched_host", "phyai_poll_status",
           "phyai_set_option", "phyai_launches_per_call", "phyai_last_error", "phyai_version",
           "phyai_suffix_attention", "phyai_suffix_attention_scratch_bytes", "phyai_op_last_error",
           "phyai_suffix_attention_static", "phyai_suffix_attention_static_capacity", "phyai_read_trace",
           "phyai_pack_prefix_kv", "phyai_postprocess_actions", "phyai_adapter_last_error", "phyai_batcher_create",
           "phyai_batcher_destroy", "phyai_batcher_submit", "phyai_batcher_next", "phyai_batcher_pending",
           "phyai_batcher_plan", "phyai_w8a8_project", "phyai_w8a8_last_error", "phyai_project_features_kv", "phyai_kv_projector_create",
           "phyai_kv_projector_run", "phyai_kv_projector_destroy")


class PhyaiError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"phyai status {STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class ConfigStruct(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in
                ("struct_size", "n_layers", "width", "mlp_dim", "n_q_heads", "n_kv_heads", "head_dim", "state_dim",
                 "action_dim", "horizon", "has_state_token", "max_prefix_len", "max_batch", "cond", "dtype")] + \
               [(n, C.c_float) for n in ("rms_eps", "rope_theta", "time_min_period", "time_max_period")] + \
               [(n, C.c_uint32) for n in ("gelu_exact", "suffix_block_causal", "engine")]


_VP = C.c_void_p
_VPP = C.POINTER(C.c_void_p)


class AttentionDesc(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("struct_size", "n_q_heads", "n_kv_heads", "head_dim", "suffix_len",
                                          "n_layers", "layer", "state_token_block_causal", "num_splits")]


class KvPackDesc(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("struct_size", "n_layers", "n_kv_heads", "head_dim", "elem_bytes", "batch",
                                          "p_max")]


class BatcherConfig(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("struct_size", "max_batch", "n_workers", "local_batch")] + [("window_ms", C.c_double)]


class WeightsStruct(C.Structure):
    _fields_ = [(n, _VP) for n in
                ("state_w", "state_b", "action_in_w", "action_in_b", "time_mlp1_w", "time_mlp1_b", "time_mlp2_w",
                 "time_mlp2_b", "action_out_w", "action_out_b", "final_norm", "final_norm_b")] + \
               [(n, _VPP) for n in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown",
                                    "norm1", "norm1_b", "norm2", "norm2_b")] + \
               [("scales", _VPP * 7)]


_lib = None


def load_library() -> C.CDLL:
    """Load ``libphyai.so`` (built by ``paper_2608_03682_b200.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_03682_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    lib.phyai_last_error.restype = C.c_char_p
    lib.phyai_version.restype = C.c_char_p
    lib.phyai_prefix_kv_bytes.restype = C.c_size_t
    lib.phyai_prefix_kv_bytes.argtypes = [C.POINTER(ConfigStruct), C.c_uint64]
    lib.phyai_expert_create.argtypes = [C.POINTER(ConfigStruct), C.POINTER(WeightsStruct), _VP, C.POINTER(_VP)]
    lib.phyai_expert_destroy.argtypes = [_VP]
    lib.phyai_expert_destroy.restype = None
    single = [_VP, _VP, C.c_uint64, C.c_uint32, _VP, _VP, C.c_uint32, _VP, _VP]
    batched = [_VP, C.c_uint32, _VP, C.c_uint64, _VP, _VP, _VP, C.c_uint32, _VP, _VP]
    lib.phyai_denoise.argtypes = single
    lib.phyai_denoise_host.argtypes = single
    lib.phyai_denoise_batched.argtypes = batched
    lib.phyai_denoise_batched_host.argtypes = batched
    lib.phyai_poll_status.argtypes = [_VP]
    lib.phyai_set_option.argtypes = [_VP, C.c_char_p, C.c_int64]
    lib.phyai_read_trace.argtypes = [_VP, _VP, C.c_size_t, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
    lib.phyai_launches_per_call.argtypes = [_VP, C.c_uint32, C.c_uint32]
    lib.phyai_launches_per_call.restype = C.c_uint64
    lib.phyai_op_last_error.restype = C.c_char_p
    lib.phyai_suffix_attention_scratch_bytes.restype = C.c_size_t
    lib.phyai_suffix_attention_scratch_bytes.argtypes = [C.POINTER(AttentionDesc), C.c_uint32]
    lib.phyai_suffix_attention.argtypes = [C.POINTER(AttentionDesc), C.c_uint32, _VP, _VP, C.c_uint64, _VP, _VP, _VP,
                                           _VP, _VP]
    lib.phyai_suffix_attention_static.argtypes = lib.phyai_suffix_attention.argtypes
    lib.phyai_suffix_attention_static_capacity.restype = C.c_size_t
    lib.phyai_pack_prefix_kv.argtypes = [C.POINTER(KvPackDesc), _VP, _VP, _VP, _VP, C.c_uint64, _VP, _VP, _VP]
    lib.phyai_postprocess_actions.argtypes = [_VP, C.c_uint32, C.c_uint32, C.c_uint32, _VP, _VP, C.c_float, C.c_float,
                                              C.c_uint32, C.c_uint32, _VP, _VP]
    lib.phyai_adapter_last_error.restype = C.c_char_p
    lib.phyai_w8a8_project.argtypes = [_VP, _VP, _VP, C.c_uint32, C.c_uint32, C.c_uint32, _VP, _VP, _VP, _VP]
    lib.phyai_w8a8_last_error.restype = C.c_char_p
    lib.phyai_project_features_kv.argtypes = [_VP, _VP, _VP, _VP, C.c_uint64, C.c_uint64, _VP, _VP]
    lib.phyai_kv_projector_create.argtypes = [_VP, _VP, _VP, C.c_uint64, _VP, C.POINTER(_VP)]
    lib.phyai_kv_projector_run.argtypes = [_VP, _VP, C.c_uint64, C.c_uint64, _VP, _VP]
    lib.phyai_kv_projector_destroy.argtypes = [_VP]
    lib.phyai_kv_projector_destroy.restype = None
    lib.phyai_batcher_create.argtypes = [C.POINTER(BatcherConfig), C.POINTER(_VP)]
    lib.phyai_batcher_destroy.argtypes = [_VP]
    lib.phyai_batcher_destroy.restype = None
    lib.phyai_batcher_submit.argtypes = [_VP, C.c_uint64]
    lib.phyai_batcher_next.argtypes = [_VP, C.c_double, C.POINTER(C.c_uint64), C.POINTER(C.c_uint32)]
    lib.phyai_batcher_pending.argtypes = [_VP]
    lib.phyai_batcher_pending.restype = C.c_uint32
    lib.phyai_batcher_plan.argtypes = [C.POINTER(BatcherConfig), C.c_uint32, C.POINTER(C.c_int32), C.POINTER(C.c_uint32)]
    _lib = lib
    return lib


def _check(status: int):
    if status != OK:
        raise PhyaiError(status, load_library().phyai_last_error().decode())


def make_config_struct(cfg, engine: str = "auto") -> ConfigStruct:
    s = ConfigStruct()
    s.struct_size = C.sizeof(ConfigStruct)
    for n in ("n_layers", "width", "mlp_dim", "n_q_heads", "n_kv_heads", "head_dim", "state_dim", "action_dim",
              "horizon", "max_prefix_len", "max_batch"):
        setattr(s, n, int(getattr(cfg, n)))
    s.has_state_token = int(bool(cfg.has_state_token))
    s.cond = CONDS[cfg.cond]
    s.dtype = DTYPES[cfg.dtype]
    s.rms_eps, s.rope_theta = cfg.rms_eps, cfg.rope_theta
    s.time_min_period, s.time_max_period = cfg.time_min_period, cfg.time_max_period
    s.gelu_exact = int(bool(cfg.gelu_exact))
    s.suffix_block_causal = int(bool(cfg.suffix_block_causal))
    s.engine = ENGINES[engine]
    return s


def prefix_kv_bytes(cfg, tokens: int) -> int:
    s = make_config_struct(cfg)
    return int(load_library().phyai_prefix_kv_bytes(C.byref(s), tokens))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


class Expert:
    """One action expert on the current CUDA device.  ``weights``: name -> CUDA tensor (per-layer
    names suffixed ``.{layer}``); for the e4m3 mode the seven big matrices are ``(codes, scales)``."""

    def __init__(self, cfg, weights: Dict[str, object], engine: str = "auto", stream=None):
        self.lib = load_library()
        self.cfg = cfg
        self._handle = _VP()
        cs = make_config_struct(cfg, engine)
        ws = WeightsStruct()
        keep = []
        L = cfg.n_layers

        def dev(t):
            if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
                raise ValueError("weights must be contiguous CUDA tensors")
            keep.append(t)
            return t.data_ptr()

        for n in ("state_w", "state_b", "action_in_w", "action_in_b", "time_mlp1_w", "time_mlp1_b", "time_mlp2_w",
                  "time_mlp2_b", "action_out_w", "action_out_b", "final_norm", "final_norm_b"):
            if n in weights:
                setattr(ws, n, dev(weights[n]))
        scale_arrays = {m: (C.c_void_p * L)() for m in BIG}
        for n in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "norm1", "norm1_b", "norm2", "norm2_b"):
            if f"{n}.0" not in weights:
                continue
            arr = (C.c_void_p * L)()
            for l in range(L):
                w = weights[f"{n}.{l}"]
                if isinstance(w, tuple):
                    arr[l] = dev(w[0])
                    scale_arrays[n][l] = dev(w[1])
                else:
                    arr[l] = dev(w)
            keep.append(arr)
            setattr(ws, n, C.cast(arr, _VPP))
        if cfg.dtype in ("w8e4m3", "w8a8e4m3", "w4a16"):
            for i, m in enumerate(BIG):
                keep.append(scale_arrays[m])
                ws.scales[i] = C.cast(scale_arrays[m], _VPP)
        _check(self.lib.phyai_expert_create(C.byref(cs), C.byref(ws), _stream_ptr(stream), C.byref(self._handle)))
        del keep  # create has repacked everything and synchronised

    # ------------------------------------------------------------------------------------------
    def close(self):
        if getattr(self, "_handle", None) is not None and self._handle.value:
            self.lib.phyai_expert_destroy(self._handle)
            self._handle = _VP()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # ------------------------------------------------------------------------------------------
    def denoise(self, prefix_kv: torch.Tensor, prefix_len: int, state: Optional[torch.Tensor], noise: torch.Tensor,
                n_steps: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """phyai_denoise: device tensors; ``prefix_kv`` [L,2,T,Hkv,dh]; returns ``out`` [H,A] (enqueued only)."""
        if out is None:
            out = torch.empty_like(noise)
        kv_tokens = 0 if prefix_kv is None else int(prefix_kv.shape[2])
        _check(self.lib.phyai_denoise(self._handle, _ptr(prefix_kv), kv_tokens, int(prefix_len), _ptr(state),
                                      _ptr(noise), int(n_steps), _ptr(out), _stream_ptr(stream)))
        return out

    def denoise_batched(self, prefix_kv: torch.Tensor, cu_prefix_lens: torch.Tensor, states: Optional[torch.Tensor],
                        noise: torch.Tensor, n_steps: int, out: Optional[torch.Tensor] = None,
                        stream=None) -> torch.Tensor:
        """phyai_denoise_batched: packed ``prefix_kv`` [L,2,T_total,Hkv,dh], device int32 ``cu_prefix_lens`` [B+1]."""
        if out is None:
            out = torch.empty_like(noise)
        batch = int(noise.shape[0])
        _check(self.lib.phyai_denoise_batched(self._handle, batch, _ptr(prefix_kv), int(prefix_kv.shape[2]),
                                              _ptr(cu_prefix_lens), _ptr(states), _ptr(noise), int(n_steps), _ptr(out),
                                              _stream_ptr(stream)))
        return out

    def denoise_host(self, prefix_kv: torch.Tensor, prefix_len: int, state, noise, n_steps: int, out: torch.Tensor,
                     stream=None) -> torch.Tensor:
        """phyai_denoise_host: all tensors are (ideally pinned) host tensors."""
        _check(self.lib.phyai_denoise_host(self._handle, _ptr(prefix_kv), int(prefix_kv.shape[2]), int(prefix_len),
                                           _ptr(state), _ptr(noise), int(n_steps), _ptr(out), _stream_ptr(stream)))
        return out

    def denoise_batched_host(self, prefix_kv, cu_prefix_lens, states, noise, n_steps: int, out, stream=None):
        batch = int(noise.shape[0])
        _check(self.lib.phyai_denoise_batched_host(self._handle, batch, _ptr(prefix_kv), int(prefix_kv.shape[2]),
                                                   _ptr(cu_prefix_lens), _ptr(states), _ptr(noise), int(n_steps),
                                                   _ptr(out), _stream_ptr(stream)))
        return out

    def poll_status(self) -> int:
        """Read-and-clear the device status word (call after synchronising); returns the status code."""
        return int(self.lib.phyai_poll_status(self._handle))

    def set_option(self, key: str, value: int):
        _check(self.lib.phyai_set_option(self._handle, key.encode(), int(value)))

    def read_trace(self) -> np.ndarray:
        """Timer stamps (ns) of the traced launches of the last call: array [slots, 16] (option "trace" = 1)."""
        buf = np.zeros(4096 * 16, dtype=np.uint64)
        n_slots, n_st = C.c_uint32(), C.c_uint32()
        _check(self.lib.phyai_read_trace(self._handle, buf.ctypes.data_as(_VP), buf.size, C.byref(n_slots),
                                         C.byref(n_st)))
        return buf.reshape(n_slots.value, n_st.value)

    def launches_per_call(self, batch: int, n_steps: int) -> int:
        return int(self.lib.phyai_launches_per_call(self._handle, batch, n_steps))


def weights_to_device(weights: Dict[str, object], device="cuda") -> Dict[str, object]:
    """Copy a generated weight dictionary to the device (tuples element-wise)."""
    out = {}
    for k, v in weights.items():
        if isinstance(v, tuple):   # (codes, scales) or (packed codes, scales, format tag)
            out[k] = tuple(t.to(device).contiguous() if hasattr(t, "to") else t for t in v)
        else:
            out[k] = v.to(device).contiguous()
    return out


def attention_desc(n_q_heads, n_kv_heads, head_dim, suffix_len, n_layers, layer, block_causal=False, num_splits=0):
    d = AttentionDesc()
    d.struct_size = C.sizeof(AttentionDesc)
    d.n_q_heads, d.n_kv_heads, d.head_dim, d.suffix_len = n_q_heads, n_kv_heads, head_dim, suffix_len
    d.n_layers, d.layer, d.state_token_block_causal, d.num_splits = n_layers, layer, int(block_causal), num_splits
    return d


def suffix_attention(desc: AttentionDesc, qkv: torch.Tensor, prefix_kv: torch.Tensor, cu_prefix_lens: torch.Tensor,
                     rope_cos_sin: Optional[torch.Tensor], entry: str = "phyai_suffix_attention", stream=None):
    """Stand-alone attention operator; returns (out bf16 [rows, Hq*dh], status_word int32 tensor)."""
    lib = load_library()
    batch = int(cu_prefix_lens.numel()) - 1
    rows = batch * desc.suffix_len
    out = torch.empty(rows, desc.n_q_heads * desc.head_dim, dtype=torch.bfloat16, device=qkv.device)
    status = torch.zeros(1, dtype=torch.int32, device=qkv.device)
    st = getattr(lib, entry)(C.byref(desc), batch, _ptr(qkv), _ptr(prefix_kv), int(prefix_kv.shape[2]),
                             _ptr(cu_prefix_lens), _ptr(rope_cos_sin), _ptr(out), _ptr(status), _stream_ptr(stream))
    if st != OK:
        raise PhyaiError(st, lib.phyai_op_last_error().decode())
    return out, status


def pack_prefix_kv(k: torch.Tensor, v: torch.Tensor, lens: torch.Tensor, kv_tokens: Optional[int] = None, stream=None):
    """Padded backbone K / V ``[L, B, p_max, Hkv, dh]`` + ``lens`` (int32 ``[B]``, device) -> the library's ragged
    layout.  Returns (prefix_kv ``[L, 2, kv_tokens, Hkv, dh]``, cu_prefix_lens int32 ``[B + 1]``, status word)."""
    lib = load_library()
    L, B, p_max, Hkv, dh = k.shape
    if kv_tokens is None:
        kv_tokens = B * p_max
    desc = KvPackDesc()
    desc.struct_size = C.sizeof(KvPackDesc)
    desc.n_layers, desc.n_kv_heads, desc.head_dim, desc.elem_bytes, desc.batch, desc.p_max = L, Hkv, dh, k.element_size(), B, p_max
    out = torch.zeros(L, 2, kv_tokens, Hkv, dh, dtype=k.dtype, device=k.device)
    cu = torch.empty(B + 1, dtype=torch.int32, device=k.device)
    status = torch.zeros(1, dtype=torch.int32, device=k.device)
    st = lib.phyai_pack_prefix_kv(C.byref(desc), _ptr(k), _ptr(v), _ptr(lens), _ptr(out), int(kv_tokens), _ptr(cu), _ptr(status),
                                  _stream_ptr(stream))
    if st != OK:
        raise PhyaiError(st, lib.phyai_adapter_last_error().decode())
    return out, cu, status


def postprocess_actions(x: torch.Tensor, q01: Optional[torch.Tensor], q99: Optional[torch.Tensor], clip=(-1.0, 1.0),
                        out_horizon: Optional[int] = None, out_dim: Optional[int] = None, stream=None) -> torch.Tensor:
    """Raw chunk ``[B, H, A]`` -> clipped, un-normalised actions ``[B, out_horizon, out_dim]``."""
    lib = load_library()
    B, H, A = x.shape
    out_horizon, out_dim = out_horizon or H, out_dim or A
    out = torch.empty(B, out_horizon, out_dim, dtype=torch.float32, device=x.device)
    lo, hi = (clip if clip is not None else (0.0, 0.0))
    st = lib.phyai_postprocess_actions(_ptr(x), B, H, A, _ptr(q01), _ptr(q99), float(lo), float(hi), out_horizon, out_dim,
                                       _ptr(out), _stream_ptr(stream))
    if st != OK:
        raise PhyaiError(st, lib.phyai_adapter_last_error().decode())
    return out


class KvProjDesc(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers", C.c_uint32), ("n_kv_heads", C.c_uint32), ("head_dim", C.c_uint32),
                ("feat_dim", C.c_uint32)]


def project_features_kv(features: torch.Tensor, wk, wv, n_kv_heads: int, head_dim: int, kv_tokens: Optional[int] = None,
                        stream=None) -> torch.Tensor:
    """Request-local K / V projections of a feature-handoff head (``phyai_project_features_kv``): ``features`` bf16
    ``[tokens, Dv]``, ``wk`` / ``wv`` lists of bf16 ``[Dv, Hkv * dh]`` -> prefix KV bf16 ``[L, 2, kv_tokens, Hkv, dh]``."""
    lib = load_library()
    tokens, Dv = features.shape
    L = len(wk)
    kv_tokens = kv_tokens or tokens
    out = torch.zeros(L, 2, kv_tokens, n_kv_heads, head_dim, dtype=torch.bfloat16, device=features.device)
    desc = KvProjDesc(C.sizeof(KvProjDesc), L, n_kv_heads, head_dim, Dv)
    ak, av = (_VP * L)(), (_VP * L)()
    for l in range(L):
        ak[l], av[l] = wk[l].data_ptr(), wv[l].data_ptr()
    st = lib.phyai_project_features_kv(C.byref(desc), _ptr(features), C.cast(ak, _VP), C.cast(av, _VP), tokens, kv_tokens,
                                       _ptr(out), _stream_ptr(stream))
    if st != OK:
        raise PhyaiError(st, lib.phyai_adapter_last_error().decode())
    return out


class KvProjector:
    """Handle form of the feature K / V projection (``phyai_kv_projector_*``): weights packed once, ``run`` only enqueues."""

    def __init__(self, wk, wv, n_kv_heads: int, head_dim: int, max_tokens: int, stream=None):
        self.lib = load_library()
        self.L, self.n_kv_heads, self.head_dim = len(wk), n_kv_heads, head_dim
        desc = KvProjDesc(C.sizeof(KvProjDesc), self.L, n_kv_heads, head_dim, wk[0].shape[0])
        ak, av = (_VP * self.L)(), (_VP * self.L)()
        for l in range(self.L):
            ak[l], av[l] = wk[l].data_ptr(), wv[l].data_ptr()
        self._h = _VP()
        st = self.lib.phyai_kv_projector_create(C.byref(desc), C.cast(ak, _VP), C.cast(av, _VP), max_tokens,
                                                _stream_ptr(stream), C.byref(self._h))
        if st != OK:
            raise PhyaiError(st, self.lib.phyai_adapter_last_error().decode())

    def run(self, features: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        tokens = features.shape[0]
        if out is None:
            out = torch.zeros(self.L, 2, tokens, self.n_kv_heads, self.head_dim, dtype=torch.bfloat16, device=features.device)
        st = self.lib.phyai_kv_projector_run(self._h, _ptr(features), tokens, out.shape[2], _ptr(out), _stream_ptr(stream))
        if st != OK:
            raise PhyaiError(st, self.lib.phyai_adapter_last_error().decode())
        return out

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.phyai_kv_projector_destroy(self._h)
            self._h = _VP()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def w8a8_project(x: torch.Tensor, w_codes: torch.Tensor, w_scales: torch.Tensor, return_codes: bool = False, stream=None):
    """Stand-alone W8A8 projection (``phyai_w8a8_project``): ``x`` bf16 ``[M, K]``, ``w_codes`` uint8 ``[K, N]``,
    ``w_scales`` float32 ``[N]`` -> float32 ``[M, N]`` (and, on request, the activation codes and scales)."""
    lib = load_library()
    M, K = x.shape
    N = w_codes.shape[1]
    y = torch.empty(M, N, dtype=torch.float32, device=x.device)
    codes = torch.empty(M, K, dtype=torch.uint8, device=x.device) if return_codes else None
    scales = torch.empty(M, dtype=torch.float32, device=x.device) if return_codes else None
    st = lib.phyai_w8a8_project(_ptr(x), _ptr(w_codes), _ptr(w_scales), M, K, N, _ptr(y), _ptr(codes), _ptr(scales),
                                _stream_ptr(stream))
    if st != OK:
        raise PhyaiError(st, lib.phyai_w8a8_last_error().decode())
    return (y, codes, scales) if return_codes else y


class Batcher:
    """Batching window of the data-parallel front-end (``phyai_batcher_*``): thread-safe queue; ``next`` returns the ids
    of the batch that is due (possibly empty after ``timeout_ms``)."""

    def __init__(self, max_batch: int, n_workers: int, local_batch: int, window_ms: float):
        self.lib = load_library()
        self.cfg = BatcherConfig(C.sizeof(BatcherConfig), max_batch, n_workers, local_batch, float(window_ms))
        h = _VP()
        st = self.lib.phyai_batcher_create(C.byref(self.cfg), C.byref(h))
        if st != OK:
            raise PhyaiError(st, "bad batcher configuration")
        self._h = h

    def submit(self, request_id: int):
        self.lib.phyai_batcher_submit(self._h, int(request_id))

    def pending(self) -> int:
        return int(self.lib.phyai_batcher_pending(self._h))

    def next(self, timeout_ms: float):
        ids = (C.c_uint64 * self.cfg.max_batch)()
        n = C.c_uint32()
        st = self.lib.phyai_batcher_next(self._h, float(timeout_ms), ids, C.byref(n))
        if st != OK:
            raise PhyaiError(st, "phyai_batcher_next failed")
        return [int(ids[i]) for i in range(n.value)]

    def plan(self, n: int):
        """(slots as a list of n_workers lists of local_batch indices, -1 = padding; number of workers with a request)"""
        total = self.cfg.n_workers * self.cfg.local_batch
        slots = (C.c_int32 * total)()
        act = C.c_uint32()
        st = self.lib.phyai_batcher_plan(C.byref(self.cfg), int(n), slots, C.byref(act))
        if st != OK:
            raise PhyaiError(st, "phyai_batcher_plan: n exceeds max_batch")
        L = self.cfg.local_batch
        return [[int(slots[w * L + j]) for j in range(L)] for w in range(self.cfg.n_workers)], int(act.value)

    def close(self):
        if self._h:
            self.lib.phyai_batcher_destroy(self._h)
            self._h = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()
