"""The C-ABI library builds, loads and exports every symbol the header declares; host-side
argument checks return status codes.  No GPU compute here."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2608_03682_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "phyai.h")).read()
    declared = set(re.findall(r"\b(phyai_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert b"sm_100a" in lib.phyai_version()


def test_config_struct_matches_header_size(lib):
    cfg = synth.tiny_config()
    s = binding.make_config_struct(cfg)
    assert s.struct_size == 22 * 4
    assert lib.phyai_prefix_kv_bytes(C.byref(s), 64) == 2 * 2 * 64 * 1 * 64 * 4
    s2 = binding.make_config_struct(synth.pi0_config())
    assert lib.phyai_prefix_kv_bytes(C.byref(s2), 816) == 18 * 2 * 816 * 256 * 2


def test_create_rejects_bad_arguments_without_touching_the_gpu(lib):
    handle = C.c_void_p()
    ws = binding.WeightsStruct()
    s = binding.make_config_struct(synth.tiny_config())
    assert lib.phyai_expert_create(None, C.byref(ws), None, C.byref(handle)) == binding.ERR_INVALID_ARG
    assert b"config" in lib.phyai_last_error()
    s.struct_size = 12
    assert lib.phyai_expert_create(C.byref(s), C.byref(ws), None, C.byref(handle)) == binding.ERR_INVALID_ARG
    s = binding.make_config_struct(synth.tiny_config())
    s.n_q_heads, s.n_kv_heads = 3, 2
    assert lib.phyai_expert_create(C.byref(s), C.byref(ws), None, C.byref(handle)) == binding.ERR_INVALID_ARG
    s = binding.make_config_struct(synth.tiny_config())
    s.head_dim = 512
    assert lib.phyai_expert_create(C.byref(s), C.byref(ws), None, C.byref(handle)) == binding.ERR_UNSUPPORTED
    assert handle.value is None
    assert lib.phyai_denoise(None, None, 0, 0, None, None, 1, None, None) == binding.ERR_INVALID_ARG
    assert lib.phyai_poll_status(None) == binding.ERR_INVALID_ARG
    assert lib.phyai_set_option(None, b"use_graph", 1) == binding.ERR_INVALID_ARG
    assert lib.phyai_launches_per_call(None, 1, 1) == 0
    lib.phyai_expert_destroy(None)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device failure")
def test_without_a_cuda_device_create_fails_loudly(lib):
    """No CPU fallback: with valid-looking arguments but no device, create reports a CUDA error."""
    handle = C.c_void_p()
    s = binding.make_config_struct(synth.tiny_config())
    ws = binding.WeightsStruct()
    st = lib.phyai_expert_create(C.byref(s), C.byref(ws), None, C.byref(handle))
    assert st == binding.ERR_CUDA and b"no CPU fallback" in lib.phyai_last_error()
