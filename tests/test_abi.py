"""The C-ABI library builds, loads without a GPU and exports what include/ssd.h declares.
Only host-side argument handling is exercised here (no kernel is launched)."""
import ctypes
import os
import re

import pytest

from paper_2505_15380_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build_library()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "ssd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ssd_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert "ssd_verify" in names and "ssd_draft_step" in names and "ssd_kv_commit" in names
    for n in names:
        assert hasattr(L, n), f"{n} declared in ssd.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_size_queries_follow_the_shape_arithmetic(L):
    cfg = binding.make_config(synth.workload(1).target)
    arena = L.ssd_model_arena_bytes(ctypes.byref(cfg))
    streamed = synth.workload(1).target.streamed_weight_bytes()
    embed = (6564 + 32768) * 896 * 2
    # a bf16 model is held three times: row-major for the generic kernels, packed in the operand
    # order of the warp-level instruction for the persistent small-batch kernel (plus its small
    # tables), and in 128-row tiles for the tcgen05 projections of batched forwards (whose last
    # tile of the LM head is padded)
    assert 3 * streamed + embed - (1 << 20) <= arena <= 3 * streamed + embed + (3 << 20)
    cfg0 = binding.make_config(synth.workload(0).target)           # fp32: one copy only
    arena0 = L.ssd_model_arena_bytes(ctypes.byref(cfg0))
    streamed0 = synth.workload(0).target.streamed_weight_bytes()
    assert streamed0 + 512 * 128 * 4 <= arena0 <= streamed0 + 512 * 128 * 4 + 64 * 256
    assert L.ssd_kv_bytes(ctypes.byref(cfg), 1, 512) == 12288 * 512
    assert L.ssd_workspace_bytes(ctypes.byref(cfg), 1, 4, 512) > 0
    assert L.ssd_workspace_bytes(ctypes.byref(cfg), 1, 16, 512) == 0      # gamma + 1 > 16 rows
    assert L.ssd_workspace_bytes(ctypes.byref(cfg), 1, 4, 3) == 0         # capacity < gamma + 1


@pytest.mark.parametrize("field,value", [("head_dim", 48), ("n_q_heads", 5), ("d_model", 100),
                                         ("weight_dtype", 2), ("qkv_bias", 0), ("vocab_out", 1),
                                         ("n_layers", 0), ("vocab_out", 60000)])
def test_bad_configs_are_rejected(L, field, value):
    cfg = binding.make_config(synth.workload(0).target)
    setattr(cfg, field, value)
    assert L.ssd_model_arena_bytes(ctypes.byref(cfg)) == 0
    h = ctypes.c_void_p()
    buf = ctypes.create_string_buffer(16)
    assert L.ssd_model_create(ctypes.byref(cfg), buf, 16, 256, 1 << 20, ctypes.byref(h)) == -2


def test_null_and_alignment_errors_without_touching_a_device(L):
    cfg = binding.make_config(synth.workload(0).target)
    h = ctypes.c_void_p()
    buf = ctypes.create_string_buffer(16)
    assert L.ssd_model_create(None, buf, 16, 256, 1 << 20, ctypes.byref(h)) == -1
    assert L.ssd_model_create(ctypes.byref(cfg), buf, 16, 257, 1 << 30, ctypes.byref(h)) == -5
    assert L.ssd_model_create(ctypes.byref(cfg), buf, 16, 256, 1024, ctypes.byref(h)) == -6
    assert L.ssd_model_create(ctypes.byref(cfg), buf, 16, 256, 1 << 30, ctypes.byref(h)) == -2
    assert L.ssd_verify(None, None, None, None, None, None, None, None, None, None) == -1
    assert L.ssd_draft_step(None, None, None, 1, None, None, None, None, None) == -1
    assert L.ssd_kv_commit(None, None, None, None) == -1
    assert L.ssd_streams_set_attention_kernel(None, 0) == -1 and L.ssd_streams_set_path(None, 0) == -1
    assert L.ssd_strerror(0) == b"ok" and b"gamma" in L.ssd_strerror(-3)
    assert L.ssd_strerror(-99) == b"unknown error"


def test_product_path_has_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    shape = synth.workload(0).target
    with pytest.raises(binding.SsdError, match="no CUDA device"):
        binding.Model(shape, synth.weights_blob(shape, synth.make_weights(shape, 0)))
