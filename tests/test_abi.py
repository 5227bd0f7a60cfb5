"""The C-ABI library builds, loads, and exports every function include/mlora.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2604_18655_b200 import build
    return build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mlora.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mlora_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_main_calls():
    names = declared_functions()
    for f in ("mlora_create", "mlora_set_adapter", "mlora_prefill_shared", "mlora_decode_step", "mlora_verify_tree"):
        assert f in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} declared in mlora.h but not exported"


def test_binding_covers_every_declared_symbol(libpath):
    from paper_2604_18655_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()
    binding.lib()


def test_host_side_argument_errors_need_no_gpu(libpath):
    from paper_2604_18655_b200 import binding as mb
    L = mb.lib()
    assert L.mlora_create(None, None) == -1
    assert b"null" in L.mlora_last_error(None)
    assert L.mlora_decode_step(None, 1, None, None, None, None) == -1
    assert L.mlora_destroy(None) == 0
    assert L.mlora_linear_workspace_bytes(None, 8, 16) == 0
    assert L.mlora_attention_workspace_bytes(8, 1, 32, 8, 128, 512, 65) > 0


def test_unsupported_rope_style_is_refused_on_the_host(libpath):
    """rope_style other than 0 (half-split pairs) is rejected before anything touches a device."""
    from paper_2604_18655_b200 import binding as mb
    L = mb.lib()
    d = mb.ModelDesc()
    d.n_layers, d.d_model, d.n_q_heads, d.n_kv_heads, d.head_dim, d.d_ffn = 1, 64, 1, 1, 64, 64
    d.group_size, d.max_tree, d.max_streams, d.max_prefix, d.max_suffix = 64, 1, 1, 1, 1
    arr = (ctypes.c_void_p * 8)(*([1] * 8))
    d.qweight, d.scales, d.rms_attn, d.rms_ffn = arr, arr, arr, arr
    d.rope_style = 1
    out = ctypes.c_void_p()
    assert L.mlora_create(ctypes.byref(d), ctypes.byref(out)) == -6
    assert b"rope_style" in L.mlora_last_error(None)
