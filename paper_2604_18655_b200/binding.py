"""ctypes binding of include/mlora.h: same names, argument marshalling only.

Tensors are torch CUDA tensors (torch supplies device memory and the stream); pointers are passed with
``data_ptr()``.  There is no fallback: if ``libmlora.so`` is missing or a call fails, an exception is raised.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmlora.so")

MLORA_OK = 0
ERR_NAMES = {0: "OK", -1: "ERR_ARG", -2: "ERR_STATE", -3: "ERR_CAPACITY", -4: "ERR_CUDA", -5: "ERR_TIMEOUT",
             -6: "ERR_UNSUPPORTED"}
PROF_FAMILIES = ("gemm", "shrink", "attn", "attn_merge", "rope_kv", "misc")


class MloraError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


class ModelDesc(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32), ("group_size", C.c_int32),
        ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("rope_style", C.c_int32), ("lora_rank", C.c_int32), ("lora_targets", C.c_int32),
        ("max_adapters", C.c_int32), ("max_streams", C.c_int32), ("max_prefix", C.c_int32),
        ("max_suffix", C.c_int32), ("max_tree", C.c_int32),
        ("embed", C.c_void_p), ("qweight", C.POINTER(C.c_void_p)), ("scales", C.POINTER(C.c_void_p)),
        ("rms_attn", C.POINTER(C.c_void_p)), ("rms_ffn", C.POINTER(C.c_void_p)), ("rms_final", C.c_void_p),
        ("cuda_stream", C.c_void_p),
    ]


_lib = None

_SIGS = {
    "mlora_create": (C.c_int, [C.POINTER(ModelDesc), C.POINTER(C.c_void_p)]),
    "mlora_destroy": (C.c_int, [C.c_void_p]),
    "mlora_set_adapter": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_float]),
    "mlora_prefill_shared": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]),
    "mlora_prefill_shared_h": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]),
    "mlora_decode_step": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "mlora_decode_step_host": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "mlora_decode_step_h": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "mlora_verify_tree": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.c_void_p, C.c_void_p]),
    "mlora_reset_streams": (C.c_int, [C.c_void_p]),
    "mlora_sync_status": (C.c_int, [C.c_void_p]),
    "mlora_last_error": (C.c_char_p, [C.c_void_p]),
    "mlora_export_kv": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_int32),
                                  C.c_void_p, C.c_void_p]),
    "mlora_sample_first": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]),
    "mlora_generate": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]),
    "mlora_generate_host": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]),
    "mlora_set_forecast": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32]),
    "mlora_ds2d_round": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32] + [C.c_void_p] * 6 + [C.c_int32, C.c_int32] +
                         [C.c_void_p] * 5),
    "mlora_quantize_act_int8": (C.c_int, [C.c_void_p, C.c_int64, C.c_float, C.c_void_p, C.c_void_p]),
    "mlora_linear_w4a8": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                    C.c_void_p]),
    "mlora_export_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_int32), C.c_void_p, C.c_void_p]),
    "mlora_debug_dequant": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "mlora_debug_set": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32]),
    "mlora_profile_begin": (C.c_int, [C.c_void_p]),
    "mlora_profile_end": (C.c_int, [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int32)]),
    "mlora_launch_count": (C.c_int64, [C.c_void_p]),
    "mlora_step_timeline": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64), C.c_int32, C.POINTER(C.c_int32)]),
    "mlora_weight_create": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                      C.POINTER(C.c_void_p)]),
    "mlora_weight_destroy": (C.c_int, [C.c_void_p]),
    "mlora_weight_dequant": (C.c_int, [C.c_void_p, C.c_void_p]),
    "mlora_linear_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int32, C.c_int32]),
    "mlora_linear": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                               C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t]),
    "mlora_linear_noalloc": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_int32, C.c_int32, C.c_void_p]),
    "mlora_linear_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "mlora_attention_workspace_bytes": (C.c_size_t, [C.c_int32] * 7),
    "mlora_attention": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                  C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                  C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]),
}
EXPORTS = tuple(_SIGS)


def lib():
    """Loads libmlora.so (once).  Raises if it has not been built: there is no other implementation."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_18655_b200.build` "
                               "(or __graft_entry__.build()) first; there is no fallback path")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGS.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(code):
    if code != MLORA_OK:
        raise MloraError(code, lib().mlora_last_error(None).decode())


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr_array(tensors):
    arr = (C.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else t.data_ptr()
    return arr


# ----------------------------------------------------------------------------- context-level calls
def mlora_create(cfg, qweight, scales, rms_attn, rms_ffn, rms_final=None, embed=None, *, max_adapters=8,
                 max_streams=8, max_prefix=512, max_suffix=256, max_tree=1, lora_rank=None, lora_targets=None):
    """cfg: object with n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab, group_size,
    rope_theta, rms_eps, lora_rank, lora_targets.  Tensor lists are CUDA tensors in canonical format."""
    d = ModelDesc()
    for f in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "group_size"):
        setattr(d, f, int(getattr(cfg, f)))
    d.rope_theta, d.rms_eps = float(cfg.rope_theta), float(cfg.rms_eps)
    d.rope_style = int(getattr(cfg, "rope_style", 0))
    d.lora_rank = int(cfg.lora_rank if lora_rank is None else lora_rank)
    d.lora_targets = int(cfg.lora_targets if lora_targets is None else lora_targets)
    d.max_adapters, d.max_streams, d.max_prefix = max_adapters, max_streams, max_prefix
    d.max_suffix, d.max_tree = max_suffix, max_tree
    keep = (_ptr_array(qweight), _ptr_array(scales), _ptr_array(rms_attn), _ptr_array(rms_ffn))
    d.qweight, d.scales, d.rms_attn, d.rms_ffn = keep
    d.embed = None if embed is None else embed.data_ptr()
    d.rms_final = None if rms_final is None else rms_final.data_ptr()
    d.cuda_stream = torch.cuda.current_stream().cuda_stream
    out = C.c_void_p()
    _check(lib().mlora_create(C.byref(d), C.byref(out)))
    return out


def mlora_destroy(ctx):
    _check(lib().mlora_destroy(ctx))


def mlora_set_adapter(ctx, slot, A, B, alpha):
    if A is None:
        _check(lib().mlora_set_adapter(ctx, slot, None, None, 0.0))
    else:
        _check(lib().mlora_set_adapter(ctx, slot, _ptr_array(A), _ptr_array(B), float(alpha)))


def mlora_prefill_shared(ctx, prompt_ids, out_last_logits=None):
    _check(lib().mlora_prefill_shared(ctx, _ptr(prompt_ids), prompt_ids.numel(), _ptr(out_last_logits)))


def mlora_prefill_shared_h(ctx, hidden, out_last_hidden=None):
    _check(lib().mlora_prefill_shared_h(ctx, _ptr(hidden), hidden.shape[0], _ptr(out_last_hidden)))


def mlora_decode_step(ctx, adapter_idx, tokens, out_next, out_logits=None):
    _check(lib().mlora_decode_step(ctx, adapter_idx.numel(), _ptr(adapter_idx), _ptr(tokens), _ptr(out_next),
                                   _ptr(out_logits)))


def mlora_decode_step_host(ctx, adapter_idx, tokens, out_next):
    """Host-buffer form: the three arguments are CPU int32 tensors (pinned for asynchronous copies)."""
    for t in (adapter_idx, tokens, out_next):
        assert not t.is_cuda and t.is_contiguous() and t.dtype == torch.int32
    _check(lib().mlora_decode_step_host(ctx, adapter_idx.numel(), C.c_void_p(adapter_idx.data_ptr()),
                                        C.c_void_p(tokens.data_ptr()), C.c_void_p(out_next.data_ptr())))


def mlora_decode_step_h(ctx, adapter_idx, hidden_in, hidden_out):
    _check(lib().mlora_decode_step_h(ctx, adapter_idx.numel(), _ptr(adapter_idx), _ptr(hidden_in), _ptr(hidden_out)))


def mlora_verify_tree(ctx, adapter_idx, tree_tokens, tree_parent, out_accept_len, out_accept_idx, out_next,
                      out_logits=None):
    n, T = tree_tokens.shape
    _check(lib().mlora_verify_tree(ctx, n, _ptr(adapter_idx), T, _ptr(tree_tokens), _ptr(tree_parent),
                                   _ptr(out_accept_len), _ptr(out_accept_idx), _ptr(out_next), _ptr(out_logits)))


def mlora_sample_first(ctx, logits, out_tokens):
    _check(lib().mlora_sample_first(ctx, _ptr(logits), out_tokens.numel(), _ptr(out_tokens)))


def mlora_generate(ctx, adapter_idx, first_tokens, out_tokens):
    """out_tokens: device int32 [k_steps][n_streams]"""
    k, n = out_tokens.shape
    _check(lib().mlora_generate(ctx, n, _ptr(adapter_idx), _ptr(first_tokens), k, _ptr(out_tokens)))


def mlora_generate_host(ctx, adapter_idx, first_tokens, out_tokens):
    """host (CPU) int32 tensors: adapter_idx, first_tokens [n_streams]; out_tokens [k_steps][n_streams]"""
    k, n = out_tokens.shape
    for t in (adapter_idx, first_tokens, out_tokens):
        assert not t.is_cuda and t.is_contiguous() and t.dtype == torch.int32
    _check(lib().mlora_generate_host(ctx, n, C.c_void_p(adapter_idx.data_ptr()), C.c_void_p(first_tokens.data_ptr()), k,
                                     C.c_void_p(out_tokens.data_ptr())))


def mlora_set_forecast(ctx, forecast):
    """forecast: CUDA fp16 [m][d_model] (kept alive by the caller) or None"""
    _check(lib().mlora_set_forecast(ctx, _ptr(forecast), 0 if forecast is None else forecast.shape[0]))


def mlora_ds2d_round(ctx, adapter_idx, tree_tokens, tree_parent, row_level, row_rank, forecast_of, widths, max_width,
                     out_accept_len, out_accept_idx, out_next, out_tree_tokens, out_logits=None):
    n, R = tree_tokens.shape
    _check(lib().mlora_ds2d_round(ctx, n, _ptr(adapter_idx), R, _ptr(tree_tokens), _ptr(tree_parent), _ptr(row_level),
                                  _ptr(row_rank), _ptr(forecast_of), _ptr(widths), widths.numel(), max_width,
                                  _ptr(out_accept_len), _ptr(out_accept_idx), _ptr(out_next), _ptr(out_tree_tokens),
                                  _ptr(out_logits)))


def mlora_quantize_act_int8(x_fp16, scale, out_int8):
    _check(lib().mlora_quantize_act_int8(_ptr(x_fp16), x_fp16.numel(), scale, _ptr(out_int8), _stream()))


def mlora_linear_w4a8(qweight, w_scale, qx, x_scale, y):
    """qweight uint8 [N][K/2], w_scale fp16 [N], qx int8 [M][K], y fp32 [M][N] (CUDA tensors)"""
    M, K = qx.shape
    _check(lib().mlora_linear_w4a8(_ptr(qweight), _ptr(w_scale), _ptr(qx), x_scale, M, K, qweight.shape[0], _ptr(y),
                                   _stream()))


def mlora_reset_streams(ctx):
    _check(lib().mlora_reset_streams(ctx))


def mlora_sync_status(ctx):
    _check(lib().mlora_sync_status(ctx))


def mlora_export_kv(ctx, layer, stream, first, count, k_out=None, v_out=None):
    s = C.c_int32(0)
    _check(lib().mlora_export_kv(ctx, layer, stream, first, count, C.byref(s), _ptr(k_out), _ptr(v_out)))
    return s.value


def mlora_export_state(ctx, layer, stream, k_out, v_out):
    """The stream's whole own segment of one layer into k_out / v_out; returns its suffix length."""
    s = C.c_int32(0)
    _check(lib().mlora_export_state(ctx, layer, stream, C.byref(s), _ptr(k_out), _ptr(v_out)))
    return s.value


def mlora_debug_dequant(ctx, layer, proj, out_fp16):
    _check(lib().mlora_debug_dequant(ctx, layer, proj, _ptr(out_fp16)))


def mlora_debug_set(ctx, key, value):
    _check(lib().mlora_debug_set(ctx, key, value))


def mlora_profile_begin(ctx):
    _check(lib().mlora_profile_begin(ctx))


def mlora_profile_end(ctx):
    ms = (C.c_float * len(PROF_FAMILIES))()
    cnt = (C.c_int32 * len(PROF_FAMILIES))()
    _check(lib().mlora_profile_end(ctx, ms, cnt))
    return {f: (ms[i], cnt[i]) for i, f in enumerate(PROF_FAMILIES)}


def mlora_launch_count(ctx):
    return int(lib().mlora_launch_count(ctx))


def mlora_step_timeline(ctx):
    """Stamps of the last traced decode step as a nested list [2][n_phases][12] of nanoseconds (0: no stamp)."""
    n = C.c_int32(0)
    lib().mlora_step_timeline(ctx, None, 0, C.byref(n))          # asks for the phase count only
    cnt = n.value * 24
    buf = (C.c_int64 * max(cnt, 1))()
    _check(lib().mlora_step_timeline(ctx, buf, cnt, C.byref(n)))
    vals = list(buf)
    return [[vals[(c * n.value + p) * 12:(c * n.value + p) * 12 + 12] for p in range(n.value)] for c in range(2)]


# ----------------------------------------------------------------------------- kernel-level calls
def mlora_weight_create(qweight, scales, K, N, G):
    out = C.c_void_p()
    _check(lib().mlora_weight_create(_ptr(qweight), _ptr(scales), K, N, G, _stream(), C.byref(out)))
    return out


def mlora_weight_destroy(w):
    _check(lib().mlora_weight_destroy(w))


def mlora_weight_dequant(w, out_fp16):
    _check(lib().mlora_weight_dequant(w, _ptr(out_fp16)))


def mlora_linear_workspace_bytes(w, M, rank):
    return int(lib().mlora_linear_workspace_bytes(w, M, rank))


def mlora_linear(w, x, y, workspace, row_adapter=None, A_ptrs=None, B_ptrs=None, scale=None, rank=0):
    """A_ptrs / B_ptrs: int64 CUDA tensors holding the device addresses of the adapters' A / B matrices."""
    n_ad = 0 if A_ptrs is None else A_ptrs.numel()
    _check(lib().mlora_linear(w, _ptr(x), x.shape[0], _ptr(row_adapter), _ptr(A_ptrs), _ptr(B_ptrs), _ptr(scale),
                              n_ad, rank, _ptr(y), _ptr(workspace), workspace.numel() * workspace.element_size()))


def mlora_linear_noalloc(w, x, y, row_adapter=None, A_ptrs=None, B_ptrs=None, scale=None, rank=0):
    """mlora_linear for at most 8 rows with the scratch built into the library: the call allocates nothing."""
    n_ad = 0 if A_ptrs is None else A_ptrs.numel()
    _check(lib().mlora_linear_noalloc(w, _ptr(x), x.shape[0], _ptr(row_adapter), _ptr(A_ptrs), _ptr(B_ptrs),
                                      _ptr(scale), n_ad, rank, _ptr(y)))


def mlora_linear_status(w, workspace=None):
    """Raises MloraError if a bounded wait ran out in an mlora_linear / mlora_linear_noalloc call (None: the latter)."""
    _check(lib().mlora_linear_status(w, _ptr(workspace)))


def mlora_attention_workspace_bytes(n, T, Hq, Hkv, hd, P, own_capacity):
    return int(lib().mlora_attention_workspace_bytes(n, T, Hq, Hkv, hd, P, own_capacity))


def mlora_attention(q, prefix_k, prefix_v, own_k, own_v, suffix_len, suffix_bound, tree_parent, out, workspace, status):
    n, T = tree_parent.shape
    Hq, hd = q.shape[-2], q.shape[-1]
    Hkv = own_k.shape[1]
    P = 0 if prefix_k is None else prefix_k.shape[1]
    _check(lib().mlora_attention(_ptr(q), _ptr(prefix_k), _ptr(prefix_v), P, _ptr(own_k), _ptr(own_v), own_k.shape[2],
                                 _ptr(suffix_len), suffix_bound, _ptr(tree_parent), n, T, Hq, Hkv, hd, _ptr(out),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status), _stream()))
