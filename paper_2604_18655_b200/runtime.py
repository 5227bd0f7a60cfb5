"""Convenience holder around the C-ABI context: uploads canonical-format numpy blobs with torch, keeps the
device tensors alive for as long as the context needs them, and allocates output tensors.  No arithmetic
of the method happens here."""
import numpy as np
import torch

from . import binding as mb


def _dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


class MloraModel:
    def __init__(self, synth, *, max_adapters=None, max_streams=None, max_prefix=None, max_suffix=256, max_tree=1):
        cfg = synth.cfg
        self.cfg = cfg
        self.dev = torch.device("cuda", torch.cuda.current_device())
        self.qweight = [_dev(q) for q in synth.qweight]
        self.scales = [_dev(s) for s in synth.scales]
        self.rms_attn = [_dev(g) for g in synth.rms_attn]
        self.rms_ffn = [_dev(g) for g in synth.rms_ffn]
        self.rms_final = None if synth.rms_final is None else _dev(synth.rms_final)
        self.embed = None if synth.embed is None else _dev(synth.embed)
        self.max_streams = max_streams or cfg.n_streams
        self.max_tree = max_tree
        self.ctx = mb.mlora_create(cfg, self.qweight, self.scales, self.rms_attn, self.rms_ffn, self.rms_final,
                                   self.embed, max_adapters=max_adapters or max(cfg.n_adapters, 1),
                                   max_streams=self.max_streams, max_prefix=max_prefix or cfg.prompt_len,
                                   max_suffix=max_suffix, max_tree=max_tree)
        # the canonical weights were repacked into the context's own layout: release them
        self.qweight, self.scales = None, None
        self.adapters = {}

    def close(self):
        if self.ctx is not None:
            mb.mlora_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- adapters: tensors stay referenced here until the slot is overwritten
    def set_adapter(self, slot, A, B, alpha):
        if A is None:
            mb.mlora_set_adapter(self.ctx, slot, None, None, 0.0)
            self.adapters.pop(slot, None)
            return
        dA = [None if a is None else _dev(a) for a in A]
        dB = [None if b is None else _dev(b) for b in B]
        mb.mlora_set_adapter(self.ctx, slot, dA, dB, alpha)
        self.adapters[slot] = (dA, dB)

    def _i32(self, a):
        return _dev(np.asarray(a, dtype=np.int32))

    # -- steps (host-array convenience forms; each returns numpy)
    def prefill(self, prompt_ids):
        ids = self._i32(prompt_ids)
        out = torch.empty(self.cfg.vocab, dtype=torch.float32, device=self.dev)
        mb.mlora_prefill_shared(self.ctx, ids, out)
        return out.cpu().numpy()

    def prefill_h(self, hidden):
        out = torch.empty(self.cfg.d_model, dtype=torch.float32, device=self.dev)
        mb.mlora_prefill_shared_h(self.ctx, _dev(hidden), out)
        return out.cpu().numpy()

    def decode(self, adapter_idx, tokens, want_logits=True):
        n = len(adapter_idx)
        nxt = torch.empty(n, dtype=torch.int32, device=self.dev)
        logits = torch.empty(n, self.cfg.vocab, dtype=torch.float32, device=self.dev) if want_logits else None
        mb.mlora_decode_step(self.ctx, self._i32(adapter_idx), self._i32(tokens), nxt, logits)
        return nxt.cpu().numpy(), (None if logits is None else logits.cpu().numpy())

    def decode_h(self, adapter_idx, hidden):
        n = len(adapter_idx)
        out = torch.empty(n, self.cfg.d_model, dtype=torch.float32, device=self.dev)
        mb.mlora_decode_step_h(self.ctx, self._i32(adapter_idx), _dev(hidden), out)
        return out.cpu().numpy()

    def verify(self, adapter_idx, tree_tokens, tree_parent, want_logits=True):
        tt = self._i32(tree_tokens)
        tp = self._i32(tree_parent)
        n, T = tt.shape
        acc_len = torch.empty(n, dtype=torch.int32, device=self.dev)
        acc_idx = torch.empty(n, T, dtype=torch.int32, device=self.dev)
        nxt = torch.empty(n, dtype=torch.int32, device=self.dev)
        logits = torch.empty(n * T, self.cfg.vocab, dtype=torch.float32, device=self.dev) if want_logits else None
        mb.mlora_verify_tree(self.ctx, self._i32(adapter_idx), tt, tp, acc_len, acc_idx, nxt, logits)
        return dict(accept_len=acc_len.cpu().numpy(), accept_idx=acc_idx.cpu().numpy(), next=nxt.cpu().numpy(),
                    logits=None if logits is None else logits.cpu().numpy())

    def export_kv(self, layer, stream, first, count):
        c = self.cfg
        k = torch.empty(count, c.n_kv_heads, c.head_dim, dtype=torch.float16, device=self.dev)
        v = torch.empty_like(k)
        s = mb.mlora_export_kv(self.ctx, layer, stream, first, count, k, v)
        return s, k.cpu().numpy(), v.cpu().numpy()

    def suffix_len(self, stream):
        return mb.mlora_export_kv(self.ctx, 0, stream, 0, 0, None, None)
