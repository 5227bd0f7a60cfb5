"""Model shapes of the synthetic workloads (the paper's 1B / 3B LLaMA-style decoders, Sec. 3.1)."""
from dataclasses import dataclass, replace

# Projection order used everywhere a per-layer list of seven matrices appears.
PROJ_NAMES = ("q", "k", "v", "o", "gate", "up", "down")
PROJ_BITS = {"q": 1, "k": 2, "v": 4, "o": 8, "gate": 16, "up": 32, "down": 64}


@dataclass(frozen=True)
class ModelCfg:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int            # 0 => hidden-state input/output (no embedding, no lm_head)
    group_size: int       # INT4 quantisation group length along the input dimension
    lora_rank: int
    lora_targets: int     # OR of PROJ_BITS
    n_adapters: int
    n_streams: int
    prompt_len: int
    alpha: float = 16.0
    rope_theta: float = 1e4
    rms_eps: float = 1e-5
    w_std: float = 0.02       # base weights ~ N(0, w_std)
    b_std: float = 0.01       # LoRA-B ~ N(0, b_std); LoRA-A ~ N(0, 1/r)
    tree_nodes: int = 1
    branch: tuple = ()

    def small(self, **kw):
        return replace(self, **kw)


def proj_shape(cfg: ModelCfg, proj: str):
    """(K, N) = (input features, output features) of one projection."""
    dq = cfg.n_q_heads * cfg.head_dim
    dkv = cfg.n_kv_heads * cfg.head_dim
    return {
        "q": (cfg.d_model, dq), "k": (cfg.d_model, dkv), "v": (cfg.d_model, dkv),
        "o": (dq, cfg.d_model), "gate": (cfg.d_model, cfg.d_ffn), "up": (cfg.d_model, cfg.d_ffn),
        "down": (cfg.d_ffn, cfg.d_model), "lm_head": (cfg.d_model, cfg.vocab),
    }[proj]


ALL7 = 127
QKVO = 15

# Tiny single layer, hidden-state I/O, 4 streams with 4 rank-8 adapters on q/k/v/o.
CFG0 = ModelCfg("tiny1L", 1, 512, 8, 8, 64, 1408, 0, 64, 8, QKVO, 4, 4, 128)
# ~1B: 8 streams, rank-16 adapters on all seven projections, 512-token shared prompt.
CFG1 = ModelCfg("llama1b", 16, 2048, 32, 8, 64, 5632, 32000, 128, 16, ALL7, 8, 8, 512)
# same model with 16-node draft trees (branching 4,2,2; node count includes the root)
CFG2 = replace(CFG1, name="llama1b_ds2d", tree_nodes=16, branch=(4, 2, 2))
# ~3B: rank-32 adapters, 2048-token prompt, 32-node trees (4,4,2)
CFG3 = ModelCfg("llama3b_ds2d", 28, 3072, 24, 8, 128, 8192, 32000, 128, 32, ALL7, 8, 8, 2048,
                tree_nodes=32, branch=(4, 4, 2))
