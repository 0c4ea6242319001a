"""Seeded synthetic inputs for the Mixture-of-Attentions drafter hot path.

This module only draws random tensors of the right shapes and distributions.
It contains none of the method's arithmetic, so the CPU oracle and the CUDA
path can both be fed from it without sharing any computation.

Every tensor is drawn on the CPU in fp32 from its own torch.Generator seeded
with ``SEED_BASE + 1000 * preset.index + tensor_index`` and then cast to the
preset's storage dtype, so both sides see exactly the same stored values.

Shapes follow the paper's hyper-parameter table (Section A.1, "Architecture")
scaled to the Llama-3-8B / 70B dimensions; the MLP widths keep the paper's
ratios (3x the LSA width, E/8 after self-attention, 7E/4 after cross-attention).
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import torch

SEED_BASE = 241003804


@dataclass(frozen=True)
class Preset:
    name: str
    index: int
    d_model: int          # E
    n_stack: int          # S: number of stacked per-layer activations fed to LSA
    d_stack: int          # D_in: width of one stacked activation
    vocab: int
    head_dim: int
    lsa_hq: int
    lsa_hkv: int
    lsa_mlp: int
    sa_hq: int
    sa_hkv: int
    sa_mlp: int
    ca_hq: int
    ca_hkv: int
    ca_mlp: int
    ctx: int              # context length already in the caches
    batch: int
    tree_topk: int        # B
    tree_depth: int       # D
    tree_keep: int        # m
    dtype: str            # "f32" | "bf16"
    lsa_tokens: int       # tokens per sequence fed to LSA in one drafting cycle
    outliers: bool        # 8 channels scaled 20x in activations (and caches where stated)
    cache_outliers: bool
    stack_std_ramp: bool  # std of stacked activation l is 0.5 + l/16 instead of 1
    rms_eps: float = 1e-5
    rope_theta: float = 500000.0
    # Target Layer Inference (Section 3.2): the last n_tli decoder layers of the LLM run on the drafted rows
    n_tli: int = 0
    tli_hq: int = 0
    tli_hkv: int = 0
    tli_mlp: int = 0

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def pool_size(self) -> int:
        return self.tree_topk + (self.tree_depth - 1) * self.tree_topk ** 2

    def as_dict(self) -> dict:
        return asdict(self)


PRESETS = {
    "c1": Preset("c1", 1, 256, 4, 256, 1024, 64, 4, 4, 768, 4, 4, 32, 4, 4, 448,
                 64, 1, 4, 4, 16, "f32", 64, False, False, False),
    "c2": Preset("c2", 2, 4096, 32, 4096, 128256, 128, 32, 8, 12288, 32, 8, 512, 32, 8, 7168,
                 2048, 1, 10, 6, 60, "bf16", 5, True, False, True),
    "c3": Preset("c3", 3, 4096, 33, 4096, 128256, 128, 32, 32, 12288, 32, 8, 512, 32, 8, 7168,
                 0, 1, 10, 6, 60, "bf16", 8192, True, False, True),
    "c4": Preset("c4", 4, 4096, 32, 4096, 128256, 128, 32, 8, 12288, 32, 8, 512, 32, 8, 7168,
                 32768, 1, 10, 6, 60, "bf16", 5, True, False, True),
    "c5": Preset("c5", 5, 8192, 80, 8192, 128256, 128, 64, 8, 24576, 64, 8, 1024, 64, 8, 14336,
                 4096, 16, 10, 6, 60, "bf16", 5, True, True, False),
    # the paper's own 8B drafter widths (hyper-parameter table), breadth 8 / depth 6 / 62 kept
    "p8": Preset("p8", 8, 4096, 32, 2048, 128256, 128, 16, 8, 6144, 32, 4, 512, 32, 8, 7168,
                 2048, 1, 8, 6, 62, "bf16", 5, True, False, True),
}


def scaled(p: Preset, **kw) -> Preset:
    """A copy of a preset with some fields replaced (reduced shapes for tests)."""
    d = p.as_dict()
    d.update(kw)
    return Preset(**d)


def _gen(p: Preset, tensor_index: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(SEED_BASE + 1000 * p.index + tensor_index)
    return g


def _randn(p: Preset, tensor_index: int, shape, std: float = 1.0, mean: float = 0.0) -> torch.Tensor:
    x = torch.randn(tuple(shape), generator=_gen(p, tensor_index), dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    if mean != 0.0:
        x.add_(mean)
    return x


# weight name -> (tensor_index, shape function)
def weight_shapes(p: Preset) -> dict:
    E, Din, V, dh = p.d_model, p.d_stack, p.vocab, p.head_dim
    return {
        "embed": (V, E), "lm_head": (V, E), "final_norm": (E,),
        "lsa_norm1": (Din,), "lsa_wq": (p.lsa_hq * dh, Din), "lsa_wk": (p.lsa_hkv * dh, Din),
        "lsa_wv": (p.lsa_hkv * dh, Din), "lsa_wo": (Din, p.lsa_hq * dh), "lsa_norm2": (Din,),
        "lsa_wgate": (p.lsa_mlp, Din), "lsa_wup": (p.lsa_mlp, Din), "lsa_wdown": (Din, p.lsa_mlp),
        "sa_norm1": (E,), "sa_wq": (p.sa_hq * dh, E), "sa_wk": (p.sa_hkv * dh, E),
        "sa_wv": (p.sa_hkv * dh, E), "sa_wo": (E, p.sa_hq * dh), "sa_norm2": (E,),
        "sa_wgate": (p.sa_mlp, E), "sa_wup": (p.sa_mlp, E), "sa_wdown": (E, p.sa_mlp),
        "ca_normq": (E,), "ca_normkv": (Din,), "ca_wq": (p.ca_hq * dh, E),
        "ca_wk": (p.ca_hkv * dh, Din), "ca_wv": (p.ca_hkv * dh, Din), "ca_wo": (E, p.ca_hq * dh),
        "ca_norm2": (E,), "ca_wgate": (p.ca_mlp, E), "ca_wup": (p.ca_mlp, E), "ca_wdown": (E, p.ca_mlp),
    }


WEIGHT_NAMES = list(weight_shapes(PRESETS["c1"]).keys())


def make_weights(p: Preset, only=None) -> dict:
    """Random drafter weights: matrices ~ N(0, 0.02), norm gains = 1 + N(0, 0.02).

    Returns CPU tensors in the preset's storage dtype. ``only`` restricts the
    set of names (large presets: skip what a test does not touch)."""
    out = {}
    for i, (name, shape) in enumerate(weight_shapes(p).items()):
        if only is not None and name not in only:
            continue
        is_gain = len(shape) == 1
        w = _randn(p, 100 + i, shape, std=0.02, mean=1.0 if is_gain else 0.0)
        out[name] = w.to(p.torch_dtype)
    return out


TLI_LAYER_NAMES = ["norm1", "wq", "wk", "wv", "wo", "norm2", "wgate", "wup", "wdown"]


def tli_weight_shapes(p: Preset) -> dict:
    """Shapes of the n_tli LLM decoder layers' weights, named tli{l}_{name}, l = 0 the earliest layer."""
    E, dh = p.d_model, p.head_dim
    one = {"norm1": (E,), "wq": (p.tli_hq * dh, E), "wk": (p.tli_hkv * dh, E), "wv": (p.tli_hkv * dh, E),
           "wo": (E, p.tli_hq * dh), "norm2": (E,), "wgate": (p.tli_mlp, E), "wup": (p.tli_mlp, E),
           "wdown": (E, p.tli_mlp)}
    return {f"tli{l}_{n}": one[n] for l in range(p.n_tli) for n in TLI_LAYER_NAMES}


def make_tli_weights(p: Preset) -> dict:
    """Random decoder-layer weights with the distributions of make_weights (tensor indices 200 + ...)."""
    out = {}
    for i, (name, shape) in enumerate(tli_weight_shapes(p).items()):
        is_gain = len(shape) == 1
        out[name] = _randn(p, 200 + i, shape, std=0.02, mean=1.0 if is_gain else 0.0).to(p.torch_dtype)
    return out


def make_tli_cache(p: Preset, layer: int, ctx: int | None = None) -> tuple[torch.Tensor, torch.Tensor]:
    """Synthetic LLM K and V cache of one Target-Layer-Inference layer [batch, ctx, tli_hkv, dh] ~ N(0,1)
    (keys treated as already rotated; the cache_outliers rule of make_cache applies)."""
    ctx = p.ctx if ctx is None else ctx
    outs = []
    for j in range(2):
        x = _randn(p, 300 + 10 * layer + j, (p.batch, ctx, p.tli_hkv * p.head_dim))
        if p.cache_outliers:
            ch = _outlier_channels(p, 305 + 10 * layer + j, p.tli_hkv * p.head_dim)
            x[:, :, ch] *= 20.0
        outs.append(x.view(p.batch, ctx, p.tli_hkv, p.head_dim).to(p.torch_dtype))
    return outs[0], outs[1]


def _outlier_channels(p: Preset, tensor_index: int, width: int) -> torch.Tensor:
    return torch.randperm(width, generator=_gen(p, tensor_index))[:8]


def make_h_stack(p: Preset, n_tok: int, tensor_index: int = 10) -> torch.Tensor:
    """Stacked per-layer activations [n_tok, S, D_in]."""
    x = _randn(p, tensor_index, (n_tok, p.n_stack, p.d_stack))
    if p.stack_std_ramp:
        std = 0.5 + torch.arange(p.n_stack, dtype=torch.float32) / 16.0
        x.mul_(std.view(1, -1, 1))
    if p.outliers:
        ch = _outlier_channels(p, tensor_index + 1, p.d_stack)
        x[:, :, ch] *= 20.0
    return x.to(p.torch_dtype)


def make_cache(p: Preset, which: str, ctx: int | None = None) -> tuple[torch.Tensor, torch.Tensor]:
    """Synthetic K and V cache content [batch, ctx, Hkv, dh] ~ N(0,1).

    ``which`` is "ca" (cross-attention keys/values, i.e. projected LSA outputs)
    or "sa" (self-attention prefix keys/values, treated as already rotated)."""
    ctx = p.ctx if ctx is None else ctx
    hkv = p.ca_hkv if which == "ca" else p.sa_hkv
    base = 20 if which == "ca" else 30
    outs = []
    for j in range(2):
        x = _randn(p, base + j, (p.batch, ctx, hkv * p.head_dim))
        if p.cache_outliers:
            ch = _outlier_channels(p, base + 5 + j, hkv * p.head_dim)
            x[:, :, ch] *= 20.0
        outs.append(x.view(p.batch, ctx, hkv, p.head_dim).to(p.torch_dtype))
    return outs[0], outs[1]


def make_tokens(p: Preset, n: int, tensor_index: int = 40) -> torch.Tensor:
    """Uniform token ids [batch, n] (int32)."""
    return torch.randint(0, p.vocab, (p.batch, n), generator=_gen(p, tensor_index), dtype=torch.int32)


def make_root(p: Preset, tensor_index: int = 41) -> torch.Tensor:
    """One root token id per sequence [batch] (int32): the last verified token."""
    return torch.randint(0, p.vocab, (p.batch,), generator=_gen(p, tensor_index), dtype=torch.int32)
