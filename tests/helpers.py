"""Shared test plumbing: builds the CUDA model and the CPU oracle from the same seeded tensors."""
import numpy as np
import torch

from oracle import moa_oracle as O
from paper_2410_03804_b200 import synth

CFG_KEYS = ("d_model", "n_stack", "d_stack", "vocab", "head_dim", "lsa_hq", "lsa_hkv", "lsa_mlp", "sa_hq", "sa_hkv",
            "sa_mlp", "ca_hq", "ca_hkv", "ca_mlp", "tree_topk", "tree_depth", "tree_keep", "rms_eps", "rope_theta",
            "dtype", "n_tli", "tli_hq", "tli_hkv", "tli_mlp")


def cfg_of(p: synth.Preset) -> dict:
    d = p.as_dict()
    return {k: d[k] for k in CFG_KEYS}


def tol_of(p: synth.Preset) -> float:
    """Max-abs error allowed, relative to the row's max |value|: 1e-4 on the fp32 path, 2e-2 on bf16."""
    return 1e-4 if p.dtype == "f32" else 2e-2


def np32(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float32).numpy()


def make_oracle(p: synth.Preset, weights_cpu: dict, cache_f64=True, store=None) -> O.Drafter:
    return O.Drafter(cfg_of(p), {k: np32(v) for k, v in weights_cpu.items()}, cache_f64=cache_f64, store=store)


def split_regime(p: synth.Preset, rows: int = None) -> bool:
    """bf16 forwards of up to 256 rows (every draft step) carry their activations as two bf16 terms (about 16 bits
    of mantissa), so their decisions are taken at nearly the oracle's own precision."""
    rows = p.batch * p.tree_topk if rows is None else rows
    return p.dtype == "bf16" and rows <= 256


def make_oracles(p: synth.Preset, weights_cpu: dict, cache_f64=True):
    """(values, decisions): the unrounded oracle that values are compared with, and the oracle whose
    top-B decisions are compared. The same object on the fp32 path and on bf16 forwards of up to 256 rows
    (activations carried at ~16 bits); the bf16-storage mode on larger bf16 forwards (plain 16-bit activations)."""
    w = {k: np32(v) for k, v in weights_cpu.items()}
    exact = O.Drafter(cfg_of(p), w, cache_f64=cache_f64)
    if p.dtype == "f32" or split_regime(p):
        return exact, exact
    dec = O.Drafter(cfg_of(p), w, cache_f64=cache_f64, store="bf16")
    dec._cache = exact._cache          # share the widened weights
    return exact, dec


def make_gpu(p: synth.Preset, weights_cpu: dict, max_ctx: int, lsa_chunk_tokens: int = 8, max_batch=None):
    from paper_2410_03804_b200 import moa
    w = {k: v.cuda() for k, v in weights_cpu.items()}
    return moa.MoA(cfg_of(p), w, max_batch or p.batch, max_ctx, lsa_chunk_tokens)


def assert_rows_close(got, want, tol, what=""):
    """max |got - want| per row <= tol * max |want| of that row."""
    got = np.asarray(got, np.float64).reshape(-1, np.shape(got)[-1])
    want = np.asarray(want, np.float64).reshape(-1, np.shape(want)[-1])
    assert got.shape == want.shape, (what, got.shape, want.shape)
    err = np.max(np.abs(got - want), axis=-1)
    ref = np.max(np.abs(want), axis=-1)
    bad = err > tol * ref + 1e-30
    assert not np.any(bad), f"{what}: worst rel err {np.max(err / (ref + 1e-30)):.3e} > {tol:g} (rows {np.nonzero(bad)[0][:8]})"
    return float(np.max(err / (ref + 1e-30)))


def tie_window(p: synth.Preset, z) -> float:
    """How close two of the oracle's log-probabilities must be for either order to count as correct.

    fp32 path: 1e-3. bf16 forwards of up to 256 rows: 1e-3 plus 2e-3 * max|z| -- weights,
    cache entries and tree keys / values are stored in 16 bits whatever the arithmetic, which leaves the logits
    about 1e-3 * max|z| away from the fp64 oracle's (measured: worst 1.1e-3 on configs 2 and 4, 1.7e-3 on the
    reduced shapes). Larger bf16
    forwards (plain 16-bit activations, compared with the oracle's bf16-storage mode): the value tolerance
    itself, 2e-2 * max|z|: after ~12 storage roundings the two sides' rounding decisions are uncorrelated, so a
    swap of two tokens closer than the value tolerance is consistent with logits that pass it."""
    if p.dtype == "f32":
        return 1e-3
    scale = float(np.max(np.abs(z)))
    return 1e-3 + 2e-3 * scale if split_regime(p) else 2e-2 * scale


def check_topk(gpu_ids, gpu_lp, z, tol, window=1e-3, what="", literal=None):
    """One row's top-B against the oracle's full logits z.

    Each reported log-probability must match the oracle's for that token within tol * max|z|; the j-th pick
    must be within `window` of the oracle's j-th best log-probability (either of two near-tied tokens is
    accepted); ids are distinct. Returns True when the id list equals the oracle's exactly. With `literal` (a
    list) given, appends whether the row also passes the plain 1e-3 window (no logit-scaled term)."""
    z = np.asarray(z, np.float64)
    lse = z.max() + np.log(np.exp(z - z.max()).sum())
    logp = z - lse
    order = np.lexsort((np.arange(z.shape[0]), -logp))
    B = len(gpu_ids)
    ids = [int(i) for i in gpu_ids]
    assert len(set(ids)) == B and min(ids) >= 0 and max(ids) < z.shape[0], (what, ids)
    scale = np.max(np.abs(z))
    lit = True
    for j in range(B):
        assert abs(float(gpu_lp[j]) - logp[ids[j]]) <= tol * scale, (what, j, float(gpu_lp[j]), logp[ids[j]])
        assert logp[ids[j]] >= logp[order[j]] - window, (what, j, ids[j], logp[ids[j]], logp[order[j]])
        lit = lit and logp[ids[j]] >= logp[order[j]] - 1e-3
    if literal is not None:
        literal.append(bool(lit))
    return ids == [int(i) for i in order[:B]]
