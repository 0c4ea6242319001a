"""The whole-sequence drafter pass on the GPU (through the C ABI) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import moa_oracle as O
from paper_2410_03804_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _limits(rng, n, ca_n):
    """K-step-bounded limits like the mask figure's: segments of random length, each seeing what was there at its start."""
    lim, i, seen = [], 0, max(1, ca_n // 3)
    while i < n:
        k = int(rng.integers(2, 6))
        lim += [min(seen, ca_n)] * min(k, n - i)
        i += k
        seen += k
    return np.array(lim, np.int32)


def _run(p, n_new, prefix, use_limits, max_ctx, lsa_chunk_tokens=8):
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=max_ctx, lsa_chunk_tokens=lsa_chunk_tokens)
    dr = H.make_oracle(p, w)
    nb = p.batch
    caK, caV = synth.make_cache(p, "ca")
    g.fill_cache("ca", caK.cuda(), caV.cuda())
    toks_pre = synth.make_tokens(p, max(prefix), tensor_index=42)
    flat_pre = torch.cat([toks_pre[b, :prefix[b]] for b in range(nb)])
    g.moa_sa_append(flat_pre.cuda(), prefix)
    toks = synth.make_tokens(p, max(n_new), tensor_index=43)
    flat = torch.cat([toks[b, :n_new[b]] for b in range(nb)])
    rng = np.random.default_rng(17)
    lims = [_limits(rng, n_new[b], p.ctx) for b in range(nb)] if use_limits else None
    lim_t = torch.from_numpy(np.concatenate(lims)).cuda() if use_limits else None
    hid = g.moa_drafter_prefill(flat.cuda(), n_new, ca_limit=lim_t)
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0
    assert g.sa_len[:nb].tolist() == [prefix[b] + n_new[b] for b in range(nb)]
    tol, off, worst = H.tol_of(p), 0, 0.0
    for b in range(nb):
        saK, saV = dr.sa_prefix(toks_pre[b, :prefix[b]].tolist())
        want, K, V = O.drafter_prefill(dr, toks[b, :n_new[b]].tolist(), saK, saV, H.np32(caK[b]), H.np32(caV[b]),
                                       None if lims is None else lims[b])
        worst = max(worst, H.assert_rows_close(H.np32(hid[off:off + n_new[b]].cpu()), want, tol, f"prefill hidden seq {b}"))
        n_all = prefix[b] + n_new[b]
        H.assert_rows_close(H.np32(g.sa_k[b, :n_all].cpu()), K, tol, "SA K after the pass")
        H.assert_rows_close(H.np32(g.sa_v[b, :n_all].cpu()), V, tol, "SA V after the pass")
        off += n_new[b]
    print(f"[prefill {p.name} {p.dtype}] worst hidden {worst:.2e}")
    g.close()


def test_prefill_c1_fp32_with_and_without_limits():
    p = synth.PRESETS["c1"]
    _run(p, [37], [9], False, max_ctx=128)
    _run(p, [37], [0], True, max_ctx=128)


@pytest.mark.parametrize("dtype,use_limits", [("bf16", True), ("bf16", False), ("f32", True)])
def test_prefill_reduced_llama_shape_ragged_batch(dtype, use_limits):
    """Reduced Llama-3 shape, three sequences of different lengths over different prefixes; the longest one spans
    two chunks of 256 rows (one with the two activation terms side by side in one tile, one with two tiles)."""
    p = synth.scaled(synth.PRESETS["c2"], d_model=512, n_stack=5, d_stack=384, vocab=5003, lsa_hq=8, lsa_hkv=2,
                     lsa_mlp=768, sa_hq=8, sa_hkv=2, sa_mlp=64, ca_hq=8, ca_hkv=4, ca_mlp=896, ctx=90, batch=3,
                     tree_topk=5, tree_depth=3, tree_keep=12, dtype=dtype, lsa_tokens=4)
    _run(p, [300, 1, 77], [5, 60, 0], use_limits, max_ctx=512, lsa_chunk_tokens=64)


def test_prefill_misuse_returns_status():
    p = synth.PRESETS["c1"]
    g = H.make_gpu(p, synth.make_weights(p), max_ctx=16)
    tok = torch.zeros(32, dtype=torch.int32, device="cuda")
    with pytest.raises(Exception) as e:
        g.moa_drafter_prefill(tok, [32])                  # 32 tokens do not fit a 16-position cache
    assert "capacity" in str(e.value).lower()
    g.close()
