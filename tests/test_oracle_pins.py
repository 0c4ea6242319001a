"""Pins for the CPU oracle: every function is checked against something other
than itself -- closed forms, library routines (torch), brute force on tiny
inputs, the paper's mask predicates and pool-size formula, and invariants that
a dropped term, a wrong sign/index or a transposed operand would break."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import moa_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(20241003)


def tiny_cfg(**kw):
    c = dict(d_model=16, n_stack=3, d_stack=12, vocab=24, head_dim=4,
             lsa_hq=4, lsa_hkv=2, lsa_mlp=10, sa_hq=4, sa_hkv=2, sa_mlp=6,
             ca_hq=4, ca_hkv=2, ca_mlp=14, rms_eps=1e-5, rope_theta=10000.0)
    c.update(kw)
    return c


def tiny_weights(c, scale=0.3, rng=None):
    rng = rng or np.random.default_rng(7)
    E, Din, V, dh = c["d_model"], c["d_stack"], c["vocab"], c["head_dim"]
    shp = {
        "embed": (V, E), "lm_head": (V, E), "final_norm": (E,),
        "lsa_norm1": (Din,), "lsa_wq": (c["lsa_hq"] * dh, Din), "lsa_wk": (c["lsa_hkv"] * dh, Din),
        "lsa_wv": (c["lsa_hkv"] * dh, Din), "lsa_wo": (Din, c["lsa_hq"] * dh), "lsa_norm2": (Din,),
        "lsa_wgate": (c["lsa_mlp"], Din), "lsa_wup": (c["lsa_mlp"], Din), "lsa_wdown": (Din, c["lsa_mlp"]),
        "sa_norm1": (E,), "sa_wq": (c["sa_hq"] * dh, E), "sa_wk": (c["sa_hkv"] * dh, E),
        "sa_wv": (c["sa_hkv"] * dh, E), "sa_wo": (E, c["sa_hq"] * dh), "sa_norm2": (E,),
        "sa_wgate": (c["sa_mlp"], E), "sa_wup": (c["sa_mlp"], E), "sa_wdown": (E, c["sa_mlp"]),
        "ca_normq": (E,), "ca_normkv": (Din,), "ca_wq": (c["ca_hq"] * dh, E),
        "ca_wk": (c["ca_hkv"] * dh, Din), "ca_wv": (c["ca_hkv"] * dh, Din), "ca_wo": (E, c["ca_hq"] * dh),
        "ca_norm2": (E,), "ca_wgate": (c["ca_mlp"], E), "ca_wup": (c["ca_mlp"], E), "ca_wdown": (E, c["ca_mlp"]),
    }
    w = {}
    for k, s in shp.items():
        w[k] = (1.0 + 0.1 * rng.standard_normal(s)) if len(s) == 1 else scale * rng.standard_normal(s)
    return w


def read_grid(name):
    rows = [l.split() for l in open(os.path.join(GOLD, name)) if not l.startswith("#") and l.strip()]
    return np.array(rows, dtype=np.uint8)


# ------------------------------------------------------------------ elementary
def test_softmax_rows_sum_to_one_and_shift_invariant():
    a = RNG.standard_normal((5, 33)) * 10
    p = O.softmax(a)
    assert np.all(np.abs(p.sum(-1) - 1) < 1e-12)
    assert np.allclose(p, O.softmax(a + 123.456), atol=1e-13)
    # two-way softmax is the logistic function
    x = 0.7
    assert abs(O.softmax(np.array([x, 0.0]))[0] - 1 / (1 + np.exp(-x))) < 1e-15
    # matches the library routine
    assert np.allclose(p, torch.softmax(torch.from_numpy(a), -1).numpy(), atol=1e-14)


def test_rmsnorm_closed_forms_and_library():
    g = RNG.standard_normal(7)
    # a constant vector normalises to its sign times the gain (eps -> 0)
    assert np.allclose(O.rmsnorm(np.full(7, -3.0), g, 0.0), -g, atol=1e-14)
    x = RNG.standard_normal((4, 7))
    # scale invariance at eps = 0 and unit mean square at unit gain
    assert np.allclose(O.rmsnorm(5 * x, g, 0.0), O.rmsnorm(x, g, 0.0), atol=1e-13)
    assert np.allclose(np.mean(O.rmsnorm(x, np.ones(7), 0.0) ** 2, -1), 1.0, atol=1e-13)
    # eps sits inside the square root, added to the MEAN square
    assert abs(O.rmsnorm(np.array([3.0, 4.0]), np.ones(2), 0.5)[0] - 3 / np.sqrt(12.5 + 0.5)) < 1e-15
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (7,), torch.from_numpy(g), 1e-5).numpy()
    assert np.allclose(O.rmsnorm(x, g, 1e-5), ref, atol=1e-14)


def test_silu_and_mlp_special_cases():
    assert abs(O.silu(1.0) - 0.7310585786300049) < 1e-15     # 1 / (1 + e^-1)
    assert O.silu(0.0) == 0.0
    x = RNG.standard_normal(50)
    assert np.allclose(O.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy(), atol=1e-15)
    u = RNG.standard_normal(5)
    wg, wu, wd = RNG.standard_normal((3, 5)), RNG.standard_normal((3, 5)), RNG.standard_normal((4, 3))
    assert np.all(O.swiglu_mlp(u, 0 * wg, wu, wd) == 0)        # silu(0) = 0 gates everything off
    # a single hidden unit: scalar closed form, down weight picks the output slot
    wg1 = np.zeros((1, 5)); wg1[0, 2] = 1.0
    wu1 = np.zeros((1, 5)); wu1[0, 4] = 2.0
    wd1 = np.zeros((4, 1)); wd1[3, 0] = -1.5
    out = O.swiglu_mlp(u, wg1, wu1, wd1)
    want = -1.5 * (u[2] / (1 + np.exp(-u[2]))) * 2.0 * u[4]
    assert np.allclose(out, [0, 0, 0, want], atol=1e-15)


def test_round_bf16_against_library_and_by_hand():
    x = np.concatenate([RNG.standard_normal(4000) * 10.0 ** RNG.integers(-6, 6, 4000), [0.0, -0.0, 1.0, 65504.0]])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(x), want)
    assert O.round_bf16(1 + 2.0 ** -8) == 1.0                    # tie -> even mantissa
    assert O.round_bf16(1 + 3 * 2.0 ** -8) == 1 + 2.0 ** -6      # tie -> even mantissa, upwards
    assert O.round_bf16(1 + 2.0 ** -8 + 2.0 ** -20) == 1 + 2.0 ** -7
    assert O.round_bf16(np.ones((2, 3))).shape == (2, 3)


def test_bf16_storage_mode_is_a_small_perturbation():
    c = tiny_cfg()
    w = {k: O.round_bf16(v) for k, v in tiny_weights(c).items()}
    H = O.round_bf16(RNG.standard_normal((2, c["n_stack"], c["d_stack"])))
    a = O.Drafter(c, w).lsa_forward(H)
    b = O.Drafter(c, w, store="bf16").lsa_forward(H)
    rel = np.max(np.abs(a - b)) / np.max(np.abs(a))
    assert 0 < rel < 2e-2
    # stored tensors are exactly representable in bfloat16
    Kc, Vc = O.Drafter(c, w, store="bf16").ca_kv(b)
    assert np.array_equal(O.round_bf16(Kc), Kc) and np.array_equal(O.round_bf16(Vc), Vc)


def test_linear_orientation():
    # W[n, k] with a single one routes x[k] to y[n]: catches a transposed operand
    w = np.zeros((3, 5)); w[2, 4] = 1.0
    x = np.arange(5.0)
    assert np.array_equal(O.linear(x, w), [0, 0, 4.0])
    X = RNG.standard_normal((6, 5))
    W = RNG.standard_normal((3, 5))
    assert np.allclose(O.linear(X, W), torch.nn.functional.linear(torch.from_numpy(X), torch.from_numpy(W)).numpy())


def test_rope_against_complex_rotation_and_invariants():
    dh, theta = 8, 10000.0
    x = RNG.standard_normal((3, dh))
    y = RNG.standard_normal((3, dh))
    assert np.array_equal(O.rope(x, 0, theta), x)                 # position 0 is the identity
    for pos in (1, 17, 4099):
        r = O.rope(x, pos, theta)
        z = (x[:, :dh // 2] + 1j * x[:, dh // 2:]) * np.exp(1j * pos * theta ** (-2 * np.arange(dh // 2) / dh))
        assert np.allclose(r[:, :dh // 2], z.real, atol=1e-12) and np.allclose(r[:, dh // 2:], z.imag, atol=1e-12)
        assert np.allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(x, axis=-1))
        # the score of two vectors depends on the position difference only
        assert np.allclose(np.sum(O.rope(x, pos, theta) * O.rope(y, pos, theta), -1), np.sum(x * y, -1))
        assert np.allclose(np.sum(O.rope(x, pos + 5, theta) * O.rope(y, pos, theta), -1),
                           np.sum(O.rope(x, 5, theta) * y, -1))
    # the first pair turns fastest (angle = pos), the last slowest
    e0 = np.zeros(dh); e0[0] = 1.0
    assert np.allclose(O.rope(e0, 1, theta)[[0, dh // 2]], [np.cos(1.0), np.sin(1.0)])
    assert np.array_equal(O.rope(x, 9, 0.0), x)


def test_attention_core_special_cases_and_library():
    dh = 4
    q = RNG.standard_normal(dh)
    K = RNG.standard_normal((6, dh))
    V = RNG.standard_normal((6, dh))
    assert np.allclose(O.attend(q, K[:1], V[:1]), V[0])                    # single key returns its value
    assert np.allclose(O.attend(q, 0 * K, V), V.mean(0))                   # zero keys: uniform weights
    assert np.allclose(O.attend(q, np.tile(K[:1], (6, 1)), V), V.mean(0))  # identical keys
    # scale 1/sqrt(dh): two keys, closed form
    k2 = np.stack([q, np.zeros(dh)])
    w0 = 1 / (1 + np.exp(-(q @ q) / np.sqrt(dh)))
    assert np.allclose(O.attend(q, k2, V[:2]), w0 * V[0] + (1 - w0) * V[1])
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None, None], torch.from_numpy(K)[None], torch.from_numpy(V)[None])[0, 0].numpy()
    assert np.allclose(O.attend(q, K, V), ref, atol=1e-13)
    assert [O.kv_head_of(h, 8, 2) for h in range(8)] == [0, 0, 0, 0, 1, 1, 1, 1]


def test_lm_head_topk_against_full_sort():
    E, V, B = 16, 50, 5
    o = RNG.standard_normal(E)
    g = 1 + 0.1 * RNG.standard_normal(E)
    W = RNG.standard_normal((V, E))
    ids, logp, z = O.lm_head_topk(o, g, W, 1e-5, B)
    ref_lp = torch.log_softmax(torch.from_numpy(W) @ torch.nn.functional.rms_norm(
        torch.from_numpy(o), (E,), torch.from_numpy(g), 1e-5), -1)
    assert abs(np.exp(z - (z.max() + np.log(np.exp(z - z.max()).sum()))).sum() - 1) < 1e-12
    tv, ti = torch.topk(ref_lp, B)
    assert np.array_equal(ids, ti.numpy()) and np.allclose(logp, tv.numpy(), atol=1e-12)
    assert np.all(logp <= 0) and np.all(np.diff(logp) <= 0)
    # ties go to the smaller token id
    W2 = W.copy(); W2[31] = W2[7]; W2[3] = W2[7]
    ids2, logp2, _ = O.lm_head_topk(o, g, W2, 1e-5, V)
    pos = {int(t): i for i, t in enumerate(ids2)}
    assert pos[3] + 1 == pos[7] and pos[7] + 1 == pos[31]


# ------------------------------------------------------------------ LSA
def test_lsa_mask_is_full_and_matches_figure():
    """Dependency of per-layer outputs on per-layer inputs == Figure 2's full grid."""
    c = tiny_cfg(n_stack=10)
    dr = O.Drafter(c, tiny_weights(c))
    X = RNG.standard_normal((10, c["d_stack"]))
    Z = dr.lsa_rows(X)
    dep = np.zeros((10, 10), np.uint8)
    for j in range(10):
        X2 = X.copy(); X2[j] += 0.5
        dep[:, j] = np.any(np.abs(dr.lsa_rows(X2) - Z) > 1e-9, axis=-1)
    assert np.array_equal(dep, read_grid("mask_lsa_10x10.txt"))


def test_lsa_permutation_independence_incremental():
    c = tiny_cfg()
    dr = O.Drafter(c, tiny_weights(c))
    H = RNG.standard_normal((5, c["n_stack"], c["d_stack"]))
    kv = dr.lsa_forward(H)
    assert kv.shape == (5, c["d_stack"])
    # no positional term over layers + symmetric mean: invariant to layer order
    assert np.allclose(dr.lsa_forward(H[:, [2, 0, 1]]), kv, atol=1e-12)
    # tokens are independent; appending later equals one pass
    assert np.allclose(np.stack([dr.lsa_forward(H[t:t + 1])[0] for t in range(5)]), kv, atol=0)
    assert np.allclose(np.concatenate([dr.lsa_forward(H[:2]), dr.lsa_forward(H[2:])]), kv, atol=0)
    assert dr.lsa_forward(H[:0]).shape == (0, c["d_stack"])


def test_lsa_special_cases():
    c = tiny_cfg()
    w = tiny_weights(c)
    w["lsa_wdown"] = 0 * w["lsa_wdown"]                  # switch the MLP off
    dr = O.Drafter(c, w)
    dh, hq, hkv = c["head_dim"], c["lsa_hq"], c["lsa_hkv"]
    x = RNG.standard_normal(c["d_stack"])
    # all layer rows identical -> every head returns that row's value projection
    X = np.tile(x, (c["n_stack"], 1))
    v = O.linear(O.rmsnorm(x, w["lsa_norm1"], c["rms_eps"]), w["lsa_wv"]).reshape(hkv, dh)
    o = np.concatenate([v[h // (hq // hkv)] for h in range(hq)])
    assert np.allclose(dr.lsa_token(X), x + O.linear(o, w["lsa_wo"]), atol=1e-12)
    # single layer (S = 1): same closed form
    assert np.allclose(dr.lsa_token(X[:1]), x + O.linear(o, w["lsa_wo"]), atol=1e-12)
    # zero key projection -> uniform attention -> mean of the value rows
    w2 = dict(w); w2["lsa_wk"] = 0 * w["lsa_wk"]
    dr2 = O.Drafter(c, w2)
    X = RNG.standard_normal((c["n_stack"], c["d_stack"]))
    vm = O.linear(O.rmsnorm(X, w["lsa_norm1"], c["rms_eps"]), w["lsa_wv"]).mean(0).reshape(hkv, dh)
    om = np.concatenate([vm[h // (hq // hkv)] for h in range(hq)])
    assert np.allclose(dr2.lsa_token(X), X.mean(0) + O.linear(om, w["lsa_wo"]), atol=1e-12)
    # zero out-projection and MLP: the block is the identity, the result the plain mean
    w3 = dict(w); w3["lsa_wo"] = 0 * w["lsa_wo"]
    assert np.allclose(O.Drafter(c, w3).lsa_token(X), X.mean(0), atol=1e-14)


def test_lsa_attention_matches_library_sdpa():
    """The whole attention sub-step against torch's SDPA with grouped heads."""
    c = tiny_cfg()
    w = tiny_weights(c)
    w["lsa_wdown"] = 0 * w["lsa_wdown"]
    dr = O.Drafter(c, w)
    S, dh, hq, hkv = c["n_stack"], c["head_dim"], c["lsa_hq"], c["lsa_hkv"]
    X = RNG.standard_normal((S, c["d_stack"]))
    U = torch.nn.functional.rms_norm(torch.from_numpy(X), (c["d_stack"],), torch.from_numpy(w["lsa_norm1"]), 1e-5)
    q = (U @ torch.from_numpy(w["lsa_wq"]).T).view(S, hq, dh).transpose(0, 1)[None]
    k = (U @ torch.from_numpy(w["lsa_wk"]).T).view(S, hkv, dh).transpose(0, 1)[None]
    v = (U @ torch.from_numpy(w["lsa_wv"]).T).view(S, hkv, dh).transpose(0, 1)[None]
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, enable_gqa=True)[0].transpose(0, 1).reshape(S, hq * dh)
    Y = torch.from_numpy(X) + o @ torch.from_numpy(w["lsa_wo"]).T
    assert np.allclose(dr.lsa_rows(X), Y.numpy(), atol=1e-12)


# ------------------------------------------------------------------ CA
def test_ca_input_independence_and_single_key():
    c = tiny_cfg()
    w = tiny_weights(c)
    dr = O.Drafter(c, w)
    kv = RNG.standard_normal((7, c["d_stack"]))
    Kc, Vc = dr.ca_kv(kv)
    assert Kc.shape == (7, c["ca_hkv"], c["head_dim"])
    xs = RNG.standard_normal((3, c["d_model"]))
    outs = [dr.ca_block(x, Kc, Vc) for x in xs]
    # Property "input-independence": a row's result ignores the other rows
    assert np.allclose(dr.ca_block(xs[1], Kc, Vc), outs[1], atol=0)
    # a single cached entry: attention returns exactly its value projection
    w1 = dict(w); w1["ca_wdown"] = 0 * w["ca_wdown"]
    dr1 = O.Drafter(c, w1)
    v = O.linear(O.rmsnorm(kv[0], w["ca_normkv"], c["rms_eps"]), w["ca_wv"]).reshape(c["ca_hkv"], c["head_dim"])
    o = np.concatenate([v[h // (c["ca_hq"] // c["ca_hkv"])] for h in range(c["ca_hq"])])
    assert np.allclose(dr1.ca_block(xs[0], Kc[:1], Vc[:1]), xs[0] + O.linear(o, w["ca_wo"]), atol=1e-12)
    # unmasked: every cached entry influences the result
    base = dr.ca_block(xs[0], Kc, Vc)
    for j in range(7):
        V2 = Vc.copy(); V2[j] += 1.0
        assert np.max(np.abs(dr.ca_block(xs[0], Kc, V2) - base)) > 1e-9


# ------------------------------------------------------------------ SA / tree
def test_sa_causal_mask_matches_figure():
    """x of token i depends on token j iff j <= i (Figure 2, middle grid)."""
    c = tiny_cfg()
    dr = O.Drafter(c, tiny_weights(c))
    Kc, Vc = dr.ca_kv(RNG.standard_normal((2, c["d_stack"])))
    toks = [3, 7, 1, 20, 5, 11, 2, 9, 14, 6]
    base = np.stack([o["x"] for o in O.sequential_decode(dr, [], toks, Kc, Vc, 1)])
    dep = np.zeros((10, 10), np.uint8)
    for j in range(10):
        t2 = list(toks); t2[j] = (t2[j] + 1) % c["vocab"]
        x2 = np.stack([o["x"] for o in O.sequential_decode(dr, [], t2, Kc, Vc, 1)])
        dep[:, j] = np.any(np.abs(x2 - base) > 1e-9, axis=-1)
    assert np.array_equal(dep, read_grid("mask_sa_10x10.txt"))


def _tree_setup(B=2, D=3, m=5, vocab=8, seed=3):
    c = tiny_cfg(vocab=vocab)
    w = tiny_weights(c, scale=0.6, rng=np.random.default_rng(seed))
    dr = O.Drafter(c, w)
    prefix = [1, 4, 2, 7, 0]
    saK, saV = dr.sa_prefix(prefix)
    caK, caV = dr.ca_kv(np.random.default_rng(seed + 1).standard_normal((4, c["d_stack"])))
    return c, dr, prefix, saK, saV, caK, caV


@pytest.mark.parametrize("B,D,m", [(2, 3, 5), (3, 4, 16), (1, 4, 3)])
def test_tree_paths_equal_sequential_causal_decoding(B, D, m):
    """Brute force: every forwarded node's output equals plain causal decoding
    of root + path; every pool node's score equals the sum of sequentially
    recomputed log-probs along its path."""
    c, dr, prefix, saK, saV, caK, caV = _tree_setup(B, D, m)
    root = 5
    ts, steps = O.draft_tree(dr, root, saK, saV, caK, caV, B, D, m)
    # replay the frontier history to know which node each forwarded row was
    ts2 = O.TreeState(root, B, D, m)
    for s in range(D):
        for r, f in enumerate(ts2.frontier):
            path = [root] + [ts.tok[i] for i in ts.path_to(f)] if f >= 0 else [root]
            seq = O.sequential_decode(dr, prefix, path, caK, caV, B)[-1]
            assert np.allclose(seq["x"], steps[s][r]["x"], atol=1e-11)
            assert np.allclose(seq["o_hat"], steps[s][r]["o_hat"], atol=1e-11)
            assert np.array_equal(seq["ids"], steps[s][r]["ids"])
        O.tree_expand(ts2, [r["ids"] for r in steps[s]], [r["logp"] for r in steps[s]])
    assert ts2.tok == ts.tok and ts2.parent == ts.parent
    for i in range(len(ts.tok)):
        path = [ts.tok[j] for j in ts.path_to(i)]
        outs = O.sequential_decode(dr, prefix, [root] + path[:-1], caK, caV, c["vocab"])
        total = 0.0
        for o, t in zip(outs, path):
            total += float(o["logp"][list(o["ids"]).index(t)])
        assert abs(total - float(ts.score[i])) < 1e-5


# ------------------------------------------------------------------ Target Layer Inference
def tli_cfg(n_tli=2, **kw):
    return tiny_cfg(n_tli=n_tli, tli_hq=4, tli_hkv=2, tli_mlp=10, **kw)


def tli_weights(c, rng, scale=0.5):
    E, dh = c["d_model"], c["head_dim"]
    w = {}
    for l in range(c["n_tli"]):
        shp = {"norm1": (E,), "wq": (c["tli_hq"] * dh, E), "wk": (c["tli_hkv"] * dh, E), "wv": (c["tli_hkv"] * dh, E),
               "wo": (E, c["tli_hq"] * dh), "norm2": (E,), "wgate": (c["tli_mlp"], E), "wup": (c["tli_mlp"], E),
               "wdown": (E, c["tli_mlp"])}
        for k, s in shp.items():
            w[f"tli{l}_{k}"] = (1.0 + 0.1 * rng.standard_normal(s)) if len(s) == 1 else scale * rng.standard_normal(s)
    return w


def _tli_setup(B, D, m, n_tli=2, seed=5, vocab=8):
    c = tli_cfg(n_tli, vocab=vocab)
    rng = np.random.default_rng(seed)
    w = tiny_weights(c, scale=0.6, rng=rng)
    w.update(tli_weights(c, rng))
    dr = O.Drafter(c, w)
    prefix = [1, 4, 2, 7, 0]
    saK, saV = dr.sa_prefix(prefix)
    caK, caV = dr.ca_kv(rng.standard_normal((4, c["d_stack"])))
    tliK = [rng.standard_normal((len(prefix), c["tli_hkv"], c["head_dim"])) for _ in range(n_tli)]
    tliV = [rng.standard_normal((len(prefix), c["tli_hkv"], c["head_dim"])) for _ in range(n_tli)]
    return c, w, dr, prefix, saK, saV, caK, caV, tliK, tliV


def test_tli_layer_equals_causal_library_attention_over_a_sequence():
    """Special case that reduces to library routines (Section 3.2: f^l_decoder is a plain LLM decoder
    layer): feeding a sequence row by row with a growing cache equals one pass of torch's causal
    scaled_dot_product_attention, with the rotation written as a complex multiplication."""
    import torch
    c = tli_cfg(1)
    rng = np.random.default_rng(21)
    w = tli_weights(c, rng)
    dr = O.Drafter(c, w)
    E, dh, hq, hkv, n, p0 = c["d_model"], c["head_dim"], c["tli_hq"], c["tli_hkv"], 7, 3
    X = rng.standard_normal((n, E))
    K = np.zeros((0, hkv, dh)); V = np.zeros((0, hkv, dh))
    got = []
    for t in range(n):
        o, k, v = dr.tli_layer(0, X[t], p0 + t, K, V)
        K = np.concatenate([K, k[None]]); V = np.concatenate([V, v[None]])
        got.append(o)
    got = np.stack(got)
    T = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    x = T(X)
    def norm(a, g): return a * torch.rsqrt((a * a).mean(-1, keepdim=True) + c["rms_eps"]) * T(g)
    def rot(a):                                  # [n, H, dh]; pairs (i, i + dh/2) as one complex number
        z = torch.complex(a[..., :dh // 2], a[..., dh // 2:])
        pos = torch.arange(p0, p0 + n, dtype=torch.float64)[:, None, None]
        ang = pos * c["rope_theta"] ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
        z = z * torch.polar(torch.ones_like(ang), ang)
        return torch.cat([z.real, z.imag], -1)
    u = norm(x, w["tli0_norm1"])
    q = rot((u @ T(w["tli0_wq"]).T).view(n, hq, dh)).transpose(0, 1)
    k = rot((u @ T(w["tli0_wk"]).T).view(n, hkv, dh)).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    v = (u @ T(w["tli0_wv"]).T).view(n, hkv, dh).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(0, 1).reshape(n, hq * dh)
    a = x + o @ T(w["tli0_wo"]).T
    u2 = norm(a, w["tli0_norm2"])
    ref = a + (torch.nn.functional.silu(u2 @ T(w["tli0_wgate"]).T) * (u2 @ T(w["tli0_wup"]).T)) @ T(w["tli0_wdown"]).T
    assert np.allclose(got, ref.numpy(), atol=1e-10)


def test_tli_zero_output_projections_make_the_layers_the_identity():
    """With W_o = 0 and W_down = 0 every decoder layer returns its input, so TLI = N must give exactly the
    TLI = 0 drafter (Section 3.2: TLI = 0 is the plain architecture)."""
    c, w, dr, prefix, saK, saV, caK, caV, tliK, tliV = _tli_setup(2, 3, 5)
    w0 = dict(w)
    for l in range(c["n_tli"]):
        w0[f"tli{l}_wo"] = np.zeros_like(w[f"tli{l}_wo"])
        w0[f"tli{l}_wdown"] = np.zeros_like(w[f"tli{l}_wdown"])
    ts_a, st_a = O.draft_tree(O.Drafter(c, w0), 5, saK, saV, caK, caV, 2, 3, 5, tliK=tliK, tliV=tliV)
    ts_b, st_b = O.draft_tree(O.Drafter(tiny_cfg(vocab=8), w), 5, saK, saV, caK, caV, 2, 3, 5)
    assert ts_a.tok == ts_b.tok and ts_a.parent == ts_b.parent
    for sa, sb in zip(st_a, st_b):
        for ra, rb in zip(sa, sb):
            assert np.array_equal(ra["o_hat"], rb["o_hat"]) and np.array_equal(ra["logp"], rb["logp"])
    # and with the real weights the layers do change the result
    ts_c, st_c = O.draft_tree(dr, 5, saK, saV, caK, caV, 2, 3, 5, tliK=tliK, tliV=tliV)
    assert not np.allclose(st_c[0][0]["o_hat"], st_b[0][0]["o_hat"])


@pytest.mark.parametrize("B,D,m,n_tli", [(2, 3, 5, 2), (3, 3, 9, 1)])
def test_tli_tree_paths_equal_sequential_decoding(B, D, m, n_tli):
    """Brute force (Section 3.2 with Section 2.2's tree): every forwarded node's LM-head input equals plain
    causal decoding of root + path through SA, CA and the TLI layers, each layer seeing the LLM's cache of
    that layer and the drafted ancestors' keys / values only."""
    c, w, dr, prefix, saK, saV, caK, caV, tliK, tliV = _tli_setup(B, D, m, n_tli)
    root = 5
    ts, steps = O.draft_tree(dr, root, saK, saV, caK, caV, B, D, m, tliK=tliK, tliV=tliV)
    ts2 = O.TreeState(root, B, D, m)
    for s in range(D):
        for r, f in enumerate(ts2.frontier):
            path = [root] + [ts.tok[i] for i in ts.path_to(f)] if f >= 0 else [root]
            seq = O.sequential_decode(dr, prefix, path, caK, caV, B, tliK, tliV)[-1]
            assert np.allclose(seq["o_hat"], steps[s][r]["o_hat"], atol=1e-11)
            assert np.array_equal(seq["ids"], steps[s][r]["ids"])
        O.tree_expand(ts2, [r["ids"] for r in steps[s]], [r["logp"] for r in steps[s]])
    assert ts2.tok == ts.tok
    # a sibling's keys / values are invisible: perturbing one frontier node's token leaves its siblings' rows alone
    # (checked through the prefix cache instead: changing layer 1's cache changes the result, layer order matters)
    tliK2 = [k.copy() for k in tliK]
    tliK2[-1][0] += 1.0
    _, steps2 = O.draft_tree(dr, root, saK, saV, caK, caV, B, D, m, tliK=tliK2, tliV=tliV)
    assert not np.allclose(steps2[0][0]["o_hat"], steps[0][0]["o_hat"])
    assert np.allclose(steps2[0][0]["x"], steps[0][0]["x"])


@pytest.mark.parametrize("B,D,m", [(2, 3, 5), (4, 4, 16), (10, 6, 60), (8, 6, 62), (3, 2, 50)])
def test_tree_bookkeeping_invariants(B, D, m):
    """Pool size B + (D-1) B^2 (Section 2.2); well-formed parents; kept set."""
    rng = np.random.default_rng(B * 100 + D)
    ts = O.TreeState(99, B, D, m)
    for s in range(D):
        R = len(ts.frontier)
        assert R == (1 if s == 0 else B)
        logp = -np.sort(rng.exponential(1.0, (R, B)), axis=-1).astype(np.float32)
        ids = rng.integers(0, 1000, (R, B))
        O.tree_expand(ts, ids, logp)
    n_pool = B + (D - 1) * B * B
    assert len(ts.tok) == n_pool
    for i in range(n_pool):
        p = ts.parent[i]
        assert p < i
        assert ts.depth[i] == (1 if p < 0 else ts.depth[p] + 1)
        assert p < 0 or ts.score[i] <= ts.score[p]
    tok, parent, depth, score = O.tree_finalize(ts)
    n = len(tok)
    assert n == min(m, n_pool) + 1 and parent[0] == -1 and depth[0] == 0 and tok[0] == 99
    assert np.all(parent[1:] < np.arange(1, n)) and np.all(parent[1:] >= 0)      # ancestor-closed, ordered
    assert np.all(depth[1:] == depth[parent[1:]] + 1)
    assert np.all(depth <= 255)                     # a tree position fits the paper's one byte
    # the kept scores are the largest of the pool
    if n_pool > m:
        worst_kept = np.min(score[1:])
        assert np.sum(np.array(ts.score) > worst_kept) <= m
    mask = O.tree_mask(parent)
    assert np.all(mask[:, 0] == 1) and np.all(np.diag(mask) == 1)
    assert np.array_equal(mask.sum(1), depth + 1)   # a node sees exactly its depth+1 ancestors-or-self
    assert np.all(np.triu(mask, 1) == 0)
    for i in range(1, n):
        assert np.array_equal(mask[i] - np.eye(n, dtype=np.uint8)[i], mask[parent[i]])


def test_tree_expand_frontier_and_ties_by_hand():
    ts = O.TreeState(0, 2, 2, 3)
    O.tree_expand(ts, [[10, 11]], [[-0.5, -1.0]])
    assert ts.tok == [10, 11] and ts.parent == [-1, -1] and ts.frontier == [0, 1]
    O.tree_expand(ts, [[20, 21], [22, 23]], [[-0.25, -2.0], [-0.25, -0.5]])
    # scores: -0.75, -2.5, -1.25, -1.5 -> frontier = nodes 2, 4
    assert [float(s) for s in ts.score] == [-0.5, -1.0, -0.75, -2.5, -1.25, -1.5]
    assert ts.frontier == [2, 4] and ts.parent[2:] == [0, 0, 1, 1]
    tok, parent, depth, score = O.tree_finalize(ts)
    assert tok.tolist() == [0, 10, 11, 20] and parent.tolist() == [-1, 0, 0, 1] and depth.tolist() == [0, 1, 1, 2]
    # exact ties: the lower pool index wins both in the frontier and in the final cut
    ts = O.TreeState(0, 2, 2, 2)
    O.tree_expand(ts, [[1, 2]], [[-1.0, -1.0]])
    O.tree_expand(ts, [[3, 4], [5, 6]], [[-0.0, -1.0], [-0.0, -1.0]])
    assert ts.frontier == [2, 4]
    assert O.tree_finalize(ts)[0].tolist() == [0, 1, 2]
    assert O.tree_mask([-1, 0, 0, 1, 3, 2]).tolist() == [
        [1, 0, 0, 0, 0, 0], [1, 1, 0, 0, 0, 0], [1, 0, 1, 0, 0, 0],
        [1, 1, 0, 1, 0, 0], [1, 1, 0, 1, 1, 0], [1, 0, 1, 0, 0, 1]]


def test_chain_case_equals_greedy_loop():
    """A tree with B = 1 is chain drafting: same tokens as the greedy inner loop of Algorithm 1."""
    c, dr, prefix, saK, saV, caK, caV = _tree_setup(1, 4, 4, vocab=12)
    ts, _ = O.draft_tree(dr, 5, saK, saV, caK, caV, 1, 4, 4)
    toks, lps = O.greedy_chain(dr, prefix, 5, caK, caV, 4)
    assert ts.tok == toks
    assert np.allclose(np.cumsum(np.float32(lps)), np.array(ts.score), atol=1e-5)
    tok, parent, depth, _ = O.tree_finalize(ts)
    assert parent.tolist() == [-1, 0, 1, 2, 3] and depth.tolist() == [0, 1, 2, 3, 4]
    assert np.array_equal(O.tree_mask(parent), np.tril(np.ones((5, 5), np.uint8)))


def test_fp32_inputs_agree_with_fp64():
    c = tiny_cfg()
    w = tiny_weights(c)
    w32 = {k: v.astype(np.float32) for k, v in w.items()}
    H = RNG.standard_normal((2, c["n_stack"], c["d_stack"]))
    a = O.Drafter(c, w).lsa_forward(H)
    b = O.Drafter(c, w32).lsa_forward(H.astype(np.float32))
    assert np.max(np.abs(a - b)) < 1e-5 * np.max(np.abs(a))


# ------------------------------------------------------------------ verification (greedy acceptance)
def _random_tree(rng, n, vocab, width=3):
    """A random kept tree: parent[i] < i, sibling tokens distinct."""
    tok, parent = [int(rng.integers(vocab))], [-1]
    for i in range(1, n):
        for _ in range(100):
            q = int(rng.integers(0, i))
            t = int(rng.integers(vocab))
            sibs = [tok[c] for c in range(1, i) if parent[c] == q]
            if t not in sibs and len(sibs) < width:
                break
        tok.append(t)
        parent.append(q)
    return tok, parent


@pytest.mark.parametrize("seed", range(12))
def test_verify_greedy_equals_token_by_token_greedy_decoding(seed):
    """Brute force (Section 2.2, step 2: discard everything after the first mismatch): with an LLM that is a
    deterministic function of the token path, the accepted tokens are the longest prefix of the LLM's own greedy
    continuation that exists in the tree as a root path, and the bonus token is the continuation's next token."""
    rng = np.random.default_rng(seed)
    vocab, n = 5, 30
    tok, parent = _random_tree(rng, n, vocab)
    table = {}
    def llm_logits(path):                     # a fixed random logit row per token path
        if path not in table:
            table[path] = np.random.default_rng(hash(path) % (2 ** 32)).standard_normal(vocab)
        return table[path]
    def path_of(i):
        p = []
        while i >= 0:
            p.append(tok[i]); i = parent[i]
        return tuple(reversed(p))
    logits = np.stack([llm_logits(path_of(i)) for i in range(n)])
    slots, nxt, choice = O.verify_greedy(tok, parent, logits)
    # token-by-token greedy decoding from the root, no tree involved
    seq = [tok[0]]
    paths = {path_of(i) for i in range(n)}
    while True:
        g = int(np.argmax(llm_logits(tuple(seq))))
        if tuple(seq + [g]) in paths:
            seq.append(g)
        else:
            bonus = g
            break
    assert [tok[i] for i in slots] == seq
    assert nxt == bonus
    assert slots[0] == 0 and all(parent[b] == a for a, b in zip(slots, slots[1:]))
    assert choice == [int(np.argmax(r)) for r in logits]


def test_verify_greedy_special_cases():
    """A chain whose every token is the LLM's choice is accepted whole; a wrong first token rejects everything;
    ties go to the smaller token id; unused slots (parent < 0) never match."""
    V = 6
    tok, parent = [2, 4, 1, 3], [-1, 0, 1, 2]
    z = np.full((4, V), -1.0)
    z[0, 4] = z[1, 1] = z[2, 3] = z[3, 5] = 2.0
    slots, nxt, _ = O.verify_greedy(tok, parent, z)
    assert slots == [0, 1, 2, 3] and nxt == 5
    z2 = z.copy(); z2[0, 4] = -1.0; z2[0, 0] = 3.0
    assert O.verify_greedy(tok, parent, z2)[:2] == ([0], 0)
    z3 = z.copy(); z3[0, 1] = 2.0                       # tie between ids 1 and 4 at the root: id 1 wins, no child has it
    assert O.verify_greedy(tok, parent, z3)[:2] == ([0], 1)
    tok5, parent5 = [2, 4, 4], [-1, -1, 0]              # slot 1 unused; slot 2 is the real child
    assert O.verify_greedy(tok5, parent5, z[:3])[0] == [0, 2]


# ------------------------------------------------------------------ client-server message codec
def test_pack_tree_layout_size_and_round_trip():
    """4 bytes per node (the message-size table's 4M for a tree of M nodes): 3 little-endian token bytes and
    the parent slot; pack and unpack are inverse on every valid tree."""
    msg = O.pack_tree([0x123456, 7, -1], [-1, 0, -1])
    assert msg.dtype == np.uint8 and msg.shape == (3, 4) and msg.nbytes == 4 * 3
    assert msg.tolist() == [[0x56, 0x34, 0x12, 255], [7, 0, 0, 0], [255, 255, 255, 255]]
    rng = np.random.default_rng(2)
    for _ in range(20):
        tok, parent = _random_tree(rng, 61, 128256, width=10)
        t2, p2 = O.unpack_tree(O.pack_tree(tok, parent))
        assert t2.tolist() == tok and p2.tolist() == parent


def test_quantize_rows_bounds_and_fixed_points():
    """Closed forms: |x - dequant| <= scale / 2 (up to the fp32 rounding of the row's reciprocal); the row's largest magnitude maps to +-127 exactly; codes stay
    in [-127, 127]; an all-zero row gives zeros; quantising a dequantised row returns the same codes; a row that
    is already k * s for integers |k| <= 127 (max 127) is reproduced exactly."""
    rng = np.random.default_rng(4)
    x = (rng.standard_normal((50, 333)) * rng.uniform(0.01, 30, (50, 1))).astype(np.float32)
    x[7] = 0
    q, s = O.quantize_rows(x)
    d = O.dequantize_rows(q, s)
    assert q.dtype == np.int8 and s.dtype == np.float32 and int(np.abs(q.astype(int)).max()) == 127
    assert np.all(np.abs(x - d) <= s[:, None] * (0.5 + 1e-4))       # half a step, plus the rounding of the reciprocal
    am = np.argmax(np.abs(x), axis=1)
    rows = np.arange(50)
    assert np.all(np.abs(q[rows, am])[s > 0] == 127)
    assert np.all(q[7] == 0) and s[7] == 0 and np.all(d[7] == 0)
    q2, s2 = O.quantize_rows(d)
    assert np.array_equal(q2, q)
    k = rng.integers(-127, 128, (4, 64)); k[:, 0] = 127
    y = (k * np.float32(0.25)).astype(np.float32)
    qy, sy = O.quantize_rows(y)
    assert np.array_equal(qy, k) and np.all(sy == np.float32(0.25)) and np.array_equal(O.dequantize_rows(qy, sy), y)


# ------------------------------------------------------------------ whole-sequence drafter pass
def test_drafter_prefill_equals_token_by_token_decoding_and_the_ca_mask_of_the_figure():
    """With every cached LLM position visible the one-pass drafter equals plain causal decoding token by token;
    with the K-step-bounded limits of the mask figure (K = 4 then K = 3 after a 3-token prompt) row j of the
    output depends on LLM activation i exactly where the figure's cross-attention grid (as its caption states it)
    is filled, and on token i exactly where the self-attention grid is."""
    c = tiny_cfg()
    dr = O.Drafter(c, tiny_weights(c))
    rng = np.random.default_rng(9)
    kv = rng.standard_normal((10, c["d_stack"]))
    toks = [3, 7, 1, 20, 5, 11, 2, 9, 14, 6]
    Kc, Vc = dr.ca_kv(kv)
    empty = np.zeros((0, c["sa_hkv"], c["head_dim"]))
    full, K, V = O.drafter_prefill(dr, toks, empty, empty, Kc, Vc)
    seq = O.sequential_decode(dr, [], toks, Kc, Vc, 1)
    assert np.allclose(full, np.stack([o["o_hat"] for o in seq]), atol=1e-12)
    assert np.allclose(K[-1], seq[-1]["k"], atol=1e-12) and K.shape[0] == 10
    # a prefix handed in as a cache gives the same as decoding it first
    pre, Kp, Vp = O.drafter_prefill(dr, toks[:4], empty, empty, Kc, Vc)
    rest, _, _ = O.drafter_prefill(dr, toks[4:], Kp, Vp, Kc, Vc)
    assert np.allclose(np.concatenate([pre, rest]), full, atol=1e-12)
    # the figure's limits: prompt rows causal, then K = 4 rows on 3 activations, then K = 3 rows on 7
    limits = [1, 2, 3, 3, 3, 3, 3, 7, 7, 7]
    base, _, _ = O.drafter_prefill(dr, toks, empty, empty, Kc, Vc, limits)
    dep = np.zeros((10, 10), np.uint8)
    for i in range(10):
        kv2 = kv.copy(); kv2[i] += 1.0
        K2, V2 = dr.ca_kv(kv2)
        out2, _, _ = O.drafter_prefill(dr, toks, empty, empty, K2, V2, limits)
        dep[:, i] = np.any(np.abs(out2 - base) > 1e-9, axis=-1)
    assert np.array_equal(dep, read_grid("mask_ca_10x10.txt"))
    dep_t = np.zeros((10, 10), np.uint8)
    for i in range(10):
        t2 = list(toks); t2[i] = (t2[i] + 1) % c["vocab"]
        out2, _, _ = O.drafter_prefill(dr, t2, empty, empty, Kc, Vc, limits)
        dep_t[:, i] = np.any(np.abs(out2 - base) > 1e-9, axis=-1)
    assert np.array_equal(dep_t, read_grid("mask_sa_10x10.txt"))


# ------------------------------------------------------------------ whole-block recomputations (MLP legs on)
def _T(a):
    return torch.tensor(np.asarray(a), dtype=torch.float64)


def _t_norm(a, g, eps):
    return a * torch.rsqrt((a * a).mean(-1, keepdim=True) + eps) * _T(g)


def _t_mlp(u, w, block):
    return (torch.nn.functional.silu(u @ _T(w[block + "_wgate"]).T) * (u @ _T(w[block + "_wup"]).T)) @ _T(w[block + "_wdown"]).T


def _t_rot(a, pos, theta):
    """[n, H, dh] rotated at positions pos [n]: the pair (i, i + dh/2) as one complex number times e^{i pos theta_i}."""
    dh = a.shape[-1]
    z = torch.complex(a[..., :dh // 2], a[..., dh // 2:])
    ang = pos[:, None, None] * theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    z = z * torch.polar(torch.ones_like(ang), ang)
    return torch.cat([z.real, z.imag], -1)


def _lsa_block_library(c, w, X):
    """Section 3.1.1 as a decoder layer over the layer axis, written with torch routines only."""
    S, dh, hq, hkv, eps = X.shape[0], c["head_dim"], c["lsa_hq"], c["lsa_hkv"], c["rms_eps"]
    x = _T(X)
    u = _t_norm(x, w["lsa_norm1"], eps)
    q = (u @ _T(w["lsa_wq"]).T).view(S, hq, dh).transpose(0, 1)
    k = (u @ _T(w["lsa_wk"]).T).view(S, hkv, dh).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    v = (u @ _T(w["lsa_wv"]).T).view(S, hkv, dh).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v).transpose(0, 1).reshape(S, hq * dh)
    y = x + o @ _T(w["lsa_wo"]).T
    return (y + _t_mlp(_t_norm(y, w["lsa_norm2"], eps), w, "lsa")).numpy()


def _sa_block_library(c, w, toks, p0):
    """Section 3.1.2 "Self-Attention" over a token sequence at positions p0, p0+1, ...: one causal pass."""
    n, dh, hq, hkv, eps = len(toks), c["head_dim"], c["sa_hq"], c["sa_hkv"], c["rms_eps"]
    e = _T(w["embed"])[torch.tensor(toks)]
    u = _t_norm(e, w["sa_norm1"], eps)
    pos = torch.arange(p0, p0 + n, dtype=torch.float64)
    q = _t_rot((u @ _T(w["sa_wq"]).T).view(n, hq, dh), pos, c["rope_theta"]).transpose(0, 1)
    k = _t_rot((u @ _T(w["sa_wk"]).T).view(n, hkv, dh), pos, c["rope_theta"]).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    v = (u @ _T(w["sa_wv"]).T).view(n, hkv, dh).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(0, 1).reshape(n, hq * dh)
    a = e + o @ _T(w["sa_wo"]).T
    return (a + _t_mlp(_t_norm(a, w["sa_norm2"], eps), w, "sa")).numpy()


def _ca_block_library(c, w, xs, kv):
    """Section 3.1.2 "Cross-Attention": queries from the rows xs, keys / values from the LSA outputs kv, no mask."""
    n, m, dh, hq, hkv, eps = xs.shape[0], kv.shape[0], c["head_dim"], c["ca_hq"], c["ca_hkv"], c["rms_eps"]
    x = _T(xs)
    ukv = _t_norm(_T(kv), w["ca_normkv"], eps)
    q = (_t_norm(x, w["ca_normq"], eps) @ _T(w["ca_wq"]).T).view(n, hq, dh).transpose(0, 1)
    k = (ukv @ _T(w["ca_wk"]).T).view(m, hkv, dh).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    v = (ukv @ _T(w["ca_wv"]).T).view(m, hkv, dh).transpose(0, 1).repeat_interleave(hq // hkv, 0)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v).transpose(0, 1).reshape(n, hq * dh)
    cc = x + o @ _T(w["ca_wo"]).T
    return (cc + _t_mlp(_t_norm(cc, w["ca_norm2"], eps), w, "ca")).numpy()


def _oracle_sa_rows(dr, toks, p0):
    """The oracle's SA block fed token by token with a growing key / value set."""
    c = dr.c
    K = np.zeros((0, c["sa_hkv"], c["head_dim"])); V = np.zeros((0, c["sa_hkv"], c["head_dim"]))
    out = []
    for i, t in enumerate(toks):
        e, q, k, v = dr.sa_qkv(t, p0 + i)
        K = np.concatenate([K, k[None]]); V = np.concatenate([V, v[None]])
        out.append(dr.sa_block(e, q, K, V))
    return np.stack(out)


def _block_pin_inputs():
    c = tiny_cfg(n_stack=5)
    rng = np.random.default_rng(77)
    w = tiny_weights(c, scale=0.5, rng=rng)            # every matrix non-zero, every gain different from 1
    X = rng.standard_normal((c["n_stack"], c["d_stack"])) * 1.5
    toks, p0 = [3, 17, 5, 5, 22, 0, 9], 4
    xs = rng.standard_normal((3, c["d_model"]))
    kv = rng.standard_normal((4, c["d_stack"]))
    return c, w, X, toks, p0, xs, kv


def test_lsa_block_with_mlp_equals_library_recomputation():
    """The whole LSA block of one token, attention and MLP legs both on, against torch (Section 3.1.1; the
    6144-wide MLP of the hyper-parameter table): pins the second pre-norm (on Y, with its own gain), the SwiGLU
    leg and both residuals."""
    c, w, X, *_ = _block_pin_inputs()
    assert np.allclose(O.Drafter(c, w).lsa_rows(X), _lsa_block_library(c, w, X), atol=1e-10)


def test_sa_block_with_mlp_equals_causal_library_attention_over_a_sequence():
    """sa_qkv + sa_block over a short sequence against one causal torch pass with the rotation as a complex
    product (Section 3.1.2 "Self-Attention"): pins the pre-norm gain, the rotation of q and k but not v, the
    residual from the embedding, the second pre-norm and the MLP leg."""
    c, w, _, toks, p0, *_ = _block_pin_inputs()
    assert np.allclose(_oracle_sa_rows(O.Drafter(c, w), toks, p0), _sa_block_library(c, w, toks, p0), atol=1e-10)


def test_ca_block_with_mlp_and_several_keys_equals_library_recomputation():
    """ca_kv + ca_block with four cached entries against torch (Section 3.1.2 "Cross-Attention"): with more than
    one key the query leg (its own norm gain and W_q) matters; the MLP leg is on."""
    c, w, _, _, _, xs, kv = _block_pin_inputs()
    dr = O.Drafter(c, w)
    Kc, Vc = dr.ca_kv(kv)
    got = np.stack([dr.ca_block(x, Kc, Vc) for x in xs])
    assert np.allclose(got, _ca_block_library(c, w, xs, kv), atol=1e-10)


def test_block_pins_catch_planted_mistakes():
    """Each plausible slip, planted in a copy of the oracle on the CPU, must break one of the three pins above."""
    c, w, X, toks, p0, xs, kv = _block_pin_inputs()

    class MlpNormsX(O.Drafter):                      # MLP leg normalises X instead of Y
        def lsa_rows(self, X):
            self._x = np.asarray(X, np.float64)
            return super().lsa_rows(X)

        def mlp(self, u, block):
            if block == "lsa":
                u = O.rmsnorm(self._x, self.w("lsa_norm2"), self.c["rms_eps"])
            return super().mlp(u, block)

    class MlpUsesNorm1(O.Drafter):                   # MLP pre-norm takes the attention pre-norm's gain
        def w(self, name):
            return super().w("lsa_norm1" if name == "lsa_norm2" else name)

    class RotatesV(O.Drafter):                       # v rotated like k
        def sa_qkv(self, tok, pos):
            e, q, k, v = super().sa_qkv(tok, pos)
            return e, q, k, O.rope(v, pos, self.c["rope_theta"])

    class SaWrongGain(O.Drafter):
        def w(self, name):
            return super().w("sa_norm2" if name == "sa_norm1" else name)

    class SaDropsResidual(O.Drafter):                # a = W_o o without the embedding
        def sa_block(self, e, q, K, V):
            return super().sa_block(np.zeros_like(e), q, K, V)

    class CaQueryGain(O.Drafter):                    # query pre-norm uses the MLP pre-norm's gain
        def w(self, name):
            return super().w("ca_norm2" if name == "ca_normq" else name)

    class CaQueryTransposedHeads(O.Drafter):         # W_q rows permuted: heads read in the wrong order
        def w(self, name):
            m = super().w(name)
            return m[::-1] if name == "ca_wq" else m

    lsa_ref, sa_ref, ca_ref = _lsa_block_library(c, w, X), _sa_block_library(c, w, toks, p0), _ca_block_library(c, w, xs, kv)
    for cls in (MlpNormsX, MlpUsesNorm1):
        assert not np.allclose(cls(c, w).lsa_rows(X), lsa_ref, atol=1e-6), cls.__name__
    for cls in (RotatesV, SaWrongGain, SaDropsResidual):
        assert not np.allclose(_oracle_sa_rows(cls(c, w), toks, p0), sa_ref, atol=1e-6), cls.__name__
    for cls in (CaQueryGain, CaQueryTransposedHeads):
        dr = cls(c, w)
        Kc, Vc = dr.ca_kv(kv)
        assert not np.allclose(np.stack([dr.ca_block(x, Kc, Vc) for x in xs]), ca_ref, atol=1e-6), cls.__name__
