"""Parity of the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances: hidden states and log-probabilities within
max-abs 1e-4 (fp32 path) / 2e-2 (bf16 path) of the row's max |value|; token ids and tree structure
bit-exact except where the oracle's competing log-probabilities differ by less than the tie window
(1e-3 on the fp32 path; helpers.tie_window derives the bf16 ones). bf16 forwards of up to 256 rows (every draft
step) carry their activations as two bf16 terms, so their top-B decisions are compared with the unrounded fp64
oracle directly; larger bf16 passes (plain 16-bit activations) would be compared with the oracle in its
bf16-storage mode, their values with the unrounded oracle.
"""
import numpy as np
import pytest
import torch

from oracle import moa_oracle as O
from paper_2410_03804_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def oracle_cycle(p, dr, h_stack, prompt, root, ca_cache, sa_cache, forced=None, seqs=None, tli_cache=None):
    """The oracle's side of one drafting cycle, for the sequences listed in seqs (default: all).
    forced[b] = per-step (ids, logp) to expand with. Per-sequence results are dicts keyed by b."""
    nb = p.batch
    seqs = list(range(nb)) if seqs is None else list(seqs)
    out = {"kv": {}, "caK": {}, "caV": {}, "saK": {}, "saV": {}, "trees": {}}
    for b in seqs:
        if ca_cache is None:
            n = h_stack.shape[0] // nb
            out["kv"][b] = dr.lsa_forward(H.np32(h_stack[b * n:(b + 1) * n]))
            out["caK"][b], out["caV"][b] = dr.ca_kv(out["kv"][b])
        else:
            out["caK"][b], out["caV"][b] = H.np32(ca_cache[0][b]), H.np32(ca_cache[1][b])
        if sa_cache is None:
            out["saK"][b], out["saV"][b] = dr.sa_prefix(prompt[b].tolist())
        else:
            out["saK"][b], out["saV"][b] = H.np32(sa_cache[0][b]), H.np32(sa_cache[1][b])
        out["trees"][b] = O.draft_tree(dr, int(root[b]), out["saK"][b], out["saV"][b], out["caK"][b], out["caV"][b],
                                       p.tree_topk, p.tree_depth, p.tree_keep,
                                       forced=None if forced is None else forced[b],
                                       tliK=None if tli_cache is None else [H.np32(k[b]) for k, _ in tli_cache],
                                       tliV=None if tli_cache is None else [H.np32(v[b]) for _, v in tli_cache])
    return out


def run_cycle(p, g, oracles, h_stack, prompt, root, ca_cache=None, sa_cache=None, seqs=None, tli_cache=None):
    """One drafting cycle on both sides. The tree follows the deciding oracle's top-B (teacher forcing);
    values are compared with the unrounded oracle walking the same tree. With seqs given, the oracle runs
    only on those sequences of the batch (sampled outputs); the others expand with the GPU's own lists."""
    exact, dec = oracles
    tol = H.tol_of(p)
    nb = p.batch
    B, D = p.tree_topk, p.tree_depth
    seqs = list(range(nb)) if seqs is None else list(seqs)
    od = oracle_cycle(p, dec, h_stack, prompt, root, ca_cache, sa_cache, seqs=seqs, tli_cache=tli_cache)
    forced = {b: [([r["ids"] for r in rows], [r["logp"] for r in rows]) for rows in od["trees"][b][1]] for b in seqs}
    ox = od if exact is dec else oracle_cycle(p, exact, h_stack, prompt, root, ca_cache, sa_cache, forced, seqs=seqs,
                                              tli_cache=tli_cache)
    stats = dict(rows=0, exact=0, literal=0, worst_hidden=0.0, worst_logp=0.0)
    literal = []
    if ca_cache is None:
        n_tok = [h_stack.shape[0] // nb] * nb
        n = n_tok[0]
        kv = g.moa_lsa_forward(h_stack.cuda(), n_tok)
        torch.cuda.synchronize()
        stats["lsa"] = 0.0
        for b in seqs:
            stats["lsa"] = max(stats["lsa"], H.assert_rows_close(H.np32(kv[b * n:(b + 1) * n].cpu()), ox["kv"][b], tol,
                                                                 "LSA kv"))
            H.assert_rows_close(H.np32(g.ca_k[b, :n].cpu()), ox["caK"][b], tol, "CA K cache")
            H.assert_rows_close(H.np32(g.ca_v[b, :n].cpu()), ox["caV"][b], tol, "CA V cache")
        assert g.ca_len[:nb].tolist() == n_tok
    else:
        g.fill_cache("ca", ca_cache[0].cuda(), ca_cache[1].cuda())
    if sa_cache is None:
        n = prompt.shape[1]
        g.moa_sa_append(prompt.reshape(-1).cuda(), [n] * nb)
        torch.cuda.synchronize()
        for b in seqs:
            H.assert_rows_close(H.np32(g.sa_k[b, :n].cpu()), ox["saK"][b], tol, "SA K cache")
            H.assert_rows_close(H.np32(g.sa_v[b, :n].cpu()), ox["saV"][b], tol, "SA V cache")
        assert g.sa_len[:nb].tolist() == [n] * nb
    else:
        g.fill_cache("sa", sa_cache[0].cuda(), sa_cache[1].cuda())
    for l, (k, v) in enumerate(tli_cache or []):
        g.fill_tli_cache(l, k.cuda(), v.cuda())
    g.moa_tree_begin(root.cuda())
    outs = None
    for s in range(D):
        ids, lp, hid = g.moa_draft_step(want_hidden=True)
        torch.cuda.synchronize()
        ids, lp, hid = ids.cpu().numpy(), lp.cpu().numpy(), H.np32(hid.cpu())
        rs = 1 if s == 0 else B
        f_ids, f_lp = ids.copy(), lp.copy()          # unsampled sequences follow the GPU's own choices
        for b in seqs:
            for r in range(rs):
                gr = b * rs + r
                rx, rd = ox["trees"][b][1][s][r], od["trees"][b][1][s][r]
                stats["worst_hidden"] = max(stats["worst_hidden"], H.assert_rows_close(
                    hid[gr][None], rx["o_hat"][None], tol, f"hidden s{s} r{gr}"))
                # values against the unrounded oracle, decisions against the deciding oracle
                zx = rx["z"]
                lpx = zx - (zx.max() + np.log(np.exp(zx - zx.max()).sum()))
                lp_err = np.max(np.abs(lp[gr] - lpx[ids[gr]])) / np.max(np.abs(zx))
                stats["worst_logp"] = max(stats["worst_logp"], float(lp_err))
                assert lp_err <= tol, f"logp s{s} r{gr}"
                stats["exact"] += H.check_topk(ids[gr], lp[gr], rd["z"], tol, H.tie_window(p, rd["z"]), f"topk s{s} r{gr}",
                                               literal)
                stats["rows"] += 1
                f_ids[gr] = rd["ids"]
                f_lp[gr] = rd["logp"].astype(np.float32)
        outs = g.moa_tree_expand(torch.from_numpy(f_ids).cuda(), torch.from_numpy(f_lp).cuda())
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0
    tok, parent, depth, score, n = [t.cpu().numpy() for t in outs]
    for b in seqs:
        otok, opar, odep, osc = O.tree_finalize(od["trees"][b][0])
        k = len(otok)
        assert n[b] == k and np.array_equal(tok[b, :k], otok) and np.array_equal(parent[b, :k], opar)
        assert np.array_equal(depth[b, :k], odep) and np.array_equal(score[b, :k].view(np.int32), osc.view(np.int32))
    for b in range(nb):                              # properties that hold for every sequence, sampled or not
        k = int(n[b])
        assert 1 <= k <= p.tree_keep + 1 and parent[b, 0] == -1 and depth[b, 0] == 0
        assert np.all(parent[b, 1:k] < np.arange(1, k)) and np.all(parent[b, 1:k] >= 0)
        assert np.array_equal(depth[b, 1:k], depth[b, parent[b, 1:k]] + 1)
        assert np.all(score[b, 1:k] <= score[b, parent[b, 1:k]])
    stats["literal"] = int(sum(literal))       # rows whose every pick is within 1e-3 of the oracle's pick of that rank
    print(f"[parity {p.name} {p.dtype}] {stats}")
    return stats


def test_c1_full_cycle_fp32():
    """Config 1 end to end: LSA over the 64 prompt tokens, SA prefix, depth-4 / top-4 / keep-16 tree."""
    p = synth.PRESETS["c1"]
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=p.ctx + 8, lsa_chunk_tokens=24)     # 64 tokens -> three ragged passes
    stats = run_cycle(p, g, H.make_oracles(p, w), synth.make_h_stack(p, p.lsa_tokens), synth.make_tokens(p, p.ctx),
                      synth.make_root(p))
    assert stats["rows"] == 1 + 3 * 4
    assert stats["exact"] == stats["rows"]


def test_c1_free_running_tree_matches_oracle():
    """The GPU's own choices (no teacher forcing) give the oracle's tree on config 1."""
    p = synth.PRESETS["c1"]
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=p.ctx + 8, lsa_chunk_tokens=64)
    dr = H.make_oracle(p, w)
    h = synth.make_h_stack(p, p.lsa_tokens)
    prompt, root = synth.make_tokens(p, p.ctx), synth.make_root(p)
    g.moa_lsa_forward(h.cuda(), [p.lsa_tokens], want_kv=False)
    g.moa_sa_append(prompt.reshape(-1).cuda(), [p.ctx])
    g.moa_tree_begin(root.cuda())
    for s in range(p.tree_depth):
        ids, lp, _ = g.moa_draft_step()
        outs = g.moa_tree_expand(ids, lp)
    tok, parent, depth, score, n = [t.cpu().numpy() for t in outs]
    caK, caV = dr.ca_kv(dr.lsa_forward(H.np32(h)))
    saK, saV = dr.sa_prefix(prompt[0].tolist())
    ts, _ = O.draft_tree(dr, int(root[0]), saK, saV, caK, caV, p.tree_topk, p.tree_depth, p.tree_keep)
    otok, opar, odep, osc = O.tree_finalize(ts)
    # near-ties (< 1e-3) could legitimately differ; at this seed there are none
    assert np.array_equal(tok[0, :n[0]], otok) and np.array_equal(parent[0, :n[0]], opar)
    assert np.allclose(score[0, :n[0]], osc, atol=1e-3)
    from paper_2410_03804_b200 import moa
    mask = moa.moa_tree_attn_mask(torch.from_numpy(parent[:, :n[0]].copy()).cuda()).cpu().numpy()
    assert np.array_equal(mask[0], O.tree_mask(opar))


@pytest.mark.parametrize("dtype,batch", [("bf16", 1), ("bf16", 3), ("f32", 2)])
def test_reduced_llama_shape(dtype, batch):
    """A reduced Llama-3-shaped drafter: GQA 8/2 x 128, ragged vocab, several sequences,
    stacked activations with the std ramp and outlier channels of config 2."""
    p = synth.scaled(synth.PRESETS["c2"], d_model=512, n_stack=5, d_stack=384, vocab=5003, lsa_hq=8, lsa_hkv=2,
                     lsa_mlp=768, sa_hq=8, sa_hkv=2, sa_mlp=64, ca_hq=8, ca_hkv=4, ca_mlp=896, ctx=37, batch=batch,
                     tree_topk=5, tree_depth=3, tree_keep=12, dtype=dtype, lsa_tokens=37)
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=64, lsa_chunk_tokens=16)
    stats = run_cycle(p, g, H.make_oracles(p, w), synth.make_h_stack(p, p.lsa_tokens * batch),
                      synth.make_tokens(p, p.ctx), synth.make_root(p))
    assert stats["rows"] == batch * (1 + 2 * 5)


@pytest.mark.parametrize("dtype,batch,n_tli", [("bf16", 2, 2), ("f32", 2, 1), ("bf16", 1, 4)])
def test_target_layer_inference_reduced_llama_shape(dtype, batch, n_tli):
    """Target Layer Inference (Section 3.2): the last n_tli LLM decoder layers (Llama-3-8B head layout, reduced
    widths) run on the drafted rows over synthetic LLM caches of those layers plus the drafted ancestors."""
    p = synth.scaled(synth.PRESETS["c2"], d_model=512, d_stack=512, n_stack=6, vocab=4099, lsa_hq=4, lsa_hkv=2, lsa_mlp=768,
                     sa_hq=4, sa_hkv=2, sa_mlp=64, ca_hq=4, ca_hkv=2, ca_mlp=896, ctx=150, batch=batch, tree_topk=4,
                     tree_depth=4, tree_keep=20, dtype=dtype, lsa_tokens=7, n_tli=n_tli, tli_hq=8, tli_hkv=2,
                     tli_mlp=1408)
    w = synth.make_weights(p)
    w.update(synth.make_tli_weights(p))
    g = H.make_gpu(p, w, max_ctx=p.ctx + 16, lsa_chunk_tokens=16)
    tli_cache = [synth.make_tli_cache(p, l) for l in range(n_tli)]
    stats = run_cycle(p, g, H.make_oracles(p, w), synth.make_h_stack(p, p.lsa_tokens * batch),
                      synth.make_tokens(p, p.ctx), synth.make_root(p), tli_cache=tli_cache)
    assert stats["rows"] == batch * (1 + 3 * 4)
    # the layers are really in the path: without them the drafter's output differs
    g0 = H.make_gpu(synth.scaled(p, n_tli=0), synth.make_weights(p), max_ctx=p.ctx + 16, lsa_chunk_tokens=16)
    g0.moa_sa_append(synth.make_tokens(p, p.ctx).reshape(-1).cuda(), [p.ctx] * batch)
    g0.moa_lsa_forward(synth.make_h_stack(p, p.lsa_tokens * batch).cuda(), [p.lsa_tokens] * batch)
    g0.moa_tree_begin(synth.make_root(p).cuda())
    _, _, h0 = g0.moa_draft_step(want_hidden=True)
    g.moa_tree_begin(synth.make_root(p).cuda())
    _, _, h1 = g.moa_draft_step(want_hidden=True)
    torch.cuda.synchronize()
    assert not torch.allclose(h0.float(), h1.float(), rtol=0, atol=1e-2 * float(h0.float().abs().max()))


def test_maximum_rows_per_step_256():
    """The largest forward the library takes: 16 sequences x breadth 16 = 256 rows (two-term activations as two
    256-row tiles per stage, 64 queries per kv head in the attention, 16-wide top lists), depth 2, reduced widths."""
    p = synth.scaled(synth.PRESETS["c5"], d_model=256, n_stack=2, d_stack=128, vocab=2051, lsa_hq=2, lsa_hkv=2,
                     lsa_mlp=128, sa_hq=4, sa_hkv=1, sa_mlp=64, ca_hq=4, ca_hkv=2, ca_mlp=448, ctx=70, batch=16,
                     tree_topk=16, tree_depth=2, tree_keep=40, lsa_tokens=2)
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=80, lsa_chunk_tokens=32)
    caK, caV = synth.make_cache(p, "ca")
    saK, saV = synth.make_cache(p, "sa")
    stats = run_cycle(p, g, H.make_oracles(p, w), None, None, synth.make_root(p), ca_cache=(caK, caV), sa_cache=(saK, saV),
                      seqs=[0, 7, 15])
    assert stats["rows"] == 3 * (1 + 16)


@pytest.mark.parametrize("batch,topk", [(13, 10), (24, 8), (15, 15)])
def test_row_counts_between_128_and_256(batch, topk):
    """Forwards of 130, 192 and 225 rows: activation tiles of 160, 192 and 256 rows, two tiles (high- and low-order
    terms) per stage; the step-0 forward of each (13, 24, 15 rows) takes the one-tile form."""
    p = synth.scaled(synth.PRESETS["c5"], d_model=256, n_stack=2, d_stack=128, vocab=2051, lsa_hq=2, lsa_hkv=2,
                     lsa_mlp=128, sa_hq=4, sa_hkv=1, sa_mlp=64, ca_hq=4, ca_hkv=2, ca_mlp=448, ctx=70, batch=batch,
                     tree_topk=topk, tree_depth=3, tree_keep=30, lsa_tokens=2)
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=80, lsa_chunk_tokens=32)
    caK, caV = synth.make_cache(p, "ca")
    saK, saV = synth.make_cache(p, "sa")
    stats = run_cycle(p, g, H.make_oracles(p, w), None, None, synth.make_root(p), ca_cache=(caK, caV), sa_cache=(saK, saV),
                      seqs=[0, batch - 1])
    assert stats["rows"] == 2 * (1 + 2 * topk)


def test_synthetic_caches_and_ragged_lengths():
    """Caches given directly (as in configs 2, 4, 5) with a different length per sequence."""
    p = synth.scaled(synth.PRESETS["c5"], d_model=256, n_stack=3, d_stack=256, vocab=777, lsa_hq=4, lsa_hkv=2,
                     lsa_mlp=256, sa_hq=4, sa_hkv=2, sa_mlp=32, ca_hq=4, ca_hkv=1, ca_mlp=448, ctx=50, batch=2,
                     tree_topk=3, tree_depth=3, tree_keep=7, head_dim=64)
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=64)
    exact, dec = H.make_oracles(p, w)
    caK, caV = synth.make_cache(p, "ca")
    saK, saV = synth.make_cache(p, "sa")
    g.fill_cache("ca", caK.cuda(), caV.cuda())
    g.fill_cache("sa", saK.cuda(), saV.cuda())
    lens_ca, lens_sa = [50, 1], [33, 0]
    g.moa_state_set_len("ca", lens_ca)
    g.moa_state_set_len("sa", lens_sa)
    root = synth.make_root(p)
    g.moa_tree_begin(root.cuda())

    def trees_of(dr, forced):
        return [O.draft_tree(dr, int(root[b]), H.np32(saK[b, :lens_sa[b]]), H.np32(saV[b, :lens_sa[b]]),
                             H.np32(caK[b, :lens_ca[b]]), H.np32(caV[b, :lens_ca[b]]), 3, 3, 7,
                             forced=None if forced is None else forced[b]) for b in range(2)]
    td = trees_of(dec, None)
    forced = [[([r["ids"] for r in rows], [r["logp"] for r in rows]) for rows in td[b][1]] for b in range(2)]
    tx = trees_of(exact, forced)
    tol = H.tol_of(p)
    for s in range(3):
        ids, lp, hid = g.moa_draft_step(want_hidden=True)
        ids, lp, hid = ids.cpu().numpy(), lp.cpu().numpy(), H.np32(hid.cpu())
        rs = 1 if s == 0 else 3
        f_ids, f_lp = np.zeros((2 * rs, 3), np.int32), np.zeros((2 * rs, 3), np.float32)
        for b in range(2):
            for r in range(rs):
                H.assert_rows_close(hid[b * rs + r][None], tx[b][1][s][r]["o_hat"][None], tol, f"hidden s{s} b{b} r{r}")
                H.check_topk(ids[b * rs + r], lp[b * rs + r], td[b][1][s][r]["z"], tol, H.tie_window(p, td[b][1][s][r]["z"]))
                f_ids[b * rs + r], f_lp[b * rs + r] = td[b][1][s][r]["ids"], td[b][1][s][r]["logp"]
        g.moa_tree_expand(torch.from_numpy(f_ids).cuda(), torch.from_numpy(f_lp).cuda())


def test_api_misuse_returns_status_and_launches_nothing():
    from paper_2410_03804_b200.moa import MoaError
    p = synth.PRESETS["c1"]
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=16)
    with pytest.raises(MoaError, match="ERR_STATE"):
        g.batch = 1
        g.moa_draft_step()                                   # no tree begun
    with pytest.raises(MoaError, match="ERR_CAPACITY"):
        g.moa_sa_append(torch.zeros(17, dtype=torch.int32).cuda(), [17])
    with pytest.raises(MoaError, match="ERR_CAPACITY"):
        g.moa_lsa_forward(synth.make_h_stack(p, 17).cuda(), [17])
    with pytest.raises(MoaError, match="ERR_SHAPE"):
        g.moa_sa_append(torch.zeros(2, dtype=torch.int32).cuda(), [1, 1])    # batch 2 > max_batch 1
    g.moa_tree_begin(synth.make_root(p).cuda())
    small = g.ws_bytes
    g.ws_bytes = 1024
    with pytest.raises(MoaError, match="ERR_WORKSPACE"):
        g.moa_draft_step()
    g.ws_bytes = small
    g.moa_lsa_forward(synth.make_h_stack(p, 0).cuda(), [0])    # empty input is fine
    torch.cuda.synchronize()
    assert int(g.ca_len[0]) == 0
    bad = dict(H.cfg_of(p)); bad["head_dim"] = 96
    with pytest.raises(MoaError, match="ERR_SHAPE"):
        from paper_2410_03804_b200 import moa
        moa.MoA(bad, {k: v.cuda() for k, v in w.items()}, 1, 16)


@pytest.mark.parametrize("dtype,lsa_tokens", [("bf16", 6), ("f32", 6), ("bf16", 60)])
def test_device_side_capacity_guard_when_the_host_count_is_stale(dtype, lsa_tokens):
    """A recorded graph replays cache appends with the host-side capacity check frozen at capture time. Here the host
    count is set back by hand (the state a replay is in): the kernels must drop the rows that would land beyond
    max_ctx, clamp the device count and raise the status word. Sequence 1's cache region lies right behind
    sequence 0's, so a missing guard would show there, inside the allocation. 60 tokens x 5 layers = 300 rows takes the
    dense-regime LSA pass (one persistent kernel), 6 tokens the weight-streaming launch chain."""
    p = synth.scaled(synth.PRESETS["c2"], d_model=512, n_stack=5, d_stack=384, vocab=5003, lsa_hq=8, lsa_hkv=2,
                     lsa_mlp=768, sa_hq=8, sa_hkv=2, sa_mlp=64, ca_hq=8, ca_hkv=4, ca_mlp=896, ctx=0, batch=1,
                     tree_topk=5, tree_depth=2, tree_keep=8, dtype=dtype)
    w = synth.make_weights(p)
    cap = lsa_tokens + lsa_tokens // 2                     # the second append overflows by half of its rows
    g = H.make_gpu(p, w, max_ctx=cap, lsa_chunk_tokens=64, max_batch=2)
    g.moa_tree_begin(synth.make_root(p).cuda())            # clears the status word
    for t in (g.sa_k, g.sa_v, g.ca_k, g.ca_v):
        t[1].fill_(7.0)                                    # sentinel in the neighbour's region
    n = lsa_tokens
    toks = synth.make_tokens(p, 2 * n, tensor_index=47)[0]
    h = synth.make_h_stack(p, 2 * n)
    g.moa_sa_append(toks[:n].contiguous().cuda(), [n])
    g.moa_lsa_forward(h[:n].cuda(), [n], want_kv=False)
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0 and g.sa_len[:1].tolist() == [n] and g.ca_len[:1].tolist() == [n]
    k_before, ck_before = g.sa_k[0, :n].clone(), g.ca_k[0, :n].clone()
    g._sa_len_host[0] = 0                                  # the host's view at capture time
    g._ca_len_host[0] = 0
    g.moa_sa_append(toks[n:].contiguous().cuda(), [n])
    torch.cuda.synchronize()
    assert g.moa_state_status() == 6                       # MOA_ERR_CAPACITY, raised on the device
    assert g.sa_len[:1].tolist() == [cap]
    g.moa_tree_begin(synth.make_root(p).cuda())
    g.moa_lsa_forward(h[n:].cuda(), [n], want_kv=False)
    torch.cuda.synchronize()
    assert g.moa_state_status() == 6
    assert g.ca_len[:1].tolist() == [cap]
    for t in (g.sa_k, g.sa_v, g.ca_k, g.ca_v):
        assert bool((t[1] == 7.0).all()), "a row was written beyond max_ctx"
    # the rows that fit were written, the earlier ones are untouched
    assert torch.equal(g.sa_k[0, :n], k_before) and torch.equal(g.ca_k[0, :n], ck_before)
    assert float(g.sa_k[0, n:cap].float().abs().max()) > 0 and float(g.ca_k[0, n:cap].float().abs().max()) > 0


def _reduced(dtype, batch, **kw):
    base = dict(d_model=512, n_stack=5, d_stack=384, vocab=5003, lsa_hq=8, lsa_hkv=2, lsa_mlp=768, sa_hq=8, sa_hkv=2,
                sa_mlp=64, ca_hq=8, ca_hkv=4, ca_mlp=896, ctx=37, batch=batch, tree_topk=5, tree_depth=3, tree_keep=12,
                dtype=dtype, lsa_tokens=37)
    base.update(kw)
    return synth.scaled(synth.PRESETS["c2"], **base)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_sequences_of_a_batch_are_independent(dtype):
    """Input-independence on the GPU (Section 3.1.2, the property that a row's cross-attention result does not depend
    on the other rows; sequences of a batch share nothing): three sequences drafted together give what each gives
    alone, up to the rounding order of a different launch shape."""
    nb = 3
    p = _reduced(dtype, nb)
    w = synth.make_weights(p)
    caK, caV = synth.make_cache(p, "ca")
    saK, saV = synth.make_cache(p, "sa")
    root = synth.make_root(p)
    tol = 2e-3 if dtype == "bf16" else 2e-5

    def run(seqs):
        g = H.make_gpu(synth.scaled(p, batch=len(seqs)), w, max_ctx=64, max_batch=len(seqs))
        g.fill_cache("ca", caK[seqs].cuda(), caV[seqs].cuda())
        g.fill_cache("sa", saK[seqs].cuda(), saV[seqs].cuda())
        g.moa_tree_begin(root[seqs].contiguous().cuda())
        hs = []
        for s in range(p.tree_depth):
            ids, lp, hid = g.moa_draft_step(want_hidden=True)
            g.moa_tree_expand(ids, lp)
            rs = 1 if s == 0 else p.tree_topk
            hs.append((H.np32(hid.cpu()).reshape(len(seqs), rs, -1), ids.cpu().numpy().reshape(len(seqs), rs, -1)))
        torch.cuda.synchronize()
        assert g.moa_state_status() == 0
        g.close()
        return hs

    together = run([0, 1, 2])
    for b in range(nb):
        alone = run([b])
        for s in range(p.tree_depth):
            if not np.array_equal(together[s][1][b], alone[s][1][0]):
                break                                    # a near-tie went the other way: later rows are other tokens
            H.assert_rows_close(together[s][0][b], alone[s][0][0], tol, f"seq {b} step {s}: together vs alone")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_lsa_tokens_are_independent_and_incremental_equals_full(dtype):
    """Layer Self-Attention treats tokens independently (Section 3.1.1), so appending tokens call by call
    (Algorithm 1, the second LSA_layer_with_mean on the newly verified tokens) gives the rows one call over all
    of them gives."""
    p = _reduced(dtype, 1)
    w = synth.make_weights(p)
    n = 21
    h = synth.make_h_stack(p, n).cuda()
    tol = 4e-3 if dtype == "bf16" else 2e-5

    def run(parts, chunk):
        g = H.make_gpu(p, w, max_ctx=64, lsa_chunk_tokens=chunk)
        kvs, t0 = [], 0
        for m in parts:
            kvs.append(g.moa_lsa_forward(h[t0:t0 + m].contiguous(), [m]).clone())
            t0 += m
        torch.cuda.synchronize()
        assert g.moa_state_status() == 0 and g.ca_len[:1].tolist() == [n]
        out = (H.np32(torch.cat(kvs).cpu()), H.np32(g.ca_k[0, :n].cpu()).reshape(n, -1), H.np32(g.ca_v[0, :n].cpu()).reshape(n, -1))
        g.close()
        return out

    full = run([n], 32)
    for parts, chunk in (([1] * n, 32), ([5, 7, 9], 32), ([n], 4)):
        got = run(parts, chunk)
        for a, b, what in zip(got, full, ("kv", "CA K rows", "CA V rows")):
            H.assert_rows_close(a, b, tol, f"{what}: parts {parts[:3]}.. chunk {chunk} vs one call")


@pytest.mark.parametrize("case", ["ragged", "wide_tree"])
def test_long_caches_take_the_tensor_core_attention_with_ragged_lengths(case):
    """Caches of 2048 positions and more run on the tcgen05 attention kernel (keys and values streamed by TMA in blocks
    of 128 positions, queries, scores, probabilities and the output accumulator in tensor memory), the tree segment
    as one more CTA of the same grid; the parts are merged by the split-KV kernel's merge.
    "ragged": two sequences with different lengths, one of them with an empty self-attention prefix (key ranges of
    zero blocks), lengths that are not multiples of the block, a last block whose second half is empty.
    "wide_tree": 16 x 8 = 128 query rows per kv head (every tensor-memory lane in use), a tree of 145 slots (two tree
    blocks, the second one ragged), lengths at and just above the 2048-position threshold."""
    if case == "ragged":
        p = synth.scaled(synth.PRESETS["c5"], d_model=256, n_stack=2, d_stack=128, vocab=1031, lsa_hq=2, lsa_hkv=2,
                         lsa_mlp=128, sa_hq=4, sa_hkv=1, sa_mlp=64, ca_hq=4, ca_hkv=2, ca_mlp=448, ctx=5000, batch=2,
                         tree_topk=4, tree_depth=3, tree_keep=9, head_dim=128)
        lens_ca, lens_sa = [5000, 4101], [4990, 0]
    else:
        p = synth.scaled(synth.PRESETS["c5"], d_model=256, n_stack=2, d_stack=128, vocab=1031, lsa_hq=2, lsa_hkv=2,
                         lsa_mlp=128, sa_hq=8, sa_hkv=1, sa_mlp=64, ca_hq=8, ca_hkv=2, ca_mlp=192, ctx=2100, batch=2,
                         tree_topk=16, tree_depth=10, tree_keep=60, head_dim=128)
        lens_ca, lens_sa = [2100, 2048], [2049, 2090]
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=p.ctx + 56)
    exact, dec = H.make_oracles(p, w)
    caK, caV = synth.make_cache(p, "ca")
    saK, saV = synth.make_cache(p, "sa")
    g.fill_cache("ca", caK.cuda(), caV.cuda())
    g.fill_cache("sa", saK.cuda(), saV.cuda())
    g.moa_state_set_len("ca", lens_ca)
    g.moa_state_set_len("sa", lens_sa)
    root = synth.make_root(p)
    g.moa_tree_begin(root.cuda())
    B, D = p.tree_topk, p.tree_depth

    def trees_of(dr, forced):
        return [O.draft_tree(dr, int(root[b]), H.np32(saK[b, :lens_sa[b]]), H.np32(saV[b, :lens_sa[b]]),
                             H.np32(caK[b, :lens_ca[b]]), H.np32(caV[b, :lens_ca[b]]), B, D, p.tree_keep,
                             forced=None if forced is None else forced[b]) for b in range(2)]
    td = trees_of(dec, None)
    forced = [[([r["ids"] for r in rows], [r["logp"] for r in rows]) for rows in td[b][1]] for b in range(2)]
    tx = trees_of(exact, forced)
    tol = H.tol_of(p)
    worst = 0.0
    for s in range(D):
        ids, lp, hid = g.moa_draft_step(want_hidden=True)
        ids, lp, hid = ids.cpu().numpy(), lp.cpu().numpy(), H.np32(hid.cpu())
        rs = 1 if s == 0 else B
        f_ids, f_lp = np.zeros((2 * rs, B), np.int32), np.zeros((2 * rs, B), np.float32)
        for b in range(2):
            for r in range(rs):
                worst = max(worst, H.assert_rows_close(hid[b * rs + r][None], tx[b][1][s][r]["o_hat"][None], tol, f"hidden s{s} b{b} r{r}"))
                H.check_topk(ids[b * rs + r], lp[b * rs + r], td[b][1][s][r]["z"], tol, H.tie_window(p, td[b][1][s][r]["z"]))
                f_ids[b * rs + r], f_lp[b * rs + r] = td[b][1][s][r]["ids"], td[b][1][s][r]["logp"]
        g.moa_tree_expand(torch.from_numpy(f_ids).cuda(), torch.from_numpy(f_lp).cuda())
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0
    print(f"[long caches, tensor-core attention, {case}] worst hidden {worst:.2e}")
