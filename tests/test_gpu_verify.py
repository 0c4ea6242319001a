"""Greedy verification of the kept tree on the GPU (through the C ABI) against the oracle: bit-exact index work."""
import numpy as np
import pytest
import torch

from oracle import moa_oracle as O
from paper_2410_03804_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _trees(rng, batch, n, vocab, width=4, unused_tail=0):
    tok = np.zeros((batch, n), np.int32)
    parent = np.full((batch, n), -1, np.int32)
    for b in range(batch):
        tok[b, 0] = rng.integers(vocab)
        for i in range(1, n - unused_tail):
            while True:
                q = int(rng.integers(0, i))
                t = int(rng.integers(vocab))
                sibs = [tok[b, c] for c in range(1, i) if parent[b, c] == q]
                if t not in sibs and len(sibs) < width:
                    break
            tok[b, i], parent[b, i] = t, q
    return tok, parent


def _logits_following_the_tree(rng, tok, parent, vocab, follow=0.75):
    """Random logits; at most slots the arg-max is planted on one child's token so that paths get accepted."""
    batch, n = tok.shape
    z = rng.standard_normal((batch, n, vocab)).astype(np.float32)
    for b in range(batch):
        for i in range(n):
            kids = [c for c in range(1, n) if parent[b, c] == i]
            if kids and rng.random() < follow:
                z[b, i, tok[b, kids[int(rng.integers(len(kids)))]]] = 9.0
    return z


def _check(tok, parent, z_t, cap):
    from paper_2410_03804_b200 import moa
    choice, acc_slot, acc_tok, acc_len, next_tok = moa.moa_verify_greedy(
        torch.from_numpy(tok).cuda(), torch.from_numpy(parent).cuda(), z_t.cuda(), cap)
    torch.cuda.synchronize()
    choice, acc_slot, acc_tok, acc_len, next_tok = [t.cpu().numpy() for t in (choice, acc_slot, acc_tok, acc_len, next_tok)]
    z = z_t.float().numpy()
    lens = []
    for b in range(tok.shape[0]):
        slots, nxt, ch = O.verify_greedy(tok[b], parent[b], z[b])
        slots = slots[:cap]
        assert np.array_equal(choice[b], ch)
        k = len(slots)
        assert acc_len[b] == k
        assert np.array_equal(acc_slot[b, :k], slots) and np.all(acc_slot[b, k:] == -1)
        assert np.array_equal(acc_tok[b, :k], tok[b][slots]) and np.all(acc_tok[b, k:] == -1)
        if k == len(O.verify_greedy(tok[b], parent[b], z[b])[0]):
            assert next_tok[b] == nxt
        lens.append(k)
    return lens


@pytest.mark.parametrize("dtype,vocab", [(torch.float32, 1024), (torch.bfloat16, 5003), (torch.float32, 4099),
                                         (torch.bfloat16, 32000)])
def test_verify_random_trees(dtype, vocab):
    """Random trees of 61 slots (config 2's kept size), several sequences, ragged vocabularies (rows of the
    logits then start off a 16-byte boundary: scalar loads), unused tail slots."""
    rng = np.random.default_rng(vocab)
    tok, parent = _trees(rng, 5, 61, vocab, unused_tail=3)
    z = torch.from_numpy(_logits_following_the_tree(rng, tok, parent, vocab)).to(dtype)
    lens = _check(tok, parent, z, cap=7)
    assert max(lens) >= 3 and min(lens) >= 1


def test_verify_ties_and_caps():
    """Equal maxima go to the smallest id (bf16 rounding makes ties common); cap cuts the path."""
    rng = np.random.default_rng(5)
    V = 777
    tok = np.array([[3, 10, 11, 12, 13, 14]], np.int32)
    parent = np.array([[-1, 0, 1, 2, 3, 4]], np.int32)
    z = np.zeros((1, 6, V), np.float32)
    for i, t in enumerate([10, 11, 12, 13, 14, 15]):
        z[0, i, t] = 1.0
        z[0, i, t + 100] = 1.0               # an equal logit at a larger id
    zt = torch.from_numpy(z).to(torch.bfloat16)
    assert _check(tok, parent, zt, cap=7) == [6]
    assert _check(tok, parent, zt, cap=3) == [3]
    z[0, 2, 5] = 1.0                          # an equal logit at a SMALLER id: the chain breaks at slot 2
    assert _check(tok, parent, torch.from_numpy(z), cap=7) == [3]


def test_verify_full_size_c5_batch16():
    """Config 5's verification input: 16 sequences x 61 kept slots x 128256 logits in bf16 (250 MB)."""
    rng = np.random.default_rng(11)
    p = synth.PRESETS["c5"]
    n = p.tree_keep + 1
    tok, parent = _trees(rng, p.batch, n, p.vocab, width=p.tree_topk)
    g = torch.Generator().manual_seed(synth.SEED_BASE + 5555)
    z = torch.randn((p.batch, n, p.vocab), generator=g, dtype=torch.float32).to(torch.bfloat16)
    for b in range(p.batch):                  # plant the LLM's choices along the trees
        for i in range(n):
            kids = [c for c in range(1, n) if parent[b, c] == i]
            if kids and rng.random() < 0.8:
                z[b, i, int(tok[b, kids[0]])] = 9.0
    lens = _check(tok, parent, z, cap=p.tree_depth + 1)
    assert max(lens) >= 3


def test_draft_verify_commit_cycle_c1():
    """Config 1, two cycles: draft a tree, verify it against synthetic LLM logits that follow one of its paths,
    append the accepted tokens to the self-attention prefix (moa_sa_append), start the next tree at the LLM's
    next token. The prefix cache then equals the oracle's prefix over prompt + accepted tokens."""
    from paper_2410_03804_b200 import moa
    p = synth.PRESETS["c1"]
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=p.ctx + 32, lsa_chunk_tokens=64)
    dr = H.make_oracle(p, w)
    prompt = synth.make_tokens(p, p.ctx)
    g.moa_lsa_forward(synth.make_h_stack(p, p.lsa_tokens).cuda(), [p.lsa_tokens])
    g.moa_sa_append(prompt.reshape(-1).cuda(), [p.ctx])
    seq = prompt[0].tolist()
    root = synth.make_root(p)
    rng = np.random.default_rng(1)
    for cycle in range(2):
        g.moa_tree_begin(root.cuda())
        outs = None
        for s in range(p.tree_depth):
            ids, lp, _ = g.moa_draft_step()
            outs = g.moa_tree_expand(ids, lp)
        tok, parent, depth, score, n = outs
        torch.cuda.synchronize()
        tok_h, par_h = tok.cpu().numpy(), parent.cpu().numpy()
        z = _logits_following_the_tree(rng, tok_h, par_h, p.vocab, follow=0.9)
        choice, acc_slot, acc_tok, acc_len, next_tok = moa.moa_verify_greedy(tok, parent, torch.from_numpy(z).cuda(),
                                                                             p.tree_depth + 1)
        torch.cuda.synchronize()
        slots, nxt, _ = O.verify_greedy(tok_h[0], par_h[0], z[0])
        k = int(acc_len[0])
        assert k == len(slots) and acc_slot[0, :k].tolist() == slots and int(next_tok[0]) == nxt
        g.moa_sa_append(acc_tok[0, :k].contiguous(), [k])
        seq += acc_tok[0, :k].tolist()
        root = next_tok.cpu()
    torch.cuda.synchronize()
    saK, saV = dr.sa_prefix(seq)
    assert g.sa_len[:1].tolist() == [len(seq)]
    H.assert_rows_close(H.np32(g.sa_k[0, :len(seq)].cpu()), saK, H.tol_of(p), "SA K after two cycles")
    H.assert_rows_close(H.np32(g.sa_v[0, :len(seq)].cpu()), saV, H.tol_of(p), "SA V after two cycles")


def test_verify_misuse_returns_status():
    from paper_2410_03804_b200 import moa
    lib = moa.load_library()
    t = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    z = torch.zeros((1, 4, 8), dtype=torch.float32, device="cuda")
    o = torch.zeros(16, dtype=torch.int32, device="cuda")
    a = lambda x: x.data_ptr()
    assert lib.moa_verify_greedy(None, a(t), 1, 4, a(z), 0, 8, 3, a(o), a(o), a(o), a(o), a(o), None) == 1
    assert lib.moa_verify_greedy(a(t), a(t), 0, 4, a(z), 0, 8, 3, a(o), a(o), a(o), a(o), a(o), None) == 2
    assert lib.moa_verify_greedy(a(t), a(t), 1, 4, a(z), 7, 8, 3, a(o), a(o), a(o), a(o), a(o), None) == 3
