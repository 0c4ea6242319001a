"""Integer stages on the GPU (tree expansion, final cut, ancestor mask) against the oracle, bit-exact."""
import numpy as np
import pytest
import torch

from oracle import moa_oracle as O
from paper_2410_03804_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _tiny_model(B, D, m, batch):
    p = synth.scaled(synth.PRESETS["c1"], tree_topk=B, tree_depth=D, tree_keep=m, batch=batch, vocab=1024)
    w = synth.make_weights(p)
    return p, H.make_gpu(p, w, max_ctx=16, max_batch=batch)


@pytest.mark.parametrize("B,D,m,batch", [(4, 4, 16, 1), (10, 6, 60, 3), (8, 6, 62, 2), (1, 5, 3, 2), (16, 3, 1000, 1),
                                         (2, 1, 2, 1)])
def test_tree_expand_and_finalize_bit_exact(B, D, m, batch):
    p, g = _tiny_model(B, D, m, batch)
    rng = np.random.default_rng(B * 1000 + D * 10 + batch)
    roots = rng.integers(0, 1024, batch).astype(np.int32)
    g.moa_tree_begin(torch.from_numpy(roots).cuda())
    trees = [O.TreeState(int(roots[b]), B, D, m) for b in range(batch)]
    outs = None
    for s in range(D):
        R = batch * (1 if s == 0 else B)
        lp = -np.sort(rng.exponential(1.0, (R, B)), axis=-1).astype(np.float32)
        if s == 2 and B > 1:
            lp[:, 1] = lp[:, 0]                    # exact ties inside a row
            lp[-1] = lp[0]                         # and across rows
        ids = rng.integers(0, 1024, (R, B)).astype(np.int32)
        outs = g.moa_tree_expand(torch.from_numpy(ids).cuda(), torch.from_numpy(lp).cuda())
        rs = 1 if s == 0 else B
        for b in range(batch):
            O.tree_expand(trees[b], ids[b * rs:(b + 1) * rs], lp[b * rs:(b + 1) * rs])
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0
    tok, parent, depth, score, n = [t.cpu().numpy() for t in outs]
    for b in range(batch):
        otok, opar, odep, osc = O.tree_finalize(trees[b])
        k = len(otok)
        assert n[b] == k
        assert np.array_equal(tok[b, :k], otok) and np.array_equal(parent[b, :k], opar)
        assert np.array_equal(depth[b, :k], odep)
        assert np.array_equal(score[b, :k].view(np.int32), osc.view(np.int32))       # bit-exact fp32 scores
        assert np.all(tok[b, k:] == -1) and np.all(parent[b, k:] == -1)
        mask = g_mask(parent[b:b + 1, :k])
        assert np.array_equal(mask[0], O.tree_mask(opar))
    # a further expansion is out of order
    from paper_2410_03804_b200.moa import MoaError
    with pytest.raises(MoaError):
        g.moa_tree_expand(torch.zeros((batch * B, B), dtype=torch.int32).cuda(),
                          torch.zeros((batch * B, B), dtype=torch.float32).cuda())


def test_tree_expand_reports_a_log_probability_that_is_not_a_number():
    """The ranks of an expansion are a permutation only under a total order. A NaN among the log-probabilities (a fault
    upstream of the tree) must rank last and raise status 11 instead of leaving frontier entries unwritten: every
    parent stays a valid slot of the kept tree."""
    B, D, m, batch = 4, 3, 8, 2
    p, g = _tiny_model(B, D, m, batch)
    rng = np.random.default_rng(7)
    g.moa_tree_begin(torch.from_numpy(rng.integers(0, 1024, batch).astype(np.int32)).cuda())
    outs = None
    for s in range(D):
        R = batch * (1 if s == 0 else B)
        lp = -np.sort(rng.exponential(1.0, (R, B)), axis=-1).astype(np.float32)
        if s < 2:
            lp[0, :] = np.nan                       # a whole row at the first steps, one entry later
        else:
            lp[-1, 1] = np.nan
        ids = rng.integers(0, 1024, (R, B)).astype(np.int32)
        outs = g.moa_tree_expand(torch.from_numpy(ids).cuda(), torch.from_numpy(lp).cuda())
    torch.cuda.synchronize()
    assert g.moa_state_status() == 11
    tok, parent, depth, score, n = [t.cpu().numpy() for t in outs]
    for b in range(batch):
        k = int(n[b])
        assert 1 <= k <= m + 1
        assert parent[b, 0] == -1 and np.all((parent[b, 1:k] >= 0) & (parent[b, 1:k] < np.arange(1, k)))
        assert np.all(depth[b, 1:k] == depth[b, parent[b, 1:k]] + 1)
        assert not np.isnan(score[b, :k]).any()


def g_mask(parent_np, packed=False):
    from paper_2410_03804_b200 import moa
    t = torch.from_numpy(np.ascontiguousarray(parent_np.astype(np.int32))).cuda()
    return moa.moa_tree_attn_mask(t, packed=packed).cpu().numpy()


@pytest.mark.parametrize("n", [1, 2, 61, 63, 64, 65, 130])
def test_mask_dense_and_packed(n):
    rng = np.random.default_rng(n)
    batch = 3
    parent = np.full((batch, n), -1, np.int32)
    for b in range(batch):
        for i in range(1, n):
            parent[b, i] = rng.integers(0, i)
    if n > 5:
        parent[2, n - 2:] = -1                    # unused tail slots
    dense = g_mask(parent)
    packed = g_mask(parent, packed=True)
    for b in range(batch):
        want = O.tree_mask(parent[b])
        for i in range(1, n):
            if parent[b, i] < 0:
                want[i] = 0
        assert np.array_equal(dense[b], want)
        bits = np.zeros((n, n), np.uint8)
        for i in range(n):
            for j in range(n):
                bits[i, j] = (int(packed[b, i, j // 64]) >> (j % 64)) & 1
        assert np.array_equal(bits, want)


def test_mask_empty_and_bad_arguments():
    from paper_2410_03804_b200 import moa
    lib = moa.load_library()
    t = torch.zeros((1, 4), dtype=torch.int32).cuda()
    out = torch.zeros(16, dtype=torch.uint8).cuda()
    assert lib.moa_tree_attn_mask(t.data_ptr(), 0, 4, out.data_ptr(), 0, None) == 0        # empty batch: nothing to do
    assert lib.moa_tree_attn_mask(t.data_ptr(), 1, 4, out.data_ptr(), 2, None) == 2        # bad packed flag
    assert lib.moa_tree_attn_mask(t.data_ptr() + 4, 1, 3, out.data_ptr(), 0, None) == 4    # misaligned
    assert lib.moa_tree_attn_mask(t.data_ptr(), -1, 4, out.data_ptr(), 0, None) == 2
