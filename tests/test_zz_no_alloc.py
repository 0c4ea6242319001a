"""moa_sa_append_static: the self-attention prefix append for callers that cannot allocate device memory
(its scratch is a fixed array inside the library). Checked against moa_sa_append on the same tokens, twice
in a row, through the C ABI, and against the oracle's prefix keys / values directly. Collected last on purpose:
every other test has run before this one."""
import pytest
import torch

from paper_2410_03804_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _small(dtype, **kw):
    base = dict(d_model=512, n_stack=2, d_stack=256, vocab=3001, lsa_hq=4, lsa_hkv=2, lsa_mlp=256, sa_hq=8, sa_hkv=2,
                sa_mlp=64, ca_hq=8, ca_hkv=2, ca_mlp=256, ctx=0, batch=2, tree_topk=4, tree_depth=2, tree_keep=6,
                dtype=dtype)
    base.update(kw)
    return synth.scaled(synth.PRESETS["c2"], **base)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_append_matches_workspace_append_twice(dtype):
    p = _small(dtype)
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=64)
    exact = H.make_oracle(p, w)
    tol = H.tol_of(p)
    n_first, n_second = [7, 4], [5, 9]
    tok1 = synth.make_tokens(p, 16, tensor_index=40)
    tok2 = synth.make_tokens(p, 16, tensor_index=42)
    flat = lambda t, n: torch.cat([t[b, :n[b]] for b in range(2)]).contiguous().cuda()

    t1, t2 = flat(tok1, n_first), flat(tok2, n_second)
    # the existing entry point: two appends in a row with the caller's workspace
    g.moa_sa_append(t1, n_first)
    g.moa_sa_append(t2, n_second)
    torch.cuda.synchronize()
    want_k, want_v = g.sa_k.clone(), g.sa_v.clone()
    assert g.sa_len[:2].tolist() == [12, 13]

    # the same two appends through the entry point that allocates nothing
    g.moa_state_set_len("sa", [0, 0])
    g.sa_k.zero_()
    g.sa_v.zero_()
    free_before = torch.cuda.mem_get_info()[0]
    g.moa_sa_append_static(t1, n_first)
    g.moa_sa_append_static(t2, n_second)
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0
    assert g.sa_len[:2].tolist() == [12, 13]
    for b, n in enumerate([12, 13]):
        H.assert_rows_close(H.np32(g.sa_k[b, :n].cpu()), H.np32(want_k[b, :n].cpu()), tol, f"static K seq {b}")
        H.assert_rows_close(H.np32(g.sa_v[b, :n].cpu()), H.np32(want_v[b, :n].cpu()), tol, f"static V seq {b}")
        assert float(g.sa_k[b, :n].float().abs().max()) > 0
        # and against the oracle itself: the sequence's tokens at positions 0 .. n-1
        toks = tok1[b, :n_first[b]].tolist() + tok2[b, :n_second[b]].tolist()
        K, V = exact.sa_prefix(toks)
        H.assert_rows_close(H.np32(g.sa_k[b, :n].cpu()).reshape(n, -1), K.reshape(n, -1), tol, f"static K vs oracle seq {b}")
        H.assert_rows_close(H.np32(g.sa_v[b, :n].cpu()).reshape(n, -1), V.reshape(n, -1), tol, f"static V vs oracle seq {b}")
    assert torch.cuda.mem_get_info()[0] >= free_before - (1 << 20)      # nothing was allocated on the device


def test_static_scratch_filled_exactly_by_32_tokens_of_width_4096():
    """The largest call the fixed scratch takes on bf16: 32 tokens of width 4096 put (32 + 32 low-order) rows of
    8 KiB into the 512 KiB region of normalised rows, to the last byte; both calls of a pair are compared with
    the oracle."""
    p = _small("bf16", d_model=4096, vocab=1024, sa_hq=4, sa_hkv=2, sa_mlp=64, ca_hq=4, ca_mlp=64, batch=1)
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=80, max_batch=1)
    exact = H.make_oracle(p, w)
    toks = synth.make_tokens(p, 64, tensor_index=41)[0]
    g.moa_sa_append_static(toks[:32].contiguous().cuda(), [32])
    g.moa_sa_append_static(toks[32:].contiguous().cuda(), [32])
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0 and g.sa_len[:1].tolist() == [64]
    K, V = exact.sa_prefix(toks.tolist())
    H.assert_rows_close(H.np32(g.sa_k[0, :64].cpu()).reshape(64, -1), K.reshape(64, -1), H.tol_of(p), "K, full scratch")
    H.assert_rows_close(H.np32(g.sa_v[0, :64].cpu()).reshape(64, -1), V.reshape(64, -1), H.tol_of(p), "V, full scratch")


def test_static_scratch_rejects_oversized_calls():
    from paper_2410_03804_b200.moa import MoaError
    p = synth.PRESETS["c1"]
    g = H.make_gpu(p, synth.make_weights(p), max_ctx=128)
    with pytest.raises(MoaError, match="ERR_WORKSPACE.*exceed the fixed scratch"):
        g.moa_sa_append_static(torch.zeros(33, dtype=torch.int32).cuda(), [33])
    torch.cuda.synchronize()
    assert int(g.sa_len[0]) == 0
    # a call inside the token limit that fails on the byte limit alone: 32 bf16 tokens of width 8192 need 1 MiB
    p8 = _small("bf16", d_model=8192, vocab=256, sa_hq=2, sa_hkv=1, sa_mlp=64, ca_hq=2, ca_hkv=1, ca_mlp=64, batch=1)
    g8 = H.make_gpu(p8, synth.make_weights(p8), max_ctx=64, max_batch=1)
    with pytest.raises(MoaError, match="ERR_WORKSPACE.*exceed the fixed scratch"):
        g8.moa_sa_append_static(torch.zeros(32, dtype=torch.int32).cuda(), [32])
    torch.cuda.synchronize()
    assert int(g8.sa_len[0]) == 0
    g8.moa_sa_append_static(torch.zeros(16, dtype=torch.int32).cuda(), [16])      # 32 rows of 16 KiB: fits exactly
    torch.cuda.synchronize()
    assert int(g8.sa_len[0]) == 16 and g8.moa_state_status() == 0
