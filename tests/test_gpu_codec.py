"""Client-server message codec on the GPU (through the C ABI) against the oracle: bit-exact bytes, codes and scales."""
import numpy as np
import pytest
import torch

from oracle import moa_oracle as O
from paper_2410_03804_b200 import synth

pytestmark = pytest.mark.gpu


def test_pack_unpack_tree_bit_exact():
    from paper_2410_03804_b200 import moa
    rng = np.random.default_rng(3)
    batch, n, V = 7, 61, 128256
    tok = rng.integers(0, V, (batch, n)).astype(np.int32)
    parent = np.stack([np.concatenate([[-1], rng.integers(0, np.arange(1, n))]) for _ in range(batch)]).astype(np.int32)
    tok[2, 50:] = -1
    parent[2, 50:] = -1                                    # unused tail slots
    msg = moa.moa_pack_tree(torch.from_numpy(tok).cuda(), torch.from_numpy(parent).cuda())
    t2, p2 = moa.moa_unpack_tree(msg)
    torch.cuda.synchronize()
    assert msg.shape == (batch, n, 4) and msg.numel() == 4 * batch * n          # 4M bytes for M nodes
    for b in range(batch):
        assert np.array_equal(msg[b].cpu().numpy(), O.pack_tree(tok[b], parent[b]))
    assert np.array_equal(t2.cpu().numpy(), tok) and np.array_equal(p2.cpu().numpy(), parent)


@pytest.mark.parametrize("dtype,rows,width", [(torch.float32, 37, 333), (torch.bfloat16, 160, 4096), (torch.bfloat16, 33, 1001),
                                              (torch.float32, 64, 2048)])
def test_quantize_rows_bit_exact(dtype, rows, width):
    """Codes and scales equal the oracle's (both decide in fp32); stacked-activation statistics of config 2
    (std ramp, outlier channels) on the wide cases; odd widths take the scalar path."""
    from paper_2410_03804_b200 import moa
    g = torch.Generator().manual_seed(synth.SEED_BASE + rows * 7 + width)
    x = torch.randn((rows, width), generator=g) * (0.5 + torch.arange(rows).float()[:, None] / 16)
    x[:, torch.randperm(width, generator=g)[:8]] *= 20.0
    x[3] = 0
    x = x.to(dtype)
    codes, scales = moa.moa_quantize_rows(x.cuda())
    deq = moa.moa_dequantize_rows(codes, scales, dtype=dtype)
    torch.cuda.synchronize()
    q_o, s_o = O.quantize_rows(x.float().numpy())
    assert np.array_equal(codes.cpu().numpy(), q_o)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32))
    d_o = torch.from_numpy(O.dequantize_rows(q_o, s_o)).to(dtype)
    assert torch.equal(deq.cpu(), d_o)
    err = (deq.cpu().float() - x.float()).abs()
    assert bool((err <= scales.cpu()[:, None] * 0.5 * 1.01 + (1e-2 * x.float().abs() if dtype == torch.bfloat16 else 0)).all())


def test_quantized_lsa_input_feeds_the_lsa_step():
    """The server's message path on config 1: stacked activations quantised to 8 bits, dequantised on the client
    and fed to Layer Self-Attention; the result equals the oracle's LSA on the oracle's dequantised rows."""
    from paper_2410_03804_b200 import moa
    from tests import helpers as H
    p = synth.PRESETS["c1"]
    w = synth.make_weights(p)
    g = H.make_gpu(p, w, max_ctx=p.ctx + 8, lsa_chunk_tokens=16)
    h = synth.make_h_stack(p, 9)
    flat = h.reshape(-1, p.d_stack).cuda()
    codes, scales = moa.moa_quantize_rows(flat)
    hq = moa.moa_dequantize_rows(codes, scales, dtype=flat.dtype).reshape(h.shape)
    kv = g.moa_lsa_forward(hq, [9])
    torch.cuda.synchronize()
    q_o, s_o = O.quantize_rows(H.np32(h).reshape(-1, p.d_stack))
    kv_o = H.make_oracle(p, w).lsa_forward(O.dequantize_rows(q_o, s_o).reshape(h.shape))
    H.assert_rows_close(H.np32(kv.cpu()), kv_o, H.tol_of(p), "LSA on dequantised input")


def test_codec_misuse_returns_status():
    from paper_2410_03804_b200 import moa
    lib = moa.load_library()
    t = torch.zeros(16, dtype=torch.int32, device="cuda")
    assert lib.moa_pack_tree(None, t.data_ptr(), 4, t.data_ptr(), None) == 1
    assert lib.moa_pack_tree(t.data_ptr(), t.data_ptr(), -1, t.data_ptr(), None) == 2
    assert lib.moa_pack_tree(t.data_ptr(), t.data_ptr(), 4, t.data_ptr() + 1, None) == 4
    assert lib.moa_quantize_rows(t.data_ptr(), 5, 2, 8, t.data_ptr(), t.data_ptr(), None) == 3
    assert lib.moa_quantize_rows(t.data_ptr(), 0, 2, 0, t.data_ptr(), t.data_ptr(), None) == 2
