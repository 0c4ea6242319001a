"""The debug build of the library (-DMOA_CHECKS): indices the host logic guarantees are checked on the device where
they are used, and a violation raises the status word. Run in a child process, because a process loads one variant
of the library; reduced shapes only."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
import numpy as np, torch
sys.path.insert(0, %r)
from paper_2410_03804_b200 import synth
from tests import helpers as H
from tests.test_gpu_parity import run_cycle
p = synth.scaled(synth.PRESETS["c2"], d_model=512, n_stack=5, d_stack=384, vocab=5003, lsa_hq=8, lsa_hkv=2, lsa_mlp=768,
                 sa_hq=8, sa_hkv=2, sa_mlp=64, ca_hq=8, ca_hkv=4, ca_mlp=896, ctx=37, batch=2, tree_topk=5, tree_depth=3,
                 tree_keep=12, dtype="bf16", lsa_tokens=37)
w = synth.make_weights(p)
g = H.make_gpu(p, w, max_ctx=64, lsa_chunk_tokens=16)
assert g.lib.moa_trace_begin is not None
# a whole cycle against the oracle with every check armed: the status word must stay clear
stats = run_cycle(p, g, H.make_oracles(p, w), synth.make_h_stack(p, p.lsa_tokens * 2), synth.make_tokens(p, p.ctx), synth.make_root(p))
assert stats["rows"] == 2 * (1 + 2 * 5) and g.moa_state_status() == 0
# a token id outside the vocabulary: the normal library clamps it silently, the checking variant also reports it
g.moa_tree_begin(synth.make_root(p).cuda())
g.moa_state_set_len("sa", [0, 0])
bad = torch.tensor([3, p.vocab + 5, 7, 1], dtype=torch.int32).cuda()
g.moa_sa_append(bad, [2, 2])
torch.cuda.synchronize()
assert g.moa_state_status() == 6, g.moa_state_status()
print("checks build ok")
'''


def test_checks_build_runs_clean_and_reports_a_bad_token_id():
    from paper_2410_03804_b200 import build
    build.build(checks=True)
    env = dict(os.environ, MOA_CHECKS_BUILD="1")
    res = subprocess.run([sys.executable, "-c", CHILD % ROOT], capture_output=True, text=True, env=env, cwd=ROOT, timeout=900)
    assert res.returncode == 0 and "checks build ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]
