"""The give-up paths of the kernels (GPU only).  Every device-side wait is bounded; here the bound is set to a few
milliseconds and block 0 of one kernel family is told never to request its first tile, so a wait behind that tile
runs out.  The kernel must come back (no hang, no fault), the status word must say RMM_ERR_TIMEOUT, and once the
status has been read (which clears the workspace header) an ordinary call on the same workspace must match the oracle.
Each case runs in a child process, so that a kernel that did not come back would be a failed test with a time limit
rather than a stuck test session.  No input here faults: the "failure" is a copy that is never asked for."""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

PRELUDE = """
import numpy as np, torch
import oracle
import paper_2608_13426_b200 as rmm
from paper_2608_13426_b200 import binding, synth
binding.poison_outputs(True)
torch.cuda.set_device(0)
TIMEOUT = 5
def rel(got, want):
    return float(np.linalg.norm(np.asarray(got, dtype=np.float64) - want) / np.linalg.norm(want))
def expect_timeout(fn, family):
    launches = rmm.rmm_launch_count()
    rmm.rmm_debug_control("wait_limit_ms", 5.0)
    rmm.rmm_debug_control("withhold", family)
    fn()
    torch.cuda.synchronize()                      # the kernel came back
    rmm.rmm_debug_control("withhold", 0)
    rmm.rmm_debug_control("wait_limit_ms", 0.0)
    assert rmm.rmm_launch_count() > launches
    assert rmm.rmm_status_read() == TIMEOUT, "the kernel did not report the expired wait"
    assert rmm.rmm_status_read() == 0             # cleared by the read
"""

CASES = {
    "gemm": """
A, B = synth.mlp_product(300, 512, 256, seed=1)
Ad, Bd = A.cuda(), B.cuda()
idx = torch.arange(0, 512, 2, dtype=torch.int32, device="cuda")
expect_timeout(lambda: rmm.rmm_reduced_gemm(Ad, Bd, idx), 1)
Y = rmm.rmm_reduced_gemm(Ad, Bd, idx)
assert rel(Y.float().cpu().numpy(), oracle.reduced_gemm(A, B, idx.cpu().numpy())) <= 1e-2
assert rmm.rmm_status_read() == 0
""",
    "gemm_rows_of_b_fetched_in_kernel": """
A, B = synth.mlp_product(100, 512, 512, seed=2)
Ad, Bd = A.cuda(), B.cuda()
idx = torch.arange(1, 512, 2, dtype=torch.int32, device="cuda")
expect_timeout(lambda: rmm.rmm_reduced_gemm(Ad, Bd, idx), 1)
Y = rmm.rmm_reduced_gemm(Ad, Bd, idx)
assert rel(Y.float().cpu().numpy(), oracle.reduced_gemm(A, B, idx.cpu().numpy())) <= 1e-2
assert rmm.rmm_status_read() == 0
""",
    "score": """
A = synth.heavy_tailed_activations(256, 64, seed=3)
Ad = A.cuda()
expect_timeout(lambda: rmm.rmm_score_select(Ad, rho=0.5), 2)
idx, _, e, _ = rmm.rmm_score_select(Ad, rho=0.5, want_energy=True)
e64, _ = oracle.score(A)
assert np.allclose(e.cpu().numpy(), e64, rtol=3e-7)
assert np.array_equal(idx.cpu().numpy(), oracle.select(e.double().cpu().numpy(), 32)[0])
assert rmm.rmm_status_read() == 0
""",
    "attn": """
Q, K, V = synth.attention_qkv(1, 1, 1, 128, 128, 64, seed=4)
Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
expect_timeout(lambda: rmm.rmm_reduced_attn(Qd, Kd, Vd, True, 0.5, 1.0), 3)
O, feat, _ = rmm.rmm_reduced_attn(Qd, Kd, Vd, True, 0.5, 1.0, want_idx=True)
Oo = oracle.attn(Q, K, V, True, 0.5, 1.0, idx_feat=feat.cpu().numpy())[0]
assert rel(O.float().cpu().numpy(), Oo) <= 1e-2
assert rmm.rmm_status_read() == 0
""",
    "front": """
A, B = synth.mlp_product(300, 2560, 256, seed=5)
Ad, Bd = A.cuda(), B.cuda()
expect_timeout(lambda: rmm.rmm_product(Ad, Bd, rho=0.5), 4)
Y, idx = rmm.rmm_product(Ad, Bd, rho=0.5)
e64, _ = oracle.score(A)
assert np.array_equal(idx.cpu().numpy(), oracle.select(e64, 1280)[0])
assert rel(Y.float().cpu().numpy(), oracle.reduced_gemm(A, B, idx.cpu().numpy())) <= 1e-2
assert rmm.rmm_status_read() == 0
""",
    "pack": """
A = synth.heavy_tailed_activations(40, 20000, seed=6)
B = synth.weight(20000, 256, seed=7)
Ad, Bd = A.cuda(), B.cuda()
idx = torch.arange(0, 20000, 4, dtype=torch.int32, device="cuda")
expect_timeout(lambda: rmm.rmm_reduced_gemm(Ad, Bd, idx), 5)
Y = rmm.rmm_reduced_gemm(Ad, Bd, idx)
assert rel(Y.float().cpu().numpy(), oracle.reduced_gemm(A, B, idx.cpu().numpy())) <= 1e-2
assert rmm.rmm_status_read() == 0
""",
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_expired_wait_is_reported_and_the_workspace_recovers(case):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    env = dict(os.environ, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", PRELUDE + CASES[case]], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
