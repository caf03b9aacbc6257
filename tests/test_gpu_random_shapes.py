"""Seeded random shapes through the whole path (GPU only): products and attention against the oracle.  The fixed
parametrisations elsewhere pin the known edges; this file walks shapes nobody thought of."""
import numpy as np
import pytest
import torch

import paper_2608_13426_b200 as rmm
from paper_2608_13426_b200 import synth
from test_gpu_parity import TOL_BF16, check_attention, check_index_set, rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _device():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    torch.cuda.set_device(0)
    yield
    assert rmm.rmm_status_read() == 0


@pytest.mark.parametrize("case", range(24))
def test_random_product(oracle, case):
    rng = np.random.default_rng(1000 + case)
    M = int(rng.integers(1, 700))
    K = int(rng.integers(1, 90)) * 8 if case % 3 else int(rng.integers(1, 700))
    N = int(rng.integers(1, 90)) * 8 if case % 4 else int(rng.integers(1, 700))
    rho = float(rng.choice([0.1, 0.25, 0.4, 0.5, 0.75, 0.9, 1.0]))
    A = synth.heavy_tailed_activations(M, K, seed=case)
    B = synth.weight(K, N, seed=case + 1)
    k = oracle.keep_count(rho, K)
    Y, idx = rmm.rmm(A.cuda(), B.cuda(), rho)
    e64, _ = oracle.score(A)
    idx_np = idx.cpu().numpy()
    check_index_set(idx_np, e64, k)
    want = oracle.reduced_gemm(A, B, idx_np)
    got = Y.float().cpu().numpy()
    assert np.linalg.norm(got - want) <= TOL_BF16 * max(np.linalg.norm(want), 1e-6), (M, K, N, rho)


@pytest.mark.parametrize("case", range(16))
def test_random_attention(oracle, case):
    rng = np.random.default_rng(2000 + case)
    Hkv = int(rng.integers(1, 4))
    Hq = Hkv * int(rng.integers(1, 4))
    B = int(rng.integers(1, 3))
    Lq = int(rng.integers(1, 520))
    Lk = int(rng.integers(max(1, Lq - 100), Lq + 300)) if case % 2 else Lq
    Dh = int(rng.choice([32, 64, 72, 128]))
    causal = bool(rng.integers(0, 2))
    rho_d = float(rng.choice([0.25, 0.5, 0.75, 1.0]))
    rho_t = float(rng.choice([0.25, 0.5, 0.8, 1.0]))
    assert check_attention(oracle, B, Hq, Hkv, Lq, Lk, Dh, causal, rho_d, rho_t, seed=3000 + case), (B, Hq, Hkv, Lq, Lk, Dh, causal, rho_d, rho_t)
