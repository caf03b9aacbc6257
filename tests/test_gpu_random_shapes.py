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


@pytest.mark.parametrize("case", range(12))
def test_random_masked_attention(oracle, case):
    """Additive masks of random shape (full, per head, per sequence, shared; random holes and biases) on random attention
    shapes: aligned mask rows with rho_t = 1 take the masked one-pass kernel, everything else the composed form."""
    rng = np.random.default_rng(4000 + case)
    g = torch.Generator().manual_seed(4000 + case)
    Hkv = int(rng.integers(1, 3))
    Hq = Hkv * int(rng.integers(1, 4))
    B = int(rng.integers(1, 3))
    Lq = int(rng.integers(1, 400))
    Lk = (int(rng.integers(max(1, Lq - 60), Lq + 200)) + 3) // 4 * 4 if case % 3 else int(rng.integers(max(1, Lq - 60), Lq + 200))
    Dh = int(rng.choice([32, 64, 128]))
    causal = bool(rng.integers(0, 2))
    rho_d = float(rng.choice([0.25, 0.5, 1.0]))
    rho_t = 1.0 if case % 2 else float(rng.choice([0.5, 0.8]))
    shape = [(B, Hq, Lq, Lk), (1, Hq, Lq, Lk), (B, 1, Lq, Lk), (Lq, Lk), (1, 1, 1, Lk)][case % 5]
    M = torch.randn(*shape, generator=g) * 1.5
    M[torch.rand(*shape, generator=g) < 0.25] = -float("inf")
    M[..., 0] = 0.0                                                           # (with the causal mask rows may still see nothing)
    assert check_attention(oracle, B, Hq, Hkv, Lq, Lk, Dh, causal, rho_d, rho_t, seed=4100 + case, mask=M), \
        (B, Hq, Hkv, Lq, Lk, Dh, causal, rho_d, rho_t, shape)


@pytest.mark.parametrize("case", range(10))
def test_random_scored_and_8_bit_products(oracle, case):
    """Random shapes through the product that scores its own output and through the 8-bit product."""
    rng = np.random.default_rng(5000 + case)
    M = int(rng.integers(1, 1500))
    K = int(rng.integers(2, 140)) * 16
    N = int(rng.integers(1, 120)) * 8
    rho = float(rng.choice([0.25, 0.5, 0.75, 1.0]))
    A = synth.heavy_tailed_activations(M, K, seed=case + 50)
    W = synth.weight(K, N, seed=case + 51, dtype=torch.float32)
    Ad = A.cuda()
    idx, _, _, _ = rmm.rmm_score_select(Ad, rho=rho)
    idx_np = idx.cpu().numpy()
    check_index_set(idx_np, oracle.score(A)[0], oracle.keep_count(rho, K))
    # the product that scores its output: energies of Y as stored, and the next selection from them
    Y, e = rmm.rmm_reduced_gemm(Ad, W.to(torch.bfloat16).cuda(), idx, want_energy=True)
    e64, _ = oracle.score(Y.cpu())
    assert np.allclose(e.cpu().numpy(), e64, rtol=3e-6, atol=1e-30), (M, K, N, rho)
    want = oracle.reduced_gemm(A, W.to(torch.bfloat16), idx_np)
    assert rel_fro(Y.float().cpu().numpy(), want) <= TOL_BF16
    k2 = oracle.keep_count(0.5, N)
    check_index_set(rmm.rmm_select(e, k=k2).cpu().numpy(), e64, k2)
    # 8-bit operands
    b_scale = float(W.abs().max()) / 448.0
    Bq = (W.t().contiguous() / b_scale).to(torch.float8_e4m3fn)
    Yq, s = rmm.rmm_reduced_gemm_q8(Ad, Bq.cuda(), b_scale, idx, out_dtype=torch.float32, want_scales=True)
    rows = sorted({0, M // 3, M - 1})
    Bv = Bq.to(torch.float64).numpy()
    for r in rows:
        Yo, so = oracle.reduced_gemm_q8(A[r:r + 1], Bv, b_scale, idx_np)
        assert float(s[r]) == float(so[0]), (M, K, N, rho, r)
        assert rel_fro(Yq[r].cpu().numpy(), Yo[0]) <= 1e-5, (M, K, N, rho, r)
