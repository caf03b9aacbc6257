"""Parity at the full sizes of the benchmark configurations (GPU only): index sets are checked in full against
the oracle, products on sampled rows that the oracle computes one by one (tile edges included)."""
import math

import numpy as np
import pytest
import torch

import paper_2608_13426_b200 as rmm
from paper_2608_13426_b200 import synth
from test_gpu_parity import TOL_BF16, check_index_set, rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _device():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    torch.cuda.set_device(0)
    yield
    assert rmm.rmm_status_read() == 0


def sample_rows(n, count, seed=0):
    edges = [0, 1, 127, 128, 129, n // 2 - 1, n // 2, n - 2, n - 1]
    extra = np.random.default_rng(seed).choice(n, count, replace=False).tolist()
    return sorted({r for r in edges + extra if 0 <= r < n})


@pytest.mark.parametrize("rho", [0.5, 0.75])
def test_attention_prefill_qk_head_dim_reduction(oracle, rho):
    """7B-class prefill: 32 heads, seq 4096, head_dim 128, 4 outlier dims per head x10; index set per head from Q,
    S~ = Q[:, I] K[:, I]^T / sqrt(128) written as a batched product with K-contiguous B."""
    H, L, Dh = 32, 4096, 128
    Q, K, _ = synth.attention_qkv(1, H, H, L, L, Dh, seed=0)
    Qd, Kd = Q[0].cuda(), K[0].cuda()
    kd = oracle.keep_count(rho, Dh)
    idx, _, _, _ = rmm.rmm_score_select(Qd, rho=rho)
    S = rmm.rmm_reduced_gemm(Qd, Kd.transpose(1, 2), idx, scale=1.0 / math.sqrt(Dh))
    assert S.shape == (H, L, L) and S.dtype == torch.bfloat16
    idx_np = idx.cpu().numpy()
    rows = sample_rows(L, 3)
    for h in range(H):
        e64, _ = oracle.score(Q[0, h])
        check_index_set(idx_np[h], e64, kd)
        for r in rows:
            want = oracle.reduced_gemm(Q[0, h], K[0, h].T, idx_np[h], rows=(r, r + 1))[r] / math.sqrt(Dh)
            assert rel_fro(S[h, r].float().cpu().numpy(), want) <= TOL_BF16


@pytest.mark.parametrize("rho", [0.25, 0.5])
def test_long_context_pv_sequence_reduction(oracle, rho):
    """Long-context PV: seq 16384, head_dim 128, P = causal softmax given as a bf16 input, keys selected per head.
    Eight of the 32 heads (P alone is 0.5 GB per head; heads are independent problems of identical shape)."""
    H, L, Dh = 8, 16384, 128
    P = synth.attention_probs(L, H, Dh, seed=3, causal=True, device="cuda")
    V = synth.gaussian((H, L, Dh), 1.0, seed=5).cuda()
    kt = oracle.keep_count(rho, L)
    idx, _, _, ret = rmm.rmm_score_select(P, rho=rho, want_retained=True)
    O = rmm.rmm_reduced_gemm(P, V, idx)
    idx_np = idx.cpu().numpy()
    Pc, Vc = P.cpu(), V.cpu()
    rows = sample_rows(L, 4)
    for h in range(H):
        e64, _ = oracle.score(Pc[h])
        check_index_set(idx_np[h], e64, kt)
        _, kept = oracle.select(e64, kt)
        assert float(ret[h]) == pytest.approx(kept / e64.sum(), rel=1e-5)
        for r in rows:
            want = oracle.reduced_gemm(Pc[h], Vc[h], idx_np[h], rows=(r, r + 1))[r]
            got = O[h, r].float().cpu().numpy()
            assert np.linalg.norm(got - want) <= TOL_BF16 * max(np.linalg.norm(want), 1e-3)


def test_70b_class_projection_sampled(oracle):
    """70B-class K/V projection: 32768 tokens x 8192 hidden -> 1024, activations with 1 % heavy-tailed channels;
    the score pass and the select run at full size, the product is checked on sampled rows."""
    M, K, N = 32768, 8192, 1024
    A = synth.heavy_tailed_activations(M, K, seed=7, device="cuda")
    B = synth.weight(K, N, seed=8, device="cuda")
    Ac, Bc = A.cpu(), B.cpu()
    e64, _ = oracle.score(Ac)
    for rho in (0.25, 0.75):
        k = oracle.keep_count(rho, K)
        Y, idx = rmm.rmm(A, B, rho)
        idx_np = idx.cpu().numpy()
        check_index_set(idx_np, e64, k)
        for r in sample_rows(M, 6, seed=1):
            want = oracle.reduced_gemm(Ac, Bc, idx_np, rows=(r, r + 1))[r]
            assert rel_fro(Y[r].float().cpu().numpy(), want) <= TOL_BF16


def test_70b_class_down_projection_index_set(oracle):
    """70B-class down projection: contraction over the 28672-wide intermediate axis (select in its own launch,
    keys cached in shared memory); index set in full, product on sampled rows of a 4096-token slice."""
    M, K, N = 4096, 28672, 8192
    A = synth.heavy_tailed_activations(M, K, seed=9, device="cuda")
    B = synth.weight(K, N, seed=10, device="cuda")
    Ac, Bc = A.cpu(), B.cpu()
    e64, _ = oracle.score(Ac)
    k = oracle.keep_count(0.5, K)
    Y, idx = rmm.rmm(A, B, 0.5)
    idx_np = idx.cpu().numpy()
    check_index_set(idx_np, e64, k)
    for r in sample_rows(M, 3, seed=2):
        want = oracle.reduced_gemm(Ac, Bc, idx_np, rows=(r, r + 1))[r]
        assert rel_fro(Y[r].float().cpu().numpy(), want) <= TOL_BF16


def test_70b_class_down_projection_selected_from_the_up_projection_epilogue(oracle):
    """70B-class MLP at full size: the up projection (32768 x 8192 x 28672, CTA pairs) accumulates the column energies
    of the activations it writes in its epilogue; the down projection's index set, selected from them with no pass over
    the 1.9 GB of activations, must lie inside the strict tie band of the oracle's scores of those activations."""
    M, K, N = 32768, 8192, 28672
    X = synth.heavy_tailed_activations(M, K, seed=21, device="cuda")
    W = synth.weight(K, N, seed=22, device="cuda")
    H, e = rmm.rmm_reduced_gemm(X, W, None, want_energy=True)
    k = rmm.rmm_keep_count(0.5, N)
    idx = rmm.rmm_select(e, k=k)
    assert rmm.rmm_status_read() == 0
    e64, _ = oracle.score(H.cpu())
    check_index_set(idx.cpu().numpy(), e64, k)
    assert np.allclose(e.cpu().numpy(), e64, rtol=3e-6)
    for r in sample_rows(M, 2, seed=5):                                # and the activations themselves, on sampled rows
        want = oracle.reduced_gemm(X.cpu(), W.cpu(), np.arange(K, dtype=np.int32), rows=(r, r + 1))[r]
        assert rel_fro(H[r].float().cpu().numpy(), want) <= TOL_BF16


def test_70b_class_down_projection_with_8_bit_operands(oracle):
    """The 8-bit form at the size and in the launch configuration the benchmark times (32768 x 28672 x 8192, rho = 0.5: the
    streaming quantising gather and CTA-pair tiles on the fp8 tensor cores): row steps bit for bit and outputs on sampled
    rows against the oracle's product of the dequantised operands."""
    M, K, N = 32768, 28672, 8192
    A = synth.heavy_tailed_activations(M, K, seed=31, device="cuda")
    W = synth.weight(K, N, seed=32, dtype=torch.float32, device="cuda")
    b_scale = float(W.abs().max()) / 448.0
    Bq = (W.t().contiguous() / b_scale).to(torch.float8_e4m3fn)                   # stored [N, K]
    del W
    idx, _, _, _ = rmm.rmm_score_select(A, rho=0.5)
    Y, s = rmm.rmm_reduced_gemm_q8(A, Bq, b_scale, idx, want_scales=True)
    assert rmm.rmm_status_read() == 0
    idx_np = idx.cpu().numpy()
    Bv = Bq.cpu().to(torch.float64).numpy()
    for r in sample_rows(M, 3, seed=6):
        Yo, so = oracle.reduced_gemm_q8(A[r:r + 1].cpu(), Bv, b_scale, idx_np)
        assert float(s[r]) == float(so[0]), r
        assert rel_fro(Y[r].float().cpu().numpy(), Yo[0]) <= TOL_BF16, r
    assert torch.isfinite(Y.float()).all()


def check_token_sets(oracle, tok, It, P, band=1e-4):
    """Token sets of the fused sweeps against the oracle's P (evaluated on the GPU's feature sets): Theorem 1's
    criterion (retained energy within 1e-6 of the optimum) and equality outside a 1e-4 band."""
    kt = tok.shape[-1]
    a2 = (P ** 2).sum(axis=0)
    assert np.all(np.diff(tok) > 0) and tok.min() >= 0 and tok.max() < P.shape[1]
    assert a2[tok].sum() >= (1 - 1e-6) * a2[It].sum()
    s = np.sqrt(a2)
    tau = np.sort(s)[::-1][kt - 1]
    diff = np.setxor1d(tok, It)
    assert np.all(np.abs(s[diff] - tau) <= band * s.max())


def test_reduced_attention_multi_tile(oracle):
    """Reduced attention across several tiles and head groups: 8 query / 2 kv heads, 1536 x 1536, causal.  O of every
    head is compared with the oracle evaluated on the GPU's own feature and token sets."""
    B, Hq, Hkv, L, Dh = 1, 8, 2, 1536, 128
    Q, K, V = synth.attention_qkv(B, Hq, Hkv, L, L, Dh, seed=11)
    O, idx_feat, idx_tok = rmm.rmm_reduced_attn(Q.cuda(), K.cuda(), V.cuda(), True, 0.5, 0.5, want_idx=True)
    feat, tok = idx_feat.cpu().numpy(), idx_tok.cpu().numpy()
    for h in range(Hq):
        check_index_set(feat[0, h], oracle.score(Q[0, h])[0], 64)
    _, _, It, P = oracle.attn(Q, K, V, True, 0.5, 0.5, round_p=True, want_p=True, idx_feat=feat)
    Oo = oracle.attn(Q, K, V, True, 0.5, 0.5, round_p=True, idx_feat=feat, idx_tok=tok)[0]
    for h in range(Hq):
        check_token_sets(oracle, tok[0, h], It[0, h], P[0, h])
        assert rel_fro(O[0, h].float().cpu().numpy(), Oo[0, h]) <= TOL_BF16


@pytest.mark.parametrize("rho_t", [1.0, 0.5])
def test_long_context_fused_attention(oracle, rho_t):
    """Fused reduced attention at 8192 tokens (a key ring that wraps many times, several items per block, all four
    kernel modes): 2 query heads on 1 kv head, head_dim 128, causal, rho_d = 0.5.  O of both heads is compared with
    the oracle evaluated on the GPU's own sets."""
    B, Hq, Hkv, L, Dh = 1, 2, 1, 8192, 128
    Q, K, V = synth.attention_qkv(B, Hq, Hkv, L, L, Dh, seed=21)
    O, idx_feat, idx_tok = rmm.rmm_reduced_attn(Q.cuda(), K.cuda(), V.cuda(), True, 0.5, rho_t, want_idx=True)
    feat = idx_feat.cpu().numpy()
    for h in range(Hq):
        check_index_set(feat[0, h], oracle.score(Q[0, h])[0], 64)
    tok = None
    if rho_t < 1.0:
        tok = idx_tok.cpu().numpy()
        _, _, It, P = oracle.attn(Q, K, V, True, 0.5, rho_t, round_p=True, want_p=True, idx_feat=feat)
        for h in range(Hq):
            check_token_sets(oracle, tok[0, h], It[0, h], P[0, h])
        del P
    Oo = oracle.attn(Q, K, V, True, 0.5, rho_t, round_p=True, idx_feat=feat, idx_tok=tok)[0]
    for h in range(Hq):
        assert rel_fro(O[0, h].float().cpu().numpy(), Oo[0, h]) <= TOL_BF16


# ------------------------------------------------------------------------------------------------
# 70B-class layer at the sizes the benchmark times (32768 prefill tokens): index sets in full, products on tile-edge
# and seeded rows that the oracle computes one by one
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,K,N", [("gate_up", 8192, 28672), ("q_o", 8192, 8192), ("down", 28672, 8192)])
def test_70b_class_layer_products_full_size(oracle, name, K, N):
    M = 32768
    A = synth.heavy_tailed_activations(M, K, seed=13, device="cuda")
    B = synth.weight(K, N, seed=14, device="cuda")
    Ac, Bc = A.cpu(), B.cpu()
    e64, _ = oracle.score(Ac)
    rows = sample_rows(M, 4, seed=3) + [255, 256, 257]          # 256: the edge of a CTA pair's tile
    for rho in (0.25, 0.5):
        k = oracle.keep_count(rho, K)
        Y, idx = rmm.rmm(A, B, rho)
        idx_np = idx.cpu().numpy()
        check_index_set(idx_np, e64, k)
        Yr = Y[rows].float().cpu().numpy()
        assert np.isfinite(Y.float().sum().item())               # no element of the 32768 x N output was left unwritten
        del Y
        for i, r in enumerate(rows):
            want = oracle.reduced_gemm(Ac, Bc, idx_np, rows=(r, r + 1))[r]
            assert rel_fro(Yr[i], want) <= TOL_BF16, (name, rho, r)
    assert rmm.rmm_status_read() == 0


def test_70b_class_attention_full_size(oracle):
    """64 query heads on 8 kv heads, 32768 tokens, head_dim 128, causal, rho_d = 0.5 (feature reduction, one fused
    pass).  Feature sets of every head in full; O of two query heads (from different kv groups) on sampled query rows,
    against the oracle evaluated on the GPU's feature sets for those rows only."""
    Hq, Hkv, L, Dh = 64, 8, 32768, 128
    Q, K, V = synth.attention_qkv(1, Hq, Hkv, L, L, Dh, seed=17, device="cuda")
    O, idx_feat, _ = rmm.rmm_reduced_attn(Q, K, V, True, 0.5, 1.0, want_idx=True)
    assert bool(torch.isfinite(O.float().sum()))
    feat = idx_feat.cpu().numpy()
    for h in range(Hq):
        check_index_set(feat[0, h], oracle.score(Q[0, h].cpu())[0], 64)
    rows = sample_rows(L, 6, seed=4)
    for h in (5, 62):
        g = h // (Hq // Hkv)
        Qh, Kg, Vg = Q[:, h:h + 1].cpu(), K[:, g:g + 1].cpu(), V[:, g:g + 1].cpu()
        Oo = oracle.attn(Qh, Kg, Vg, True, 0.5, 1.0, round_p=True, idx_feat=feat[:, h:h + 1], rows=rows)[0]
        got = O[0, h][rows].float().cpu().numpy()
        for i, r in enumerate(rows):
            assert rel_fro(got[i], Oo[0, 0, i]) <= TOL_BF16, (h, r)
    assert rmm.rmm_status_read() == 0
