"""Pins of the CPU oracle against what the paper and the mathematics fix (CPU only).

Each test names the passage it pins.  None of them re-types the oracle's own loops: they use
exact rational arithmetic, brute-force enumeration, closed forms, inequalities the paper
proves, and library routines (numpy matmul, torch softmax / scaled_dot_product_attention).
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2608_13426_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def rand_bf16(shape, seed, std=1.0):
    return synth.gaussian(shape, std, seed)


# --------------------------------------------------------------------------------------------
# keep count: |I| = ceil(rho d), Sec. 3.2
# --------------------------------------------------------------------------------------------
def test_keep_count_exact_rationals(oracle):
    """ceil(p/q * K) in exact integer arithmetic for a grid of decimal-looking ratios."""
    for q in (2, 3, 4, 5, 8, 10, 16, 20, 25, 100, 128, 1000):
        for p in range(1, q + 1):
            for K in (1, 2, 7, 8, 9, 10, 64, 100, 127, 128, 129, 512, 1000, 4096, 8192, 28672, 32768):
                want = max(1, min(K, math.ceil(Fraction(p, q) * K)))
                assert oracle.keep_count(p / q, K) == want, (p, q, K)


def test_keep_count_large_axes_and_near_integers(oracle):
    """The snap to an integer is a matter of a few ulps at any size: on axes of 2^15 .. 2^30 a ratio that is
    integral in exact arithmetic gives that integer, and a ratio a little above j / K (from 1e-7 down to a few
    hundred ulps) gives j + 1, as exact rational arithmetic on the double that was passed says."""
    for K in (32768, 28672, 1 << 20, (1 << 24) + 3, 1 << 30):
        for q in (3, 5, 7, 10, 100, 1000):
            for p in (1, q // 2, q - 1):
                rho = p / q
                exact = Fraction(p, q) * K
                if exact.denominator == 1:                      # integral in exact arithmetic: no rounding up
                    assert oracle.keep_count(rho, K) == int(exact), (p, q, K)
                else:
                    assert oracle.keep_count(rho, K) == math.ceil(Fraction(rho) * K), (p, q, K)
        for j in (1, K // 3, K - 2):
            for above in (1e-3, 1e-5, 1e-7 * K / 32768):
                rho = (j + above) / K                           # genuinely fractional: ceil gives j + 1
                assert math.ceil(Fraction(rho) * K) == j + 1
                assert oracle.keep_count(rho, K) == j + 1, (j, above, K)
            assert oracle.keep_count(j / K, K) == j             # j / K itself rounds to j even if the product is a hair off


def test_keep_count_paper_values(oracle):
    for line in open(os.path.join(GOLDEN, "keep_count_paper.txt")):
        if line.startswith("#") or not line.strip():
            continue
        p, q, d, k = map(int, line.split())
        assert oracle.keep_count(p / q, d) == k


def test_keep_count_domain(oracle):
    """rho in (0, 1] only (Sec. 3.2); the count is always in [1, K]."""
    for bad in (0.0, -0.1, 1.0000001, 2.0, float("nan"), float("inf")):
        assert oracle.keep_count(bad, 16) == -1
    assert oracle.keep_count(0.5, 0) == -1
    assert oracle.keep_count(1e-12, 16) == 1
    assert oracle.keep_count(1.0, 16) == 16
    for K in (1, 5, 33):
        assert oracle.keep_count(1.0 / K, K) == 1
    for K in (2, 5, 33):
        assert oracle.keep_count((K - 1) / K, K) == K - 1


# --------------------------------------------------------------------------------------------
# score: s_j = ||A[:, j]||_2, Sec. 3.2
# --------------------------------------------------------------------------------------------
def test_score_closed_forms(oracle):
    M, K = 37, 9
    A = np.zeros((M, K), np.float32)
    A[:, 0] = 3.0                      # constant column: |c| sqrt(M)
    A[5, 1] = -7.0                     # single entry: |a|
    A[:, 2] = np.arange(M)             # sum i^2 = (M-1)M(2M-1)/6
    A[0, 3], A[1, 3] = 3.0, 4.0        # 3-4-5
    e, s = oracle.score(A)
    assert s[0] == pytest.approx(3.0 * math.sqrt(M), rel=1e-15)
    assert s[1] == 7.0
    assert e[2] == (M - 1) * M * (2 * M - 1) / 6
    assert s[3] == 5.0
    assert np.all(s[4:] == 0.0)


def test_score_exact_against_rational_sum(oracle):
    """bf16 inputs widen exactly and the compensated sum is the exact sum, correctly rounded to
    within 1 ulp: compare with Python's exactly rounded fsum on exact rational squares."""
    A = rand_bf16((301, 17), seed=11)
    e, s = oracle.score(A)
    Af = A.to(torch.float64).numpy()      # torch's own bf16 -> fp64 widening, not the oracle's
    for j in range(A.shape[1]):
        want = math.fsum(float(x) * float(x) for x in Af[:, j])
        assert abs(e[j] - want) <= 2 * np.spacing(want)
        assert s[j] == pytest.approx(math.sqrt(want), rel=1e-15)


def test_score_reads_columns_not_rows(oracle):
    """A transposed-operand mistake would give row norms: make them differ."""
    A = np.zeros((4, 3), np.float64)
    A[0] = [1.0, 2.0, 3.0]
    e, s = oracle.score(A)
    assert list(e) == [1.0, 4.0, 9.0]
    e2, _ = oracle.score(A.T)               # strided view, no copy
    assert list(e2) == [14.0, 0.0, 0.0, 0.0]


# --------------------------------------------------------------------------------------------
# select: TopK, Sec. 3.2; Theorem 1 (minimax optimality) and Eq. 3
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("K,k", [(5, 2), (8, 3), (10, 5), (12, 7), (13, 1), (9, 9)])
def test_select_brute_force_optimal(oracle, K, k):
    """Over all C(K,k) subsets the selected one attains max sum_{j in I} e_j, i.e. minimises the
    residual ||A[:, I-bar]||_F of Eq. 3, and is the unique maximiser when keys are distinct."""
    A = rand_bf16((23, K), seed=100 + K)
    e, _ = oracle.score(A)
    assert len(set(e.tolist())) == K
    idx, kept = oracle.select(e, k)
    assert len(idx) == k and list(idx) == sorted(set(idx.tolist()))
    best, best_sets = -1.0, []
    for sub in itertools.combinations(range(K), k):
        v = math.fsum(e[list(sub)])
        if v > best:
            best, best_sets = v, [sub]
        elif v == best:
            best_sets.append(sub)
    assert best_sets == [tuple(idx.tolist())]
    assert kept == pytest.approx(best, rel=1e-14)
    # Eq. 3: the inner maximum equals the Frobenius norm of the discarded columns
    Af = bf16_to_f64(A)
    rest = [j for j in range(K) if j not in set(idx.tolist())]
    assert math.sqrt(max(0.0, e.sum() - kept)) == pytest.approx(np.linalg.norm(Af[:, rest]), rel=1e-12, abs=1e-12)


def test_select_ties_go_to_lowest_index(oracle):
    key = np.array([1.0, 5.0, 5.0, 5.0, 0.5, 5.0, 9.0])
    idx, _ = oracle.select(key, 3)          # 9.0 and two of the four 5.0s
    assert idx.tolist() == [1, 2, 6]
    idx, _ = oracle.select(np.full(10, 2.5), 4)
    assert idx.tolist() == [0, 1, 2, 3]


def test_duplicate_columns_straddling_threshold(oracle):
    """Two bit-identical columns, one place left: the lower index is kept."""
    A = rand_bf16((40, 12), seed=5).clone()
    e, _ = oracle.score(A)
    order = np.argsort(-e, kind="stable")
    k = 5
    a, b = int(order[k - 1]), int(order[k])    # the threshold column and the first one out
    lo, hi = min(a, b), max(a, b)
    A[:, hi] = A[:, lo]
    e2, _ = oracle.score(A)
    assert e2[lo] == e2[hi]
    idx, _ = oracle.select(e2, oracle.keep_count(k / 12, 12))
    assert lo in idx.tolist() and hi not in idx.tolist()


def test_select_nesting_and_monotone_energy(oracle):
    """I(rho1) is a subset of I(rho2) for rho1 < rho2, and eps_A(rho) is non-increasing (Sec. 3.4)."""
    A, _, _ = synth.outlier_product(M=32, K=96, N=8, seed=3)
    e, _ = oracle.score(A)
    prev, prev_eps = set(), 1.0
    for rho in (0.1, 0.25, 0.5, 0.7, 0.75, 0.9, 1.0):
        idx, kept = oracle.select(e, oracle.keep_count(rho, 96))
        cur = set(idx.tolist())
        assert prev <= cur
        eps = 1.0 - kept / e.sum()
        assert eps <= prev_eps + 1e-15
        prev, prev_eps = cur, eps
    assert prev == set(range(96)) and abs(prev_eps) < 1e-15


def test_printed_energy_example(oracle):
    """Top 70 % of dimensions holding 95 % of the energy gives eps_A(0.7) = 0.05 (golden file)."""
    rho, retained, eps = [float(x) for x in
                          [l for l in open(os.path.join(GOLDEN, "energy_example.txt")) if l[0] != "#"][0].split()]
    K, M = 20, 6
    k = oracle.keep_count(rho, K)
    assert k == 14
    energies = np.empty(K)
    big = np.linspace(1.0, 2.0, k)
    small = np.linspace(0.1, 0.2, K - k)
    energies[::-1][:k] = big / big.sum() * retained         # large ones at the high indices
    energies[: K - k] = small / small.sum() * (1.0 - retained)
    A = np.zeros((M, K))
    A[0] = np.sqrt(energies)                                 # column j has norm sqrt(energy_j)
    e, _ = oracle.score(A)
    idx, kept = oracle.select(e, k)
    assert idx.tolist() == list(range(K - k, K))
    assert 1.0 - kept / e.sum() == pytest.approx(eps, abs=1e-12)


# --------------------------------------------------------------------------------------------
# reduced product: RMM_rho(A, B) = A[:, I] B[I, :], Sec. 3.2
# --------------------------------------------------------------------------------------------
def test_rho_one_is_the_dense_product_exactly(oracle):
    A, B, _ = synth.outlier_product(M=17, K=40, N=9, seed=2)
    Y, idx, _ = oracle.rmm(A, B, 1.0)
    assert idx.tolist() == list(range(40))
    D = oracle.dense_gemm(A, B)
    assert np.array_equal(Y, D)
    assert np.allclose(D, bf16_to_f64(A) @ bf16_to_f64(B), rtol=1e-13, atol=1e-13)


def test_reduced_product_library_special_cases(oracle):
    """Equals a library matmul on pre-gathered contiguous operands, and a dense product with the
    other columns zeroed; a transposed or mis-indexed operand fails here (M, K, N all distinct)."""
    A, B, _ = synth.outlier_product(M=19, K=48, N=11, seed=4)
    Y, idx, _ = oracle.rmm(A, B, 0.4)
    assert len(idx) == 20
    Af, Bf = bf16_to_f64(A), bf16_to_f64(B)
    assert np.allclose(Y, np.ascontiguousarray(Af[:, idx]) @ np.ascontiguousarray(Bf[idx, :]), rtol=1e-13, atol=1e-13)
    Az = np.zeros_like(Af)
    Az[:, idx] = Af[:, idx]
    assert np.allclose(Y, Az @ Bf, rtol=1e-13, atol=1e-13)
    # strided operands (B stored N x K, i.e. a transposed view) give the same numbers
    Bt = np.ascontiguousarray(Bf.T)
    assert np.array_equal(oracle.reduced_gemm(Af, Bt.T, idx), oracle.reduced_gemm(Af, Bf, idx))
    # a sample of rows equals those rows of the full result
    part = oracle.reduced_gemm(A, B, idx, rows=(3, 7))
    assert np.array_equal(part[3:7], Y[3:7]) and not part[:3].any() and not part[7:].any()


def test_permutation_of_contraction_axis(oracle):
    """AB = sum_j A[:,j] B[j,:] (Eq. 1) does not depend on the order of j: permuting the axis
    permutes I and leaves Y unchanged."""
    A, B, _ = synth.outlier_product(M=21, K=64, N=10, seed=6)
    perm = torch.randperm(64, generator=torch.Generator().manual_seed(9))
    Y, idx, _ = oracle.rmm(A, B, 0.5)
    Yp, idxp, _ = oracle.rmm(A[:, perm].contiguous(), B[perm, :].contiguous(), 0.5)
    assert sorted(perm[idxp.tolist()].tolist()) == idx.tolist()
    assert np.allclose(Y, Yp, rtol=1e-12, atol=1e-12)


def test_rank_one_closed_form_meets_bound_with_equality(oracle):
    """A = u alpha^T, B = b v^T, unit u, v, non-negative alpha, b: s_j = alpha_j,
    RMM = (sum_{j in I} alpha_j b_j) u v^T and the error norm equals sum_{j not in I} alpha_j b_j
    (Eq. 2 with equality).  With b = alpha / ||alpha_Ibar|| on the discarded set (Remark 1) the error
    equals ||A[:, I-bar]||_F (Eq. 3)."""
    rng = np.random.default_rng(7)
    n, d, m, k = 9, 14, 6, 6
    u = rng.standard_normal(n); u /= np.linalg.norm(u)
    v = rng.standard_normal(m); v /= np.linalg.norm(v)
    alpha = rng.uniform(0.1, 3.0, d)
    b = rng.uniform(0.1, 2.0, d)
    A = np.outer(u, alpha)
    B = np.outer(b, v)
    e, s = oracle.score(A)
    assert np.allclose(s, alpha, rtol=1e-13)
    idx, _ = oracle.select(e, k)
    assert set(idx.tolist()) == set(np.argsort(-alpha)[:k].tolist())
    Y = oracle.reduced_gemm(A, B, idx)
    assert np.allclose(Y, (alpha[idx] * b[idx]).sum() * np.outer(u, v), rtol=1e-12, atol=1e-13)
    rest = np.setdiff1d(np.arange(d), idx)
    err = np.linalg.norm(oracle.dense_gemm(A, B) - Y)
    assert err == pytest.approx((alpha[rest] * b[rest]).sum(), rel=1e-12)
    b2 = np.zeros(d)
    b2[rest] = alpha[rest] / np.linalg.norm(alpha[rest])
    B2 = np.outer(b2, v)
    err2 = np.linalg.norm(oracle.dense_gemm(A, B2) - oracle.reduced_gemm(A, B2, idx))
    assert err2 == pytest.approx(np.linalg.norm(A[:, rest]), rel=1e-12)


@pytest.mark.parametrize("rho", [0.25, 0.5, 0.75])
def test_error_bounds_hold(oracle, rho):
    """||AB - Y||_F <= sum_{j not in I} s_j ||B[j,:]|| (Eq. 2) <= ||A_Ibar||_F ||B_Ibar||_F (Eq. 4),
    and the normalised form <= sqrt(eps_A eps_B) (Eq. 6); eps_A is the minimum over a random
    sample of other index sets of the same size (Theorem 1)."""
    A, B, _ = synth.outlier_product(M=33, K=80, N=12, seed=8)
    Y, idx, e = oracle.rmm(A, B, rho)
    Af, Bf = bf16_to_f64(A), bf16_to_f64(B)
    rest = np.setdiff1d(np.arange(80), idx)
    err = np.linalg.norm(Af @ Bf - Y)
    b_norm = np.linalg.norm(Bf, axis=1)
    bound2 = (np.sqrt(e[rest]) * b_norm[rest]).sum()
    bound4 = np.linalg.norm(Af[:, rest]) * np.linalg.norm(Bf[rest])
    assert err <= bound2 * (1 + 1e-12) <= bound4 * (1 + 1e-12)
    eps_a = np.linalg.norm(Af[:, rest]) ** 2 / np.linalg.norm(Af) ** 2
    eps_b = np.linalg.norm(Bf[rest]) ** 2 / np.linalg.norm(Bf) ** 2
    assert err / (np.linalg.norm(Af) * np.linalg.norm(Bf)) <= math.sqrt(eps_a * eps_b) * (1 + 1e-12)
    rng = np.random.default_rng(1)
    for _ in range(200):
        other = rng.choice(80, size=len(idx), replace=False)
        rest_o = np.setdiff1d(np.arange(80), other)
        assert np.linalg.norm(Af[:, rest]) <= np.linalg.norm(Af[:, rest_o]) * (1 + 1e-12)


# --------------------------------------------------------------------------------------------
# bf16 rounding used for P
# --------------------------------------------------------------------------------------------
def test_round_bf16_matches_library_conversion(oracle):
    x = torch.randn(4000, generator=torch.Generator().manual_seed(3), dtype=torch.float32)
    x = torch.cat([x, x * 1e-3, x * 1e-30, x * 1e30, torch.tensor([0.0, 1.0, 1.00390625, 1.01171875, 3.0e38])])
    want = x.to(torch.bfloat16).to(torch.float64)
    got = torch.tensor([oracle.round_bf16(float(v)) for v in x.to(torch.float64)], dtype=torch.float64)
    assert torch.equal(want, got)
    # ties to even, directly from double: 1 + 2^-8 is exactly half way between 1 and 1 + 2^-7
    assert oracle.round_bf16(1.0 + 2.0 ** -8) == 1.0
    assert oracle.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 1.0 + 2.0 ** -7
    assert oracle.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6


# --------------------------------------------------------------------------------------------
# attention, Sec. 3.3
# --------------------------------------------------------------------------------------------
def sdpa_reference(Q, K, V, causal):
    """Textbook softmax attention by the library, fp64, grouped-query heads repeated."""
    Q, K, V = Q.double(), K.double(), V.double()
    Hq, Hkv = Q.shape[1], K.shape[1]
    K = K.repeat_interleave(Hq // Hkv, dim=1)
    V = V.repeat_interleave(Hq // Hkv, dim=1)
    Lq, Lk = Q.shape[2], K.shape[2]
    mask = None
    if causal:
        mask = torch.ones(Lq, Lk, dtype=torch.bool).tril(diagonal=Lk - Lq)
    return torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=mask)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("Hq,Hkv,Lq,Lk", [(4, 4, 12, 12), (4, 2, 9, 15), (8, 1, 7, 7)])
def test_attention_rho_one_is_textbook_attention(oracle, causal, Hq, Hkv, Lq, Lk):
    Q, K, V = synth.attention_qkv(2, Hq, Hkv, Lq, Lk, 16, seed=20, n_outlier=2)
    O, idx_feat, idx_tok, _ = oracle.attn(Q, K, V, causal, 1.0, 1.0, round_p=False)
    assert idx_tok is None and np.array_equal(idx_feat[0, 0], np.arange(16))
    want = sdpa_reference(Q, K, V, causal).numpy()
    assert np.allclose(O, want, rtol=1e-11, atol=1e-12)


def test_attention_feature_reduction_per_query_head(oracle):
    """I is chosen per query head from Q alone, K is gathered on the same dims, the scale keeps the
    full 1/sqrt(d_h): zeroing the unselected dims of Q and calling the library gives the same O."""
    B, Hq, Hkv, Lq, Lk, Dh = 1, 4, 2, 10, 14, 16
    Q, K, V = synth.attention_qkv(B, Hq, Hkv, Lq, Lk, Dh, seed=21, n_outlier=3)
    O, idx_feat, _, _ = oracle.attn(Q, K, V, True, 0.5, 1.0, round_p=False)
    Qz = torch.zeros_like(Q)
    for h in range(Hq):
        e, _ = oracle.score(Q[0, h])
        want_idx, _ = oracle.select(e, 8)
        assert np.array_equal(idx_feat[0, h], want_idx)
        Qz[0, h][:, want_idx.tolist()] = Q[0, h][:, want_idx.tolist()]
    assert len({tuple(idx_feat[0, h]) for h in range(Hq)}) > 1       # heads really differ
    want = sdpa_reference(Qz, K, V, True).numpy()
    assert np.allclose(O, want, rtol=1e-11, atol=1e-12)


def test_attention_token_reduction(oracle):
    """a_t = ||P[:, t]||_2 over query rows, T = TopK, O = P[:, T] V[T, :] without renormalisation:
    checked against library softmax + matmul, with T verified as the energy-optimal set."""
    B, Hq, Hkv, Lq, Lk, Dh = 1, 2, 1, 11, 13, 8
    Q, K, V = synth.attention_qkv(B, Hq, Hkv, Lq, Lk, Dh, seed=22, n_outlier=0)
    O, _, idx_tok, P = oracle.attn(Q, K, V, False, 1.0, 0.4, round_p=False, want_p=True)
    kt = 6
    assert idx_tok.shape == (1, 2, kt)
    for h in range(Hq):
        S = (Q[0, h].double() @ K[0, 0].double().T) / math.sqrt(Dh)
        Pl = torch.softmax(S, dim=-1).numpy()
        assert np.allclose(P[0, h], Pl, rtol=1e-12, atol=1e-15)
        a2 = (Pl * Pl).sum(axis=0)
        T = idx_tok[0, h]
        rest = np.setdiff1d(np.arange(Lk), T)
        assert list(T) == sorted(T) and a2[T].min() >= a2[rest].max()
        want = Pl[:, T] @ V[0, 0].double().numpy()[T, :]
        assert np.allclose(O[0, h], want, rtol=1e-11, atol=1e-13)
    # no renormalisation: with V = 1 the output is the kept probability mass, strictly below 1
    ones = torch.ones_like(V)
    O1, _, idx1, P1 = oracle.attn(Q, K, ones, False, 1.0, 0.4, round_p=False, want_p=True)
    mass = np.stack([P1[0, h][:, idx1[0, h]].sum(axis=1) for h in range(Hq)])
    assert np.allclose(O1[0, :, :, 0], mass, rtol=1e-12) and (mass < 1.0).all()


def test_attention_rounded_p_is_scored_and_multiplied(oracle):
    """With rounding on, P holds bf16 values, and the very same values are scored and multiplied."""
    Q, K, V = synth.attention_qkv(1, 2, 2, 9, 12, 8, seed=23, n_outlier=1)
    O, _, idx_tok, P = oracle.attn(Q, K, V, True, 0.75, 0.5, round_p=True, want_p=True)
    Pt = torch.from_numpy(P)
    assert torch.equal(Pt, Pt.to(torch.bfloat16).to(torch.float64))
    for h in range(2):
        a2 = (P[0, h] ** 2).sum(axis=0)
        T, _ = oracle.select(a2, 6)
        assert np.array_equal(T, idx_tok[0, h])
        want = P[0, h][:, T] @ V[0, h].double().numpy()[T, :]
        assert np.allclose(O[0, h], want, rtol=1e-12, atol=1e-14)
    # causal, Lq < Lk: query i sees keys t <= i + (Lk - Lq)
    assert P[0, 0][0, 4:].sum() == 0.0 and P[0, 0][0, 3] > 0.0


def test_attention_on_given_sets(oracle):
    """Sec. 3.3 defines S~ = Q[:, I] K[:, I]^T / sqrt(d_h) and O~ = P[:, T] V[T, :] for any I and T.  Handing the
    oracle's own choice back reproduces its result bit for bit; a foreign feature set equals the library on Q with
    the other dims zeroed; a foreign token set equals P[:, T] V[T, :] from the returned P; sets are reported back."""
    B, Hq, Hkv, Lq, Lk, Dh = 2, 4, 2, 9, 13, 16
    Q, K, V = synth.attention_qkv(B, Hq, Hkv, Lq, Lk, Dh, seed=24, n_outlier=2)
    O, If, It, P = oracle.attn(Q, K, V, True, 0.5, 0.5, round_p=True, want_p=True)
    O2, If2, It2, P2 = oracle.attn(Q, K, V, True, 0.5, 0.5, round_p=True, want_p=True, idx_feat=If, idx_tok=It)
    assert np.array_equal(O, O2) and np.array_equal(P, P2) and np.array_equal(If, If2) and np.array_equal(It, It2)
    # only one of the two handed in: the other is still chosen by TopK
    O3, _, It3, _ = oracle.attn(Q, K, V, True, 0.5, 0.5, round_p=True, idx_feat=If)
    assert np.array_equal(O3, O) and np.array_equal(It3, It)

    # a foreign feature set (not the TopK one), unrounded P: library attention on Q with the other dims zeroed
    rng = np.random.default_rng(0)
    kd = 8
    feat = np.stack([np.sort(rng.choice(Dh, kd, replace=False)) for _ in range(B * Hq)]).reshape(B, Hq, kd).astype(np.int32)
    assert not np.array_equal(feat, If)
    Of, Iff, _, _ = oracle.attn(Q, K, V, True, 0.5, 1.0, round_p=False, idx_feat=feat)
    assert np.array_equal(Iff, feat)
    Qz = torch.zeros_like(Q)
    for b in range(B):
        for h in range(Hq):
            Qz[b, h][:, feat[b, h].tolist()] = Q[b, h][:, feat[b, h].tolist()]
    assert np.allclose(Of, sdpa_reference(Qz, K, V, True).numpy(), rtol=1e-11, atol=1e-12)

    # a foreign token set: O = P[:, T] V[T, :] with the P of the same call, no renormalisation
    kt = oracle.keep_count(0.5, Lk)
    tok = np.stack([np.sort(rng.choice(Lk, kt, replace=False)) for _ in range(B * Hq)]).reshape(B, Hq, kt).astype(np.int32)
    Ot, _, Itt, Pt = oracle.attn(Q, K, V, True, 0.5, 0.5, round_p=True, want_p=True, idx_feat=If, idx_tok=tok)
    assert np.array_equal(Itt, tok) and np.array_equal(Pt, P)       # P does not depend on T
    for b in range(B):
        for h in range(Hq):
            want = P[b, h][:, tok[b, h]] @ V[b, h // (Hq // Hkv)].double().numpy()[tok[b, h], :]
            assert np.allclose(Ot[b, h], want, rtol=1e-12, atol=1e-14)
    assert not np.allclose(Ot, O)


def test_attention_with_an_additive_mask(oracle):
    """Sec. 3.3: P = softmax(S~ + M) with M the optional causal or attention mask.  (i) The causal mask written out as
    an additive 0 / -inf matrix reproduces causal = True exactly; (ii) a finite additive bias with some keys hidden
    equals the library's attention with that float mask, per head and broadcast over heads; (iii) a mask entry moves
    the logit it belongs to: hiding one key of one head zeroes that column of P and nothing in other heads; (iv) rows
    whose keys are all hidden give zeros; (v) token scores are taken on the masked P."""
    B, Hq, Hkv, Lq, Lk, Dh = 2, 4, 2, 9, 13, 16
    Q, K, V = synth.attention_qkv(B, Hq, Hkv, Lq, Lk, Dh, seed=26, n_outlier=2)
    tri = np.where(np.tril(np.ones((Lq, Lk), bool), k=Lk - Lq), 0.0, -np.inf)
    for rho_d, rho_t in ((1.0, 1.0), (0.5, 0.5)):
        want = oracle.attn(Q, K, V, True, rho_d, rho_t, want_p=True)
        got = oracle.attn(Q, K, V, False, rho_d, rho_t, want_p=True, mask=tri)
        assert np.array_equal(got[0], want[0]) and np.array_equal(got[3], want[3]) and np.array_equal(got[1], want[1])
        both = oracle.attn(Q, K, V, True, rho_d, rho_t, mask=tri)                      # the two masks compose
        assert np.array_equal(both[0], want[0])
    # (ii) a float mask against the library, unrounded P, no reduction
    rng = np.random.default_rng(5)
    M4 = rng.normal(0.0, 2.0, (B, Hq, Lq, Lk))
    M4[rng.random(M4.shape) < 0.2] = -np.inf
    M4[..., 0] = 0.5                                                                   # every row keeps a key
    for M in (M4, M4[0, 0], M4[:, :1], M4[:1]):                                        # full, [Lq,Lk], per batch, per head
        O, _, _, _ = oracle.attn(Q, K, V, False, 1.0, 1.0, round_p=False, mask=M)
        Mt = torch.from_numpy(np.broadcast_to(M, (B, Hq, Lq, Lk)).copy())
        Kr, Vr = K.double().repeat_interleave(Hq // Hkv, 1), V.double().repeat_interleave(Hq // Hkv, 1)
        want = torch.nn.functional.scaled_dot_product_attention(Q.double(), Kr, Vr, attn_mask=Mt).numpy()
        assert np.allclose(O, want, rtol=1e-11, atol=1e-12)
    # (iii) one hidden key of one head
    M = np.zeros((B, Hq, Lq, Lk))
    M[1, 2, :, 5] = -np.inf
    base = oracle.attn(Q, K, V, False, 0.5, 1.0, want_p=True)
    got = oracle.attn(Q, K, V, False, 0.5, 1.0, want_p=True, mask=M)
    assert np.all(got[3][1, 2][:, 5] == 0.0) and np.all(base[3][1, 2][:, 5] > 0.0)
    keep = np.ones((B, Hq), bool)
    keep[1, 2] = False
    assert np.array_equal(got[3][keep], base[3][keep]) and not np.array_equal(got[0][1, 2], base[0][1, 2])
    # (iv) rows with every key hidden
    M = np.zeros((Lq, Lk))
    M[3] = -np.inf
    O, _, _, P = oracle.attn(Q, K, V, False, 1.0, 1.0, want_p=True, mask=M)
    assert np.all(O[:, :, 3] == 0.0) and np.all(P[:, :, 3] == 0.0) and np.isfinite(O).all()
    # (v) hidden keys have zero score and are never kept while visible ones remain
    M = np.zeros((Lq, Lk))
    M[:, [1, 4, 7]] = -np.inf
    _, _, It, P = oracle.attn(Q, K, V, False, 1.0, 0.5, want_p=True, mask=M)
    assert not np.isin(It, [1, 4, 7]).any() and np.all(P[..., [1, 4, 7]] == 0.0)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_on_sampled_query_rows(oracle, causal):
    """Steps 2-4 of Sec. 3.3 and the final product are row by row: evaluating a subset of the query rows gives
    exactly those rows of the full result (the feature set still comes from every row of Q)."""
    B, Hq, Hkv, Lq, Lk, Dh = 1, 4, 2, 21, 30, 16
    Q, K, V = synth.attention_qkv(B, Hq, Hkv, Lq, Lk, Dh, seed=25, n_outlier=2)
    rows = [0, 3, 20, 7]
    O, If, _, P = oracle.attn(Q, K, V, causal, 0.5, 1.0, round_p=True, want_p=True)
    Or, Ifr, _, Pr = oracle.attn(Q, K, V, causal, 0.5, 1.0, round_p=True, want_p=True, rows=rows)
    assert Or.shape == (B, Hq, 4, Dh) and Pr.shape == (B, Hq, 4, Lk)
    assert np.array_equal(Ifr, If) and np.array_equal(Or, O[:, :, rows]) and np.array_equal(Pr, P[:, :, rows])
    # with token reduction the set must be handed in (scores need every row); then rows are again independent
    O5, _, It, _ = oracle.attn(Q, K, V, causal, 0.5, 0.4, round_p=True)
    O5r, _, Itr, _ = oracle.attn(Q, K, V, causal, 0.5, 0.4, round_p=True, idx_tok=It, rows=rows)
    assert np.array_equal(Itr, It) and np.array_equal(O5r, O5[:, :, rows])
    with pytest.raises(AssertionError):
        oracle.attn(Q, K, V, causal, 0.5, 0.4, rows=rows)


# --------------------------------------------------------------------------------------------
# 8-bit operands (appendix "Compatibility with quantization"): the e4m3 rounding, the per-row step, the product
# --------------------------------------------------------------------------------------------
def test_e4m3_rounding_against_the_library_and_the_definition(oracle):
    grid = oracle.e4m3_grid()
    assert len(grid) == 127 and grid[0] == 0.0 and grid[1] == 2.0 ** -9 and grid[-1] == 448.0
    assert np.all(np.diff(grid) > 0)
    # every value of the format is a fixed point, in both signs
    assert np.array_equal(oracle.round_e4m3(grid), grid) and np.array_equal(oracle.round_e4m3(-grid), -grid)
    # the library's conversion (round to nearest even) on a dense sweep inside the range
    g = torch.Generator().manual_seed(5)
    x = torch.cat([torch.randn(200000, generator=g) * 100, torch.randn(50000, generator=g) * 0.01, torch.linspace(-448, 448, 100001)])
    x = x[x.abs() <= 448].float()
    want = x.to(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_e4m3(x.numpy()), want)
    # hand-made ties: half way between neighbours goes to the even mantissa code
    assert oracle.round_e4m3([1.0625])[0] == 1.0          # 1.0 (code ..000) | 1.125 (..001)
    assert oracle.round_e4m3([1.1875])[0] == 1.25         # 1.125 (..001) | 1.25 (..010)
    assert oracle.round_e4m3([2.0 ** -10])[0] == 0.0      # 0 | smallest subnormal 2^-9: tie to the even code 0
    assert oracle.round_e4m3([3 * 2.0 ** -10])[0] == 2.0 ** -8
    # saturation instead of overflow
    assert np.array_equal(oracle.round_e4m3([449.0, 1e9, -1e9]), [448.0, 448.0, -448.0])


def test_row_quantisation_and_8_bit_product(oracle):
    # steps: the row maximum maps onto 448 exactly; an all-zero row has step 1 and codes 0
    A = np.array([[448.0, -224.0, 1.0, 0.0], [0.0, 0.0, 0.0, 0.0], [3.0, -7.0, 0.5, 0.25]], dtype=np.float32)
    q, s = oracle.quantize_rows_e4m3(A)
    assert s[0] == 1.0 and np.array_equal(q[0], [448.0, -224.0, 1.0, 0.0])
    assert s[1] == 1.0 and not q[1].any()
    assert s[2] == np.float32(7.0) / np.float32(448.0) and q[2, 1] == -448.0 and q[2, 0] == 192.0 and q[2, 2] == 32.0
    # operands whose codes are exact: entries 0, +-1, +-2, +-4, +-8 with row maximum 8 (step 8 / 448, codes a * 56 are all
    # values of the format), so the quantised product equals the plain one up to the fp32 rounding of the step
    rng = np.random.default_rng(0)
    M, K, N = 5, 24, 7
    Aint = (rng.choice([0.0, 1.0, 2.0, 4.0, 8.0], size=(M, K)) * rng.choice([-1.0, 1.0], size=(M, K))).astype(np.float32)
    Aint[:, 0] = 8.0
    Bq = rng.choice(oracle.e4m3_grid()[:40], size=(N, K)) * rng.choice([-1.0, 1.0], size=(N, K))
    idx = np.array([0, 5, 2, 23, 11, 7], dtype=np.int32)
    Y, s = oracle.reduced_gemm_q8(Aint, Bq, 0.5, idx)
    assert np.all(s == np.float32(8.0) / np.float32(448.0))
    want = (Aint[:, idx].astype(np.float64) @ Bq[:, idx].T) * 0.5
    assert np.allclose(Y, want, rtol=1e-7, atol=0)               # (the fp32 step 8/448 is not a power of two: 6e-8 relative)
    # against the library end to end: torch's own conversion of A / step, dequantised, matmul in fp64
    A2 = synth.heavy_tailed_activations(33, 64, seed=3)
    idx2 = np.sort(rng.choice(64, 20, replace=False)).astype(np.int32)
    Bq2 = (torch.randn(9, 64, generator=torch.Generator().manual_seed(1)) * 0.3).to(torch.float8_e4m3fn)
    Y2, s2 = oracle.reduced_gemm_q8(A2, Bq2.to(torch.float64).numpy(), 0.02, idx2)
    Asel = A2.float()[:, idx2.tolist()]
    st = Asel.abs().amax(dim=1) / 448.0
    qt = (Asel / st[:, None]).to(torch.float8_e4m3fn).to(torch.float64)
    want2 = (qt * st.double()[:, None]) @ (Bq2.to(torch.float64)[:, idx2.tolist()].T * float(np.float32(0.02)))
    assert np.array_equal(s2, st.numpy()) and np.allclose(Y2, want2.numpy(), rtol=1e-12, atol=1e-300)
