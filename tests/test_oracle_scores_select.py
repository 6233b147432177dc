"""Pins for the oracle's importance scores (Eq. 3-7) and keep set (Eq. 8)."""
import os

import numpy as np

from oracle import xsv_oracle as orc


def _kv(path):
    d = {}
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split(";")
            d[k.strip()] = np.array([float(x) for x in v.split()])
    return d


def test_scores_hand_worked(golden_dir):
    g = _kv(os.path.join(golden_dir, "scores_worked.txt"))
    Q = np.stack([g["Q0"].reshape(5, 2), g["Q1"].reshape(5, 2)])
    K = np.stack([g["K0"].reshape(2, 2), g["K1"].reshape(2, 2)])
    S = orc.importance_scores(Q, K, n_special=1, g=2)
    assert np.allclose(S, g["S"], rtol=0, atol=1e-15)


def test_scores_constant_inputs_closed_form():
    # constant q and k everywhere: every pooled row is q, every K_bar row is k, S = d*q*k
    H, F, d, Tp = 4, 37, 16, 9
    Q = np.full((H, F, d), 0.75)
    K = np.full((H, Tp, d), -1.5)
    S = orc.importance_scores(Q, K, n_special=5, g=16)
    assert np.allclose(S, d * 0.75 * -1.5, rtol=1e-14)


def test_scores_pooling_structure():
    # Special rows count once each, patch rows 1/(group size) each: a query that is
    # non-zero only in one special row / one patch row gives a score that shows the weight.
    H, d, n_sp, g = 2, 4, 2, 4
    F = n_sp + 2 * g + 3                      # short last group of 3
    n_pooled = n_sp + 3
    K = np.zeros((H, 1, d)); K[:, 0, 1] = 2.0   # K_bar = (0,2,0,0)
    for row, w in [(0, 1.0), (n_sp + 1, 1.0 / g), (F - 1, 1.0 / 3)]:
        Q = np.zeros((H, F, d)); Q[0, row, 1] = 1.0
        S = orc.importance_scores(Q, K, n_sp, g)
        assert np.isclose(S[0], w * 2.0 / H / n_pooled, rtol=1e-14)


def test_scores_linearity_identity_and_head_symmetry():
    rng = np.random.default_rng(5)
    H, F, d, Tp = 16, 261, 64, 300
    Q = rng.standard_normal((H, F, d)); K = rng.standard_normal((H, Tp, d)) * 3
    S = orc.importance_scores(Q, K, 5, 16)
    S2 = orc.importance_scores_collapsed(Q, K, 5, 16)
    assert np.max(np.abs(S - S2)) <= 1e-12 * np.max(np.abs(S))
    # S has no head axis: permuting heads of Q and, independently, of K changes nothing
    assert np.allclose(S, orc.importance_scores(Q[rng.permutation(H)], K[rng.permutation(H)], 5, 16),
                       rtol=1e-11, atol=1e-12)
    # independent evaluation with einsum over the un-averaged tensors
    Qp = orc.pooled_query(Q, 5, 16)
    S3 = np.einsum("hic,gjc->j", Qp, K) / (H * H * Qp.shape[1])
    assert np.max(np.abs(S - S3)) <= 1e-12 * np.max(np.abs(S))
    assert Qp.shape[1] == 5 + 16              # 256 patches / 16


def test_select_hand_worked(golden_dir):
    for line in open(os.path.join(golden_dir, "select_worked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tf, tc, lmax, s, kept = [f.strip() for f in line.split(";")]
        S = np.array([float(v) for v in s.split()])
        T = int(tf) + S.shape[0] + int(tc)
        got = orc.keep_positions(S, int(tf), int(tc), T, int(lmax))
        assert got.tolist() == [int(v) for v in kept.split()]


def test_select_against_pairwise_definition():
    # token i is selected iff fewer than k tokens beat it, where j beats i when
    # S[j] > S[i], or S[j] == S[i] and j < i.
    rng = np.random.default_rng(11)
    for trial in range(300):
        n = int(rng.integers(1, 24))
        S = rng.integers(-3, 4, n).astype(np.float64) if trial % 2 else rng.standard_normal(n)
        for k in {0, 1, n // 2, n - 1, n}:
            got = set(orc.select_middle(S, k).tolist())
            exp = set()
            for i in range(n):
                beaten = sum(1 for j in range(n) if S[j] > S[i] or (S[j] == S[i] and j < i))
                if beaten < k:
                    exp.add(i)
            assert got == exp and len(got) == min(k, n)
