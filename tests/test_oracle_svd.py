"""Pins of the checker's SVD, rank rule and split (Eq. 3; AB-decomposition bullet of
Section "Methodology") against closed forms, LAPACK, Eckart-Young, exact recovery and
planted spectra.  CPU only."""
import os

import numpy as np
import pytest

from oracle import ab_oracle as orc
from paper_2405_01067_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "closed_form_svd.txt")


def _golden():
    out = []
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        shp, ent, sv = [p.strip() for p in line.split("|")]
        m, n = map(int, shp.split())
        out.append((np.array(list(map(float, ent.split()))).reshape(m, n),
                    np.array(list(map(float, sv.split())))))
    return out


@pytest.mark.parametrize("W,sv", _golden())
def test_closed_form_singular_values(W, sv):
    U, s, Vt, _ = orc.jacobi_svd(W)
    assert np.allclose(s, sv, rtol=1e-13, atol=1e-13)
    assert np.allclose((U * s) @ Vt, W, atol=1e-13)


@pytest.mark.parametrize("m,n", [(40, 24), (24, 40), (33, 33), (17, 1), (1, 9), (64, 48)])
def test_against_lapack(m, n):
    rng = np.random.default_rng(m * 131 + n)
    W = rng.standard_normal((m, n))
    U, s, Vt, _ = orc.jacobi_svd(W)
    s_ref = np.linalg.svd(W, compute_uv=False)
    assert np.allclose(s, s_ref, rtol=1e-12, atol=1e-13)
    k = len(s)
    assert np.allclose(U.T @ U, np.eye(k), atol=1e-12)
    assert np.allclose(Vt @ Vt.T, np.eye(k), atol=1e-12)
    assert np.allclose((U * s) @ Vt, W, atol=1e-12)
    assert np.all(np.diff(s) <= 0)
    # leading-r reconstruction agrees with LAPACK's (sign-invariant comparison)
    U2, s2, Vt2 = np.linalg.svd(W, full_matrices=False)
    r = max(1, k // 3)
    assert np.allclose((U[:, :r] * s[:r]) @ Vt[:r], (U2[:, :r] * s2[:r]) @ Vt2[:r], atol=1e-10)


def test_eckart_young_and_balance():
    rng = np.random.default_rng(5)
    W = rng.standard_normal((48, 30))
    for r in (1, 7, 30):
        A, B, s, rk = orc.svd_split(W, r, 0.0)
        assert rk == r and A.shape == (48, r) and B.shape == (r, 30)
        err = np.linalg.norm(W - A @ B)
        assert np.isclose(err ** 2, np.sum(s[r:] ** 2), rtol=1e-10, atol=1e-20)
        if r < 30:
            assert np.isclose(np.linalg.norm(W - A @ B, 2), s[r], rtol=1e-10)
        # A^T A = B B^T = diag(sigma_r)
        assert np.allclose(A.T @ A, np.diag(s[:r]), atol=1e-12)
        assert np.allclose(B @ B.T, np.diag(s[:r]), atol=1e-12)


def test_no_rank_r_matrix_is_closer():
    rng = np.random.default_rng(6)
    W = rng.standard_normal((20, 14))
    A, B, _, _ = orc.svd_split(W, 4, 0.0)
    best = np.linalg.norm(W - A @ B)
    for _ in range(50):
        P = rng.standard_normal((20, 4))
        C = np.linalg.lstsq(P, W, rcond=None)[0]
        assert np.linalg.norm(W - P @ C) >= best - 1e-12


@pytest.mark.parametrize("m,n,r", [(50, 30, 6), (30, 50, 6), (64, 64, 16)])
def test_exact_recovery_and_fixed_point(m, n, r):
    rng = np.random.default_rng(m + n + r)
    W = rng.standard_normal((m, r)) @ rng.standard_normal((r, n))
    A, B, s, rk = orc.svd_split(W, r, 0.0)
    assert rk == r
    assert np.allclose(A @ B, W, atol=1e-11)
    assert np.all(s[r:] < 1e-12 * s[0])
    # recombine -> split -> recombine is a fixed point
    W2 = orc.recombine(A, B)
    A2, B2, s2, _ = orc.svd_split(W2, r, 0.0)
    assert np.allclose(orc.recombine(A2, B2), W2, atol=1e-11)
    assert np.allclose(s2[:r], s[:r], rtol=1e-11)
    # asking for more rank than W has must not inject anything
    A3, B3, _, rk3 = orc.svd_split(W, r + 5, 0.0)
    assert rk3 == r + 5 and np.allclose(A3 @ B3, W, atol=1e-11)


def test_planted_spectrum_and_rank_rule():
    rng = np.random.default_rng(8)
    sig = np.exp(-np.arange(192) / 64.0)
    W = synth.planted_matrix(rng, 200, 192, sig).astype(np.float64)   # float32-rounded entries
    A, B, s, rk = orc.svd_split(W, 192, 0.1)
    assert np.allclose(s[:150], sig[:150], rtol=2e-6)
    # exp(-i/64) >= 0.1  <=>  i <= 147.37: 148 values are kept
    assert rk == 148
    assert A.shape == (200, 148) and B.shape == (148, 192)


def test_rank_rule_cases():
    s = np.array([4.0, 2.0, 1.0, 0.4, 0.399999])
    assert orc.rank_rule(s, 0.0, 5) == 5
    assert orc.rank_rule(s, 0.0, 3) == 3           # capped at r_max
    assert orc.rank_rule(s, 0.1, 5) == 4           # 0.4 == 0.1 * 4 is kept (only smaller values go)
    assert orc.rank_rule(s, 0.25, 5) == 3
    assert orc.rank_rule(s, 0.5, 5) == 2
    assert orc.rank_rule(s, 1.0, 5) == 1
    assert orc.rank_rule(s, 7.0, 5) == 1           # never below one
    assert orc.rank_rule(np.array([]), 0.1, 3) == 0


def test_transposition_does_not_change_the_result():
    rng = np.random.default_rng(9)
    W = rng.standard_normal((12, 31))
    A, B, s, _ = orc.svd_split(W, 5, 0.0)
    At, Bt, st, _ = orc.svd_split(W.T, 5, 0.0)
    assert np.allclose(s, st, rtol=1e-12)
    assert np.allclose(A @ B, (At @ Bt).T, atol=1e-11)


def test_rank_deficient_input_converges():
    rng = np.random.default_rng(10)
    W = rng.standard_normal((40, 8)) @ rng.standard_normal((8, 32))
    U, s, Vt, sweeps = orc.jacobi_svd(W)
    assert sweeps < 30
    assert np.allclose(s[:8], np.linalg.svd(W, compute_uv=False)[:8], rtol=1e-12)
    assert np.all(s[8:] < 1e-12 * s[0])
    assert np.allclose(np.zeros((3, 4)), (lambda r: (r[0] * r[1]) @ r[2])(orc.jacobi_svd(np.zeros((3, 4)))[:3]))


def test_group_sync_chain():
    d = synth.vit_sync_matrix(3, 0, 96, 64, K=4, scale=1)
    Ak = synth.group_copies(d["A"], d["noise_A"])
    Bk = synth.group_copies(d["B"], d["noise_B"])
    out = orc.group_sync(Ak, Bk, d["r"], 0.1)
    W = np.mean(Ak.astype(np.float64), 0) @ np.mean(Bk.astype(np.float64), 0)
    assert np.allclose(out["W"], W, atol=1e-13)
    s_ref = np.linalg.svd(W, compute_uv=False)
    assert out["r"] == max(1, min(d["r"], int(np.sum(s_ref >= 0.1 * s_ref[0]))))
    U, s, Vt = np.linalg.svd(W)
    r = out["r"]
    assert np.allclose(out["A"] @ out["B"], (U[:, :r] * s[:r]) @ Vt[:r], atol=1e-10)
