"""Pins of the offline-solve oracle (Algorithm 1 steps 1-6) against what the paper and the mathematics fix: a
hand-worked instance, Theorem 1 with Eckart-Young (the remaining loss is the tail energy of the projected error),
the identity-Gram special case (reduces to a library SVD), a closed form for diagonal inputs, optimality against
the plain SVD and against perturbations, an independent formulation through the d x d matrix dW G dW^T, and
invariances.  CPU only."""
import os
import numpy as np
import pytest

from oracle import eora_solve_oracle as sol
import eora_inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "solve_hand_example.txt")


def test_hand_worked_two_by_two():
    vals = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        key, *rest = line.split()
        vals[key] = [float(v) for v in rest]
    w = np.eye(2); w_hat = np.zeros((2, 2)); x = np.array([[2.0, 0.0], [0.0, 1.0]])
    out = sol.solve(w, w_hat, x, 1)
    ba = out["B"] @ out["A"]
    assert np.allclose(ba.ravel(), vals["BA"], atol=1e-12)
    assert np.isclose(out["sigma"][0], vals["sigma"][0])
    assert np.isclose(sol.layer_loss(out["dW"], out["B"], out["A"], x), vals["loss"][0])
    b2 = np.array([[0.0], [1.0]]); a2 = np.array([[0.0, 1.0]])          # the other direction a plain SVD may keep
    assert np.isclose(sol.layer_loss(out["dW"], b2, a2, x), vals["loss_if_e2_kept"][0])


@pytest.mark.parametrize("d,k,n,r", [(24, 16, 40, 4), (16, 32, 64, 7), (20, 20, 12, 5)])
def test_loss_is_tail_energy_of_projected_error(d, k, n, r):
    """Theorem 1 + Eckart-Young: || (dW - B'A) X~ ||_F^2 = sum of the squared singular values of dW' beyond r.
    (20, 20, 12): fewer calibration columns than channels, so the Gram matrix is singular and the clamp is active.)"""
    w, w_hat, x = gen.make_solve_case(1, d, k, n)
    out = sol.solve(w, w_hat, x, r)
    loss = sol.layer_loss(out["dW"], out["B"], out["A"], x)
    tail = np.sqrt(np.sum(out["sigma_all"][r:] ** 2))
    assert np.isclose(loss, tail, rtol=1e-6, atol=1e-9 * np.linalg.norm(out["dW"] @ x))
    # and the singular values of dW' are those of dW X~ (same Gram matrix), computed without any of the steps
    s_direct = np.linalg.svd(out["dW"].astype(np.float64) @ x.astype(np.float64), compute_uv=False)
    m = min(len(s_direct), len(out["sigma_all"]))
    assert np.allclose(out["sigma_all"][:m], s_direct[:m], rtol=1e-6, atol=1e-8 * s_direct[0])


def test_identity_gram_reduces_to_library_svd():
    d, k, r = 12, 10, 3
    rng = np.random.default_rng(2)
    w = rng.standard_normal((d, k)); w_hat = np.zeros((d, k))
    qmat, _ = np.linalg.qr(rng.standard_normal((k, k)))
    x = 3.0 * qmat                                   # X~ X~^T = 9 I
    out = sol.solve(w, w_hat, x, r)
    b, a = sol.plain_svd(w, r)
    assert np.allclose(out["B"] @ out["A"], b @ a, atol=1e-10)
    assert np.allclose(out["sigma"], 3.0 * np.linalg.svd(w, compute_uv=False)[:r])


def test_diagonal_closed_form():
    """dW = diag(delta), X~ X~^T = diag(g): the projected error is diag(delta_i sqrt(g_i)), so the r kept directions
    are the r largest |delta_i| sqrt(g_i), each restored exactly, the others not at all."""
    delta = np.array([0.5, -2.0, 1.0, 0.1, 3.0]); g = np.array([100.0, 1.0, 9.0, 400.0, 0.01])
    x = np.diag(np.sqrt(g))
    out = sol.solve(np.diag(delta), np.zeros((5, 5)), x, 2)
    score = np.abs(delta) * np.sqrt(g)               # 5, 2, 3, 2, 0.3 -> indices 0 and 2
    keep = np.argsort(-score)[:2]
    expect = np.zeros((5, 5)); expect[keep, keep] = delta[keep]
    assert sorted(keep.tolist()) == [0, 2]
    assert np.allclose(out["B"] @ out["A"], expect, atol=1e-12)
    assert np.allclose(np.sort(out["sigma"]), np.sort(score[keep]))


@pytest.mark.parametrize("seed", [3, 4])
def test_never_worse_than_plain_svd_and_locally_optimal(seed):
    d, k, n, r = 24, 32, 96, 6
    w, w_hat, x = gen.make_solve_case(seed, d, k, n)
    out = sol.solve(w, w_hat, x, r)
    loss = sol.layer_loss(out["dW"], out["B"], out["A"], x)
    b, a = sol.plain_svd(out["dW"], r)
    assert loss <= sol.layer_loss(out["dW"], b, a, x) * (1 + 1e-12)
    assert loss < 0.97 * sol.layer_loss(out["dW"], b, a, x)            # anisotropic activations: strictly better
    rng = np.random.default_rng(seed)
    for _ in range(20):                                                 # no perturbation of (B', A) lowers the loss
        db = rng.standard_normal(out["B"].shape) * 1e-3 * np.abs(out["B"]).max()
        da = rng.standard_normal(out["A"].shape) * 1e-3 * np.abs(out["A"]).max()
        assert sol.layer_loss(out["dW"], out["B"] + db, out["A"] + da, x) >= loss * (1 - 1e-12)
    # alternating least squares in the weighted norm from a random start reaches the same loss from above
    g = sol.gram(x)
    bb = rng.standard_normal((d, r)); aa = rng.standard_normal((r, k))
    for _ in range(400):
        aa = np.linalg.solve(bb.T @ bb, bb.T @ out["dW"])               # best A for fixed B (G cancels: it is invertible here)
        bb = out["dW"] @ g @ aa.T @ np.linalg.inv(aa @ g @ aa.T)        # best B for fixed A
    als = sol.layer_loss(out["dW"], bb, aa, x)
    assert als >= loss * (1 - 1e-9) and als <= loss * (1 + 1e-3)


def test_full_rank_restores_the_error():
    d, k, n = 6, 9, 30
    w, w_hat, x = gen.make_solve_case(5, d, k, n)
    out = sol.solve(w, w_hat, x, d)
    assert np.allclose(out["B"] @ out["A"], out["dW"], atol=1e-9 * np.abs(out["dW"]).max() + 1e-12)


def test_equals_projection_on_top_eigenvectors_of_dw_g_dwt():
    """Independent route: B'A = U U^T dW with U the top-r eigenvectors of dW (X~ X~^T) dW^T -- no square roots, no
    inverse; and B' = U S', A = S'^{-1} U^T dW up to the sign of each pair."""
    d, k, n, r = 18, 14, 50, 5
    w, w_hat, x = gen.make_solve_case(6, d, k, n)
    out = sol.solve(w, w_hat, x, r)
    m = out["dW"] @ sol.gram(x) @ out["dW"].T
    lam, u = np.linalg.eigh(m)
    u = u[:, ::-1][:, :r]; lam = lam[::-1][:r]
    assert np.allclose(out["sigma"], np.sqrt(lam), rtol=1e-8)
    assert np.allclose(out["B"] @ out["A"], u @ (u.T @ out["dW"]), atol=1e-10 * np.abs(out["dW"]).max() * k)
    for i in range(r):
        sgn = np.sign(np.dot(out["B"][:, i], u[:, i]))
        assert np.allclose(out["B"][:, i], sgn * u[:, i] * np.sqrt(lam[i]), rtol=1e-6, atol=1e-12)
        assert np.allclose(out["A"][i], sgn * (u[:, i] @ out["dW"]) / np.sqrt(lam[i]), rtol=1e-6, atol=1e-12)


def test_invariances_and_floor():
    d, k, n, r = 10, 12, 8, 3                         # n < k: singular Gram matrix
    w, w_hat, x = gen.make_solve_case(7, d, k, n)
    base = sol.solve(w, w_hat, x, r)
    ba = base["B"] @ base["A"]
    perm = np.random.default_rng(8).permutation(n)
    for other in (sol.solve(w, w_hat, 5.0 * x, r), sol.solve(w, w_hat, x[:, perm], r), sol.solve(w, w_hat, x, r, floor=1e-10)):
        # the product is what is unique; compare it where it acts: on the calibration activations and as a matrix
        assert np.allclose((other["B"] @ other["A"]) @ x, ba @ x, atol=1e-8 * np.linalg.norm(ba @ x))
    assert np.allclose(sol.solve(w, w_hat, 5.0 * x, r)["B"] @ sol.solve(w, w_hat, 5.0 * x, r)["A"], ba, atol=1e-6 * np.abs(ba).max())
    a_lib, b_lib = sol.to_library_layout(base["B"], base["A"])
    assert a_lib.shape == (k, r) and b_lib.shape == (r, d)
    xs = np.random.default_rng(9).standard_normal((4, k))
    assert np.allclose((xs @ a_lib) @ b_lib, (ba @ xs.T).T)            # the inference path's  (X A) B  is  (B'A X)^T
