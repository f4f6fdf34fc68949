"""GPU parity of the offline solve (Algorithm 1 steps 1-6, include/eora_solve.h) against the float64 oracle.

What is unique is compared tightly: the remaining layer-wise loss (Theorem 1: the optimum is the tail energy of the
projected error), the top singular values, and -- where the spectrum has a gap at r -- the product B'A and the
sign-aligned factors.  Where neighbouring singular values are close, individual vectors near the cut are not unique to
working precision; there the product is checked through the loss and through the properties every valid answer has
(rank r, B' = U'S' with orthonormal U', A = S'^{-1} U'^T dW)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_solve_oracle as sol
import eora_inputs as gen
import paper_2410_21271_b200 as eora

LOSS_RTOL = 1e-3          # remaining loss within 0.1 % of the optimum (fp32 contractions, finite iteration)
SIGMA_RTOL = 2e-3


def run_solve(w, w_hat, x, r, **kw):
    import torch
    tw, th, tx = (torch.from_numpy(np.ascontiguousarray(v)).cuda() for v in (w, w_hat, x))
    b, a, s = eora.solve(tw, th, tx, r, **kw)
    loss_dev = eora.solve_loss(tw, th, tx, b, a)
    torch.cuda.synchronize()
    return b.cpu().numpy().astype(np.float64), a.cpu().numpy().astype(np.float64), s.cpu().numpy().astype(np.float64), loss_dev


@pytest.mark.parametrize("d,k,n,r", [(96, 64, 200, 8), (200, 160, 120, 16), (130, 70, 33, 5), (64, 300, 500, 12), (256, 256, 512, 64),
                                     (256, 192, 300, 120), (320, 256, 400, 128), (264, 192, 300, 128)])   # iterates 152 and 160 wide: the 160-column product; 264 rows: the padded one
def test_solve_matches_oracle_loss_and_spectrum(d, k, n, r):
    w, w_hat, x = gen.make_solve_case(11, d, k, n)
    ref = sol.solve(w, w_hat, x, r)
    b, a, s, loss_dev = run_solve(w, w_hat, x, r)
    opt = sol.layer_loss(ref["dW"], ref["B"], ref["A"], x)
    got = sol.layer_loss(ref["dW"], b, a, x)
    assert got >= opt * (1 - 1e-6)                       # nothing beats the optimum (Eckart-Young)
    assert got <= opt * (1 + LOSS_RTOL), (got, opt)
    assert np.isclose(loss_dev, got, rtol=1e-4)          # the library's own loss evaluation
    assert np.allclose(s, ref["sigma"], rtol=SIGMA_RTOL), (s[:4], ref["sigma"][:4])
    assert np.all(np.diff(s) <= 1e-6 * s[0])             # descending
    # structure every valid answer has: B' = U'S' with orthonormal U', A = S'^{-1} U'^T dW
    u = b / s[None, :]
    assert np.allclose(u.T @ u, np.eye(r), atol=5e-4)
    assert np.allclose(a, (u.T @ ref["dW"]) / s[:, None], rtol=0, atol=2e-3 * np.abs(a).max())


@pytest.mark.parametrize("d,k,n,r", [(160, 128, 256, 8), (96, 200, 150, 12)])
def test_solve_gapped_spectrum_elementwise(d, k, n, r):
    """The error is rank r plus noise a hundred times smaller: the top-r subspace is well separated, so the product and
    the factors themselves are comparable (each pair up to its sign)."""
    w, w_hat, x = gen.make_solve_case(12, d, k, n, kind="gap", rank_signal=r)
    ref = sol.solve(w, w_hat, x, r)
    b, a, s, _ = run_solve(w, w_hat, x, r)
    ba, ba_ref = b @ a, ref["B"] @ ref["A"]
    assert np.linalg.norm(ba - ba_ref) <= 2e-3 * np.linalg.norm(ba_ref)
    assert np.allclose(s, ref["sigma"], rtol=1e-3)
    for i in range(r):
        sgn = np.sign(np.dot(b[:, i], ref["B"][:, i]))
        assert np.linalg.norm(b[:, i] - sgn * ref["B"][:, i]) <= 2e-2 * np.linalg.norm(ref["B"][:, i]), i
        assert np.linalg.norm(a[i] - sgn * ref["A"][i]) <= 2e-2 * np.linalg.norm(ref["A"][i]), i


def test_solve_compensates_the_layer():
    """Steps 1-7 end to end: the compensated layer W^ X + B'A X is closer to W X than the compressed one and than the
    plain-SVD compensation of the same rank, by the amounts the oracle computes."""
    d, k, n, r = 192, 256, 384, 32
    w, w_hat, x = gen.make_solve_case(13, d, k, n)
    ref = sol.solve(w, w_hat, x, r)
    b, a, s, _ = run_solve(w, w_hat, x, r)
    none = np.linalg.norm(ref["dW"] @ x.astype(np.float64))
    bs, as_ = sol.plain_svd(ref["dW"], r)
    plain = sol.layer_loss(ref["dW"], bs, as_, x)
    got = sol.layer_loss(ref["dW"], b, a, x)
    assert got < plain < none
    # Pythagoras for an orthogonal projection: what is kept plus what is left is the whole error
    assert np.isclose(got ** 2 + np.sum(s ** 2), none ** 2, rtol=1e-4)


def test_solve_iterations_and_argument_errors():
    import torch
    d, k, n, r = 128, 96, 160, 8
    w, w_hat, x = gen.make_solve_case(14, d, k, n)
    ref = sol.solve(w, w_hat, x, r)
    opt = sol.layer_loss(ref["dW"], ref["B"], ref["A"], x)
    few = run_solve(w, w_hat, x, r, iters=1, oversample=4)
    many = run_solve(w, w_hat, x, r, iters=40, oversample=32)
    l_few, l_many = sol.layer_loss(ref["dW"], few[0], few[1], x), sol.layer_loss(ref["dW"], many[0], many[1], x)
    assert opt * (1 - 1e-6) <= l_many <= l_few and l_many <= opt * (1 + 2e-4)
    cfg = eora.eora_solve_config(d, k, n, r, 0, 0)
    assert eora.eora_solve_workspace_bytes(cfg) > 4 * (d * k + k * k + d * d)
    assert eora.eora_solve_workspace_bytes(eora.eora_solve_config(d, k, n, 0, 0, 0)) == 0
    assert eora.eora_solve_workspace_bytes(eora.eora_solve_config(d, k, n, 600, 0, 0)) == 0
    tw = torch.from_numpy(w).cuda()
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    out = torch.empty((d, r), device="cuda"); oa = torch.empty((r, k), device="cuda"); os_ = torch.empty(r, device="cuda")
    assert eora.eora_solve(cfg, tw, tw, torch.from_numpy(x).cuda(), out, oa, os_, ws, check=False) == eora.EORA_ERR_BAD_SHAPE
    assert eora.lib().eora_solve(None, None, None, None, None, None, None, None, 0, None) == eora.EORA_ERR_NULL_ARG


def test_solve_large_against_oracle():
    """2048 x 2048, 1024 calibration columns (fewer than channels: singular Gram matrix), rank 128."""
    d, k, n, r = 2048, 2048, 1024, 128
    w, w_hat, x = gen.make_solve_case(15, d, k, n, bits=3)
    ref = sol.solve(w, w_hat, x, r)
    b, a, s, loss_dev = run_solve(w, w_hat, x, r)
    opt = sol.layer_loss(ref["dW"], ref["B"], ref["A"], x)
    got = sol.layer_loss(ref["dW"], b, a, x)
    assert opt * (1 - 1e-6) <= got <= opt * (1 + LOSS_RTOL), (got, opt)
    assert np.isclose(loss_dev, got, rtol=1e-3)
    assert np.allclose(s, ref["sigma"], rtol=SIGMA_RTOL)


def test_solves_side_by_side_on_three_streams():
    """Three different layers solved at the same time, each on its own stream with its own workspace: every one meets the
    oracle's optimum, so the solves share no state."""
    import torch
    cases = [(200, 160, 120, 16, 21), (256, 256, 512, 64, 22), (130, 300, 260, 24, 23)]
    streams = [torch.cuda.Stream() for _ in cases]
    ins, outs = [], []
    for (d, k, n, r, seed) in cases:
        w, w_hat, x = gen.make_solve_case(seed, d, k, n)
        ins.append((w, w_hat, x, tuple(torch.from_numpy(np.ascontiguousarray(v)).cuda() for v in (w, w_hat, x))))
    torch.cuda.synchronize()
    for rep in range(2):                                  # the second round runs with every stream already busy
        outs = []
        for st, (d, k, n, r, _), (_, _, _, dev) in zip(streams, cases, ins):
            with torch.cuda.stream(st):
                outs.append(eora.solve(dev[0], dev[1], dev[2], r, stream=st))
    torch.cuda.synchronize()
    for (d, k, n, r, _), (w, w_hat, x, _), (b, a, s) in zip(cases, ins, outs):
        ref = sol.solve(w, w_hat, x, r)
        opt = sol.layer_loss(ref["dW"], ref["B"], ref["A"], x)
        got = sol.layer_loss(ref["dW"], b.cpu().numpy(), a.cpu().numpy(), x)
        assert opt * (1 - 1e-6) <= got <= opt * (1 + LOSS_RTOL), (d, k, n, r, got, opt)
        assert np.allclose(s.cpu().numpy(), ref["sigma"], rtol=SIGMA_RTOL)
