"""The allocation-free entry point (collected last on purpose).

eora_linear_forward_noalloc serves callers that cannot call cudaMalloc -- a plug-in running inside a
framework that owns all device memory, or a loop that must not allocate -- by reading the weights from
the caller's buffers and keeping its scratch in a fixed array inside the library.  Here it is called
through the C ABI twice in a row (the shared array keeps the first call's contents) and compared with the
handle-based forward on the same inputs, within the tolerance the other parity tests use.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_oracle as orc
import eora_inputs as gen
import paper_2410_21271_b200 as eora
from helpers import REL_FRO_TOL, MAX_ABS_TOL


def _buffers(wf, af, bf, device="cuda:0"):
    import torch
    def dev(a):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint32:
            a = a.view(np.int32)
        return torch.from_numpy(a).to(device)
    keep = [dev(wf["codes"]), dev(wf["scales"]), dev(wf["zeros"]), dev(af["data"]), dev(bf["data"])]
    w = eora.eora_linear_weights()
    w.w_codes, w.w_scales, w.w_zeros, w.a, w.b = [t.data_ptr() for t in keep]
    return w, keep


def _cfg(K, N, r, bits):
    c = eora.eora_linear_config()
    c.d_in, c.d_out, c.rank = K, N, r
    c.w_format, c.w_bits, c.w_group = eora.EORA_W_QUANT, bits, 128
    c.ab_format, c.ab_group, c.x_dtype, c.y_dtype, c.max_m, c.kernel_policy = eora.EORA_AB_F16, 128, 0, 0, 64, 0
    return c


def test_noalloc_matches_handle_forward_twice_in_a_row():
    import torch
    cases = [(4, 512, 96, 64, 5, 71), (3, 384, 160, 128, 9, 72)]     # second call: other shape, larger t
    for bits, K, N, r, M, seed in cases:
        wf = gen.make_backbone_quant(seed, K, N, bits, 128)
        af, bf = gen.make_ab_f16(seed, K, N, r)
        x = torch.from_numpy(gen.make_x(seed + 1, M, K)).to("cuda:0")
        L = eora.Layer(wf, af, bf, max_m=M)
        y_ref = L.forward(x).float().cpu().numpy().astype(np.float64)
        w, keep = _buffers(wf, af, bf)
        y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda:0")
        eora.eora_linear_forward_noalloc(_cfg(K, N, r, bits), w, x, M, y)
        torch.cuda.synchronize()
        got = y.float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        d = got - y_ref
        assert np.linalg.norm(d) / np.linalg.norm(y_ref) <= REL_FRO_TOL
        assert np.abs(d).max() <= MAX_ABS_TOL * np.abs(y_ref).max()
        # and against the float64 oracle (Eq. 4 written out), like every other entry point
        y_orc = orc.forward(x.cpu().numpy(), "f16", wf, af, bf)
        rel, mabs = orc.parity_errors(got, y_orc)
        assert rel <= REL_FRO_TOL and mabs <= MAX_ABS_TOL, (rel, mabs)
        L.close()
        del keep


def test_noalloc_rejects_sizes_beyond_the_fixed_scratch():
    import torch
    K, N, r = 256, 64, 512
    M = eora.EORA_NOALLOC_MAX_T_ELEMS // r + 1
    wf = gen.make_backbone_quant(73, K, N, 4, 128)
    af, bf = gen.make_ab_f16(73, K, N, r)
    w, keep = _buffers(wf, af, bf)
    x = torch.zeros((M, K), dtype=torch.float16, device="cuda:0")
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda:0")
    st = eora.eora_linear_forward_noalloc(_cfg(K, N, r, 4), w, x, M, y, check=False)
    assert st == eora.EORA_ERR_M_TOO_LARGE
    assert "max_m" in eora.eora_status_string(st) or "exceeds" in eora.eora_status_string(st)
    torch.cuda.synchronize()
    del keep
