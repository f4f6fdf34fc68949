"""Shared helpers of the GPU parity tests: build a layer from generator output, run it through
the C ABI, compare with the CPU oracle."""
import numpy as np

from oracle import eora_oracle as orc
import eora_inputs as gen

REL_FRO_TOL = 2e-3     # ||Y - y||_F / ||y||_F   (y: float64 oracle, unrounded)
MAX_ABS_TOL = 1e-2     # max|Y - y| / max|y|


def make_case(seed, K, N, r, *, w="q4", ab="f16", group=128):
    if w in ("q4", "q3"):
        wf = gen.make_backbone_quant(seed, K, N, 4 if w == "q4" else 3, group)
    elif w == "sp24":
        wf = gen.make_sparse24(seed, K, N)
    elif w == "sq4":
        wf = gen.make_sparse24_quant(seed, K, N, 4, group)
    else:
        raise ValueError(w)
    if r == 0:
        af = bf = None
    elif ab == "f16":
        af, bf = gen.make_ab_f16(seed, K, N, r)
    else:
        af, bf = gen.make_ab_quant(seed, K, N, r, ab)
    return wf, af, bf


def x_to_torch(x, x_dtype, device="cuda:0"):
    import torch
    if x_dtype == "f16":
        return torch.from_numpy(x).to(device)
    return torch.from_numpy(x.view(np.int16)).to(device).view(torch.bfloat16)


def run_layer(layer, x, x_dtype):
    import torch
    xt = x_to_torch(x, x_dtype)
    y = layer.forward(xt)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    return y.float().cpu().numpy().astype(np.float64)


def check_parity(y, y_ref, what=""):
    rel, mabs = orc.parity_errors(y, y_ref)
    assert np.all(np.isfinite(y)), what
    assert rel <= REL_FRO_TOL, f"{what}: rel Frobenius {rel:.3e}"
    assert mabs <= MAX_ABS_TOL, f"{what}: max abs {mabs:.3e}"
    return rel, mabs


def expected_family(M, K):
    """The kernel family a plain layer takes under EORA_POLICY_AUTO when both families support it (the rule in
    include/eora_linear.h): decode up to 16 tokens, tensor-core beyond 64, in between whichever is cheaper."""
    import paper_2410_21271_b200 as eora
    if M > 64 or (M > 16 and ((M + 7) // 8) * 30 > K // 64):
        return eora.EORA_PATH_PREFILL
    return eora.EORA_PATH_DECODE
