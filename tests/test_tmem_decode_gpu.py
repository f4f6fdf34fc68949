"""GPU parity of the tensor-memory decode family (kernel_policy = EORA_POLICY_TMEM_DECODE): the same layer, Eq. 4,
with the weights unpacked to bytes into tensor memory and multiplied by tcgen05.mma (kind::i8) against the activations
as 16-bit block fixed point.  Compared element by element with the float64 oracle on the same seeded inputs."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_oracle as orc
import eora_inputs as gen
import paper_2410_21271_b200 as eora
from helpers import make_case, run_layer, check_parity, x_to_torch

POL = eora.EORA_POLICY_TMEM_DECODE

CASES = [
    # w, K, N, r, M, x_dtype, group
    ("q3", 256, 128, 0, 1, "f16", 128),
    ("q4", 256, 128, 0, 1, "f16", 128),
    ("q3", 512, 256, 128, 1, "f16", 128),
    ("q4", 512, 96, 64, 3, "f16", 128),
    ("q3", 384, 160, 64, 8, "f16", 128),
    ("q3", 1024, 224, 128, 16, "bf16", 128),
    ("q4", 256, 64, 24, 7, "f16", 128),
    ("q4", 1152, 352, 128, 63, "f16", 128),
    ("q3", 768, 96, 64, 2, "f16", 256),
    ("q4", 512, 96, 64, 1, "f16", 512),          # channel-wise
    ("q3", 1024, 224, 128, 33, "f16", 128),
]


@pytest.mark.parametrize("w,K,N,r,M,xd,group", CASES)
def test_forward_matches_oracle(w, K, N, r, M, xd, group):
    wf, af, bf = make_case(41, K, N, r, w=w, group=group)
    x = gen.make_x(42, M, K, xd)
    L = eora.Layer(wf, af, bf, max_m=M, x_dtype=xd, kernel_policy=POL)
    assert L.path(M) == eora.EORA_PATH_DECODE and L.launches(M) == (M + 15) // 16
    y_ref = orc.forward(x, xd, wf, af, bf)
    for rep in range(2):                       # the second call finds the scratch as the first one left it
        check_parity(run_layer(L, x, xd), y_ref, f"tmem decode {w} K{K} N{N} r{r} M{M} rep {rep}")
    L.close()


@pytest.mark.parametrize("w", ["q4", "q3"])
def test_one_hot_rows_read_back_exact_weights(w):
    """X = e_k, rank 0, fp32 output: the power-of-two block scale makes the fixed-point activations exact, so y[n] is the
    dequantised weight itself, bit for bit."""
    K, N = 512, 96
    wf, _, _ = make_case(25, K, N, 0, w=w)
    ks = [0, 1, 10, 21, 63, 64, 127, 128, 300, 511]
    x = np.zeros((len(ks), K), dtype=np.float16)
    for i, k in enumerate(ks):
        x[i, k] = 1.0
    L = eora.Layer(wf, None, None, max_m=len(ks), y_dtype="f32", kernel_policy=POL)
    y = run_layer(L, x, "f16")
    q = orc.unpack_codes(wf["codes"], wf["bits"], K); z = orc.unpack_zeros(wf["zeros"], wf["bits"], N)
    W = orc.deq_fp32(q, z, wf["scales"], 128).astype(np.float64)
    assert np.array_equal(y, W[ks])
    L.close()


def test_extreme_activations():
    """All-zero input, one huge value among tiny ones, a wide dynamic range: the block fixed point (one power-of-two scale
    per token and 128 reduction elements) must stay inside the tolerance."""
    K, N, r = 512, 96, 64
    wf, af, bf = make_case(37, K, N, r, w="q3")
    L = eora.Layer(wf, af, bf, max_m=1, kernel_policy=POL)
    rng = np.random.default_rng(38)
    xs = [np.zeros((1, K), dtype=np.float16)]
    x = (rng.standard_normal((1, K)) * 1e-3).astype(np.float16); x[0, 17] = 3000.0; xs.append(x)
    x = (rng.standard_normal((1, K)) * np.exp(rng.uniform(-6, 3, (1, K)))).astype(np.float16); xs.append(x)
    x = (rng.standard_normal((1, K)) * 200).astype(np.float16); xs.append(x)
    for i, x in enumerate(xs):
        y = run_layer(L, x, "f16")
        ref = orc.forward(x, "f16", wf, af, bf)
        if not ref.any():
            assert not y.any()
        else:
            check_parity(y, ref, f"extreme activations case {i}")
    L.close()


@pytest.mark.parametrize("M", [1, 8])
def test_fullsize_q_shape_and_fused_qkv(M):
    import torch
    K, r = 4096, 128
    parts = [gen.make_backbone_quant(60 + i, K, n, 3, 128) for i, n in enumerate((4096, 1024, 1024))]
    abs_ = [gen.make_ab_f16(60 + i, K, n, r) for i, n in enumerate((4096, 1024, 1024))]
    x = gen.make_x(61, M, K)
    F = eora.FusedLayers([(w, a, b) for w, (a, b) in zip(parts, abs_)], max_m=M, kernel_policy=POL)
    ys = F.forward(x_to_torch(x, "f16"))
    torch.cuda.synchronize()
    assert F.device_status() == 0
    for w, (a, b), y in zip(parts, abs_, ys):
        check_parity(y.float().cpu().numpy().astype(np.float64), orc.forward(x, "f16", w, a, b), f"fused tmem decode M{M}")
    F.close()


def test_formats_it_does_not_serve_fall_back():
    """Quantised adapters, 2:4 backbones and groups that do not fill a 128-element unit are served by the other families."""
    wf, af, bf = make_case(43, 512, 96, 64, w="q4", ab="q4")
    L = eora.Layer(wf, af, bf, max_m=4, kernel_policy=POL)
    x = gen.make_x(44, 4, 512)
    check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), "fallback")
    L.close()
