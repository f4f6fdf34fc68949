"""GPU parity of the backbone that is 2:4 sparse AND 4-bit quantised (the paper's appendix on sparsity &
quantisation error compensation): storage bit for bit, then the forward through every kernel family against the
float64 oracle.  Tolerances as in the other parity tests."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_oracle as orc
import eora_inputs as gen
import paper_2410_21271_b200 as eora
from helpers import make_case, run_layer, check_parity, expected_family

SHAPES = gen.LLAMA3_8B_SHAPES


@pytest.mark.parametrize("K,N,group", [(256, 64, 128), (512, 96, 64), (384, 32, 192), (512, 160, 512)])
def test_storage_bit_exact(K, N, group):
    """The library's re-tiled copy, element by element: (q - z) * s at the kept positions, 0 elsewhere."""
    wf, _, _ = make_case(90, K, N, 0, w="sq4", group=group)
    L = eora.Layer(wf, None, None, max_m=1)
    W = orc.dequant_matrix(wf)
    assert np.array_equal(L.dump(1).cpu().numpy().astype(np.float64), W.astype(np.float32).astype(np.float64))
    with pytest.raises(eora.EoraError):                 # there is no dense code matrix to dump
        L.dump(0)
    L.close()


def test_one_hot_rows_through_the_fast_path():
    """X = e_k, rank 0, fp32 output: the decode kernel's own unpack + expansion, bit for bit (the product of a
    4-bit difference and an fp16 scale is exact in fp32)."""
    K, N = 512, 96
    wf, _, _ = make_case(91, K, N, 0, w="sq4")
    ks = [0, 1, 2, 3, 5, 63, 64, 127, 128, 130, 257, 511]
    x = np.zeros((len(ks), K), dtype=np.float16)
    for i, k in enumerate(ks):
        x[i, k] = 1.0
    L = eora.Layer(wf, None, None, max_m=8, y_dtype="f32")        # the decode family: at most eight tokens per call
    assert L.path(8) == eora.EORA_PATH_DECODE
    y = np.concatenate([run_layer(L, x[i:i + 8], "f16") for i in range(0, len(ks), 8)])
    assert np.array_equal(y, orc.dequant_matrix(wf)[ks])
    L.close()


CASES = [
    # ab, K, N, r, M, x dtype, group
    ("f16", 256, 64, 64, 1, "f16", 128),
    ("f16", 512, 96, 128, 3, "bf16", 128),
    ("q4", 512, 160, 128, 8, "f16", 128),
    ("q8", 384, 96, 40, 19, "f16", 128),
    ("q3", 1024, 224, 64, 64, "f16", 128),
    ("f16", 1024, 352, 0, 1, "f16", 128),
    ("f16", 512, 96, 64, 5, "f16", 64),
    ("f16", 768, 96, 64, 2, "f16", 256),
    ("f16", 512, 96, 64, 1, "f16", 512),            # channel-wise
    ("f16", 640, 160, 64, 100, "f16", 128),         # tensor-core family
    ("q4", 1024, 512, 128, 300, "bf16", 128),
    ("f16", 384, 288, 24, 130, "f16", 192),
]


@pytest.mark.parametrize("policy", [eora.EORA_POLICY_GENERIC, eora.EORA_POLICY_AUTO])
@pytest.mark.parametrize("ab,K,N,r,M,xd,group", CASES)
def test_forward_matches_oracle(policy, ab, K, N, r, M, xd, group):
    wf, af, bf = make_case(92, K, N, r, w="sq4", ab=ab, group=group)
    x = gen.make_x(93, M, K, xd)
    L = eora.Layer(wf, af, bf, max_m=M, x_dtype=xd, kernel_policy=policy)
    if policy == eora.EORA_POLICY_AUTO:
        assert L.path(M) == expected_family(M, K)
    y_ref = orc.forward(x, xd, wf, af, bf)
    for rep in range(2):                                # second call: the scratch was restored
        check_parity(run_layer(L, x, xd), y_ref, f"sq4/{ab} K{K} N{N} r{r} M{M} g{group} path{L.path(M)} call {rep}")
    L.close()


@pytest.mark.parametrize("name,M", [("k", 1), ("q", 1), ("down", 8), ("k", 2048)])
def test_fullsize(name, M):
    """LLaMA3-8B layer shapes, rank 128: the decode family element by element, the prefill family on sampled outputs."""
    K, N = SHAPES[name]
    wf, af, bf = make_case(94, K, N, 128, w="sq4")
    x = gen.make_x(95, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    if M <= 64:
        assert L.path(M) == eora.EORA_PATH_DECODE
        rel, _ = check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), f"{name} M{M}")
        assert 5e-5 < rel < 1e-3
    else:
        assert L.path(M) == eora.EORA_PATH_PREFILL
        y = run_layer(L, x, "f16")
        rng = np.random.default_rng(0)
        mi, ni = rng.integers(0, M, 96), rng.integers(0, N, 96)
        mi[:4] = [0, M - 1, 0, M - 1]; ni[:4] = [0, 0, N - 1, N - 1]
        ref = orc.forward_at(x, "f16", wf, af, bf, mi, ni)
        d = y[mi, ni] - ref
        assert np.all(np.isfinite(y))
        assert np.linalg.norm(d) / np.linalg.norm(ref) <= 2e-3 and np.abs(d).max() <= 1e-2 * np.abs(ref).max()
    L.close()


def test_argument_errors():
    wf, af, bf = make_case(96, 256, 64, 64, w="sq4")
    cfg, wts, keep = eora._marshal(wf, af, bf, max_m=1, x_dtype="f16", y_dtype="f16", kernel_policy=eora.EORA_POLICY_AUTO,
                                   device="cuda:0")
    meta = wts.w_meta
    wts.w_meta = None
    assert eora.eora_linear_create_status(cfg, wts) == eora.EORA_ERR_NULL_ARG
    wts.w_meta = meta + 4
    assert eora.eora_linear_create_status(cfg, wts) == eora.EORA_ERR_MISALIGNED
    wts.w_meta = meta
    cfg.w_bits = 3
    assert eora.eora_linear_create_status(cfg, wts) == eora.EORA_ERR_UNSUPPORTED
    cfg.w_bits, cfg.w_group = 4, 96
    assert eora.eora_linear_create_status(cfg, wts) == eora.EORA_ERR_BAD_SHAPE
