"""GPU parity of the fused-layer entry points (several layers that read the same X behind one handle and one
launch): every output is compared with the CPU oracle's forward of its own layer, and with the plain
per-layer handle.  Tolerances as in the other parity tests."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_oracle as orc
import eora_inputs as gen
import paper_2410_21271_b200 as eora
from helpers import make_case, check_parity, x_to_torch

SHAPES = gen.LLAMA3_8B_SHAPES


def run_fused(F, x, xd):
    import torch
    ys = F.forward(x_to_torch(x, xd))
    torch.cuda.synchronize()
    assert F.device_status() == 0
    return [y.float().cpu().numpy().astype(np.float64) for y in ys]


CASES = [
    # w, ab, K, [N...], r, M, x dtype
    ("q4", "f16", 256, [64, 32], 64, 1, "f16"),
    ("q3", "f16", 512, [96, 32, 64], 128, 3, "f16"),
    ("q4", "q4", 512, [96, 160], 128, 8, "f16"),
    ("q4", "q8", 384, [64, 64, 32, 96], 40, 5, "bf16"),
    ("q3", "f16", 1024, [224, 96], 0, 2, "f16"),
    ("q3", "f16", 640, [160, 352], 256, 19, "f16"),          # three passes of eight tokens
    ("sp24", "f16", 512, [96, 64], 64, 2, "f16"),            # 2:4 backbones
    ("sq4", "q4", 512, [64, 160, 32], 128, 9, "f16"),        # 2:4 with 4-bit kept values
]


@pytest.mark.parametrize("w,ab,K,Ns,r,M,xd", CASES)
def test_fused_matches_oracle_small(w, ab, K, Ns, r, M, xd):
    layers = [make_case(50 + i, K, N, r, w=w, ab=ab) for i, N in enumerate(Ns)]
    x = gen.make_x(51, M, K, xd)
    F = eora.FusedLayers(layers, max_m=M, x_dtype=xd)
    assert F.launches(M) == (M + 7) // 8
    for rep in range(2):                                   # second call: the scratch was restored
        ys = run_fused(F, x, xd)
        for i, (wf, af, bf) in enumerate(layers):
            check_parity(ys[i], orc.forward(x, xd, wf, af, bf), f"layer {i} call {rep}")
    F.close()


@pytest.mark.parametrize("w,ab,K,Ns,r,M,xd", [
    ("q4", "f16", 2048, [256, 128], 128, 17, "f16"),
    ("q3", "q4", 1024, [128, 128, 384], 64, 64, "f16"),
    ("q4", "q8", 2048, [128, 256], 256, 40, "bf16"),
    ("q3", "f16", 1536, [384, 128], 0, 33, "f16"),
])
def test_fused_few_tokens_tensor_core_family(w, ab, K, Ns, r, M, xd):
    """17 to 64 tokens on a fused handle whose layers are whole tiles of 128 rows: one launch of the tensor-core family
    (plus the one for t), every layer with its own slice of t and its own output."""
    layers = [make_case(70 + i, K, N, r, w=w, ab=ab) for i, N in enumerate(Ns)]
    x = gen.make_x(71, M, K, xd)
    F = eora.FusedLayers(layers, max_m=64, x_dtype=xd)
    assert F.launches(M) <= 3
    for rep in range(2):
        ys = run_fused(F, x, xd)
        for i, (wf, af, bf) in enumerate(layers):
            check_parity(ys[i], orc.forward(x, xd, wf, af, bf), f"layer {i} call {rep}")
    x8 = gen.make_x(72, 8, K, xd)              # and the decode family on the same handle
    ys = run_fused(F, x8, xd)
    for i, (wf, af, bf) in enumerate(layers):
        check_parity(ys[i], orc.forward(x8, xd, wf, af, bf), f"layer {i} M=8")
    F.close()


def test_fused_fullsize_64_tokens():
    names = ("q", "k", "v")
    K = SHAPES[names[0]][0]
    layers = [make_case(80 + i, K, SHAPES[nm][1], 128, w="q4", ab="q4") for i, nm in enumerate(names)]
    x = gen.make_x(81, 64, K)
    F = eora.FusedLayers(layers, max_m=64)
    ys = run_fused(F, x, "f16")
    for i, (wf, af, bf) in enumerate(layers):
        check_parity(ys[i], orc.forward(x, "f16", wf, af, bf), names[i])
    F.close()


@pytest.mark.parametrize("names,w", [(("q", "k", "v"), "q3"), (("gate", "up"), "q3"), (("q", "k", "v"), "q4")])
def test_fused_fullsize(names, w):
    K = SHAPES[names[0]][0]
    layers = [make_case(60 + i, K, SHAPES[nm][1], 128, w=w) for i, nm in enumerate(names)]
    x = gen.make_x(61, 1, K)
    F = eora.FusedLayers(layers, max_m=1)
    ys = run_fused(F, x, "f16")
    for i, (wf, af, bf) in enumerate(layers):
        rel, _ = check_parity(ys[i], orc.forward(x, "f16", wf, af, bf), names[i])
        assert 5e-5 < rel < 1e-3
    F.close()


@pytest.mark.parametrize("pinned", [(True, True), (True, False), (False, False)])
def test_fused_forward_host(pinned):
    """The host entry point: every combination of page-locked (written by the kernel) and pageable (staged) results."""
    import torch
    K, Ns, r, M = 512, [96, 160], 128, 5
    layers = [make_case(80 + i, K, N, r, w="q3") for i, N in enumerate(Ns)]
    x = gen.make_x(81, M, K)
    F = eora.FusedLayers(layers, max_m=M)
    xh = torch.from_numpy(x.copy()).pin_memory()
    yh = [torch.full((M, N), float("nan"), dtype=torch.float16) for N in Ns]
    yh = [y.pin_memory() if p else y for y, p in zip(yh, pinned)]
    for rep in range(2):
        for y in yh:
            y.fill_(float("nan"))
        F.forward_host(xh, yh)
        assert F.device_status() == 0
        for i, (wf, af, bf) in enumerate(layers):
            check_parity(yh[i].float().numpy().astype(np.float64), orc.forward(x, "f16", wf, af, bf), f"layer {i} call {rep}")
    F.close()


def test_fused_argument_errors():
    import torch
    K = 256
    la = make_case(70, K, 64, 64)
    lb = make_case(71, K, 32, 64)
    lc = make_case(72, K, 32, 128)                         # other rank
    ld = make_case(73, 512, 32, 64)                        # other d_in
    m = dict(max_m=4, x_dtype="f16", y_dtype="f16", kernel_policy=eora.EORA_POLICY_AUTO, device="cuda:0")
    def status(ls, **kw):
        mm = dict(m); mm.update(kw)
        parts = [eora._marshal(*l, **mm) for l in ls]
        return eora.eora_linear_create_fused([p[0] for p in parts], [p[1] for p in parts], check=False)
    assert status([la, lb]) == eora.EORA_OK
    assert status([la, lc]) == eora.EORA_ERR_BAD_SHAPE
    assert status([la, ld]) == eora.EORA_ERR_BAD_SHAPE
    assert status([la, lb], max_m=65) == eora.EORA_ERR_UNSUPPORTED
    assert status([la] * 5) == eora.EORA_ERR_BAD_SHAPE
    F = eora.FusedLayers([la, lb], max_m=4)
    x = torch.zeros((4, K), dtype=torch.float16, device="cuda:0")
    y = torch.zeros((4, 96), dtype=torch.float16, device="cuda:0")
    assert eora.eora_linear_forward(F.handle, x, 1, y, check=False) == eora.EORA_ERR_UNSUPPORTED
    assert eora.eora_linear_forward_fused(F.handle, x, 5, [y, y], check=False) == eora.EORA_ERR_M_TOO_LARGE
    assert eora.eora_linear_forward_fused(F.handle, x, 1, [y, None], check=False) == eora.EORA_ERR_NULL_ARG
    torch.cuda.synchronize()
    F.close()


@pytest.mark.parametrize("w,ab,K,Ns,r,M,xd", [
    ("q4", "f16", 1024, [256, 128, 128], 128, 65, "f16"),     # a 128-row layer: tiles of 128 rows throughout
    ("q3", "q4", 512, [512, 256], 64, 300, "f16"),            # whole 256-row tiles, two token tiles with a ragged tail
    ("q4", "q8", 1024, [128, 384], 256, 130, "bf16"),
    ("q4", "f16", 768, [256, 256], 0, 257, "f16"),            # no adapter
    ("sp24", "f16", 512, [128, 256], 128, 96, "f16"),
])
def test_fused_many_tokens_tensor_core_family(w, ab, K, Ns, r, M, xd):
    """More than 64 tokens on a fused handle: the tensor-core family writes every layer's tiles to that layer's output
    and takes that layer's slice of t; compared with the oracle's forward of each layer, whole outputs."""
    layers = [make_case(90 + i, K, N, r, w=w, ab=ab) for i, N in enumerate(Ns)]
    x = gen.make_x(91, M, K, xd)
    F = eora.FusedLayers(layers, max_m=M, x_dtype=xd)
    assert F.launches(M) <= 3
    for rep in range(2):
        ys = run_fused(F, x, xd)
        for i, (wf, af, bf) in enumerate(layers):
            check_parity(ys[i], orc.forward(x, xd, wf, af, bf), f"layer {i} call {rep}")
    for m2 in (1, 8, 40):                                   # and the other families on the same handle
        x2 = gen.make_x(92, m2, K, xd)
        ys = run_fused(F, x2, xd)
        for i, (wf, af, bf) in enumerate(layers):
            check_parity(ys[i], orc.forward(x2, xd, wf, af, bf), f"layer {i} M={m2}")
    F.close()


@pytest.mark.parametrize("names", [("q", "k", "v"), ("gate", "up")])
def test_fused_fullsize_prefill_sampled(names):
    """M = 2048 at the full sizes (gate | up takes the launch whose last row tiles are covered by small tiles): sampled
    outputs of every layer, with the corners, the last columns and both sides of tile borders among them."""
    import torch
    K = SHAPES[names[0]][0]
    M = 2048
    layers = [make_case(95 + i, K, SHAPES[nm][1], 128, w="q4") for i, nm in enumerate(names)]
    x = gen.make_x(96, M, K)
    F = eora.FusedLayers(layers, max_m=M)
    assert F.launches(M) == 2
    ys = run_fused(F, x, "f16")
    rng = np.random.default_rng(5)
    for i, (wf, af, bf) in enumerate(layers):
        y = ys[i]
        N = y.shape[1]
        mi = rng.integers(0, M, 64); ni = rng.integers(0, N, 64)
        mi[:4] = [0, M - 1, 0, M - 1]; ni[:4] = [0, 0, N - 1, N - 1]
        ni[4:16] = N - 1 - rng.integers(0, min(N, 512), 12)
        ni[16:24] = np.clip(128 * rng.integers(1, max(2, N // 128), 8) - rng.integers(0, 2, 8), 0, N - 1)
        mi[24:32] = np.clip(128 * rng.integers(1, max(2, M // 128), 8) - rng.integers(0, 2, 8), 0, M - 1)
        ref = orc.forward_at(x, "f16", wf, af, bf, mi, ni)
        d = y[mi, ni] - ref
        assert np.all(np.isfinite(y)), names[i]
        assert np.linalg.norm(d) / np.linalg.norm(ref) <= 2e-3, names[i]
        assert np.abs(d).max() <= 1e-2 * np.abs(ref).max(), names[i]
    F.close()


def test_fused_forward_host_many_tokens():
    """The host entry point above 64 tokens: results go through the staging buffer (side by side) and the copy engine."""
    import torch
    K, Ns, r, M = 512, [128, 256], 64, 100
    layers = [make_case(97 + i, K, N, r, w="q4") for i, N in enumerate(Ns)]
    x = gen.make_x(98, M, K)
    F = eora.FusedLayers(layers, max_m=M)
    xh = torch.from_numpy(x.copy()).pin_memory()
    yh = [torch.full((M, N), float("nan"), dtype=torch.float16).pin_memory() for N in Ns]
    for rep in range(2):
        F.forward_host(xh, yh)
        assert F.device_status() == 0
        for i, (wf, af, bf) in enumerate(layers):
            check_parity(yh[i].float().numpy().astype(np.float64), orc.forward(x, "f16", wf, af, bf), f"layer {i} call {rep}")
    F.close()
