"""GPU parity at the full LLaMA3-8B layer sizes, in the launch configuration bench.py times.

Decode cases (M <= 64) are compared element by element with the float64 oracle (its forward is cheap at
small M).  Prefill cases (M = 2048) are compared on sampled outputs that the oracle computes one by one
(forward_at), plus the whole output for the smallest shape.  Tolerances as everywhere: rel. Frobenius
<= 2e-3, max|diff| <= 1e-2 * max|y| (for sampled checks the norms run over the samples)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_oracle as orc
import eora_inputs as gen
import paper_2410_21271_b200 as eora
from helpers import make_case, run_layer, check_parity, x_to_torch

SHAPES = gen.LLAMA3_8B_SHAPES


def sampled_check(L, wf, af, bf, x, xd, n_samples=96, seed=0):
    y = run_layer(L, x, xd)
    rng = np.random.default_rng(seed)
    M, N = y.shape
    mi = rng.integers(0, M, n_samples)
    ni = rng.integers(0, N, n_samples)
    mi[:4] = [0, M - 1, 0, M - 1]; ni[:4] = [0, 0, N - 1, N - 1]          # corners: first / last tile edges
    # the last output columns (a launch may cover them with tiles of another size) and both sides of tile borders
    ni[4:20] = N - 1 - rng.integers(0, min(N, 512), 16)
    ni[20:28] = np.clip(128 * rng.integers(1, max(2, N // 128), 8) - rng.integers(0, 2, 8), 0, N - 1)
    mi[28:36] = np.clip(128 * rng.integers(1, max(2, M // 128), 8) - rng.integers(0, 2, 8), 0, M - 1)
    ref = orc.forward_at(x, xd, wf, af, bf, mi, ni)
    got = y[mi, ni]
    d = got - ref
    assert np.all(np.isfinite(y))
    assert np.linalg.norm(d) / np.linalg.norm(ref) <= 2e-3
    assert np.abs(d).max() <= 1e-2 * np.abs(ref).max()


# config 1 and 2: 4-bit / 3-bit backbone, fp16 rank-128 adapter, decode
@pytest.mark.parametrize("name", ["q", "k", "gate", "down"])
@pytest.mark.parametrize("w,M", [("q4", 1), ("q3", 1), ("q3", 8), ("q3", 16)])
def test_decode_fullsize(name, w, M):
    K, N = SHAPES[name]
    wf, af, bf = make_case(31, K, N, 128, w=w)
    x = gen.make_x(32, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    assert L.path(M) == (eora.EORA_PATH_DECODE if M <= 8 else eora.EORA_PATH_PREFILL)
    y = run_layer(L, x, "f16")
    rel, _ = check_parity(y, orc.forward(x, "f16", wf, af, bf), f"{name} {w} M{M}")
    assert 5e-5 < rel < 1e-3          # fp16 output rounding alone is ~2e-4: far off means a harness bug
    L.close()


# config 3: quantised adapter
@pytest.mark.parametrize("name,ab,r,M", [("q", "q4", 128, 1), ("k", "q4", 512, 16), ("q", "q8", 128, 64),
                                         ("down", "q4", 128, 1), ("gate", "q8", 512, 1)])
def test_decode_quantised_adapter_fullsize(name, ab, r, M):
    K, N = SHAPES[name]
    wf, af, bf = make_case(33, K, N, r, w="q4", ab=ab)
    x = gen.make_x(34, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    # eight decode passes (M = 64) cost more than one walk over the k-blocks with the tensor-core family
    assert L.path(M) == (eora.EORA_PATH_PREFILL if M > 8 else eora.EORA_PATH_DECODE)
    check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), f"{name} {ab} r{r} M{M}")
    L.close()


# config 4: prefill
def test_prefill_fullsize_whole_output():
    K, N = SHAPES["k"]
    M = 2048
    wf, af, bf = make_case(35, K, N, 128, w="q4")
    x = gen.make_x(36, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    assert L.path(M) == eora.EORA_PATH_PREFILL
    rel, _ = check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), "k prefill")
    assert 5e-5 < rel < 1e-3
    L.close()


@pytest.mark.parametrize("name,r,xd", [("q", 128, "f16"), ("q", 512, "bf16"), ("gate", 64, "f16"), ("down", 128, "bf16")])
def test_prefill_fullsize_sampled(name, r, xd):
    K, N = SHAPES[name]
    M = 2048
    wf, af, bf = make_case(37, K, N, r, w="q4")
    x = gen.make_x(38, M, K, xd)
    L = eora.Layer(wf, af, bf, max_m=M, x_dtype=xd)
    assert L.path(M) == eora.EORA_PATH_PREFILL
    sampled_check(L, wf, af, bf, x, xd)
    L.close()


def test_prefill_weights_are_the_rounded_dequantised_values():
    """X = identity block, rank 0, fp32 out: Y is the fp16-rounded dequantised weight, bit for bit."""
    K, N = 512, 256
    wf, _, _ = make_case(39, K, N, 0, w="q4")
    x = np.eye(K, dtype=np.float16)
    L = eora.Layer(wf, None, None, max_m=K, y_dtype="f32")
    assert L.path(K) == eora.EORA_PATH_PREFILL
    y = run_layer(L, x, "f16")
    q = orc.unpack_codes(wf["codes"], 4, K); z = orc.unpack_zeros(wf["zeros"], 4, N)
    assert np.array_equal(y, orc.deq_fp16(q, z, wf["scales"], 128).astype(np.float64))
    L.close()


# config 5: 2:4 backbone
@pytest.mark.parametrize("name,M", [("k", 1), ("q", 1), ("k", 2048)])
def test_sparse24_fullsize(name, M):
    K, N = SHAPES[name]
    wf, af, bf = make_case(41, K, N, 128, w="sp24")
    x = gen.make_x(42, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    if M == 1:
        assert L.path(M) == eora.EORA_PATH_DECODE
        check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), f"{name} sp24 M1")
    else:
        assert L.path(M) == eora.EORA_PATH_PREFILL
        sampled_check(L, wf, af, bf, x, "f16")
    L.close()


def test_prefill_small_formats():
    """Every adapter format and odd sizes through the tensor-core path."""
    for (w, ab, K, N, r, M, yd) in [("q3", "q4", 512, 352, 128, 130, "f16"), ("q4", "q8", 640, 96, 64, 257, "bf16"),
                                    ("sp24", "f16", 384, 288, 24, 100, "f32"), ("q3", "f16", 1024, 512, 0, 300, "f16")]:
        wf, af, bf = make_case(43, K, N, r, w=w, ab=ab)
        x = gen.make_x(44, M, K)
        L = eora.Layer(wf, af, bf, max_m=M, y_dtype=yd)
        assert L.path(M) == eora.EORA_PATH_PREFILL
        y = run_layer(L, x, "f16")
        rel, mabs = orc.parity_errors(y, orc.forward(x, "f16", wf, af, bf))
        assert rel <= 2e-3 and mabs <= 1e-2, (w, ab, rel, mabs)
        y2 = run_layer(L, x, "f16")           # scratch (the split-K sums of t) must have been restored
        rel2, mabs2 = orc.parity_errors(y2, orc.forward(x, "f16", wf, af, bf))
        assert rel2 <= 2e-3 and mabs2 <= 1e-2, (w, ab, rel2, mabs2)
        L.close()


def test_mid_size_m_takes_the_tensor_core_family():
    """Up to 8 tokens: one decode pass; from 9 on one launch of the tensor-core family, which for up to 64 tokens splits
    the reduction axis over several CTAs per tile (sums in fp32 scratch, tickets, restored by the last CTA)."""
    for name, Ms in [("q", (9, 24, 64)), ("down", (16, 57)), ("k", (33,))]:
        K, N = SHAPES[name]
        wf, af, bf = make_case(45, K, N, 128, w="q4")
        L = eora.Layer(wf, af, bf, max_m=64)
        for M in (1, 8):
            assert L.path(M) == eora.EORA_PATH_DECODE, (name, M)
        for M in (9, 16, 17, 24, 48, 64):
            assert L.path(M) == eora.EORA_PATH_PREFILL, (name, M)
        for M in Ms:
            x = gen.make_x(46, M, K)
            for rep in range(2):               # second call: sums and tickets were restored
                check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), f"{name} q4 M{M} call {rep}")
        L.close()


@pytest.mark.parametrize("w,ab,K,N,r,M,xd,yd", [
    ("q4", "f16", 2048, 384, 128, 17, "f16", "f16"),      # 32 k-blocks: four CTAs per tile
    ("q3", "q4", 1152, 160, 64, 40, "f16", "f32"),        # 18 k-blocks in two uneven shares, rows past the matrix
    ("q4", "q8", 4096, 96, 512, 64, "bf16", "bf16"),      # rank 512: t has four row tiles
    ("sp24", "f16", 2048, 256, 0, 33, "f16", "f16"),      # no adapter
    ("sq4", "q3", 1024, 128, 128, 64, "f16", "f16"),
    ("q3", "f16", 640, 224, 32, 20, "f16", "f16"),        # too few k-blocks to split: one CTA per tile
])
def test_few_tokens_split_reduction(w, ab, K, N, r, M, xd, yd):
    wf, af, bf = make_case(47, K, N, r, w=w, ab=ab)
    x = gen.make_x(48, M, K, xd)
    L = eora.Layer(wf, af, bf, max_m=64, x_dtype=xd, y_dtype=yd)
    assert L.path(M) == eora.EORA_PATH_PREFILL
    ref = orc.forward(x, xd, wf, af, bf)
    for rep in range(3):
        y = run_layer(L, x, xd)
        rel, mabs = orc.parity_errors(y, ref)
        assert rel <= 2e-3 and mabs <= 1e-2, (rep, rel, mabs)
    x1 = gen.make_x(49, 1, K, xd)              # the decode family on the same handle afterwards
    y1 = run_layer(L, x1, xd)
    rel, mabs = orc.parity_errors(y1, orc.forward(x1, xd, wf, af, bf))
    assert rel <= 2e-3 and mabs <= 1e-2, ("M=1 after split launches", rel, mabs)
    L.close()


# ---- full-size cells that take other tile / wave paths than the small cases ------------------------------------------
def sampled_check_last_tiles(L, wf, af, bf, x, xd, n_samples=64, seed=1):
    """Samples aimed at the last 128-row tiles of the output (a launch may cover them with tiles of another size) and at
    the last tokens."""
    y = run_layer(L, x, xd)
    rng = np.random.default_rng(seed)
    M, N = y.shape
    mi = rng.integers(0, M, n_samples)
    ni = N - 1 - rng.integers(0, min(N, 640), n_samples)
    mi[: n_samples // 4] = M - 1 - rng.integers(0, min(M, 128), n_samples // 4)
    ref = orc.forward_at(x, xd, wf, af, bf, mi, ni)
    d = y[mi, ni] - ref
    assert np.all(np.isfinite(y))
    assert np.linalg.norm(d) / np.linalg.norm(ref) <= 2e-3
    assert np.abs(d).max() <= 1e-2 * np.abs(ref).max()


@pytest.mark.parametrize("w", ["sp24", "sq4"])
@pytest.mark.parametrize("name", ["gate", "down"])
def test_sparse_backbones_fullsize_single_token(w, name):
    K, N = SHAPES[name]
    wf, af, bf = make_case(47, K, N, 128, w=w)
    x = gen.make_x(48, 1, K)
    L = eora.Layer(wf, af, bf, max_m=1)
    assert L.path(1) == eora.EORA_PATH_DECODE
    check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), f"{name} {w} M1")
    L.close()


@pytest.mark.parametrize("w", ["sp24", "sq4"])
@pytest.mark.parametrize("name", ["q", "gate", "down"])
def test_sparse_backbones_fullsize_prefill(w, name):
    """gate at M = 2048 is the launch whose last row tiles are covered by 128 x 128 tiles."""
    K, N = SHAPES[name]
    M = 2048
    wf, af, bf = make_case(49, K, N, 128, w=w)
    x = gen.make_x(50, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    assert L.path(M) == eora.EORA_PATH_PREFILL
    sampled_check(L, wf, af, bf, x, "f16", n_samples=64)
    sampled_check_last_tiles(L, wf, af, bf, x, "f16")
    L.close()


def test_quantised_adapter_rank512_m64_on_gate():
    K, N = SHAPES["gate"]
    wf, af, bf = make_case(57, K, N, 512, w="q4", ab="q4")
    x = gen.make_x(58, 64, K)
    L = eora.Layer(wf, af, bf, max_m=64)
    check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), "gate q4 adapters r512 M64")
    L.close()


def test_quantised_adapter_prefill_last_tiles_on_gate():
    K, N = SHAPES["gate"]
    M = 2048
    wf, af, bf = make_case(59, K, N, 128, w="q4", ab="q4")
    x = gen.make_x(60, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    sampled_check_last_tiles(L, wf, af, bf, x, "f16")
    L.close()


@pytest.mark.parametrize("M", [1, 16])
def test_three_bit_adapter_fullsize(M):
    K, N = SHAPES["q"]
    wf, af, bf = make_case(61, K, N, 128, w="q4", ab="q3")
    x = gen.make_x(62, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    check_parity(run_layer(L, x, "f16"), orc.forward(x, "f16", wf, af, bf), f"q 3-bit adapters M{M}")
    L.close()


def test_fused_qkv_fullsize_eight_tokens():
    import torch
    K, r, M = 4096, 128, 8
    parts = [(gen.make_backbone_quant(63 + i, K, n, 3, 128),) + gen.make_ab_f16(63 + i, K, n, r) for i, n in enumerate((4096, 1024, 1024))]
    x = gen.make_x(66, M, K)
    F = eora.FusedLayers(parts, max_m=M)
    ys = F.forward(x_to_torch(x, "f16"))
    torch.cuda.synchronize()
    assert F.device_status() == 0
    for (w, a, b), y in zip(parts, ys):
        check_parity(y.float().cpu().numpy().astype(np.float64), orc.forward(x, "f16", w, a, b), "fused q|k|v M8")
    F.close()


@pytest.mark.parametrize("name,M", [("q", 3072), ("q", 1536), ("k", 4096), ("gate", 1024)])
def test_prefill_other_token_counts_sampled(name, M):
    """Token counts at which the launch picks another tiling than at M = 2048 (rows per CTA are chosen by counting the
    waves of both tilings; q at M = 3072 takes tiles of 128 rows)."""
    K, N = SHAPES[name]
    wf, af, bf = make_case(41, K, N, 128, w="q4")
    x = gen.make_x(42, M, K)
    L = eora.Layer(wf, af, bf, max_m=M)
    assert L.path(M) == eora.EORA_PATH_PREFILL
    sampled_check(L, wf, af, bf, x, "f16")
    L.close()
