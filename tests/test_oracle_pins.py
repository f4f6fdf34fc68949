"""Pins for the CPU oracle: every check here compares the oracle with something that is not
the oracle -- hand-packed words, hand-evaluated numbers, bit-by-bit brute force, library
matmuls on independently built matrices, algebraic invariants."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import eora_oracle as orc
import eora_inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- helpers
def scalar_code(words, bits, k, n):
    """Independent scalar reader: assemble the code of (k, n) one stream bit at a time."""
    v = 0
    for b in range(bits):
        p = bits * k + b
        bit = (int(words[p // 32][n]) >> (p % 32)) & 1
        v |= bit << b
    return v


def scalar_zero(zwords, bits, g, n):
    v = 0
    for b in range(bits):
        p = bits * n + b
        v |= ((int(zwords[g][p // 32]) >> (p % 32)) & 1) << b
    return v


def scalar_dense(fmt):
    """Dense matrix as exact Fractions from a 'quant' fmt, element by element."""
    K, N, bits, grp = fmt["rows"], fmt["cols"], fmt["bits"], fmt["group"]
    W = [[None] * N for _ in range(K)]
    for k in range(K):
        for n in range(N):
            q = scalar_code(fmt["codes"], bits, k, n)
            z = scalar_zero(fmt["zeros"], bits, k // grp, n)
            s = Fraction(float(fmt["scales"][k // grp][n]))
            W[k][n] = (q - z) * s
    return W


def scalar_forward(X, W, A, B):
    """Exact rational y = X.W + (X.A).B with per-element loops (lists of Fractions)."""
    M, K, N = len(X), len(W), len(W[0])
    r = len(B)
    y = [[Fraction(0)] * N for _ in range(M)]
    for m in range(M):
        t = [sum(X[m][k] * A[k][j] for k in range(K)) for j in range(r)]
        for n in range(N):
            acc = sum(X[m][k] * W[k][n] for k in range(K))
            acc += sum(t[j] * B[j][n] for j in range(r))
            y[m][n] = acc
    return y


def fr(a):
    return [[Fraction(float(v)) for v in row] for row in np.asarray(a)]


def read_kv(path):
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(":", 1)
        out[k.strip()] = v.split()
    return out


# --------------------------------------------------------------------------- a1 unpack
def test_unpack4_hand_packed():
    w = np.array([[0x76543210, 0xFFFFFFFF, 0x00900000]], dtype=np.uint32)
    q = orc.unpack_codes(w, 4, 8)
    assert q[:, 0].tolist() == [0, 1, 2, 3, 4, 5, 6, 7]
    assert q[:, 1].tolist() == [15] * 8
    assert q[:, 2].tolist() == [0, 0, 0, 0, 0, 9, 0, 0]


def test_unpack3_hand_packed():
    for line in open(os.path.join(GOLDEN, "unpack3_hand_packed.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, rule, words = [p.strip() for p in line.split(";")]
        words = np.array([[int(x, 16)] for x in words.split()], dtype=np.uint32)
        want = [eval(rule, {"j": j}) for j in range(32)]
        got = orc.unpack_codes(words, 3, 32)[:, 0].tolist()
        assert got == want, name


def test_unpack3_straddling_codes():
    # code 10 = stream bits 30..32, code 21 = bits 63..65: set only those
    w = np.zeros((3, 1), dtype=np.uint32)
    w[0, 0] = 0b01 << 30          # low two bits of code 10 = 01
    w[1, 0] = 0b1 | (1 << 31)     # top bit of code 10 = 1 -> code 10 = 0b101 = 5 ; bit 63 -> low bit of code 21
    w[2, 0] = 0b11                # bits 64,65 -> code 21 = 0b111 = 7
    q = orc.unpack_codes(w, 3, 32)[:, 0]
    want = [0] * 32
    want[10], want[21] = 5, 7
    assert q.tolist() == want


@pytest.mark.parametrize("bits", [3, 4])
def test_unpack_matches_bit_by_bit(bits):
    rng = np.random.default_rng(7)
    K, N = 64, 5
    words = rng.integers(0, 2**32, size=(bits * K // 32, N), dtype=np.uint32)
    q = orc.unpack_codes(words, bits, K)
    for k in range(K):
        for n in range(N):
            assert q[k, n] == scalar_code(words, bits, k, n)
    zw = rng.integers(0, 2**32, size=(3, bits * 32 // 32), dtype=np.uint32)
    z = orc.unpack_zeros(zw, bits, 32)
    for g in range(3):
        for n in range(32):
            assert z[g, n] == scalar_zero(zw, bits, g, n)


@pytest.mark.parametrize("bits", [3, 4])
def test_pack_then_unpack_is_identity(bits):
    rng = np.random.default_rng(11)
    codes = rng.integers(0, 2**bits, size=(96, 7))
    assert np.array_equal(orc.unpack_codes(gen.pack_stream(codes, bits), bits, 96), codes)


# --------------------------------------------------------------------------- a2 dequant
def test_dequant_hand_value():
    s = np.array([[0x191F]], dtype=np.uint16)                 # fp16 nearest to 0.0025
    assert float(orc.to_f64(s, "f16")[0, 0]) == 0.0025005340576171875
    w = orc.dequant_groupwise(np.array([[5]]), np.array([[8]]), s.view(np.float16), 1)
    assert float(w[0, 0]) == -0.0075016021728515625          # (5 - 8) * s, exact in binary


def test_dequant_group_indexing():
    # K=4, group=2: rows 0,1 use group 0; rows 2,3 use group 1 -- distinct z and s per group/col
    q = np.array([[1, 2], [3, 4], [5, 6], [7, 0]])
    z = np.array([[1, 0], [2, 3]])
    s = np.array([[0.5, 2.0], [0.25, 1.0]], dtype=np.float16)
    w = orc.dequant_groupwise(q, z, s, 2)
    assert w.tolist() == [[0.0, 4.0], [1.0, 8.0], [0.75, 3.0], [1.25, -3.0]]


def test_dequant_fp32_is_exact_for_every_scale():
    # every positive finite fp16 scale x every (q - z) of 4-bit and 8-bit codes
    bits = np.arange(1, 0x7C00, dtype=np.uint16)
    s64 = bits.view(np.float16).astype(np.float64)
    s32 = bits.view(np.float16).astype(np.float32)
    for d in list(range(-15, 16)) + [-255, -254, -129, 127, 253, 255]:
        exact = s64 * d
        assert np.array_equal((s32 * np.float32(d)).astype(np.float64), exact)
    # and the oracle's own fp32 export returns that value
    q = np.array([[5, 0], [15, 7]]); z = np.array([[8, 15]])
    s = np.array([[0.0025, 0.0031]], dtype=np.float16)
    w32 = orc.deq_fp32(q, z, s, 2)
    assert w32.dtype == np.float32
    assert float(w32[0, 0]) == -3 * float(s[0, 0]) and float(w32[1, 1]) == -8 * float(s[0, 1])
    w16 = orc.deq_fp16(q, z, s, 2)
    assert w16.dtype == np.float16 and float(w16[1, 0]) == float(np.float16(7 * float(s[0, 0])))


def test_deq_fp16_rounds_to_nearest_even_hand_worked():
    """Hand-worked ties.  s = 1 + 3 * 2^-10 (fp16 bits 0x3C03); 3 s = 3 + 9 * 2^-10 lies exactly between the fp16 neighbours
    3 + 8 * 2^-10 (bits 0x4204, even mantissa) and 3 + 10 * 2^-10 (0x4205): round-to-nearest-even takes 0x4204, rounding
    halves up would take 0x4205.  With s = 1 + 2^-10 (0x3C01), 3 s = 3 + 3 * 2^-10 is the tie between 0x4201 and 0x4202 and
    goes UP to the even 0x4202; truncation would give 0x4201.  Negative products mirror both.  The products have at most
    5 + 11 significant bits, so an fp32 intermediate holds them exactly and cannot double-round."""
    s = np.array([[0x3C03, 0x3C01, 0x3C03, 0x3C01]], dtype=np.uint16).view(np.float16)
    q = np.array([[3, 3, 0, 0]], dtype=np.int64)
    z = np.array([[0, 0, 3, 3]], dtype=np.int64)
    w16 = orc.deq_fp16(q, z, s, 1)
    assert w16.view(np.uint16).tolist() == [[0x4204, 0x4202, 0xC204, 0xC202]]
    w32 = orc.deq_fp32(q, z, s, 1)
    assert [float(v) for v in w32[0]] == [3 + 9 / 1024, 3 + 3 / 1024, -(3 + 9 / 1024), -(3 + 3 / 1024)]   # exact in fp32


def test_q8_per_channel():
    codes = np.array([[0, 255], [128, 1]], dtype=np.uint8)
    fmt = {"kind": "q8", "rows": 2, "cols": 2, "codes": codes,
           "scales": np.array([0.5, 0.25], dtype=np.float16), "zeros": np.array([128, 1], dtype=np.uint8)}
    assert orc.dequant_matrix(fmt).tolist() == [[-64.0, 63.5], [0.0, 0.0]]


# --------------------------------------------------------------------------- forward
def test_worked_example_eq4():
    g = read_kv(os.path.join(GOLDEN, "worked_example_eq4.txt"))
    codes = np.array([[int(g["packed_col0"][0], 16), int(g["packed_col1"][0], 16)]], dtype=np.uint32)
    zeros = np.array([[int(g["packed_zeros"][0], 16)]], dtype=np.uint32)
    scales = np.array([[float(v) for v in g["scales"]]], dtype=np.float16)
    wf = {"kind": "quant", "bits": 4, "group": 8, "rows": 8, "cols": 2,
          "codes": codes, "scales": scales, "zeros": zeros}
    q = orc.unpack_codes(codes, 4, 8)
    assert q[:, 0].tolist() == [int(v) for v in g["codes_col0"]]
    assert q[:, 1].tolist() == [int(v) for v in g["codes_col1"]]
    assert orc.unpack_zeros(zeros, 4, 2).tolist() == [[int(v) for v in g["zeros"]]]
    W = orc.dequant_matrix(wf)
    assert W[:, 0].tolist() == [float(v) for v in g["w_col0"]]
    assert W[:, 1].tolist() == [float(v) for v in g["w_col1"]]
    x = np.array([[float(v) for v in g["x"]]], dtype=np.float16)
    A = {"kind": "f16", "data": np.array([[float(v)] for v in g["A"]], dtype=np.float16)}
    B = {"kind": "f16", "data": np.array([[float(v) for v in g["B"]]], dtype=np.float16)}
    y0 = orc.forward(x, "f16", wf, None, None)
    assert y0.tolist() == [[float(v) for v in g["xw"]]]
    y = orc.forward(x, "f16", wf, A, B)
    assert y.tolist() == [[float(v) for v in g["y"]]]
    ys = orc.forward_at(x, "f16", wf, A, B, np.array([0, 0]), np.array([1, 0]))
    assert ys.tolist() == [float(g["y"][1]), float(g["y"][0])]


@pytest.mark.parametrize("bits,K,N,r,M", [(4, 128, 32, 0, 1), (4, 256, 32, 32, 3), (3, 128, 64, 32, 1),
                                          (3, 256, 32, 0, 3)])
def test_forward_brute_force_exact_rationals(bits, K, N, r, M):
    """Tiny shapes against a scalar, bit-by-bit, exact-rational evaluation of Eq. 4.  Non-square
    shapes with distinct K, N, r, M catch transposed operands and swapped indices."""
    wf = gen.make_backbone_quant(100 + bits, K, N, bits, 128)
    x = gen.make_x(5, M, K, "f16")
    if r:
        af, bf = gen.make_ab_f16(6, K, N, r)
        A, B = fr(af["data"]), fr(bf["data"])
    else:
        af = bf = None
        A, B = [[] for _ in range(K)], []
    want = scalar_forward(fr(x), scalar_dense(wf), A, B)
    got = orc.forward(x, "f16", wf, af, bf)
    for m in range(M):
        for n in range(N):
            w = float(want[m][n])
            assert abs(got[m, n] - w) <= 1e-12 * max(1.0, abs(w)), (m, n)
    # sampled entry points agree with the same rationals
    mi = np.array([M - 1, 0]); ni = np.array([N - 1, 3])
    s = orc.forward_at(x, "f16", wf, af, bf, mi, ni)
    for i in range(2):
        assert abs(s[i] - float(want[mi[i]][ni[i]])) <= 1e-12


def test_rank0_and_zero_adapter_reduce_to_plain_matmul():
    import torch
    K, N, M, r = 256, 96, 4, 32
    wf = gen.make_backbone_quant(1, K, N, 4, 128)
    x = gen.make_x(2, M, K, "f16")
    af, bf = gen.make_ab_f16(3, K, N, r)
    # textbook X.W from a matrix assembled element-wise by the scalar reader, multiplied by torch
    Wd = np.array([[float(v) for v in row] for row in scalar_dense(wf)], dtype=np.float64)
    ref = (torch.from_numpy(x.astype(np.float64)) @ torch.from_numpy(Wd)).numpy()
    y_r0 = orc.forward(x, "f16", wf, None, None)
    assert np.allclose(y_r0, ref, rtol=0, atol=1e-12)
    zeroA = {"kind": "f16", "data": np.zeros_like(af["data"])}
    zeroB = {"kind": "f16", "data": np.zeros_like(bf["data"])}
    assert np.array_equal(orc.forward(x, "f16", wf, zeroA, bf), y_r0)
    assert np.array_equal(orc.forward(x, "f16", wf, af, zeroB), y_r0)
    empty = ({"kind": "f16", "data": np.zeros((K, 0), np.float16)}, {"kind": "f16", "data": np.zeros((0, N), np.float16)})
    assert np.array_equal(orc.forward(x, "f16", wf, *empty), y_r0)
    # and with the adapter on, the difference is exactly the textbook low-rank term
    y = orc.forward(x, "f16", wf, af, bf)
    lr = (torch.from_numpy(x.astype(np.float64)) @ torch.from_numpy(af["data"].astype(np.float64))
          @ torch.from_numpy(bf["data"].astype(np.float64))).numpy()
    assert np.allclose(y - y_r0, lr, rtol=0, atol=1e-12)


@pytest.mark.parametrize("bits", [3, 4])
def test_one_hot_and_identity_inputs(bits):
    K, N, r = 128, 32, 32
    wf = gen.make_backbone_quant(9, K, N, bits, 128)
    af, bf = gen.make_ab_f16(10, K, N, r)
    A = af["data"].astype(np.float64); B = bf["data"].astype(np.float64)
    for k in (0, 10, 21, 127):                                  # 10 and 21 straddle words when bits = 3
        x = np.zeros((1, K), dtype=np.float16); x[0, k] = 1.0
        y = orc.forward(x, "f16", wf, af, bf)[0]
        for n in (0, 7, N - 1):
            wkn = (scalar_code(wf["codes"], bits, k, n) - scalar_zero(wf["zeros"], bits, 0, n)) \
                * float(wf["scales"][0][n])
            want = wkn + math.fsum(A[k, j] * B[j, n] for j in range(r))
            assert abs(y[n] - want) <= 1e-15
    eye = np.eye(K, dtype=np.float16)
    Y = orc.forward(eye, "f16", wf, af, bf)
    Wd = np.array([[float(v) for v in row] for row in scalar_dense(wf)])
    assert np.allclose(Y, Wd + A @ B, rtol=0, atol=1e-15)


def test_linearity_in_x():
    K, N, r = 256, 64, 32
    wf = gen.make_backbone_quant(21, K, N, 3, 128)
    af, bf = gen.make_ab_f16(22, K, N, r)
    x1 = gen.make_x(23, 2, K).astype(np.float64); x2 = gen.make_x(24, 2, K).astype(np.float64)
    f = lambda x: orc.forward(x, "f64", wf, af, bf)
    assert np.allclose(f(0.75 * x1 + x2), 0.75 * f(x1) + f(x2), rtol=0, atol=1e-12)


def test_bf16_input_conversion():
    bits = np.array([[0x3F80, 0xC000, 0x3DCD, 0x0000]], dtype=np.uint16)      # 1.0, -2.0, 0.10009765625, 0
    assert orc.to_f64(bits, "bf16").tolist() == [[1.0, -2.0, 0.10009765625, 0.0]]
    assert gen.f32_to_bf16_bits(np.array([1.0, -2.0, 0.1, 1.00390625], np.float32)).tolist() == \
        [0x3F80, 0xC000, 0x3DCD, 0x3F80]      # 0.1 rounds up; 1 + 2^-8 is a tie -> even


# --------------------------------------------------------------------------- cross-format
def test_3bit_equals_4bit_on_codes_below_8():
    rng = np.random.default_rng(3)
    K, N = 128, 32
    q = rng.integers(0, 8, size=(K, N)); z = rng.integers(0, 8, size=(1, N))
    s = gen.make_scales(rng, (1, N))
    fmts = []
    for bits in (3, 4):
        fmts.append({"kind": "quant", "bits": bits, "group": 128, "rows": K, "cols": N,
                     "codes": gen.pack_stream(q, bits), "scales": s,
                     "zeros": np.ascontiguousarray(gen.pack_stream(np.ascontiguousarray(z.T), bits).T)})
    x = gen.make_x(1, 2, K)
    assert np.array_equal(orc.forward(x, "f16", fmts[0], None, None), orc.forward(x, "f16", fmts[1], None, None))


@pytest.mark.parametrize("abf", ["q4", "q3", "q8"])
def test_quantised_adapter_equals_dense_adapter(abf):
    K, N, r = 256, 64, 128
    wf = gen.make_backbone_quant(31, K, N, 4, 128)
    aq, bq = gen.make_ab_quant(32, K, N, r, abf)
    x = gen.make_x(33, 3, K)
    # dense adapter rebuilt element by element from the integer codes of the quantiser itself
    a16, b16 = gen.make_ab_f16(32, K, N, r)
    if abf in ("q4", "q3"):
        bits = 4 if abf == "q4" else 3
        ra, rb = gen.rtn_quantize(a16["data"], bits, 128), gen.rtn_quantize(b16["data"], bits, 128)
        ga, gb = 128, 128
    else:
        ra, rb = gen.rtn_quantize(a16["data"], 8, K), gen.rtn_quantize(b16["data"], 8, r)
        ga, gb = K, r
    def dense(rq, grp):
        rows, cols = rq["q"].shape
        out = np.empty((rows, cols))
        for i in range(rows):
            for j in range(cols):
                out[i, j] = (int(rq["q"][i, j]) - int(rq["z"][i // grp, j])) * float(rq["scales"][i // grp, j])
        return out
    Ad, Bd = dense(ra, ga), dense(rb, gb)
    y_q = orc.forward(x, "f16", wf, aq, bq)
    y_d = orc.forward(x, "f16", wf, {"kind": "f64", "data": Ad}, {"kind": "f64", "data": Bd})
    assert np.allclose(y_q, y_d, rtol=0, atol=1e-13)


def test_sparse24_equals_dense_on_expanded_matrix():
    K, N, r = 128, 48, 32
    sp = gen.make_sparse24(41, K, N)
    # independent scalar expansion
    Wd = np.zeros((K, N))
    for n in range(N):
        for j in range(K // 4):
            nib = (int(sp["meta"][n][j // 8]) >> (4 * (j % 8))) & 0xF
            p0, p1 = nib & 3, nib >> 2
            assert 0 <= p0 < p1 <= 3
            Wd[4 * j + p0, n] = float(sp["values"][n][2 * j])
            Wd[4 * j + p1, n] = float(sp["values"][n][2 * j + 1])
    assert np.array_equal(orc.dequant_matrix(sp), Wd)
    assert np.all((Wd.reshape(K // 4, 4, N) != 0).sum(axis=1) <= 2)
    af, bf = gen.make_ab_f16(42, K, N, r)
    x = gen.make_x(43, 2, K)
    y = orc.forward(x, "f16", sp, af, bf)
    y_d = orc.forward(x, "f16", {"kind": "f64", "data": Wd}, af, bf)
    assert np.array_equal(y, y_d)


def test_sparse24_hand_packed():
    # one quad: positions (1, 3) -> nibble 1 | 3<<2 = 0xD, values (2.0, -4.0)
    vals = np.zeros((1, 16), dtype=np.float16); vals[0, 0], vals[0, 1] = 2.0, -4.0
    vals[0, 2], vals[0, 3] = 1.0, 3.0                                    # quad 1: positions (0, 2) -> 0x8
    meta = np.array([[0xD | (0x8 << 4) | 0x44444440 << 4 & 0xFFFFFF00]], dtype=np.uint32)
    meta[0, 0] = 0xD | (0x8 << 4) | 0x44444400                           # remaining quads: (0,1) = 0x4
    W = orc.expand_sparse24(vals, meta, 32, 1)[:, 0]
    assert W[:8].tolist() == [0.0, 2.0, 0.0, -4.0, 1.0, 0.0, 3.0, 0.0]


def test_sparse24_quant_scalar_expansion():
    """2:4 + 4-bit (appendix on sparsity & quantisation compensation): bit-by-bit scalar unpack of every stored
    field, independent of the oracle's vectorised helpers."""
    K, N, group = 256, 16, 128
    sq = gen.make_sparse24_quant(44, K, N, 4, group)
    codes, scales, zeros, meta = sq["codes"], sq["scales"], sq["zeros"], sq["meta"]
    assert codes.shape == (K // 16, N) and scales.shape == (K // group, N) and zeros.shape == (K // group, N // 8)
    Wd = np.zeros((K, N))
    for n in range(N):
        for j in range(K // 4):
            nib = (int(meta[n][j // 8]) >> (4 * (j % 8))) & 0xF
            pos = (nib & 3, nib >> 2)
            for i in range(2):
                c = 2 * j + i                                       # index among the kept values
                q = (int(codes[c // 8][n]) >> (4 * (c % 8))) & 0xF
                g = (4 * j) // group                                # group of the ORIGINAL k
                z = (int(zeros[g][n // 8]) >> (4 * (n % 8))) & 0xF
                Wd[4 * j + pos[i], n] = (q - z) * float(scales[g][n])
    assert np.array_equal(orc.dequant_matrix(sq), Wd)
    # the zero pattern is the 2:4 one, and the forward equals the dense forward on the expanded matrix
    assert np.all((Wd.reshape(K // 4, 4, N) != 0).sum(axis=1) <= 2)
    af, bf = gen.make_ab_f16(45, K, N, 32)
    x = gen.make_x(46, 3, K)
    assert np.array_equal(orc.forward(x, "f16", sq, af, bf), orc.forward(x, "f16", {"kind": "f64", "data": Wd}, af, bf))


def test_sparse24_quant_hand_packed():
    # K = 32, one column, group 32 (16 kept values): scale 0.5, zero 3; quad 0 keeps positions (1, 3) with codes
    # (7, 0), quad 1 positions (0, 2) with codes (3, 15); the other quads positions (0, 1) with code 3 (-> 0)
    codes = np.zeros((2, 1), dtype=np.uint32)
    codes[0, 0] = 7 | 0 << 4 | 3 << 8 | 15 << 12 | 0x33330000
    codes[1, 0] = 0x33333333
    scales = np.array([[0.5]], dtype=np.float16)
    zeros = np.array([[3]], dtype=np.uint32)
    meta = np.array([[0xD | (0x8 << 4) | 0x44444400]], dtype=np.uint32)
    W = orc.expand_sparse24_quant(codes, scales, zeros, meta, 4, 32, 32, 1)[:, 0]
    assert W[:8].tolist() == [0.0, 2.0, 0.0, -1.5, 0.0, 0.0, 6.0, 0.0]
    assert not W[8:].any()


def test_sparse24_quant_tracks_the_sparse_matrix():
    """The generator quantises the kept values of the seeded 2:4 matrix: same pattern, error within half a step."""
    K, N, group = 512, 32, 128
    sp, sq = gen.make_sparse24(47, K, N), gen.make_sparse24_quant(47, K, N, 4, group)
    assert np.array_equal(sp["meta"], sq["meta"])
    Ws, Wq = orc.dequant_matrix(sp), orc.dequant_matrix(sq)
    step = np.repeat(sq["scales"].astype(np.float64), group, axis=0)       # [K][N]
    assert np.all(np.abs(Ws - Wq) <= 0.5 * step * (1 + 1e-3) + 1e-12)
    assert np.all(Wq[Ws == 0] == 0)
    # group-size-K (channel-wise) and a group of 64 go through the same code
    for g in (64, K):
        Wg = orc.dequant_matrix(gen.make_sparse24_quant(47, K, N, 4, g))
        assert np.all(Wg[Ws == 0] == 0) and np.abs(Wg - Ws).max() < 0.02


# --------------------------------------------------------------------------- generator properties
@pytest.mark.parametrize("bits,group", [(4, 128), (8, 256)])
def test_rtn_quantiser_error_bound_and_idempotence(bits, group):
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((256, 16)) * 0.02).astype(np.float16)
    r = gen.rtn_quantize(x, bits, group)
    G = 256 // group
    s = r["scales"].astype(np.float64)
    deq = (r["q"].reshape(G, group, 16) - r["z"][:, None, :]) * s[:, None, :]
    err = np.abs(deq - x.astype(np.float64).reshape(G, group, 16))
    # in-range values are within half a step (+ one fp32 rounding of x/s near a tie)
    lo = (0 - r["z"]) * s; hi = (2**bits - 1 - r["z"]) * s
    xin = x.astype(np.float64).reshape(G, group, 16)
    inside = (xin >= lo[:, None, :]) & (xin <= hi[:, None, :])
    assert np.all(err[inside] <= 0.5 * np.broadcast_to(s[:, None, :], err.shape)[inside] * (1 + 1e-6))
    assert r["q"].min() >= 0 and r["q"].max() <= 2**bits - 1
    # quantising the dequantised codes again with the same grid returns the same codes
    q2 = np.clip(np.rint(deq / s[:, None, :]) + r["z"][:, None, :], 0, 2**bits - 1)
    assert np.array_equal(q2.reshape(256, 16), r["q"])


def test_generator_is_seeded_and_shaped():
    a = gen.make_backbone_quant(1, 256, 64, 3, 128); b = gen.make_backbone_quant(1, 256, 64, 3, 128)
    assert a["codes"].shape == (24, 64) and a["zeros"].shape == (2, 6) and a["scales"].shape == (2, 64)
    assert np.array_equal(a["codes"], b["codes"]) and np.array_equal(a["scales"], b["scales"])
    c = gen.make_backbone_quant(2, 256, 64, 3, 128)
    assert not np.array_equal(a["codes"], c["codes"])
    s = a["scales"].astype(np.float64)
    assert s.min() >= 0.00199 and s.max() < 0.01
    q = orc.unpack_codes(gen.make_backbone_quant(3, 4096, 64, 4, 128)["codes"], 4, 4096)
    assert abs(q.mean() - 7.5) < 0.1 and q.min() == 0 and q.max() == 15
    assert set(gen.LLAMA3_8B_SHAPES) == {"q", "k", "v", "o", "gate", "up", "down"}


def test_parity_metric():
    ref = np.array([[3.0, -4.0]])
    rel, mabs = orc.parity_errors(np.array([[3.0, -4.5]]), ref)
    assert rel == pytest.approx(0.1) and mabs == pytest.approx(0.125)
