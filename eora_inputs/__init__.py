"""Seeded synthetic inputs for the EoRA compensated linear layer.

Shared by the CPU oracle's tests and the CUDA parity tests / benchmark: it only
makes data (random codes, scales, zero-points, activations, adapters and their
round-to-nearest quantised forms, 2:4 patterns) in the library's interchange
layout.  It holds none of the forward arithmetic and imports neither the oracle
nor the CUDA package.

Recipe (LLaMA3-8B-shaped linear layers stand in for the paper's GPTQ / SparseGPT
compressed LLaMA weights, which need the real checkpoints):
  backbone codes  : uniform b-bit codes  -> uniformly random packed words
  zero-points     : uniform b-bit codes  -> uniformly random packed words
  scales          : fp16(0.002 + |N(0, sigma=1e-3)|)
  A [K][r], B [r][N] : fp16(N(0, 0.02^2))
  X [M][K]        : fp16 or bf16 of N(0, 1)
  quantised A/B   : round-to-nearest asymmetric from the fp16 matrices (see rtn_quantize)
  2:4 backbone    : per quad of 4 consecutive k two random positions, values fp16(N(0, 0.02^2))
"""
from __future__ import annotations

import numpy as np

# (d_in, d_out) of the seven linear layers of one LLaMA3-8B block
LLAMA3_8B_SHAPES = {
    "q": (4096, 4096),
    "k": (4096, 1024),
    "v": (4096, 1024),
    "o": (4096, 4096),
    "gate": (4096, 14336),
    "up": (4096, 14336),
    "down": (14336, 4096),
}
LLAMA3_8B_BLOCKS = 32

BASE_SEED = 0x241021271


def _rng(seed: int, *tags: int) -> np.random.Generator:
    return np.random.default_rng([BASE_SEED, int(seed), *[int(t) for t in tags]])


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    return r.astype(np.uint16)


def pack_stream(codes: np.ndarray, bits: int) -> np.ndarray:
    """Pack integer codes [count][C] into an LSB-first bit stream along axis 0:
    uint32 [bits*count/32][C]; code k occupies stream bits [bits*k, bits*k+bits)."""
    codes = np.asarray(codes)
    count, C = codes.shape
    assert (bits * count) % 32 == 0
    assert codes.min(initial=0) >= 0 and codes.max(initial=0) < (1 << bits)
    acc = np.zeros((bits * count // 32, C), dtype=np.uint64)
    c64 = codes.astype(np.uint64)
    for k in range(count):
        i, off = divmod(bits * k, 32)
        acc[i] |= (c64[k] << np.uint64(off)) & np.uint64(0xFFFFFFFF)
        if off + bits > 32:
            acc[i + 1] |= c64[k] >> np.uint64(32 - off)
    return acc.astype(np.uint32)


def make_x(seed: int, M: int, K: int, dtype: str = "f16") -> np.ndarray:
    """Activations ~ N(0,1).  'f16' -> np.float16 [M][K]; 'bf16' -> uint16 bit patterns [M][K]."""
    x = _rng(seed, 1).standard_normal((M, K), dtype=np.float32)
    if dtype == "f16":
        return x.astype(np.float16)
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)


def make_scales(rng: np.random.Generator, shape) -> np.ndarray:
    return (0.002 + np.abs(rng.standard_normal(shape, dtype=np.float32)) * 1e-3).astype(np.float16)


def make_backbone_quant(seed: int, K: int, N: int, bits: int, group: int = 128) -> dict:
    """Group-wise asymmetric b-bit backbone in the interchange layout."""
    assert bits in (3, 4) and K % group == 0 and (bits * K) % 32 == 0 and (bits * N) % 32 == 0
    rng = _rng(seed, 2, bits)
    codes = rng.integers(0, 2**32, size=(bits * K // 32, N), dtype=np.uint32)
    zeros = rng.integers(0, 2**32, size=(K // group, bits * N // 32), dtype=np.uint32)
    scales = make_scales(rng, (K // group, N))
    return {"kind": "quant", "bits": bits, "group": group, "rows": K, "cols": N,
            "codes": codes, "scales": scales, "zeros": zeros}


def make_ab_f16(seed: int, K: int, N: int, r: int) -> tuple[dict, dict]:
    """fp16 adapter: A [K][r], B [r][N], entries N(0, 0.02^2)."""
    rng = _rng(seed, 3)
    A = (rng.standard_normal((K, r), dtype=np.float32) * 0.02).astype(np.float16)
    B = (rng.standard_normal((r, N), dtype=np.float32) * 0.02).astype(np.float16)
    return {"kind": "f16", "data": A}, {"kind": "f16", "data": B}


def rtn_quantize(mat: np.ndarray, bits: int, group: int) -> dict:
    """Round-to-nearest asymmetric quantisation of a fp16 matrix [rows][cols] with groups of
    `group` consecutive rows (the reduction axis) per column.

    Per group G: lo = min(0, min G), hi = max(0, max G), s = fp16((hi - lo) / (2^b - 1)) (1 if 0),
    z = clamp(rint(-lo / s), 0, 2^b - 1), q = clamp(rint(x / s) + z, 0, 2^b - 1); rint is
    round-half-even; float32 arithmetic with the rounded s.
    Returns {'q': int codes [rows][cols], 'scales': fp16 [rows/group][cols], 'z': int [rows/group][cols]}.
    """
    x = np.asarray(mat, dtype=np.float16).astype(np.float32)
    rows, cols = x.shape
    assert rows % group == 0
    G = rows // group
    xg = x.reshape(G, group, cols)
    lo = np.minimum(xg.min(axis=1), 0.0).astype(np.float32)
    hi = np.maximum(xg.max(axis=1), 0.0).astype(np.float32)
    qmax = np.float32(2**bits - 1)
    s = ((hi - lo) / qmax).astype(np.float16)
    s = np.where(s.astype(np.float32) == 0.0, np.float16(1.0), s).astype(np.float16)
    s32 = s.astype(np.float32)
    z = np.clip(np.rint(-lo / s32), 0, qmax).astype(np.float32)
    q = np.clip(np.rint(xg / s32[:, None, :]) + z[:, None, :], 0, qmax)
    return {"q": q.reshape(rows, cols).astype(np.int64), "scales": s, "z": z.astype(np.int64)}


def quantize_matrix_bits(mat: np.ndarray, bits: int, group: int) -> dict:
    """fp16 [rows][cols] -> b-bit (3 or 4) group-wise interchange format (groups along rows)."""
    rows, cols = mat.shape
    g = min(group, rows)
    r = rtn_quantize(mat, bits, g)
    return {"kind": "quant", "bits": bits, "group": g, "rows": rows, "cols": cols,
            "codes": pack_stream(r["q"], bits), "scales": r["scales"],
            "zeros": np.ascontiguousarray(pack_stream(np.ascontiguousarray(r["z"].T), bits).T)}


def quantize_matrix_4bit(mat: np.ndarray, group: int) -> dict:
    return quantize_matrix_bits(mat, 4, group)


def quantize_matrix_8bit(mat: np.ndarray) -> dict:
    """fp16 [rows][cols] -> 8-bit per-channel format: one (scale, zero) per column."""
    rows, cols = mat.shape
    r = rtn_quantize(mat, 8, rows)
    return {"kind": "q8", "rows": rows, "cols": cols, "codes": r["q"].astype(np.uint8),
            "scales": r["scales"].reshape(cols), "zeros": r["z"].reshape(cols).astype(np.uint8)}


def make_ab_quant(seed: int, K: int, N: int, r: int, ab_format: str, group: int = 128) -> tuple[dict, dict]:
    """Quantised adapter derived from the seeded fp16 one.  ab_format: 'q4', 'q3' (group-wise) or 'q8'."""
    a16, b16 = make_ab_f16(seed, K, N, r)
    if ab_format == "q4":
        return quantize_matrix_4bit(a16["data"], group), quantize_matrix_4bit(b16["data"], group)
    if ab_format == "q3":
        return quantize_matrix_bits(a16["data"], 3, group), quantize_matrix_bits(b16["data"], 3, group)
    if ab_format == "q8":
        return quantize_matrix_8bit(a16["data"]), quantize_matrix_8bit(b16["data"])
    raise ValueError(ab_format)


def make_sparse24(seed: int, K: int, N: int) -> dict:
    """2:4 structured-sparse fp16 backbone: compressed values [N][K/2] + 2-bit positions."""
    assert K % 32 == 0
    rng = _rng(seed, 4)
    values = (rng.standard_normal((N, K // 2), dtype=np.float32) * 0.02).astype(np.float16)
    # the six (p0 < p1) position pairs of a quad, as nibbles p0 | p1 << 2
    pairs = np.array([0 | 1 << 2, 0 | 2 << 2, 0 | 3 << 2, 1 | 2 << 2, 1 | 3 << 2, 2 | 3 << 2], dtype=np.uint32)
    nib = pairs[rng.integers(0, 6, size=(N, K // 4))]
    nib = nib.reshape(N, K // 32, 8)
    meta = np.zeros((N, K // 32), dtype=np.uint32)
    for i in range(8):
        meta |= nib[:, :, i] << np.uint32(4 * i)
    return {"kind": "sparse24", "rows": K, "cols": N, "values": values, "meta": meta}


def make_sparse24_quant(seed: int, K: int, N: int, bits: int = 4, group: int = 128) -> dict:
    """2:4 structured-sparse backbone whose kept values are quantised group-wise: the seeded 2:4 matrix,
    its [K/2][N] kept values rounded to `bits` with groups of `group` original k (group/2 kept values)."""
    sp = make_sparse24(seed, K, N)
    g = min(group, K)
    assert g % 2 == 0 and K % g == 0
    kept = np.ascontiguousarray(sp["values"].T)                 # [K/2][N]
    qz = quantize_matrix_bits(kept, bits, g // 2)
    return {"kind": "sparse24q", "rows": K, "cols": N, "bits": bits, "group": g, "codes": qz["codes"],
            "scales": qz["scales"], "zeros": qz["zeros"], "meta": sp["meta"]}


# ----------------------------------------------------------------------------
# inputs of the offline solve (Algorithm 1): a weight, its compressed version and calibration activations
# ----------------------------------------------------------------------------
def make_solve_case(seed: int, d: int, k: int, n: int, bits: int = 3, kind: str = "rtn", rank_signal: int = 0):
    """W [d][k] ~ N(0, 0.02^2); W^ = W rounded to a per-row uniform grid of 2^bits levels (a stand-in for the
    compressed checkpoint: the error is bounded, zero-mean noise like that of a round-to-nearest quantiser);
    X~ [k][n]: Gaussian columns with log-normal per-channel scales and a few strong channels, the shape of LLM
    activations (the paper's calibration activations need the real model).  kind == "gap": the error is a rank
    `rank_signal` matrix plus noise 100 times smaller, so the top singular subspace of the projected error is
    well separated (for element-wise comparisons)."""
    rng = _rng(seed, 0x501E, d, k, n)
    w = (rng.standard_normal((d, k)) * 0.02).astype(np.float32)
    if kind == "gap":
        u = rng.standard_normal((d, rank_signal)); v = rng.standard_normal((rank_signal, k))
        s = np.geomspace(1.0, 0.2, rank_signal)
        dw = (u * s[None, :]) @ v / np.sqrt(d * k) + rng.standard_normal((d, k)) * 1e-5
        w_hat = (w.astype(np.float64) - dw).astype(np.float32)
    else:
        amax = np.abs(w).max(axis=1, keepdims=True)
        step = 2.0 * amax / (2 ** bits - 1)
        w_hat = (np.round(w / step) * step).astype(np.float32)
    scale = np.exp(rng.standard_normal(k) * 0.8)
    strong = rng.choice(k, size=max(1, k // 64), replace=False)
    scale[strong] *= 12.0
    x = (rng.standard_normal((k, n)) * scale[:, None]).astype(np.float32)
    return w, w_hat, x
