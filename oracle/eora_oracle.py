"""CPU oracle for the EoRA compensated linear layer (test infrastructure only).

This module is the slow, plain definition of what the CUDA library computes.
It is test infrastructure: only the test-suite, the smoke check and the CPU
baseline leg of the benchmark may import it.  It shares no code with the CUDA
path and never imports it.

What it computes (paper Eq. 4 / Algorithm 1 step 7, written row-vector style):

    y = X . deq(Wq) + (X . A) . B

with X [M][K], deq(Wq) [K][N], A [K][r], B [r][N]; K = d_in, N = d_out.
The paper writes the same thing column-vector style as  W^ X + B' A X  with
W^ [d][k]; the map is K = k, N = d, A_here = A_paper^T, B_here = B'_paper^T.

Storage formats (the paper only says "asymmetric", "group size 128", "2:4" and
"quantize EoRA to 4-bit" -- Section 4.1, the group-wise appendix and Section 4.5;
the bit layouts below are this library's interchange format):

* b-bit codes (b = 3 or 4) are an LSB-first bit stream along the reduction
  axis: for a fixed column n, the b-bit code of row k occupies stream bits
  [b*k, b*k + b), and 32-bit word i of the stream is ``words[i][n]``.
  For b = 4 that is "8 codes per uint32, code k%8 at bits 4*(k%8)".
  For b = 3, 32 codes fill 3 words and codes 10 and 21 of each 32 straddle
  a word boundary.
* zero-points use the same b-bit stream, but along n: ``zeros[g][i]`` is word i
  of the stream of group-row g.  The stored value is the zero-point itself.
* scales are fp16 [K/g][N].
* dequantisation: w[k][n] = (q[k][n] - z[k/g][n]) * s[k/g][n].
* 8-bit per-channel: uint8 codes [K][N], one fp16 scale and one uint8 zero per
  column n (the group spans the whole reduction axis).
* 2:4 sparse: fp16 values [N][K/2] (the two kept values of every quad of
  consecutive k, in increasing-k order) and uint32 meta [N][K/32]; quad j owns
  nibble (meta[n][j/8] >> 4*(j%8)) & 0xF = p0 | p1 << 2 with 0 <= p0 < p1 <= 3,
  and w[4j+p0][n] = values[n][2j], w[4j+p1][n] = values[n][2j+1], others 0.
* 2:4 sparse AND 4-bit (the appendix on sparsity & quantisation error compensation;
  the paper prunes to 2:4 and quantises to 4 bits without fixing a storage):
  the K/2 kept values of a column are a group-wise asymmetric 4-bit matrix
  [K/2][N] in the layout above (codes uint32 [K/16][N]); a group covers `group`
  consecutive k of the ORIGINAL axis, i.e. group/2 kept values, so scales are
  fp16 [K/group][N] and zeros [K/group][N/8]; meta as for 2:4.
  w[4j+p0][n] = (q[2j][n] - z) * s, w[4j+p1][n] = (q[2j+1][n] - z) * s, others 0.

All floating point is float64; inputs are converted exactly from their storage
types.  No blocking, no fusion: unpack, dequantise, two matrix products.
"""
from __future__ import annotations

import numpy as np


# ----------------------------------------------------------------------------
# storage-type conversions (exact)
# ----------------------------------------------------------------------------
def f16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """IEEE binary16 bit patterns (uint16) -> float64, exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return bits.view(np.float16).astype(np.float64)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float64, exactly (bf16 = top half of fp32)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def to_f64(x: np.ndarray, dtype: str) -> np.ndarray:
    """Convert a stored tensor to float64.  dtype: 'f16' (np.float16 or uint16 bits),
    'bf16' (uint16 bits), 'f32', 'f64'."""
    if dtype == "f16":
        if x.dtype == np.float16:
            return x.astype(np.float64)
        return f16_bits_to_f64(x)
    if dtype == "bf16":
        return bf16_bits_to_f64(x)
    if dtype in ("f32", "f64"):
        return np.asarray(x).astype(np.float64)
    raise ValueError(dtype)


# ----------------------------------------------------------------------------
# a1: unpack
# ----------------------------------------------------------------------------
def unpack_stream(words: np.ndarray, bits: int, count: int) -> np.ndarray:
    """Unpack `count` b-bit codes per column from an LSB-first bit stream that
    runs along axis 0 of `words` (uint32 [ceil(bits*count/32)][C]).

    Returns int64 [count][C].  Code k is stream bits [bits*k, bits*k+bits).
    """
    words = np.asarray(words)
    assert words.dtype == np.uint32 and words.ndim == 2
    assert words.shape[0] * 32 >= bits * count
    w = words.astype(np.uint64)
    out = np.empty((count, words.shape[1]), dtype=np.int64)
    mask = np.uint64((1 << bits) - 1)
    for k in range(count):
        p = bits * k
        i, off = divmod(p, 32)
        v = w[i] >> np.uint64(off)
        if off + bits > 32:                      # the code straddles words i and i+1
            v = v | (w[i + 1] << np.uint64(32 - off))
        out[k] = (v & mask).astype(np.int64)
    return out


def unpack_codes(w_codes: np.ndarray, bits: int, K: int) -> np.ndarray:
    """Backbone / adapter codes: stream along the reduction axis.  -> int64 [K][N]."""
    return unpack_stream(w_codes, bits, K)


def unpack_zeros(w_zeros: np.ndarray, bits: int, N: int) -> np.ndarray:
    """Zero-points: stream along n for every group-row.  uint32 [G][bits*N/32] -> int64 [G][N]."""
    return unpack_stream(np.ascontiguousarray(np.asarray(w_zeros).T), bits, N).T.copy()


# ----------------------------------------------------------------------------
# a2: dequantise
# ----------------------------------------------------------------------------
def dequant_groupwise(q: np.ndarray, z: np.ndarray, s_f16: np.ndarray, group: int) -> np.ndarray:
    """w[k][n] = (q[k][n] - z[k/group][n]) * s[k/group][n], float64.

    q int64 [K][N]; z int64 [K/group][N]; s_f16 fp16 (or uint16 bits) [K/group][N].
    """
    K, N = q.shape
    assert K % group == 0 and z.shape == (K // group, N) and s_f16.shape == (K // group, N)
    s = to_f64(s_f16, "f16")
    w = np.empty((K, N), dtype=np.float64)
    for g in range(K // group):
        rows = slice(g * group, (g + 1) * group)
        w[rows] = (q[rows] - z[g][None, :]).astype(np.float64) * s[g][None, :]
    return w


def dequant_matrix(fmt: dict) -> np.ndarray:
    """Dense float64 [rows][cols] matrix from any of the stored formats.

    fmt['kind'] is one of
      'f16'    : fmt['data'] fp16 [rows][cols]
      'f64'    : fmt['data'] float64 [rows][cols], used as is
      'quant'  : b-bit group-wise asymmetric: 'codes', 'scales', 'zeros', 'bits', 'group', 'rows', 'cols'
      'q8'     : 8-bit per-channel: 'codes' uint8 [rows][cols], 'scales' fp16 [cols], 'zeros' uint8 [cols]
      'sparse24': 'values' fp16 [cols][rows/2], 'meta' uint32 [cols][rows/32], 'rows', 'cols'
      'sparse24q': 2:4 + 4-bit: 'codes', 'scales', 'zeros' of the kept values ([rows/2][cols], groups of
                 group/2), 'meta' uint32 [cols][rows/32], 'bits' (4), 'group', 'rows', 'cols'
    rows is the reduction axis of the product the matrix is used in.
    """
    kind = fmt["kind"]
    if kind == "f16":
        return to_f64(fmt["data"], "f16")
    if kind == "f64":
        return np.asarray(fmt["data"], dtype=np.float64)
    if kind == "quant":
        q = unpack_codes(fmt["codes"], fmt["bits"], fmt["rows"])
        z = unpack_zeros(fmt["zeros"], fmt["bits"], fmt["cols"])
        return dequant_groupwise(q, z, fmt["scales"], fmt["group"])
    if kind == "q8":
        q = np.asarray(fmt["codes"]).astype(np.int64)
        z = np.asarray(fmt["zeros"]).astype(np.int64)
        s = to_f64(fmt["scales"], "f16")
        return (q - z[None, :]).astype(np.float64) * s[None, :]
    if kind == "sparse24":
        return expand_sparse24(fmt["values"], fmt["meta"], fmt["rows"], fmt["cols"])
    if kind == "sparse24q":
        return expand_sparse24_quant(fmt["codes"], fmt["scales"], fmt["zeros"], fmt["meta"], fmt["bits"],
                                     fmt["group"], fmt["rows"], fmt["cols"])
    raise ValueError(kind)


def deq_fp32(q: np.ndarray, z: np.ndarray, s_f16: np.ndarray, group: int) -> np.ndarray:
    """(float)(q - z) * (float)s in float32.  The product of a <=9-bit integer and an
    11-bit significand has <= 20 significant bits, so this float32 is the exact product."""
    w64 = dequant_groupwise(q, z, s_f16, group)
    w32 = w64.astype(np.float32)
    return w32


def deq_fp16(q: np.ndarray, z: np.ndarray, s_f16: np.ndarray, group: int) -> np.ndarray:
    """Round-to-nearest-even fp16 of the exact product (what a tensor-core operand holds)."""
    return dequant_groupwise(q, z, s_f16, group).astype(np.float16)


# ----------------------------------------------------------------------------
# a7: 2:4 expansion
# ----------------------------------------------------------------------------
def expand_sparse24(values: np.ndarray, meta: np.ndarray, K: int, N: int) -> np.ndarray:
    """Dense float64 [K][N] from compressed 2:4 storage (see module docstring)."""
    return scatter24(to_f64(values, "f16"), meta, K, N)


def expand_sparse24_quant(codes, scales, zeros, meta, bits: int, group: int, K: int, N: int) -> np.ndarray:
    """Dense float64 [K][N] of a backbone that is 2:4 sparse with its kept values quantised (appendix on
    sparsity & quantisation error compensation): dequantise the K/2 kept values of every column (a group
    of `group` original k holds group/2 of them), then put them where the metadata says."""
    assert group % 2 == 0 and K % group == 0
    q = unpack_codes(codes, bits, K // 2)
    z = unpack_zeros(zeros, bits, N)
    kept = dequant_groupwise(q, z, scales, group // 2)          # [K/2][N]
    return scatter24(np.ascontiguousarray(kept.T), meta, K, N)


def scatter24(vals: np.ndarray, meta: np.ndarray, K: int, N: int) -> np.ndarray:
    """vals float64 [N][K/2] (kept values in increasing-k order) -> dense [K][N] by the position nibbles."""
    meta = np.asarray(meta)
    assert vals.shape == (N, K // 2) and meta.shape == (N, K // 32) and meta.dtype == np.uint32
    w = np.zeros((K, N), dtype=np.float64)
    cols = np.arange(N)
    for j in range(K // 4):
        nib = (meta[:, j // 8] >> np.uint32(4 * (j % 8))) & np.uint32(0xF)
        p0 = (nib & np.uint32(3)).astype(np.int64)
        p1 = (nib >> np.uint32(2)).astype(np.int64)
        if not np.all(p0 < p1):
            raise ValueError("2:4 metadata must satisfy p0 < p1")
        w[4 * j + p0, cols] = vals[:, 2 * j]
        w[4 * j + p1, cols] = vals[:, 2 * j + 1]
    return w


# ----------------------------------------------------------------------------
# a3..a6: forward (paper Eq. 4)
# ----------------------------------------------------------------------------
def forward(x: np.ndarray, x_dtype: str, w_fmt: dict, a_fmt: dict | None, b_fmt: dict | None) -> np.ndarray:
    """y = X . deq(Wq) + (X . A) . B  in float64.  a_fmt/b_fmt None means rank 0.

    t = X . A is NOT rounded before it multiplies B.  The result is left in float64
    (it is not rounded to the output type)."""
    X = to_f64(x, x_dtype)
    W = dequant_matrix(w_fmt)
    y = X @ W
    if a_fmt is not None and b_fmt is not None:
        A = dequant_matrix(a_fmt)
        B = dequant_matrix(b_fmt)
        if A.shape[1] > 0:
            t = X @ A
            y = y + t @ B
    return y


def forward_at(x: np.ndarray, x_dtype: str, w_fmt: dict, a_fmt: dict | None, b_fmt: dict | None,
               m_idx: np.ndarray, n_idx: np.ndarray) -> np.ndarray:
    """The entries y[m_idx[i]][n_idx[i]] of `forward`, each computed on its own as two
    dot products -- for sampled parity at sizes where the full product is too slow."""
    X = to_f64(x, x_dtype)
    W = dequant_matrix(w_fmt)
    have_ab = a_fmt is not None and b_fmt is not None
    if have_ab:
        A = dequant_matrix(a_fmt)
        B = dequant_matrix(b_fmt)
    out = np.empty(len(m_idx), dtype=np.float64)
    for i, (m, n) in enumerate(zip(m_idx, n_idx)):
        v = float(np.dot(X[m], W[:, n]))
        if have_ab and A.shape[1] > 0:
            v += float(np.dot(X[m] @ A, B[:, n]))
        out[i] = v
    return out


# ----------------------------------------------------------------------------
# comparison rule
# ----------------------------------------------------------------------------
REL_FRO_TOL = 2e-3      # ||Y - y||_F / ||y||_F
MAX_ABS_TOL = 1e-2      # max|Y - y| / max|y|


def parity_errors(y_test: np.ndarray, y_ref: np.ndarray) -> tuple[float, float]:
    """(relative Frobenius error, max abs error / max|y_ref|), y_ref in float64 and unrounded."""
    y_test = np.asarray(y_test, dtype=np.float64)
    d = y_test - y_ref
    den = float(np.linalg.norm(y_ref))
    mx = float(np.max(np.abs(y_ref))) if y_ref.size else 0.0
    rel = float(np.linalg.norm(d)) / den if den > 0 else float(np.linalg.norm(d))
    mabs = float(np.max(np.abs(d))) / mx if mx > 0 else (float(np.max(np.abs(d))) if d.size else 0.0)
    return rel, mabs
