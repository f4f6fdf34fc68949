"""Algorithmic bytes and flops of the compensated linear layer (host-side accounting only).

"Algorithmic" = what Eq. 4 must move / compute given the storage formats, independent of how a
kernel tiles it: every weight byte once, X once, Y once.
"""
from __future__ import annotations


def matrix_bytes(kind: str, rows: int, cols: int, *, bits: int = 4, group: int = 128) -> int:
    """Bytes of a stored [rows (reduction)][cols] matrix.
    kind: 'f16' | 'quant' (b-bit codes + fp16 scale + b-bit zero per group and column)
          | 'q8' (uint8 codes + fp16 scale + uint8 zero per column) | 'sparse24' (fp16 values for half
          the entries + 2 bits of position per kept value) | 'sparse24q' (b-bit codes for half the entries
          + 2 bits of position per kept value + fp16 scale and b-bit zero per group of `group` original rows)."""
    if kind == "f16":
        return 2 * rows * cols
    if kind == "quant":
        g = min(group, rows)
        groups = rows // g
        return rows * cols * bits // 8 + groups * cols * 2 + groups * cols * bits // 8
    if kind == "q8":
        return rows * cols + cols * 2 + cols
    if kind == "sparse24":
        return (rows // 2) * cols * 2 + (rows // 4) * cols * 4 // 8
    if kind == "sparse24q":
        g = min(group, rows)
        groups = rows // g
        return (rows // 2) * cols * bits // 8 + (rows // 4) * cols * 4 // 8 + groups * cols * 2 + groups * cols * bits // 8
    raise ValueError(kind)


def adapter_bytes(ab: str, K: int, N: int, r: int, group: int = 128) -> int:
    """Bytes of A [K][r] plus B [r][N].  ab: 'f16' | 'q4' | 'q3' | 'q8'."""
    if r == 0:
        return 0
    if ab == "f16":
        return matrix_bytes("f16", K, r) + matrix_bytes("f16", r, N)
    if ab in ("q4", "q3"):
        b = 4 if ab == "q4" else 3
        return matrix_bytes("quant", K, r, bits=b, group=group) + matrix_bytes("quant", r, N, bits=b, group=group)
    if ab == "q8":
        return matrix_bytes("q8", K, r) + matrix_bytes("q8", r, N)
    raise ValueError(ab)


def backbone_bytes(w: str, K: int, N: int, group: int = 128) -> int:
    """w: 'q4' | 'q3' | 'sp24' | 'sq4' (2:4 with 4-bit kept values)."""
    if w == "q4":
        return matrix_bytes("quant", K, N, bits=4, group=group)
    if w == "q3":
        return matrix_bytes("quant", K, N, bits=3, group=group)
    if w == "sp24":
        return matrix_bytes("sparse24", K, N)
    if w == "sq4":
        return matrix_bytes("sparse24q", K, N, bits=4, group=group)
    raise ValueError(w)


def forward_bytes(w: str, ab: str, K: int, N: int, r: int, M: int, *, group: int = 128, y_bytes: int = 2) -> int:
    """Algorithmic bytes of one forward: weights + adapter + X (fp16/bf16) + Y."""
    return backbone_bytes(w, K, N, group) + adapter_bytes(ab, K, N, r, group) + 2 * M * K + y_bytes * M * N


def forward_flops(K: int, N: int, r: int, M: int) -> int:
    """2*M*(K*N + r*(K+N)): the dense contraction and the two thin products; dequantisation is not credited."""
    return 2 * M * (K * N + r * (K + N))


def adapter_params_per_block(shapes: dict, r: int) -> int:
    """Adapter parameters of one transformer block: sum over its linear layers of r*(K+N)."""
    return sum(r * (K + N) for (K, N) in shapes.values())
