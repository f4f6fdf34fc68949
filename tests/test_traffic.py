"""Byte / flop accounting used for the roofline numbers, pinned to the paper's model-size table
and to hand arithmetic."""
import os

import eora_inputs as gen
from paper_2410_21271_b200 import traffic

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_adapter_bytes_match_paper_model_size_table():
    shapes = gen.LLAMA3_8B_SHAPES
    assert traffic.adapter_params_per_block(shapes, 1) == 81920
    for line in open(os.path.join(GOLDEN, "model_size_adapter_overhead.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        _, base, r, bits, total = [p.strip() for p in line.split(";")]
        overhead_gb = float(total) - float(base)
        ab = "f16" if bits == "16" else "q4"
        ours = gen.LLAMA3_8B_BLOCKS * sum(traffic.adapter_bytes(ab, K, N, int(r)) for K, N in shapes.values())
        lo, hi = ours / 2**30, ours / 1e9           # GiB and GB readings
        assert lo - 0.03 <= overhead_gb <= hi + 0.03, (line, lo, hi)


def test_forward_bytes_hand_arithmetic():
    # 4096 x 4096, 4-bit g128, fp16 r=128, M=1: codes 8,388,608 + 32 groups x 4096 x (2 + 0.5)
    # + A/B 2*128*8192 + X, Y 2*(4096+4096)
    assert traffic.forward_bytes("q4", "f16", 4096, 4096, 128, 1) == 8388608 + 327680 + 2097152 + 16384
    assert traffic.forward_bytes("q3", "f16", 4096, 4096, 0, 1) == 6291456 + 32 * 4096 * 2 + 32 * 4096 * 3 // 8 + 16384
    assert traffic.backbone_bytes("sp24", 4096, 4096) == 4096 * 2048 * 2 + 4096 * 1024 // 2
    # 2:4 + 4-bit: half a byte per kept value, half a byte of positions per quad, scale + zero per group of 128 k
    assert traffic.backbone_bytes("sq4", 4096, 4096) == 4096 * 2048 // 2 + 4096 * 1024 // 2 + 32 * 4096 * 2 + 32 * 4096 // 2
    assert traffic.matrix_bytes("q8", 4096, 128) == 4096 * 128 + 3 * 128
    assert traffic.forward_flops(4096, 4096, 128, 2048) == 2 * 2048 * (4096 * 4096 + 128 * 8192)
