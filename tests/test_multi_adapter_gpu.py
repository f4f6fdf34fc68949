"""GPU parity of the multi-adapter entry points: one backbone, several adapters, every token names its own
(or none).  Each output row is compared with the CPU oracle's forward of that token with that adapter."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_oracle as orc
import eora_inputs as gen
import paper_2410_21271_b200 as eora
from helpers import make_case, check_parity, x_to_torch


def adapters_for(K, N, r, ab, n, seed):
    out = []
    for j in range(n):
        if ab == "f16":
            out.append(gen.make_ab_f16(seed + j, K, N, r))
        else:
            out.append(gen.make_ab_quant(seed + j, K, N, r, ab))
    return out


def reference(x, xd, wf, adapters, ids):
    rows = []
    for i, j in enumerate(ids):
        af, bf = adapters[j] if 0 <= j < len(adapters) else (None, None)
        rows.append(orc.forward(x[i:i + 1], xd, wf, af, bf)[0])
    return np.stack(rows)


CASES = [
    # w, ab, K, N, r, n_adapters, ids, x dtype
    ("q4", "f16", 256, 64, 64, 2, [0], "f16"),
    ("q4", "f16", 256, 64, 64, 2, [1], "f16"),
    ("q3", "f16", 512, 96, 128, 3, [2, 0, -1, 1, 1], "f16"),
    ("q4", "q4", 512, 160, 128, 4, [3, 3, 0, -1, 2, 1, 0, 2], "f16"),
    ("q3", "q8", 384, 96, 40, 2, [1, -1, 0], "bf16"),
    ("q4", "q3", 640, 96, 64, 3, list(range(-1, 3)) * 5, "f16"),          # 20 tokens: three passes
    ("sp24", "f16", 512, 96, 64, 2, [1, 0, 0], "f16"),
    ("sq4", "f16", 512, 96, 64, 3, [2, -1, 0, 1, 1], "f16"),
    ("q4", "f16", 256, 64, 64, 1, [0, -1], "f16"),                         # a single adapter that can be off
    ("q3", "f16", 4096, 1024, 128, 8, [7], "f16"),                         # k-shaped layer, full size
]


@pytest.mark.parametrize("w,ab,K,N,r,n,ids,xd", CASES)
def test_multi_adapter_matches_oracle(w, ab, K, N, r, n, ids, xd):
    import torch
    wf, _, _ = make_case(80, K, N, 0, w=w)
    adapters = adapters_for(K, N, r, ab, n, 81)
    M = len(ids)
    x = gen.make_x(82, M, K, xd)
    L = eora.MultiAdapterLayer(wf, adapters, max_m=M, x_dtype=xd)
    ref = reference(x, xd, wf, adapters, ids)
    for rep in range(2):                                   # second call: the scratch was restored
        y = L.forward(x_to_torch(x, xd), ids)
        torch.cuda.synchronize()
        assert L.device_status() == 0
        check_parity(y.float().cpu().numpy().astype(np.float64), ref, f"call {rep}")
    L.close()


def test_tokens_without_adapter_equal_the_plain_backbone():
    """Adapter id -1 must give exactly what a rank-0 layer gives (fp32 output, bit for bit)."""
    import torch
    K, N, r = 512, 96, 64
    wf, _, _ = make_case(83, K, N, 0, w="q4")
    adapters = adapters_for(K, N, r, "f16", 2, 84)
    x = gen.make_x(85, 2, K)
    Lm = eora.MultiAdapterLayer(wf, adapters, max_m=2, y_dtype="f32")
    L0 = eora.Layer(wf, None, None, max_m=2, y_dtype="f32")
    xt = x_to_torch(x, "f16")
    ym = Lm.forward(xt, [-1, -1]); y0 = L0.forward(xt)
    torch.cuda.synchronize()
    # the partial sums are added in a different order (atomics), so compare within fp32 rounding of the sums
    assert np.allclose(ym.cpu().numpy(), y0.cpu().numpy(), rtol=0, atol=2e-6 * np.abs(y0.cpu().numpy()).max())
    Lm.close(); L0.close()


def test_multi_adapter_argument_errors():
    import torch
    K, N, r = 256, 64, 64
    wf, _, _ = make_case(86, K, N, 0, w="q4")
    adapters = adapters_for(K, N, r, "f16", 2, 87)
    L = eora.MultiAdapterLayer(wf, adapters, max_m=4)
    x = torch.zeros((4, K), dtype=torch.float16, device="cuda:0")
    y = torch.zeros((4, N), dtype=torch.float16, device="cuda:0")
    assert eora.eora_linear_forward(L.handle, x, 1, y, check=False) == eora.EORA_ERR_UNSUPPORTED
    assert eora.eora_linear_forward_multi(L.handle, x, 5, [0] * 5, y, check=False) == eora.EORA_ERR_M_TOO_LARGE
    Lp = eora.Layer(wf, *adapters[0], max_m=4)
    assert eora.eora_linear_forward_multi(Lp.handle, x, 1, [0], y, check=False) == eora.EORA_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    L.close(); Lp.close()
