"""GPU tests of the boundary's robustness: the bounded device-side wait running out (and the handle staying usable),
memory accounting, and handles given to the wrong entry point.  Nothing here faults or hangs a GPU: the wait that runs
out returns by itself."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import eora_oracle as orc
import eora_inputs as gen
import paper_2410_21271_b200 as eora
from helpers import make_case, run_layer, check_parity, x_to_torch


@pytest.mark.parametrize("policy", [eora.EORA_POLICY_AUTO, eora.EORA_POLICY_TMEM_DECODE])
def test_wait_that_runs_out_is_reported_and_the_handle_recovers(policy):
    import torch
    K, N, r, M = 1024, 512, 128, 3
    wf, af, bf = make_case(51, K, N, r, w="q3")
    x = gen.make_x(52, M, K)
    y_ref = orc.forward(x, "f16", wf, af, bf)
    L = eora.Layer(wf, af, bf, max_m=M, kernel_policy=policy)
    check_parity(run_layer(L, x, "f16"), y_ref, "before")
    assert eora.eora_linear_set_wait_limit(L.handle, 2000) == eora.EORA_OK            # two microseconds
    assert eora.eora_linear_selftest_wait_timeout(L.handle) == eora.EORA_OK
    torch.cuda.synchronize()                                                           # returns: the wait gave up by itself
    assert L.device_status() == eora.EORA_ERR_DEVICE_TIMEOUT
    assert L.device_status() == 0                                                      # reading it cleared it
    assert eora.eora_linear_set_wait_limit(L.handle, 0) == eora.EORA_OK               # back to the default
    # the debris the self-test left in the scratch (a partial sum, a ticket) is gone: the next forward is correct
    check_parity(run_layer(L, x, "f16"), y_ref, "after the timeout")
    check_parity(run_layer(L, x, "f16"), y_ref, "and once more")
    L.close()


def test_staging_is_allocated_by_the_first_host_call_only():
    """A handle whose activations live on the device owns its weights and a small scratch; the [max_m][d_in] +
    [max_m][d_out] staging buffers appear with the first forward_host (paper Section 4.5: the memory saving is the point)."""
    import torch
    K, N, r, M = 1024, 512, 128, 64
    wf, af, bf = make_case(53, K, N, r, w="q4")
    L = eora.Layer(wf, af, bf, max_m=M)
    assert eora.eora_linear_staging_bytes(L.handle) == 0
    scratch = eora.eora_linear_scratch_bytes(L.handle)
    # scratch: t (fp16, prefill) + sums of eight tokens + tickets, and for handles that take 17 to 64 tokens the fp32
    # sums of a launch that splits its reduction axis ([64][d_out] and [64][rank]); no staging in it
    assert scratch < M * K * 2 + 64 * (N + r) * 4 + 4096
    x = gen.make_x(54, M, K)
    xh = torch.from_numpy(x.copy()).pin_memory()
    yh = torch.empty((M, N), dtype=torch.float16).pin_memory()
    L.forward_host(xh, yh)
    assert eora.eora_linear_staging_bytes(L.handle) >= M * K * 2 + M * N * 2
    assert eora.eora_linear_scratch_bytes(L.handle) == scratch
    check_parity(yh.float().numpy().astype(np.float64), orc.forward(x, "f16", wf, af, bf), "forward_host")
    L.close()


def test_weight_bytes_of_a_llama3_8b_block():
    """Byte accounting: the re-tiled copy of a 3-bit group-128 layer with fp16 rank-128 adapters stays within 3 % of the
    algorithmic weight bytes (codes + scales + zeros + A + B)."""
    from paper_2410_21271_b200 import traffic
    K, N, r = 4096, 1024, 128
    wf = gen.make_backbone_quant(55, K, N, 3, 128)
    af, bf = gen.make_ab_f16(55, K, N, r)
    L = eora.Layer(wf, af, bf, max_m=1)
    algo = traffic.forward_bytes("q3", "f16", K, N, r, 1) - 2 * (K + N)
    assert algo <= eora.eora_linear_weight_bytes(L.handle) <= 1.03 * algo + 4096
    L.close()


def test_multi_adapter_handle_is_refused_by_the_fused_entry_points():
    import torch
    K, N, r = 512, 96, 64
    wf, af, bf = make_case(56, K, N, r)
    Lm = eora.MultiAdapterLayer(wf, [(af, bf), (af, bf)], max_m=2)
    x = torch.zeros((2, K), dtype=torch.float16, device="cuda:0")
    y = torch.zeros((2, N), dtype=torch.float16, device="cuda:0")
    assert eora.eora_linear_forward_fused(Lm.handle, x, 2, [y], check=False) == eora.EORA_ERR_UNSUPPORTED
    assert eora.eora_linear_forward(Lm.handle, x, 2, y, check=False) == eora.EORA_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    Lm.close()


def test_host_forwards_enqueued_back_to_back():
    """The enqueue-only host-buffer forwards: several layers and a fused pair on one stream, one synchronisation, every
    result against the oracle; a second round reuses the handles' staging buffers."""
    import torch
    K = 512
    cases = [make_case(60 + i, K, N, 64, w="q4") for i, N in enumerate((96, 256, 160))]
    Ls = [eora.Layer(wf, af, bf, max_m=8) for wf, af, bf in cases]
    fused = [make_case(70 + i, K, N, 64, w="q3") for i, N in enumerate((128, 64))]
    F = eora.FusedLayers(fused, max_m=8)
    for M in (1, 5):
        xs = [gen.make_x(80 + i, M, K) for i in range(4)]
        hx = [torch.from_numpy(x.copy()).pin_memory() for x in xs]
        hy = [torch.zeros((M, N), dtype=torch.float16).pin_memory() for N in (96, 256, 160)]
        hf = [torch.zeros((M, N), dtype=torch.float16).pin_memory() for N in (128, 64)]
        for L, x, y in zip(Ls, hx, hy):
            L.forward_host(x, y, sync=False)
        F.forward_host(hx[3], hf, sync=False)
        torch.cuda.synchronize()
        for (wf, af, bf), x, y in zip(cases, xs, hy):
            check_parity(y.numpy().astype(np.float64), orc.forward(x, "f16", wf, af, bf), f"enqueued M{M}")
        for (wf, af, bf), y in zip(fused, hf):
            check_parity(y.numpy().astype(np.float64), orc.forward(xs[3], "f16", wf, af, bf), f"enqueued fused M{M}")
    for L in Ls:
        assert L.device_status() == 0
        L.close()
    F.close()
