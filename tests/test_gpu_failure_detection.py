"""The library's failure detection on the device: every wait inside the tensor-core kernels is bounded, and a wait
that runs out ends the kernel through its normal exit with a status word that patdnn_check reports.

Nothing here faults, traps or hangs the GPU: the test shortens the bound to about a millisecond and asks the producer
warp (patdnn_debug_wait) to leave out the loads of one iteration, so the consumer's wait for them simply runs out.
"""
import numpy as np
import pytest

from paper_2001_00138_b200 import build, synth
from util import TOL_F32, assert_close, oracle_layer

pytestmark = pytest.mark.gpu

E_DEVICE_TIMEOUT = 8


@pytest.mark.parametrize("ks", [1, 4])
def test_a_wait_that_runs_out_is_reported_and_the_handle_keeps_working(ks, monkeypatch):
    import torch
    build.build_library()
    from paper_2001_00138_b200 import binding as B
    # one-tile-per-CTA kernel, alone (ks = 1) and as clusters of four that split the channel/tap loop
    monkeypatch.setenv("PATDNN_DEBUG", f"ksplit={ks},halo=0,tail=0")
    L = synth.make_layer("timeout", F=192, C=160, N=1, H=20, W=24, seed=77 + ks, prune=0.6, bias_std=0.1, x_dist="normal")
    layer = B.encode(L.weights, L.mask, L.patterns, N=1, H=20, W=24, relu=True, bias=L.bias, variant=B.VARIANT_DENSE_TC)
    plan = layer.plan()
    assert plan["channel_splits"] == ks and plan["grid_y"] == 1 and plan["grid_z"] == 1
    st = torch.cuda.current_stream().cuda_stream
    x = torch.from_numpy(L.x).cuda()
    out = torch.zeros((1, 192, 20, 24), device="cuda")
    ref = oracle_layer(L)

    layer.conv(x, out, st)
    layer.check()
    assert_close(out.cpu().numpy(), ref, TOL_F32, "before the expired wait")

    layer.debug_wait(1024, 3)                      # ~1 ms per wait; the loads of the third iteration never arrive
    layer.conv(x, out, st)
    with pytest.raises(B.PatdnnError) as e:
        layer.check()
    assert e.value.status == E_DEVICE_TIMEOUT
    layer.check()                                  # the report cleared the status word

    layer.debug_wait(0, 0)                         # back to normal: same handle, same buffers
    out.fill_(float("nan"))
    layer.conv(x, out, st)
    layer.check()
    assert_close(out.cpu().numpy(), ref, TOL_F32, "after the expired wait")
    layer.free()
