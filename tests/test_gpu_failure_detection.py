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


def test_a_wait_that_runs_out_in_the_persistent_multi_layer_kernel(monkeypatch):
    """The chained kernel has mbarrier waits AND a barrier over all its CTAs.  With one iteration's activation loads
    withheld in every CTA, the MMA threads' waits run out, the status word stops every other wait and grid barrier,
    the kernel returns, patdnn_check on the run's first handle reports the timeout (and clears the barrier words), and
    the same stack then runs normally.  (The kernel is opt-in: PATDNN_DEBUG=chain=1.)"""
    monkeypatch.setenv("PATDNN_DEBUG", "chain=1")
    import oracle
    import torch
    build.build_library()
    from paper_2001_00138_b200 import binding as B
    N, H, W, chans = 1, 14, 14, [256, 256, 128, 192]
    x = synth.make_layer("x", F=1, C=chans[0], N=N, H=H, W=W, seed=5, x_dist="normal").x
    cur, handles = x, []
    for i in range(3):
        L = synth.make_layer(f"t{i}", F=chans[i + 1], C=chans[i], N=N, H=H, W=W, seed=700 + i, prune=0.5, bias_std=0.2,
                             draw_input=False, w_std=float(np.sqrt(2.0 / (4 * chans[i] * 0.5))))
        handles.append(B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, relu=True, bias=L.bias, variant=B.VARIANT_DENSE_TC))
        cur = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
    stack = B.Stack(handles, [0, 0, 0])
    st = torch.cuda.current_stream().cuda_stream
    xt = torch.from_numpy(x).cuda()
    out = torch.zeros(cur.shape, device="cuda")
    B.reset_launch_count()
    stack.run(xt, out, st)
    handles[0].check()
    assert B.launch_count() == 2, "layout kernel + one persistent kernel"
    assert_close(out.cpu().numpy(), cur, TOL_F32 * 3 ** 0.5, "before the expired wait")

    handles[0].debug_wait(1024, 1)                 # the first iteration's activation tile never arrives
    stack.run(xt, out, st)
    with pytest.raises(B.PatdnnError) as e:
        handles[0].check()
    assert e.value.status == E_DEVICE_TIMEOUT
    handles[0].debug_wait(0, 0)
    out.fill_(float("nan"))
    stack.run(xt, out, st)
    for h in handles:
        h.check()
    assert_close(out.cpu().numpy(), cur, TOL_F32 * 3 ** 0.5, "after the expired wait")
    stack.free()
    for h in handles:
        h.free()

