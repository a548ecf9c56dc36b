"""The allocation-free entry point (patdnn_conv_static) must give what patdnn_conv gives.

It exists for callers that cannot allocate device memory while they run a layer (a loop that replays captured work,
a plug-in living inside another program's memory pool, a process whose allocator is frozen after start-up): the
scratch of the tensor-core path then comes from a fixed 16 MiB device array inside the library instead of a buffer
owned by the handle.  This file is collected last on purpose, so that a failure here cannot hide other results.
"""
import numpy as np
import pytest

from paper_2001_00138_b200 import build, synth
from util import TOL_F32, assert_close, oracle_layer

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_the_allocating_one_twice_in_a_row():
    import torch
    build.build_library()
    from paper_2001_00138_b200 import binding as B
    L = synth.make_layer("noalloc", F=96, C=80, N=2, H=28, W=28, seed=4242, prune=0.5, bias_std=0.1, x_dist="normal")
    layer = B.encode(L.weights, L.mask, L.patterns, N=2, H=28, W=28, relu=True, bias=L.bias,
                     variant=B.VARIANT_DENSE_TC)
    st = torch.cuda.current_stream().cuda_stream
    ref = oracle_layer(L)
    x = torch.from_numpy(L.x).cuda()
    base = torch.empty((2, 96, 28, 28), device="cuda")
    layer.conv(x, base, st)
    layer.check()
    assert_close(base.cpu().numpy(), ref, TOL_F32, "patdnn_conv")
    # two calls in a row through the C ABI, the second on a different input: the shared array keeps the first call's
    # contents, and the second call must not be disturbed by them
    x2 = torch.from_numpy(np.ascontiguousarray(L.x[::-1])).cuda()
    ref2 = oracle_layer(L, x=np.ascontiguousarray(L.x[::-1]))
    out1 = torch.full_like(base, float("nan"))
    out2 = torch.full_like(base, float("nan"))
    layer.conv_static(x, out1, st)
    layer.conv_static(x2, out2, st)
    layer.check()
    assert_close(out1.cpu().numpy(), base.cpu().numpy(), TOL_F32, "patdnn_conv_static, first call")
    assert_close(out2.cpu().numpy(), ref2, TOL_F32, "patdnn_conv_static, second call")
    layer.free()


def test_static_scratch_entry_point_refuses_layers_beyond_its_limit_and_forwards_cuda_core_layers():
    import torch
    from paper_2001_00138_b200 import binding as B
    st = torch.cuda.current_stream().cuda_stream
    big = synth.make_layer("big", F=32, C=64, N=5, H=128, W=128, seed=1, prune=0.5, draw_input=False)   # 20 MiB of scratch
    layer = B.encode(big.weights, big.mask, big.patterns, N=5, H=128, W=128, variant=B.VARIANT_DENSE_TC)
    x = torch.zeros((5, 64, 128, 128), device="cuda")
    out = torch.empty((5, 32, 128, 128), device="cuda")
    with pytest.raises(B.PatdnnError) as e:
        layer.conv_static(x, out, st)
    assert e.value.status == 12
    layer.free()
    L = synth.config1()
    layer = B.encode(L.weights, L.mask, L.patterns, N=1, H=32, W=32, bias=L.bias, variant=B.VARIANT_TILED)
    x = torch.from_numpy(L.x).cuda()
    out = torch.empty((1, 32, 32, 32), device="cuda")
    layer.conv_static(x, out, st)
    layer.check()
    assert_close(out.cpu().numpy(), oracle_layer(L), TOL_F32, "tiled layer through patdnn_conv_static")
    layer.free()
