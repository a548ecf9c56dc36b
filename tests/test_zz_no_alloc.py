"""The allocation-free entry point (patdnn_conv_static) must give what patdnn_conv gives.

It exists for callers that cannot allocate device memory while they run a layer (a loop that replays captured work,
a plug-in living inside another program's memory pool, a process whose allocator is frozen after start-up): the
scratch of the tensor-core path then comes from a fixed 16 MiB device array inside the library instead of a buffer
owned by the handle.  This file is collected last on purpose, so that a failure here cannot hide other results.
"""
import numpy as np
import pytest

from paper_2001_00138_b200 import build, synth
from util import TOL_F16, TOL_F32, assert_close, oracle_layer

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


def test_handles_of_different_layouts_share_the_array_and_nothing_is_allocated():
    """Four handles with different channel padding, image size, storage type and kernel (one tile per CTA; persistent
    kernel with a K-split tail launch) take turns on the one array: each result must equal the oracle whatever the
    previous call left behind -- in particular the zero padding of the channels 80..127 after a call that filled them --
    and the amount of free device memory must not move while they run."""
    import torch
    build.build_library()
    from paper_2001_00138_b200 import binding as B
    st = torch.cuda.current_stream().cuda_stream
    specs = [  # (F, C, N, H, W, dtype)
        (64, 128, 2, 28, 28, "f32"),       # every channel of the 128-wide rows is written with data
        (96, 80, 2, 28, 28, "f32"),        # channels 80..127 are padding and must read as zero
        (128, 100, 3, 14, 14, "f16"),      # one operand plane, several images per tile
        (128, 64, 2, 112, 112, "f32"),     # 196 tiles: persistent kernel plus a K-split tail launch, 6.4 MB of the array
    ]
    cases = []
    for i, (F, C, N, H, W, dtype) in enumerate(specs):
        L = synth.make_layer(f"share{i}", F=F, C=C, N=N, H=H, W=W, seed=500 + i, prune=0.5, bias_std=0.1, x_dist="normal",
                             dtype=dtype, w_std=float(np.sqrt(2.0 / (4 * C * 0.5))))
        h = B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, relu=True, bias=L.bias,
                     dtype=B.F16 if dtype == "f16" else B.F32, variant=B.VARIANT_DENSE_TC)
        tdt = torch.float16 if dtype == "f16" else torch.float32
        x = torch.from_numpy(L.x).to("cuda", dtype=tdt)
        out = torch.empty((N, F, H, W), device="cuda", dtype=tdt)
        cases.append((L, h, x, out, oracle_layer(L), TOL_F16 if dtype == "f16" else TOL_F32))
    assert cases[3][1].plan()["grid_z"] > 1, "the 112x112 layer is planned with a tail launch"
    for _, h, x, out, _, _ in cases:               # first calls: address look-up, tensor maps, module loading
        h.conv_static(x, out, st)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for order in ([0, 1, 2, 3], [3, 1, 0, 2, 1]):
        for i in order:
            L, h, x, out, ref, tol = cases[i]
            out.fill_(float("nan"))
            h.conv_static(x, out, st)
            h.check()
            assert_close(out.float().cpu().numpy(), ref, tol, f"handle {i} after order {order}")
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "patdnn_conv_static must not allocate or free device memory"
    for _, h, _, _, _, _ in cases:
        h.free()


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
