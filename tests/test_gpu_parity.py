"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs."""
import os

import numpy as np
import pytest

from paper_2001_00138_b200 import build, synth
from util import TOL_F16, TOL_F32, assert_close, chain_tol, gpu_layer, oracle_layer

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build_library()
    from paper_2001_00138_b200 import binding
    binding.load()
    return binding


VARIANTS = {"auto": 0, "noopt": 1, "reorder": 2, "tiled": 3, "dense": 4, "prun": 5}


@pytest.mark.parametrize("variant", ["tiled", "dense", "reorder", "noopt", "prun"])
def test_config1(variant):
    L = synth.config1()
    got, plan = gpu_layer(L, variant=VARIANTS[variant])
    assert plan["variant"] == VARIANTS[variant]
    assert_close(got, oracle_layer(L), TOL_F32, f"config1/{variant}")


# (N, C, F, H, W, n_patterns, prune): ragged tails in every dimension, widths that are not multiples of 4 or 2,
# single rows/columns, batches that straddle a warp's tile range, more filters than one CTA holds.
ODD_SHAPES = [
    (2, 3, 5, 5, 5, 8, 0.0), (1, 4, 20, 7, 7, 8, 0.3), (3, 8, 33, 14, 14, 12, 0.5), (2, 16, 64, 9, 13, 8, 0.6),
    (1, 5, 7, 1, 1, 4, 0.0), (1, 6, 40, 2, 30, 6, 0.2), (5, 9, 17, 3, 4, 8, 0.4), (2, 20, 130, 16, 16, 8, 0.7),
    (1, 3, 16, 40, 36, 8, 0.0), (4, 12, 24, 6, 10, 12, 0.9), (1, 33, 70, 18, 66, 8, 0.5), (7, 2, 3, 4, 8, 8, 0.0),
    (1, 1000, 1000, 7, 7, 8, 0.8), (2, 100, 300, 15, 17, 12, 0.6),      # channel counts beyond any tile, not multiples of 64
]


@pytest.mark.parametrize("shape", ODD_SHAPES)
@pytest.mark.parametrize("variant", ["tiled", "dense", "reorder", "prun"])
def test_odd_shapes(shape, variant):
    N, C, F, H, W, npat, prune = shape
    L = synth.make_layer("odd", F=F, C=C, N=N, H=H, W=W, seed=hash(shape) % 10000, n_patterns=npat, prune=prune,
                         bias_std=0.2, x_dist="normal", relu=(F % 2 == 1))
    if variant == "prun" and C > 600:
        # the pattern-run kernel keeps all channels of a 9 x 9 patch in shared memory (C <= ~630): asked for by name on a
        # wider layer it is refused when the layer is encoded, not at run time
        from paper_2001_00138_b200 import binding as B
        with pytest.raises(B.PatdnnError) as e:
            B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, variant=VARIANTS["prun"])
        assert e.value.status == 2
        return
    got, _ = gpu_layer(L, variant=VARIANTS[variant])
    assert_close(got, oracle_layer(L), TOL_F32, f"{shape}/{variant}")


def test_noopt_matches_on_pruned_layer():
    L = synth.make_layer("n", F=24, C=18, N=2, H=11, W=9, seed=31, prune=0.5, bias_std=0.1)
    got, _ = gpu_layer(L, variant=VARIANTS["noopt"])
    assert_close(got, oracle_layer(L), TOL_F32, "noopt")


def test_empty_filters_and_caller_order():
    L = synth.make_layer("e", F=40, C=12, N=2, H=10, W=12, seed=77, prune=0.5, bias_std=0.5)
    L.mask[3] = 0
    L.mask[17] = 0
    ref = oracle_layer(L)
    for variant in ("tiled", "dense", "reorder", "prun"):
        got, _ = gpu_layer(L, variant=VARIANTS[variant])
        assert_close(got, ref, TOL_F32, variant)
        assert np.all(got[:, 3] == max(L.bias[3], 0.0))
        got, _ = gpu_layer(L, variant=VARIANTS[variant], order=synth.random_filter_order(40, 5))
        assert_close(got, ref, TOL_F32, variant + "/random order")


def test_output_is_fully_written_and_input_untouched():
    import torch
    from paper_2001_00138_b200 import binding as B
    L = synth.make_layer("w", F=19, C=7, N=3, H=13, W=10, seed=8, prune=0.4)
    layer = B.encode(L.weights, L.mask, L.patterns, N=3, H=13, W=10, relu=True, bias=L.bias)
    x = torch.from_numpy(L.x).cuda()
    x0 = x.clone()
    canary = torch.full((3 * 19 * 13 * 10 + 64,), -7.0, device="cuda")
    out = canary[32:-32].view(3, 19, 13, 10)
    layer.conv(x, out, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert torch.equal(x, x0)
    assert torch.all(canary[:32] == -7.0) and torch.all(canary[-32:] == -7.0)
    assert torch.all(out >= 0)
    layer.free()


def test_config2_full_size():
    L = synth.config2()
    ref = oracle_layer(L)
    got, plan = gpu_layer(L)
    assert plan["variant"] in (3, 4)
    assert_close(got, ref, TOL_F32, "config2")
    for variant in ("tiled", "dense"):
        got, plan = gpu_layer(L, variant=VARIANTS[variant])
        assert plan["variant"] == VARIANTS[variant]
        assert_close(got, ref, TOL_F32, "config2/" + variant)
    got, _ = gpu_layer(L, via_host=True)
    assert_close(got, ref, TOL_F32, "config2 via host buffers")


@pytest.mark.parametrize("i", range(4))
@pytest.mark.parametrize("N", [1, 3, 32])
def test_resnet_shapes_fp16(i, N):
    """The four ResNet-50-shaped fp16 layers at batch 1, a ragged batch and the full batch of 32, whole output."""
    L = synth.resnet50_layer(i, N=N)
    ref = oracle_layer(L)
    for variant in ("auto", "tiled", "dense", "reorder", "prun"):
        if N == 32 and variant == "reorder":
            continue                      # the generic kernel adds nothing at full batch
        if variant == "tiled" and L.W % 2:
            continue                      # odd-width fp16 rows are not 4-byte aligned: no tiled kernel for them
        got, _ = gpu_layer(L, variant=VARIANTS[variant])
        assert_close(got, ref, TOL_F16, f"resnet {i} N={N} {variant}")


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("shape", [(4, 3, 64, 64, 64), (6, 4, 96, 40, 72), (10, 7, 64, 33, 50), (3, 1, 130, 71, 90)])
def test_small_channel_layers_gather_their_operand_in_the_kernel(shape, dtype):
    """9*C <= 64 on the persistent tensor-core kernel: one launch per call (no gathered tensor is written first), image
    borders, ragged tiles and the zero tail of the 64-deep operand rows included."""
    import torch
    from paper_2001_00138_b200 import binding as B
    N, C, F, H, W = shape
    L = synth.make_layer("g", F=F, C=C, N=N, H=H, W=W, seed=4242 + C, n_patterns=8, prune=0.2 if C > 1 else 0.0,
                         bias_std=0.3, x_dist="normal", dtype=dtype)
    B.reset_launch_count()
    got, plan = gpu_layer(L, variant=VARIANTS["dense"])
    assert plan["variant"] == VARIANTS["dense"]
    assert B.launch_count() == 1
    assert_close(got, oracle_layer(L), TOL_F16 if dtype == "f16" else TOL_F32, f"gather {shape} {dtype}")


@pytest.mark.parametrize("generated", [True, False])
@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("shape", [(3, 3, 64, 13, 9), (2, 1, 40, 32, 32), (1, 4, 64, 7, 50), (5, 2, 17, 6, 6)])
def test_few_channel_first_layer_writes_the_next_layers_operands(shape, dtype, generated, monkeypatch):
    """CUDA-core layer with C <= 4 and F <= 64 followed by a tensor-core layer: the stack runs ONE kernel for the first
    layer that writes the second layer's split operands (no NCHW tensor, no layout kernel), then the GEMM.  Both forms of
    that kernel: the code generated for the layer at run time (kept weights as immediates) and the static one."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    N, C, F, H, W = shape
    if not generated:
        monkeypatch.setenv("PATDNN_DEBUG", "jit=0")
    dt = B.F16 if dtype == "f16" else B.F32
    tdt = torch.float16 if dtype == "f16" else torch.float32
    L0 = synth.make_layer("f0", F=F, C=C, N=N, H=H, W=W, seed=77 + C, prune=0.0, bias_std=0.3, x_dist="normal", dtype=dtype)
    L1 = synth.make_layer("f1", F=48, C=F, N=N, H=H, W=W, seed=78 + C, prune=0.5, bias_std=0.3, draw_input=False, dtype=dtype,
                          w_std=0.2)
    h0 = B.encode(L0.weights, L0.mask, L0.patterns, N=N, H=H, W=W, dtype=dt, relu=True, bias=L0.bias, variant=VARIANTS["reorder"])
    h1 = B.encode(L1.weights, L1.mask, L1.patterns, N=N, H=H, W=W, dtype=dt, relu=False, bias=L1.bias, variant=VARIANTS["dense"])
    mid = oracle.conv3x3(L0.x, L0.weights, L0.mask, L0.bias, True)
    if dtype == "f16":
        mid = mid.astype(np.float16).astype(np.float32)          # the layer boundary stores fp16
    ref = oracle.conv3x3(mid, L1.weights, L1.mask, L1.bias, False)
    stack = B.Stack([h0, h1], [0, 0])
    assert stack.generated() == (1 if generated else 0), "the generated kernel must be the one that runs (no silent fallback)"
    out = torch.empty((N, 48, H, W), device="cuda", dtype=tdt)
    B.reset_launch_count()
    stack.run(torch.from_numpy(L0.x).to("cuda", dtype=tdt), out, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert B.launch_count() == 2
    assert_close(out.float().cpu().numpy(), ref, chain_tol(2, TOL_F16 if dtype == "f16" else TOL_F32),
                 f"fused first layer {shape} {dtype}")
    stack.free()
    h0.free()
    h1.free()


@pytest.mark.parametrize("npat,prune", [(4, 0.0), (6, 0.5), (8, 0.75), (12, 0.9)])
def test_sweep_points_reduced_batch(npat, prune):
    L = synth.sweep_layer(npat, prune, N=3)
    ref = oracle_layer(L)
    for variant in ("auto", "tiled", "dense", "prun"):
        got, _ = gpu_layer(L, variant=VARIANTS[variant])
        assert_close(got, ref, TOL_F32, f"sweep p{npat} prune{prune} {variant}")
    got, _ = gpu_layer(L, order=synth.random_filter_order(512, 1))
    assert_close(got, ref, TOL_F32, f"sweep p{npat} prune{prune} random filter order")


@pytest.mark.parametrize("npat,prune", [(4, 0.9), (6, 0.75), (8, 0.0), (12, 0.5), (8, 0.9)])
def test_sweep_points_full_batch(npat, prune):
    """Sweep points at the full batch of 64 (the launch configuration the sweep is timed in), whole output, with the
    filter reorder and with a seeded random filter order."""
    L = synth.sweep_layer(npat, prune, N=64)
    ref = oracle_layer(L)
    for variant in ("auto", "tiled", "prun"):
        got, plan = gpu_layer(L, variant=VARIANTS[variant])
        assert_close(got, ref, TOL_F32, f"sweep N=64 p{npat} prune{prune} {variant}")
    assert plan["variant"] == VARIANTS["prun"] and plan["entries"] >= L.K, "lane entries = kept kernels + padding"
    got, _ = gpu_layer(L, order=synth.random_filter_order(512, 7))
    assert_close(got, ref, TOL_F32, f"sweep N=64 p{npat} prune{prune} random filter order")


@pytest.mark.parametrize("scale,N", [(4, 2), (7, 5)])
def test_vgg_stack_reduced_spatial_per_layer_and_chained(scale, N):
    """All 13 layers at 1/4 spatial size (56x56 input) and at 1/7 (the 32x32 input of the CIFAR-sized network, down to
    2x2 images): each GPU layer is fed the oracle's input for that layer (binding check), and the chained GPU stack is
    compared with the chained oracle."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    x = synth.vgg16_input(N, scale)
    layers, handles = [], []
    cur = x
    for i in range(13):
        L = synth.vgg16_layer(i, N=N, spatial_scale=scale)
        ref = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
        got, _ = gpu_layer(L, x=cur)
        assert_close(got, ref, TOL_F32, f"vgg layer {i + 1}")
        cur = oracle.maxpool2x2(ref) if i in synth.VGG16_POOL_AFTER else ref
        layers.append(L)
        handles.append(B.encode(L.weights, L.mask, L.patterns, N=N, H=L.H, W=L.W, relu=True, bias=L.bias))
    pools = [1 if i in synth.VGG16_POOL_AFTER else 0 for i in range(13)]
    stack = B.Stack(handles, pools)
    assert stack.out_shape() == cur.shape
    xt = torch.from_numpy(x).cuda()
    out = torch.empty(cur.shape, device="cuda")
    stack.run(xt, out, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert_close(out.cpu().numpy(), cur, chain_tol(13, TOL_F32), "vgg chained")
    out_h = np.empty(cur.shape, dtype=np.float32)
    stack.run_host(x, out_h)
    # same kernels, and the cluster reduction of K-split partial tiles adds in rank order: the same bits
    assert np.array_equal(out_h, out.cpu().numpy()), "vgg chained through host buffers"
    stack.free()
    for h in handles:
        h.free()


@pytest.mark.parametrize("variants", [("dense", "dense", "dense"), ("tiled", "dense", "tiled"), ("dense", "tiled", "dense"),
                                      ("reorder", "dense", "dense")])
@pytest.mark.parametrize("hw", [(7, 7), (13, 9), (6, 10), (5, 7)])
def test_small_stack_with_odd_sizes_and_pools(variants, hw):
    """Three chained layers with a pool after the first two, on extents that are odd before and after pooling, with
    every hand-over between the kernel families (NCHW <-> channels-innermost split operands, pooled or not)."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    N, (H, W) = 3, hw
    chans = [5, 70, 24, 9]
    x = synth.make_layer("x", F=1, C=chans[0], N=N, H=H, W=W, seed=5, x_dist="normal").x
    cur, handles, h, w = x, [], H, W
    for i in range(3):
        L = synth.make_layer(f"s{i}", F=chans[i + 1], C=chans[i], N=N, H=h, W=w, seed=900 + i, prune=0.4, bias_std=0.3,
                             draw_input=False)
        handles.append(B.encode(L.weights, L.mask, L.patterns, N=N, H=h, W=w, relu=True, bias=L.bias,
                                variant=VARIANTS[variants[i]]))
        cur = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
        if i < 2 and h >= 2 and w >= 2:
            cur = oracle.maxpool2x2(cur)
            h, w = h // 2, w // 2
    pools = [1 if (i < 2) else 0 for i in range(3)]
    assert cur.shape[2:] == (h, w) and h >= 1 and w >= 1
    stack = B.Stack(handles, pools)
    assert stack.out_shape() == cur.shape
    out = torch.empty(cur.shape, device="cuda")
    B.reset_launch_count()
    stack.run(torch.from_numpy(x).cuda(), out, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    if variants == ("dense", "dense", "dense"):
        # three GEMMs, both pools taken in their epilogues; the first layer (9*C <= 64) either gathers its operand rows
        # from the caller's NCHW input itself or has one layout kernel in front
        assert B.launch_count() in (3, 4)
    assert_close(out.cpu().numpy(), cur, chain_tol(3, TOL_F32), f"stack {variants} {hw}")
    stack.free()
    for hd in handles:
        hd.free()


@pytest.mark.parametrize("i,N", [(0, 32), (1, 32), (2, 32), (5, 32), (8, 32), (12, 32), (3, 1), (8, 1), (11, 1)])
def test_vgg_full_size_standalone(i, N):
    """Full-size layers called alone (NCHW in, NCHW out) in the benchmark's launch configuration; the whole output is
    compared with the oracle."""
    import torch
    from paper_2001_00138_b200 import binding as B
    L = synth.vgg16_layer(i, N=N)
    rng = np.random.Generator(np.random.PCG64(900 + i))
    x = rng.random((N, L.C, L.H, L.W), dtype=np.float32)
    layer = B.encode(L.weights, L.mask, L.patterns, N=N, H=L.H, W=L.W, relu=True, bias=L.bias)
    xt = torch.from_numpy(x).cuda()
    out = torch.full((N, L.F, L.H, L.W), float("nan"), device="cuda")
    layer.conv(xt, out, torch.cuda.current_stream().cuda_stream)
    layer.check()
    got = out.cpu().numpy()
    if i == 0:
        assert layer.plan()["generated"] == 1, "the RGB layer under AUTO runs code generated for it"
    if (i, N) in ((5, 32), (8, 32)):
        assert layer.plan()["grid_z"] > 1, "these tile counts are not whole rounds of CTAs: a tail launch is planned"
    layer.free()
    assert_close(got, oracle_layer(L, x=x), TOL_F32, f"vgg L{i + 1} N={N}")


@pytest.mark.parametrize("variant,dtype", [("auto", "f16"), ("tiled", "f16"), ("prun", "f16"), ("auto", "f32")])
def test_batch_holding_more_than_two_to_the_31_elements(variant, dtype):
    """64 -> 64 @ 128x128 at batch 2112: input and output hold 2.2e9 elements each, so every offset that includes the
    image index needs 64 bits.  The first and last images and those on both sides of the 2^32-byte and 2^31-element
    boundaries (images 1024 and 2048) are compared whole with the oracle."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    N, C, F, H, W = 2112, 64, 64, 128, 128
    if torch.cuda.mem_get_info()[0] < 40e9:
        pytest.skip("needs ~30 GB of free device memory")
    L = synth.make_layer("big", F=F, C=C, N=1, H=H, W=W, seed=4242, prune=0.5, dtype=dtype, bias_std=0.1, draw_input=False)
    tdt = torch.float16 if dtype == "f16" else torch.float32
    xt = torch.rand((N, C, H, W), device="cuda", dtype=tdt, generator=torch.Generator(device="cuda").manual_seed(11))
    out = torch.full((N, F, H, W), float("nan"), device="cuda", dtype=tdt)
    layer = B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, dtype=B.F16 if dtype == "f16" else B.F32, relu=True,
                     bias=L.bias, variant=VARIANTS[variant])
    try:
        layer.conv(xt, out, torch.cuda.current_stream().cuda_stream)
        layer.check()
        if variant != "auto":
            assert layer.plan()["variant"] == VARIANTS[variant]
    finally:
        layer.free()
    sel = [0, 1, 1023, 1024, 2047, 2048, N - 2, N - 1]
    assert bool(torch.isfinite(out[::97]).all())
    ref = oracle.conv3x3(xt[sel].float().cpu().numpy(), L.weights, L.mask, L.bias, True)
    assert_close(out[sel].float().cpu().numpy(), ref, TOL_F16 if dtype == "f16" else TOL_F32, f"big batch {variant}/{dtype}")


@pytest.mark.parametrize("ks", [1, 2, 4, 8])
def test_tensor_core_path_with_cluster_split_of_the_channel_loop(ks, monkeypatch):
    """Small batches split the (channel block, tap) loop over the CTAs of a cluster and sum through distributed shared
    memory; every split factor must give the same layer."""
    monkeypatch.setenv("PATDNN_DEBUG", f"ksplit={ks}")
    L = synth.make_layer("ks", F=192, C=160, N=1, H=20, W=24, seed=900 + ks, prune=0.6, bias_std=0.1, x_dist="normal")
    got, plan = gpu_layer(L, variant=VARIANTS["dense"])
    assert plan["variant"] == 4
    assert_close(got, oracle_layer(L), TOL_F32, f"cluster split {ks}")
    Lh = synth.resnet50_layer(1, N=2)
    got, _ = gpu_layer(Lh, variant=VARIANTS["dense"])
    assert_close(got, oracle_layer(Lh), TOL_F16, f"cluster split {ks}, fp16")


def test_maxpool_matches_oracle():
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    x = np.random.Generator(np.random.PCG64(6)).standard_normal((3, 5, 14, 10)).astype(np.float32)
    xt = torch.from_numpy(x).cuda()
    out = torch.empty((3, 5, 7, 5), device="cuda")
    B.maxpool2x2(xt, out, 3, 5, 14, 10, B.F32, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), oracle.maxpool2x2(x))


def test_pipelined_host_entry_point_matches_the_blocking_one():
    """submit_host/wait_host over a stream of different batches: every result equals run_host's for that batch, with two
    batches in flight; a third submission without a wait is refused."""
    import torch
    from paper_2001_00138_b200 import binding as B
    N, H, W = 2, 20, 24
    chans = [3, 64, 32]
    handles = []
    for i in range(2):
        L = synth.make_layer(f"p{i}", F=chans[i + 1], C=chans[i], N=N, H=H, W=W, seed=40 + i, prune=0.3 * i, bias_std=0.2,
                             draw_input=False, w_std=0.3)
        handles.append(B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, relu=True, bias=L.bias))
    stack = B.Stack(handles, [0, 1])
    rng = np.random.Generator(np.random.PCG64(5))
    xs = [torch.from_numpy(rng.standard_normal((N, 3, H, W)).astype(np.float32)).pin_memory() for _ in range(5)]
    ref = []
    for x in xs:
        o = np.empty(stack.out_shape(), dtype=np.float32)
        stack.run_host(x.numpy(), o)
        ref.append(o)
    outs = [torch.empty(stack.out_shape(), dtype=torch.float32).pin_memory() for _ in xs]
    s = torch.cuda.current_stream().cuda_stream
    stack.submit_host(xs[0].numpy(), outs[0].numpy(), s)
    stack.submit_host(xs[1].numpy(), outs[1].numpy(), s)
    with pytest.raises(B.PatdnnError):
        stack.submit_host(xs[2].numpy(), outs[2].numpy(), s)
    for i in range(2, 5):
        stack.wait_host()
        stack.submit_host(xs[i].numpy(), outs[i].numpy(), s)
    stack.wait_host()
    stack.wait_host()
    stack.wait_host()                                       # nothing outstanding: returns at once
    for o, r in zip(outs, ref):
        assert np.array_equal(o.numpy(), r)
    stack.free()
    for h in handles:
        h.free()


@pytest.mark.parametrize("hw", [(24, 24), (14, 10)])
def test_fp16_stack_with_pools(hw):
    """fp16 storage end to end: four layers, two pools; the oracle chain rounds every layer boundary to fp16 like the
    stored activations (a pool commutes with that rounding)."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    N, (H, W) = 3, hw
    chans = [3, 64, 64, 96, 40]
    pools = [0, 1, 1, 0]
    x = synth.make_layer("x", F=1, C=3, N=N, H=H, W=W, seed=9, x_dist="normal", dtype="f16").x
    cur, handles, h, w = x.astype(np.float32), [], H, W
    for i in range(4):
        L = synth.make_layer(f"h{i}", F=chans[i + 1], C=chans[i], N=N, H=h, W=w, seed=300 + i, prune=0.0 if i == 0 else 0.5,
                             bias_std=0.2, draw_input=False, dtype="f16", w_std=float(np.sqrt(2.0 / (4 * chans[i] * 0.6))))
        handles.append(B.encode(L.weights, L.mask, L.patterns, N=N, H=h, W=w, dtype=B.F16, relu=True, bias=L.bias))
        cur = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
        if pools[i]:
            cur = oracle.maxpool2x2(cur)
            h, w = h // 2, w // 2
        if i < 3:
            cur = cur.astype(np.float16).astype(np.float32)
    stack = B.Stack(handles, pools)
    assert stack.out_shape() == cur.shape
    out = torch.empty(cur.shape, device="cuda", dtype=torch.float16)
    stack.run(torch.from_numpy(x).to("cuda", dtype=torch.float16), out, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for hd in handles:
        hd.check()
    assert_close(out.float().cpu().numpy(), cur, chain_tol(4, TOL_F16), f"fp16 stack {hw}")
    stack.free()
    for hd in handles:
        hd.free()


def test_empty_batch_is_a_no_op():
    import torch
    from paper_2001_00138_b200 import binding as B
    L = synth.make_layer("z", F=16, C=8, N=1, H=6, W=6, seed=3, draw_input=False)
    for variant in ("auto", "dense", "tiled", "reorder", "prun"):
        h = B.encode(L.weights, L.mask, L.patterns, N=0, H=6, W=6, relu=True, bias=L.bias, variant=VARIANTS[variant])
        x = torch.empty((0, 8, 6, 6), device="cuda")
        y = torch.empty((0, 16, 6, 6), device="cuda")
        h.conv(x, y, torch.cuda.current_stream().cuda_stream)
        h.check()
        h.free()


@pytest.mark.parametrize("shape", [(20, 96, 256, 56, 56), (37, 64, 300, 28, 28), (41, 128, 512, 16, 16)])
def test_cta_pair_kernel(shape, monkeypatch):
    """The opt-in cta_group::2 kernel (two CTAs per 256-pixel x 256-filter tile, each loading half of the weights): same
    layer as the default kernels, odd pixel-tile counts and padded filter tiles included."""
    import torch
    from paper_2001_00138_b200 import binding as B
    monkeypatch.setenv("PATDNN_DEBUG", "pair=1")
    N, C, F, H, W = shape
    L = synth.make_layer("pair", F=F, C=C, N=N, H=H, W=W, seed=N + F, prune=0.6, bias_std=0.2, draw_input=False,
                         w_std=float(np.sqrt(2.0 / (4 * C * 0.4))))
    rng = np.random.Generator(np.random.PCG64(N))
    x = rng.random((N, C, H, W), dtype=np.float32)
    layer = B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, relu=True, bias=L.bias, variant=VARIANTS["dense"])
    plan = layer.plan()
    assert plan["grid_x"] == 148 and plan["grid_y"] > 148          # 74 clusters of two CTAs
    out = torch.full((N, F, H, W), float("nan"), device="cuda")
    layer.conv(torch.from_numpy(x).cuda(), out, torch.cuda.current_stream().cuda_stream)
    layer.check()
    got = out.cpu().numpy()
    import oracle
    assert_close(got, oracle.conv3x3(x, L.weights, L.mask, L.bias, True), TOL_F32, f"CTA-pair kernel {shape}")
    layer.free()


def _fuzz_cases(n, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    cases = []
    for _ in range(n):
        N = int(rng.choice([1, 1, 2, 3, 5, 9, 17, 40]))
        C = int(rng.choice([1, 2, 3, 4, 7, 8, 16, 31, 64, 65, 100, 130, 200]))
        F = int(rng.choice([1, 3, 8, 16, 33, 64, 65, 100, 128, 129, 200, 260]))
        H = int(rng.integers(1, 41))
        W = int(rng.integers(1, 41))
        cases.append((N, C, F, H, W, str(rng.choice(["f32", "f16"])), float(rng.choice([0.0, 0.3, 0.7])), bool(rng.integers(2)),
                      9000 + len(cases)))
    return cases


@pytest.mark.parametrize("case", _fuzz_cases(36, 2024))
def test_random_layers_all_planner_paths(case):
    """Seeded random shapes through the planner (AUTO) and the tensor-core variant: whatever kernel, box, split, tail or
    gather the plan picks, the layer equals the oracle."""
    N, C, F, H, W, dtype, prune, relu, seed = case
    if N * F * H * W * C > 3e8:
        N = 1
    L = synth.make_layer("fz", F=F, C=C, N=N, H=H, W=W, seed=seed, n_patterns=8, prune=prune, bias_std=0.2,
                         x_dist="normal", dtype=dtype, relu=relu)
    ref = oracle_layer(L)
    tol = TOL_F16 if dtype == "f16" else TOL_F32
    for variant in ("auto", "dense", "prun"):
        got, _ = gpu_layer(L, variant=VARIANTS[variant])
        assert_close(got, ref, tol, f"{case}/{variant}")


@pytest.mark.parametrize("seed", range(10))
def test_random_stacks(seed):
    """Seeded random three- and four-layer stacks (channel counts, extents, pools, variants): every hand-over between the
    kernel families and every fused pool/first-layer path the stack chooses must reproduce the chained oracle."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    rng = np.random.Generator(np.random.PCG64(7000 + seed))
    nl = int(rng.integers(3, 5))
    N = int(rng.choice([1, 2, 4, 9]))
    H, W = int(rng.integers(8, 41)), int(rng.integers(8, 41))
    chans = [int(rng.choice([1, 3, 4, 16, 40]))] + [int(rng.choice([16, 64, 64, 96, 130])) for _ in range(nl)]
    pools = [int(rng.integers(2)) for _ in range(nl)]
    x = rng.standard_normal((N, chans[0], H, W)).astype(np.float32)
    cur, handles, h, w = x, [], H, W
    for i in range(nl):
        if pools[i] and (h < 2 or w < 2):
            pools[i] = 0
        L = synth.make_layer(f"rs{i}", F=chans[i + 1], C=chans[i], N=N, H=h, W=w, seed=8000 + 10 * seed + i,
                             prune=0.0 if i == 0 else 0.5, bias_std=0.2, draw_input=False,
                             w_std=float(np.sqrt(2.0 / (4 * chans[i] * (1.0 if i == 0 else 0.5)))))
        variant = VARIANTS[str(rng.choice(["auto", "auto", "dense", "reorder"]))]
        handles.append(B.encode(L.weights, L.mask, L.patterns, N=N, H=h, W=w, relu=True, bias=L.bias, variant=variant))
        cur = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
        if pools[i]:
            cur = oracle.maxpool2x2(cur)
            h, w = h // 2, w // 2
    stack = B.Stack(handles, pools)
    assert stack.out_shape() == cur.shape
    out = torch.empty(cur.shape, device="cuda")
    stack.run(torch.from_numpy(x).cuda(), out, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for hd in handles:
        hd.check()
    assert_close(out.cpu().numpy(), cur, chain_tol(nl, TOL_F32), f"random stack {seed}: {chans} pools {pools} {H}x{W} N={N}")
    stack.free()
    for hd in handles:
        hd.free()


@pytest.mark.parametrize("C,prune", [(1, 0.0), (3, 0.75), (5, 0.8), (7, 0.9)])
def test_auto_keeps_few_channel_fp32_layers_exact_whatever_the_pattern_set(C, prune):
    """Few input channels, heavy pruning and a pattern set outside the tiled kernel's built-in table: with one or two
    products per output the hi/lo split of the tensor-core path would sit at the edge of 1e-4, so AUTO must keep such
    fp32 layers on an FP32 kernel (here the generic FKW kernel), and the result must hold the tolerance."""
    rng = np.random.Generator(np.random.PCG64(4000 + C))
    pats = np.asarray([0b000101011, 0b110100010, 0b011000101, 0b101010001], dtype=np.uint16)   # four 4-of-9 masks, none built in
    assert all(bin(int(m)).count("1") == 4 for m in pats) and not set(int(m) for m in pats) & set(synth.PATTERN_MASKS)
    N, F, H, W = 2, 48, 19, 23
    w = rng.standard_normal((F, C, 3, 3)).astype(np.float32) * 3.0
    pid = rng.integers(0, len(pats), size=(F, C)).astype(np.int32)
    pid[rng.random((F, C)) < prune] = -1
    mask = synth.mask_from_pid(pid, pats)
    bias = (rng.standard_normal(F) * 0.2).astype(np.float32)
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    layer = B.encode(w, mask, pats, N=N, H=H, W=W, relu=False, bias=bias)
    assert layer.plan()["variant"] in (VARIANTS["reorder"], VARIANTS["tiled"]), "not the tensor-core variant"
    out = torch.full((N, F, H, W), float("nan"), device="cuda")
    layer.conv(torch.from_numpy(x).cuda(), out, torch.cuda.current_stream().cuda_stream)
    layer.check()
    layer.free()
    assert_close(out.cpu().numpy(), oracle.conv3x3(x, w, mask, bias, False), TOL_F32, f"AUTO, C={C}, prune={prune}")

