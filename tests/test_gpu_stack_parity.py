"""Parity of the code paths that exist only inside a stack, and of the benchmark's own configuration.

Inside a stack a layer does not write an NCHW tensor: its epilogue writes the next tensor-core layer's split,
channels-innermost operands (after the 2x2 maximum where a pool follows), and a few-channel first layer runs as one
FP32 kernel that does the same.  To hold those paths to the single-layer tolerance, a layer is followed by an
identity layer (one kept kernel per filter on its own channel, centre weight 1): the stack's output then equals the
first layer's (pooled) output up to the operand split (2^-16 relative), so it can be compared with the oracle's
result for that ONE layer at 1e-4 (fp32) / 2e-3 (fp16).
"""
import numpy as np
import pytest

from paper_2001_00138_b200 import build, synth
from util import TOL_F16, TOL_F32, assert_close, chain_tol, identity_layer

pytestmark = pytest.mark.gpu

DENSE = 4


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build_library()
    from paper_2001_00138_b200 import binding
    binding.load()
    return binding


def _run_with_identity(L, x, pool, variant=0, dtype="f32"):
    """Stack [L, identity] (pool after L if asked); returns (output as float32 numpy, launches, plan of L)."""
    import torch
    from paper_2001_00138_b200 import binding as B
    N, C, H, W = x.shape
    dt = B.F16 if dtype == "f16" else B.F32
    tdt = torch.float16 if dtype == "f16" else torch.float32
    h0 = B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, dtype=dt, relu=L.relu, bias=L.bias, variant=variant)
    h2, w2 = (H // 2, W // 2) if pool else (H, W)
    wi, mi, pi = identity_layer(L.F)
    h1 = B.encode(wi, mi, pi, N=N, H=h2, W=w2, dtype=dt, relu=False, variant=DENSE)
    stack = B.Stack([h0, h1], [1 if pool else 0, 0])
    assert stack.out_shape() == (N, L.F, h2, w2)
    out = torch.full((N, L.F, h2, w2), float("nan"), device="cuda", dtype=tdt)
    B.reset_launch_count()
    stack.run(torch.from_numpy(x).to("cuda", dtype=tdt), out, torch.cuda.current_stream().cuda_stream)
    h0.check()
    h1.check()
    launches = B.launch_count()
    plan = h0.plan()
    got = out.float().cpu().numpy()
    stack.free()
    h0.free()
    h1.free()
    return got, launches, plan


def _oracle_one_layer(L, x, pool):
    import oracle
    ref = oracle.conv3x3(x, L.weights, L.mask, L.bias, L.relu)
    return oracle.maxpool2x2(ref) if pool else ref


@pytest.mark.parametrize("N", [32, 1])
@pytest.mark.parametrize("i", range(13))
def test_every_benchmark_layer_in_its_in_stack_form(i, N):
    """Each layer of the VGG-shaped benchmark stack, at full size and at both benchmark batch sizes, planned and
    launched as the stack launches it (operands written for a tensor-core successor, pool fused where the stack fuses
    it, K-split tail launches, cluster splits, the generated first-layer kernel), checked in full against the oracle
    at the single-layer tolerance."""
    L = synth.vgg16_layer(i, N=N)
    pool = i in synth.VGG16_POOL_AFTER
    if i == 0:
        x = synth.vgg16_input(N)
    else:
        x = np.random.Generator(np.random.PCG64(900 + i)).random((N, L.C, L.H, L.W), dtype=np.float32)
    got, launches, plan = _run_with_identity(L, x, pool)
    if i == 0:
        assert plan["variant"] != DENSE and launches == 2, "first layer: one FP32 kernel that writes the operands, then the GEMM"
    else:
        assert plan["variant"] == DENSE
        # no layout kernel and no pooling kernel behind the first layer: its GEMM (plus a K-split tail launch where
        # the plan has one) and the identity's GEMM (ditto) -- or one persistent kernel for both at batch 1; the only
        # layout kernel is the one in front of the stack
        assert launches <= 1 + 2 + 2
    assert_close(got, _oracle_one_layer(L, x, pool), TOL_F32, f"vgg L{i + 1} N={N} in-stack")


# (N, C, F, H, W, pool, dtype, variant of the first layer, prune)
IN_STACK_CASES = [
    (3, 5, 70, 13, 9, True, "f32", 4, 0.4),        # gathered operand (9*C <= 64), odd extents, pooled epilogue
    (3, 5, 70, 13, 9, False, "f32", 4, 0.4),
    (2, 70, 24, 6, 10, True, "f32", 4, 0.4),
    (4, 96, 130, 20, 24, True, "f32", 4, 0.6),     # filter tiles padded beyond the successor's channels
    (1, 160, 192, 20, 24, False, "f32", 4, 0.6),   # small grid: cluster split of the channel loop
    (1, 160, 192, 20, 24, True, "f32", 4, 0.6),
    (9, 64, 64, 40, 40, True, "f32", 4, 0.5),      # persistent kernel, pooled boxes
    (9, 64, 64, 40, 40, False, "f32", 4, 0.5),
    (3, 64, 96, 24, 24, True, "f16", 4, 0.5),
    (3, 64, 96, 14, 10, False, "f16", 4, 0.5),
    (2, 128, 128, 28, 28, True, "f16", 4, 0.7),
    (5, 3, 64, 33, 50, False, "f32", 0, 0.0),      # few-channel first layer under AUTO: FP32 kernel writing the operands
    (5, 3, 64, 33, 50, False, "f16", 0, 0.0),
    (2, 4, 40, 7, 50, False, "f32", 2, 0.2),
    (3, 16, 64, 12, 12, True, "f32", 3, 0.3),      # CUDA-core layer in front: NCHW hand-over through the layout kernel
    (3, 16, 64, 12, 12, False, "f32", 2, 0.3),
]


# the run-time generated kernel only exists for few-channel first layers (C <= 4): those cases also run with the
# static kernel in its place
IN_STACK_RUNS = [(case, True) for case in IN_STACK_CASES] + [(case, False) for case in IN_STACK_CASES if case[1] <= 4]


@pytest.mark.parametrize("chained", [True, False])
@pytest.mark.parametrize("case,generated", IN_STACK_RUNS)
def test_in_stack_paths_at_the_single_layer_tolerance(case, generated, chained, monkeypatch):
    """chained = False: one kernel per layer, epilogues that write the successor's operands (the default);
    chained = True: the stack may run consecutive small tensor-core layers as one persistent kernel (opt-in)."""
    N, C, F, H, W, pool, dtype, variant, prune = case
    opts = ["chain=1"] if chained else []
    if not generated:
        opts.append("jit=0")
    if opts:
        monkeypatch.setenv("PATDNN_DEBUG", ",".join(opts))
    L = synth.make_layer("in_stack", F=F, C=C, N=N, H=H, W=W, seed=1234 + C + F, prune=prune, bias_std=0.3,
                         x_dist="normal", dtype=dtype, w_std=float(np.sqrt(2.0 / (4 * C * (1 - prune)))))
    got, _, _ = _run_with_identity(L, L.x, pool, variant=variant, dtype=dtype)
    ref = _oracle_one_layer(L, L.x, pool)
    assert_close(got, ref, TOL_F16 if dtype == "f16" else TOL_F32, f"in-stack {case}")


@pytest.mark.parametrize("N", [32, 1])
def test_benchmark_stack_whole_images_against_the_chained_oracle(N):
    """The object bench.py times: the 13-layer stack at 224x224, built the same way, run once through
    patdnn_stack_run; the whole output of the first and the last image is compared with the oracle chained over
    those images alone.  The chain allowance is sqrt(13) single-layer allowances (see util.chain_tol)."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    layers = [synth.vgg16_layer(i, N=N) for i in range(13)]
    handles = [B.encode(L.weights, L.mask, L.patterns, N=N, H=L.H, W=L.W, relu=True, bias=L.bias) for L in layers]
    pools = [1 if i in synth.VGG16_POOL_AFTER else 0 for i in range(13)]
    stack = B.Stack(handles, pools)
    assert stack.generated() == 1, "the RGB layer runs the code generated for it, as in the benchmark"
    x = synth.vgg16_input(N)
    out = torch.full(stack.out_shape(), float("nan"), device="cuda")
    stack.run(torch.from_numpy(x).cuda(), out, torch.cuda.current_stream().cuda_stream)
    for h in handles:
        h.check()
    got = out.cpu().numpy()
    assert np.all(np.isfinite(got))
    # the same call through host buffers: same kernels, same order of every sum, so the same bits
    out_h = np.empty(stack.out_shape(), dtype=np.float32)
    stack.run_host(x, out_h)
    assert np.array_equal(out_h, got)
    imgs = sorted({0, N - 1})
    cur = np.ascontiguousarray(x[imgs])
    for i, L in enumerate(layers):
        cur = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
        if pools[i]:
            cur = oracle.maxpool2x2(cur)
    worst = assert_close(got[imgs], cur, chain_tol(13, TOL_F32), f"benchmark stack N={N}, images {imgs}")
    print(f"benchmark stack N={N}: worst |gpu - oracle| / (1e-4 * max(|o|, rms)) over images {imgs} = "
          f"{worst * chain_tol(13, TOL_F32) / TOL_F32:.2f} (allowed {chain_tol(13, TOL_F32) / TOL_F32:.2f})")
    stack.free()
    for h in handles:
        h.free()


# chains of tensor-core layers small enough for the persistent multi-layer kernel
# (N, H, W, channels per layer boundary, pool flags, dtype)
CHAIN_CASES = [
    (1, 28, 28, [64, 128, 128, 256, 192], [0, 1, 0, 0], "f32"),
    (1, 14, 14, [512, 512, 512, 512], [0, 0, 0], "f32"),
    (2, 20, 24, [96, 130, 70, 64], [1, 0, 1], "f32"),          # ragged filter tiles and channel blocks, two pools
    (3, 12, 16, [64, 64, 200, 40, 64, 96], [0, 1, 0, 0, 1], "f32"),
    (1, 56, 56, [128, 256, 256], [0, 1], "f32"),                # 28 pixel tiles x 2 filter tiles per layer
    (2, 14, 10, [64, 96, 128, 40], [0, 1, 0], "f16"),
    (1, 24, 24, [64, 64, 64, 96, 40], [1, 1, 0, 0], "f16"),
    (5, 9, 7, [70, 33, 129, 64], [0, 0, 0], "f32"),             # odd extents (no pool), several images per tile
]


@pytest.mark.parametrize("case", CHAIN_CASES)
def test_chained_layers_in_one_persistent_kernel(case, monkeypatch):
    """Runs of small tensor-core layers: after the layout kernel in front, the whole run is ONE launch; the result must
    equal the chained oracle and the host-buffer call must give the same bits."""
    import oracle
    import torch
    from paper_2001_00138_b200 import binding as B
    monkeypatch.setenv("PATDNN_DEBUG", "chain=1")               # the persistent multi-layer kernel is opt-in
    N, H, W, chans, pools, dtype = case
    dt = B.F16 if dtype == "f16" else B.F32
    tdt = torch.float16 if dtype == "f16" else torch.float32
    tol = TOL_F16 if dtype == "f16" else TOL_F32
    nl = len(chans) - 1
    x = synth.make_layer("x", F=1, C=chans[0], N=N, H=H, W=W, seed=77, x_dist="normal", dtype=dtype).x
    cur, handles, h, w = x.astype(np.float32), [], H, W
    for i in range(nl):
        L = synth.make_layer(f"ch{i}", F=chans[i + 1], C=chans[i], N=N, H=h, W=w, seed=600 + i, prune=0.5, bias_std=0.2,
                             draw_input=False, dtype=dtype, w_std=float(np.sqrt(2.0 / (4 * chans[i] * 0.5))))
        handles.append(B.encode(L.weights, L.mask, L.patterns, N=N, H=h, W=w, dtype=dt, relu=True, bias=L.bias, variant=DENSE))
        cur = oracle.conv3x3(cur, L.weights, L.mask, L.bias, True)
        if pools[i]:
            cur = oracle.maxpool2x2(cur)
            h, w = h // 2, w // 2
        if dtype == "f16" and i < nl - 1:
            cur = cur.astype(np.float16).astype(np.float32)       # the layer boundary stores fp16
    stack = B.Stack(handles, pools)
    assert stack.out_shape() == cur.shape
    out = torch.full(cur.shape, float("nan"), device="cuda", dtype=tdt)
    B.reset_launch_count()
    stack.run(torch.from_numpy(x).to("cuda", dtype=tdt), out, torch.cuda.current_stream().cuda_stream)
    for hd in handles:
        hd.check()
    assert B.launch_count() == 2, "one layout kernel, then one persistent kernel for the whole run"
    got = out.float().cpu().numpy()
    assert_close(got, cur, chain_tol(nl, tol), f"chained run {case}")
    out_h = np.empty(cur.shape, dtype=np.float16 if dtype == "f16" else np.float32)
    stack.run_host(np.ascontiguousarray(x.astype(out_h.dtype)), out_h)
    assert np.array_equal(out_h.astype(np.float32), got)
    stack.free()
    for hd in handles:
        hd.free()

