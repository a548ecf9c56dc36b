"""Host logic of the library, run without a GPU: the C ABI loads and exports what the header declares, and the
encoder's FKW arrays equal the reference statement bit for bit."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import fkw_ref
from paper_2001_00138_b200 import build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    build.build_library()
    from paper_2001_00138_b200 import binding
    binding.load()
    return binding


def test_library_exports_every_declared_symbol(B):
    header = open(os.path.join(ROOT, "include", "patdnn.h")).read()
    declared = set(re.findall(r"PATDNN_API[^;(]*?\b(patdnn_\w+)\s*\(", header))
    assert declared == set(B.EXPORTED_SYMBOLS)
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert "sm_100a" in B.version()


def _compare(B, L, dtype="f32", order=None):
    dt = B.F16 if dtype == "f16" else B.F32
    layer = B.encode(L.weights, L.mask, L.patterns, N=max(L.N, 1), H=L.H, W=L.W, dtype=dt, bias=L.bias,
                     order=order, host_only=True)
    got = layer.export()
    ref = fkw_ref.encode(L.weights, L.mask, L.patterns, order=order, dtype=dtype)
    for name in ("offset", "reorder", "index", "stride"):
        assert got[name].dtype == np.int32 and np.array_equal(got[name], ref[name]), name
    if dtype == "f16":
        assert got["weight"].dtype == np.uint16 and np.array_equal(got["weight"], ref["weight"])
    else:
        assert np.array_equal(got["weight"].view(np.uint32), ref["weight"].view(np.uint32))
    fkw_ref.check_fkw_invariants(got, len(L.patterns), L.F, L.C)
    dense = layer.decode()
    expect = L.masked_weights()
    if dtype == "f16":
        expect = expect.astype(np.float16).astype(np.float32)
    assert np.array_equal(dense.view(np.uint32), expect.view(np.uint32))
    layer.free()
    return got


def test_config1_arrays_bit_exact(B):
    got = _compare(B, synth.config1())
    assert got["offset"][-1] == 512


@pytest.mark.parametrize("prune", [0.0, 0.5, 0.9])
@pytest.mark.parametrize("npat", [4, 8, 12])
def test_random_layers_bit_exact(B, prune, npat):
    L = synth.make_layer("t", F=48, C=40, N=1, H=8, W=8, seed=100 + npat, n_patterns=npat, prune=prune,
                         bias_std=0.1, draw_input=False)
    _compare(B, L)


def test_fp16_weights_bit_exact(B):
    L = synth.make_layer("h", F=32, C=24, N=1, H=8, W=8, seed=5, prune=0.7, dtype="f16", draw_input=False)
    _compare(B, L, dtype="f16")
    # values that stress the float -> half rounding: ties, subnormals, overflow, tiny
    special = np.asarray([0.0, -0.0, 1.0, 1.0009765625, 1.00048828125, 1.00146484375, 65504.0, 65519.0, 65520.0,
                          1e-8, 5.9604645e-08, 2.9802322e-08, 2.98023224e-08 * 1.0001, 6.1e-5, 6.0975552e-05, -3.3e-7,
                          1e5, -1e9, 0.33333334, 1234.5678], dtype=np.float32)
    L2 = synth.make_layer("s", F=5, C=4, N=1, H=8, W=8, seed=6, dtype="f32", draw_input=False)
    w = L2.weights.copy()
    w.reshape(-1)[:special.size] = special
    w.reshape(-1)[special.size:2 * special.size] = -special
    L2.weights = w
    layer = B.encode(L2.weights, L2.mask, L2.patterns, N=1, H=8, W=8, dtype=B.F16, host_only=True)
    with np.errstate(over="ignore"):
        ref = fkw_ref.encode(L2.weights, L2.mask, L2.patterns, dtype="f16")
    assert np.array_equal(layer.export()["weight"], ref["weight"])
    layer.free()


def test_caller_order_and_empty_filters(B):
    L = synth.make_layer("o", F=16, C=12, N=1, H=8, W=8, seed=9, prune=0.3, draw_input=False)
    L.mask[5] = 0
    L.mask[11] = 0
    L.pid[5] = -1
    L.pid[11] = -1
    got = _compare(B, L)
    assert list(got["reorder"][:2]) == [5, 11]
    _compare(B, L, order=synth.random_filter_order(16, seed=3))


def test_vgg_shaped_layer_bit_exact(B):
    L = synth.vgg16_layer(4, N=1)          # 128 -> 256, 60 % of the kernels removed
    got = _compare(B, L)
    lengths = np.diff(got["offset"])
    assert np.all(np.diff(lengths) >= 0)


def test_error_codes(B):
    L = synth.make_layer("e", F=4, C=4, N=1, H=8, W=8, seed=2, draw_input=False)
    bad = L.mask.copy()
    bad[1, 2] = 0
    bad[1, 2, 0, 0] = 1
    with pytest.raises(B.PatdnnError) as e:
        B.encode(L.weights, bad, L.patterns, N=1, H=8, W=8, host_only=True)
    assert e.value.status == 4
    with pytest.raises(B.PatdnnError) as e:
        B.encode(L.weights, L.mask, [0x01B, 0x01B], N=1, H=8, W=8, host_only=True)
    assert e.value.status == 3
    with pytest.raises(B.PatdnnError) as e:
        B.encode(L.weights, L.mask, [0x007], N=1, H=8, W=8, host_only=True)
    assert e.value.status == 3
    with pytest.raises(B.PatdnnError) as e:
        B.encode(L.weights, L.mask, L.patterns, N=1, H=8, W=8, order=[0, 0, 1, 2], host_only=True)
    assert e.value.status == 5
    with pytest.raises(B.PatdnnError) as e:
        B.encode(L.weights, L.mask, L.patterns, N=1, H=0, W=8, host_only=True)
    assert e.value.status == 2
    with pytest.raises(B.PatdnnError) as e:
        B.encode(L.weights, L.mask, L.patterns, N=1, H=8, W=8, dtype=7, host_only=True)
    assert e.value.status == 9
    lib = B.load()
    assert lib.patdnn_encode(None, None, None, 0, None, None) == 1
    assert lib.patdnn_conv(None, None, None, None) == 1
    assert lib.patdnn_free(None) == 0
    assert b"permutation" in lib.patdnn_strerror(5)


def test_size_limits_are_refused_at_encode_time(B):
    L = synth.make_layer("lim", F=4, C=4, N=1, H=8, W=8, seed=2, draw_input=False)
    for kw in (dict(N=1, H=65536, W=8), dict(N=1, H=8, W=65536), dict(N=65536, H=8, W=8),
               dict(N=1, H=32768, W=32768)):                 # the last: 4 * 2^30 elements in one image
        with pytest.raises(B.PatdnnError) as e:
            B.encode(L.weights, L.mask, L.patterns, host_only=True, **kw)
        assert e.value.status == 2, kw
    # one image may come close to 2^31 elements, and a batch may hold more than that
    B.encode(L.weights, L.mask, L.patterns, N=1, H=16384, W=16384, host_only=True).free()
    B.encode(L.weights, L.mask, L.patterns, N=4096, H=1024, W=1024, host_only=True).free()


def test_host_only_handle_refuses_to_run(B):
    L = synth.config1()
    layer = B.encode(L.weights, L.mask, L.patterns, N=1, H=32, W=32, host_only=True)
    with pytest.raises(B.PatdnnError) as e:
        layer.conv(4096, 8192)
    assert e.value.status == 7
    info = layer.plan()
    assert info["variant"] == B.VARIANT_TILED and info["tile_cols"] == 4
    assert info["filters_per_warp"] * info["tile_rows"] * info["tile_cols"] in (64, 128)   # fp32 accumulators per thread
    assert info["entries"] >= 512 and info["smem_bytes"] <= 227 * 1024
    layer.free()


def test_patterns_outside_the_builtin_table_fall_back_to_the_generic_kernel(B):
    pats = np.asarray([0x00F, 0x1E0], dtype=np.uint16)        # legal 4-entry patterns without the centre tap
    pid = np.random.Generator(np.random.PCG64(1)).integers(0, 2, size=(6, 5)).astype(np.int32)
    mask = synth.mask_from_pid(pid, pats)
    w = np.random.Generator(np.random.PCG64(2)).standard_normal((6, 5, 3, 3)).astype(np.float32)
    layer = B.encode(w, mask, pats, N=1, H=8, W=8, host_only=True)
    assert layer.plan()["variant"] == B.VARIANT_REORDER
    ref = fkw_ref.encode(w, mask, pats)
    assert np.array_equal(layer.export()["index"], ref["index"])
    with pytest.raises(B.PatdnnError):
        B.encode(w, mask, pats, N=1, H=8, W=8, variant=B.VARIANT_TILED, host_only=True)
    layer.free()


def test_pattern_run_step_lists_cover_every_kept_kernel():
    """Host side of the pattern-run kernel: the warp-uniform step lists hold every kept kernel once plus zero-weight
    padding (whole steps of 32 lanes); a layer whose input tile cannot stay in shared memory is refused."""
    from paper_2001_00138_b200 import binding as B, synth
    for F, C, prune in ((70, 40, 0.8), (512, 96, 0.9), (33, 7, 0.0)):
        L = synth.make_layer("steps", F=F, C=C, N=2, H=9, W=11, seed=F + C, prune=prune, draw_input=False)
        h = B.encode(L.weights, L.mask, L.patterns, N=2, H=9, W=11, variant=B.VARIANT_PATTERN_RUN, host_only=True)
        p = h.plan()
        h.free()
        assert p["variant"] == B.VARIANT_PATTERN_RUN and p["tile_rows"] == 7 and p["tile_cols"] == 7
        assert p["entries"] % 32 == 0 and p["entries"] >= L.K
        if prune == 0.0:
            assert p["entries"] <= 1024                            # 231 kernels: two warp groups, the second with one filter
    L = synth.make_layer("wide", F=16, C=700, N=1, H=7, W=7, seed=3, prune=0.5, draw_input=False)
    with pytest.raises(B.PatdnnError) as e:
        B.encode(L.weights, L.mask, L.patterns, N=1, H=7, W=7, variant=B.VARIANT_PATTERN_RUN, host_only=True)
    assert e.value.status == 2

