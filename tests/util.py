"""Shared helpers for the tests: tolerance rule and thin runners around the binding and the oracle."""
import numpy as np

TOL_F32 = 1e-4     # max relative error, fp32 storage
TOL_F16 = 2e-3     # fp16 storage, fp32 accumulate


def assert_close(got: np.ndarray, ref: np.ndarray, tol: float, what: str = "") -> float:
    """|got - ref| <= tol * max(|ref|, rms(ref)) element by element; returns the worst ratio to that bound."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    bound = tol * np.maximum(np.abs(ref), max(rms, 1e-30))
    err = np.abs(got - ref)
    worst = float((err / bound).max()) if ref.size else 0.0
    if worst > 1.0:
        i = np.unravel_index(np.argmax(err / bound), ref.shape)
        raise AssertionError(f"{what}: |{got[i]} - {ref[i]}| exceeds {tol} * max(|ref|, rms={rms:.4g}) at {i} "
                             f"(ratio {worst:.2f})")
    return worst


def oracle_layer(L, x=None):
    import oracle
    return oracle.conv3x3(L.x if x is None else x, L.weights, L.mask, L.bias, L.relu)


def gpu_layer(L, x=None, variant=0, order=None, via_host=False):
    """Encode L, run it on the GPU through the C ABI, return the output as float32 numpy."""
    import torch
    from paper_2001_00138_b200 import binding as B
    x = L.x if x is None else x
    dt = B.F16 if L.dtype == "f16" else B.F32
    tdt = torch.float16 if L.dtype == "f16" else torch.float32
    N, C, H, W = x.shape
    layer = B.encode(L.weights, L.mask, L.patterns, N=N, H=H, W=W, dtype=dt, relu=L.relu, bias=L.bias,
                     order=order, variant=variant)
    try:
        if via_host:
            xin = np.ascontiguousarray(x.astype(np.float16 if L.dtype == "f16" else np.float32))
            out = np.empty((N, L.F, H, W), dtype=xin.dtype)
            layer.conv_host(xin, out)
            return out.astype(np.float32), layer.plan()
        xt = torch.from_numpy(x).to("cuda", dtype=tdt).contiguous()
        out = torch.full((N, L.F, H, W), float("nan"), device="cuda", dtype=tdt)
        layer.conv(xt, out, torch.cuda.current_stream().cuda_stream)
        layer.check()                 # synchronises; raises if a bounded device-side wait expired
        return out.float().cpu().numpy(), layer.plan()
    finally:
        layer.free()


def chain_tol(n_layers: int, tol: float) -> float:
    """Bound for a chain of n_layers compared with the chained oracle: sqrt(n_layers) * tol.

    Every layer adds its own rounding error, bounded by `tol` relative to max(|o|, rms); the chains of these tests are
    He-scaled, so an input perturbation passes a layer with rms gain of about one, and the per-layer errors are
    independent rounding noise that adds in quadrature.  (Measured on the 13-layer benchmark stack: 1.3 * tol.)
    Single layers, and layers checked through an identity successor, use `tol` itself."""
    return float(np.sqrt(n_layers)) * tol


def identity_layer(F: int):
    """(weights, mask, patterns) of a C = F layer that copies its input: one kept kernel per filter, on the channel
    of the same number, whose pattern's centre weight is 1.0 and whose other three kept weights are 0.0."""
    from paper_2001_00138_b200 import synth
    pats = synth.pattern_set(8)
    taps = synth.mask_to_taps(int(pats[0]))
    w = np.zeros((F, F, 3, 3), dtype=np.float32)
    m = np.zeros((F, F, 3, 3), dtype=np.uint8)
    for f in range(F):
        for t in taps:
            m[f, f, t // 3, t % 3] = 1
        w[f, f, 1, 1] = 1.0
    return w, m, pats
