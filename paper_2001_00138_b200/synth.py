"""Seeded synthetic layers shaped like the paper's pattern-pruned 3x3 convolutions.

This module only *produces inputs*: dense weights, a 0/1 mask that satisfies the
paper's two constraint sets (Section 4.2, Eq. 1: every kept kernel matches one
pattern of the set, connectivity-pruned kernels are all zero), a bias, and an
input feature map.  It holds none of the convolution or FKW/FKR arithmetic and
imports neither the CUDA binding nor the CPU oracle; both are fed from here.

The trained VGG-16 / ResNet-50 weights and the ImageNet / CIFAR-10 images the
paper evaluates on are not available, so the shapes and the sparsity structure
follow the paper (Section 4.3: 8 patterns, uniform connectivity rate with a
smaller rate in the first layer) while the values are seeded random numbers.
The two projections of Section 4.2 (best pattern by L2 norm, keep the kernels
with the largest L2 norm) are used here only to turn dense random weights into
a legal pruned layer.

Random draws come from ``numpy.random.Generator(PCG64(seed))`` in the fixed
order  weights -> pattern ids (only for uniformly drawn patterns) -> bias ->
input.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

# Tap numbering t = 3*r + s (r = kernel row, s = kernel column); bit t of a
# pattern mask says tap t is kept.  All twelve contain the centre tap 4
# (Section 4.1: the central weight is never pruned).  A set of size k is the
# first k entries.
PATTERN_TAPS: Tuple[Tuple[int, int, int, int], ...] = (
    (0, 1, 3, 4), (1, 2, 4, 5), (3, 4, 6, 7), (4, 5, 7, 8),
    (1, 3, 4, 5), (3, 4, 5, 7), (1, 3, 4, 7), (1, 4, 5, 7),
    (0, 1, 2, 4), (4, 6, 7, 8), (0, 3, 4, 6), (2, 4, 5, 8),
)
PATTERN_MASKS: Tuple[int, ...] = tuple(sum(1 << t for t in taps) for taps in PATTERN_TAPS)


def pattern_set(k: int) -> np.ndarray:
    """First ``k`` pattern masks as uint16 (k in 1..12)."""
    if not 1 <= k <= len(PATTERN_MASKS):
        raise ValueError("pattern set size must be in 1..12")
    return np.asarray(PATTERN_MASKS[:k], dtype=np.uint16)


def mask_to_taps(m: int) -> List[int]:
    return [t for t in range(9) if (m >> t) & 1]


@dataclass
class Layer:
    """One synthetic pruned 3x3 convolution (stride 1, pad 1)."""
    name: str
    F: int
    C: int
    N: int
    H: int
    W: int
    dtype: str                  # "f32" or "f16" (storage type of weights/activations)
    relu: bool
    weights: np.ndarray         # float32 [F, C, 3, 3]; dense values (entries outside the mask are arbitrary)
    mask: np.ndarray            # uint8   [F, C, 3, 3]
    patterns: np.ndarray        # uint16  [P]
    bias: np.ndarray            # float32 [F]
    x: Optional[np.ndarray]     # float32 [N, C, H, W] (fp16-representable values when dtype == "f16"); None if not drawn
    pid: np.ndarray = field(repr=False, default=None)   # int32 [F, C], -1 = pruned kernel
    seed: int = 0

    @property
    def K(self) -> int:
        return int((self.pid >= 0).sum())

    @property
    def nonzero_macs(self) -> int:
        """Nominal multiply-accumulates on kept weights: 4 per kept kernel per output pixel."""
        return 4 * self.K * self.H * self.W * self.N

    def masked_weights(self) -> np.ndarray:
        return np.where(self.mask != 0, self.weights, np.float32(0.0)).astype(np.float32)


def _round_f16(a: np.ndarray) -> np.ndarray:
    return a.astype(np.float16).astype(np.float32)


def best_pattern_ids(w: np.ndarray, patterns: Sequence[int]) -> np.ndarray:
    """Per kernel, the pattern keeping the largest sum of squared weights (ties -> lowest id)."""
    F, C = w.shape[:2]
    sq = w.reshape(F, C, 9).astype(np.float64) ** 2
    energy = np.stack([sq[:, :, mask_to_taps(int(m))].sum(axis=2) for m in patterns], axis=2)
    return np.argmax(energy, axis=2).astype(np.int32)      # argmax returns the first maximum


def connectivity_prune(w: np.ndarray, pid: np.ndarray, patterns: Sequence[int], rate: float) -> np.ndarray:
    """Remove floor(rate*F*C) kernels with the smallest L2 norm of their 4 kept weights.

    Layer-global; ties remove the smaller linear index f*C+c first.  Returns pid with -1 where pruned.
    """
    F, C = pid.shape
    n_remove = int(np.floor(rate * F * C + 1e-9))
    if n_remove <= 0:
        return pid.copy()
    sq = w.reshape(F, C, 9).astype(np.float64) ** 2
    keepbits = np.zeros((len(patterns), 9), dtype=np.float64)
    for i, m in enumerate(patterns):
        keepbits[i, mask_to_taps(int(m))] = 1.0
    norms = (sq * keepbits[pid]).sum(axis=2).reshape(-1)
    order = np.argsort(norms, kind="stable")
    out = pid.reshape(-1).copy()
    out[order[:n_remove]] = -1
    return out.reshape(F, C)


def mask_from_pid(pid: np.ndarray, patterns: Sequence[int]) -> np.ndarray:
    F, C = pid.shape
    bits = np.zeros((len(patterns) + 1, 9), dtype=np.uint8)     # last row = pruned kernel
    for i, m in enumerate(patterns):
        bits[i, mask_to_taps(int(m))] = 1
    return bits[pid].reshape(F, C, 3, 3)                        # pid == -1 indexes the last (all-zero) row


def make_layer(name: str, *, F: int, C: int, N: int, H: int, W: int, seed: int,
               n_patterns: int = 8, prune: float = 0.0, dtype: str = "f32", relu: bool = True,
               w_std: float = 1.0, pattern_choice: str = "best", bias_std: float = 0.0,
               x_dist: str = "uniform_pm1", draw_input: bool = True) -> Layer:
    """Draw one layer.  ``pattern_choice``: "best" (largest-magnitude pattern) or "uniform" (seeded random id).

    ``x_dist``: "uniform_pm1" U(-1,1), "uniform01" U(0,1), "normal" N(0,1).
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    pats = pattern_set(n_patterns)
    w = (rng.standard_normal((F, C, 3, 3)) * w_std).astype(np.float32)
    if dtype == "f16":
        w = _round_f16(w)
    if pattern_choice == "uniform":
        pid = rng.integers(0, n_patterns, size=(F, C)).astype(np.int32)
    elif pattern_choice == "best":
        pid = best_pattern_ids(w, pats)
    else:
        raise ValueError(pattern_choice)
    pid = connectivity_prune(w, pid, pats, prune)
    if bias_std > 0:
        bias = (rng.standard_normal(F) * bias_std).astype(np.float32)
    else:
        bias = np.zeros(F, dtype=np.float32)
    x = None
    if draw_input:
        x = draw_activations(rng, (N, C, H, W), x_dist, dtype)
    return Layer(name=name, F=F, C=C, N=N, H=H, W=W, dtype=dtype, relu=relu, weights=w,
                 mask=mask_from_pid(pid, pats), patterns=pats, bias=bias, x=x, pid=pid, seed=seed)


def draw_activations(rng: np.random.Generator, shape, dist: str, dtype: str) -> np.ndarray:
    if dist == "uniform_pm1":
        x = rng.random(shape, dtype=np.float32) * 2.0 - 1.0
    elif dist == "uniform01":
        x = rng.random(shape, dtype=np.float32)
    elif dist == "normal":
        x = rng.standard_normal(shape, dtype=np.float32)
    else:
        raise ValueError(dist)
    x = x.astype(np.float32)
    return _round_f16(x) if dtype == "f16" else x


# ----------------------------------------------------------------------------------------------
# The five workload families (shapes after the paper's VGG-16 / ResNet-50 3x3 layers)
# ----------------------------------------------------------------------------------------------

def config1() -> Layer:
    """Small correctness layer: C16 -> F32, 32x32, batch 1, uniformly drawn patterns, no connectivity pruning."""
    return make_layer("cfg1_c16f32_32", F=32, C=16, N=1, H=32, W=32, seed=1001, n_patterns=8, prune=0.0,
                      w_std=0.1, pattern_choice="uniform", bias_std=0.01, x_dist="uniform_pm1")


def config2(draw_input: bool = True) -> Layer:
    """VGG-shaped layer: C256 -> F256, 56x56, batch 1, best-of-8 pattern, half of the kernels removed."""
    return make_layer("cfg2_c256f256_56", F=256, C=256, N=1, H=56, W=56, seed=2002, n_patterns=8, prune=0.5,
                      w_std=1.0, pattern_choice="best", bias_std=0.0, x_dist="uniform_pm1", draw_input=draw_input)


# (C, F, spatial) of the 13 VGG-16 3x3 convolutions; a 2x2 max-pool follows layers 2, 4, 7, 10 (1-based).
VGG16_CONVS: Tuple[Tuple[int, int, int], ...] = (
    (3, 64, 224), (64, 64, 224), (64, 128, 112), (128, 128, 112), (128, 256, 56), (256, 256, 56),
    (256, 256, 56), (256, 512, 28), (512, 512, 28), (512, 512, 28), (512, 512, 14), (512, 512, 14),
    (512, 512, 14),
)
VGG16_POOL_AFTER: Tuple[int, ...] = (1, 3, 6, 9)     # 0-based layer indices followed by a 2x2 max-pool


def vgg16_layer(i: int, N: int, spatial_scale: int = 1, draw_input: bool = False) -> Layer:
    """Layer i (0-based) of the VGG-16 stack: layer 0 keeps every kernel, later layers keep 40 %.

    ``spatial_scale`` divides the 224-pixel input side (for reduced-size parity runs: 224/scale must stay >= 16).
    Weight scale is He-style on the kept fan-in, N(0, 2 / (4 * C * keep)), so activations stay O(1) through the
    thirteen ReLU layers.
    """
    C, F, S = VGG16_CONVS[i]
    keep = 1.0 if i == 0 else 0.4
    S = S // spatial_scale
    return make_layer(f"vgg16_L{i + 1:02d}_c{C}f{F}_{S}", F=F, C=C, N=N, H=S, W=S, seed=3000 + i + 1,
                      n_patterns=8, prune=1.0 - keep, w_std=float(np.sqrt(2.0 / (4.0 * C * keep))),
                      pattern_choice="best", bias_std=0.01, x_dist="uniform01", draw_input=draw_input)


def vgg16_input(N: int, spatial_scale: int = 1) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(3000))
    S = 224 // spatial_scale
    return draw_activations(rng, (N, 3, S, S), "uniform01", "f32")


RESNET50_CONVS: Tuple[Tuple[int, int], ...] = ((64, 56), (128, 28), (256, 14), (512, 7))


def resnet50_layer(i: int, N: int, draw_input: bool = True) -> Layer:
    """ResNet-50-shaped 3x3 layer i (C = F), fp16 storage, 70 % of the kernels removed."""
    C, S = RESNET50_CONVS[i]
    return make_layer(f"resnet50_c{C}_{S}_n{N}", F=C, C=C, N=N, H=S, W=S, seed=4000 + i, n_patterns=8,
                      prune=0.7, dtype="f16", w_std=1.0, pattern_choice="best", bias_std=0.0,
                      x_dist="normal", draw_input=draw_input)


SWEEP_PATTERNS = (4, 6, 8, 12)
SWEEP_PRUNE = (0.0, 0.5, 0.75, 0.9)


def sweep_layer(n_patterns: int, prune: float, N: int = 64, draw_input: bool = True) -> Layer:
    """C = F = 512, 14x14 sweep point (pattern-set size x connectivity rate)."""
    point = SWEEP_PATTERNS.index(n_patterns) * len(SWEEP_PRUNE) + SWEEP_PRUNE.index(prune)
    return make_layer(f"sweep_p{n_patterns}_prune{int(prune * 100)}", F=512, C=512, N=N, H=14, W=14,
                      seed=5000 + point, n_patterns=n_patterns, prune=prune, w_std=1.0, pattern_choice="best",
                      bias_std=0.0, x_dist="uniform_pm1", draw_input=draw_input)


def random_filter_order(F: int, seed: int) -> np.ndarray:
    """Seeded random filter permutation (the 'no filter reorder' arm of the sweep)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.permutation(F).astype(np.int32)
