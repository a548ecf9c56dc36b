"""The synthetic generator must hand out layers that satisfy the paper's constraint sets.  CPU only."""
import numpy as np
import pytest

from oracle import fkw_ref
from paper_2001_00138_b200 import synth


def test_config1_structure():
    L = synth.config1()
    assert (L.F, L.C, L.H, L.W, L.N) == (32, 16, 32, 32, 1)
    assert fkw_ref.check_layer_constraints(L.weights, L.mask, L.patterns) == 512
    assert L.nonzero_macs == 4 * 512 * 1024
    assert L.x.min() >= -1 and L.x.max() <= 1


@pytest.mark.parametrize("prune", [0.0, 0.5, 0.9])
def test_connectivity_pruning_keeps_the_largest_kernels(prune):
    L = synth.make_layer("p", F=20, C=30, N=1, H=4, W=4, seed=9, prune=prune, draw_input=False)
    n_removed = int(np.floor(prune * 600 + 1e-9))
    assert fkw_ref.check_layer_constraints(L.weights, L.mask, L.patterns, max_kept=600 - n_removed) == 600 - n_removed
    norms = ((L.weights.astype(np.float64) ** 2) * synth.mask_from_pid(
        synth.best_pattern_ids(L.weights, L.patterns), L.patterns)).sum(axis=(2, 3))
    kept, gone = norms[L.pid >= 0], norms[L.pid < 0]
    if gone.size:
        assert gone.max() <= kept.min()


def test_best_pattern_has_least_distortion():
    L = synth.make_layer("b", F=6, C=7, N=1, H=4, W=4, seed=10, n_patterns=12, draw_input=False)
    sq = L.weights.reshape(6, 7, 9).astype(np.float64) ** 2
    for f in range(6):
        for c in range(7):
            energies = [sq[f, c, synth.mask_to_taps(int(m))].sum() for m in L.patterns]
            assert L.pid[f, c] == int(np.argmax(energies))


def test_fp16_layers_hold_representable_values():
    L = synth.resnet50_layer(3, N=1)
    assert np.array_equal(L.weights, L.weights.astype(np.float16).astype(np.float32))
    assert np.array_equal(L.x, L.x.astype(np.float16).astype(np.float32))
    assert L.K == 512 * 512 - int(np.floor(0.7 * 512 * 512 + 1e-9))


def test_vgg_shapes_are_the_nine_unique_ones():
    assert len(synth.VGG16_CONVS) == 13 and len(set(synth.VGG16_CONVS)) == 9
    L = synth.vgg16_layer(0, N=1)
    assert L.K == 192
    L = synth.vgg16_layer(5, N=1)
    assert L.K == 256 * 256 - int(np.floor(0.6 * 256 * 256 + 1e-9))


def test_seeds_reproduce():
    a, b = synth.config1(), synth.config1()
    assert np.array_equal(a.weights, b.weights) and np.array_equal(a.x, b.x) and np.array_equal(a.mask, b.mask)
