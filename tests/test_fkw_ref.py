"""Pins for the reference FKW / FKR statement: the paper's worked example, round trips, invariants.  CPU only."""
import os

import numpy as np
import pytest

from oracle import fkw_ref
from paper_2001_00138_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fkw_worked_example.txt")


def _read_golden():
    vals, kernels = {}, []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.split("#")[0].split()
            if not line:
                continue
            if line[0] == "kernel":
                kernels.append(tuple(int(v) for v in line[1:]))
            else:
                vals[line[0]] = [int(v) for v in line[1:]]
    return vals, kernels


def test_worked_example_of_section_5_3():
    vals, kernels = _read_golden()
    F, C, P = vals["F"][0], vals["C"][0], vals["P"][0]
    pats = synth.pattern_set(P)
    pid = np.full((F, C), -1, dtype=np.int32)
    for f, c, p in kernels:
        pid[f, c] = p
    mask = synth.mask_from_pid(pid, pats)
    w = np.arange(F * C * 9, dtype=np.float32).reshape(F, C, 3, 3) + 1
    fkw = fkw_ref.encode(w, mask, pats)
    assert list(np.diff(fkw["offset"])) == vals["lengths"]
    assert list(fkw["offset"]) == vals["offset"]
    assert list(fkw["reorder"]) == vals["reorder"]
    assert list(fkw["index"][:2]) == vals["index_prefix"]
    assert list(fkw["stride"][0]) == vals["stride0"]
    assert [4 * int(n) for n in np.diff(fkw["offset"])] == vals["weights_per_filter"]
    # the first stored kernel is filter 0 / channel 3 with pattern id 0: its four weights in ascending tap order
    taps = synth.mask_to_taps(int(pats[0]))
    assert list(fkw["weight"][0]) == [w[0, 3].reshape(9)[t] for t in taps]
    fkw_ref.check_fkw_invariants(fkw, P, F, C)


def test_natural_pattern_count_and_centre_tap():
    """Section 4.1: the centre weight is always kept, so there are C(8,3) = 56 natural patterns."""
    import itertools
    naturals = {sum(1 << t for t in combo) | (1 << 4)
                for combo in itertools.combinations([t for t in range(9) if t != 4], 3)}
    assert len(naturals) == 56
    assert all(m in naturals for m in synth.PATTERN_MASKS)
    assert len(set(synth.PATTERN_MASKS)) == 12


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("prune", [0.0, 0.6])
def test_round_trip_is_bit_exact(dtype, prune):
    L = synth.make_layer("rt", F=24, C=20, N=1, H=4, W=4, seed=77, n_patterns=8, prune=prune, dtype=dtype,
                         draw_input=False)
    fkw = fkw_ref.encode(L.weights, L.mask, L.patterns, dtype=dtype)
    fkw_ref.check_fkw_invariants(fkw, 8, L.F, L.C)
    dense = fkw_ref.decode(fkw, L.patterns, L.F, L.C)
    assert np.array_equal(dense.view(np.uint32), L.masked_weights().view(np.uint32))
    assert int(fkw["offset"][-1]) == L.K == L.F * L.C - int(np.floor(prune * L.F * L.C + 1e-9))


def test_similarity_against_brute_force_and_prefix_formula():
    rng = np.random.Generator(np.random.PCG64(3))
    P = 5
    for _ in range(50):
        L = int(rng.integers(0, 12))
        a = np.sort(rng.integers(0, P, size=L))
        b = np.sort(rng.integers(0, P, size=L))
        brute = sum(1 for i in range(L) if a[i] == b[i])
        ca = np.concatenate([[0], np.cumsum(np.bincount(a, minlength=P))])
        cb = np.concatenate([[0], np.cumsum(np.bincount(b, minlength=P))])
        closed = sum(max(0, min(ca[p + 1], cb[p + 1]) - max(ca[p], cb[p])) for p in range(P))
        assert fkw_ref.similarity(a, b) == brute == closed


def test_filter_reorder_groups_equal_lengths():
    """After the reorder, filters of equal length are contiguous and lengths never decrease (Section 6.4, the
    filter-length distribution before/after FKR); neighbours are at least as similar as in a random order."""
    L = synth.make_layer("fkr", F=64, C=48, N=1, H=4, W=4, seed=12, prune=0.6, draw_input=False)
    order = fkw_ref.filter_reorder(L.pid)
    assert sorted(order) == list(range(L.F))
    lengths = [(L.pid[f] >= 0).sum() for f in order]
    assert lengths == sorted(lengths)
    seqs = {f: fkw_ref.sorted_pattern_sequence(L.pid[f]) for f in range(L.F)}

    def adjacent(o):
        return sum(fkw_ref.similarity(seqs[a], seqs[b]) for a, b in zip(o, o[1:]) if len(seqs[a]) == len(seqs[b]))

    rnd = sorted(range(L.F), key=lambda f: (len(seqs[f]), (f * 2654435761) % 97))
    assert adjacent(order) >= adjacent(rnd)


def test_empty_filters_come_first_and_caller_order_is_respected():
    L = synth.make_layer("e", F=6, C=5, N=1, H=4, W=4, seed=2, prune=0.0, draw_input=False)
    L.mask[3] = 0
    fkw = fkw_ref.encode(L.weights, L.mask, L.patterns)
    assert fkw["reorder"][0] == 3 and fkw["offset"][1] == 0
    order = [5, 4, 3, 2, 1, 0]
    fkw2 = fkw_ref.encode(L.weights, L.mask, L.patterns, order=order)
    assert list(fkw2["reorder"]) == order
    assert np.array_equal(fkw_ref.decode(fkw2, L.patterns, 6, 5), L.masked_weights())
    with pytest.raises(fkw_ref.ConstraintViolation):
        fkw_ref.encode(L.weights, L.mask, L.patterns, order=[0, 0, 1, 2, 3, 4])


def test_constraint_violations_are_rejected():
    L = synth.make_layer("v", F=4, C=4, N=1, H=4, W=4, seed=2, draw_input=False)
    bad = L.mask.copy()
    bad[1, 2] = 0
    bad[1, 2, 0, 0] = 1                                   # one kept entry: not a 4-entry pattern
    with pytest.raises(fkw_ref.ConstraintViolation):
        fkw_ref.encode(L.weights, bad, L.patterns)
    with pytest.raises(fkw_ref.ConstraintViolation):
        fkw_ref.check_pattern_set([0x01B, 0x01B])
    with pytest.raises(fkw_ref.ConstraintViolation):
        fkw_ref.check_pattern_set([0x007])
    with pytest.raises(fkw_ref.ConstraintViolation):     # a legal pattern that is not in the (smaller) set
        fkw_ref.encode(L.weights, L.mask, synth.pattern_set(2))


def test_weight_reduction_arithmetic():
    """Section 4.3: 4-entry patterns (9/4) times 3.6x connectivity pruning give about 8x fewer CONV weights."""
    assert abs(9 / 4 * 3.6 - 8.1) < 1e-12
    L = synth.make_layer("r", F=60, C=60, N=1, H=4, W=4, seed=4, prune=1 - 1 / 3.6, draw_input=False)
    kept = fkw_ref.check_layer_constraints(L.weights, L.mask, L.patterns, max_kept=L.F * L.C)
    assert abs(L.F * L.C * 9 / (4 * kept) - 8.1) < 0.05


def test_index_structure_is_far_smaller_than_csr():
    """Section 6.4 reports that FKW needs roughly a tenth of CSR's index bytes; with equal index widths FKW stores
    one index per kernel where CSR stores one per weight, so the saving tends to 3/4 and grows with narrower ids."""
    F = C = 256
    K = int(F * C * 0.4)
    b = fkw_ref.storage_bytes(F, C, K, 8)
    assert 1 - b["fkw_index"] / b["csr_index"] > 0.70
    b16 = fkw_ref.storage_bytes(F, C, K, 8, index_bytes=2)
    assert b16["fkw_index"] * 2 == b["fkw_index"]


def test_storage_saving_with_the_widths_that_fit_section_6_4():
    """Section 6.4 prints 93.4 % (index) and 46.7 % (total) saved at 18x.  One byte of index per kept kernel against
    four bytes per weight in CSR gives 1 - 1/16 and 1 - 17/32 when the per-filter arrays are negligible; the
    function must reach those closed forms from below as filters get longer, and the 18x layer must sit near them."""
    P = 8
    last = 0.0
    for per_filter in (16, 64, 256, 4096, 1 << 16):
        F = 8
        b = fkw_ref.storage_bytes(F, per_filter * 4, F * per_filter, P, index_bytes=1, filter_bytes=2, csr_index_bytes=4)
        idx = 1 - b["fkw_index"] / b["csr_index"]
        tot = 1 - (b["fkw_index"] + b["weights"]) / (b["csr_index"] + b["weights"])
        assert last < idx < 15 / 16 and tot < 15 / 32
        last = idx
    assert abs(idx - 15 / 16) < 1e-3 and abs(tot - 15 / 32) < 1e-3
    # by hand for a tiny case: F = 2 filters, K = 3 kernels, P = 2 patterns
    b = fkw_ref.storage_bytes(2, 4, 3, 2, index_bytes=1, filter_bytes=2, csr_index_bytes=4)
    assert b["fkw_index"] == 3 * 2 + 2 * 2 + 3 * 1 + 2 * 3 * 2          # offset[3], reorder[2], index[3], stride[2][3]
    assert b["csr_index"] == 3 * 4 + 12 * 4 and b["weights"] == 48
    # 512 x 512 layer at an overall rate of 18x: 64 kernels per filter
    b = fkw_ref.storage_bytes(512, 512, 512 * 64, P, index_bytes=1, filter_bytes=2, csr_index_bytes=4)
    idx = 1 - b["fkw_index"] / b["csr_index"]
    assert 0.90 < idx < 0.9375                                            # the paper prints 93.4 %

