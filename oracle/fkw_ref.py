"""Reference statement of the FKW storage format and the filter-kernel reorder (FKR).  Test infrastructure only.

Written from Sections 5.2 and 5.3 of the paper, in the paper's order and with its array names
(offset, reorder, index, stride, weight); plain Python loops, no cleverness.  It is used to check the library's
host encoder bit for bit and never runs on the product path.  Where the paper leaves a choice open the reading is
stated at the function that takes it.

Conventions
-----------
* tap t = 3*r + s of a 3x3 kernel; a pattern is a 9-bit mask with exactly four bits; the pattern id of a kernel is
  the 0-based position of its mask in the caller's pattern set (the paper's example numbers its patterns from 1).
* a kernel whose nine mask entries are all zero was removed by connectivity pruning ("empty"); every other kernel
  must equal one pattern of the set (Section 4.2, the two constraint sets of Eq. 1).

Pins: the worked example of Section 5.3, an encode/decode round trip, structural invariants and a brute-force
similarity count (see tests).  The tie-breaking and chaining details of the filter reorder are this module's own
reading ("parity unpinned": the paper only says the most similar filters end up next to each other).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np


class ConstraintViolation(ValueError):
    """The layer does not satisfy the pattern / connectivity constraint sets of Section 4.2."""


def check_pattern_set(patterns: Sequence[int]) -> List[int]:
    pats = [int(p) for p in patterns]
    if not 1 <= len(pats) <= 32:
        raise ConstraintViolation("pattern set must hold 1..32 patterns")
    for p in pats:
        if p < 0 or p >= 512 or bin(p).count("1") != 4:
            raise ConstraintViolation(f"pattern 0x{p:03x} is not a 4-entry 3x3 pattern")
    if len(set(pats)) != len(pats):
        raise ConstraintViolation("duplicate pattern in the set")
    return pats


def classify(mask: np.ndarray, patterns: Sequence[int]) -> np.ndarray:
    """Pattern id per (filter, channel) kernel, -1 for an empty kernel (Section 4.2: W in S_k and S'_k)."""
    pats = check_pattern_set(patterns)
    F, C = mask.shape[:2]
    m = mask.reshape(F, C, 9)
    pid = np.full((F, C), -1, dtype=np.int32)
    for f in range(F):
        for c in range(C):
            bits = 0
            for t in range(9):
                v = int(m[f, c, t])
                if v not in (0, 1):
                    raise ConstraintViolation("mask entries must be 0 or 1")
                bits |= v << t
            if bits == 0:
                continue
            if bits not in pats:
                raise ConstraintViolation(f"kernel ({f},{c}) has mask 0x{bits:03x}, which is not in the pattern set")
            pid[f, c] = pats.index(bits)
    return pid


def kernel_reorder(pid_row: np.ndarray) -> List[int]:
    """Kernel reorder (Section 5.2): kernels with the same pattern are grouped together inside a filter.

    Reading: groups in ascending pattern id, ascending input channel inside a group.
    """
    kept = [(int(p), c) for c, p in enumerate(pid_row) if p >= 0]
    kept.sort()
    return [c for _, c in kept]


def sorted_pattern_sequence(pid_row: np.ndarray) -> np.ndarray:
    return np.sort(np.asarray([int(p) for p in pid_row if p >= 0], dtype=np.int64))


def similarity(seq_a: np.ndarray, seq_b: np.ndarray) -> int:
    """Filter similarity for two filters of equal length (Section 5.2): the number of positions holding the same
    pattern id once each filter's kernels are ordered by pattern id."""
    assert len(seq_a) == len(seq_b)
    return int(np.count_nonzero(np.asarray(seq_a) == np.asarray(seq_b)))


def filter_reorder(pid: np.ndarray) -> List[int]:
    """Filter reorder (Section 5.2): filters of equal length (number of non-empty kernels) become neighbours and,
    inside such a group, the most similar filters are placed next to each other.

    Reading: groups in ascending length (filters with no kernel first); inside a group a greedy chain that starts
    at the smallest original filter id and keeps appending the unplaced filter most similar to the last placed one,
    ties going to the smallest original id.
    """
    F = pid.shape[0]
    seqs = [sorted_pattern_sequence(pid[f]) for f in range(F)]
    lengths = sorted(set(len(s) for s in seqs))
    order: List[int] = []
    for L in lengths:
        group = [f for f in range(F) if len(seqs[f]) == L]
        last = group.pop(0)
        order.append(last)
        while group:
            best, best_sim = None, -1
            for f in group:                       # ascending id, strict '>' keeps the smallest id on ties
                s = similarity(seqs[last], seqs[f])
                if s > best_sim:
                    best, best_sim = f, s
            group.remove(best)
            order.append(best)
            last = best
    return order


def encode(weights: np.ndarray, mask: np.ndarray, patterns: Sequence[int],
           order: Optional[Sequence[int]] = None, dtype: str = "f32") -> Dict[str, np.ndarray]:
    """The five FKW arrays of Section 5.3 for one layer, after FKR.

    offset[i]   kernels stored before filter position i (F+1 entries, offset[F] = K);
    reorder[i]  original output channel of the filter at position i (where its result is written);
    index[k]    input channel of stored kernel k;
    stride[i]   per filter, cumulative kernel counts per pattern (P+1 entries, stride[i][0] = 0, stride[i][P] =
                length; patterns with no kernel repeat the previous value);
    weight[k]   the four kept weights of kernel k in ascending tap order (float32 bits; for dtype "f16" the values
                rounded to nearest-even half precision, returned as uint16 bit patterns).

    ``order`` replaces the filter reorder by a caller-given permutation (the kernel reorder still applies).
    """
    pats = check_pattern_set(patterns)
    P = len(pats)
    F, C = weights.shape[:2]
    pid = classify(mask, pats)
    if order is None:
        order = filter_reorder(pid)
    else:
        order = [int(o) for o in order]
        if sorted(order) != list(range(F)):
            raise ConstraintViolation("order is not a permutation of the filters")
    w = np.ascontiguousarray(weights, dtype=np.float32).reshape(F, C, 9)
    offset = [0]
    index: List[int] = []
    stride: List[List[int]] = []
    wrows: List[np.ndarray] = []
    for f in order:
        chans = kernel_reorder(pid[f])
        row = [0] * (P + 1)
        for c in chans:
            row[int(pid[f, c]) + 1] += 1
        for p in range(P):
            row[p + 1] += row[p]
        stride.append(row)
        for c in chans:
            taps = [t for t in range(9) if (pats[int(pid[f, c])] >> t) & 1]
            index.append(c)
            wrows.append(w[f, c, taps])
        offset.append(offset[-1] + len(chans))
    K = offset[-1]
    wt = np.stack(wrows).astype(np.float32) if K else np.zeros((0, 4), dtype=np.float32)
    if dtype == "f16":
        wt = wt.astype(np.float16).view(np.uint16)
    elif dtype != "f32":
        raise ValueError(dtype)
    return {
        "offset": np.asarray(offset, dtype=np.int32),
        "reorder": np.asarray(order, dtype=np.int32),
        "index": np.asarray(index, dtype=np.int32),
        "stride": np.asarray(stride, dtype=np.int32).reshape(F, P + 1),
        "weight": wt,
    }


def decode(fkw: Dict[str, np.ndarray], patterns: Sequence[int], F: int, C: int) -> np.ndarray:
    """Dense [F, C, 3, 3] float32 weights rebuilt from the five arrays (zeros where nothing is stored)."""
    pats = check_pattern_set(patterns)
    P = len(pats)
    wt = fkw["weight"]
    if wt.dtype == np.uint16:
        wt = wt.view(np.float16).astype(np.float32)
    dense = np.zeros((F, C, 9), dtype=np.float32)
    for i in range(F):
        f = int(fkw["reorder"][i])
        base = int(fkw["offset"][i])
        for p in range(P):
            taps = [t for t in range(9) if (pats[p] >> t) & 1]
            for j in range(int(fkw["stride"][i, p]), int(fkw["stride"][i, p + 1])):
                k = base + j
                dense[f, int(fkw["index"][k]), taps] = wt[k]
    return dense.reshape(F, C, 3, 3)


def check_fkw_invariants(fkw: Dict[str, np.ndarray], P: int, F: int, C: int) -> None:
    """Structural facts any FKW encoding of a layer must satisfy (raises AssertionError)."""
    offset, reorder, index, stride = fkw["offset"], fkw["reorder"], fkw["index"], fkw["stride"]
    K = int(offset[-1])
    assert offset.shape == (F + 1,) and offset[0] == 0
    assert np.all(np.diff(offset) >= 0)
    assert sorted(int(r) for r in reorder) == list(range(F))
    assert index.shape == (K,) and fkw["weight"].shape == (K, 4)
    assert stride.shape == (F, P + 1)
    for i in range(F):
        L = int(offset[i + 1] - offset[i])
        assert stride[i, 0] == 0 and stride[i, P] == L
        assert np.all(np.diff(stride[i]) >= 0)
        for p in range(P):
            run = index[offset[i] + stride[i, p]: offset[i] + stride[i, p + 1]]
            assert np.all((run >= 0) & (run < C))
            assert np.all(np.diff(run) > 0), "channels inside one (filter, pattern) run must ascend strictly"


def check_layer_constraints(weights: np.ndarray, mask: np.ndarray, patterns: Sequence[int],
                            max_kept: Optional[int] = None) -> int:
    """Section 4.2: each kept kernel has exactly four mask entries forming a set pattern; pruned kernels are empty;
    at most ``max_kept`` kernels are non-empty.  Returns the number of kept kernels."""
    pid = classify(mask, patterns)
    F, C = pid.shape
    wm = (weights * mask).reshape(F, C, 9)
    kept = 0
    for f in range(F):
        for c in range(C):
            n_mask = int(mask[f, c].sum())
            if pid[f, c] < 0:
                assert n_mask == 0 and not wm[f, c].any()
            else:
                assert n_mask == 4
                kept += 1
    if max_kept is not None:
        assert kept <= max_kept
    return kept


def storage_bytes(F: int, C: int, K: int, P: int, weight_bytes: int = 4, index_bytes: int = 4,
                  filter_bytes: int = None, csr_index_bytes: int = None) -> Dict[str, int]:
    """Bytes of the FKW arrays versus a CSR matrix over the same 4K non-zeros (Section 6.4's comparison).

    ``index_bytes`` is the width of one ``index[]`` entry (one per kept kernel), ``filter_bytes`` the width of the
    per-filter entries (offset, reorder, stride; default: the same), ``csr_index_bytes`` the width of CSR's column
    indices and row pointers (default: the same).  The paper's figures (93.4 % of the index bytes and 46.7 % of the
    total saved at 18x) are matched by about one byte of index per kernel against four bytes per weight in CSR:
    1 - 1/16 = 93.75 % and 1 - 17/32 = 46.9 % in the limit of long filters.
    """
    fb = index_bytes if filter_bytes is None else filter_bytes
    cb = index_bytes if csr_index_bytes is None else csr_index_bytes
    fkw_index = (F + 1) * fb + F * fb + K * index_bytes + F * (P + 1) * fb
    csr_index = (F + 1) * cb + 4 * K * cb                            # row pointers + one column index per weight
    return {"fkw_index": fkw_index, "csr_index": csr_index, "weights": 4 * K * weight_bytes}
