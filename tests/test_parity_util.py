"""CPU checks of the parity helpers themselves: the rule that decides whether a selection that
differs from the oracle's is still a legal nucleus must accept a swap between tied cubes and reject
every planted mistake (a missing cube, an extra cube, a wrong boundary)."""
import numpy as np

import oracle

import parity_util as pu


def _row(n=40, seed=3, tie=False):
    rng = np.random.default_rng(seed)
    D = 64
    q = rng.standard_normal(D).astype(np.float32)
    kbar = rng.standard_normal((n, D))
    if tie:
        kbar[7] = kbar[21]                       # two cubes with exactly equal probability
    sel, probs, margin = oracle.select_row(q, kbar, n, 1.0 / 8.0, 0.9)
    return sel, probs, margin


def test_identical_sets_and_planted_mistakes():
    sel, probs, _ = _row()
    assert pu.check_nucleus_legal(probs, sel, sel, 0.9) is None
    order = np.argsort(-probs)
    k = int(sel.sum())
    # drop the most probable cube: no longer a prefix of the order
    bad = sel.copy(); bad[order[0]] = 0
    assert pu.check_nucleus_legal(probs, sel, bad, 0.9) is not None
    # add the next two cubes: size differs by two
    bad = sel.copy(); bad[order[k]] = 1; bad[order[k + 1]] = 1
    assert pu.check_nucleus_legal(probs, sel, bad, 0.9) is not None
    # add the next cube (not tied with the boundary cube): not minimal
    bad = sel.copy(); bad[order[k]] = 1
    assert pu.check_nucleus_legal(probs, sel, bad, 0.9) is not None
    # drop the boundary cube: mass below p
    bad = sel.copy(); bad[order[k - 1]] = 0
    assert pu.check_nucleus_legal(probs, sel, bad, 0.9) is not None
    # a cube beyond the row's candidates
    wide = np.concatenate([sel, [1]]).astype(np.uint8)
    assert pu.check_nucleus_legal(probs, np.concatenate([sel, [0]]).astype(np.uint8), wide, 0.9) is not None


def test_swap_between_tied_boundary_cubes_is_legal():
    """Build a row whose boundary falls between two exactly tied cubes: either of them may be taken."""
    probs = np.array([0.5, 0.2, 0.1, 0.1, 0.06, 0.04])
    o = np.array([1, 1, 1, 0, 0, 0], np.uint8)          # p = 0.8: {0, 1, 2} by the lower-index rule
    g = np.array([1, 1, 0, 1, 0, 0], np.uint8)          # the tied twin instead
    assert pu.check_nucleus_legal(probs, o, g, 0.8) is None
    g2 = np.array([1, 1, 0, 0, 1, 0], np.uint8)         # a cube that is not tied
    assert pu.check_nucleus_legal(probs, o, g2, 0.8) is not None
    # Top-K: same size required
    assert pu.check_nucleus_legal(probs, o, g, 0.8, top_k=3) is None
    assert pu.check_nucleus_legal(probs, o, np.array([1, 1, 1, 1, 0, 0], np.uint8), 0.8, top_k=3) is not None
