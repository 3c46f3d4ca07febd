"""Pins of the oracle's context drop-off / drop-in (Sec. 3.1) and of the counter-based generator it
draws from, against things other than itself: the generator's published known-answer vectors, the
identity case, set relations that the definition forces, and closed-form expectations."""
import math
import os

import numpy as np
import pytest

import oracle
from oracle import Oracle
from paper_2508_21058_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_generator_reproduces_published_known_answers():
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert list(oracle.philox4x32(w[0:4], w[4:6])) == w[6:10]
        n += 1
    assert n == 3


def _routed(name, heads=1):
    wl = W.workload(name)
    wl.n_heads = heads
    x = {n: W.as_u16(t) for n, t in W.generate(wl, "cpu", ("q", "k")).items()}
    orc = Oracle.from_workload(wl)
    return wl, orc, orc.route(x["q"], orc.chunk_pool(x["k"]))


def _legal(wl, orc, c):
    lay = wl.layout
    none = np.full(orc.k, -1, np.int32)
    mask = orc.token_mask(int(lay.chunk_off[c]), none)
    anchors = {j for j in range(lay.n_chunks) if mask[lay.chunk_off[j]]}
    return {j for j in range(lay.n_chunks) if j not in anchors and (j < c or not wl.causal)}


def test_no_drop_and_no_insertion_is_the_identity():
    wl, orc, sel = _routed("mini2", 2)
    out, nd, nm, na = orc.context_drop(sel, 0.0, 0.0, 5)
    assert np.array_equal(out, sel) and not nd.any() and not nm.any() and not na.any()


@pytest.mark.parametrize("name,p_max,lam", [("mini2", 0.9, 0.0), ("mini9", 0.5, 1.5), ("mini6", 1.0, 3.0), ("mini5", 0.7, 2.0)])
def test_removed_picks_are_a_subset_and_added_chunks_are_new_legal_candidates(name, p_max, lam):
    wl, orc, sel = _routed(name)
    out, nd, nm, na = orc.context_drop(sel, p_max, lam, 11)
    tc = wl.layout.token_chunk()
    k = wl.top_k
    legal = {}
    for i in range(0, wl.n_tokens, 3):
        c = int(tc[i])
        if c not in legal:
            legal[c] = _legal(wl, orc, c)
        before = [int(j) for j in sel[0, i]]
        after = [int(j) for j in out[0, i]]
        kept = {j for j in after if j >= 0 and j in before}
        added = [j for j in after if j >= 0 and j not in before]
        n_sel = sum(j >= 0 for j in before)
        assert len(set(j for j in after if j >= 0)) == sum(j >= 0 for j in after)        # no chunk twice
        assert len(kept) == n_sel - nd[0, i]                                             # exactly n_dropped removed
        assert all(after[s] == before[s] for s in range(k) if after[s] in kept)          # kept picks stay in their slots
        assert 0 <= nd[0, i] <= min(n_sel, math.floor(p_max * k))
        assert len(added) == na[0, i] <= nm[0, i]
        assert all(j in legal[c] for j in added)                                         # never an anchor or a future chunk
        free_before = k - n_sel + nd[0, i]
        n_eligible = len(legal[c]) - n_sel
        assert na[0, i] == min(nm[0, i], free_before, n_eligible)                        # stops only for lack of room or of chunks
        if lam == 0.0:
            assert nm[0, i] == 0 and not added


def test_drop_count_and_poisson_draw_follow_their_closed_forms():
    """Over many rows: E[floor(U a)] = sum_{j=1}^{floor(a)} (1 - j / a) with a = p_max k, the Poisson draw has
    mean and variance lambda, and every pick of a full row is equally likely to be the one removed."""
    wl, orc, sel = _routed("mini6", 3)          # k = 12, rows late in the stream have all 12 picks
    k = wl.top_k
    p_max, lam = 0.8, 1.7
    out, nd, nm, na = orc.context_drop(sel, p_max, lam, 2024)
    full = np.all(sel >= 0, axis=-1)
    assert full.sum() > 5000
    a = p_max * k
    want = sum(1.0 - j / a for j in range(1, int(math.floor(a)) + 1))
    got = nd[full].mean()
    assert abs(got - want) < 4 * math.sqrt(k * k / 12.0 / full.sum()) + 1e-9, (got, want)
    n = nm.size
    assert abs(nm.mean() - lam) < 5 * math.sqrt(lam / n)
    assert abs(nm.var() - lam) < 0.05
    pmf0 = (nm == 0).mean()
    assert abs(pmf0 - math.exp(-lam)) < 5 * math.sqrt(math.exp(-lam) / n)
    # which slot loses its pick: uniform over the slots of full rows that dropped exactly one
    one = full & (nd == 1)
    gone = (sel[one] >= 0) & np.array([[sel[one][r, s] not in out[one][r] for s in range(k)] for r in range(one.sum())])
    assert np.all(gone.sum(-1) == 1)
    counts = gone.sum(0)
    assert counts.sum() == one.sum() and counts.min() > 0.6 * one.sum() / k and counts.max() < 1.4 * one.sum() / k


def test_different_seeds_and_rows_draw_differently_but_a_seed_repeats():
    wl, orc, sel = _routed("mini2", 2)
    a = orc.context_drop(sel, 0.9, 1.0, 1)[0]
    b = orc.context_drop(sel, 0.9, 1.0, 1)[0]
    c = orc.context_drop(sel, 0.9, 1.0, 2)[0]
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    assert not np.array_equal(a[0], a[1]) or not np.array_equal(sel[0], sel[1])
