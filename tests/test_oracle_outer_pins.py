"""Pins of the oracle's outer-loop (shot-level) routing, Appendix "Outer Loop Context Routing": a numpy
restatement through library reductions (mean, einsum, argsort), closed forms on constructed inputs, the
candidate rule (only shots that end before the query block begins), ties and padding."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_2508_21058_b200 import workloads as W


def _f64(u16):
    return torch.from_numpy(u16.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


def _bits(a):
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _shot_ranges(lay):
    ids = lay.chunk_shot
    out = []
    for s in np.unique(ids):
        cs = np.nonzero(ids == s)[0]
        out.append((int(lay.chunk_off[cs[0]]), int(lay.chunk_off[cs[-1] + 1])))
    return out


@pytest.mark.parametrize("name,shot,M", [("mini2", 2, 1), ("mini3", 3, 2), ("mini4", 2, 5)])
def test_outer_route_equals_library_restatement(name, shot, M):
    wl = W.workload(name)
    x = {n: W.as_u16(t) for n, t in W.generate(wl, "cpu", ("q", "k")).items()}
    orc = Oracle.from_workload(wl)
    rng = _shot_ranges(wl.layout)
    assert orc.num_shots() == len(rng)
    q0, q1 = rng[shot][0] + 7, rng[shot][1] - 3              # a block inside shot `shot`
    desc, sc, sel = orc.outer_route(x["q"], x["k"], q0, q1, M)
    Q, K = _f64(x["q"]), _f64(x["k"])
    want_desc = np.stack([K[:, a:b].mean(1) for a, b in rng], 1)          # [H, S, d]
    xg = Q[:, q0:q1].mean(1)
    want_sc = np.einsum("hd,hsd->hs", xg, want_desc)
    assert np.max(np.abs(desc - want_desc)) < 1e-12 and np.max(np.abs(sc - want_sc)) < 1e-10
    for h in range(wl.n_heads):
        cands = [s for s, (a, b) in enumerate(rng) if b <= q0]
        assert cands == list(range(shot))                                 # exactly the earlier shots
        order = sorted(cands, key=lambda s: (-want_sc[h, s], s))[:M]
        assert [int(v) for v in sel[h, :len(order)]] == order
        assert np.all(sel[h, len(order):] == -1)


def test_outer_route_closed_forms_ties_and_candidate_rule():
    lay = W.make_layout(4, 8, 2, 16)                     # 4 shots of 8 + 32 tokens
    d, H = 64, 1
    L = lay.n_tokens
    rng = _shot_ranges(lay)
    K = np.zeros((H, L, d), np.float32)
    Q = np.zeros((H, L, d), np.float32)
    for s, (a, b) in enumerate(rng):
        K[0, a:b, s] = 2.0                              # shot s: constant key 2 e_s  -> descriptor 2 e_s exactly
    K[0, rng[1][0]:rng[1][1], 0] = 2.0                  # shot 1 also carries e_0: ties with shot 0 on an e_0 query
    q0, q1 = rng[3][0], rng[3][1]
    Q[0, q0:q1, 0] = 1.0                                # block mean e_0 (+ e_2 half the time below)
    Q[0, q0:q1:2, 2] = 3.0                              # mean 1.5 e_2
    orc = Oracle(H, L, d, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 1)
    desc, sc, sel = orc.outer_route(_bits(Q), _bits(K), q0, q1, 3)
    assert np.allclose(desc[0, 2], 2.0 * np.eye(d)[2], atol=0) and np.allclose(desc[0, 1, :2], [2.0, 2.0], atol=0)
    assert np.allclose(sc[0], [2.0, 2.0, 3.0, 0.0], atol=1e-15)
    assert list(sel[0]) == [2, 0, 1]                    # best first; the tie goes to the earlier shot
    # a block that starts inside shot 2: only shots 0 and 1 end before it; shot 2 and 3 are not candidates
    desc, sc, sel = orc.outer_route(_bits(Q), _bits(K), rng[2][0] + 5, rng[3][1], 3)
    assert set(int(v) for v in sel[0] if v >= 0) == {0, 1} and sel[0, 2] == -1
    # the first shot has no history at all
    assert np.all(orc.outer_route(_bits(Q), _bits(K), 3, rng[0][1], 2)[2] == -1)
