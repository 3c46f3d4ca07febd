"""Outer-loop (shot-level) context routing on the GPU against the oracle, and the path it feeds: the reduced
stream's chunk table against an independent construction, the gathered rows bit for bit, and the inner path
(pool -> route -> attend) on the reduced stream against the oracle run on the same reduced inputs."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_2508_21058_b200 import MocError, MocPlan
from paper_2508_21058_b200 import workloads as W

import parity_utils as PU

pytestmark = pytest.mark.gpu


def _shot_ranges(lay):
    out = []
    for s in np.unique(lay.chunk_shot):
        cs = np.nonzero(lay.chunk_shot == s)[0]
        out.append((int(lay.chunk_off[cs[0]]), int(lay.chunk_off[cs[-1] + 1]), int(cs[0]), int(cs[-1]) + 1))
    return out


def _outer(wl, block_shot, M):
    x = W.generate(wl, "cuda", ("q", "k", "v"))
    plan = MocPlan.from_workload(wl)
    g = PU.Guarded()
    ws = g.empty((plan.workspace_bytes(False),), torch.uint8)
    S = plan.moc_outer_num_shots()
    rng = _shot_ranges(wl.layout)
    assert S == len(rng)
    q0, q1 = rng[block_shot][0], rng[block_shot][1]
    desc = g.empty((plan.H, plan.C, plan.d), torch.float32)
    sdesc = g.empty((plan.H, S, plan.d), torch.float32)
    scores = g.empty((plan.H, S), torch.float32)
    sel = g.empty((plan.H, M), torch.int32)
    plan.moc_chunk_pool(x["k"], desc, ws)
    plan.moc_outer_route(x["q"], desc, q0, q1, M, sdesc, scores, sel, ws)
    torch.cuda.synchronize()
    g.check()
    return x, plan, rng, (q0, q1), sdesc, scores, sel


@pytest.mark.parametrize("name,block_shot,M", [("mini2", 2, 1), ("mini3", 3, 2), ("mini4", 1, 3), ("cfg2", 6, 3)])
def test_outer_route_matches_oracle(name, block_shot, M):
    wl = W.workload(name)
    if name == "cfg2":
        wl.n_heads = 4
    x, plan, rng, (q0, q1), sdesc, scores, sel = _outer(wl, block_shot, M)
    h = {n: W.as_u16(t) for n, t in x.items()}
    orc = Oracle.from_workload(wl)
    d64, s64, sel64 = orc.outer_route(h["q"], h["k"], q0, q1, M)
    assert np.max(np.abs(sdesc.cpu().numpy() - d64)) <= PU.DESC_ATOL
    assert np.max(np.abs(scores.cpu().numpy() - s64)) <= 1e-4
    got = sel.cpu().numpy()
    near = 0
    for hh in range(wl.n_heads):
        if list(got[hh]) == list(sel64[hh]):
            continue
        # differing picks must be candidates within the near-tie window of the oracle's M-th best score
        cands = [s for s, r in enumerate(rng) if r[1] <= q0]
        kth = min(s64[hh, s] for s in sel64[hh] if s >= 0)
        for s in set(got[hh]) ^ set(sel64[hh]):
            assert s in cands and abs(s64[hh, s] - kth) <= PU.NEAR_TIE
        near += 1
    PU.report(name + "-outer", "outer_routing", {"streams": wl.n_heads, "shots": len(rng), "top_m": M, "near_tie_streams": near,
                                                "desc_max_abs": float(np.max(np.abs(sdesc.cpu().numpy() - d64))),
                                                "score_max_abs": float(np.max(np.abs(scores.cpu().numpy() - s64)))})
    assert near <= 1


def test_outer_to_inner_path_on_the_reduced_stream():
    wl = W.workload("mini3")                  # 4 shots; route the last shot's block to 2 earlier shots
    M, block_shot, stream = 2, 3, 1
    x, plan, rng, (q0, q1), sdesc, scores, sel = _outer(wl, block_shot, M)
    lay = wl.layout
    picks = [int(s) for s in sel[stream].cpu().numpy()]
    off, shot, mod, tok = plan.moc_outer_reduced_layout(picks, q0, q1)
    # independent construction: text chunks, picked shots, the block's shot, in stream order
    keep = [c for c in range(lay.n_chunks)
            if lay.chunk_mod[c] == 1 or any(rng[s][2] <= c < rng[s][3] for s in picks + [block_shot])]
    want_tok = np.concatenate([np.arange(lay.chunk_off[c], lay.chunk_off[c + 1]) for c in keep])
    assert np.array_equal(tok, want_tok)
    assert np.array_equal(np.diff(off), np.diff(lay.chunk_off)[keep])
    assert np.array_equal(shot, lay.chunk_shot[keep]) and np.array_equal(mod, lay.chunk_mod[keep])
    assert 0 < len(tok) < lay.n_tokens
    # gather, then the inner path on the reduced stream (one plan for it; every stream uses this stream's selection)
    tok_d = torch.from_numpy(tok).cuda()
    red = {}
    for n in ("q", "k", "v"):
        red[n] = torch.empty((wl.n_heads, len(tok), wl.head_dim), dtype=torch.bfloat16, device="cuda")
        plan.moc_gather_tokens(x[n], tok_d, red[n])
        assert torch.equal(red[n], x[n][:, tok_d.long()])
    inner = MocPlan(wl.n_heads, len(tok), wl.head_dim, off, shot, mod, wl.top_k, wl.win_back, wl.win_fwd, wl.causal)
    desc, sel_in, O, lse, ws = inner.forward(red["q"], red["k"], red["v"])
    torch.cuda.synchronize()
    assert inner.moc_get_status(ws)[0] == 0
    orc = Oracle(wl.n_heads, len(tok), wl.head_dim, off, shot, mod, wl.top_k, wl.win_back, wl.win_fwd, wl.causal)
    h = {n: W.as_u16(t) for n, t in red.items()}
    red_wl = W.Workload("reduced", wl.n_heads, wl.head_dim, W.Layout(off, shot, mod), wl.top_k, wl.win_back, wl.win_fwd, wl.causal)
    sel_np = sel_in.cpu().numpy()
    PU.assert_routing(red_wl, orc, h["q"], orc.chunk_pool(h["k"]), sel_np)
    O_ref, lse_ref = orc.attend(h["q"], h["k"], h["v"], sel_np)
    PU.assert_attention_close(PU.attention_errors(O.float().cpu().numpy().reshape(-1, wl.head_dim), lse.cpu().numpy().reshape(-1),
                                                  O_ref, lse_ref), "mini3-outer-inner")


def test_outer_route_argument_errors():
    wl = W.workload("mini2")
    x, plan, rng, (q0, q1), sdesc, scores, sel = _outer(wl, 1, 1)
    ws = plan.new_workspace()
    desc = torch.zeros((plan.H, plan.C, plan.d), dtype=torch.float32, device="cuda")
    for bad in ((5, 5, 1), (-1, 9, 1), (0, wl.n_tokens + 1, 1), (0, 8, 99)):
        with pytest.raises(MocError) as e:
            plan.moc_outer_route(x["q"], desc, bad[0], bad[1], bad[2], sdesc, scores, sel, ws)
        assert e.value.code == -2
    with pytest.raises(MocError) as e:
        plan.moc_outer_reduced_layout([99], q0, q1)
    assert e.value.code == -2
