"""Parity of the CUDA library (through its C-ABI binding) against the CPU oracle,
element by element on small workloads and on sampled rows at the benchmark sizes."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_2508_21058_b200 import MocError, MocPlan
from paper_2508_21058_b200 import workloads as W

import parity_utils as PU

pytestmark = pytest.mark.gpu

SMALL = ["cfg0", "mini1", "mini2", "mini2t", "mini3", "mini4", "mini5", "mini6", "mini7", "mini8", "mini9", "mini10", "mini11", "midi2"]


def _forward_parity(name, scalar, rows_per_head=None):
    wl = W.workload(name)
    run = PU.GpuRun(wl, scalar_attend=scalar).forward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    rec = None if scalar else name
    # step 1: descriptors
    desc64 = orc.chunk_pool(x["k"])
    desc_gpu = run.desc.cpu().numpy()
    assert np.max(np.abs(desc_gpu - desc64)) <= PU.DESC_ATOL
    if rec:
        PU.report(rec, "descriptors", {"max_abs": float(np.max(np.abs(desc_gpu - desc64)))})
    # steps 2-5: indices (oracle routed from its own fp64 descriptors)
    sel_gpu = run.sel.cpu().numpy()
    n, near = PU.assert_routing(wl, orc, x["q"], desc64, sel_gpu, rec)
    # step 6: attention over the GPU's own selection (equal to the oracle's up to the near ties above)
    rows = None if rows_per_head is None else W.sample_rows(wl, rows_per_head)
    O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], sel_gpu, rows)
    O_gpu, lse_gpu = run.O.float().cpu().numpy(), run.lse.cpu().numpy()
    if rows is None:
        O_g, l_g = O_gpu.reshape(-1, wl.head_dim), lse_gpu.reshape(-1)
    else:
        O_g, l_g = O_gpu[rows[:, 0], rows[:, 1]], lse_gpu[rows[:, 0], rows[:, 1]]
    err = PU.attention_errors(O_g, l_g, O_ref, lse_ref)
    PU.assert_attention_close(err, rec)
    return run, err, near, n


@pytest.mark.parametrize("name", SMALL)
def test_forward_small_scalar_kernels(name):
    _forward_parity(name, scalar=True, rows_per_head=None if name != "midi2" else 400)


@pytest.mark.parametrize("name", SMALL)
def test_forward_small(name):
    _forward_parity(name, scalar=False, rows_per_head=None if name != "midi2" else 400)


def _backward_parity(name, scalar, n_rows=64, heads=None, record=None):
    wl = W.workload(name)
    if heads is not None:
        wl.n_heads = heads
    run = PU.GpuRun(wl, tensors=("q", "k", "v", "do"), scalar_attend=scalar).forward().backward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    sel_gpu = run.sel.cpu().numpy()
    lay = wl.layout
    rows = W.sample_rows(wl, n_rows)
    dQ_g = run.dQ.float().cpu().numpy()
    dK_g, dV_g = run.dK.float().cpu().numpy(), run.dV.float().cpu().numpy()
    for n, (key_head, chunk) in enumerate(((0, 0), (wl.n_heads - 1, lay.n_chunks // 2), (0, lay.n_chunks - 2))):
        t0, t1 = int(lay.chunk_off[chunk]), int(lay.chunk_off[chunk + 1])
        dQ, dK, dV = orc.attend_bwd(x["q"], x["k"], x["v"], x["do"], sel_gpu, rows, key_head, (t0, t1))
        rec = record if n == 0 else None
        PU.assert_grad_close(dQ_g[rows[:, 0], rows[:, 1]], dQ, rec, "dQ")
        PU.assert_grad_close(dK_g[key_head, t0:t1], dK, rec, "dK_first_chunk")
        PU.assert_grad_close(dV_g[key_head, t0:t1], dV, rec, "dV_first_chunk")


@pytest.mark.parametrize("name", ["cfg0", "mini2", "mini4", "mini3"])
def test_backward_small_scalar_kernels(name):
    _backward_parity(name, scalar=True)


@pytest.mark.parametrize("name", ["cfg0", "mini1", "mini2", "mini2t", "mini3", "mini4", "mini5", "mini6", "mini7", "mini8", "mini9", "mini10", "mini11", "midi2"])
def test_backward_small(name):
    _backward_parity(name, scalar=False, n_rows=64 if name != "midi2" else 200)


def test_backward_benchmark_length_sampled():
    """The single-shot clip at its full length (two heads: heads are independent): dQ on sampled rows, dK / dV
    of the caption chunk (selected by every query), of a middle frame and of the last-but-one frame."""
    _backward_parity("cfg1", scalar=False, n_rows=96, heads=2, record="cfg1")


def _backward_full_length(name, chunk, n_rows, record, what):
    """One head of a multi-shot layout at its full length: dQ on sampled rows (edges and interior), dK / dV of
    one key chunk (the oracle recomputes the forward of every query that attends to it)."""
    wl = W.workload(name)
    wl.n_heads = 1
    run = PU.GpuRun(wl, tensors=("q", "k", "v", "do")).forward().backward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    sel_gpu = run.sel.cpu().numpy()
    lay = wl.layout
    rows = W.sample_rows(wl, n_rows)
    t0, t1 = int(lay.chunk_off[chunk]), int(lay.chunk_off[chunk + 1])
    dQ, dK, dV = orc.attend_bwd(x["q"], x["k"], x["v"], x["do"], sel_gpu, rows, 0, (t0, t1))
    PU.assert_grad_close(run.dQ.float().cpu().numpy()[rows[:, 0], rows[:, 1]], dQ, record, "dQ")
    PU.assert_grad_close(run.dK.float().cpu().numpy()[0, t0:t1], dK, record, "dK_" + what)
    PU.assert_grad_close(run.dV.float().cpu().numpy()[0, t0:t1], dV, record, "dV_" + what)


def test_backward_training_length_sampled():
    """The minute-scale training layout at its full length, one head: dQ on sampled rows and dK / dV of one
    frame in the middle of the stream (its queries are its shot window and the rows that routed to it)."""
    wl = W.workload("cfg4")
    chunk = wl.layout.n_chunks // 2 + 3
    assert int(wl.layout.chunk_mod[chunk]) == 0           # a video frame
    _backward_full_length("cfg4", chunk, 512, "cfg4", "mid_frame")


def test_backward_caption_chunk_at_multi_shot_length():
    """dK / dV of a caption chunk of the 8-shot stream at its full length (one head): every one of the 264k
    queries attends to it, so its key tiles see the longest query stream the backward has."""
    wl = W.workload("cfg2")
    chunk = int(np.nonzero(wl.layout.chunk_mod == 1)[0][3])          # the caption of the fourth shot
    _backward_full_length("cfg2", chunk, 512, "cfg2", "caption")


def test_route_is_deterministic_and_lists_invert_selection():
    wl = W.workload("mini2")
    run = PU.GpuRun(wl).forward()
    sel1 = run.sel.clone()
    run.forward()
    assert torch.equal(sel1, run.sel)
    # selected pairs from the library's counts == pair count of the oracle's explicit masks
    orc = Oracle.from_workload(wl)
    assert run.plan.moc_selected_pairs(run.ws) == orc.pair_count(run.sel.cpu().numpy())


def test_edge_cases_k0_and_single_chunk():
    # k = 0: anchors only
    wl = W.workload("mini2")
    wl.top_k = 0
    for scalar in (True, False):
        run = PU.GpuRun(wl, scalar_attend=scalar).forward()
        x = run.host_inputs()
        orc = Oracle.from_workload(wl)
        O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], np.zeros((wl.n_heads, wl.n_tokens, 0), np.int32))
        err = PU.attention_errors(run.O.float().cpu().numpy().reshape(-1, wl.head_dim), run.lse.cpu().numpy().reshape(-1),
                                  O_ref, lse_ref)
        PU.assert_attention_close(err)
    # one chunk: plain dense attention, every pick is -1
    lay = W.make_layout(1, 0, 1, 300)
    wl1 = W.Workload("one", 2, 128, lay, 3, 0, 0)
    for scalar in (True, False):
        run = PU.GpuRun(wl1, scalar_attend=scalar).forward()
        assert bool(torch.all(run.sel == -1))
        x = run.host_inputs()
        orc = Oracle.from_workload(wl1)
        O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], run.sel.cpu().numpy())
        err = PU.attention_errors(run.O.float().cpu().numpy().reshape(-1, 128), run.lse.cpu().numpy().reshape(-1), O_ref, lse_ref)
        PU.assert_attention_close(err)


def test_all_tie_scores_pick_lowest_indices():
    wl = W.workload("mini2")
    run = PU.GpuRun(wl)
    run.x["q"].zero_()
    run.forward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    sel_orc = orc.route(x["q"], orc.chunk_pool(x["k"]))
    assert np.array_equal(run.sel.cpu().numpy(), sel_orc)          # exact, including order
    # all logits are zero: LSE = log(#selected keys)
    pairs_row = np.array([orc.token_mask(i, sel_orc[0, i]).sum() for i in range(0, wl.n_tokens, 37)])
    assert np.max(np.abs(run.lse[0, ::37].cpu().numpy() - np.log(pairs_row))) < 1e-4


@pytest.mark.parametrize("name", ["mini8", "mini9", "mini10", "mini11", "mini7"])
def test_equal_descriptors_keep_index_order(name):
    """Groups of frames with identical keys have identical descriptors, so every query scores them
    equally: inside the sorted pick list equal scores must stay in ascending chunk order while better
    chunks arriving later push the list down, and the one that falls off must be the highest index.
    Covers the one-pass list, the extraction rounds with 4 / 32 / 64 entries and the passes beyond 64 picks."""
    wl = W.workload(name)
    lay = wl.layout
    run = PU.GpuRun(wl)
    video = [c for c in range(lay.n_chunks) if lay.chunk_mod[c] == 0 and lay.chunk_shot[c] == 0]
    L0 = int(lay.chunk_off[video[0] + 1] - lay.chunk_off[video[0]])
    same = [c for c in video if int(lay.chunk_off[c + 1] - lay.chunk_off[c]) == L0]
    # frames 0, 3, 6, ... of the first shot share their keys; so do frames 1, 4, 7, ...
    for grp in (same[0::3], same[1::3]):
        src = run.x["k"][:, int(lay.chunk_off[grp[0]]):int(lay.chunk_off[grp[0]]) + L0].clone()
        for c in grp[1:]:
            run.x["k"][:, int(lay.chunk_off[c]):int(lay.chunk_off[c]) + L0] = src
    run.forward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    desc64 = orc.chunk_pool(x["k"])
    PU.assert_routing(wl, orc, x["q"], desc64, run.sel.cpu().numpy())


def test_argument_errors_launch_nothing():
    wl = W.workload("mini1")
    lay = wl.layout
    from paper_2508_21058_b200 import launch_count
    n0 = launch_count()
    bad_off = lay.chunk_off.copy(); bad_off[2] = bad_off[1]
    with pytest.raises(MocError) as e:
        MocPlan(2, lay.n_tokens, 128, bad_off, lay.chunk_shot, lay.chunk_mod, 2)
    assert e.value.code == -3
    with pytest.raises(MocError) as e:
        MocPlan(2, lay.n_tokens, 96, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 2)
    assert e.value.code == -2
    plan = MocPlan.from_workload(wl)
    x = W.generate(wl, "cuda", ("k",))
    desc = torch.empty((wl.n_heads, wl.n_chunks, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(MocError) as e:
        plan.moc_chunk_pool(x["k"], desc, None)
    assert e.value.code == -5
    with pytest.raises(MocError) as e:
        plan.moc_chunk_pool(None, desc, plan.new_workspace())
    assert e.value.code == -1
    ws = plan.new_workspace()
    with pytest.raises(MocError) as e:
        plan.moc_chunk_pool(x["k"].view(torch.int16).flatten()[1:].view(torch.bfloat16), desc, ws)
    assert e.value.code == -4
    assert launch_count() == n0


SWEEP = [f"cfg3-m{m}-p{p}" for m in (1560, 1024, 512, 256) for p in (8, 15, 25)]


@pytest.mark.parametrize("name,rows_per_head,heads",
                         [("cfg1", 2048, None), ("cfg2", 2048, None), ("cfg4", 2048, 6)] + [(n, 2048, 1) for n in SWEEP])
def test_forward_benchmark_size_sampled(name, rows_per_head, heads):
    """The benchmark workloads at their full length, in the launch configuration bench.py times (cfg1 and the
    multi-shot stream with all 24 heads, the training layout on 6 heads, every chunk-size / sparsity point of
    the sweep on one head: heads are independent).  Indices are compared on EVERY row; attention on 2048 rows
    per head, half of them chunk edges and half uniform picks over the stream."""
    wl = W.workload(name)
    if heads is not None:
        wl.n_heads = heads
    run = PU.GpuRun(wl).forward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    desc64 = orc.chunk_pool(x["k"])
    derr = float(np.max(np.abs(run.desc.cpu().numpy() - desc64)))
    PU.report(name, "descriptors", {"max_abs": derr})
    assert derr <= PU.DESC_ATOL
    sel_gpu = run.sel.cpu().numpy()
    PU.assert_routing(wl, orc, x["q"], desc64, sel_gpu, name)
    rows = W.sample_rows(wl, rows_per_head)
    O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], sel_gpu, rows)
    hh, ii = (torch.from_numpy(rows[:, a].astype(np.int64)).cuda() for a in (0, 1))
    O_g = run.O[hh, ii].float().cpu().numpy()
    l_g = run.lse[hh, ii].cpu().numpy()
    PU.assert_attention_close(PU.attention_errors(O_g, l_g, O_ref, lse_ref), name)
    pairs = run.plan.moc_selected_pairs(run.ws)
    PU.report(name, "workload", {"heads": wl.n_heads, "tokens": wl.n_tokens, "chunks": wl.n_chunks, "top_k": wl.top_k,
                                 "selected_pairs": int(pairs), "workspace_bytes": run.plan.workspace_bytes(False)})
    assert pairs > 0
