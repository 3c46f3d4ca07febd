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
    # step 1: descriptors
    desc64 = orc.chunk_pool(x["k"])
    desc_gpu = run.desc.cpu().numpy()
    assert np.max(np.abs(desc_gpu - desc64)) <= PU.DESC_ATOL
    # steps 2-5: indices (oracle routed from its own fp64 descriptors)
    sel_gpu = run.sel.cpu().numpy()
    n, near, hard, ex, order_bad = PU.compare_routing(wl, orc, x["q"], desc64, sel_gpu)
    assert hard == 0, ex
    assert near <= max(2, int(2e-3 * n)), (near, n)
    assert order_bad <= near + max(2, int(2e-3 * n))
    # step 6: attention over the GPU's own selection (equal to the oracle's up to the near ties above)
    rows = None if rows_per_head is None else W.sample_rows(wl, rows_per_head)
    O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], sel_gpu, rows)
    O_gpu, lse_gpu = run.O.float().cpu().numpy(), run.lse.cpu().numpy()
    if rows is None:
        O_g, l_g = O_gpu.reshape(-1, wl.head_dim), lse_gpu.reshape(-1)
    else:
        O_g, l_g = O_gpu[rows[:, 0], rows[:, 1]], lse_gpu[rows[:, 0], rows[:, 1]]
    err = PU.attention_errors(O_g, l_g, O_ref, lse_ref)
    PU.assert_attention_close(err)
    return run, err, near, n


@pytest.mark.parametrize("name", SMALL)
def test_forward_small_scalar_kernels(name):
    _forward_parity(name, scalar=True, rows_per_head=None if name != "midi2" else 400)


@pytest.mark.parametrize("name", SMALL)
def test_forward_small(name):
    _forward_parity(name, scalar=False, rows_per_head=None if name != "midi2" else 400)


def _backward_parity(name, scalar, n_rows=64, heads=None):
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
    for key_head, chunk in ((0, 0), (wl.n_heads - 1, lay.n_chunks // 2), (0, lay.n_chunks - 2)):
        t0, t1 = int(lay.chunk_off[chunk]), int(lay.chunk_off[chunk + 1])
        dQ, dK, dV = orc.attend_bwd(x["q"], x["k"], x["v"], x["do"], sel_gpu, rows, key_head, (t0, t1))
        assert np.max(np.abs(dQ_g[rows[:, 0], rows[:, 1]] - dQ)) <= PU.GRAD_MAX_ABS
        assert np.max(np.abs(dK_g[key_head, t0:t1] - dK)) <= PU.GRAD_MAX_ABS
        assert np.max(np.abs(dV_g[key_head, t0:t1] - dV)) <= PU.GRAD_MAX_ABS
        # not vacuous: relative L2 as well
        for g, r in ((dQ_g[rows[:, 0], rows[:, 1]], dQ), (dK_g[key_head, t0:t1], dK), (dV_g[key_head, t0:t1], dV)):
            assert np.sqrt(np.sum((g - r) ** 2) / np.sum(r ** 2)) < 2e-2


@pytest.mark.parametrize("name", ["cfg0", "mini2", "mini4", "mini3"])
def test_backward_small_scalar_kernels(name):
    _backward_parity(name, scalar=True)


@pytest.mark.parametrize("name", ["cfg0", "mini1", "mini2", "mini2t", "mini3", "mini4", "mini5", "mini6", "mini7", "mini8", "mini9", "mini10", "mini11", "midi2"])
def test_backward_small(name):
    _backward_parity(name, scalar=False, n_rows=64 if name != "midi2" else 200)


def test_backward_benchmark_length_sampled():
    """The single-shot clip at its full length (two heads: heads are independent): dQ on sampled rows, dK / dV
    of the caption chunk (selected by every query), of a middle frame and of the last-but-one frame."""
    _backward_parity("cfg1", scalar=False, n_rows=96, heads=2)


def test_backward_training_length_sampled():
    """The minute-scale training layout at its full length, one head: dQ on sampled rows and dK / dV of one
    frame in the middle of the stream (its queries are its shot window and the rows that routed to it; a caption
    chunk is attended by all 528k queries, which the oracle cannot afford here - the single-shot test covers it)."""
    wl = W.workload("cfg4")
    wl.n_heads = 1
    run = PU.GpuRun(wl, tensors=("q", "k", "v", "do")).forward().backward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    sel_gpu = run.sel.cpu().numpy()
    lay = wl.layout
    rows = W.sample_rows(wl, 64)
    chunk = lay.n_chunks // 2 + 3
    assert int(lay.chunk_mod[chunk]) == 0           # a video frame
    t0, t1 = int(lay.chunk_off[chunk]), int(lay.chunk_off[chunk + 1])
    dQ, dK, dV = orc.attend_bwd(x["q"], x["k"], x["v"], x["do"], sel_gpu, rows, 0, (t0, t1))
    dQ_g = run.dQ.float().cpu().numpy()[rows[:, 0], rows[:, 1]]
    dK_g, dV_g = run.dK.float().cpu().numpy()[0, t0:t1], run.dV.float().cpu().numpy()[0, t0:t1]
    for g, r in ((dQ_g, dQ), (dK_g, dK), (dV_g, dV)):
        assert np.max(np.abs(g - r)) <= PU.GRAD_MAX_ABS
        assert np.sqrt(np.sum((g - r) ** 2) / np.sum(r ** 2)) < 2e-2


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
    n, near, hard, ex, order_bad = PU.compare_routing(wl, orc, x["q"], desc64, run.sel.cpu().numpy())
    assert hard == 0, ex
    assert near <= max(2, int(2e-3 * n)), (near, n)
    assert order_bad <= near + max(2, int(2e-3 * n)), order_bad


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


@pytest.mark.parametrize("name,rows_per_head,heads", [("cfg1", 96, None), ("cfg2", 192, 3), ("cfg4", 192, 2), ("cfg3-m512-p8", 128, 1), ("cfg3-m256-p15", 96, 1)])
def test_forward_benchmark_size_sampled(name, rows_per_head, heads):
    """The benchmark workload in the launch configuration bench.py times; attention
    checked on sampled rows (frame, caption and shot edges plus uniform picks), indices on
    every row of a sample of heads."""
    wl = W.workload(name)
    if heads is not None:       # the multi-shot stream at its full length, on a few heads (each head is independent)
        wl.n_heads = heads
    run = PU.GpuRun(wl).forward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    desc64 = orc.chunk_pool(x["k"])
    assert np.max(np.abs(run.desc.cpu().numpy() - desc64)) <= PU.DESC_ATOL
    sel_gpu = run.sel.cpu().numpy()
    n, near, hard, ex, _ = PU.compare_routing(wl, orc, x["q"], desc64, sel_gpu)
    assert hard == 0, ex
    assert near <= int(2e-3 * n), (near, n)
    rows = W.sample_rows(wl, rows_per_head)
    O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], sel_gpu, rows)
    hh, ii = (torch.from_numpy(rows[:, a].astype(np.int64)).cuda() for a in (0, 1))
    O_g = run.O[hh, ii].float().cpu().numpy()
    l_g = run.lse[hh, ii].cpu().numpy()
    PU.assert_attention_close(PU.attention_errors(O_g, l_g, O_ref, lse_ref))
    assert run.plan.moc_selected_pairs(run.ws) > 0
