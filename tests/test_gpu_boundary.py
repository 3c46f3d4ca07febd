"""Contract of the C ABI beyond plain parity: a workspace that does not hold the plan's lists is refused
on the device without a fault, an edited selection is honoured after moc_lists_from_sel, a bounded wait
that runs out is reported and leaves the GPU usable, the workspace budget, and the debug build."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_2508_21058_b200 import MocError, MocPlan
from paper_2508_21058_b200 import workloads as W

import parity_utils as PU

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

ERR_WORKSPACE, ERR_TIMEOUT, ERR_TOO_LARGE = -5, -8, -9


def _outputs(plan, with_grads=False):
    O = torch.full((plan.H, plan.L, plan.d), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((plan.H, plan.L), 7.0, dtype=torch.float32, device="cuda")
    return O, lse


@pytest.mark.parametrize("fill", [0, 0xA5])
def test_unrouted_workspace_is_refused_on_the_device(fill):
    """moc_attend / moc_attend_bwd on a workspace that moc_route never wrote (zero-filled, or full of a
    byte pattern): every block returns at once, nothing is written, the status says MOC_ERR_WORKSPACE."""
    wl = W.workload("mini2")
    x = W.generate(wl, "cuda", ("q", "k", "v", "do"))
    plan = MocPlan.from_workload(wl)
    ws = torch.full((plan.workspace_bytes(True),), fill, dtype=torch.uint8, device="cuda")
    ws[:64] = 0                                   # status words: no error recorded, no cookie
    sel = torch.full((plan.H, plan.L, plan.k), -1, dtype=torch.int32, device="cuda")
    O, lse = _outputs(plan)
    plan.moc_attend(x["q"], x["k"], x["v"], sel, O, lse, ws)
    torch.cuda.synchronize()
    assert plan.moc_get_status(ws)[0] == ERR_WORKSPACE
    assert bool(torch.all(O == 7.0)) and bool(torch.all(lse == 7.0))
    ws[:64] = 0
    grads = [torch.full_like(O, 7.0) for _ in range(3)]
    plan.moc_attend_bwd(x["q"], x["k"], x["v"], O, lse, x["do"], sel, *grads, ws)
    torch.cuda.synchronize()
    assert plan.moc_get_status(ws)[0] == ERR_WORKSPACE
    assert all(bool(torch.all(g == 7.0)) for g in grads)
    # the same workspace, once routed, works
    desc = torch.empty((plan.H, plan.C, plan.d), dtype=torch.float32, device="cuda")
    plan.moc_chunk_pool(x["k"], desc, ws)
    plan.moc_route(x["q"], desc, sel, ws)
    plan.moc_attend(x["q"], x["k"], x["v"], sel, O, lse, ws)
    torch.cuda.synchronize()
    assert plan.moc_get_status(ws)[0] == 0
    assert not bool(torch.any(O == 7.0).all())


def test_workspace_routed_by_another_plan_is_refused():
    wl_a, wl_b = W.workload("mini2"), W.workload("mini2t")     # same stream, another window: other lists
    wl_b.n_heads = wl_a.n_heads
    x = W.generate(wl_a, "cuda", ("q", "k", "v"))
    plan_a, plan_b = MocPlan.from_workload(wl_a), MocPlan.from_workload(wl_b)
    assert plan_a.workspace_bytes() == plan_b.workspace_bytes()
    ws = plan_a.new_workspace()
    desc, sel, O, lse, _ = plan_a.forward(x["q"], x["k"], x["v"], ws)
    torch.cuda.synchronize()
    assert plan_a.moc_get_status(ws)[0] == 0
    O2, lse2 = _outputs(plan_b)
    plan_b.moc_attend(x["q"], x["k"], x["v"], sel, O2, lse2, ws)
    torch.cuda.synchronize()
    assert plan_b.moc_get_status(ws)[0] == ERR_WORKSPACE
    assert bool(torch.all(O2 == 7.0))


def _edited_selection(wl, sel, rng):
    """A selection the router would not have produced: picks removed, picks swapped for other legal
    chunks, holes in the middle of a row, plus entries that must be dropped (an anchor, a future chunk,
    a repeat, an index out of range)."""
    lay = wl.layout
    tc = lay.token_chunk()
    H, L, k = sel.shape
    out = sel.copy()
    illegal = np.zeros_like(out, dtype=bool)
    for h in range(H):
        for i in rng.choice(L, L // 3, replace=False):
            c = int(tc[i])
            s = int(rng.randint(k))
            what = rng.randint(6)
            if what == 0:
                out[h, i, s] = -1                                   # a hole
            elif what == 1 and c > 0:
                out[h, i, s] = int(rng.randint(c))                  # any earlier chunk (may be an anchor or a repeat)
            elif what == 2:
                out[h, i, s] = c                                    # own chunk: an anchor
            elif what == 3 and c + 1 < lay.n_chunks:
                out[h, i, s] = c + 1                                # a future chunk
            elif what == 4:
                out[h, i, s] = lay.n_chunks + 5                     # out of range
            elif what == 5 and k > 1:
                out[h, i, s] = out[h, i, (s + 1) % k]               # a repeat
    return out


def _clean_like_the_contract(wl, orc, sel):
    """What moc_lists_from_sel must leave in sel_idx, written from the header's rule."""
    lay = wl.layout
    tc = lay.token_chunk()
    out = sel.copy()
    anchors = {}
    for h in range(sel.shape[0]):
        for i in range(sel.shape[1]):
            c = int(tc[i])
            if c not in anchors:
                anchors[c] = PU.anchor_chunks(orc, lay, c)
            seen = set()
            for s in range(sel.shape[2]):
                j = int(sel[h, i, s])
                ok = 0 <= j < lay.n_chunks and j not in anchors[c] and (j < c or not wl.causal) and j not in seen
                if ok:
                    seen.add(j)
                else:
                    out[h, i, s] = -1
    return out


@pytest.mark.parametrize("name", ["mini2", "mini9", "mini5"])
def test_edited_selection_is_honoured_after_lists_from_sel(name):
    wl = W.workload(name)
    run = PU.GpuRun(wl, tensors=("q", "k", "v", "do")).forward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    edited = _edited_selection(wl, run.sel.cpu().numpy(), np.random.RandomState(5))
    want = _clean_like_the_contract(wl, orc, edited)
    assert np.any(want != run.sel.cpu().numpy())
    run.sel.copy_(torch.from_numpy(edited).cuda())
    run.plan.moc_lists_from_sel(run.sel, run.ws)
    run.attend_only()
    sel_now = run.sel.cpu().numpy()
    assert np.array_equal(sel_now, want)                                       # illegal entries blanked, the rest untouched
    assert run.plan.moc_selected_pairs(run.ws) == orc.pair_count(want)
    O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], want)
    err = PU.attention_errors(run.O.float().cpu().numpy().reshape(-1, wl.head_dim), run.lse.cpu().numpy().reshape(-1), O_ref, lse_ref)
    PU.assert_attention_close(err)
    # and the backward over the same edited selection
    run.backward()
    rows = W.sample_rows(wl, 48)
    lay = wl.layout
    chunk = 1
    t0, t1 = int(lay.chunk_off[chunk]), int(lay.chunk_off[chunk + 1])
    dQ, dK, dV = orc.attend_bwd(x["q"], x["k"], x["v"], x["do"], want, rows, 0, (t0, t1))
    PU.assert_grad_close(run.dQ.float().cpu().numpy()[rows[:, 0], rows[:, 1]], dQ)
    PU.assert_grad_close(run.dK.float().cpu().numpy()[0, t0:t1], dK, what="dK")
    PU.assert_grad_close(run.dV.float().cpu().numpy()[0, t0:t1], dV, what="dV")


def test_lists_from_sel_of_the_routers_own_selection_changes_nothing():
    wl = W.workload("mini2")
    run = PU.GpuRun(wl).forward()
    sel0, O0, lse0 = run.sel.clone(), run.O.clone(), run.lse.clone()
    pairs0 = run.plan.moc_selected_pairs(run.ws)
    run.plan.moc_lists_from_sel(run.sel, run.ws)
    run.attend_only()
    assert torch.equal(run.sel, sel0)
    assert run.plan.moc_selected_pairs(run.ws) == pairs0
    assert float((run.O.float() - O0.float()).abs().max()) <= 1e-2           # the same rows, grouped into other tiles
    assert float((run.lse - lse0).abs().max()) <= 1e-3


def test_a_wait_that_runs_out_is_reported_and_the_gpu_stays_usable():
    """A block waits on a barrier nothing arrives on, through the library's bounded wait with a 2 ms limit:
    it must give up, record MOC_ERR_TIMEOUT with the probe's code, and return; the attention kernels then
    refuse to start on that workspace (status set) until routing clears it, after which all is as before."""
    wl = W.workload("mini2")
    run = PU.GpuRun(wl).forward()
    O0 = run.O.clone()
    run.plan.debug_set_wait_limit_us(2000)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    run.plan.debug_wait_probe(run.ws, 777)
    t1.record()
    torch.cuda.synchronize()
    assert 1.5 <= t0.elapsed_time(t1) <= 200.0                       # gave up after the stated limit, not the default second
    assert run.plan.moc_get_status(run.ws) == (ERR_TIMEOUT, 777)
    run.O.fill_(7.0)
    run.plan.moc_attend(run.x["q"], run.x["k"], run.x["v"], run.sel, run.O, run.lse, run.ws)
    torch.cuda.synchronize()
    assert bool(torch.all(run.O == 7.0))                             # a workspace with an error recorded runs nothing
    run.plan.debug_set_wait_limit_us(0)
    run.forward()                                                    # routing clears the status
    assert float((run.O.float() - O0.float()).abs().max()) <= 1e-2


def test_workspace_budget_groups_heads_and_results_do_not_change():
    wl = W.workload("mini2")
    wl.n_heads = 5
    run = PU.GpuRun(wl, tensors=("q", "k", "v", "do")).forward().backward()
    full = run.plan.workspace_bytes(False)
    ref = [t.clone() for t in (run.sel, run.O, run.lse, run.dQ, run.dK, run.dV)]
    small = PU.GpuRun(wl, tensors=("q", "k", "v", "do"))
    per_head = 2 * wl.n_tokens * wl.top_k * wl.head_dim
    small.plan.moc_plan_set_workspace_budget(full - 3 * per_head)   # room for two heads' partials: groups of 2, 2, 1
    assert small.plan.workspace_bytes(False) <= full - 3 * per_head
    small.ws = small.g.empty((small.plan.workspace_bytes(True),), torch.uint8)
    small.forward().backward()
    got = (small.sel, small.O, small.lse, small.dQ, small.dK, small.dV)
    assert torch.equal(got[0], ref[0])
    for a, b in zip(got[1:], ref[1:]):
        assert float((a.float() - b.float()).abs().max()) <= 1e-2
    with pytest.raises(MocError) as e:
        small.plan.moc_plan_set_workspace_budget(per_head // 2)
    assert e.value.code == ERR_TOO_LARGE


def test_debug_build_checks_every_workspace_index_and_finds_nothing():
    """The same sources built with -DMOC_DEBUG check every index taken from the workspace; on a sound run
    they must stay silent (status 0) and give the same answers.  Runs in a child process: a process loads
    one variant of the library."""
    code = (
        "import numpy as np, torch, sys\n"
        "sys.path.insert(0, %r); sys.path.insert(0, %r)\n"
        "import parity_utils as PU\n"
        "from oracle import Oracle\n"
        "from paper_2508_21058_b200 import workloads as W, lib_path\n"
        "assert lib_path().endswith('libmoc_debug.so')\n"
        "for name in ('mini2', 'mini9', 'mini7'):\n"
        "    wl = W.workload(name)\n"
        "    run = PU.GpuRun(wl, tensors=('q', 'k', 'v', 'do')).forward().backward()\n"
        "    x = run.host_inputs(); orc = Oracle.from_workload(wl)\n"
        "    sel = run.sel.cpu().numpy()\n"
        "    PU.assert_routing(wl, orc, x['q'], orc.chunk_pool(x['k']), sel)\n"
        "    O_ref, lse_ref = orc.attend(x['q'], x['k'], x['v'], sel)\n"
        "    PU.assert_attention_close(PU.attention_errors(run.O.float().cpu().numpy().reshape(-1, wl.head_dim), run.lse.cpu().numpy().reshape(-1), O_ref, lse_ref))\n"
        "    run.plan.moc_lists_from_sel(run.sel, run.ws); run.attend_only()\n"
        "print('DEBUG_BUILD_OK')\n"
    ) % (ROOT, os.path.join(ROOT, "tests"))
    from paper_2508_21058_b200 import build as libbuild
    libbuild.build(debug=True)                  # a no-op when libmoc_debug.so is up to date with the sources
    env = dict(os.environ, MOC_LIBRARY="debug", MOC_PARITY_DIR=os.path.join(PU.OUT_ROOT, "parity_debug"))
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, timeout=600)
    assert res.returncode == 0 and "DEBUG_BUILD_OK" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]
