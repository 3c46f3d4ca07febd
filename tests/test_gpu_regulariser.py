"""Context drop-off / drop-in (Sec. 3.1) on the GPU against the oracle: the edited selection is integer work and
must match bit for bit (same generator, same single-precision decisions), and attention and its backward over
the edited selection must match the oracle's within the usual tolerances."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_2508_21058_b200 import MocError
from paper_2508_21058_b200 import workloads as W

import parity_utils as PU

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,p_max,lam,seed", [("mini2", 0.9, 1.0, 3), ("mini9", 0.5, 2.5, 2 ** 40 + 17), ("mini6", 1.0, 0.7, 5),
                                                  ("mini5", 0.6, 1.5, 9), ("mini7", 0.4, 4.0, 1), ("cfg0", 1.0, 1.0, 123)])
def test_context_drop_matches_oracle_bit_for_bit_and_attention_follows(name, p_max, lam, seed):
    wl = W.workload(name)
    run = PU.GpuRun(wl, tensors=("q", "k", "v", "do")).forward()
    x = run.host_inputs()
    orc = Oracle.from_workload(wl)
    routed = run.sel.cpu().numpy()
    want, nd, nm, na = orc.context_drop(routed, p_max, lam, seed)
    assert nd.sum() > 0 and na.sum() > 0                     # the case does remove and add
    run.plan.moc_context_drop(run.sel, p_max, lam, seed, run.ws)
    run.attend_only()
    got = run.sel.cpu().numpy()
    assert np.array_equal(got, want)
    assert run.plan.moc_selected_pairs(run.ws) == orc.pair_count(want)
    O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], want)
    err = PU.attention_errors(run.O.float().cpu().numpy().reshape(-1, wl.head_dim), run.lse.cpu().numpy().reshape(-1), O_ref, lse_ref)
    PU.assert_attention_close(err, name + "-dropped")
    run.backward()
    rows = W.sample_rows(wl, 48)
    lay = wl.layout
    t0, t1 = int(lay.chunk_off[1]), int(lay.chunk_off[2])
    dQ, dK, dV = orc.attend_bwd(x["q"], x["k"], x["v"], x["do"], want, rows, 0, (t0, t1))
    PU.assert_grad_close(run.dQ.float().cpu().numpy()[rows[:, 0], rows[:, 1]], dQ)
    PU.assert_grad_close(run.dK.float().cpu().numpy()[0, t0:t1], dK, what="dK")
    PU.assert_grad_close(run.dV.float().cpu().numpy()[0, t0:t1], dV, what="dV")


def test_context_drop_identity_and_argument_range():
    wl = W.workload("mini2")
    run = PU.GpuRun(wl).forward()
    before = run.sel.clone()
    run.plan.moc_context_drop(run.sel, 0.0, 0.0, 7, run.ws)
    run.attend_only()
    assert torch.equal(run.sel, before)
    for bad in ((1.5, 0.0), (-0.1, 0.0), (0.5, 9.0), (float("nan"), 1.0)):
        with pytest.raises(MocError) as e:
            run.plan.moc_context_drop(run.sel, bad[0], bad[1], 7, run.ws)
        assert e.value.code == -2


def test_context_drop_at_benchmark_length():
    """The multi-shot stream at its full length, two heads: every row's edited selection against the oracle."""
    wl = W.workload("cfg2")
    wl.n_heads = 2
    run = PU.GpuRun(wl).forward()
    orc = Oracle.from_workload(wl)
    want, nd, nm, na = orc.context_drop(run.sel.cpu().numpy(), 0.5, 1.0, 99)
    run.plan.moc_context_drop(run.sel, 0.5, 1.0, 99, run.ws)
    run.attend_only()
    assert np.array_equal(run.sel.cpu().numpy(), want)
    x = run.host_inputs()
    rows = W.sample_rows(wl, 256)
    O_ref, lse_ref = orc.attend(x["q"], x["k"], x["v"], want, rows)
    hh, ii = (torch.from_numpy(rows[:, a].astype(np.int64)).cuda() for a in (0, 1))
    PU.assert_attention_close(PU.attention_errors(run.O[hh, ii].float().cpu().numpy(), run.lse[hh, ii].cpu().numpy(), O_ref, lse_ref),
                              "cfg2-dropped")
    PU.report("cfg2-dropped", "regulariser", {"rows": int(nd.size), "picks_removed": int(nd.sum()), "chunks_added": int(na.sum()),
                                              "selection_mismatches": 0})
