"""The workspace-free descriptor entry point (scratch in a fixed array inside the library,
for callers that cannot allocate device memory when they call) must give what the regular
entry point gives.  Collected last on purpose: it shares one scratch array per GPU with
every other call of that entry point, so it runs after everything else has been checked."""
import numpy as np
import pytest
import torch

from paper_2508_21058_b200 import MocError, MocPlan
from paper_2508_21058_b200 import workloads as W

import parity_utils as PU

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["mini2", "midi2", "cfg0"])
def test_noalloc_pool_matches_workspace_pool_twice_in_a_row(name):
    wl = W.workload(name)
    x = W.generate(wl, "cuda", ("k",))
    plan = MocPlan.from_workload(wl)
    ws = plan.new_workspace()
    ref = torch.empty((wl.n_heads, wl.n_chunks, wl.head_dim), dtype=torch.float32, device="cuda")
    plan.moc_chunk_pool(x["k"], ref, ws)
    torch.cuda.synchronize()
    for call in range(2):                      # second call meets the first call's leftovers
        out = torch.full_like(ref, float("nan"))
        plan.moc_chunk_pool_noalloc(x["k"], out)
        torch.cuda.synchronize()
        assert float((out - ref).abs().max()) <= PU.DESC_ATOL, (name, call)
    # a different problem right after, through the same array
    wl2 = W.workload("mini1")
    x2 = W.generate(wl2, "cuda", ("k",))
    plan2 = MocPlan.from_workload(wl2)
    ref2 = torch.empty((wl2.n_heads, wl2.n_chunks, wl2.head_dim), dtype=torch.float32, device="cuda")
    out2 = torch.empty_like(ref2)
    plan2.moc_chunk_pool(x2["k"], ref2, plan2.new_workspace())
    plan2.moc_chunk_pool_noalloc(x2["k"], out2)
    torch.cuda.synchronize()
    assert float((out2 - ref2).abs().max()) <= PU.DESC_ATOL


def test_noalloc_pool_rejects_problems_beyond_its_fixed_scratch():
    lay = W.make_layout(1, 0, 1000, 8)          # 24 heads x 1000 chunks: the per-chunk counters alone pass 64 KiB
    plan = MocPlan(24, lay.n_tokens, 128, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 6, 1, 1)
    k = torch.zeros((1, 8, 128), dtype=torch.bfloat16, device="cuda")     # never read: the call is refused first
    desc = torch.zeros((24, lay.n_chunks, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(MocError) as e:
        plan.moc_chunk_pool_noalloc(k, desc)
    assert e.value.code == -9
