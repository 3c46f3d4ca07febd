"""The workspace-free descriptor entry point (scratch in a fixed array inside the library, for callers
that cannot allocate device memory when they call: the GPU already handed over in full to a framework's
memory pool, a fixed start-up budget, a loop where cudaMalloc is forbidden) must give what the regular
entry point gives.  Collected last on purpose: it shares one scratch array per GPU with every other call
of that entry point, so it runs after everything else has been checked."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_2508_21058_b200 import MocError, MocPlan
from paper_2508_21058_b200 import workloads as W

import parity_utils as PU

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["mini2", "midi2", "cfg0"])
def test_noalloc_pool_matches_workspace_pool_and_oracle_twice_in_a_row(name):
    wl = W.workload(name)
    x = W.generate(wl, "cuda", ("k",))
    plan = MocPlan.from_workload(wl)
    out = torch.full((wl.n_heads, wl.n_chunks, wl.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    ref = torch.empty_like(out)
    ws = plan.new_workspace()
    torch.cuda.synchronize()
    # The no-allocation call is the FIRST pooling call of this fresh plan, and device memory in use must be
    # the same before and after it (the array's address was looked up when the plan was created).
    free0, _ = torch.cuda.mem_get_info()
    plan.moc_chunk_pool_noalloc(x["k"], out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    plan.moc_chunk_pool(x["k"], ref, ws)
    torch.cuda.synchronize()
    desc64 = Oracle.from_workload(wl).chunk_pool(W.as_u16(x["k"]))
    assert np.max(np.abs(out.cpu().numpy() - desc64)) <= PU.DESC_ATOL            # against the oracle itself
    assert float((out - ref).abs().max()) <= PU.DESC_ATOL, name
    out2 = torch.full_like(ref, float("nan"))                                    # second call meets the first call's leftovers
    plan.moc_chunk_pool_noalloc(x["k"], out2)
    torch.cuda.synchronize()
    assert float((out2 - ref).abs().max()) <= PU.DESC_ATOL, name
    assert np.max(np.abs(out2.cpu().numpy() - desc64)) <= PU.DESC_ATOL
    # a different problem right after, through the same array
    wl2 = W.workload("mini1")
    x2 = W.generate(wl2, "cuda", ("k",))
    plan2 = MocPlan.from_workload(wl2)
    ref2 = torch.empty((wl2.n_heads, wl2.n_chunks, wl2.head_dim), dtype=torch.float32, device="cuda")
    out3 = torch.empty_like(ref2)
    plan2.moc_chunk_pool(x2["k"], ref2, plan2.new_workspace())
    plan2.moc_chunk_pool_noalloc(x2["k"], out3)
    torch.cuda.synchronize()
    assert float((out3 - ref2).abs().max()) <= PU.DESC_ATOL


def test_noalloc_pool_rejects_problems_beyond_its_fixed_scratch():
    # the per-chunk counters: 24 heads x 1000 chunks x 4 bytes pass 64 KiB
    lay = W.make_layout(1, 0, 1000, 8)
    plan = MocPlan(24, lay.n_tokens, 128, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 6, 1, 1)
    k = torch.zeros((1, 8, 128), dtype=torch.bfloat16, device="cuda")     # never read: the call is refused first
    desc = torch.zeros((24, lay.n_chunks, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(MocError) as e:
        plan.moc_chunk_pool_noalloc(k, desc)
    assert e.value.code == -9
    # the partial sums: 24 heads x 344 slices of 256 tokens x 128 x 4 bytes = 4.03 MiB pass 4 MiB, while the
    # counters (24 x 43 chunks) are far below their limit
    lay = W.make_layout(1, 0, 43, 2048)
    plan = MocPlan(24, lay.n_tokens, 128, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 2, 0, 0)
    desc = torch.zeros((24, lay.n_chunks, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(MocError) as e:
        plan.moc_chunk_pool_noalloc(k, desc)
    assert e.value.code == -9
    # one slice fewer per head fits (4 MiB exactly is allowed): 24 x 341.33 -> use 23 heads of the same stream
    plan = MocPlan(23, lay.n_tokens, 128, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 2, 0, 0)
    kk = torch.ones((23, lay.n_tokens, 128), dtype=torch.bfloat16, device="cuda")
    desc = torch.zeros((23, lay.n_chunks, 128), dtype=torch.float32, device="cuda")
    plan.moc_chunk_pool_noalloc(kk, desc)
    torch.cuda.synchronize()
    assert bool(torch.all(desc == 1.0))
