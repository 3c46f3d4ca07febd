"""Helpers shared by the GPU parity tests: run the CUDA library through its C-ABI
binding, run the CPU oracle on the same bf16 bit patterns, and compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import Oracle
from paper_2508_21058_b200 import MocPlan
from paper_2508_21058_b200 import workloads as W

NEAR_TIE = 1e-4            # raw-score window inside which either pick is accepted
O_MAX_ABS, O_MEAN_ABS = 2e-2, 2e-3
LSE_MAX_ABS = 2e-3
GRAD_MAX_ABS = 5e-2
DESC_ATOL = 5e-6


class GpuRun:
    """Inputs on the GPU, the plan, and the outputs of pool -> route -> attend."""

    def __init__(self, wl, tensors=("q", "k", "v"), scalar_attend=False, device="cuda"):
        self.wl = wl
        self.x = W.generate(wl, device, tensors)
        self.plan = MocPlan.from_workload(wl, scalar_attend=scalar_attend)
        self.ws = self.plan.new_workspace(with_bwd=("do" in tensors), device=device)

    def forward(self):
        p, x = self.plan, self.x
        self.desc, self.sel, self.O, self.lse, _ = p.forward(x["q"], x["k"], x["v"], self.ws)
        torch.cuda.synchronize()
        st, det = p.moc_get_status(self.ws)
        assert st == 0, f"device status {st} detail {det}"
        return self

    def backward(self):
        p, x = self.plan, self.x
        self.dQ, self.dK, self.dV = (torch.empty_like(x["q"]) for _ in range(3))
        p.moc_attend_bwd(x["q"], x["k"], x["v"], self.O, self.lse, x["do"], self.sel, self.dQ, self.dK, self.dV, self.ws)
        torch.cuda.synchronize()
        st, det = p.moc_get_status(self.ws)
        assert st == 0, f"device status {st} detail {det}"
        return self

    def host_inputs(self):
        return {n: W.as_u16(t) for n, t in self.x.items()}


def anchor_chunks(orc: Oracle, lay, c: int) -> set:
    """Anchor chunk set of a query in chunk c, read off the oracle's token mask."""
    none = np.full(orc.k, -1, np.int32)
    mask = orc.token_mask(int(lay.chunk_off[c]), none)
    return {j for j in range(lay.n_chunks) if mask[lay.chunk_off[j]]}


def compare_routing(wl, orc: Oracle, q_u16, desc64, sel_gpu: np.ndarray, heads=None):
    """Index parity.  Returns (n_rows, n_near_tie_rows, n_hard_mismatch_rows, examples).
    A row whose GPU and oracle pick sets differ is a near-tie row if every chunk in the
    symmetric difference is a legal candidate whose oracle score lies within NEAR_TIE of
    the oracle's k-th best score; anything else is a hard mismatch."""
    lay = wl.layout
    sel_orc, sel_score, _ = orc.route(q_u16, desc64, with_scores=True)
    a = np.sort(sel_gpu, axis=-1)
    b = np.sort(sel_orc, axis=-1)
    differ = np.any(a != b, axis=-1)
    hh, ii = np.nonzero(differ)
    near, hard, examples = 0, 0, []
    if len(hh):
        tc = lay.token_chunk()
        rows = np.stack([hh, ii], 1).astype(np.int32)
        sc = orc.scores(q_u16, desc64, rows)
        cache = {}
        for r, (h, i) in enumerate(rows):
            c = int(tc[i])
            if c not in cache:
                cache[c] = anchor_chunks(orc, lay, c)
            g = {int(j) for j in sel_gpu[h, i] if j >= 0}
            o = {int(j) for j in sel_orc[h, i] if j >= 0}
            valid = sel_score[h, i][sel_orc[h, i] >= 0]
            ok = len(g) == len(o) and len(valid) > 0
            if ok:
                kth = valid.min()
                for j in g ^ o:
                    legal = (j not in cache[c]) and (j < c or not wl.causal) and 0 <= j < lay.n_chunks
                    if not legal or abs(sc[r, j] - kth) > NEAR_TIE:
                        ok = False
            if ok:
                near += 1
            else:
                hard += 1
                if len(examples) < 5:
                    examples.append((int(h), int(i), sorted(g), sorted(o)))
    # order inside a row: descending oracle score, ties ascending index (checked on equal-set rows)
    same = ~differ
    order_bad = int(np.sum(np.any((sel_gpu != sel_orc) & same[..., None], axis=-1)))
    return differ.size, near, hard, examples, order_bad


def attention_errors(O_gpu: np.ndarray, lse_gpu: np.ndarray, O_ref: np.ndarray, lse_ref: np.ndarray):
    diff = np.abs(O_gpu.astype(np.float64) - O_ref)
    rel_l2 = float(np.sqrt(np.sum(diff ** 2) / max(np.sum(O_ref ** 2), 1e-300)))
    return {"max_abs": float(diff.max()), "mean_abs": float(diff.mean()), "rel_l2": rel_l2,
            "lse_max_abs": float(np.max(np.abs(lse_gpu.astype(np.float64) - lse_ref)))}


def assert_attention_close(err):
    assert err["max_abs"] <= O_MAX_ABS, err
    assert err["mean_abs"] <= O_MEAN_ABS, err
    assert err["lse_max_abs"] <= LSE_MAX_ABS, err
    assert err["rel_l2"] <= 2e-2, err          # guards against a vacuous pass when |O| is small
