"""Helpers shared by the GPU parity tests: run the CUDA library through its C-ABI
binding, run the CPU oracle on the same bf16 bit patterns, and compare.

Every device buffer the library writes (outputs and the workspace) is allocated between two
poisoned guard bands that are verified after the calls: a kernel that writes outside a
buffer fails the test even when the stray write lands in memory nobody reads.

Every comparison can be recorded (``report``): one JSON file per workload under
the parity records folder (``PARITY_DIR``: ``$MOC_PARITY_DIR`` if set) with the rows compared, the near-tie and
hard-mismatch counts and the error figures, from which the committed parity table is made."""
from __future__ import annotations

import json
import os

import numpy as np
import torch

from oracle import Oracle
from paper_2508_21058_b200 import MocPlan
from paper_2508_21058_b200 import workloads as W

NEAR_TIE = 1e-4            # raw-score window inside which either pick is accepted
NEAR_TIE_ROW_FRACTION = 5e-4   # at most this fraction of rows may be near-tie rows (plus two rows on tiny inputs)
O_MAX_ABS, O_MEAN_ABS = 2e-2, 2e-3
LSE_MAX_ABS = 2e-3
GRAD_MAX_ABS = 5e-2
DESC_ATOL = 5e-6
GUARD = 4096
POISON = 0xA5

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
OUT_ROOT = os.path.join(ROOT, "gpurun_out")          # where a run leaves its outputs
PARITY_DIR = os.environ.get("MOC_PARITY_DIR", os.path.join(OUT_ROOT, "parity"))


def near_tie_budget(n_rows: int) -> int:
    return max(2, int(NEAR_TIE_ROW_FRACTION * n_rows))


def report(workload: str, section: str, values: dict):
    """Merge `values` under `section` into the workload's parity record."""
    out_dir = PARITY_DIR
    try:
        os.makedirs(out_dir, exist_ok=True)
        path = os.path.join(out_dir, f"{workload}.json")
        rec = {}
        if os.path.exists(path):
            with open(path) as f:
                rec = json.load(f)
        rec.setdefault(section, {}).update(values)
        with open(path, "w") as f:
            json.dump(rec, f, indent=1, sort_keys=True)
    except OSError:
        pass


class Guarded:
    """Device buffers with poisoned bands on both sides."""

    def __init__(self, device="cuda"):
        self.device = device
        self.bufs = []

    def empty(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 256
        raw = torch.full((GUARD + n + pad + GUARD,), POISON, dtype=torch.uint8, device=self.device)
        self.bufs.append((raw, n))
        return raw[GUARD:GUARD + n].view(dtype).view(shape)

    def check(self):
        for raw, n in self.bufs:
            assert bool(torch.all(raw[:GUARD] == POISON)), "a kernel wrote before a buffer"
            assert bool(torch.all(raw[GUARD + n:] == POISON)), "a kernel wrote past a buffer"


class GpuRun:
    """Inputs on the GPU, the plan, and the outputs of pool -> route -> attend."""

    def __init__(self, wl, tensors=("q", "k", "v"), scalar_attend=False, device="cuda", plan_kw=None):
        self.wl = wl
        self.x = W.generate(wl, device, tensors)
        self.plan = MocPlan.from_workload(wl, scalar_attend=scalar_attend, **(plan_kw or {}))
        self.g = Guarded(device)
        self.with_bwd = "do" in tensors
        self.ws = self.g.empty((self.plan.workspace_bytes(self.with_bwd),), torch.uint8)

    def check_status(self):
        torch.cuda.synchronize()
        st, det = self.plan.moc_get_status(self.ws)
        assert st == 0, f"device status {st} detail {det}"
        self.g.check()

    def alloc_forward(self):
        p, g = self.plan, self.g
        self.desc = g.empty((p.H, p.C, p.d), torch.float32)
        self.sel = g.empty((p.H, p.L, p.k), torch.int32)
        self.O = g.empty((p.H, p.L, p.d), torch.bfloat16)
        self.lse = g.empty((p.H, p.L), torch.float32)

    def forward(self):
        p, x = self.plan, self.x
        if not hasattr(self, "desc"):
            self.alloc_forward()
        p.moc_chunk_pool(x["k"], self.desc, self.ws)
        p.moc_route(x["q"], self.desc, self.sel, self.ws)
        p.moc_attend(x["q"], x["k"], x["v"], self.sel, self.O, self.lse, self.ws)
        self.check_status()
        return self

    def attend_only(self):
        p, x = self.plan, self.x
        p.moc_attend(x["q"], x["k"], x["v"], self.sel, self.O, self.lse, self.ws)
        self.check_status()
        return self

    def backward(self):
        p, x = self.plan, self.x
        if not hasattr(self, "dQ"):
            self.dQ, self.dK, self.dV = (self.g.empty((p.H, p.L, p.d), torch.bfloat16) for _ in range(3))
        p.moc_attend_bwd(x["q"], x["k"], x["v"], self.O, self.lse, x["do"], self.sel, self.dQ, self.dK, self.dV, self.ws)
        self.check_status()
        return self

    def host_inputs(self):
        return {n: W.as_u16(t) for n, t in self.x.items()}


def anchor_chunks(orc: Oracle, lay, c: int) -> set:
    """Anchor chunk set of a query in chunk c, read off the oracle's token mask."""
    none = np.full(orc.k, -1, np.int32)
    mask = orc.token_mask(int(lay.chunk_off[c]), none)
    return {j for j in range(lay.n_chunks) if mask[lay.chunk_off[j]]}


def compare_routing(wl, orc: Oracle, q_u16, desc64, sel_gpu: np.ndarray, heads=None):
    """Index parity.  Returns (n_rows, n_near_tie_rows, n_hard_mismatch_rows, examples, order_bad, order_near).
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
    # order inside a row (checked on equal-set rows): descending oracle score, equal scores by ascending index.
    # Two picks whose oracle scores lie within NEAR_TIE of each other may come in either order (the kernel
    # accumulates the same products in fp32); any other difference in order is counted as bad.
    same = ~differ
    oh, oi = np.nonzero(np.any((sel_gpu != sel_orc) & same[..., None], axis=-1))
    order_near, order_bad = 0, 0
    for h, i in zip(oh, oi):
        score_of = {int(j): float(sc_) for j, sc_ in zip(sel_orc[h, i], sel_score[h, i]) if j >= 0}
        g = [int(j) for j in sel_gpu[h, i]]
        live = [j for j in g if j >= 0]
        ok = g[:len(live)] == live                                  # padding only at the end
        for a, b in zip(live[:-1], live[1:]):
            if score_of[a] < score_of[b] - NEAR_TIE or (score_of[a] == score_of[b] and a > b):
                ok = False
        order_near += ok
        order_bad += not ok
    return differ.size, near, hard, examples, order_bad, order_near


def assert_routing(wl, orc, q_u16, desc64, sel_gpu, record=None):
    n, near, hard, ex, order_bad, order_near = compare_routing(wl, orc, q_u16, desc64, sel_gpu)
    if record:
        report(record, "routing", {"rows": int(n), "heads": int(sel_gpu.shape[0]), "near_tie_rows": int(near),
                                   "hard_mismatch_rows": int(hard), "order_near_tie_rows": int(order_near),
                                   "order_wrong_rows": int(order_bad),
                                   "near_tie_window": NEAR_TIE, "near_tie_row_budget": near_tie_budget(n)})
    assert hard == 0, ex
    assert near <= near_tie_budget(n), (near, n)
    assert order_bad == 0, order_bad           # same set, and the order is wrong by more than a near tie
    return n, near


def attention_errors(O_gpu: np.ndarray, lse_gpu: np.ndarray, O_ref: np.ndarray, lse_ref: np.ndarray):
    diff = np.abs(O_gpu.astype(np.float64) - O_ref)
    rel_l2 = float(np.sqrt(np.sum(diff ** 2) / max(np.sum(O_ref ** 2), 1e-300)))
    return {"rows": int(O_ref.shape[0]), "max_abs": float(diff.max()), "mean_abs": float(diff.mean()), "rel_l2": rel_l2,
            "lse_max_abs": float(np.max(np.abs(lse_gpu.astype(np.float64) - lse_ref)))}


def assert_attention_close(err, record=None):
    if record:
        report(record, "attention", err)
    assert err["max_abs"] <= O_MAX_ABS, err
    assert err["mean_abs"] <= O_MEAN_ABS, err
    assert err["lse_max_abs"] <= LSE_MAX_ABS, err
    assert err["rel_l2"] <= 2e-2, err          # guards against a vacuous pass when |O| is small


def grad_errors(g: np.ndarray, ref: np.ndarray):
    diff = np.abs(g.astype(np.float64) - ref)
    return {"rows": int(ref.shape[0]), "max_abs": float(diff.max()), "mean_abs": float(diff.mean()),
            "rel_l2": float(np.sqrt(np.sum(diff ** 2) / max(np.sum(ref ** 2), 1e-300)))}


def assert_grad_close(g, ref, record=None, what="dQ"):
    err = grad_errors(g, ref)
    if record:
        report(record, "backward_" + what, err)
    assert err["max_abs"] <= GRAD_MAX_ABS, (what, err)
    assert err["rel_l2"] < 2e-2, (what, err)          # not vacuous
