"""Host-side logic that needs no GPU: the multi-rank path of the benchmark (independent replicas,
slowest-rank timing, whole-job value) run as two gloo ranks on the CPU, per-rank seeding of the
workloads, and that the C-ABI library exports every symbol its header declares."""
import ctypes
import os
import re
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import Oracle
    from paper_2508_21058_b200 import workloads as W
    # every rank is a replica with its own seed and no data-path exchange
    wl = W.workload("cfg0", seed=rank)
    x = W.generate(wl, "cpu", ("q", "k", "v"))
    orc = Oracle.from_workload(wl)
    h = {n: W.as_u16(t) for n, t in x.items()}
    sel = orc.route(h["q"], orc.chunk_pool(h["k"]))
    pairs = orc.pair_count(sel)
    local_ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
    ms = bench.max_over_ranks_ms(local_ms, world, "cpu")
    value = bench.job_value(bench.step_flops(wl, pairs, False), world, ms)
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([ms, value, pairs, float(x["q"].float().sum())]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_slowest_rank_and_whole_job_value(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [np.load(tmp_path / f"r{i}.npy") for i in range(world)]
    assert r[0][0] == r[1][0] == 20.0                  # max over ranks, seen by every rank
    assert r[0][3] != r[1][3]                          # different seeds, different inputs
    sys.path.insert(0, ROOT)
    import bench
    from paper_2508_21058_b200 import workloads as W
    wl = W.workload("cfg0")
    for i in range(world):
        assert r[i][1] == pytest.approx(world * 4.0 * wl.head_dim * r[i][2] / 20e-3 / 1e12)


def test_library_exports_every_declared_symbol():
    sys.path.insert(0, ROOT)
    from paper_2508_21058_b200 import build, lib_path
    build.build()
    lib = ctypes.CDLL(lib_path())
    header = open(os.path.join(ROOT, "include", "moc.h")).read()
    names = set(re.findall(r"\b(moc_[a-z_0-9]+)\s*\(", header))
    assert {"moc_plan_create", "moc_chunk_pool", "moc_route", "moc_attend", "moc_attend_bwd",
            "moc_chunk_pool_noalloc"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_plan_rejects_bad_arguments_without_a_device():
    """Argument checks that precede any CUDA call give their codes on a machine with no GPU."""
    sys.path.insert(0, ROOT)
    from paper_2508_21058_b200 import MocError, MocPlan
    from paper_2508_21058_b200 import workloads as W
    lay = W.make_layout(1, 8, 2, 16)
    with pytest.raises(MocError) as e:
        MocPlan(2, lay.n_tokens, 96, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 2)
    assert e.value.code == -2
    bad = lay.chunk_off.copy(); bad[1] = 0
    with pytest.raises(MocError) as e:
        MocPlan(2, lay.n_tokens, 64, bad, lay.chunk_shot, lay.chunk_mod, 2)
    assert e.value.code == -3
    with pytest.raises(MocError) as e:
        MocPlan(2, lay.n_tokens, 64, lay.chunk_off, lay.chunk_shot, lay.chunk_mod, 600)
    assert e.value.code == -2


def test_roofline_objects_follow_from_the_segment_times():
    """The fractions the benchmark prints are plain arithmetic on the segment times, the pair count and the
    peaks: recomputed here by hand; the attention peak is the sustained one only for a long timed region."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2508_21058_b200 import workloads as W
    wl = W.workload("cfg1")
    peaks = {"hbm_gbs": 6000.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    pairs = 5_000_000_000
    r = {"seg": [0.05, 0.06, 3.5], "pairs": pairs, "timed_ms": 80.0}
    roof, routing = bench.rooflines(wl, r, peaks, "measured")
    att = 4.0 * wl.head_dim * pairs / 3.5e-3 / 1e12
    assert roof["achieved"] == pytest.approx(att) and roof["peak"] == 1600.0
    assert roof["frac"] == pytest.approx(att / 1600.0) == pytest.approx(roof["frac_of_burst"])
    assert roof["frac_of_sustained"] == pytest.approx(att / 1400.0)
    H, L, d, C, k = wl.n_heads, wl.n_tokens, wl.head_dim, wl.n_chunks, wl.top_k
    bytes_ = 2.0 * 2 * L * d * H + 4.0 * k * L * H + 2 * 4.0 * C * d * H
    assert routing["achieved"] == pytest.approx(bytes_ / 0.11e-3 / 1e9)
    assert routing["frac"] == pytest.approx(routing["achieved"] / 6000.0)
    roof_long, _ = bench.rooflines(wl, dict(r, timed_ms=1300.0), peaks, "measured")
    assert roof_long["peak"] == 1400.0 and roof_long["frac"] == pytest.approx(att / 1400.0)


def test_traffic_figure_is_dropped_when_the_kernel_source_has_changed(tmp_path, monkeypatch):
    sys.path.insert(0, ROOT)
    import hashlib
    import bench
    (tmp_path / "profiles").mkdir()
    (tmp_path / "k.cu").write_text("kernel v1")
    sha = hashlib.sha1(b"kernel v1").hexdigest()
    (tmp_path / "profiles" / "traffic.txt").write_text(f"# comment\nmoc_attend cfgX 1.5e+09 {sha} k.cu\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.measured_traffic("moc_attend", "cfgX") == 1.5e9
    assert bench.measured_traffic("moc_attend", "other") is None
    (tmp_path / "k.cu").write_text("kernel v2")
    assert bench.measured_traffic("moc_attend", "cfgX") is None


def test_both_arms_describe_the_workload_with_the_same_config():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2508_21058_b200 import workloads as W
    wl = W.workload("cfg2")
    a, b = bench.config_of(wl, False, 1), bench.config_of(W.workload("cfg2"), False, 1)
    assert a == b and a["workload"] == "cfg2" and a["tokens"] == 264128 and a["top_k"] == 6 and a["backward"] is False
