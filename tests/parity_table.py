"""Turns the per-workload parity records that the GPU tests leave (one JSON per workload in the parity records
folder, ``$MOC_PARITY_DIR`` if set) into one markdown table:  python tests/parity_table.py > profiles/parity_full_size.md"""
import glob
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def main():
    src = os.environ.get("MOC_PARITY_DIR", os.path.join(ROOT, "gpurun_out", "parity"))      # the default of tests/parity_utils.py
    recs = {os.path.basename(f)[:-5]: json.load(open(f)) for f in sorted(glob.glob(os.path.join(src, "*.json")))}
    order = [n for n in ("cfg0", "cfg1", "cfg2", "cfg4") if n in recs] + sorted(n for n in recs if n.startswith("cfg3")) + \
        sorted(n for n in recs if not n.startswith("cfg"))
    out = ["# Parity of the CUDA path against the fp64 oracle, per workload",
           "",
           "Written by `python tests/parity_table.py` from the records that `python -m pytest tests -m gpu` leaves under",
           "the parity records folder (one B200).  Routing is compared on EVERY row of the heads listed; a near-tie row is one whose",
           "GPU and oracle pick sets differ only in chunks whose oracle score lies within 1e-4 of the oracle's k-th score;",
           "`order` counts rows with equal sets whose order differs (`~` inside the near-tie window, `!` beyond it - must be 0).",
           "Attention is compared on sampled rows (half chunk edges, half uniform) at the full-size workloads and on every row",
           "of the small ones.  Bars: hard mismatches 0, near-tie rows <= 5e-4 of rows, O max-abs 2e-2, mean-abs 2e-3,",
           "LSE 2e-3, relative L2 2e-2, gradients max-abs 5e-2 and relative L2 2e-2.",
           "",
           "| workload | heads | routed rows | near-tie rows | hard | order ~ / ! | attn rows | O max-abs | O mean-abs | O rel-L2 | LSE max-abs | desc max-abs |",
           "|---|---|---|---|---|---|---|---|---|---|---|---|"]
    grads = []
    for n in order:
        r = recs[n]
        ro, at, de = r.get("routing", {}), r.get("attention", {}), r.get("descriptors", {})
        if ro or at:
            out.append("| %s | %s | %s | %s | %s | %s / %s | %s | %s | %s | %s | %s | %s |" % (
                n, ro.get("heads", ""), ro.get("rows", ""), ro.get("near_tie_rows", ""), ro.get("hard_mismatch_rows", ""),
                ro.get("order_near_tie_rows", ""), ro.get("order_wrong_rows", ""), at.get("rows", ""),
                "%.2e" % at["max_abs"] if at else "", "%.2e" % at["mean_abs"] if at else "", "%.2e" % at["rel_l2"] if at else "",
                "%.2e" % at["lse_max_abs"] if at else "", "%.1e" % de["max_abs"] if de else ""))
        for key, v in sorted(r.items()):
            if key.startswith("backward_"):
                grads.append("| %s | %s | %d | %.2e | %.2e | %.2e |" % (n, key[len("backward_"):], v["rows"], v["max_abs"], v["mean_abs"], v["rel_l2"]))
    out += ["", "## Backward (gradients against the oracle's, selection held constant)", "",
            "| workload | gradient | rows | max-abs | mean-abs | rel-L2 |", "|---|---|---|---|---|---|"] + grads
    extra = []
    for n in order:
        r = recs[n]
        if "outer_routing" in r:
            v = r["outer_routing"]
            extra.append("- `%s`: outer-loop routing of %d streams over %d shots, top-%d: %d stream(s) differ within the near-tie window; shot "
                         "descriptors max-abs %.1e, scores max-abs %.1e." % (n, v["streams"], v["shots"], v["top_m"], v["near_tie_streams"],
                                                                             v["desc_max_abs"], v["score_max_abs"]))
        if "regulariser" in r:
            v = r["regulariser"]
            extra.append("- `%s`: context drop-off / drop-in on %d rows: %d picks removed, %d chunks added, edited selection equal to the "
                         "oracle's bit for bit (%d mismatches)." % (n, v["rows"], v["picks_removed"], v["chunks_added"], v["selection_mismatches"]))
    if extra:
        out += ["", "## Other paths", ""] + extra
    sys.stdout.write("\n".join(out) + "\n")


if __name__ == "__main__":
    main()
