"""Turn a report of measured parity counts (written by `GS_PARITY_MEASURE=1 GS_PARITY_REPORT=<file> pytest tests -m gpu`
on a B200) into tests/parity_bounds.json, the records that gpu_helpers.check_bound holds later runs to (at most
twice the record).  Usage: python tests/make_parity_bounds.py <report.json> [--merge | --max]
(--merge keeps the records of the cases the report does not cover, e.g. after re-measuring one test file; --max also
keeps, per record, the larger of the stored value and the new measurement: the gradient sums are accumulated by
atomics, so a count of near-threshold values varies by a few from run to run, and the record is the largest seen)."""
import json
import os
import sys


def main(path, merge=False, keep_max=False):
    rows = json.load(open(path))
    dst = os.path.join(os.path.dirname(os.path.abspath(__file__)), "parity_bounds.json")
    old = json.load(open(dst)) if (merge or keep_max) and os.path.exists(dst) else {}
    out = {}
    for r in rows:
        par = r.get("parameter", "")
        for k, v in r.items():
            if k in ("case", "check", "parameter"):
                continue
            name = "|".join((r["case"], r["check"], par, k))
            out[name] = max(out.get(name, 0), v)          # a case visited twice keeps its larger measurement
    if keep_max:
        out = {k: max(v, old.get(k, v)) for k, v in out.items()}
    out = {**old, **out}
    with open(dst, "w") as f:
        json.dump(dict(sorted(out.items())), f, indent=0)
    print(f"{len(out)} records -> {dst}")


if __name__ == "__main__":
    main(sys.argv[1], merge="--merge" in sys.argv[2:], keep_max="--max" in sys.argv[2:])
