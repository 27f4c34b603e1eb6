"""Turn a report of measured parity counts (written by `GS_PARITY_MEASURE=1 GS_PARITY_REPORT=<file> pytest tests -m gpu`
on a B200) into tests/parity_bounds.json, the records that gpu_helpers.check_bound holds later runs to (at most
twice the record).  Usage: python tests/make_parity_bounds.py <report.json> [--merge]
(--merge keeps the records of the cases the report does not cover, e.g. after re-measuring one test file)."""
import json
import os
import sys


def main(path, merge=False):
    rows = json.load(open(path))
    dst = os.path.join(os.path.dirname(os.path.abspath(__file__)), "parity_bounds.json")
    old = json.load(open(dst)) if merge and os.path.exists(dst) else {}
    out = {}
    for r in rows:
        par = r.get("parameter", "")
        for k, v in r.items():
            if k in ("case", "check", "parameter"):
                continue
            name = "|".join((r["case"], r["check"], par, k))
            out[name] = max(out.get(name, 0), v)          # a case visited twice keeps its larger measurement
    out = {**old, **out}
    with open(dst, "w") as f:
        json.dump(dict(sorted(out.items())), f, indent=0)
    print(f"{len(out)} records -> {dst}")


if __name__ == "__main__":
    main(sys.argv[1], merge="--merge" in sys.argv[2:])
