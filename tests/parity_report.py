"""Summarises parity_errors.jsonl (written by a `-m gpu` test session into PARITY_REPORT_DIR, default parity_report/
at the repository root) as a markdown table:
per tensor, the worst raw figures over all comparisons of that tensor in the chosen tests.

    python tests/parity_report.py [substring of the test id ...]
"""
import json
import os
import sys
from collections import defaultdict

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def main(argv):
    path = os.path.join(os.environ.get("PARITY_REPORT_DIR") or os.path.join(ROOT, "parity_report"), "parity_errors.jsonl")
    recs = [json.loads(l) for l in open(path)]
    if argv:
        recs = [r for r in recs if any(a in r["test"] for a in argv)]
    groups = defaultdict(list)
    for r in recs:
        base = r["tensor"].split("[")[0].split(" ")[0]
        groups[(base, r["kind"])].append(r)
    print("| tensor | tolerance class | comparisons | max rel err (|ref| >= rms/16) | max abs err / rms | worst err / tol | worst err / tol without allowance |")
    print("|---|---|---|---|---|---|---|")
    for (name, kind), rs in sorted(groups.items()):
        print("| %s | %s | %d | %.2e | %.2e | %.2f | %.2f |" % (
            name, kind, len(rs), max(r["max_rel_err_big"] for r in rs), max(r["max_abs_err_over_rms"] for r in rs),
            max(r["worst_over_tol"] for r in rs), max(r["worst_over_tol_no_extra"] for r in rs)))


if __name__ == "__main__":
    main(sys.argv[1:])
