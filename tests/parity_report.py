"""Turn the parity log that the GPU tests write (one JSON record per compared tensor: error, noise floor,
allowance; see harness.log_parity) into a short table.

  LP_PARITY_LOG=parity.jsonl python -m pytest tests -m gpu -q
  python tests/parity_report.py parity.jsonl > summary.md
"""
import collections
import json
import sys

import numpy as np


def main(path):
    recs = [json.loads(line) for line in open(path)]
    bf = [r for r in recs if r["dtype"] == "bf16"]
    groups = collections.OrderedDict()
    for r in bf:
        groups.setdefault((r["test"].split("::")[-1], r["workload"]), []).append(r)
    print("| test | workload | tensors compared | error > 2e-2 | largest error (tensor; its floor; allowed) | largest floor | failed |")
    print("|---|---|---|---|---|---|---|")
    for (test, workload), rs in groups.items():
        worst = max(rs, key=lambda r: r["err"] / r["allowed"])
        big = max(rs, key=lambda r: r["err"])
        print("| `%s` | %s | %d | %d | %.4f (`%s`; %.4f; %.4f) | %.4f | %d |" % (
            test, workload, len(rs), sum(r["err"] >= 2e-2 for r in rs), big["err"], big["tensor"], big["floor"],
            big["allowed"], max(r["floor"] for r in rs), sum(not r["err"] < r["allowed"] for r in rs)))
        del worst
    ratio = np.array([r["err"] / r["floor"] for r in bf if r["floor"] > 0.02])
    print()
    print("Records: %d (bf16: %d, fp32: %d).  Error / floor over the %d bf16 records with a floor above 0.02: "
          "median %.2f, 90 %% %.2f, 99 %% %.2f, max %.2f." % (
              len(recs), len(bf), len(recs) - len(bf), ratio.size, *np.percentile(ratio, [50, 90, 99, 100])))
    f32 = [r for r in recs if r["dtype"] == "f32"]
    if f32:
        print("fp32 records: largest error %.2e (allowed 1e-4)." % max(r["err"] for r in f32))


if __name__ == "__main__":
    main(sys.argv[1])
