"""Writes tests/golden/config_optima.txt: the oracle's optimum for the named synthetic configs.

Only the seeded generators and the CPU oracle are called here; nothing comes from the CUDA
path.  Each line: name, input checksum, beta* as a C99 hex float (bit-exact), m, cuts, nodes.

    python tests/golden/make_golden.py
"""
from __future__ import annotations

import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from paper_2210_12219_b200 import workloads as W  # noqa: E402


def main():
    lines = ["# name checksum beta_hex m | cuts | nodes   (written by make_golden.py from oracle.dp_fact)"]
    cases = [W.config_tiny(), W.config_resnet50_shaped(), W.config_deeper_cnn(), W.config_large()]
    cases += W.config_batched(8)
    cases += [W.config_geometric(14, 64, 0), W.config_geometric(10, 64, 1, link="pairwise")]
    for inst in cases:
        sol = oracle.dp_fact(inst, oracle.max_threads())
        m, cuts, nodes = sol.plan()
        beta = "inf" if sol.status == oracle.INFEASIBLE else float(sol.beta_ms).hex()
        lines.append("%s %d %s %d | %s | %s" % (inst.name, inst.checksum(), beta, m,
                                                 " ".join(map(str, cuts)), " ".join(map(str, nodes))))
    with open(os.path.join(HERE, "config_optima.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")
    print("\n".join(lines))


if __name__ == "__main__":
    main()
