"""Writes tests/golden/c5_skew_13b_select_bias.txt: the selection bias b (Eq. final_gate) that
skews the routed load of the 13B-shaped workload towards Zipf(1.2) shares.  Calls only the
oracle: router scores on the workload's seeded tokens (Eq. router), then the paper's bias
update rule (Section 4.3) with the clipped Zipf shares as target, iterated to convergence.
Run from the repository root:  python tests/golden/make_c5_select_bias.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import cmoe_oracle as oracle  # noqa: E402
from paper_2502_04416_b200 import workloads as wl  # noqa: E402

NAME = "c5_skew_13b"


def main():
    w = wl.WORKLOADS[NAME]
    inp = wl.make_inputs(w)
    lay = inp.layers[0]
    s = oracle.router_scores(inp.x, lay.w_gate, lay.w_up, lay.rep_idx)
    target = wl.zipf_target_shares(w.shape.n_routed, w.shape.top_k, w.zipf_s)
    b, counts = oracle.fit_select_bias(s, w.shape.top_k, target)
    share = counts / counts.sum()
    path = os.path.join(ROOT, "tests", "golden", f"{NAME}_select_bias.txt")
    with open(path, "w") as f:
        f.write(f"# selection bias b[j], j = 0..{len(b) - 1}, for workload {NAME} (seed {w.seed}, T = {w.t_max});\n")
        f.write("# written by tests/golden/make_c5_select_bias.py from the oracle's router scores and the\n")
        f.write("# paper's bias-update rule; target shares = Zipf(1.2) clipped at 1/N_k.\n")
        f.write("# achieved shares: " + " ".join(f"{p:.4f}" for p in share) + "\n")
        f.write("# max |share - target| = %.4f\n" % np.abs(share - target).max())
        for v in b:
            f.write(f"{np.float32(v):.9g}\n")
    print(path, "max dev", np.abs(share - target).max())


if __name__ == "__main__":
    main()
