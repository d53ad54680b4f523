"""Writes tests/golden/c1_oracle_trace.txt: what the CPU oracle retains, block by block, on the smallest
benchmark configuration (C1: 24x24 vision tokens + 32 text tokens, blocks of 64, budget 128, fp32 inputs),
plus a few log-sum-exp values and scores.  The paper prints no worked numeric example, so this file pins
the oracle against silent changes of its own arithmetic (a regression fixture), not against the paper;
what ties the oracle to the paper are the pins in tests/test_oracle_pins.py.  Calls only oracle/ and the
input generator:  python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle.kvc_oracle import KVCOracle                      # noqa: E402
from paper_2604_16734_b200.workloads import CONFIGS, Workload  # noqa: E402


def trace_lines():
    cfg = CONFIGS["C1"]
    q, k, v = (x.double().numpy() for x in Workload(cfg).layer(0))
    orc = KVCOracle(1, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.budget, cfg.obs_window)
    lines = ["# block pos0 n | evicted | sha1 of the retained positions | first 8 retained | lse[row 0, head 0] | max score"]
    for pos0, n in cfg.chunks():
        res = orc.prefill_chunk(0, q[pos0:pos0 + n], k[pos0:pos0 + n], v[pos0:pos0 + n], pos0)
        ret = res.retained_pos[0]
        digest = hashlib.sha1(np.asarray(ret, dtype=np.int64).tobytes()).hexdigest()[:16]
        top = f"{res.score[0].max():.9e}" if res.evicted else "-"
        lines.append(f"{pos0} {n} | {int(res.evicted)} | {digest} | {' '.join(map(str, ret[:8].tolist()))} | "
                     f"{res.lse[0, 0]:.9e} | {top}")
    return lines


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_oracle_trace.txt")
    with open(path, "w") as f:
        f.write("\n".join(trace_lines()) + "\n")
    print("wrote", path)
