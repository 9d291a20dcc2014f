"""Writes tests/golden/config0_oracle.txt: reference values of the float64 oracle on the tiny configuration
(1 layer, 1 KV head, 1 query head, 4,096 fp32 pre-RoPE keys at positions 0..4095, query position 4,096,
budget 512, the 17 power-of-two offsets of Section 4.2).  Calls only the oracle and the seeded input generator.
The stored values guard the oracle against unintended change; they are not an independent pin (those are in
tests/test_oracle_pins.py).

    python tests/golden/make_config0_oracle.py
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle                                              # noqa: E402
from paper_2604_04921_b200 import workloads as W          # noqa: E402


def compute():
    sp = W.SPECS["tiny"]
    w = W.make_workload(sp, "cpu")
    k_pre = w.k_pre_fp32[0, 0, 0].double().numpy()
    raw = oracle.score_raw(k_pre, np.arange(sp.n_keys), sp.n_keys, w.q_center[0].double().numpy(),
                           w.q_mean_norm[0].double().numpy(), theta=sp.theta)
    _, s_final = oracle.normalize(raw)
    idx = oracle.select(s_final, sp.budget)
    return raw[0], s_final, idx


def render(raw, s_final, idx):
    probes = [0, 1, 2, 3, 511, 512, 1000, 2047, 2048, 4000, 4094, 4095]
    lines = ["# oracle on the tiny configuration; written by tests/golden/make_config0_oracle.py",
             "# slot  raw_score  final_score"]
    lines += [f"{i} {raw[i]:.12e} {s_final[i]:.12e}" for i in probes]
    lines.append(f"mean_raw {raw.mean():.12e}")
    lines.append(f"std_raw {raw.std():.12e}")
    lines.append(f"threshold_final {np.sort(s_final)[::-1][511]:.12e}")
    lines.append("kept_first16 " + " ".join(str(int(i)) for i in idx[:16]))
    lines.append("kept_sha256 " + hashlib.sha256(idx.astype("<i4").tobytes()).hexdigest())
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config0_oracle.txt")
    with open(out, "w") as f:
        f.write(render(*compute()))
    print("wrote", out)
