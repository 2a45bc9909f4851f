"""Writes tests/golden/oracle_f32_cases.txt: final states of the binary32 oracle on a few small
cases, as hexadecimal bit patterns. Calls nothing but the oracle. Re-run only when a change to
the oracle's arithmetic is intended (and say why in the commit message).

    python tests/golden/make_oracle_golden.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
import oracle  # noqa: E402

COORDS = np.array([0, 1, 2, 3, 1000, 4095, 2**32 + 6, 2**32 + 7], np.uint64)
CASES = {
    "nesterov_reset": dict(m=4, tau=4, T=3, alpha=1.0, beta=0.6, gamma=0.05, mu=0.9, sigma=0.1),
    "nesterov_average_wd": dict(m=5, tau=3, T=3, alpha=0.9, beta=0.7, gamma=0.1, mu=0.9, weight_decay=1e-4, a_lo=0.1,
                                a_hi=1.0, c_std=0.05, sigma=0.01, buffer_policy="average"),
    "adam_maintain": dict(m=3, tau=5, T=2, alpha=1.0, beta=0.5, gamma=5e-4, base="adam", adam_b1=0.9, adam_b2=0.98,
                          adam_eps=1e-8, a_lo=0.1, a_hi=1.0, c_std=0.02, sigma=0.01, buffer_policy="maintain"),
    "sgp_nesterov_reset": dict(m=8, tau=6, T=2, alpha=1.0, beta=0.6, gamma=0.1, base="sgp_nesterov", mu=0.9,
                               weight_decay=1e-4, a_lo=0.1, a_hi=1.0, c_std=0.05, sigma=0.01),
    "sgp_adam_no_average": dict(m=3, tau=4, T=2, alpha=1.0, beta=0.6, gamma=5e-4, base="sgp_adam", adam_b1=0.9,
                                adam_b2=0.98, adam_eps=1e-8, sigma=0.01, buffer_policy="maintain", no_average=True),
    "supplied_hash": dict(m=4, tau=3, T=2, alpha=1.0, beta=0.6, gamma=0.05, mu=0.9, sigma=0.1, grad_mode="supplied"),
}


def lines():
    for name, kw in CASES.items():
        out = oracle.run(oracle.make_config(**kw), j=COORDS, precision="f32")
        for key in ("x", "anchor", "u", "h", "v"):
            bits = np.ascontiguousarray(out[key], np.float32).reshape(-1).view(np.uint32)
            yield f"{name} {key} " + " ".join(f"{b:08x}" for b in bits)


if __name__ == "__main__":
    path = os.path.join(HERE, "oracle_f32_cases.txt")
    with open(path, "w") as f:
        f.write("# binary32 oracle, final state at coordinates " + " ".join(str(int(c)) for c in COORDS) + "\n")
        f.write("# written by tests/golden/make_oracle_golden.py (calls only oracle/); row-major, workers outermost\n")
        for line in lines():
            f.write(line + "\n")
    print(path)
