"""Writes tests/golden/oracle_cfg0.txt from the fp64 oracle alone (no CUDA code is involved).

The paper prints no worked numeric example, so this file is not a value from the paper: it freezes
what the pinned oracle computes on the tiny config, so that a later change to the oracle's arithmetic
shows up as a diff of this file and has to be justified.

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ea_oracle  # noqa: E402
from paper_2510_00636_b200 import inputs  # noqa: E402  (seeded input generator only)


def compute():
    cfg = inputs.CONFIGS[0].tempered(2.0)
    q, k, v, pos = inputs.generate_layer(cfg)
    ref = ea_oracle.compress(inputs.bits(q), inputs.bits(k), inputs.bits(v), pos.numpy(), cfg.n_future,
                             cfg.rope_base, cfg.eps, cfg.n_kept)
    keys = [0, 1, 17, 100, 255, 256, 511]
    return {
        "logits_head0": ref["logits"][0, 0, keys],
        "logits_head3": ref["logits"][0, 3, keys],
        "scores_kv0": ref["scores"][0, 0, keys],
        "scores_kv1": ref["scores"][0, 1, keys],
        "kept_kv0_first16": ref["kept_idx"][0, 0, :16].astype(np.float64),
        "kept_kv1_last16": ref["kept_idx"][0, 1, -16:].astype(np.float64),
        "kept_sum": np.array([ref["kept_idx"][0, 0].sum(), ref["kept_idx"][0, 1].sum()], np.float64),
    }


def main():
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_cfg0.txt")
    with open(out, "w") as f:
        f.write("# fp64 oracle on cfg0-tiny with outlier scale x2 (seed 0); written by make_golden.py\n")
        f.write("# no value of the paper: the paper prints no worked example (Sec. 2.2 gives formulas only)\n")
        for name, vals in compute().items():
            f.write(name + " " + " ".join(repr(float(x)) for x in vals) + "\n")
    print(out)


if __name__ == "__main__":
    main()
