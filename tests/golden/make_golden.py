"""Writes the stored expected values under tests/golden/ by calling only the CPU oracle.

    python tests/golden/make_golden.py

The paper prints no worked numeric example of the optimizer step, so there is no value of the
paper's to store. What is stored instead are outputs of the oracle on tiny seeded cases, so that a
later change to the oracle's arithmetic shows up as a diff of these files (a change must name, in
its commit message, the passage of the paper that justifies it).
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import lordo_oracle as lo  # noqa: E402


def tiny_run(variant: int, form: int) -> np.ndarray:
    rng = np.random.default_rng(123)
    m, n, r, K = 8, 8, 8 if variant == 1 else 4, 2
    cfg = lo.OracleConfig(mats=((m, n, r),), K=K, H=2, variant=variant, beta2=0.999, eps=1e-8, clip_rho=1.0,
                          outer=lo.OUTER_NESTEROV, outer_lr=0.8, outer_momentum=0.9, seed=5, state_dtype="f64", w_dtype="f64",
                          e_dtype="f64")
    orc = lo.LordoOracle(cfg, [rng.standard_normal((m, n)) * 0.02])
    grads = [[rng.standard_normal((K, m, n))] for _ in range(4)]
    lo.run_rounds(orc, lambda rnd, h: grads[2 * rnd + h], 2, 0.004, 0.9, 0.9, form)
    return orc.W[0][0]


def main():
    np.savetxt(os.path.join(HERE, "generator_seed7_purpose2_mat5_index3_replica2_4x8.txt"),
               lo.random_matrix(7, 2, 5, 3, 2, 4, 8), fmt="%d",
               header="oracle.random_matrix(7, 2, 5, 3, 2, 4, 8): centred Binomial(64, 1/2) integers of the counter-based generator")
    for variant, form, name in ((0, 2, "global_fullqhm"), (1, 1, "local_lowqhm")):
        np.savetxt(os.path.join(HERE, f"tiny_8x8_{name}_weights.txt"), tiny_run(variant, form), fmt="%.17e",
                   header=f"oracle weights of worker 0 after 2 rounds of 2 steps, 8x8, Algorithm {1 + variant}, QHM form {form} (fp64 states)")


if __name__ == "__main__":
    main()
