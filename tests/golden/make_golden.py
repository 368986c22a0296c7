"""Writes the stored expected values under tests/golden/ by calling ONLY the CPU oracle
(and the seeded input generators).  The paper prints no iterates or worked numerical example,
so nothing here is a value of the paper's: these files freeze the oracle's own output on the
first configuration as stated (n = 4 directed ring, least squares p = 10, 50 rows per worker,
alpha = 0.01, 200 rounds, seed 0), so that an accidental change of the oracle's arithmetic or of
the generators shows up as a diff.  A deliberate change re-runs this script and says why in
its commit message.

    python tests/golden/make_golden.py
"""

from __future__ import annotations

import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import from_workload, make_model, run_schedule   # noqa: E402
from workloads import build_config                            # noqa: E402


def compute():
    wl = build_config("ls_ring4", seed=0)
    orc = from_workload(wl, make_model(wl).grad)
    run_schedule(orc, wl.schedule)
    return orc


def main():
    orc = compute()
    head = ("R-FAST oracle, configuration 1 as stated (Algorithm 1 over the seeded schedule), after 200 rounds.\n"
            "Not a value printed in the paper (it prints none); written by tests/golden/make_golden.py.\n")
    np.savetxt(os.path.join(HERE, "ls_ring4_x_after_200_rounds.txt"), orc.X(), fmt="%.17e",
               header=head + "x_i, one row per node")
    np.savetxt(os.path.join(HERE, "ls_ring4_z_after_200_rounds.txt"), orc.Z(), fmt="%.17e",
               header=head + "tracker z_i, one row per node")
    np.savetxt(os.path.join(HERE, "ls_ring4_stamps.txt"),
               np.array([orc.t + orc.tau_v + orc.tau_rho]), fmt="%d",
               header=head + "local counters t_i (4), then tau_v per G_R edge (4), then tau_rho per G_C edge (4)")


if __name__ == "__main__":
    main()
