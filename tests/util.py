"""Helpers shared by the tests (no method arithmetic of the product lives here)."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def example_jobs():
    """The two jobs of tests/golden/worked_example.txt as a job table."""
    from paper_2108_03645_b200.inputs import JOB_DTYPE
    jobs = np.zeros(2, dtype=JOB_DTYPE)
    jobs[0] = (64, 128, 0, 5, 0.02, 0.0005, 0.01, 1.0)
    jobs[1] = (128, 64, 0, 5, 0.05, 0.001, 0.02, 1.0)
    return jobs


def golden_rows(kind):
    rows = []
    with open(os.path.join(GOLDEN, "worked_example.txt")) as fh:
        for line in fh:
            line = line.strip()
            if line.startswith(kind + " "):
                rows.append(line.split()[1:])
    return rows
