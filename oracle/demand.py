"""Eq. 3 of the paper (Section 5.1): expected number of distinct adapters a batch needs.

    Low_lora = sum_i (1 - (1 - prob_i)^BS)

Used here only to check the synthetic batch generator's adapter popularity sampling.
Pin: uniform popularity over n adapters gives n (1 - (1 - 1/n)^BS); BS = 1 gives 1.
"""
import numpy as np


def expected_distinct(prob, batch_size):
    prob = np.asarray(prob, dtype=np.float64)
    return float(np.sum(1.0 - (1.0 - prob) ** batch_size))
