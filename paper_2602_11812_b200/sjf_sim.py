"""Host-side simulator of length-aware batching (the consumer of the predictions; paper Sec. 4.4, App. B).

A static-batching model: requests are ordered by predicted output length (shortest job first),
cut into batches of `batch_size`, and every batch decodes until its longest member finishes, so a
batch of true lengths L_1..L_k allocates k * max(L) token slots for sum(L) useful ones.
Metrics follow the paper's appendix definitions:
  padding ratio = (R_allocated - R_actual) / R_actual,
  job completion time = completion - submission (all jobs submitted at t = 0, batches run back to back,
  one time unit per decode step),
  throughput = completed jobs / total time.
No GPU work; inputs are synthetic length arrays.  MAE is included for completeness.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class BatchingResult:
    padding_ratio: float
    mean_jct: float
    throughput: float
    total_time: float
    order: np.ndarray


def mean_absolute_error(y_true, y_pred) -> float:
    y_true = np.asarray(y_true, dtype=np.float64)
    y_pred = np.asarray(y_pred, dtype=np.float64)
    return float(np.abs(y_true - y_pred).mean())


def simulate_batches(true_len, order, batch_size: int) -> BatchingResult:
    """Runs the requests in the given order, `batch_size` at a time."""
    true_len = np.asarray(true_len, dtype=np.int64)
    order = np.asarray(order, dtype=np.int64)
    if sorted(order.tolist()) != list(range(len(true_len))):
        raise ValueError("order must be a permutation of the requests")
    if batch_size <= 0:
        raise ValueError("batch_size must be positive")
    allocated, t, jct_sum = 0, 0, 0.0
    for i in range(0, len(order), batch_size):
        lens = true_len[order[i:i + batch_size]]
        steps = int(lens.max())
        allocated += steps * len(lens)
        jct_sum += float((t + lens).sum())          # a job leaves when its own last token is out
        t += steps
    actual = int(true_len.sum())
    return BatchingResult(padding_ratio=(allocated - actual) / actual, mean_jct=jct_sum / len(true_len),
                          throughput=len(true_len) / t, total_time=float(t), order=order)


def sjf_order(pred_len) -> np.ndarray:
    """Shortest predicted job first; ties keep submission order."""
    return np.argsort(np.asarray(pred_len, dtype=np.float64), kind="stable")


def compare_policies(true_len, pred_len, batch_size: int) -> dict:
    """FCFS, SJF on the predictions, and SJF on the true lengths (the bound a perfect predictor reaches)."""
    n = len(true_len)
    return dict(fcfs=simulate_batches(true_len, np.arange(n), batch_size),
                sjf_predicted=simulate_batches(true_len, sjf_order(pred_len), batch_size),
                sjf_oracle=simulate_batches(true_len, sjf_order(true_len), batch_size),
                mae=mean_absolute_error(true_len, pred_len))
