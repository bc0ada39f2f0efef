"""Reporting conventions (host arithmetic only; no data path).

The paper's bandwidth table (section 5.3.3, Table 1) reports per-direction GB/s and an end-to-end
time for a fixed payload per direction: with the directions run one after the other ("u") the
end-to-end time is the sum of the two transfer times; with both in flight ("b") it is the time of
the slower one.  GB means 1e9 bytes here; GiB figures are given beside it where useful.
"""
from __future__ import annotations

import statistics
from typing import Iterable, Sequence


def e2e_ms(bytes_out: float, bytes_in: float, d2h_gbs: float, h2d_gbs: float, concurrent: bool) -> float:
    t_out = bytes_out / (d2h_gbs * 1e9) * 1e3 if bytes_out else 0.0
    t_in = bytes_in / (h2d_gbs * 1e9) * 1e3 if bytes_in else 0.0
    return max(t_out, t_in) if concurrent else t_out + t_in


def gbs(nbytes: float, ms: float) -> float:
    return nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0


def duplex_ideal_ms(bytes_out: float, bytes_in: float, p_d2h: float, p_h2d: float, p_bi: float) -> float:
    """Best time the probed link allows for an unbalanced rotation: both directions share the
    measured bidirectional rate until the smaller payload is done, the rest runs alone."""
    small = min(bytes_out, bytes_in)
    rest_out, rest_in = bytes_out - small, bytes_in - small
    t = 2 * small / (p_bi * 1e9)
    t += rest_out / (p_d2h * 1e9) + rest_in / (p_h2d * 1e9)
    return t * 1e3


def percentile(xs: Sequence[float], q: float) -> float:
    xs = sorted(xs)
    if not xs:
        return float("nan")
    k = (len(xs) - 1) * q
    lo, hi = int(k), min(int(k) + 1, len(xs) - 1)
    return xs[lo] + (xs[hi] - xs[lo]) * (k - lo)


def median(xs: Iterable[float]) -> float:
    return statistics.median(list(xs))


def reduce_over_ranks(x: float, op: str, dist=None, device: str = "cpu") -> float:
    """Maximum or sum of a per-rank number over the ranks of an initialised ``torch.distributed`` group
    (``dist`` is the module; ``None`` = single process).  Replicas are timed as the slowest rank and
    their bytes are added: job GB/s = sum of bytes / max of time."""
    if dist is None:
        return float(x)
    import torch
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def replicas_gbs(bytes_per_rank: float, ms_per_rank: float, dist=None, device: str = "cpu") -> float:
    """Whole-job GB/s of independent replicas: every rank's bytes over the slowest rank's time."""
    total = reduce_over_ranks(bytes_per_rank, "sum", dist, device)
    slowest = reduce_over_ranks(ms_per_rank, "max", dist, device)
    return gbs(total, slowest)
