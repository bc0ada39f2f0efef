"""The reporting convention must reproduce the paper's Table 1 arithmetic."""
import pytest

from conftest import read_golden
from paper_2601_20309_b200 import metrics as M


def test_table1_end_to_end_times():
    g = read_golden("table1.txt")
    payload = g["payload_gb"] * 1e9
    for row in ("naive", "ms", "ms_mk", "ideal"):
        d2h, h2d, e2e, conc = g[row]
        got = M.e2e_ms(payload, payload, d2h, h2d, bool(conc))
        assert got == pytest.approx(e2e, rel=2e-3), row


def test_duplex_ideal_and_percentiles():
    # balanced: both payloads at the bidirectional rate
    assert M.duplex_ideal_ms(1e9, 1e9, 50, 50, 80) == pytest.approx(25.0)
    # unbalanced: the remainder of the larger payload runs alone
    assert M.duplex_ideal_ms(1e9, 3e9, 50, 40, 80) == pytest.approx(25.0 + 50.0)
    assert M.percentile([1, 2, 3, 4, 5], 0.5) == 3 and M.percentile([1, 2], 0.5) == 1.5
    assert M.gbs(2e9, 1000.0) == pytest.approx(2.0)
