"""Pins for the communication-volume model (Eq. 1, Eq. 2, Eq. 4) against the
values the paper prints in Table 1."""
import os

import pytest

from oracle import td_oracle as ora

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_tcv.txt")


def _rows():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        rows.append(line.split())
    return rows


def _printed(tok):
    """(value, absolute tolerance) of a printed table cell: half a unit in the last
    printed digit, a whole unit where the paper truncated instead of rounding."""
    if tok.endswith("K"):
        body = tok[:-1]
        digits = len(body.split(".")[1]) if "." in body else 0
        return float(body) * 1000.0, 1000.0 * 10.0 ** (-digits)
    digits = len(tok.split(".")[1]) if "." in tok else 0
    return float(tok), 10.0 ** (-digits)


def test_table1_has_six_rows():
    assert len(_rows()) == 6


@pytest.mark.parametrize("row", _rows())
def test_tcv_matches_table1(row):
    G, N, PL, n, SL, M = map(float, row[:6])
    tcv = ora.tcv(G, N, 4, PL, n, SL, M)
    want, tol = _printed(row[6])
    assert abs(tcv - want) <= tol, (tcv, want)
    t100, tol100 = _printed(row[7])
    assert abs(tcv * 1024.0 / 100.0 - t100) <= max(tol100, 1e-3 * t100)
    t1k, tol1k = _printed(row[8])
    assert abs(tcv - t1k) <= tol1k


def test_eq4_reduces_to_eq2():
    # one warehouse, no controller broadcast: Eq. 4 is Eq. 2
    args = (256, 8, 4, 2048, 5, 8192, 3)
    assert ora.tcv_dock(*args, 0, 1) == pytest.approx(ora.tcv(*args), rel=1e-15)
    # S warehouses share the payload evenly
    assert ora.tcv_dock(*args, 0, 16) == pytest.approx(ora.tcv(*args) / 16, rel=1e-15)
    # the metadata term grows by 8*M*(G*N*B) per extra controller
    d = ora.tcv_dock(*args, 6, 1) - ora.tcv_dock(*args, 5, 1)
    assert d == pytest.approx(256 * 8 * 4 * 8 * 3 / 1024 ** 3, rel=1e-12)


def test_eq1_terms():
    # CV counts the prompt once, n response-length items and M scalars per sample
    assert ora.cv(1, 1, 1, 7, 0, 0, 0) * 1024 ** 3 == pytest.approx(7)
    assert ora.cv(1, 1, 1, 0, 3, 5, 0) * 1024 ** 3 == pytest.approx(15)
    assert ora.cv(2, 3, 4, 0, 0, 0, 5) * 1024 ** 3 == pytest.approx(2 * 3 * 4 * 5)
    # and Eq. 2 is 2 prompts + 3 response blocks + 8 scalar blocks
    assert ora.tcv(1, 1, 1, 1, 0, 0, 0) * 1024 ** 3 == pytest.approx(2)
    assert ora.tcv(1, 1, 1, 0, 1, 1, 0) * 1024 ** 3 == pytest.approx(3)
    assert ora.tcv(1, 1, 1, 0, 0, 0, 1) * 1024 ** 3 == pytest.approx(8)
