"""td_model_bytes (Eq. 1, Eq. 2, Eq. 4 of "Distributed Transfer Dock Strategy") against the
values the paper prints in Table 1 and against hand-worked cases.  Host arithmetic: no GPU."""
import os

import pytest

from paper_2507_19017_b200 import binding as td

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_tcv.txt")
GB = float(1 << 30)


def _rows():
    return [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]


def _printed(tok):
    """(value, tolerance) of a printed cell: one unit in the last printed digit."""
    if tok.endswith("K"):
        body = tok[:-1]
        digits = len(body.split(".")[1]) if "." in body else 0
        return float(body) * 1000.0, 1000.0 * 10.0 ** (-digits)
    digits = len(tok.split(".")[1]) if "." in tok else 0
    return float(tok), 10.0 ** (-digits)


@pytest.mark.parametrize("row", _rows())
def test_tcv_matches_table1(row):
    G, N, PL, n, SL, M = map(int, row[:6])
    _cv, tcv, _dock = td.model_bytes(G, N, PL, n, SL, M, 4, 0, 1)
    want, tol = _printed(row[6])
    assert abs(tcv / GB - want) <= tol
    t100, tol100 = _printed(row[7])                 # seconds over a 100 MB/s link
    assert abs(tcv / (100.0 * (1 << 20)) - t100) <= max(tol100, 1e-3 * t100)
    t1k, tol1k = _printed(row[8])                   # seconds over a 1 GB/s link
    assert abs(tcv / GB - t1k) <= tol1k


def test_terms_by_hand():
    # Eq. 1: the prompt once, n response-length items, M scalars, per sample and byte width
    assert td.model_bytes(1, 1, 7, 0, 0, 0, 1)[0] == 7
    assert td.model_bytes(1, 1, 0, 3, 5, 0, 1)[0] == 15
    assert td.model_bytes(2, 3, 0, 0, 0, 5, 4)[0] == 2 * 3 * 4 * 5
    # Eq. 2: two prompts, three response blocks, eight scalar blocks
    assert td.model_bytes(1, 1, 1, 0, 0, 0, 1)[1] == 2
    assert td.model_bytes(1, 1, 0, 1, 1, 0, 1)[1] == 3
    assert td.model_bytes(1, 1, 0, 0, 0, 1, 1)[1] == 8
    # Eq. 4: one warehouse and no controller is Eq. 2; S warehouses share evenly; each extra
    # controller adds 8*M per sample
    a = (256, 8, 2048, 5, 8192, 3, 4)
    assert td.model_bytes(*a, 0, 1)[2] == td.model_bytes(*a)[1]
    assert td.model_bytes(*a, 0, 16)[2] == td.model_bytes(*a)[1] / 16
    assert td.model_bytes(*a, 6, 1)[2] - td.model_bytes(*a, 5, 1)[2] == 256 * 8 * 4 * 8 * 3


def test_rejects_overflow_and_zero_warehouses():
    with pytest.raises(td.TdError):
        td.model_bytes(1 << 40, 1 << 40, 1, 0, 0, 0, 1)
    with pytest.raises(td.TdError):
        td.model_bytes(1, 1, 1, 0, 0, 0, 1, 0, 0)
