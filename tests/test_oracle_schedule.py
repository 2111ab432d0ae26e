"""Pins for the oracle's retention schedule: the paper's printed table rows and closed forms."""
import math
import os

import pytest

from oracle.st3_oracle import Schedule, conserved_fraction_bp

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pvtp_conserved_fraction.txt")


def _rows():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            model, L, S, R, C = line.split()
            out.append((model, int(L), int(S), float(R), float(C)))
    return out


def test_golden_has_all_rows():
    assert len(_rows()) == 60


@pytest.mark.parametrize("model,L,S,R,C", _rows())
def test_conserved_fraction_matches_paper_tables(model, L, S, R, C):
    r_bp = round(R * 100)
    assert abs(r_bp - R * 100) < 1e-9          # every printed R is a whole number of basis points
    assert conserved_fraction_bp(L, S, r_bp) == round(C * 100)


def test_printed_eq9_disagrees_only_when_S_divides_L_minus_3():
    """Eq. 9 as printed (floor((L-3)/S)) is off by one R exactly for the S = 1 rows."""
    bad = 0
    for model, L, S, R, C in _rows():
        printed = 100.0 - ((L - 3) // S) * R - 50.0
        if abs(printed - C) > 1e-9:
            bad += 1
            assert (L - 3) % S == 0
    assert bad == 10


def test_first_three_layers_exempt_and_stage_heads():
    s = Schedule(num_layers=32, num_visual=576, stride=7, step_ratio_bp=1225, tau=256)
    assert [s.stage(l) for l in range(4)] == [-1, -1, -1, 0]
    heads = [l for l in range(32) if l >= 3 and (l - 3) % 7 == 0]       # Algorithm 1's condition
    assert heads == [3, 10, 17, 24, 31]
    for l in range(3, 32):
        assert s.stage(l) == sum(1 for h in heads if h <= l) - 1


def test_worked_counts_7b_13b_next():
    s7 = Schedule(num_layers=32, num_visual=576, stride=7, step_ratio_bp=1225, tau=256)
    n = [s7.n0(l) for l in range(32)]
    assert n[:3] == [576] * 3 and n[3:10] == [288] * 7 and n[10:17] == [217] * 7
    assert n[17:24] == [146] * 7 and n[24:31] == [76] * 7 and n[31] == 5
    assert sum(n) == 6822
    s13 = Schedule(num_layers=40, num_visual=576, stride=4, step_ratio_bp=500, tau=512)
    n13 = [s13.n0(l) for l in range(40)]
    assert n13[3::4] == [288, 259, 230, 201, 172, 144, 115, 86, 57, 28]
    assert sum(n13) == 7964
    sn = Schedule(num_layers=32, num_visual=2880, stride=7, step_ratio_bp=1225, tau=1024)
    assert sorted(set(sn.n0(l) for l in range(32)), reverse=True) == [2880, 1440, 1087, 734, 381, 28]
    assert sum(sn.n0(l) for l in range(32)) == 34162


def test_beta_closed_forms():
    s = Schedule(num_layers=32, num_visual=576, stride=7, step_ratio_bp=1225, tau=50)
    assert s.beta(0) == 1.0
    assert s.beta(50) == 0.0 and s.beta(51) == 0.0 and s.beta(10 ** 6) == 0.0
    assert abs(s.beta(25) - math.sqrt(0.5)) < 1e-15          # cos(pi/4)
    b = [s.beta(t) for t in range(0, 51)]
    d1 = [b[i + 1] - b[i] for i in range(50)]
    assert all(x < 0 for x in d1)                            # strictly decreasing on [0, tau]
    d2 = [d1[i + 1] - d1[i] for i in range(48)]              # (last interval ends on the cut-off)
    assert all(x < 0 for x in d2)                            # concave: decay accelerates


def test_vta_counts():
    s = Schedule(num_layers=32, num_visual=576, stride=7, step_ratio_bp=1225, tau=256)
    assert s.n(3, 128) == 203                                # floor(288 * cos(pi/4))
    assert s.n(3, 0) == 288 and s.n(3, 1) == 287
    for l in range(32):
        assert s.n(l, 256) == (576 if l < 3 else 0)
        assert s.n(l, 300) == (576 if l < 3 else 0)
    for t in range(0, 257):                                  # monotone in depth and in time
        col = [s.n(l, t) for l in range(32)]
        assert all(col[i] >= col[i + 1] for i in range(31))
    for l in range(32):
        row = [s.n(l, t) for t in range(0, 258)]
        assert all(row[i] >= row[i + 1] for i in range(257))


def test_anneal_variants_and_disable():
    base = dict(num_layers=32, num_visual=576, stride=7, step_ratio_bp=1225, tau=50)
    none = Schedule(anneal="none", **base)
    assert all(none.n(l, 40) == none.n0(l) for l in range(32))
    lin = Schedule(anneal="linear", **base)
    assert lin.beta(25) == 0.5 and lin.beta(50) == 0.0
    ex = Schedule(anneal="exp", sigma=20.0, **base)
    assert abs(ex.beta(20) - math.exp(-1)) < 1e-15
    off = Schedule(disable_trim=True, **base)
    assert all(off.n(l, t) == 576 for l in range(32) for t in (0, 1, 49, 50, 99))
