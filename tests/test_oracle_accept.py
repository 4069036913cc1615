"""Pins for the oracle's acceptance rule (Sec. 3.4, Eq. 7) and confidences."""
import itertools
import os

import numpy as np
import pytest

from oracle import sdlm_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "gamma_worked_example.txt")


def _examples():
    out, conf = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        if parts[0] == "conf":
            conf = [float(x) for x in parts[1:]]
        else:
            out.append((conf, float(parts[0]), int(parts[1])))
    return out


@pytest.mark.parametrize("conf,tau,gamma", _examples())
def test_gamma_hand_worked(conf, tau, gamma):
    assert orc.accepted_length(conf, tau)[0] == gamma


def _first_failure_scan(conf, tau):
    """Independent statement: walk the prefix, stop at the first running product below tau."""
    prod, n = 1.0, 0
    for c in conf:
        prod *= c
        if prod < tau:
            break
        n += 1
    return max(n, 1)


def test_gamma_exhaustive_small_blocks():
    levels = [0.2, 0.6, 0.9, 1.0]
    taus = [0.0, 0.1, 0.2, 0.35, 0.5, 0.54, 0.6, 0.81, 0.9, 0.95, 1.0, 1.1]
    for D in (1, 2, 3, 4):
        for conf in itertools.product(levels, repeat=D):
            for tau in taus:
                g, _ = orc.accepted_length(conf, tau)
                assert 1 <= g <= D
                assert g == _first_failure_scan(conf, tau), (conf, tau)


def test_gamma_bounds_and_monotone_in_tau():
    rng = np.random.default_rng(0)
    for _ in range(200):
        D = int(rng.integers(1, 9))
        conf = rng.random(D)
        prev = D + 1
        for tau in np.linspace(-0.2, 1.2, 29):
            g, margin = orc.accepted_length(conf, tau)
            assert 1 <= g <= D
            assert g <= prev          # raising tau can only shorten the prefix
            assert margin >= 0
            prev = g
        assert orc.accepted_length(conf, 0.0)[0] == D
        assert orc.accepted_length(conf, 1.0 + 1e-9)[0] == 1


def test_gamma_margin_reports_distance_to_threshold():
    g, margin = orc.accepted_length([0.5, 0.5], 0.26)
    assert g == 1 and margin == pytest.approx(0.01)


def test_confidence_mode_selects_column():
    z = np.array([[0.0, 1.0, 3.0, -2.0]])
    st = orc.softmax_statistics(z)
    assert np.array_equal(orc.confidences(st, orc.CONF_LOGIT), st.p_top1)
    assert np.array_equal(orc.confidences(st, orc.CONF_ENTROPY), st.conf_entropy)
