"""Link model and draft-length controller (Eq. 7-9, 18-22): the oracle against hand-worked values
and closed forms, and the library's host functions against the oracle (no GPU needed)."""
import math

import pytest

from oracle import controller_oracle as O
from paper_2605_02218_b200 import api, build


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.load_library()


def test_oracle_hand_values():
    # Eq. 7: 6 drafted ids of 32 bits and their 6 float16 logits
    assert O.uplink_bits(6, 32, 6, 16) == 288
    # Eq. 8: accepted -> 8 + 32 bits; rejected -> 8 + |W| * 16 bits
    assert O.downlink_bits(True, 8, 32, 8, 151674, 16) == 40
    assert O.downlink_bits(False, 8, 32, 8, 151674, 16) == 8 + 151674 * 16
    # Eq. 9 with the paper's link (5 MHz, 10 dB): rate 5e6 * log2(11) = 17.297 Mbit/s
    assert O.comm_latency(17297158.09, 5e6, 10.0) == pytest.approx(1.0, rel=1e-8)
    assert O.comm_latency(8 + 151674 * 16, 5e6, 10.0) == pytest.approx(0.140299, rel=1e-5)
    # Eq. 18 from p = 1 with eta = 0.5: one acceptance keeps 1, one rejection halves it
    assert O.ema_update(1.0, 0.5, 1, 1) == 1.0 and O.ema_update(1.0, 0.5, 1, 0) == 0.5
    assert O.ema_update(0.5, 0.5, 3, 2) == pytest.approx(((0.5 * 0.5 + 0.5) * 0.5 + 0.5) * 0.5)
    # Eq. 20-22
    assert O.phi(0.3, 0.0, 0.4, 0.8, 0.1) == -1 and O.phi(0.9, 0.05, 0.4, 0.8, 0.1) == 1
    assert O.phi(0.9, 0.2, 0.4, 0.8, 0.1) == 0 and O.phi(0.6, 0.0, 0.4, 0.8, 0.1) == 0
    assert O.next_draft_length(4, 0.9, 0.05, 0.4, 0.8, 0.1, 1.5, 1, 16) == 6
    assert O.next_draft_length(5, 0.3, 0.05, 0.4, 0.8, 0.1, 2.0, 1, 16) == 3      # 2.5 rounds away from zero
    assert O.next_draft_length(12, 0.9, 0.05, 0.4, 0.8, 0.1, 1.5, 1, 16) == 16    # clipped
    assert O.next_draft_length(1, 0.1, 0.05, 0.4, 0.8, 0.1, 1.5, 2, 16) == 2      # clipped from below


def test_ema_closed_form_and_bounds():
    # n ones then m zeros: p -> (1 - eta)^m (1 - (1 - eta)^n (1 - p))
    for p0, eta, k, n in [(1.0, 0.1, 8, 5), (0.2, 0.3, 6, 6), (0.7, 0.05, 10, 0), (0.5, 0.9, 4, 1)]:
        want = (1 - eta) ** (k - n) * (1 - (1 - eta) ** n * (1 - p0))
        assert O.ema_update(p0, eta, k, n) == pytest.approx(want, rel=1e-12)
        assert 0.0 <= O.ema_update(p0, eta, k, n) <= 1.0
    assert O.ema_update(0.5, 0.2, 5, 5) > 0.5 > O.ema_update(0.5, 0.2, 5, 0)


def test_latency_properties():
    base = O.comm_latency(1e6, 5e6, 10.0)
    assert O.comm_latency(2e6, 5e6, 10.0) == pytest.approx(2 * base)
    assert O.comm_latency(1e6, 10e6, 10.0) == pytest.approx(base / 2)
    assert O.comm_latency(1e6, 5e6, 20.0) < base
    assert O.comm_latency(1e6, 1.0, 0.0) == pytest.approx(1e6)            # 0 dB: log2(2) = 1 bit/s/Hz


def test_library_matches_oracle(lib):
    assert lib.covspec_uplink_bits(6, 32, 6, 16) == O.uplink_bits(6, 32, 6, 16)
    for acc in (0, 1):
        assert lib.covspec_downlink_bits(acc, 8, 32, 8, 151674, 16) == O.downlink_bits(bool(acc), 8, 32, 8, 151674, 16)
    for bits, bw, snr in [(2426792.0, 5e6, 10.0), (288.0, 1e6, -3.0), (1e9, 2e7, 25.5)]:
        assert lib.covspec_comm_latency(bits, bw, snr) == pytest.approx(O.comm_latency(bits, bw, snr), rel=1e-14)
    for p0, eta, k, n in [(1.0, 0.1, 8, 5), (0.2, 0.3, 6, 6), (0.7, 0.05, 10, 0), (0.5, 0.9, 4, 1)]:
        assert lib.covspec_ema_update(p0, eta, k, n) == pytest.approx(O.ema_update(p0, eta, k, n), rel=1e-15)
    grid = [(k, p, t) for k in (1, 2, 3, 5, 8, 13) for p in (0.1, 0.4, 0.6, 0.8, 0.95) for t in (0.01, 0.1, 0.5)]
    for k, p, t in grid:
        for s in (1.25, 1.5, 2.0):
            got = lib.covspec_draft_length(k, p, t, 0.4, 0.8, 0.1, s, 1, 12)
            assert got == O.next_draft_length(k, p, t, 0.4, 0.8, 0.1, s, 1, 12), (k, p, t, s)
    assert lib.covspec_draft_length(4, 0.9, 0.0, 0.4, 0.8, 0.1, 1.0, 1, 8) == -1     # s must exceed 1
    assert lib.covspec_draft_length(4, 0.9, 0.0, 0.4, 0.8, 0.1, 1.5, 9, 8) == -1
