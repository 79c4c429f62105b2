"""CPU oracle for the scalar controller and link formulas of CoVSpec (Eq. 7-9, 18-22).

TEST INFRASTRUCTURE ONLY: plain Python floats (float64), each formula written out as the paper
states it; the exponential moving average is applied update by update.  Shares no code with the
library.  Pinned by tests/test_controller.py (hand-worked values, the closed form of a run of
updates, monotonicity and clipping properties).
Readings: the accepted tokens update the average before the rejected ones; round() rounds halves
away from zero; payload sizes are in bits and the latency in seconds for a bandwidth in hertz.
"""
import math


def uplink_bits(n_draft, b_id, n_logit_draft, b_logit):
    """Eq. 7."""
    return n_draft * b_id + n_logit_draft * b_logit


def downlink_bits(all_accepted, b_acc, b_bonus, b_rej, vocab, b_logit_tar):
    """Eq. 8."""
    return b_acc + b_bonus if all_accepted else b_rej + vocab * b_logit_tar


def comm_latency(bits, bandwidth_hz, snr_db):
    """Eq. 9 / Eq. 19: bits over the Shannon rate B log2(1 + 10^(SNR/10))."""
    return bits / (bandwidth_hz * math.log2(1.0 + 10.0 ** (snr_db / 10.0)))


def ema_update(p_hat, eta, k, n_acc):
    """Eq. 18, applied n_acc times with a = 1 and then k - n_acc times with a = 0."""
    for _ in range(n_acc):
        p_hat = (1.0 - eta) * p_hat + eta * 1.0
    for _ in range(k - n_acc):
        p_hat = (1.0 - eta) * p_hat + eta * 0.0
    return p_hat


def phi(p_hat, t_rej, p_low, p_up, t_ref):
    """Eq. 20."""
    if p_hat <= p_low:
        return -1
    if p_hat >= p_up and t_rej <= t_ref:
        return 1
    return 0


def next_draft_length(k, p_hat, t_rej, p_low, p_up, t_ref, s, k_min, k_max):
    """Eq. 21-22: k <- clip(round(k * s^phi), k_min, k_max)."""
    x = k * s ** phi(p_hat, t_rej, p_low, p_up, t_ref)
    r = math.floor(x + 0.5) if x >= 0 else -math.floor(-x + 0.5)
    return min(k_max, max(k_min, int(r)))
