"""Pins for the oracle's softmax statistics (Sec. 3.4, Eq. 8 and Eq. 9)."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import sdlm_oracle as orc
import sdlm_synth as syn


def test_uniform_logits_closed_form():
    V = 1000
    st = orc.softmax_statistics(np.full((2, V), 3.25))
    assert st.token.tolist() == [0, 0]                       # lowest index wins an exact tie
    assert st.p_top1 == pytest.approx(1.0 / V, rel=1e-12)
    assert st.entropy == pytest.approx(math.log(V), rel=1e-12)
    assert st.conf_entropy == pytest.approx(0.0, abs=1e-12)
    assert st.top2_gap == pytest.approx(0.0, abs=0)


@pytest.mark.parametrize("L", [0.5, 4.0, 12.0])
def test_one_dominant_logit_closed_form(L):
    V, pos = 513, 77
    z = np.zeros((1, V)); z[0, pos] = L
    st = orc.softmax_statistics(z)
    p = math.exp(L) / (math.exp(L) + V - 1)
    q = 1.0 / (math.exp(L) + V - 1)
    H = -(p * math.log(p) + (V - 1) * q * math.log(q))
    assert st.token[0] == pos
    assert st.p_top1[0] == pytest.approx(p, rel=1e-12)
    assert st.entropy[0] == pytest.approx(H, rel=1e-12)
    assert st.conf_entropy[0] == pytest.approx(1 - H / math.log(V), rel=1e-12)
    assert st.top2_gap[0] == pytest.approx(L, rel=1e-12)
    assert st.max_logit[0] == L
    assert st.lse[0] == pytest.approx(math.log(math.exp(L) + V - 1), rel=1e-12)


def test_matches_scipy_routines_and_invariants():
    rng = np.random.default_rng(1)
    z = rng.normal(size=(16, 301)) * 3.0
    st = orc.softmax_statistics(z)
    logp = scipy.special.log_softmax(z, axis=-1)
    assert np.array_equal(st.token, np.argmax(z, axis=-1))
    assert np.allclose(st.p_top1, np.exp(np.max(logp, axis=-1)), rtol=1e-12, atol=0)
    assert np.allclose(st.entropy, scipy.stats.entropy(np.exp(logp), axis=-1), rtol=1e-10, atol=0)
    assert np.allclose(st.lse, scipy.special.logsumexp(z, axis=-1), rtol=1e-12, atol=0)
    assert np.all(st.entropy >= 0) and np.all(st.entropy <= math.log(z.shape[1]) + 1e-12)
    assert np.all((st.conf_entropy >= -1e-12) & (st.conf_entropy <= 1))
    # adding a constant to every logit changes no probability
    st2 = orc.softmax_statistics(z + 123.0)
    assert np.array_equal(st.token, st2.token)
    assert np.allclose(st.p_top1, st2.p_top1, rtol=1e-10)
    assert np.allclose(st.entropy, st2.entropy, rtol=1e-9)
    srt = np.sort(z, axis=-1)
    assert np.allclose(st.top2_gap, srt[:, -1] - srt[:, -2], atol=0)


def test_extreme_logits_do_not_overflow_and_zero_prob_terms_vanish():
    z = np.array([[1000.0, -1000.0, 0.0], [-1e4, -1e4 + 1.0, -1e4]])
    st = orc.softmax_statistics(z)
    assert st.token.tolist() == [0, 1]
    assert st.p_top1[0] == pytest.approx(1.0)
    assert st.entropy[0] == pytest.approx(0.0, abs=1e-300)
    p = math.e / (math.e + 2)
    assert st.p_top1[1] == pytest.approx(p, rel=1e-12)


def test_tie_takes_lowest_index():
    z = np.array([[1.0, 5.0, 5.0, 2.0, 5.0]])
    assert orc.softmax_statistics(z).token[0] == 1


def test_logits_are_hidden_times_weight_transposed():
    """z[r, n] = sum_c hidden[r, c] W[n, c]: checked against an explicit loop on a tiny case
    with non-square shapes, so a transposed operand or wrong axis cannot pass."""
    rng = np.random.default_rng(2)
    hid = syn.f32_to_bf16_bits(rng.normal(size=(3, 8)).astype(np.float32))
    w = syn.f32_to_bf16_bits(rng.normal(size=(5, 8)).astype(np.float32))
    z = orc.logits_fp64(hid, w, chunk=2)
    hf, wf = syn.bf16_bits_to_f32(hid).astype(np.float64), syn.bf16_bits_to_f32(w).astype(np.float64)
    for r in range(3):
        for n in range(5):
            acc = 0.0
            for c in range(8):
                acc += hf[r, c] * wf[n, c]
            assert z[r, n] == pytest.approx(acc, rel=1e-14, abs=1e-14)
    z2 = orc.logits_fp64(hid, w, w64=orc.widen(w))
    assert np.allclose(z, z2, rtol=1e-14, atol=1e-14)


def test_widen_is_exact_bf16_to_double():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x3DCD, 0x0000, 0x7F7F], dtype=np.uint16)
    exp = [1.0, -1.0, 2.0, 0.10009765625, 0.0, 3.3895313892515355e38]
    assert orc.widen(bits).tolist() == exp
