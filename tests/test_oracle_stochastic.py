"""Pins for the oracle's unbiased (stochastic-rounding) quantizer: the generator against its
published known-answer vectors, the quantizer against exact rational arithmetic, the property
the convergence theorem asks for (E[Q(x)] = x, Theorem 3.1) and the structure of the levels.
No GPU is involved."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import BF16, FP16

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_philox_known_answer_vectors():
    n = 0
    for line in open(os.path.join(ROOT, "tests", "golden", "philox4x32_10_kat.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        w = [int(x, 16) for x in line]
        assert list(oracle.philox4x32_10(w[0:4], w[4:6])) == w[6:10]
        n += 1
    assert n == 3


def _offsets(seed, epoch, stream_id, chunk):
    """r - 1/2 of the 8 elements of a chunk as exact rationals, from the generator's raw words:
    element j takes 16 bits, low half of word j//2 first."""
    w = oracle.philox4x32_10([chunk, stream_id, epoch & 0xFFFFFFFF, epoch >> 32],
                             [seed & 0xFFFFFFFF, seed >> 32])
    halves = w.view(np.uint16)                       # little-endian: low half first
    return [Fraction(2 * int(h) + 1, 1 << 17) - Fraction(1, 2) for h in halves]


@pytest.mark.parametrize("bits", range(1, 9))
def test_codes_equal_exact_stochastic_floor(bits):
    """k = floor(d/Delta - 1/2 + r) with Delta = s / (2^(b-1) - 1/2), in exact rationals, for
    random groups; elements whose exact value sits within fp32 rounding of an integer may land
    on either side."""
    rng = np.random.default_rng(300 + bits)
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    for trial in range(30):
        G = 16
        d = (rng.standard_normal(G) * float(np.exp(rng.uniform(-10, 6)))).astype(np.float32)
        seed, epoch, sid, first = int(rng.integers(1 << 62)), int(rng.integers(1 << 40)), int(rng.integers(1 << 20)), 8 * int(rng.integers(1000))
        k, delta = oracle.quantize_group_stochastic(d, bits, seed, epoch, sid, first)
        s = max(abs(Fraction(float(x))) for x in d)
        delta_exact = s / (Fraction(1 << (bits - 1)) - Fraction(1, 2))
        assert abs(Fraction(float(delta)) - delta_exact) <= delta_exact * Fraction(1, 1 << 23)
        rc = _offsets(seed, epoch, sid, first // 8) + _offsets(seed, epoch, sid, first // 8 + 1)
        for j in range(G):
            t = Fraction(float(d[j])) / delta_exact + rc[j]
            want = min(max(t.numerator // t.denominator, lo), hi)
            near_edge = abs(t - round(t)) <= Fraction(1, 1 << 17) * max(1, abs(t))
            if near_edge:
                assert abs(int(k[j]) - want) <= 1
            else:
                assert int(k[j]) == want, (bits, trial, j)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_levels_cover_the_whole_range_and_the_extremes_are_exact(bits):
    rng = np.random.default_rng(400 + bits)
    top = (1 << (bits - 1)) - 0.5
    for trial in range(20):
        d = (rng.standard_normal(8) * 3).astype(np.float32)
        k, delta = oracle.quantize_group_stochastic(d, bits, 5, trial, 7)
        s = float(np.abs(d).max())
        assert abs(float(delta) - s / top) <= s / top * 2.0 ** -22
        q = np.array([oracle.reconstruct(kk, delta) for kk in k], np.float64)
        assert k.min() >= -(1 << (bits - 1)) and k.max() <= (1 << (bits - 1)) - 1
        assert np.abs(q).max() <= s * (1 + 2.0 ** -21)                 # levels stay inside [-s, s]
        assert (np.abs(d - q) < float(delta) * (1 + 2.0 ** -20)).all()  # a neighbouring level, never further
        j = int(np.abs(d).argmax())                                    # the largest element is a level itself
        assert k[j] == ((1 << (bits - 1)) - 1 if d[j] > 0 else -(1 << (bits - 1)))
        assert abs(q[j] - d[j]) <= s * 2.0 ** -21


def test_values_on_a_level_never_move_and_midpoints_split_evenly():
    # b = 2, s = 1.5: Delta = 1, levels -1.5, -0.5, 0.5, 1.5
    d = np.array([1.5, 0.5, -0.5, -1.5, 0.0, 1.0, -1.0, 0.25], np.float32)
    ks = np.array([oracle.quantize_group_stochastic(d, 2, 99, e, 3)[0] for e in range(4000)])
    assert (ks[:, 0] == 1).all() and (ks[:, 1] == 0).all() and (ks[:, 2] == -1).all() and (ks[:, 3] == -2).all()
    for col, lower in ((4, -1), (5, 0), (6, -2)):                      # midway between two levels
        assert set(np.unique(ks[:, col])) == {lower, lower + 1}
        assert abs((ks[:, col] == lower).mean() - 0.5) < 5 * 0.5 / np.sqrt(4000)
    assert abs((ks[:, 7] == 0).mean() - 0.75) < 5 * np.sqrt(0.75 * 0.25 / 4000)    # 0.25 is 1/4 of the way from 0.5 down to -0.5


@pytest.mark.parametrize("bits", [2, 4, 6])
def test_unbiased_in_expectation(bits):
    """E[Q(d)] = d for every element, outliers and the group maximum included (Theorem 3.1's
    assumption on Q; the proof uses it for the backward term)."""
    rng = np.random.default_rng(500 + bits)
    d = (rng.standard_normal(16)).astype(np.float32)
    d[3] *= 6                                                          # sets the scale
    n = 6000
    acc = np.zeros(16)
    delta = None
    for e in range(n):
        k, delta = oracle.quantize_group_stochastic(d, bits, 1234, e, 42)
        acc += (k + 0.5) * float(delta)
    mean = acc / n
    sigma = float(delta) / 2                                           # a two-point variable: std <= Delta/2
    assert (np.abs(mean - d) <= 5 * sigma / np.sqrt(n) + 1e-6).all()


def test_zero_group_and_determinism():
    k, delta = oracle.quantize_group_stochastic(np.zeros(8, np.float32), 4, 1, 2, 3)
    assert delta == 0 and not k.any()
    d = np.linspace(-1, 1, 64).astype(np.float32)                      # 62 elements with a real choice
    a = oracle.quantize_group_stochastic(d, 3, 11, 5, 9)[0]
    assert np.array_equal(a, oracle.quantize_group_stochastic(d, 3, 11, 5, 9)[0])          # same counters, same codes
    others = [oracle.quantize_group_stochastic(d, 3, *args)[0] for args in
              ((12, 5, 9), (11, 6, 9), (11, 5, 10), (11, 1 << 32 | 5, 9))]
    assert all(not np.array_equal(a, o) for o in others)               # seed, epoch (both words), stream id all matter
    assert not np.array_equal(a, oracle.quantize_group_stochastic(d, 3, 11, 5, 9, first_elem=8)[0])


def _rand_act(rng, shape, dtype, scale=1.0):
    import torch
    x = (rng.standard_normal(shape) * scale).astype(np.float32)
    if dtype == FP16:
        return x.astype(np.float16).view(np.uint16)
    return torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("dtype", [FP16, BF16])
def test_stateful_path_with_stochastic_rounding(dtype):
    """The receiver is untouched by the rounding mode: it rebuilds (k + 1/2) * Delta from what
    it is sent, and both copies of m stay identical (Algorithm 2)."""
    rng = np.random.default_rng(17)
    N, seq, hidden, bits, group = 4, 3, 64, 3, 16
    snd = oracle.Side(N, seq, hidden, bits, group, dtype)
    rcv = oracle.Side(N, seq, hidden, bits, group, dtype)
    ids = np.array([2, 0], np.int32)
    for epoch in range(4):
        snd.set_rounding(True, seed=77, epoch=epoch)
        act = _rand_act(rng, (2, seq, hidden), dtype)
        p, s, first = snd.encode(act, ids)
        out, _ = rcv.decode(p, s, ids, raw=act if epoch == 0 else None)
        assert np.array_equal(snd.m(), rcv.m()) and np.array_equal(out, rcv.m()[ids])
        assert snd.checksum() == rcv.checksum()
        if epoch:
            codes = oracle.get_codes(p[0], seq * hidden, bits)
            assert codes.min() >= -4 and codes.max() <= 3
    # per group the codes are those of the bare stochastic quantizer at the group's place in the stream
    snd.set_rounding(True, seed=77, epoch=9)
    before = snd.m()[2].reshape(-1).copy()
    act = _rand_act(rng, (1, seq, hidden), dtype)
    p, s, _ = snd.encode(act, np.array([2], np.int32))
    to_f = (lambda v: v.view(np.float16).astype(np.float32)) if dtype == FP16 else \
        (lambda v: (v.astype(np.uint32) << 16).view(np.float32))
    d = to_f(act.reshape(-1)) - to_f(before)
    g = 5
    k, delta = oracle.quantize_group_stochastic(d[g * group:(g + 1) * group], bits, 77, 9, 2, first_elem=g * group)
    assert np.array_equal(oracle.get_codes(p[0], seq * hidden, bits)[g * group:(g + 1) * group], k)
    assert s.reshape(-1)[g] == delta


def test_gradient_quantization_stochastic():
    rng = np.random.default_rng(23)
    G, n, bits = 64, 64 * 6, 4
    g16 = _rand_act(rng, (n,), FP16, 1e-3)
    p, s = oracle.quant_grad_stochastic(g16, bits, G, seed=5, epoch=1)
    gf = g16.view(np.float16).astype(np.float32)
    for grp in (0, 3, 5):
        k, delta = oracle.quantize_group_stochastic(gf[grp * G:(grp + 1) * G], bits, 5, 1, 0xFFFFFFFF, first_elem=grp * G)
        assert np.array_equal(oracle.get_codes(p, n, bits)[grp * G:(grp + 1) * G], k) and s[grp] == delta
    # unbiased over epochs, through the ordinary dequantizer
    acc = np.zeros(n)
    N = 1500
    for e in range(N):
        p, s = oracle.quant_grad_stochastic(g16, bits, G, seed=5, epoch=e)
        acc += oracle.dequant_grad(p, s, n, bits, G, FP16).view(np.float16).astype(np.float64)
    sigma = np.repeat(s, G) / 2 + np.abs(gf) * 2.0 ** -11            # two-point rounding + the fp16 output rounding
    assert (np.abs(acc / N - gf) <= 5 * sigma / np.sqrt(N) + np.abs(gf) * 2.0 ** -11).all()
    assert not np.array_equal(p, oracle.quant_grad_stochastic(g16, bits, G, seed=5, epoch=0)[0])
