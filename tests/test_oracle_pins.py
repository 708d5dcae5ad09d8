"""Pins for the CPU oracle: everything here checks the oracle against something
other than itself -- library conversion tables, hand-worked vectors, exact
rational arithmetic, the invariants the paper states, and published mixer
vectors.  No GPU is involved.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, FP16


# --------------------------------------------------------------------------- conversions

def test_half_to_float_all_patterns_match_numpy():
    pats = np.arange(65536, dtype=np.uint16)
    want = pats.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(p)) for p in pats], np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got.view(np.uint32)[~nan], want.view(np.uint32)[~nan])


def _float_probes(rng):
    halves = np.arange(0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mids = (halves[:-1] + halves[1:]) / 2            # exact ties between neighbours
    vals = [halves, mids, mids * (1 + 2.0 ** -20), mids * (1 - 2.0 ** -20)]
    vals.append(np.array([65504.0, 65519.99, 65520.0, 65520.01, 65536.0, 1e9, 2.0 ** -24, 2.0 ** -25,
                          2.0 ** -25 * (1 + 2.0 ** -20), 2.0 ** -26, 0.0, 2.0 ** -14, 2.0 ** -14 * (1 - 2.0 ** -12)]))
    vals.append(rng.standard_normal(20000) * np.exp(rng.uniform(-20, 12, 20000)))
    v = np.concatenate(vals).astype(np.float32)
    return np.concatenate([v, -v])


def test_float_to_half_matches_numpy_round_to_nearest_even():
    v = _float_probes(np.random.default_rng(0))
    with np.errstate(over="ignore"):
        want = v.astype(np.float16).view(np.uint16)
    got = np.array([oracle.float_to_half(float(x)) for x in v], np.uint16)
    assert np.array_equal(got, want)


def test_bf16_conversions_match_torch():
    rng = np.random.default_rng(1)
    pats = np.arange(65536, dtype=np.int64)
    bf = torch.tensor(pats.astype(np.uint16).view(np.int16)).view(torch.bfloat16)
    want = bf.float().numpy()
    got = np.array([oracle.bf16_to_float(int(p)) for p in pats], np.float32)
    nan = np.isnan(want)
    assert np.array_equal(got.view(np.uint32)[~nan], want.view(np.uint32)[~nan])
    # float -> bf16: exact values, ties, near-ties, random
    fin = want[np.isfinite(want)].astype(np.float64)
    fin = np.sort(np.unique(fin))
    mids = (fin[:-1] + fin[1:]) / 2
    v = np.concatenate([fin, mids, mids * (1 + 2.0 ** -20), mids * (1 - 2.0 ** -20),
                        rng.standard_normal(20000) * np.exp(rng.uniform(-60, 60, 20000))])
    v = v[np.abs(v) < 3.0e38].astype(np.float32)
    want16 = torch.tensor(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got16 = np.array([oracle.float_to_bf16(float(x)) for x in v], np.uint16)
    assert np.array_equal(got16, want16)


# --------------------------------------------------------------------------- bitstream

@pytest.mark.parametrize("bits", range(1, 9))
def test_bitstream_layout_is_lsb_first(bits):
    rng = np.random.default_rng(bits)
    n = 64
    codes = rng.integers(-(1 << (bits - 1)), 1 << (bits - 1), n)
    stream = oracle.put_codes(codes, bits)
    assert stream.shape[0] == n * bits // 8
    # independent statement of the layout: numpy's little-endian bit unpacking
    flat = np.unpackbits(stream, bitorder="little")[: n * bits].reshape(n, bits)
    fields = (flat * (1 << np.arange(bits))).sum(1)
    assert np.array_equal(fields, codes & ((1 << bits) - 1))
    assert np.array_equal(oracle.get_codes(stream, n, bits), codes)


# --------------------------------------------------------------------------- hand-worked vectors

def test_golden_vectors_bare_quantizer(golden_vectors):
    assert {c["bits"] for c in golden_vectors} == {1, 2, 3, 4, 6, 8}
    for c in golden_vectors:
        d = np.array(c["d"], np.float32)
        k, delta = oracle.quantize_group(d, c["bits"])
        assert list(k) == c["k"], c["name"]
        assert float(delta) == c["scale"], c["name"]
        assert oracle.put_codes(k, c["bits"]).tobytes() == c["bytes"], c["name"]
        q = [float(oracle.reconstruct(kk, delta)) for kk in k]
        assert q == c["qhat"], c["name"]


def test_golden_vectors_through_encode_and_decode(golden_vectors):
    """Same vectors through the stateful path: m = 0 after a first visit with a zero
    activation, then a = d (rounded to fp16).  m afterwards is exactly qhat."""
    for c in golden_vectors:
        G = len(c["d"])
        snd = oracle.Side(2, 1, G, c["bits"], G, FP16)
        rcv = oracle.Side(2, 1, G, c["bits"], G, FP16)
        ids = np.array([1], np.int32)
        zero = np.zeros((1, 1, G), np.uint16)
        p, s, first = snd.encode(zero, ids)
        assert first[0] == 1 and not p.any() and not s.any()
        out, _ = rcv.decode(p, s, ids, raw=zero)
        act = np.array(c["d"], np.float32).astype(np.float16).view(np.uint16).reshape(1, 1, G)
        p, s, first = snd.encode(act, ids)
        assert first[0] == 0
        assert p.tobytes() == c["bytes"], c["name"]
        assert s.shape == (1, 1) and float(s[0, 0]) == c["scale"]
        out, _ = rcv.decode(p, s, ids)
        want = np.array(c["qhat"], np.float16).view(np.uint16)
        assert np.array_equal(out.reshape(-1), want), c["name"]
        assert np.array_equal(snd.m()[1].reshape(-1), want)
        assert np.array_equal(rcv.m()[1].reshape(-1), want)
        assert not snd.m()[0].any()


# --------------------------------------------------------------------------- exact-arithmetic brute force

def _exact_reference(d, bits):
    """Interval number by definition, in exact rationals; also the nearest-centre search."""
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    s = max(abs(Fraction(float(x))) for x in d)
    delta = s / (1 << (bits - 1))
    ks, edge = [], []
    for x in d:
        q = Fraction(float(x)) / delta
        k = q.numerator // q.denominator          # floor
        ks.append(min(max(k, lo), hi))
        edge.append(abs(q - round(q)) <= Fraction(1, 1 << 20) * max(1, abs(q)))
        # the same code is the nearest interval centre (ties to the upper centre)
        best = min(range(lo, hi + 1), key=lambda c: (abs(Fraction(float(x)) - (c + Fraction(1, 2)) * delta), -c))
        if not edge[-1]:
            assert best == ks[-1]
    return ks, edge, delta


@pytest.mark.parametrize("bits", range(1, 9))
def test_codes_equal_exact_floor_of_quotient(bits):
    rng = np.random.default_rng(100 + bits)
    for trial in range(40):
        G = int(rng.choice([8, 16]))
        scale = float(np.exp(rng.uniform(-12, 8)))
        d = (rng.standard_normal(G) * scale).astype(np.float32)
        if trial % 5 == 0:
            d[rng.integers(G)] *= 30        # an outlier sets the scale
        if trial % 7 == 0:
            d = np.round(d / scale * 4).astype(np.float32) * np.float32(2.0 ** -3)   # many exact edges
        if not d.any():
            d[0] = 1.0
        k, delta = oracle.quantize_group(d, bits)
        ks, edge, delta_exact = _exact_reference(d, bits)
        assert Fraction(float(delta)) == delta_exact          # power-of-two scaling is exact
        for j in range(G):
            if edge[j]:
                assert abs(int(k[j]) - ks[j]) <= 1
            else:
                assert int(k[j]) == ks[j], (bits, trial, j)


# --------------------------------------------------------------------------- invariants of Q

@pytest.mark.parametrize("bits", range(1, 9))
def test_error_bound_and_code_range(bits):
    """|d - Q(d)| <= Delta/2 = max|d| / 2^b: the contraction the convergence proof needs
    (assumption on Q in Theorem 3.1, used in the proof's first lemma), in sup-norm."""
    rng = np.random.default_rng(200 + bits)
    for _ in range(50):
        G = 64
        d = (rng.standard_normal(G) * np.exp(rng.uniform(-10, 10))).astype(np.float32)
        k, delta = oracle.quantize_group(d, bits)
        assert k.min() >= -(1 << (bits - 1)) and k.max() <= (1 << (bits - 1)) - 1
        assert float(delta) == float(np.abs(d).max()) * 2.0 ** (1 - bits)
        q = np.array([oracle.reconstruct(kk, delta) for kk in k], np.float64)
        err = np.abs(d.astype(np.float64) - q)
        # Delta/2, plus the fp32 rounding of the quotient at an interval edge and of the centre
        assert err.max() <= float(delta) / 2 + float(np.abs(d).max()) * 2.0 ** -21
        assert np.abs(q).max() <= np.abs(d).max()          # centres stay inside [-s, s]


def test_zero_and_vanishing_groups():
    for bits in (2, 4, 8):
        k, delta = oracle.quantize_group(np.zeros(8, np.float32), bits)
        assert delta == 0 and not k.any()
        tiny = np.full(8, 1e-39, np.float32)                  # subnormal: Delta < FLT_MIN
        k, delta = oracle.quantize_group(tiny, bits)
        assert delta == 0 and not k.any()
    big = np.array([np.finfo(np.float32).tiny * 8, 0, 0, 0, 0, 0, 0, 0], np.float32)
    k, delta = oracle.quantize_group(big, 2)
    assert delta > 0 and k[0] == 1


def test_eight_bit_fixed_point_of_the_uniform_quantizer():
    """Values that already sit on interval centres survive quantize -> dequantize unchanged."""
    delta = np.float32(0.03125)
    k0 = np.array([-128, -77, -1, 0, 1, 50, 100, 127], np.int32)
    d = ((k0 + 0.5) * delta).astype(np.float32)
    d[0] = -128 * delta                                        # keeps max|d| = 128*Delta
    k, got_delta = oracle.quantize_group(d, 8)
    assert got_delta == delta
    assert np.array_equal(k, k0)
    g16 = d.astype(np.float16)
    assert np.array_equal(g16.astype(np.float32), d)           # representable in fp16
    p, s = oracle.quant_grad(g16.view(np.uint16), 8, 8, FP16)
    out = oracle.dequant_grad(p, s, 8, 8, 8, FP16).view(np.float16)
    assert np.array_equal(out[1:], g16[1:])


# --------------------------------------------------------------------------- invariants of the stateful algorithm

def _rand_act(rng, shape, dtype, scale=1.0):
    x = (rng.standard_normal(shape) * scale).astype(np.float32)
    if dtype == FP16:
        return x.astype(np.float16).view(np.uint16)
    return torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _to_f64(bits16, dtype):
    if dtype == FP16:
        return bits16.view(np.float16).astype(np.float64)
    return torch.tensor(bits16.view(np.int16)).view(torch.bfloat16).double().numpy()


@pytest.mark.parametrize("dtype", [FP16, BF16])
@pytest.mark.parametrize("bits,group", [(2, 16), (3, 8), (4, 32), (6, 8), (8, 16)])
def test_sender_and_receiver_buffers_stay_identical(dtype, bits, group):
    """Algorithm 2: both networks apply m <- m + Delta_m to their own copy; the receiver's
    activation is its m.  First visit: the message is the activation itself."""
    rng = np.random.default_rng(7)
    N, seq, hidden, nb = 6, 3, 32, 2
    snd = oracle.Side(N, seq, hidden, bits, group, dtype)
    rcv = oracle.Side(N, seq, hidden, bits, group, dtype)
    base = _rand_act(rng, (N, seq, hidden), dtype)
    for epoch in range(4):
        order = rng.permutation(N).astype(np.int32)
        for c in range(N // nb):
            ids = order[c * nb:(c + 1) * nb]
            act = base[ids] if epoch == 0 else _rand_act(rng, (nb, seq, hidden), dtype)
            if epoch >= 2:
                act = base[ids]                                  # revisit the same activation
            before = snd.m()[ids].copy()
            p, s, first = snd.encode(act, ids)
            assert p.shape == (nb, seq * hidden * bits // 8)     # b bits per element on the wire
            out, first_r = rcv.decode(p, s, ids, raw=act if epoch == 0 else None)
            assert np.array_equal(first, first_r)
            assert np.array_equal(first, np.full(nb, epoch == 0, np.uint8))
            assert np.array_equal(snd.m(), rcv.m())
            assert np.array_equal(out, rcv.m()[ids])
            assert snd.checksum() == rcv.checksum()
            if epoch == 0:
                assert np.array_equal(snd.m()[ids], act)          # delta_xi = 0 on the first visit
                assert not p.any() and not s.any()
            else:
                # per group: |a - m_new| <= Delta/2 + rounding of m to 16 bits
                a = _to_f64(act, dtype).reshape(nb, -1, group)
                m_new = _to_f64(snd.m()[ids], dtype).reshape(nb, -1, group)
                m_old = _to_f64(before, dtype).reshape(nb, -1, group)
                smax = np.abs(a - m_old).max(-1)
                assert np.allclose(s.reshape(nb, -1), smax * 2.0 ** (1 - bits), rtol=1e-6, atol=0)
                ulp = np.abs(m_new).max(-1) * (2.0 ** -10 if dtype == FP16 else 2.0 ** -7)
                assert (np.abs(a - m_new).max(-1) <= smax / 2 ** bits * (1 + 1e-6) + ulp).all()
    assert snd.seen().all() and rcv.seen().all()
    assert snd.status() == 0 and rcv.status() == 0


def test_step_change_decays_geometrically():
    """Self-correcting loop: if the activation stops moving after a jump D, each further
    visit shrinks the message error by the factor 2^-b (contraction with c_Q = 2^-b),
    down to the resolution of the 16-bit storage."""
    rng = np.random.default_rng(3)
    bits, group, hidden = 3, 16, 64
    snd = oracle.Side(1, 2, hidden, bits, group, FP16)
    ids = np.array([0], np.int32)
    a0 = _rand_act(rng, (1, 2, hidden), FP16)
    snd.encode(a0, ids)
    a1 = (a0.view(np.float16).astype(np.float32) + rng.standard_normal((1, 2, hidden)).astype(np.float32)
          ).astype(np.float16).view(np.uint16)
    D = np.abs(_to_f64(a1, FP16) - _to_f64(a0, FP16)).reshape(-1, group).max(-1)
    for visit in range(1, 5):
        snd.encode(a1, ids)
        err = np.abs(_to_f64(a1, FP16) - _to_f64(snd.m()[0:1], FP16)).reshape(-1, group).max(-1)
        floor_ = np.abs(_to_f64(a1, FP16)).reshape(-1, group).max(-1) * 2.0 ** -10
        assert (err <= D * 2.0 ** (-bits * visit) * (1 + 1e-6) + 2 * floor_).all(), visit


def test_zero_delta_is_a_fixed_point():
    """c_Q = 0 case of the theory: an unchanged activation sends all-zero codes and scales
    and leaves m as it is."""
    rng = np.random.default_rng(4)
    snd = oracle.Side(3, 2, 32, 4, 16, FP16)
    ids = np.array([2, 0], np.int32)
    act = _rand_act(rng, (2, 2, 32), FP16)
    snd.encode(act, ids)
    m0 = snd.m().copy()
    p, s, first = snd.encode(act, ids)
    assert not first.any() and not p.any() and not s.any()
    assert np.array_equal(snd.m(), m0)


def test_bad_ids_are_skipped_and_reported():
    rng = np.random.default_rng(5)
    snd = oracle.Side(4, 1, 16, 2, 8, FP16)
    rcv = oracle.Side(4, 1, 16, 2, 8, FP16)
    act = _rand_act(rng, (3, 1, 16), FP16)
    ids = np.array([1, 9, 1], np.int32)                 # out of range, then a repeat
    p, s, first = snd.encode(act, ids)
    assert snd.status() == (oracle.ST_BAD_ID | oracle.ST_DUP_ID)
    assert snd.status() == 0                            # reading clears
    assert list(snd.seen()) == [0, 1, 0, 0]
    assert np.array_equal(snd.m()[1], act[0])
    out, _ = rcv.decode(p, s, np.array([1, 2], np.int32), raw=None)     # first visits without a raw message
    assert rcv.status() == oracle.ST_NO_RAW
    assert not out.any() and not rcv.seen().any() and not rcv.m().any()


# --------------------------------------------------------------------------- gradients

@pytest.mark.parametrize("bits", [4, 6, 8])
def test_gradient_quantization_is_the_same_q_without_a_buffer(bits):
    rng = np.random.default_rng(6)
    G, n = 64, 64 * 10
    g = _rand_act(rng, (n,), FP16, 1e-3)
    p, s = oracle.quant_grad(g, bits, G, FP16)
    assert p.shape[0] == n * bits // 8 and s.shape[0] == n // G
    out = oracle.dequant_grad(p, s, n, bits, G, FP16)
    gf = _to_f64(g, FP16).reshape(-1, G)
    of = _to_f64(out, FP16).reshape(-1, G)
    smax = np.abs(gf).max(-1)
    assert np.array_equal(s.astype(np.float64), smax * 2.0 ** (1 - bits))
    ulp = smax * 2.0 ** -10
    assert (np.abs(gf - of).max(-1) <= smax / 2 ** bits * (1 + 1e-6) + ulp).all()
    # group by group it is exactly quantize_group + reconstruct
    k, delta = oracle.quantize_group(gf[3].astype(np.float32), bits)
    assert np.array_equal(oracle.get_codes(p, n, bits).reshape(-1, G)[3], k)


# --------------------------------------------------------------------------- checksum

def test_mixer_reproduces_published_splitmix64_stream():
    # splitmix64 seeded with 1234567: the widely published first five outputs
    want = [6457827717110365317, 3203168211198807973, 9817491932198370423,
            4593380528125082431, 16408922859458223821]
    assert [oracle.mix64(i + 1, 1234567) for i in range(5)] == want


def test_checksum_definition_and_sensitivity():
    rng = np.random.default_rng(8)
    side = oracle.Side(3, 2, 8, 2, 8, FP16)
    act = _rand_act(rng, (2, 2, 8), FP16)
    side.encode(act, np.array([2, 0], np.int32))
    m = side.m().reshape(-1)
    words = sum(m[e::4].astype(np.uint64) << np.uint64(16 * e) for e in range(4))      # little-endian 64-bit words
    assert np.array_equal(words, np.ascontiguousarray(m).view(np.uint64))
    want = sum(oracle.mix64(i, int(w)) for i, w in enumerate(words))
    want += sum(oracle.mix64((1 << 40) + x, int(f)) for x, f in enumerate(side.seen()))
    assert side.checksum() == want % (1 << 64)
    other = oracle.Side(3, 2, 8, 2, 8, FP16)
    act2 = act.copy()
    act2[1, 1, 7] ^= 1                                    # one bit of one element
    other.encode(act2, np.array([2, 0], np.int32))
    assert other.checksum() != side.checksum()
    swapped = oracle.Side(3, 2, 8, 2, 8, FP16)
    swapped.encode(act, np.array([0, 2], np.int32))       # same rows under other ids
    assert swapped.checksum() != side.checksum()
