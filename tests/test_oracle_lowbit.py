"""Pins for the oracle's low-precision store of previous messages (the paper's "mz" ablation:
z bits per element of m).  The store is the messages' own quantizer Q applied to m, so the pins
are: the wiring of the steps against the separately pinned bare quantizer, the two error bounds
(message: Delta/2 around the dequantized store; storage: Delta_m/2), identity of the two sides,
and what the method promises -- the error stays at the resolution of the message quantizer plus
that of the store, and shrinks to the store's resolution when the activation stops moving."""
import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, FP16


def _rand_act(rng, shape, dtype, scale=1.0):
    x = (rng.standard_normal(shape) * scale).astype(np.float32)
    if dtype == FP16:
        return x.astype(np.float16).view(np.uint16)
    return torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _f32(bits16, dtype):
    if dtype == FP16:
        return bits16.view(np.float16).astype(np.float32)
    return (bits16.astype(np.uint32) << 16).view(np.float32)


@pytest.mark.parametrize("dtype", [FP16, BF16])
@pytest.mark.parametrize("bits,m_bits,group", [(4, 8, 16), (2, 2, 8), (3, 4, 32), (8, 8, 8), (4, 5, 16)])
def test_wiring_bounds_and_identity_of_the_two_sides(dtype, bits, m_bits, group):
    rng = np.random.default_rng(bits * 10 + m_bits)
    N, seq, hidden, nb = 5, 3, 64, 2
    E = seq * hidden
    snd = oracle.SideLow(N, seq, hidden, bits, group, dtype, m_bits)
    rcv = oracle.SideLow(N, seq, hidden, bits, group, dtype, m_bits)
    base = _rand_act(rng, (N, seq, hidden), dtype)
    ulp = 2.0 ** -10 if dtype == FP16 else 2.0 ** -7
    for epoch in range(4):
        for ids in (np.array([3, 0], np.int32), np.array([4, 1], np.int32)):
            act = base[ids] if epoch == 0 else _rand_act(rng, (nb, seq, hidden), dtype)
            codes_before = snd.m_codes()[ids].copy()
            scales_before = snd.m_scales()[ids].copy()
            p, s, first = snd.encode(act, ids)
            out, first_r = rcv.decode(p, s, ids, raw=act if epoch == 0 else None)
            assert np.array_equal(first, first_r) and first.all() == (epoch == 0)
            assert p.shape == (nb, E * bits // 8) and snd.m_codes().shape == (N, E * m_bits // 8)
            # the two sides hold the same store
            assert np.array_equal(snd.m_codes(), rcv.m_codes())
            assert np.array_equal(snd.m_scales().view(np.uint32), rcv.m_scales().view(np.uint32))
            assert snd.checksum() == rcv.checksum()
            a = _f32(act.reshape(nb, E), dtype)
            for y in range(nb):
                if epoch == 0:
                    assert np.array_equal(out[y].reshape(-1), act[y].reshape(-1))          # the raw message itself
                    assert not p[y].any() and not s[y].any()
                    m_new = a[y]
                else:
                    # wiring, group by group, from the separately pinned pieces
                    km = oracle.get_codes(codes_before[y], E, m_bits)
                    m_deq = np.array([oracle.reconstruct(k, d) for k, d in zip(km, np.repeat(scales_before[y], group))], np.float32)
                    d = a[y] - m_deq
                    m_new = np.empty(E, np.float32)
                    for g in range(E // group):
                        sl = slice(g * group, (g + 1) * group)
                        k, delta = oracle.quantize_group(d[sl], bits)
                        assert np.array_equal(oracle.get_codes(p[y], E, bits)[sl], k) and s[y, g] == delta
                        q = np.array([oracle.reconstruct(kk, delta) for kk in k], np.float32)
                        m_new[sl] = m_deq[sl] + q
                        # message bound: the new m is within Delta/2 of the activation
                        # (plus the fp32 rounding of the quotient at an interval edge and of the sum)
                        assert np.abs(a[y][sl] - m_new[sl]).max() <= float(delta) / 2 + np.abs(d[sl]).max() * 2.0 ** -21 + np.abs(m_new[sl]).max() * 2.0 ** -23
                    want_out = m_new.astype(np.float16).view(np.uint16) if dtype == FP16 else \
                        torch.tensor(m_new).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
                    assert np.array_equal(out[y].reshape(-1), want_out)
                # storage: Q_z(m_new), error at most Delta_m / 2 = max|m_new| / 2^z per group
                sid = ids[y]
                for g in (0, E // group - 1):
                    sl = slice(g * group, (g + 1) * group)
                    k, dm = oracle.quantize_group(m_new[sl], m_bits)
                    assert np.array_equal(oracle.get_codes(snd.m_codes()[sid], E, m_bits)[sl], k)
                    assert snd.m_scales()[sid, g] == dm
                stored = snd.m_values()[sid]
                smax = np.abs(m_new.astype(np.float64)).reshape(-1, group).max(-1)
                assert (np.abs(stored - m_new).reshape(-1, group).max(-1) <= smax / 2 ** m_bits + smax * 2.0 ** -20).all()
    assert snd.seen()[[0, 1, 3, 4]].all() and not snd.seen()[2]
    assert not snd.m_codes()[2].any() and not snd.m_scales()[2].any()                   # "initialized to 0"
    assert snd.status() == 0 and rcv.status() == 0


def test_error_settles_at_the_resolution_of_the_store():
    """The activation stops moving: each further visit sends the (small) storage error, and the
    receiver's activation stays within Delta/2 of the truth with Delta <= max|storage error| * 2^(1-b)."""
    rng = np.random.default_rng(5)
    bits, m_bits, group, hidden = 4, 8, 16, 64
    snd = oracle.SideLow(1, 2, hidden, bits, group, FP16, m_bits)
    rcv = oracle.SideLow(1, 2, hidden, bits, group, FP16, m_bits)
    ids = np.zeros(1, np.int32)
    a = _rand_act(rng, (1, 2, hidden), FP16)
    af = _f32(a.reshape(-1), FP16).astype(np.float64)
    p, s, _ = snd.encode(a, ids)
    rcv.decode(p, s, ids, raw=a)
    smax = np.abs(af).reshape(-1, group).max(-1)
    for visit in range(3):
        p, s, _ = snd.encode(a, ids)
        out, _ = rcv.decode(p, s, ids)
        err = np.abs(_f32(out.reshape(-1), FP16).astype(np.float64) - af).reshape(-1, group).max(-1)
        # what is left to send is the storage error (<= smax / 2^8) plus the last message error (1/16 of it):
        # Delta <= 1.1 * smax * 2^-8 * 2^(1-4), and the receiver is within Delta / 2 (+ fp16 rounding) of the truth
        assert (s.reshape(-1) <= 1.1 * smax * 2.0 ** (-8 + 1 - bits)).all()
        assert (err <= 1.1 * smax * 2.0 ** -8 * 2.0 ** -4 + smax * 2.0 ** -10).all()
        assert (np.abs(snd.m_values()[0] - af).reshape(-1, group).max(-1) <= smax * 2.0 ** -8 * 1.1).all()


def test_low_precision_digest_definition():
    rng = np.random.default_rng(6)
    side = oracle.SideLow(3, 2, 32, 4, 16, FP16, 8)
    side.encode(_rand_act(rng, (2, 2, 32), FP16), np.array([2, 0], np.int32))
    words = side.m_codes().reshape(-1).view(np.uint32)
    want = sum(oracle.mix64(i, int(w)) for i, w in enumerate(words))
    want += sum(oracle.mix64(len(words) + i, int(w)) for i, w in enumerate(side.m_scales().reshape(-1).view(np.uint32)))
    want += sum(oracle.mix64((1 << 40) + x, int(f)) for x, f in enumerate(side.seen()))
    assert side.checksum() == want % (1 << 64)


def test_low_precision_bad_ids():
    rng = np.random.default_rng(7)
    snd = oracle.SideLow(4, 1, 16, 2, 8, FP16, 8)
    rcv = oracle.SideLow(4, 1, 16, 2, 8, FP16, 8)
    act = _rand_act(rng, (3, 1, 16), FP16)
    p, s, first = snd.encode(act, np.array([1, 9, 1], np.int32))
    assert snd.status() == (oracle.ST_BAD_ID | oracle.ST_DUP_ID) and list(snd.seen()) == [0, 1, 0, 0]
    out, _ = rcv.decode(p, s, np.array([1, 2], np.int32), raw=None)
    assert rcv.status() == oracle.ST_NO_RAW and not out.any() and not rcv.seen().any()


@pytest.mark.parametrize("dtype", [FP16, BF16])
def test_binary32_store(dtype):
    """m kept in binary32 (m_bits = 32): m_new = m + Q(a - m) is stored as it is, the receiver's
    activation is T(m_new); wiring against the separately pinned bare quantizer, the message
    bound, identity of the two sides, and geometric decay of the error of a halted activation
    without the floor that a 16-bit store has."""
    rng = np.random.default_rng(41)
    N, seq, hidden, bits, group = 3, 2, 64, 3, 16
    E = seq * hidden
    snd = oracle.SideLow(N, seq, hidden, bits, group, dtype, 32)
    rcv = oracle.SideLow(N, seq, hidden, bits, group, dtype, 32)
    ids = np.array([2, 0], np.int32)
    a0 = _rand_act(rng, (2, seq, hidden), dtype)
    p, s, first = snd.encode(a0, ids)
    out, _ = rcv.decode(p, s, ids, raw=a0)
    assert first.all() and np.array_equal(out, a0) and snd.m_codes().shape == (N, E * 4)
    assert np.array_equal(snd.m_codes()[ids].view(np.float32), _f32(a0.reshape(2, E), dtype))     # stored exactly
    a1 = _rand_act(rng, (2, seq, hidden), dtype)
    for visit in range(1, 6):
        before = snd.m_codes()[ids].view(np.float32).copy()
        p, s, first = snd.encode(a1, ids)
        out, _ = rcv.decode(p, s, ids)
        assert not first.any()
        assert np.array_equal(snd.m_codes(), rcv.m_codes()) and snd.checksum() == rcv.checksum()
        a = _f32(a1.reshape(2, E), dtype)
        for y in range(2):
            d = a[y] - before[y]
            m_new = np.empty(E, np.float32)
            for g in range(E // group):
                sl = slice(g * group, (g + 1) * group)
                k, delta = oracle.quantize_group(d[sl], bits)
                assert np.array_equal(oracle.get_codes(p[y], E, bits)[sl], k) and s[y, g] == delta
                m_new[sl] = before[y][sl] + np.array([oracle.reconstruct(kk, delta) for kk in k], np.float32)
            assert np.array_equal(snd.m_codes()[ids[y]].view(np.float32), m_new)
            want_out = m_new.astype(np.float16).view(np.uint16) if dtype == FP16 else \
                torch.tensor(m_new).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
            assert np.array_equal(out[y].reshape(-1), want_out)
        # the error of the store against the halted activation shrinks by 2^-b per visit, with no 16-bit floor
        D = np.abs(a - _f32(a0.reshape(2, E), dtype)).reshape(2, -1, group).max(-1)
        err = np.abs(a - snd.m_codes()[ids].view(np.float32)).reshape(2, -1, group).max(-1)
        assert (err <= D * 2.0 ** (-bits * visit) * (1 + 1e-4) + np.abs(a).reshape(2, -1, group).max(-1) * 2.0 ** -21).all()
    assert err.max() < 1e-3 * D.max()                      # far below what fp16 / bf16 storage could hold


@pytest.mark.parametrize("m_bits", [8, 32])
def test_stochastic_messages_over_the_low_precision_store(m_bits):
    """Unbiased rounding applies to the message only: its codes are those of the separately
    pinned bare stochastic quantizer on a - m_deq (stream = sample id, place = the group's first
    element); the store is re-quantized with the interval number as always, so the receiver,
    which never sees the rounding mode, ends with the same store."""
    rng = np.random.default_rng(43)
    N, seq, hidden, bits, group = 3, 2, 64, 3, 16
    E = seq * hidden
    snd = oracle.SideLow(N, seq, hidden, bits, group, FP16, m_bits)
    rcv = oracle.SideLow(N, seq, hidden, bits, group, FP16, m_bits)
    ids = np.array([2, 0], np.int32)

    def stored(side, sample):
        if m_bits == 32:
            return side.m_codes()[sample].view(np.float32).copy()
        k = oracle.get_codes(side.m_codes()[sample], E, m_bits)
        steps = np.repeat(side.m_scales()[sample], group)
        return np.array([oracle.reconstruct(int(kk), float(dd)) for kk, dd in zip(k, steps)], np.float32)

    a0 = _rand_act(rng, (2, seq, hidden), FP16)
    snd.set_rounding(True, seed=91, epoch=0)
    p, s, first = snd.encode(a0, ids)
    rcv.decode(p, s, ids, raw=a0)
    assert first.all() and not p.any()
    differs = False
    for epoch in range(1, 4):
        snd.set_rounding(True, seed=91, epoch=epoch)
        act = _rand_act(rng, (2, seq, hidden), FP16)
        before = [stored(snd, int(i)) for i in ids]
        p, s, first = snd.encode(act, ids)
        out, _ = rcv.decode(p, s, ids)
        assert not first.any()
        assert np.array_equal(snd.m_codes(), rcv.m_codes()) and np.array_equal(snd.m_scales(), rcv.m_scales())
        assert snd.checksum() == rcv.checksum()
        a = _f32(act.reshape(2, E), FP16)
        for y in range(2):
            d = a[y] - before[y]
            m_new = np.empty(E, np.float32)
            for g in range(E // group):
                sl = slice(g * group, (g + 1) * group)
                k, delta = oracle.quantize_group_stochastic(d[sl], bits, 91, epoch, int(ids[y]), first_elem=g * group)
                assert np.array_equal(oracle.get_codes(p[y], E, bits)[sl], k) and s[y, g] == delta
                differs |= not np.array_equal(k, oracle.quantize_group(d[sl], bits)[0])
                m_new[sl] = before[y][sl] + np.array([oracle.reconstruct(int(kk), delta) for kk in k], np.float32)
                if m_bits != 32:                              # the store's own quantizer: interval number
                    km, dm = oracle.quantize_group(m_new[sl], m_bits)
                    assert np.array_equal(oracle.get_codes(snd.m_codes()[ids[y]], E, m_bits)[sl], km)
                    assert snd.m_scales()[ids[y], g] == dm
            if m_bits == 32:
                assert np.array_equal(stored(snd, int(ids[y])), m_new)
            assert np.array_equal(out[y].reshape(-1), m_new.astype(np.float16).view(np.uint16))
    assert differs                                            # the mode did change some codes
