"""Seeded random shapes through the whole boundary, every element against the CPU oracle.

The hand-picked cases elsewhere sit on the corners that were thought of; these walk the space in
between: bit width, type, group size, sequence length, hidden size, samples per call and value
recipe are drawn from a fixed seed, so that a failure names a case that can be run again.  Three
families: small calls (ragged rows, single chunks, calls that leave multiprocessors idle), calls
around the size from which the receiver's grid ends in smaller CTAs (a few samples more or fewer than
two waves of full-size CTAs, odd and ragged row counts), and gradients of random length; the small shapes
also go through the optional modes (stochastic rounding, low-precision and binary32 stores, the store in
host memory with and without prefetch)."""
import random

import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from codec_harness import DT, Guarded, bits16, check_guards, run_boundary
from fixtures import synth
from test_gpu_lowbit import run_lowbit

pytestmark = pytest.mark.gpu

KINDS = ("normal", "outlier", "student_t3")


def _small_case(i):
    rng = random.Random(9000 + i)
    group = rng.choice((8, 8, 16, 32, 64, 128, 256, 24, 40, 72, 104, 288, 8 * rng.randint(1, 60)))
    hidden = group * rng.randint(1, max(1, 1536 // group))
    seq = rng.choice((1, 2, 3, 5, 8, 13, 21, 34, 40))
    n_batch = rng.randint(1, 9)
    n_samples = n_batch * rng.randint(1, 3)
    return synth.Boundary(f"fuzz-small-{i}", n_samples, n_batch, seq, hidden, rng.choice(("fp16", "bf16")),
                          rng.randint(1, 8), group, rng.randint(2, 3), rng.choice(KINDS),
                          rng.choice((0.02, 0.3, 1.0)), seed=9000 + i)


def _power_of_two_group(cfg):
    """The low-precision stores take groups of 8 to 256 elements in powers of two: the nearest one below."""
    g = 8
    while g * 2 <= min(cfg.group, 256) and cfg.hidden % (g * 2) == 0:
        g *= 2
    return synth.Boundary(cfg.name, cfg.n_samples, cfg.n_batch, cfg.seq, cfg.hidden, cfg.dtype, cfg.bits, g,
                          cfg.epochs, cfg.kind, cfg.drift, seed=cfg.seed)


def _large_case(i):
    """One call of about two waves of four-row CTAs (six resident per multiprocessor): the number of
    samples is drawn on either side of that size."""
    rng = random.Random(9500 + i)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    group = rng.choice((8, 16, 64))
    hidden = group * rng.randint(1024 // group, 2048 // group)
    rows = rng.randint(20, 60) + rng.random()                     # rows of 256 chunks per sample, ragged
    seq = max(1, round(rows * 2048 / hidden))
    rows = -(-seq * hidden // 2048)
    ctas_per_sample = -(-rows // 4)
    n_batch = max(2, 2 * 6 * sms // ctas_per_sample + rng.randint(-3, 6))
    return synth.Boundary(f"fuzz-large-{i}", n_batch, n_batch, seq, hidden, rng.choice(("fp16", "bf16")),
                          rng.choice((2, 3, 4, 6)), group, 3, rng.choice(KINDS), 0.1, seed=9500 + i)


@pytest.mark.parametrize("i", range(48))
def test_small_random_shapes(i):
    run_boundary(_small_case(i))


@pytest.mark.parametrize("i", range(10))
def test_random_shapes_around_the_tapered_grid(i):
    cfg = _large_case(i)
    assert cfg.n_batch <= 4096
    run_boundary(cfg)


@pytest.mark.parametrize("i", range(32))
def test_random_gradient_lengths(i):
    """aq_quant_grad / aq_dequant_grad on lengths drawn around the multiples of what one CTA takes
    (6144 elements for the dequantizer, twice that for the sixteen-elements-per-lane quantizer) and
    of a warp's share, values spread over many binades; guard regions behind every output."""
    rng = random.Random(9800 + i)
    group = rng.choice((8, 16, 32, 64, 128, 256, 24, 56, 200, 8 * rng.randint(1, 80)))
    bits = rng.randint(1, 8)
    dtype = rng.choice(("fp16", "bf16"))
    td = torch.float16 if dtype == "fp16" else torch.bfloat16
    tile = rng.choice((256, 6144, 12288))
    n = max(group, (tile * rng.randint(1, 40) + rng.randint(-3, 3) * group) // group * group)
    gen = torch.Generator().manual_seed(9800 + i)
    x = torch.randn(n, generator=gen) * torch.exp2(torch.randint(-12, 6, (n,), generator=gen).float())
    x[torch.rand(n, generator=gen) < 0.01] = 0.0
    grad = x.to(td).cuda()
    h = aq.aq_create(1, 1, group, 4, group)
    try:
        aq.aq_configure(h, aq.AQ_DTYPE, DT[dtype][0])
        guards = (Guarded(n * bits // 8, torch.uint8), Guarded(n // group, torch.float32), Guarded(n, td))
        packed, scales, out = (g.t for g in guards)
        aq.aq_quant_grad(h, grad, n, bits, packed, scales)
        aq.aq_dequant_grad(h, packed, scales, n, bits, out)
        torch.cuda.synchronize()
        check_guards(*guards)
        p_o, s_o = oracle.quant_grad(bits16(grad), bits, group, DT[dtype][1])
        o_o = oracle.dequant_grad(p_o, s_o, n, bits, group, DT[dtype][1])
        assert np.array_equal(packed.cpu().numpy(), p_o), (n, bits, group, dtype)
        assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32)), (n, bits, group, dtype)
        assert np.array_equal(bits16(out), o_o), (n, bits, group, dtype)
        assert aq.aq_status(h) == 0
    finally:
        aq.aq_destroy(h)


@pytest.mark.parametrize("i", range(24))
def test_small_random_shapes_through_the_optional_modes(i):
    rng = random.Random(9900 + i)
    cfg = _small_case(100 + i)
    mode = i % 4
    if mode == 0:                                    # unbiased stochastic rounding of the messages
        run_boundary(cfg, stochastic_seed=rng.getrandbits(40))
    elif mode == 1:                                  # previous messages kept in 2, 4, 8 bits or binary32
        run_lowbit(_power_of_two_group(cfg), rng.choice((2, 4, 8, 32)), stochastic_seed=rng.choice((None, 77)))
    elif mode == 2:                                  # m in page-locked host memory; some calls prefetched
        pattern = rng.getrandbits(16) | 1
        run_boundary(cfg, hosted=True, prefetch=lambda k: (pattern >> (k % 16)) & 1 == 1)
    else:                                            # low-precision store in host memory
        run_lowbit(_power_of_two_group(cfg), rng.choice((2, 4, 8)), hosted=True, prefetch=lambda k: k % 2 == 0)
