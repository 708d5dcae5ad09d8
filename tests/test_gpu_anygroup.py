"""Group sizes whose eight-element pieces are not a power of two within one warp: 24, 40, 48, 96 ...
elements, and groups longer than 256 up to a whole hidden row (Section 4.1 "Baselines" normalises "a
vector"; which vector is the caller's choice).  They run on kernels of their own; the oracle is the
same definition for every group size, and everything is compared bit for bit as elsewhere."""
import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from codec_harness import DT, Guarded, bits16, check_guards, run_boundary
from fixtures import synth

pytestmark = pytest.mark.gpu

# (group, hidden): 3, 5, 6, 12 and 30 lanes inside one warp-tile; 40, 64 and 200 lanes: several per lane
SHAPES = [(24, 96), (40, 640), (48, 1536), (96, 768), (240, 1200), (320, 1600), (512, 1536), (1600, 1600)]


@pytest.mark.parametrize("group,hidden", SHAPES)
@pytest.mark.parametrize("dtype,bits", [("fp16", 4), ("bf16", 2), ("fp16", 3), ("bf16", 7)])
def test_boundary_with_other_group_sizes(group, hidden, dtype, bits):
    cfg = synth.Boundary("anygroup", 8, 4, 7, hidden, dtype, bits, group, 3, "outlier", 0.2, seed=group + bits)
    run_boundary(cfg)


@pytest.mark.parametrize("group,hidden", [(24, 1200), (1600, 1600)])
def test_larger_calls_and_a_single_token(group, hidden):
    # enough groups for several CTAs per sample, then one token per sample (a single group when group == hidden)
    run_boundary(synth.Boundary("anygroup-long", 6, 3, 150, hidden, "fp16", 4, group, 3, "student_t3", 0.1, seed=group))
    run_boundary(synth.Boundary("anygroup-token", 4, 2, 1, hidden, "bf16", 5, group, 3, "normal", 0.5, seed=group + 1))


@pytest.mark.parametrize("group,hidden", [(48, 1536), (320, 1600)])
def test_stochastic_rounding_and_hosted_store_with_other_group_sizes(group, hidden):
    cfg = synth.Boundary("anygroup-modes", 8, 4, 9, hidden, "fp16", 3, group, 3, "outlier", 0.3, seed=group + 7)
    run_boundary(cfg, stochastic_seed=99)
    run_boundary(cfg, hosted=True, prefetch=lambda k: k % 2 == 0)


@pytest.mark.parametrize("group", [24, 40, 96, 320, 1600])
@pytest.mark.parametrize("dtype,bits", [("fp16", 8), ("bf16", 4), ("fp16", 6), ("bf16", 1)])
def test_gradients_with_other_group_sizes(group, dtype, bits):
    td = torch.float16 if dtype == "fp16" else torch.bfloat16
    n = group * 517                                    # ragged against every tile of the kernels
    gen = torch.Generator().manual_seed(group * 10 + bits)
    x = torch.randn(n, generator=gen) * torch.exp2(torch.randint(-10, 5, (n,), generator=gen).float())
    x[:group] = 0.0                                    # a dead group
    grad = x.to(td).cuda()
    h = aq.aq_create(1, 1, group, 4, group)
    try:
        aq.aq_configure(h, aq.AQ_DTYPE, DT[dtype][0])
        for stochastic in (False, True):
            if stochastic:
                aq.aq_configure(h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
                aq.aq_configure(h, aq.AQ_SEED, 4242)
                aq.aq_configure(h, aq.AQ_EPOCH, 17)
            guards = (Guarded(n * bits // 8, torch.uint8), Guarded(n // group, torch.float32), Guarded(n, td))
            packed, scales, out = (g.t for g in guards)
            aq.aq_quant_grad(h, grad, n, bits, packed, scales)
            aq.aq_dequant_grad(h, packed, scales, n, bits, out)
            torch.cuda.synchronize()
            check_guards(*guards)
            if stochastic:
                p_o, s_o = oracle.quant_grad_stochastic(bits16(grad), bits, group, 4242, 17, DT[dtype][1])
            else:
                p_o, s_o = oracle.quant_grad(bits16(grad), bits, group, DT[dtype][1])
            o_o = oracle.dequant_grad(p_o, s_o, n, bits, group, DT[dtype][1])
            assert np.array_equal(packed.cpu().numpy(), p_o), (stochastic, "codes")
            assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32)), (stochastic, "steps")
            assert np.array_equal(bits16(out), o_o), (stochastic, "out")
        assert aq.aq_status(h) == 0
    finally:
        aq.aq_destroy(h)


def test_what_other_group_sizes_do_not_offer():
    """The low-precision and binary32 stores have kernels for groups of 8 to 256 elements in powers of
    two only, and say so."""
    for create in (lambda: aq.aq_create_lowbit(4, 2, 96, 4, 24, 4), lambda: aq.aq_create_fp32(4, 2, 96, 4, 24),
                   lambda: aq.aq_create_hosted_lowbit(4, 2, 96, 4, 24, 8)):
        with pytest.raises(aq.AqError) as e:
            create()
        assert e.value.code == aq.AQ_EUNSUPPORTED
