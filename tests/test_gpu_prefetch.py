"""Hosted store with the previous messages fetched ahead of the call (aq_prefetch): the calls
run on staged rows in device memory and write them back; every output and the whole state must
equal the oracle's, exactly as for calls that work on the host block in place."""
import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from fixtures import synth
from codec_harness import GpuSide, Guarded, bits16, check_guards, run_boundary

pytestmark = pytest.mark.gpu


def test_prefetched_calls_match_the_oracle():
    always = lambda k: True
    run_boundary(synth.TINY, hosted=True, prefetch=always)
    run_boundary(synth.shrink(synth.GPT2_XL, 8, seq=128, epochs=3), n_batch=4, hosted=True, prefetch=always)
    run_boundary(synth.shrink(synth.DEBERTA_XXL, 16, seq=32), hosted=True, stochastic_seed=5, prefetch=always)
    cfg = synth.Boundary("staged-ragged", 6, 3, 37, 136, "bf16", 3, 8, 3, "outlier", 0.3, seed=511)
    run_boundary(cfg, hosted=True, prefetch=always)


def test_prefetched_and_in_place_calls_mix():
    """Staged calls write back on another stream; calls on the host block in place, the digest
    and the checkpoint reads in between must all see the rows that came back."""
    cfg = synth.Boundary("staged-mix", 12, 2, 16, 128, "fp16", 4, 64, 4, "normal", 0.1, seed=512)
    run_boundary(cfg, hosted=True, prefetch=lambda k: k % 3 != 1)
    run_boundary(cfg, hosted=True, prefetch=lambda k: k % 2 == 1)


def test_same_samples_in_consecutive_prefetched_calls():
    """Every call visits the same samples: each prefetch must pick up what the call before it
    has just written back."""
    cfg = synth.Boundary("staged-repeat", 4, 4, 8, 256, "fp16", 2, 32, 5, "normal", 0.2, seed=513)
    run_boundary(cfg, hosted=True, prefetch=lambda k: True)


def test_prefetch_of_many_rows_goes_through_one_kernel():
    """More than 64 rows, or rows below 64 KB, are gathered into the staging block and scattered
    back by one kernel over the mapped host block instead of one copy per row: the largest batch
    of the smallest samples, and a hundred rows of 96 KB."""
    cfg = synth.Boundary("staged-wide", 4096, 4096, 1, 64, "fp16", 4, 64, 2, "normal", 0.1, seed=517)
    run_boundary(cfg, hosted=True, prefetch=lambda k: True, check_all_m=False)
    cfg = synth.Boundary("staged-hundred", 200, 100, 32, 1536, "bf16", 2, 128, 3, "student_t3", 0.02, seed=518)
    run_boundary(cfg, hosted=True, prefetch=lambda k: k != 2, check_all_m=False)


def test_prefetch_of_bad_and_repeated_ids():
    cfg = synth.Boundary("staged-ids", 8, 6, 4, 64, "fp16", 4, 64, 3, "normal", 0.1, seed=514)
    gs, gr = GpuSide(cfg, 6, hosted=True), GpuSide(cfg, 6, hosted=True)
    os_, or_ = (oracle.Side(8, 4, 64, 4, 64, oracle.FP16) for _ in range(2))
    try:
        guards = (Guarded((6, cfg.packed_bytes), torch.uint8), Guarded((6, cfg.groups), torch.float32), Guarded((6, 4, 64), torch.float16))
        packed, scales, out = (g.t for g in guards)
        for epoch in range(3):
            ids = torch.tensor([3, 7, 3, -2, 0, 8], dtype=torch.int32)       # a repeat, two out of range
            act = synth.activation(cfg, torch.arange(6), epoch, device="cuda")
            aq.aq_prefetch(gs.h, ids)
            aq.aq_prefetch(gr.h, ids)
            aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
            aq.aq_configure(gr.h, aq.AQ_RAW, act)
            aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
            torch.cuda.synchronize()
            check_guards(*guards)
            p_o, s_o, f_o = os_.encode(bits16(act), ids.numpy())
            out_o, fr_o = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
            assert np.array_equal(packed.cpu().numpy(), p_o) and np.array_equal(scales.cpu().numpy(), s_o)
            assert np.array_equal(bits16(out), out_o)
            assert np.array_equal(gs.first.cpu().numpy(), f_o) and np.array_equal(gr.first.cpu().numpy(), fr_o)
            assert aq.aq_status(gs.h) == os_.status() == (aq.AQ_ST_BAD_ID | aq.AQ_ST_DUP_ID)
            assert aq.aq_status(gr.h) == or_.status()
            assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
        assert np.array_equal(gs.m_all(), os_.m()) and np.array_equal(gr.m_all(), or_.m())
    finally:
        gs.close(), gr.close(), os_.close(), or_.close()


def test_call_with_other_ids_than_prefetched_skips_those_samples():
    """Position 1 was prefetched for sample 1 and the call brings sample 5: that sample is
    skipped like a bad id (zero codes and scales, neither m(1) nor m(5) touched) and the status
    says so; the other positions work as usual."""
    cfg = synth.Boundary("staged-stale", 8, 4, 4, 64, "fp16", 4, 64, 2, "normal", 0.1, seed=515)
    g, ref = GpuSide(cfg, 4, hosted=True), GpuSide(cfg, 4)
    try:
        packed = torch.empty((4, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
        scales = torch.empty((4, cfg.groups), dtype=torch.float32, device="cuda")
        packed_r, scales_r = torch.empty_like(packed), torch.empty_like(scales)
        all_ids = torch.arange(8, dtype=torch.int32)
        for half in range(2):                                  # every sample seen once, both handles alike
            ids = all_ids[half * 4:half * 4 + 4].contiguous()
            act = synth.activation(cfg, ids, 0, device="cuda")
            aq.aq_encode(g.h, act, ids.cuda(), packed, scales)
            aq.aq_encode(ref.h, act, ids.cuda(), packed_r, scales_r)
        before = g.m_all()
        fetched = torch.tensor([0, 1, 2, 3], dtype=torch.int32)
        brought = torch.tensor([0, 5, 2, 3], dtype=torch.int32)
        act = synth.activation(cfg, brought, 1, device="cuda")
        aq.aq_prefetch(g.h, fetched)
        aq.aq_encode(g.h, act, brought.cuda(), packed, scales)
        aq.aq_encode(ref.h, act, torch.tensor([0, -1, 2, 3], dtype=torch.int32).cuda(), packed_r, scales_r)
        torch.cuda.synchronize()
        assert aq.aq_status(g.h) == aq.AQ_ST_STAGED
        assert aq.aq_status(ref.h) == aq.AQ_ST_BAD_ID
        assert torch.equal(packed, packed_r) and torch.equal(scales, scales_r)
        assert not packed[1].any() and not scales[1].any()
        assert g.first.cpu().tolist() == [0, 0, 0, 0]
        after = g.m_all()
        assert np.array_equal(after, ref.m_all())
        for untouched in (1, 4, 5, 6, 7):
            assert np.array_equal(after[untouched], before[untouched])
        for updated in (0, 2, 3):
            assert not np.array_equal(after[updated], before[updated])
        assert aq.aq_state_checksum(g.h) == aq.aq_state_checksum(ref.h)
    finally:
        g.close(), ref.close()


def test_prefetch_before_the_host_buffer_calls():
    cfg = synth.Boundary("staged-host", 6, 3, 8, 128, "bf16", 3, 64, 3, "normal", 0.1, seed=516)
    gs, gr = GpuSide(cfg, 3, hosted=True), GpuSide(cfg, 3, hosted=True)
    os_, or_ = (oracle.Side(6, 8, 128, 3, 64, oracle.BF16) for _ in range(2))
    try:
        packed = torch.empty((3, cfg.packed_bytes), dtype=torch.uint8).pin_memory()
        scales = torch.empty((3, cfg.groups), dtype=torch.float32).pin_memory()
        out = torch.empty((3, 8, 128), dtype=torch.bfloat16).pin_memory()
        for epoch in range(3):
            order = synth.epoch_order(cfg, epoch)
            for c in range(2):
                ids = order[c * 3:c * 3 + 3].contiguous()
                act = synth.activation(cfg, ids, epoch, device="cpu").pin_memory()
                aq.aq_prefetch(gs.h, ids)
                aq.aq_prefetch(gr.h, ids)
                aq.aq_encode_host(gs.h, act, ids, packed, scales)
                aq.aq_decode_host(gr.h, packed, scales, act, ids, out)
                p_o, s_o, _ = os_.encode(bits16(act), ids.numpy())
                out_o, _ = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
                assert np.array_equal(packed.numpy(), p_o) and np.array_equal(scales.numpy(), s_o)
                assert np.array_equal(bits16(out), out_o)
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
        assert aq.aq_state_checksum_noalloc(gs.h) == os_.checksum()
    finally:
        gs.close(), gr.close(), os_.close(), or_.close()


def test_prefetch_argument_checks():
    dev = aq.aq_create(4, 2, 64, 4, 64)
    hosted = aq.aq_create_hosted(4, 2, 64, 4, 64)
    try:
        ids = torch.tensor([0, 1], dtype=torch.int32)
        with pytest.raises(aq.AqError) as e:
            aq.aq_prefetch(dev, ids[:1])                       # m lives in device memory: nothing to fetch
        assert e.value.code == aq.AQ_EUNSUPPORTED
        aq.aq_configure(hosted, aq.AQ_BATCH, 2)
        with pytest.raises(aq.AqError) as e:
            aq.aq_prefetch(hosted, ids[:1])                    # not AQ_BATCH ids
        assert e.value.code == aq.AQ_EINVAL
        aq.aq_prefetch(hosted, ids)
        aq.aq_configure(hosted, aq.AQ_BATCH, 1)                # the batch size changed under the prefetch
        act = torch.zeros((1, 2, 64), dtype=torch.float16, device="cuda")
        p = torch.zeros(64, dtype=torch.uint8, device="cuda")
        s = torch.zeros(2, dtype=torch.float32, device="cuda")
        with pytest.raises(aq.AqError) as e:
            aq.aq_encode(hosted, act, ids.cuda(), p, s)
        assert e.value.code == aq.AQ_EINVAL
        aq.aq_encode(hosted, act, ids.cuda(), p, s)            # the prefetch is dropped: this one runs in place
        aq.aq_configure(hosted, aq.AQ_BATCH, 0)
        aq.aq_prefetch(hosted, ids[:0])                        # empty call: nothing to do
        assert aq.aq_status(hosted) == 0
    finally:
        aq.aq_destroy(dev), aq.aq_destroy(hosted)


@pytest.mark.parametrize("m_bits", [0, 8])
def test_prefetch_issued_while_the_previous_call_is_in_flight(m_bits):
    """The order a pipeline stage uses: the rows of call N+1 are asked for as soon as call N is
    issued, with no synchronisation anywhere -- the fetch runs beside call N's kernel and beside the
    write-back of its rows, on the second staging block.  Consecutive calls share a sample now and
    then (the fetch then has to wait for that row to come home), a call in between works on the host
    block in place, and one prefetch is replaced before it is used.  Every output is kept and compared
    at the end."""
    cfg = synth.Boundary("staged-overlap", 24, 4, 24, 1536, "bf16" if m_bits else "fp16", 4, 64, 1, "normal", 0.1, seed=519)
    nb, n_calls = 4, 18
    if m_bits:
        create = lambda: aq.aq_create_hosted_lowbit(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, m_bits)
        o_side = lambda: oracle.SideLow(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, oracle.BF16, m_bits)
    else:
        create = lambda: aq.aq_create_hosted(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group)
        o_side = lambda: oracle.Side(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, oracle.FP16)
    stream = torch.cuda.Stream()
    hs, hr = create(), create()
    os_, or_ = o_side(), o_side()
    rng = np.random.default_rng(519)
    calls = []
    for c in range(n_calls):
        ids = rng.choice(cfg.n_samples, nb, replace=False).astype(np.int32)
        if c % 3 == 1 and int(calls[-1][0][2]) not in ids[1:]:
            ids[0] = calls[-1][0][2]                              # a sample of the call before
        calls.append((torch.from_numpy(ids), synth.activation(cfg, torch.arange(nb) + 4 * c, c % 3, device="cuda")))
    outs = [(torch.empty((nb, cfg.packed_bytes), dtype=torch.uint8, device="cuda"),
             torch.empty((nb, cfg.groups), dtype=torch.float32, device="cuda"),
             torch.empty((nb, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")) for _ in range(n_calls)]
    ids_dev = [c[0].cuda() for c in calls]
    torch.cuda.synchronize()
    try:
        for h in (hs, hr):
            aq.aq_configure(h, aq.AQ_DTYPE, aq.AQ_BF16 if m_bits else aq.AQ_FP16)
            aq.aq_configure(h, aq.AQ_BATCH, nb)
            aq.aq_configure(h, aq.AQ_STREAM, stream.cuda_stream)
        in_place = {7, 13}                                        # these calls fetch nothing ahead
        aq.aq_prefetch(hs, calls[0][0]), aq.aq_prefetch(hr, calls[0][0])
        for c, (ids, act) in enumerate(calls):
            packed, scales, out = outs[c]
            aq.aq_encode(hs, act, ids_dev[c], packed, scales)
            aq.aq_configure(hr, aq.AQ_RAW, act)
            aq.aq_decode(hr, packed, scales, ids_dev[c], out)
            if c + 1 < n_calls and c + 1 not in in_place:
                if c == 4:                                        # a prefetch for other samples, replaced before its call
                    aq.aq_prefetch(hs, calls[c][0]), aq.aq_prefetch(hr, calls[c][0])
                aq.aq_prefetch(hs, calls[c + 1][0]), aq.aq_prefetch(hr, calls[c + 1][0])
        torch.cuda.synchronize()
        for c, (ids, act) in enumerate(calls):
            a_np = bits16(act)
            p_o, s_o, _ = os_.encode(a_np, ids.numpy())
            out_o, _ = or_.decode(p_o, s_o, ids.numpy(), raw=a_np)
            packed, scales, out = outs[c]
            assert np.array_equal(packed.cpu().numpy(), p_o), (c, "packed")
            assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32)), (c, "scales")
            assert np.array_equal(bits16(out), out_o), (c, "out")
        assert aq.aq_status(hs) == 0 and aq.aq_status(hr) == 0
        assert aq.aq_state_checksum(hs) == aq.aq_state_checksum(hr) == os_.checksum() == or_.checksum()
    finally:
        aq.aq_destroy(hs), aq.aq_destroy(hr), os_.close(), or_.close()
