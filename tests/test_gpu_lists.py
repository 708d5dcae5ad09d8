"""List forms of the calls (aq_encode_list / aq_decode_list): every sample of a call in a buffer of
its own, named through device arrays of pointers.  Same kernels, so the results must be those of the
CPU oracle bit for bit, and nothing may be written outside any of the scattered buffers."""
import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from fixtures import synth
from codec_harness import DT, GpuSide, Guarded, bits16

pytestmark = pytest.mark.gpu


def addresses(tensors):
    """Device array of the tensors' addresses (0 for None)."""
    return torch.tensor([0 if t is None else t.data_ptr() for t in tensors], dtype=torch.int64, device="cuda")


class Scattered:
    """The buffers of one call, one guarded allocation per sample and kind."""

    def __init__(self, cfg, nb):
        self.act = [Guarded((cfg.seq, cfg.hidden), cfg.torch_dtype) for _ in range(nb)]
        self.packed = [Guarded(cfg.packed_bytes, torch.uint8) for _ in range(nb)]
        self.scales = [Guarded(cfg.groups, torch.float32) for _ in range(nb)]
        self.out = [Guarded((cfg.seq, cfg.hidden), cfg.torch_dtype) for _ in range(nb)]

    def check(self):
        for kind in (self.act, self.packed, self.scales, self.out):
            for g in kind:
                g.check("a scattered buffer")


@pytest.mark.parametrize("cfg,nb", [
    (synth.shrink(synth.GPT2_XL, 12, seq=40, epochs=3), 4),
    (synth.shrink(synth.DEBERTA_XXL, 16, seq=24), 8),
    (synth.shrink(synth.SWEEP_FWD, 6, seq=16), 3),
    (synth.Boundary("list-ragged", 6, 3, 37, 136, "bf16", 5, 8, 3, "outlier", 0.3, seed=71), 3),
    (synth.Boundary("list-group-40", 6, 3, 11, 640, "fp16", 3, 40, 3, "outlier", 0.3, seed=72), 3),
    (synth.Boundary("list-group-row", 4, 2, 9, 1600, "bf16", 4, 1600, 3, "normal", 0.3, seed=73), 2),
])
def test_list_forms_match_the_oracle(cfg, nb):
    gs, gr = GpuSide(cfg, nb), GpuSide(cfg, nb)
    od = DT[cfg.dtype][1]
    os_, or_ = (oracle.Side(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, od) for _ in range(2))
    bufs = Scattered(cfg, nb)
    act_l, packed_l = addresses([g.t for g in bufs.act]), addresses([g.t for g in bufs.packed])
    scales_l, out_l = addresses([g.t for g in bufs.scales]), addresses([g.t for g in bufs.out])
    try:
        aq.aq_configure(gr.h, aq.AQ_RAW_LIST, act_l)                  # first visits: the raw message is the activation
        for epoch in range(cfg.epochs):
            order = synth.epoch_order(cfg, epoch)
            for c in range(cfg.n_samples // nb):
                ids = order[c * nb:(c + 1) * nb].contiguous()
                act = synth.activation(cfg, ids, epoch, device="cuda")
                for y in range(nb):
                    bufs.act[y].t.copy_(act[y])
                    bufs.packed[y].t.fill_(0xAB), bufs.scales[y].t.fill_(-7.0), bufs.out[y].t.fill_(3.0)
                ids_d = ids.cuda()
                aq.aq_encode_list(gs.h, act_l, ids_d, packed_l, scales_l)
                aq.aq_decode_list(gr.h, packed_l, scales_l, ids_d, out_l)
                torch.cuda.synchronize()
                bufs.check()
                a_np = bits16(act)
                p_o, s_o, f_o = os_.encode(a_np, ids.numpy())
                out_o, fr_o = or_.decode(p_o, s_o, ids.numpy(), raw=a_np)
                for y in range(nb):
                    assert np.array_equal(bufs.packed[y].t.cpu().numpy(), p_o[y]), (epoch, c, y, "packed")
                    assert np.array_equal(bufs.scales[y].t.cpu().numpy().view(np.uint32), s_o[y].view(np.uint32)), (epoch, c, y)
                    assert np.array_equal(bits16(bufs.out[y].t), out_o[y]), (epoch, c, y, "out")
                assert np.array_equal(gs.first.cpu().numpy()[:nb], f_o) and np.array_equal(gr.first.cpu().numpy()[:nb], fr_o)
            assert aq.aq_status(gs.h) == 0 and aq.aq_status(gr.h) == 0
            assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
        assert np.array_equal(gs.m_all(), os_.m()) and np.array_equal(gr.m_all(), or_.m())
    finally:
        gs.close(), gr.close(), os_.close(), or_.close()


def test_list_and_base_pointer_forms_mix_on_one_handle():
    """A call in one form, the next in the other: the state does not care how a call named its buffers."""
    cfg = synth.Boundary("list-mix", 8, 4, 9, 256, "fp16", 4, 64, 3, "normal", 0.05, seed=72)
    nb = 4
    gs, gr = GpuSide(cfg, nb), GpuSide(cfg, nb)
    os_, or_ = (oracle.Side(8, 9, 256, 4, 64, oracle.FP16) for _ in range(2))
    bufs = Scattered(cfg, nb)
    lists = [addresses([g.t for g in kind]) for kind in (bufs.act, bufs.packed, bufs.scales, bufs.out)]
    packed = torch.empty((nb, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
    scales = torch.empty((nb, cfg.groups), dtype=torch.float32, device="cuda")
    out = torch.empty((nb, cfg.seq, cfg.hidden), dtype=torch.float16, device="cuda")
    try:
        aq.aq_configure(gr.h, aq.AQ_RAW_LIST, lists[0])
        call = 0
        for epoch in range(3):
            order = synth.epoch_order(cfg, epoch)
            for c in range(2):
                ids = order[c * nb:(c + 1) * nb].contiguous()
                act = synth.activation(cfg, ids, epoch, device="cuda")
                ids_d = ids.cuda()
                if call % 2 == 0:
                    for y in range(nb):
                        bufs.act[y].t.copy_(act[y])
                    aq.aq_encode_list(gs.h, lists[0], ids_d, lists[1], lists[2])
                    aq.aq_decode_list(gr.h, lists[1], lists[2], ids_d, lists[3])
                    torch.cuda.synchronize()
                    bufs.check()
                    got_p = np.stack([g.t.cpu().numpy() for g in bufs.packed])
                    got_o = np.stack([bits16(g.t) for g in bufs.out])
                else:
                    aq.aq_encode(gs.h, act, ids_d, packed, scales)
                    aq.aq_configure(gr.h, aq.AQ_RAW, act)
                    aq.aq_decode(gr.h, packed, scales, ids_d, out)
                    torch.cuda.synchronize()
                    got_p, got_o = packed.cpu().numpy(), bits16(out)
                call += 1
                p_o, s_o, _ = os_.encode(bits16(act), ids.numpy())
                out_o, _ = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
                assert np.array_equal(got_p, p_o) and np.array_equal(got_o, out_o), (epoch, c)
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
    finally:
        gs.close(), gr.close(), os_.close(), or_.close()


def test_bad_pointers_in_a_list_skip_the_sample_and_are_reported():
    cfg = synth.Boundary("list-bad", 6, 3, 5, 128, "fp16", 4, 64, 1, "normal", 0.1, seed=73)
    nb = 3
    gs, gr = GpuSide(cfg, nb), GpuSide(cfg, nb)
    os_, or_ = (oracle.Side(6, 5, 128, 4, 64, oracle.FP16) for _ in range(2))
    bufs = Scattered(cfg, nb)
    try:
        ids = torch.tensor([4, 0, 2], dtype=torch.int32)
        act = synth.activation(cfg, ids, 0, device="cuda")
        for y in range(nb):
            bufs.act[y].t.copy_(act[y])
            bufs.packed[y].t.fill_(0xAB), bufs.scales[y].t.fill_(-7.0), bufs.out[y].t.fill_(3.0)
        act_l = addresses([g.t for g in bufs.act])
        packed_l = addresses([g.t for g in bufs.packed])
        scales_l = addresses([g.t for g in bufs.scales])
        out_l = addresses([g.t for g in bufs.out])
        packed_bad = packed_l.clone()
        packed_bad[1] += 4                                            # sample 1: a pointer that is not 16-byte aligned
        act_bad = act_l.clone()
        act_bad[2] = 0                                                # sample 2: no activation
        aq.aq_encode_list(gs.h, act_bad, ids.cuda(), packed_bad, scales_l)
        assert aq.aq_status(gs.h) == aq.AQ_ST_BAD_PTR
        bufs.check()
        # sample 0 went through; nothing was read or written for the other two, which stay unseen
        p_o, s_o, _ = os_.encode(bits16(act[:1]), ids[:1].numpy())
        assert np.array_equal(bufs.packed[0].t.cpu().numpy(), p_o[0])
        for y in (1, 2):
            assert (bufs.packed[y].t == 0xAB).all() and (bufs.scales[y].t == -7.0).all()
        assert [gs.m_row(i)[1] for i in (4, 0, 2)] == [1, 0, 0]
        assert aq.aq_state_checksum(gs.h) == os_.checksum()
        # receiver: a null raw entry is "no raw message" (reported as such), a null output pointer is a bad pointer
        raw_l = act_l.clone()
        raw_l[1] = 0
        out_bad = out_l.clone()
        out_bad[2] = 0
        aq.aq_configure(gr.h, aq.AQ_RAW_LIST, raw_l)
        for y in range(nb):
            bufs.packed[y].t.zero_(), bufs.scales[y].t.zero_()
        aq.aq_decode_list(gr.h, packed_l, scales_l, ids.cuda(), out_bad)
        assert aq.aq_status(gr.h) == (aq.AQ_ST_BAD_PTR | aq.AQ_ST_NO_RAW)
        bufs.check()
        assert np.array_equal(bits16(bufs.out[0].t), bits16(act[0]))          # first visit: the raw message
        assert not bufs.out[1].t.any()                                         # skipped: zeros
        assert (bufs.out[2].t == 3.0).all()                                    # untouched
        assert [gr.m_row(i)[1] for i in (4, 0, 2)] == [1, 0, 0]
        # low-precision stores have no list form
        low = aq.aq_create_lowbit(4, 2, 64, 4, 64, 8)
        try:
            with pytest.raises(aq.AqError) as e:
                aq.aq_encode_list(low, act_l, ids.cuda(), packed_l, scales_l)
            assert e.value.code == aq.AQ_EUNSUPPORTED
        finally:
            aq.aq_destroy(low)
    finally:
        gs.close(), gr.close(), os_.close(), or_.close()
