"""Drives one boundary through the CUDA library (sender + receiver handles) and through the
CPU oracle on the same seeded inputs, comparing every output bit for bit."""
import numpy as np
import torch

import oracle
import paper_2206_01299_b200 as aq
from fixtures import synth

DT = {"fp16": (aq.AQ_FP16, oracle.FP16), "bf16": (aq.AQ_BF16, oracle.BF16)}


def bits16(t: torch.Tensor) -> np.ndarray:
    """16-bit float tensor (any device) -> numpy uint16 bit patterns."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


GUARD_BYTES = 512
GUARD_FILL = 0x5A


class Guarded:
    """A device buffer with GUARD_BYTES of a known pattern in front of it and behind it.  `.t` is
    the buffer itself (the view handed to the library); check() fails when a kernel wrote outside
    it.  Stands in for a memory checker: a store one word past the end of an output lands here."""

    def __init__(self, shape, dtype, device="cuda"):
        shape = (shape,) if isinstance(shape, int) else tuple(shape)
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.body = (n + 15) // 16 * 16                       # the tail guard starts at the next 16-byte boundary at the latest
        self.n = n
        self.raw = torch.full((GUARD_BYTES + self.body + GUARD_BYTES,), GUARD_FILL, dtype=torch.uint8, device=device)
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)

    def check(self, what=""):
        front = self.raw[:GUARD_BYTES].cpu().numpy()
        behind = self.raw[GUARD_BYTES + self.n:].cpu().numpy()
        assert (front == GUARD_FILL).all(), f"write in front of {what}"
        assert (behind == GUARD_FILL).all(), f"write behind {what}"


class GpuSide:
    def __init__(self, cfg, n_batch, stream=None, hosted=False):
        self.cfg = cfg
        create = aq.aq_create_hosted if hosted else aq.aq_create
        self.h = create(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group)
        aq.aq_configure(self.h, aq.AQ_DTYPE, DT[cfg.dtype][0])
        aq.aq_configure(self.h, aq.AQ_BATCH, n_batch)
        if stream is not None:
            aq.aq_configure(self.h, aq.AQ_STREAM, stream.cuda_stream)
        self.first_guarded = Guarded(max(n_batch, 1), torch.uint8)
        self.first = self.first_guarded.t
        self.first.zero_()
        aq.aq_configure(self.h, aq.AQ_FIRST_FLAGS, self.first)

    def close(self):
        if self.h:
            aq.aq_destroy(self.h)
            self.h = None

    def m_row(self, sample_id):
        buf = np.empty(self.cfg.elems, np.uint16)
        seen = aq.aq_export_sample(self.h, int(sample_id), buf)
        return buf.reshape(self.cfg.seq, self.cfg.hidden), seen

    def m_all(self):
        return np.stack([self.m_row(i)[0] for i in range(self.cfg.n_samples)])


def guarded_outputs(cfg, nb):
    """(packed, scales, out) of a call of nb samples as Guarded buffers."""
    return (Guarded((nb, cfg.packed_bytes), torch.uint8), Guarded((nb, cfg.groups), torch.float32),
            Guarded((nb, cfg.seq, cfg.hidden), cfg.torch_dtype))


def check_guards(*guarded):
    for i, g in enumerate(guarded):
        g.check(f"output buffer {i}")


def run_boundary(cfg, n_batch=None, epochs=None, check_all_m=True, order_fn=None, act_fn=None, stochastic_seed=None,
                 hosted=False, prefetch=None, l2_prefetch=None):
    """Every call of every epoch: GPU sender -> GPU receiver and oracle sender -> oracle
    receiver; packed, scales, first flags, out and (per epoch) both m arrays and the state
    digests must agree exactly.  prefetch (hosted handles): a function of the call's running
    number saying whether the two sides fetch that call's previous messages ahead of it."""
    nb = n_batch or cfg.n_batch
    epochs = epochs or cfg.epochs
    assert cfg.n_samples % nb == 0
    gs, gr = GpuSide(cfg, nb, hosted=hosted), GpuSide(cfg, nb, hosted=hosted)
    od = DT[cfg.dtype][1]
    os_, or_ = (oracle.Side(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, od) for _ in range(2))
    g_packed = Guarded((nb, cfg.packed_bytes), torch.uint8)
    g_scales = Guarded((nb, cfg.groups), torch.float32)
    g_out = Guarded((nb, cfg.seq, cfg.hidden), cfg.torch_dtype)
    packed, scales, out = g_packed.t, g_scales.t, g_out.t
    calls = 0
    try:
        if l2_prefetch is not None:
            aq.aq_configure(gs.h, aq.AQ_L2_PREFETCH, int(l2_prefetch))
            aq.aq_configure(gr.h, aq.AQ_L2_PREFETCH, int(l2_prefetch))
        if stochastic_seed is not None:                      # only the sender rounds; the receiver needs no setting
            aq.aq_configure(gs.h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
            aq.aq_configure(gs.h, aq.AQ_SEED, stochastic_seed)
        for epoch in range(epochs):
            if stochastic_seed is not None:
                aq.aq_configure(gs.h, aq.AQ_EPOCH, (epoch << 33) | 5)          # both counter words in use
                os_.set_rounding(True, stochastic_seed, (epoch << 33) | 5)
            order = order_fn(epoch) if order_fn else synth.epoch_order(cfg, epoch)
            for c in range(cfg.n_samples // nb):
                ids = order[c * nb:(c + 1) * nb].contiguous()
                act = act_fn(ids, epoch) if act_fn else synth.activation(cfg, ids, epoch, device="cuda")
                ids_d = ids.cuda()
                packed.fill_(0xAB)
                scales.fill_(-7.0)
                out.fill_(3.0)
                if prefetch and prefetch(calls):
                    aq.aq_prefetch(gs.h, ids)
                    aq.aq_prefetch(gr.h, ids)
                calls += 1
                aq.aq_encode(gs.h, act, ids_d, packed, scales)
                aq.aq_configure(gr.h, aq.AQ_RAW, act)        # first visits: the raw message is the activation
                aq.aq_decode(gr.h, packed, scales, ids_d, out)
                torch.cuda.synchronize()
                act_np, ids_np = bits16(act), ids.numpy()
                p_o, s_o, f_o = os_.encode(act_np, ids_np)
                out_o, fr_o = or_.decode(p_o, s_o, ids_np, raw=act_np)
                assert np.array_equal(packed.cpu().numpy(), p_o), (epoch, c, "packed")
                assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32)), (epoch, c, "scales")
                assert np.array_equal(gs.first.cpu().numpy()[:nb], f_o), (epoch, c, "first (sender)")
                assert np.array_equal(gr.first.cpu().numpy()[:nb], fr_o), (epoch, c, "first (receiver)")
                assert np.array_equal(bits16(out), out_o), (epoch, c, "out")
                for g, what in ((g_packed, "packed"), (g_scales, "scales"), (g_out, "out"),
                                (gs.first_guarded, "first flags (sender)"), (gr.first_guarded, "first flags (receiver)")):
                    g.check(what)
            assert aq.aq_status(gs.h) == os_.status() and aq.aq_status(gr.h) == or_.status()
            cs = aq.aq_state_checksum(gs.h)
            assert cs == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum(), (epoch, "digest")
            if check_all_m:
                assert np.array_equal(gs.m_all(), os_.m()), (epoch, "sender m")
                assert np.array_equal(gr.m_all(), or_.m()), (epoch, "receiver m")
    finally:
        gs.close()
        gr.close()
        os_.close()
        or_.close()
