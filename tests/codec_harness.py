"""Drives one boundary through the CUDA library (sender + receiver handles) and through the
CPU oracle on the same seeded inputs, comparing every output bit for bit."""
import numpy as np
import torch

import oracle
import paper_2206_01299_b200 as aq
from paper_2206_01299_b200 import synth

DT = {"fp16": (aq.AQ_FP16, oracle.FP16), "bf16": (aq.AQ_BF16, oracle.BF16)}


def bits16(t: torch.Tensor) -> np.ndarray:
    """16-bit float tensor (any device) -> numpy uint16 bit patterns."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class GpuSide:
    def __init__(self, cfg, n_batch, stream=None, hosted=False):
        self.cfg = cfg
        create = aq.aq_create_hosted if hosted else aq.aq_create
        self.h = create(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group)
        aq.aq_configure(self.h, aq.AQ_DTYPE, DT[cfg.dtype][0])
        aq.aq_configure(self.h, aq.AQ_BATCH, n_batch)
        if stream is not None:
            aq.aq_configure(self.h, aq.AQ_STREAM, stream.cuda_stream)
        self.first = torch.zeros(max(n_batch, 1), dtype=torch.uint8, device="cuda")
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
    packed = torch.empty((nb, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
    scales = torch.empty((nb, cfg.groups), dtype=torch.float32, device="cuda")
    out = torch.empty((nb, cfg.seq, cfg.hidden), dtype=cfg.torch_dtype, device="cuda")
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
