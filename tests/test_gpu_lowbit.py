"""The low-precision store of previous messages (aq_create_lowbit: m kept in 2, 4 or 8 bits per
element) against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from fixtures import synth
from codec_harness import DT, Guarded, bits16, check_guards

pytestmark = pytest.mark.gpu


class LowSide:
    def __init__(self, cfg, n_batch, m_bits, hosted=False):
        self.cfg, self.m_bits = cfg, m_bits
        self.h = (aq.aq_create_hosted_lowbit(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, m_bits) if hosted
                  else aq.aq_create_fp32(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group) if m_bits == 32
                  else aq.aq_create_lowbit(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, m_bits))
        aq.aq_configure(self.h, aq.AQ_DTYPE, DT[cfg.dtype][0])
        aq.aq_configure(self.h, aq.AQ_BATCH, n_batch)
        self.first_guarded = Guarded(n_batch, torch.uint8)
        self.first = self.first_guarded.t
        self.first.zero_()
        aq.aq_configure(self.h, aq.AQ_FIRST_FLAGS, self.first)
        self.code_bytes = cfg.elems * m_bits // 8
        self.n_steps = 0 if m_bits == 32 else cfg.groups
        assert aq.aq_m_bytes_per_sample(self.h) == self.code_bytes + self.n_steps * 4

    def close(self):
        aq.aq_destroy(self.h)

    def state(self):
        """(codes uint8[n, code_bytes], steps float32[n, groups], seen uint8[n])"""
        n = self.cfg.n_samples
        codes = np.empty((n, self.code_bytes), np.uint8)
        steps = np.empty((n, self.n_steps), np.float32)
        seen = np.empty(n, np.uint8)
        buf = np.empty(self.code_bytes + self.n_steps * 4, np.uint8)
        for i in range(n):
            seen[i] = aq.aq_export_sample(self.h, i, buf)
            codes[i] = buf[:self.code_bytes]
            steps[i] = buf[self.code_bytes:].view(np.float32)
        return codes, steps, seen


def run_lowbit(cfg, m_bits, n_batch=None, stochastic_seed=None, hosted=False, prefetch=None):
    nb = n_batch or cfg.n_batch
    gs, gr = LowSide(cfg, nb, m_bits, hosted), LowSide(cfg, nb, m_bits, hosted)
    od = DT[cfg.dtype][1]
    os_, or_ = (oracle.SideLow(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, od, m_bits) for _ in range(2))
    g_packed = Guarded((nb, cfg.packed_bytes), torch.uint8)
    g_scales = Guarded((nb, cfg.groups), torch.float32)
    g_out = Guarded((nb, cfg.seq, cfg.hidden), cfg.torch_dtype)
    packed, scales, out = g_packed.t, g_scales.t, g_out.t
    calls = 0
    try:
        if stochastic_seed is not None:                      # only the sender rounds
            aq.aq_configure(gs.h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
            aq.aq_configure(gs.h, aq.AQ_SEED, stochastic_seed)
        for epoch in range(cfg.epochs):
            if stochastic_seed is not None:
                aq.aq_configure(gs.h, aq.AQ_EPOCH, (epoch << 33) | 3)
                os_.set_rounding(True, stochastic_seed, (epoch << 33) | 3)
            order = synth.epoch_order(cfg, epoch)
            for c in range(cfg.n_samples // nb):
                ids = order[c * nb:(c + 1) * nb].contiguous()
                act = synth.activation(cfg, ids, epoch, device="cuda")
                packed.fill_(0xAB)
                scales.fill_(-7.0)
                out.fill_(3.0)
                if prefetch and prefetch(calls):                 # hosted store: rows fetched ahead of the call
                    aq.aq_prefetch(gs.h, ids)
                    aq.aq_prefetch(gr.h, ids)
                calls += 1
                aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
                aq.aq_configure(gr.h, aq.AQ_RAW, act)
                aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
                torch.cuda.synchronize()
                a_np = bits16(act)
                p_o, s_o, f_o = os_.encode(a_np, ids.numpy())
                out_o, fr_o = or_.decode(p_o, s_o, ids.numpy(), raw=a_np)
                assert np.array_equal(packed.cpu().numpy(), p_o), (epoch, c, "packed")
                assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32)), (epoch, c, "scales")
                assert np.array_equal(gs.first.cpu().numpy(), f_o) and np.array_equal(gr.first.cpu().numpy(), fr_o)
                assert np.array_equal(bits16(out), out_o), (epoch, c, "out")
                for g, what in ((g_packed, "packed"), (g_scales, "scales"), (g_out, "out"),
                                (gs.first_guarded, "first flags (sender)"), (gr.first_guarded, "first flags (receiver)")):
                    g.check(what)
            for g_side, o_side in ((gs, os_), (gr, or_)):
                codes, steps, seen = g_side.state()
                assert np.array_equal(codes, o_side.m_codes()), (epoch, "stored codes")
                assert np.array_equal(steps.view(np.uint32), o_side.m_scales().view(np.uint32)), (epoch, "stored steps")
                assert np.array_equal(seen, o_side.seen())
            assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
            assert aq.aq_status(gs.h) == 0 and aq.aq_status(gr.h) == 0
    finally:
        gs.close()
        gr.close()
        os_.close()
        or_.close()


@pytest.mark.parametrize("m_bits", [2, 4, 8, 32])
def test_tiny_boundary_with_a_low_precision_store(m_bits):
    run_lowbit(synth.TINY, m_bits)


@pytest.mark.parametrize("m_bits", [2, 8, 32])
def test_large_shapes_reduced_id_space(m_bits):
    run_lowbit(synth.shrink(synth.GPT2_XL, 8, seq=96, epochs=3), m_bits, n_batch=4)
    run_lowbit(synth.shrink(synth.DEBERTA_XXL, 16, seq=40), m_bits)
    run_lowbit(synth.shrink(synth.SWEEP_FWD, 4, seq=64), m_bits)


@pytest.mark.parametrize("m_bits", [2, 4, 8])
def test_low_precision_store_in_host_memory(m_bits):
    """Codes and steps in page-locked host memory: the same kernels on mapped pointers, the same
    results, checkpoint reads and digest included; visited in place, fetched ahead of the call
    (codes and steps both staged and written back; rows by copies and rows by the kernel), and
    the two mixed."""
    run_lowbit(synth.TINY, m_bits, hosted=True)
    run_lowbit(synth.shrink(synth.GPT2_XL, 8, seq=96, epochs=3), m_bits, n_batch=4, hosted=True, stochastic_seed=21)
    run_lowbit(synth.TINY, m_bits, hosted=True, prefetch=lambda k: True)
    run_lowbit(synth.shrink(synth.GPT2_XL, 8, seq=96, epochs=3), m_bits, n_batch=4, hosted=True, stochastic_seed=22,
               prefetch=lambda k: k % 3 != 1)
    ragged = synth.Boundary("low-staged-ragged", 6, 3, 37, 136, "bf16", 5, 8, 3, "outlier", 0.3, seed=612)
    run_lowbit(ragged, m_bits, hosted=True, prefetch=lambda k: True)
    wide = synth.Boundary("low-staged-wide", 256, 128, 1, 64, "fp16", 4, 64, 2, "normal", 0.1, seed=613)
    run_lowbit(wide, m_bits, hosted=True, prefetch=lambda k: True)
    for not_offered in (16, 32):
        with pytest.raises(aq.AqError):
            aq.aq_create_hosted_lowbit(4, 2, 64, 4, 64, not_offered)


@pytest.mark.parametrize("m_bits", [2, 4, 8, 32])
def test_stochastic_messages_over_a_low_precision_store(m_bits):
    """The unbiased rounding applies to the message; the store is re-quantized deterministically
    and the receiver, which has no rounding setting, must end with the same store."""
    run_lowbit(synth.TINY, m_bits, stochastic_seed=0x5EED0 + m_bits)
    run_lowbit(synth.shrink(synth.GPT2_XL, 8, seq=96, epochs=3), m_bits, n_batch=4, stochastic_seed=(1 << 40) + m_bits)
    cfg = synth.Boundary("low-stoch-ragged", 6, 3, 37, 136, "bf16", 5, 8, 3, "outlier", 0.3, seed=611)
    run_lowbit(cfg, m_bits, stochastic_seed=7)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", range(1, 9))
def test_every_message_width_on_ragged_shapes(dtype, bits):
    m_bits = (2, 4, 8, 32)[bits % 4]
    cfg = synth.Boundary("low-ragged", 6, 3, 37, 136, dtype, bits, 8, 3, "outlier", 0.3, seed=120 + bits)
    run_lowbit(cfg, m_bits)
    cfg = synth.Boundary("low-groups", 4, 2, 3, 1024, dtype, bits, 256, 3, "student_t3", 0.2, seed=140 + bits)
    run_lowbit(cfg, m_bits)
    cfg = synth.Boundary("low-one-chunk", 4, 2, 1, 8, dtype, bits, 8, 3, "normal", 0.5, seed=160 + bits)
    run_lowbit(cfg, m_bits)


def test_bad_ids_import_export_and_unsupported_calls():
    cfg = synth.Boundary("low-err", 5, 4, 2, 64, "fp16", 2, 64, 1, "normal", 0.1, seed=5)
    gs, gr = LowSide(cfg, 4, 8), LowSide(cfg, 4, 8)
    os_, or_ = (oracle.SideLow(5, 2, 64, 2, 64, oracle.FP16, 8) for _ in range(2))
    try:
        guards = (Guarded((4, cfg.packed_bytes), torch.uint8), Guarded((4, cfg.groups), torch.float32), Guarded((4, 2, 64), torch.float16))
        packed, scales, out = (g.t for g in guards)
        for step, id_list in enumerate([[1, 7, 1, 3], [3, -1, 1, 3], [0, 1, 2, 3]]):
            ids = torch.tensor(id_list, dtype=torch.int32)
            act = synth.activation(cfg, torch.tensor([10, 11, 12, 13]), step, device="cuda")
            aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
            raw = act if step != 2 else None
            aq.aq_configure(gr.h, aq.AQ_RAW, raw)
            aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
            torch.cuda.synchronize()
            check_guards(*guards)
            p_o, s_o, _ = os_.encode(bits16(act), ids.numpy())
            out_o, _ = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act) if raw is not None else None)
            assert np.array_equal(packed.cpu().numpy(), p_o) and np.array_equal(scales.cpu().numpy(), s_o)
            assert np.array_equal(bits16(out), out_o)
            assert aq.aq_status(gs.h) == os_.status() and aq.aq_status(gr.h) == or_.status()
            assert aq.aq_state_checksum(gs.h) == os_.checksum() and aq.aq_state_checksum(gr.h) == or_.checksum()
        # checkpoint: export every sample of one handle into a fresh one
        fresh = LowSide(cfg, 4, 8)
        buf = np.empty(aq.aq_m_bytes_per_sample(gs.h), np.uint8)
        for i in range(cfg.n_samples):
            seen = aq.aq_export_sample(gs.h, i, buf)
            aq.aq_import_sample(fresh.h, i, buf, seen)
        assert aq.aq_state_checksum(fresh.h) == aq.aq_state_checksum(gs.h)
        fresh.close()
        # what is not built for this store says so
        with pytest.raises(aq.AqError) as e:
            aq.aq_state_checksum_noalloc(gs.h)
        assert e.value.code == aq.AQ_EUNSUPPORTED
        with pytest.raises(aq.AqError):
            aq.aq_create_lowbit(4, 2, 64, 4, 64, 3)
    finally:
        gs.close()
        gr.close()


def test_gpt2_boundary_full_id_space_with_an_8_bit_store():
    """4096 ids (3.8 GB of codes and steps per side), 32 micro-batches of 1 x 1024 x 1600 fp16 per
    launch: the launch shape that the benchmark times with --m-bits 8.  The oracle follows the
    sampled ids only, one small store each."""
    free, _ = torch.cuda.mem_get_info()
    if free < 12 * 2 ** 30:
        pytest.skip("needs 12 GiB of free device memory")
    cfg, per_launch, m_bits = synth.GPT2_XL, 32, 8
    gs, gr = LowSide(cfg, per_launch, m_bits), LowSide(cfg, per_launch, m_bits)
    guards = (Guarded((per_launch, cfg.packed_bytes), torch.uint8), Guarded((per_launch, cfg.groups), torch.float32), Guarded((per_launch, cfg.seq, cfg.hidden), cfg.torch_dtype))
    packed, scales, out = (g.t for g in guards)
    buf = np.empty(aq.aq_m_bytes_per_sample(gs.h), np.uint8)
    tracked = {}
    try:
        order = synth.epoch_order(cfg, 0)
        for epoch in range(3):
            for step in (0, 63, cfg.n_samples // per_launch - 1):
                ids = order[step * per_launch:(step + 1) * per_launch].contiguous()
                act = synth.activation(cfg, ids, epoch, device="cuda")
                aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
                aq.aq_configure(gr.h, aq.AQ_RAW, act if epoch == 0 else None)
                aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
                torch.cuda.synchronize()
                check_guards(*guards)
                for y in (0, per_launch - 1):
                    sid = int(ids[y])
                    if sid not in tracked:
                        tracked[sid] = tuple(oracle.SideLow(1, cfg.seq, cfg.hidden, cfg.bits, cfg.group, DT[cfg.dtype][1], m_bits)
                                             for _ in range(2))
                    o_s, o_r = tracked[sid]
                    zero = np.zeros(1, np.int32)
                    a_np = bits16(act[y:y + 1])
                    p_o, s_o, f_o = o_s.encode(a_np, zero)
                    out_o, _ = o_r.decode(p_o, s_o, zero, raw=a_np if epoch == 0 else None)
                    assert f_o[0] == (epoch == 0)
                    assert np.array_equal(packed[y].cpu().numpy(), p_o[0]), (epoch, step, y, "packed")
                    assert np.array_equal(scales[y].cpu().numpy().view(np.uint32), s_o[0].view(np.uint32)), (epoch, step, y)
                    assert np.array_equal(bits16(out[y]), out_o[0]), (epoch, step, y, "out")
                    for g_side, o_side in ((gs, o_s), (gr, o_r)):
                        assert aq.aq_export_sample(g_side.h, sid, buf) == 1
                        assert np.array_equal(buf[:gs.code_bytes], o_side.m_codes()[0]), (epoch, step, y, "stored codes")
                        assert np.array_equal(buf[gs.code_bytes:].view(np.uint32), o_side.m_scales()[0].view(np.uint32))
        assert aq.aq_status(gs.h) == 0 and aq.aq_status(gr.h) == 0
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h)
    finally:
        gs.close()
        gr.close()
        for pair in tracked.values():
            for side in pair:
                side.close()
