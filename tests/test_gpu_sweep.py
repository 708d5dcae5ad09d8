"""The 'Pipeline sweep' workload on one GPU (reduced sequence length and id space, same
structure): 8 stage boundaries, 16 micro-batches per macro-batch, forward 3-bit deltas and
backward 6-bit direct quantization at every boundary, the wire between sender and receiver
being a device-to-device byte copy.  Boundaries are independent (one (m, Q) pair per boundary),
so they run one after the other with one sender/receiver pair alive at a time.

Also here: the two large boundaries at their full id-space size, in the launch shape the
benchmark times, checked against the oracle on sampled sequences."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from fixtures import synth
from codec_harness import DT, GpuSide, Guarded, bits16, check_guards, guarded_outputs

pytestmark = pytest.mark.gpu


def test_pipeline_sweep_boundary_major():
    seq, n_ids, epochs = 24, 32, 3
    fwd0 = synth.shrink(synth.SWEEP_FWD, n_ids, seq=seq, epochs=epochs)
    bwd = replace(synth.SWEEP_BWD, seq=seq)
    n = fwd0.elems
    bbits = bwd.bits[0]
    assert (fwd0.bits, bbits, fwd0.group) == (3, 6, 64)
    # wire buffers: the sender's and the receiver's ends of the channel
    guards = [Guarded((1, fwd0.packed_bytes), torch.uint8), Guarded((1, fwd0.groups), torch.float32),       # tx_p, tx_s
              Guarded((1, fwd0.packed_bytes), torch.uint8), Guarded((1, fwd0.groups), torch.float32),       # rx_p, rx_s
              Guarded((1, seq, fwd0.hidden), torch.float16), Guarded((1, seq, fwd0.hidden), torch.float16),  # rx_raw, out
              Guarded(n * bbits // 8, torch.uint8), Guarded(n // bwd.group, torch.float32),                  # gtx_p, gtx_s
              Guarded(n * bbits // 8, torch.uint8), Guarded(n // bwd.group, torch.float32),                  # grx_p, grx_s
              Guarded(n, torch.float16)]                                                                     # gout
    tx_p, tx_s, rx_p, rx_s, rx_raw, out, gtx_p, gtx_s, grx_p, grx_s, gout = (g.t for g in guards)
    digests = []
    for boundary in range(synth.SWEEP_BOUNDARIES):
        cfg = replace(fwd0, stream=boundary)
        gs, gr = GpuSide(cfg, 1), GpuSide(cfg, 1)
        os_, or_ = (oracle.Side(n_ids, seq, cfg.hidden, cfg.bits, cfg.group, oracle.FP16) for _ in range(2))
        try:
            aq.aq_configure(gr.h, aq.AQ_RAW, rx_raw)
            call = 0
            for epoch in range(epochs):
                order = synth.epoch_order(cfg, epoch)
                for macro in range(n_ids // synth.SWEEP_MICRO_BATCHES):
                    for mb in range(synth.SWEEP_MICRO_BATCHES):
                        ids = order[macro * synth.SWEEP_MICRO_BATCHES + mb:][:1].contiguous()
                        ids_d = ids.cuda()
                        act = synth.activation(cfg, ids, epoch, device="cuda")
                        # forward: sender -> channel -> receiver
                        aq.aq_encode(gs.h, act, ids_d, tx_p, tx_s)
                        # the channel (same stream as both handles): on a first visit the message is the activation
                        aq.aq_wire_copy(gs.h, 0, rx_p, rx_s, rx_raw if epoch == 0 else None,
                                        tx_p, tx_s, act if epoch == 0 else None)
                        aq.aq_decode(gr.h, rx_p, rx_s, ids_d, out)
                        # backward: receiver -> channel -> sender
                        grad = synth.gradient(bwd, call, device="cuda", stream=boundary)
                        aq.aq_quant_grad(gr.h, grad, n, bbits, gtx_p, gtx_s)
                        aq.aq_wire_copy_grad(gr.h, 0, grx_p, grx_s, gtx_p, gtx_s, n, bbits)
                        aq.aq_dequant_grad(gs.h, grx_p, grx_s, n, bbits, gout)
                        torch.cuda.synchronize()
                        check_guards(*guards, gs.first_guarded, gr.first_guarded)
                        a_np = bits16(act)
                        p_o, s_o, _ = os_.encode(a_np, ids.numpy())
                        out_o, _ = or_.decode(p_o, s_o, ids.numpy(), raw=a_np if epoch == 0 else None)
                        assert np.array_equal(rx_p.cpu().numpy(), p_o), (boundary, epoch, macro, mb)
                        assert np.array_equal(rx_s.cpu().numpy().view(np.uint32), s_o.view(np.uint32))
                        assert np.array_equal(bits16(out), out_o)
                        gp_o, gs_o = oracle.quant_grad(bits16(grad), bbits, bwd.group, oracle.FP16)
                        assert np.array_equal(grx_p.cpu().numpy(), gp_o)
                        assert np.array_equal(grx_s.cpu().numpy().view(np.uint32), gs_o.view(np.uint32))
                        assert np.array_equal(bits16(gout), oracle.dequant_grad(gp_o, gs_o, n, bbits, bwd.group, oracle.FP16))
                        assert tx_p.numel() + tx_s.numel() * 4 == n * 3 // 8 + n // 64 * 4     # forward wire bytes
                        call += 1
                d = aq.aq_state_checksum(gs.h)
                assert d == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
            assert aq.aq_status(gs.h) == 0 and aq.aq_status(gr.h) == 0
            digests.append(d)
        finally:
            gs.close()
            gr.close()
            os_.close()
            or_.close()
    assert len(set(digests)) == synth.SWEEP_BOUNDARIES              # every boundary saw its own data


def test_wire_copies_of_odd_sizes_and_bad_arguments():
    """Messages whose byte counts are not multiples of 16 travel by plain copies instead of the one-launch
    kernel: the bytes that arrive are the same, and nothing lands outside the receiver's buffers."""
    cfg = synth.Boundary("wire-odd", 4, 2, 3, 64, "fp16", 3, 64, 2, "normal", 0.1, seed=55)     # 72 bytes of codes per sample
    gs = GpuSide(cfg, 2)
    try:
        tx = guarded_outputs(cfg, 2)
        rx = guarded_outputs(cfg, 2)
        ids = torch.tensor([1, 3], dtype=torch.int32, device="cuda")
        for epoch in range(2):
            act = synth.activation(cfg, [1, 3], epoch, device="cuda")
            for g in rx:
                g.t.view(torch.uint8).fill_(0xEE)
            aq.aq_encode(gs.h, act, ids, tx[0].t, tx[1].t)
            aq.aq_wire_copy(gs.h, 0, rx[0].t, rx[1].t, rx[2].t if epoch == 0 else None, tx[0].t, tx[1].t, act if epoch == 0 else None)
            torch.cuda.synchronize()
            check_guards(*tx, *rx)
            assert torch.equal(rx[0].t, tx[0].t) and torch.equal(rx[1].t.view(torch.int32), tx[1].t.view(torch.int32))
            assert torch.equal(rx[2].t, act) == (epoch == 0)
        n, bits = 3 * 64, 5                                          # 120 bytes of codes, 12 bytes of steps
        grad = torch.randn(n, device="cuda").half()
        g_tx = (Guarded(n * bits // 8, torch.uint8), Guarded(n // 64, torch.float32))
        g_rx = (Guarded(n * bits // 8, torch.uint8), Guarded(n // 64, torch.float32))
        aq.aq_quant_grad(gs.h, grad, n, bits, g_tx[0].t, g_tx[1].t)
        aq.aq_wire_copy_grad(gs.h, 0, g_rx[0].t, g_rx[1].t, g_tx[0].t, g_tx[1].t, n, bits)
        torch.cuda.synchronize()
        check_guards(*g_tx, *g_rx)
        assert torch.equal(g_rx[0].t, g_tx[0].t) and torch.equal(g_rx[1].t, g_tx[1].t)
        aq.aq_wire_copy_grad(gs.h, 0, None, None, None, None, 0, bits)                # nothing to move
        with pytest.raises(aq.AqError):
            aq.aq_wire_copy_grad(gs.h, 0, g_rx[0].t, g_rx[1].t, g_tx[0].t, g_tx[1].t, n + 1, bits)
        with pytest.raises(aq.AqError):
            aq.aq_wire_copy_grad(gs.h, 99, g_rx[0].t, g_rx[1].t, g_tx[0].t, g_tx[1].t, n, bits)
        with pytest.raises(aq.AqError):
            aq.aq_wire_copy(gs.h, 0, rx[0].t, rx[1].t, rx[2].t, tx[0].t, tx[1].t, None)
    finally:
        gs.close()


def _full_size_sampled(cfg, per_launch, steps, samples_per_launch, wire=False):
    """Full id space, the benchmark's launch shape; the oracle follows only the sampled ids.
    wire: the message crosses aq_wire_copy into the receiver's own buffers (the raw block too, on
    first visits), as between the two stages of the pipeline sweep."""
    od = DT[cfg.dtype][1]
    gs, gr = GpuSide(cfg, per_launch), GpuSide(cfg, per_launch)
    guards = guarded_outputs(cfg, per_launch)
    packed, scales, out = (g.t for g in guards)
    if wire:
        rx = guarded_outputs(cfg, per_launch)                          # the receiver's codes, steps and raw block
        guards = guards + rx
    tracked = {}                                                     # sample id -> (oracle sender, oracle receiver)
    try:
        order = synth.epoch_order(cfg, 0)
        for epoch in range(3):                                        # the same launches each epoch: first visit, then deltas
            for step in steps:
                ids = order[step * per_launch:(step + 1) * per_launch].contiguous()
                act = synth.activation(cfg, ids, epoch, device="cuda")
                aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
                if wire:
                    first = epoch == 0
                    aq.aq_wire_copy(gs.h, torch.cuda.current_device(), rx[0].t, rx[1].t, rx[2].t if first else None,
                                    packed, scales, act if first else None)
                    aq.aq_configure(gr.h, aq.AQ_RAW, rx[2].t if first else None)
                    aq.aq_decode(gr.h, rx[0].t, rx[1].t, ids.cuda(), out)
                else:
                    aq.aq_configure(gr.h, aq.AQ_RAW, act if epoch == 0 else None)
                    aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
                torch.cuda.synchronize()
                check_guards(*guards, gs.first_guarded, gr.first_guarded)
                assert gs.first.cpu().numpy().all() == (epoch == 0)
                if wire:
                    assert torch.equal(rx[0].t, packed) and torch.equal(rx[1].t.view(torch.int32), scales.view(torch.int32))
                for y in np.linspace(0, per_launch - 1, samples_per_launch).astype(int):
                    sid = int(ids[y])
                    if sid not in tracked:
                        tracked[sid] = tuple(oracle.Side(1, cfg.seq, cfg.hidden, cfg.bits, cfg.group, od) for _ in range(2))
                    o_s, o_r = tracked[sid]
                    zero = np.zeros(1, np.int32)
                    a_np = bits16(act[y:y + 1])
                    p_o, s_o, f_o = o_s.encode(a_np, zero)
                    out_o, _ = o_r.decode(p_o, s_o, zero, raw=a_np if epoch == 0 else None)
                    assert f_o[0] == (epoch == 0)
                    assert np.array_equal(packed[y].cpu().numpy(), p_o[0]), (epoch, step, y, "packed")
                    assert np.array_equal(scales[y].cpu().numpy().view(np.uint32), s_o[0].view(np.uint32)), (epoch, step, y)
                    assert np.array_equal(bits16(out[y]), out_o[0]), (epoch, step, y, "out")
                    assert np.array_equal(gs.m_row(sid)[0], o_s.m()[0]) and np.array_equal(gr.m_row(sid)[0], o_r.m()[0])
        assert aq.aq_status(gs.h) == 0 and aq.aq_status(gr.h) == 0
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h)
        assert aq.aq_state_checksum_noalloc(gs.h) == aq.aq_state_checksum(gs.h)
    finally:
        gs.close()
        gr.close()
        for pair in tracked.values():
            for side in pair:
                side.close()


def _needs_gb(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 2 ** 30:
        pytest.skip(f"needs {gb} GiB of free device memory")


def test_gpt2_boundary_full_id_space_in_the_benchmark_launch_shape():
    """4096 ids (13.4 GB of m per side), 32 micro-batches of 1 x 1024 x 1600 fp16 per launch."""
    _needs_gb(34)
    cfg = synth.GPT2_XL
    _full_size_sampled(cfg, 32, steps=[0, 1, cfg.n_samples // 32 - 1], samples_per_launch=2)


def test_sweep_boundary_full_id_space_in_the_benchmark_launch_shape():
    """One boundary of the pipeline sweep at full size: 8192 ids (26.8 GB of m per side), a macro-batch of
    16 micro-batches of 1 x 1024 x 1600 fp16 per launch, 3-bit deltas over the wire copy, three epochs;
    then the backward direction of one whole macro-batch (26,214,400 gradient elements) in 6 bits."""
    _needs_gb(60)
    cfg, per_launch = synth.SWEEP_FWD, synth.SWEEP_MICRO_BATCHES
    assert (cfg.n_samples, cfg.bits, cfg.group, cfg.elems) == (8192, 3, 64, 1024 * 1600)
    _full_size_sampled(cfg, per_launch, steps=[0, 3, cfg.n_samples // per_launch - 1], samples_per_launch=2, wire=True)
    bwd = replace(synth.SWEEP_BWD, n_batch=per_launch)
    bits, n = bwd.bits[0], bwd.elems
    assert (bits, n) == (6, 26214400)
    h = aq.aq_create(1, 1, bwd.group, cfg.bits, bwd.group)
    try:
        grad = synth.gradient(bwd, 1, device="cuda")
        guards = (Guarded(n * bits // 8, torch.uint8), Guarded(n // bwd.group, torch.float32),     # sender's end of the wire
                  Guarded(n * bits // 8, torch.uint8), Guarded(n // bwd.group, torch.float32),     # receiver's end
                  Guarded(n, torch.float16))
        tx_p, tx_s, rx_p, rx_s, gout = (g.t for g in guards)
        aq.aq_quant_grad(h, grad, n, bits, tx_p, tx_s)
        aq.aq_wire_copy_grad(h, torch.cuda.current_device(), rx_p, rx_s, tx_p, tx_s, n, bits)
        aq.aq_dequant_grad(h, rx_p, rx_s, n, bits, gout)
        torch.cuda.synchronize()
        check_guards(*guards)
        p_o, s_o = oracle.quant_grad(bits16(grad), bits, bwd.group, oracle.FP16)
        assert np.array_equal(rx_p.cpu().numpy(), p_o)
        assert np.array_equal(rx_s.cpu().numpy().view(np.uint32), s_o.view(np.uint32))
        assert np.array_equal(bits16(gout), oracle.dequant_grad(p_o, s_o, n, bits, bwd.group, oracle.FP16))
    finally:
        aq.aq_destroy(h)


@pytest.mark.parametrize("per_launch", [8, 64])
def test_deberta_boundary_full_id_space(per_launch):
    """32768 ids (25.8 GB of m per side), 256 x 1536 bf16, 2 bit, group 128: calls of its micro-batch of 8
    sequences, and of the 64 sequences (a macro-batch) that the benchmark hands to one launch."""
    _needs_gb(60)
    cfg = synth.DEBERTA_XXL
    _full_size_sampled(cfg, per_launch, steps=[0, 7, cfg.n_samples // per_launch - 1], samples_per_launch=3)


def test_gpt2_boundary_full_id_space_with_stochastic_rounding():
    """The benchmark's launch shape with the unbiased quantizer: the random stream of a sample is
    keyed by its id, so the oracle keeps the four lowest ids under their own numbers and the
    launches that hold them are run at full width."""
    _needs_gb(34)
    cfg, per_launch, seed, n_track = synth.GPT2_XL, 32, 0xA05D, 4
    gs, gr = GpuSide(cfg, per_launch), GpuSide(cfg, per_launch)
    od = DT[cfg.dtype][1]
    o_s, o_r = (oracle.Side(n_track, cfg.seq, cfg.hidden, cfg.bits, cfg.group, od) for _ in range(2))
    guards = guarded_outputs(cfg, per_launch)
    packed, scales, out = (g.t for g in guards)
    try:
        aq.aq_configure(gs.h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
        aq.aq_configure(gs.h, aq.AQ_SEED, seed)
        order = synth.epoch_order(cfg, 0)
        where = {int(sid): int(pos) for pos, sid in enumerate(order.tolist()) if sid < n_track}
        steps = sorted({pos // per_launch for pos in where.values()})
        checked, differs, before = 0, False, {}
        for epoch in range(3):
            aq.aq_configure(gs.h, aq.AQ_EPOCH, epoch)
            o_s.set_rounding(True, seed, epoch)
            for step in steps:
                ids = order[step * per_launch:(step + 1) * per_launch].contiguous()
                act = synth.activation(cfg, ids, epoch, device="cuda")
                aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
                aq.aq_configure(gr.h, aq.AQ_RAW, act if epoch == 0 else None)
                aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
                torch.cuda.synchronize()
                check_guards(*guards, gs.first_guarded, gr.first_guarded)
                for sid, pos in where.items():
                    if pos // per_launch != step:
                        continue
                    y = pos % per_launch
                    one = np.array([sid], np.int32)
                    a_np = bits16(act[y:y + 1])
                    p_o, s_o, f_o = o_s.encode(a_np, one)
                    out_o, _ = o_r.decode(p_o, s_o, one, raw=a_np if epoch == 0 else None)
                    assert f_o[0] == (epoch == 0)
                    assert np.array_equal(packed[y].cpu().numpy(), p_o[0]), (epoch, step, y, "packed")
                    assert np.array_equal(scales[y].cpu().numpy().view(np.uint32), s_o[0].view(np.uint32)), (epoch, step, y)
                    assert np.array_equal(bits16(out[y]), out_o[0]), (epoch, step, y, "out")
                    assert np.array_equal(gs.m_row(sid)[0], o_s.m()[sid]) and np.array_equal(gr.m_row(sid)[0], o_r.m()[sid])
                    checked += 1
                    if epoch:                                  # the mode is on: some codes differ from the interval number's
                        d = (act[y].float() - torch.from_numpy(before[sid].view(np.float16).astype(np.float32)).cuda()).cpu().numpy()
                        k_det = oracle.quantize_group(d.reshape(-1)[:cfg.group], cfg.bits)[0]
                        differs |= not np.array_equal(oracle.get_codes(p_o[0], cfg.elems, cfg.bits)[:cfg.group], k_det)
                    before[sid] = o_s.m()[sid].copy()
        assert checked == 3 * n_track and differs
        assert aq.aq_status(gs.h) == 0 and aq.aq_status(gr.h) == 0
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h)
    finally:
        gs.close(), gr.close(), o_s.close(), o_r.close()
