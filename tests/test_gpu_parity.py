"""CUDA library against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from fixtures import synth
from codec_harness import DT, GpuSide, Guarded, bits16, check_guards, run_boundary

pytestmark = pytest.mark.gpu


# ----------------------------------------------------------------- backward direction (stateless)

def _grad_input(n, group, dtype, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    x = torch.randn(n, generator=g) * 1e-3
    spikes = torch.rand(n, generator=g) < 0.01
    x = torch.where(spikes, x * 100, x)
    xg = x.view(-1, group)
    if xg.shape[0] >= 8:
        xg[1] = 0.0                                   # an all-zero group
        xg[2] = 1e-41                                  # a vanishing group: step below FLT_MIN
        xg[3, 0] = -0.0
        xg[4] = 2.0 ** -120                            # tiny but live
        xg[5] = torch.arange(group) - group / 2        # exact interval edges
    return x.to(dtype)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("group,n_groups", [(8, 1), (8, 333), (16, 1), (16, 333), (32, 77), (64, 4097), (128, 777), (256, 130)])
def test_quant_and_dequant_grad_match_oracle(dtype, bits, group, n_groups):
    td = torch.float16 if dtype == "fp16" else torch.bfloat16
    n = group * n_groups                               # ragged: not a multiple of the CTA tile
    h = aq.aq_create(1, 1, group, 4, group)
    try:
        aq.aq_configure(h, aq.AQ_DTYPE, DT[dtype][0])
        grad = _grad_input(n, group, td, bits * 1000 + group).cuda()
        packed = torch.full((n * bits // 8 + 16,), 0xCD, dtype=torch.uint8, device="cuda")
        scales = torch.full((n // group + 4,), -3.0, dtype=torch.float32, device="cuda")
        out = torch.full((n + 8,), 5.0, dtype=td, device="cuda")
        aq.aq_quant_grad(h, grad, n, bits, packed, scales)
        aq.aq_dequant_grad(h, packed, scales, n, bits, out)
        torch.cuda.synchronize()
        p_o, s_o = oracle.quant_grad(bits16(grad), bits, group, DT[dtype][1])
        o_o = oracle.dequant_grad(p_o, s_o, n, bits, group, DT[dtype][1])
        assert np.array_equal(packed.cpu().numpy()[: n * bits // 8], p_o)
        assert np.array_equal(scales.cpu().numpy()[: n // group].view(np.uint32), s_o.view(np.uint32))
        assert np.array_equal(bits16(out)[:n], o_o)
        # nothing written past the ends
        assert (packed.cpu().numpy()[n * bits // 8:] == 0xCD).all()
        assert (scales.cpu().numpy()[n // group:] == -3.0).all()
        assert (out.float().cpu().numpy()[n:] == 5.0).all()
    finally:
        aq.aq_destroy(h)


def test_backward_workload_full_size():
    """Config 'Backward path': 4 x 1024 x 1600 fp16 gradients, 8-bit and 4-bit, group 64."""
    cfg = synth.BACKWARD
    h = aq.aq_create(1, 1, cfg.group, 4, cfg.group)
    try:
        grad = synth.gradient(cfg, 0, device="cuda")
        n = cfg.elems
        g_np = bits16(grad)
        for bits in cfg.bits:
            guards = (Guarded(n * bits // 8, torch.uint8), Guarded(n // cfg.group, torch.float32), Guarded(n, torch.float16))
            packed, scales, out = (g.t for g in guards)
            aq.aq_quant_grad(h, grad, n, bits, packed, scales)
            aq.aq_dequant_grad(h, packed, scales, n, bits, out)
            torch.cuda.synchronize()
            check_guards(*guards)
            p_o, s_o = oracle.quant_grad(g_np, bits, cfg.group, oracle.FP16)
            o_o = oracle.dequant_grad(p_o, s_o, n, bits, cfg.group, oracle.FP16)
            assert np.array_equal(packed.cpu().numpy(), p_o)
            assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32))
            assert np.array_equal(bits16(out), o_o)
    finally:
        aq.aq_destroy(h)


def test_gradient_inputs_are_identical_on_cpu_and_gpu():
    cfg = synth.GradWorkload("g", 1, 16, 1600, "fp16", (4,), 64, seed=9)
    assert np.array_equal(bits16(synth.gradient(cfg, 3, "cuda")), bits16(synth.gradient(cfg, 3, "cpu")))
    b = synth.shrink(synth.DEBERTA_XXL, 8, seq=8)
    assert np.array_equal(bits16(synth.activation(b, [5, 2], 2, "cuda")), bits16(synth.activation(b, [5, 2], 2, "cpu")))


# ----------------------------------------------------------------- forward boundary (stateful)

def test_tiny_boundary_all_epochs():
    """Config 'Tiny boundary', complete: 64 ids, 4 x 128 x 768 fp16, 2 bit, group 128, 3 epochs."""
    run_boundary(synth.TINY)


def test_gpt2_shaped_boundary_reduced_id_space():
    """Config 'GPT2-1.5B-shaped boundary' with 8 ids instead of 4096 (same per-call shape)."""
    run_boundary(synth.shrink(synth.GPT2_XL, 8, epochs=3))


def test_gpt2_shaped_boundary_batched_launch():
    run_boundary(synth.shrink(synth.GPT2_XL, 8, seq=192, epochs=3), n_batch=4)


def test_deberta_shaped_boundary_reduced_id_space():
    """Config 'DeBERTa-1.5B-shaped boundary' with 16 ids: bf16, 2 bit, group 128, micro-batch 8."""
    run_boundary(synth.shrink(synth.DEBERTA_XXL, 16))


def test_sweep_forward_three_bit_reduced_id_space():
    """Forward half of the 'Pipeline sweep' config: 3-bit delta, group 64 (fields straddle bytes)."""
    run_boundary(synth.shrink(synth.SWEEP_FWD, 4, seq=256))


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", range(1, 9))
def test_every_bit_width_on_ragged_shapes(dtype, bits):
    # 37 x 136 elements: 629 chunks per sample -- not a multiple of a warp or of a CTA tile
    cfg = synth.Boundary("ragged", 6, 3, 37, 136, dtype, bits, 8, 3, "outlier", 0.3, seed=20 + bits)
    run_boundary(cfg)
    # one chunk per sample; the stream of a sample is `bits` bytes long
    cfg = synth.Boundary("one-chunk", 4, 2, 1, 8, dtype, bits, 8, 3, "normal", 0.5, seed=40 + bits)
    run_boundary(cfg)


@pytest.mark.parametrize("dtype,bits", [("fp16", 3), ("bf16", 4)])
def test_call_large_enough_for_the_tapered_end_of_the_decode_grid(dtype, bits):
    """128 samples of 57 rows (the last one ragged) in one call: more than two waves of four-row CTAs on
    148 multiprocessors, so the receiver's grid walks its last samples with two-row CTAs; 57 is odd, so
    either part of the grid ends each sample with a one-row CTA.  Every element is compared."""
    cfg = synth.Boundary("taper", 128, 128, 57, 2040, dtype, bits, 8, 3, "outlier", 0.2, seed=70 + bits)
    assert cfg.elems // 8 == 57 * 255 and (cfg.elems // 8) % 256 != 0
    run_boundary(cfg)


@pytest.mark.parametrize("group", [16, 32, 256])
def test_other_group_sizes(group):
    cfg = synth.Boundary("groups", 4, 2, 5, 1024, "fp16", 4, group, 3, "outlier", 0.1, seed=group)
    run_boundary(cfg)
    cfg = synth.Boundary("groups3", 4, 2, 5, 1024, "bf16", 3, group, 3, "student_t3", 0.1, seed=group)
    run_boundary(cfg)


def test_revisits_of_an_unchanged_activation_send_zeros():
    cfg = synth.Boundary("still", 4, 2, 4, 256, "fp16", 4, 64, 3, "normal", 0.0, seed=77)

    def act_fn(ids, epoch):
        return synth.activation(cfg, ids, 0, device="cuda")

    run_boundary(cfg, act_fn=act_fn)
    side = GpuSide(cfg, 2)
    try:
        ids = torch.tensor([1, 3], dtype=torch.int32, device="cuda")
        act = act_fn(ids.cpu(), 0)
        guards = (Guarded((2, cfg.packed_bytes), torch.uint8), Guarded((2, cfg.groups), torch.float32))
        packed, scales = (g.t for g in guards)
        packed.fill_(9), scales.fill_(9.0)
        aq.aq_encode(side.h, act, ids, packed, scales)
        aq.aq_encode(side.h, act, ids, packed, scales)
        torch.cuda.synchronize()
        check_guards(*guards)
        assert not packed.any() and not scales.any()
        assert np.array_equal(side.m_row(3)[0], bits16(act[1]))
    finally:
        side.close()


# ----------------------------------------------------------------- error paths and empty inputs

def test_bad_duplicate_and_rawless_ids_are_skipped_like_the_oracle():
    cfg = synth.Boundary("err", 5, 4, 2, 64, "fp16", 2, 64, 1, "normal", 0.1, seed=5)
    gs, gr = GpuSide(cfg, 4), GpuSide(cfg, 4)
    os_, or_ = (oracle.Side(5, 2, 64, 2, 64, oracle.FP16) for _ in range(2))
    try:
        guards = (Guarded((4, cfg.packed_bytes), torch.uint8), Guarded((4, cfg.groups), torch.float32), Guarded((4, 2, 64), torch.float16))
        packed, scales, out = (g.t for g in guards)
        for step, id_list in enumerate([[1, 7, 1, 3], [3, -1, 1, 3], [0, 1, 2, 3]]):
            ids = torch.tensor(id_list, dtype=torch.int32)
            act = synth.activation(cfg, torch.tensor([10, 11, 12, 13]), step, device="cuda")
            packed.fill_(1)
            scales.fill_(1)
            out.fill_(1)
            aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
            raw = act if step != 2 else None                      # last step: first visits without a raw message
            aq.aq_configure(gr.h, aq.AQ_RAW, raw)
            aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
            torch.cuda.synchronize()
            check_guards(*guards)
            p_o, s_o, f_o = os_.encode(bits16(act), ids.numpy())
            out_o, fr_o = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act) if raw is not None else None)
            assert np.array_equal(packed.cpu().numpy(), p_o)
            assert np.array_equal(scales.cpu().numpy(), s_o)
            assert np.array_equal(bits16(out), out_o)
            assert np.array_equal(gs.first.cpu().numpy(), f_o) and np.array_equal(gr.first.cpu().numpy(), fr_o)
            st_s, st_r = aq.aq_status(gs.h), aq.aq_status(gr.h)
            assert st_s == os_.status() and st_r == or_.status()
            assert aq.aq_status(gs.h) == 0                          # reading clears
            assert np.array_equal(gs.m_all(), os_.m()) and np.array_equal(gr.m_all(), or_.m())
            assert aq.aq_state_checksum(gs.h) == os_.checksum()
            assert aq.aq_state_checksum(gr.h) == or_.checksum()
        assert st_r & aq.AQ_ST_NO_RAW
    finally:
        gs.close()
        gr.close()


def test_host_side_argument_errors():
    with pytest.raises(aq.AqError):
        aq.aq_create(4, 2, 100, 4, 64)          # group does not divide hidden
    with pytest.raises(aq.AqError) as e:
        aq.aq_create_lowbit(4, 2, 96, 4, 24, 8)  # a valid group that the low-precision store has no kernel for
    assert e.value.code == aq.AQ_EUNSUPPORTED and "24" in str(e.value)
    with pytest.raises(aq.AqError) as e:
        aq.aq_create(4, 2, 96, 4, 12)           # not a whole number of 16-byte pieces
    assert e.value.code == aq.AQ_EINVAL
    with pytest.raises(aq.AqError):
        aq.aq_create(0, 2, 64, 4, 64)
    h = aq.aq_create(4, 2, 64, 4, 64)
    try:
        t = torch.zeros(256, dtype=torch.float16, device="cuda")
        ids = torch.zeros(1, dtype=torch.int32, device="cuda")
        with pytest.raises(aq.AqError) as e:
            aq.aq_encode(h, None, ids, t, t)
        assert e.value.code == aq.AQ_EINVAL
        with pytest.raises(aq.AqError):
            aq.aq_encode(h, t.data_ptr() + 2, ids, t, t)          # misaligned
        with pytest.raises(aq.AqError):
            aq.aq_quant_grad(h, t, 100, 4, t, t)                  # not a multiple of the group
        with pytest.raises(aq.AqError):
            aq.aq_quant_grad(h, t, 128, 0, t, t)
        with pytest.raises(aq.AqError):
            aq.aq_configure(h, aq.AQ_BATCH, 70000)
        with pytest.raises(aq.AqError):
            aq.aq_configure(h, 99, 0)
        # empty inputs are no-ops
        aq.aq_quant_grad(h, None, 0, 4, None, None)
        aq.aq_dequant_grad(h, None, None, 0, 4, None)
        aq.aq_configure(h, aq.AQ_BATCH, 0)
        aq.aq_encode(h, None, None, None, None)
        aq.aq_decode(h, None, None, None, None)
        assert aq.aq_status(h) == 0
        assert aq.aq_packed_bytes_per_sample(h) == 64 and aq.aq_scales_per_sample(h) == 2
    finally:
        aq.aq_destroy(h)


def test_non_default_stream_and_host_buffer_forms():
    cfg = synth.Boundary("host", 6, 3, 9, 192, "bf16", 3, 64, 3, "normal", 0.05, seed=31)
    stream = torch.cuda.Stream()
    gs, gr = GpuSide(cfg, 3, stream), GpuSide(cfg, 3, stream)
    os_, or_ = (oracle.Side(6, 9, 192, 3, 64, oracle.BF16) for _ in range(2))
    try:
        for epoch in range(3):
            order = synth.epoch_order(cfg, epoch)
            for c in range(2):
                ids = order[c * 3:(c + 1) * 3].contiguous()
                act = synth.activation(cfg, ids, epoch).pin_memory()
                packed = torch.empty((3, cfg.packed_bytes), dtype=torch.uint8).pin_memory()
                scales = torch.empty((3, cfg.groups), dtype=torch.float32).pin_memory()
                out = torch.empty_like(act).pin_memory()
                aq.aq_encode_host(gs.h, act, ids, packed, scales)
                aq.aq_decode_host(gr.h, packed, scales, act if epoch == 0 else None, ids, out)
                p_o, s_o, _ = os_.encode(bits16(act), ids.numpy())
                out_o, _ = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
                assert np.array_equal(packed.numpy(), p_o) and np.array_equal(scales.numpy(), s_o)
                assert np.array_equal(bits16(out), out_o)
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum()
        assert np.array_equal(gr.m_all(), or_.m())
    finally:
        gs.close()
        gr.close()


@pytest.mark.parametrize("n_batch", [8, 11, 32])
def test_host_buffer_forms_in_slices(n_batch):
    """From 8 samples per call on, the host-buffer calls move the batch in four pieces whose copies
    and kernels overlap (ragged pieces at 11); a call with a repeated or a bad id is not cut up,
    so that the repeat is still found.  Every output, the first-visit flags and the state must be
    those of the oracle either way."""
    cfg = synth.Boundary("host-sliced", 64, n_batch, 5, 192, "fp16", 3, 64, 3, "normal", 0.05, seed=33)
    gs, gr = GpuSide(cfg, n_batch), GpuSide(cfg, n_batch)
    os_, or_ = (oracle.Side(64, 5, 192, 3, 64, oracle.FP16) for _ in range(2))
    aq.aq_configure(gs.h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
    aq.aq_configure(gs.h, aq.AQ_SEED, 99)
    try:
        packed = torch.empty((n_batch, cfg.packed_bytes), dtype=torch.uint8).pin_memory()
        scales = torch.empty((n_batch, cfg.groups), dtype=torch.float32).pin_memory()
        out = torch.empty((n_batch, 5, 192), dtype=torch.float16).pin_memory()
        for call in range(6):
            aq.aq_configure(gs.h, aq.AQ_EPOCH, call)
            os_.set_rounding(True, 99, call)
            ids = synth.epoch_order(cfg, call)[:n_batch].clone()          # overlapping draws: first and later visits mixed
            if call == 3:
                ids[n_batch - 1] = ids[1]                                 # a repeat across two pieces
            if call == 4:
                ids[2] = 64                                               # out of range
            act = synth.activation(cfg, torch.arange(n_batch), call).pin_memory()
            packed.fill_(0xCD), scales.fill_(-1.0), out.fill_(7.0)
            aq.aq_encode_host(gs.h, act, ids, packed, scales)
            aq.aq_decode_host(gr.h, packed, scales, act, ids, out)
            p_o, s_o, f_o = os_.encode(bits16(act), ids.numpy())
            out_o, fr_o = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
            assert np.array_equal(packed.numpy(), p_o) and np.array_equal(scales.numpy(), s_o), call
            assert np.array_equal(bits16(out), out_o), call
            assert np.array_equal(gs.first.cpu().numpy()[:n_batch], f_o), call
            assert np.array_equal(gr.first.cpu().numpy()[:n_batch], fr_o), call
            assert aq.aq_status(gs.h) == os_.status() and aq.aq_status(gr.h) == or_.status()
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
        assert np.array_equal(gs.m_all(), os_.m()) and np.array_equal(gr.m_all(), or_.m())
    finally:
        gs.close(), gr.close(), os_.close(), or_.close()


def test_l2_prefetch_switch():
    """AQ_L2_PREFETCH only says whether a CTA asks for its rows ahead of its loads: results are
    the same with the key at 0, at 1 (the default), and for a hosted store with staged calls."""
    cfg = synth.shrink(synth.GPT2_XL, 8, seq=160, epochs=3)
    run_boundary(cfg, n_batch=4, l2_prefetch=0)
    run_boundary(cfg, n_batch=4, l2_prefetch=1)
    ragged = synth.Boundary("pf-ragged", 6, 3, 37, 136, "bf16", 3, 8, 3, "outlier", 0.3, seed=43)
    run_boundary(ragged, l2_prefetch=0)
    run_boundary(ragged, hosted=True, prefetch=lambda k: True, l2_prefetch=1)
    run_boundary(ragged, hosted=True, prefetch=lambda k: k % 2 == 0, l2_prefetch=0)
    h = aq.aq_create(4, 2, 64, 4, 64)
    try:
        with pytest.raises(aq.AqError):
            aq.aq_configure(h, aq.AQ_L2_PREFETCH, 2)
    finally:
        aq.aq_destroy(h)


def test_two_boundaries_run_side_by_side_on_two_streams():
    """A stage has a boundary on either side: two pairs of handles, each pair on a stream of its
    own, fed without any synchronisation in between.  Handles share no state, so each pair must
    give exactly what it gives alone."""
    cfgs = [synth.Boundary("left", 12, 4, 24, 256, "fp16", 4, 64, 3, "normal", 0.05, seed=41),
            synth.Boundary("right", 10, 5, 17, 384, "bf16", 2, 128, 3, "student_t3", 0.02, seed=42, stream=1)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    sides = [(GpuSide(c, c.n_batch, st), GpuSide(c, c.n_batch, st)) for c, st in zip(cfgs, streams)]
    oracles = [tuple(oracle.Side(c.n_samples, c.seq, c.hidden, c.bits, c.group, DT[c.dtype][1]) for _ in range(2)) for c in cfgs]
    kept = [[], []]
    try:
        n_calls = [c.epochs * (c.n_samples // c.n_batch) for c in cfgs]
        for call in range(max(n_calls)):
            for b, c in enumerate(cfgs):
                if call >= n_calls[b]:
                    continue
                per_epoch = c.n_samples // c.n_batch
                epoch, k = divmod(call, per_epoch)
                ids = synth.epoch_order(c, epoch)[k * c.n_batch:(k + 1) * c.n_batch].contiguous()
                act = synth.activation(c, ids, epoch, device="cuda")
                ids_d = ids.cuda()
                guards = (Guarded((c.n_batch, c.packed_bytes), torch.uint8), Guarded((c.n_batch, c.groups), torch.float32),
                          Guarded(tuple(act.shape), act.dtype))
                packed, scales, out = (g.t for g in guards)
                torch.cuda.current_stream().synchronize()                 # the inputs are ready; the codec calls are not waited for
                gs, gr = sides[b]
                aq.aq_encode(gs.h, act, ids_d, packed, scales)
                aq.aq_configure(gr.h, aq.AQ_RAW, act)
                aq.aq_decode(gr.h, packed, scales, ids_d, out)
                kept[b].append((ids, act, ids_d, packed, scales, out, guards))
        torch.cuda.synchronize()
        for b, c in enumerate(cfgs):
            o_s, o_r = oracles[b]
            for ids, act, _, packed, scales, out, guards in kept[b]:
                check_guards(*guards)
                p_o, s_o, _ = o_s.encode(bits16(act), ids.numpy())
                out_o, _ = o_r.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
                assert np.array_equal(packed.cpu().numpy(), p_o) and np.array_equal(scales.cpu().numpy(), s_o), c.name
                assert np.array_equal(bits16(out), out_o), c.name
            gs, gr = sides[b]
            assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == o_s.checksum() == o_r.checksum()
            assert np.array_equal(gs.m_all(), o_s.m()) and np.array_equal(gr.m_all(), o_r.m())
    finally:
        for pair in sides:
            for g in pair:
                g.close()
        for pair in oracles:
            for o in pair:
                o.close()


def test_import_export_round_trip():
    cfg = synth.Boundary("ckpt", 3, 1, 4, 64, "fp16", 4, 64, 1, "normal", 0.1, seed=8)
    a, b = GpuSide(cfg, 1), GpuSide(cfg, 1)
    try:
        ids = torch.tensor([2], dtype=torch.int32, device="cuda")
        act = synth.activation(cfg, [2], 0, device="cuda")
        p = torch.empty((1, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
        s = torch.empty((1, cfg.groups), dtype=torch.float32, device="cuda")
        aq.aq_encode(a.h, act, ids, p, s)
        for i in range(3):
            row, seen = a.m_row(i)
            aq.aq_import_sample(b.h, i, row, seen)
        assert aq.aq_state_checksum(a.h) == aq.aq_state_checksum(b.h)
        assert b.m_row(2)[1] == 1 and b.m_row(0)[1] == 0
    finally:
        a.close()
        b.close()


def test_replayed_cuda_graph_counts_every_replay_as_a_call():
    """One captured encode + decode, replayed: the first replay is a first visit, the later ones
    are delta visits of the same activation (and a second graph, other ids, interleaves)."""
    cfg = synth.Boundary("graph", 6, 2, 5, 320, "fp16", 3, 64, 1, "outlier", 0.2, seed=61)
    stream = torch.cuda.Stream()
    gs, gr = GpuSide(cfg, 2, stream), GpuSide(cfg, 2, stream)
    os_, or_ = (oracle.Side(6, 5, 320, 3, 64, oracle.FP16) for _ in range(2))
    try:
        graphs = []
        for ids_list, epoch in (([4, 1], 0), ([2, 4], 1)):
            ids = torch.tensor(ids_list, dtype=torch.int32)
            act = synth.activation(cfg, ids, epoch, device="cuda")
            ids_d = ids.cuda()
            guards = (Guarded((2, cfg.packed_bytes), torch.uint8), Guarded((2, cfg.groups), torch.float32), Guarded((2, cfg.seq, cfg.hidden), torch.float16))
            packed, scales, out = (g.t for g in guards)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                aq.aq_configure(gr.h, aq.AQ_RAW, act)
                aq.aq_encode(gs.h, act, ids_d, packed, scales)
                aq.aq_decode(gr.h, packed, scales, ids_d, out)
            graphs.append((g, ids, act, packed, scales, out, ids_d, guards))     # the graph reads ids_d: keep it alive
        for which in (0, 0, 1, 0, 1, 1):
            g, ids, act, packed, scales, out, _, guards = graphs[which]
            aq.aq_configure(gr.h, aq.AQ_RAW, act)            # host-side setting only; the graph holds its own pointer
            g.replay()
            torch.cuda.synchronize()
            check_guards(*guards, gs.first_guarded, gr.first_guarded)
            p_o, s_o, f_o = os_.encode(bits16(act), ids.numpy())
            out_o, fr_o = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
            assert np.array_equal(packed.cpu().numpy(), p_o)
            assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32))
            assert np.array_equal(bits16(out), out_o)
            assert np.array_equal(gs.first.cpu().numpy(), f_o) and np.array_equal(gr.first.cpu().numpy(), fr_o)
        assert aq.aq_state_checksum(gs.h) == aq.aq_state_checksum(gr.h) == os_.checksum() == or_.checksum()
        assert np.array_equal(gs.m_all(), os_.m())
    finally:
        gs.close()
        gr.close()


# ----------------------------------------------------------------- unbiased stochastic rounding (Philox4x32-10)

def test_stochastic_rounding_tiny_boundary():
    run_boundary(synth.TINY, stochastic_seed=0x1234567890ABCDEF)


def test_stochastic_rounding_large_shapes_reduced_id_space():
    run_boundary(synth.shrink(synth.GPT2_XL, 8, seq=160, epochs=3), n_batch=4, stochastic_seed=7)
    run_boundary(synth.shrink(synth.DEBERTA_XXL, 16, seq=64), stochastic_seed=8)
    run_boundary(synth.shrink(synth.SWEEP_FWD, 4, seq=96), stochastic_seed=9)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", range(1, 9))
def test_stochastic_rounding_every_bit_width_on_ragged_shapes(dtype, bits):
    cfg = synth.Boundary("sr-ragged", 6, 3, 37, 136, dtype, bits, 8, 3, "outlier", 0.3, seed=70 + bits)
    run_boundary(cfg, stochastic_seed=1000 + bits)
    cfg = synth.Boundary("sr-groups", 4, 2, 3, 1024, dtype, bits, 256, 3, "student_t3", 0.2, seed=90 + bits)
    run_boundary(cfg, stochastic_seed=2000 + bits)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", [1, 3, 4, 6, 8])
def test_stochastic_gradient_quantization_matches_oracle(dtype, bits):
    td = torch.float16 if dtype == "fp16" else torch.bfloat16
    group, n_groups = 64, 4097
    n = group * n_groups
    h = aq.aq_create(1, 1, group, 4, group)
    try:
        aq.aq_configure(h, aq.AQ_DTYPE, DT[dtype][0])
        aq.aq_configure(h, aq.AQ_ROUNDING, aq.AQ_ROUND_STOCHASTIC)
        aq.aq_configure(h, aq.AQ_SEED, 424242)
        grad = _grad_input(n, group, td, 5000 + bits).cuda()
        guards = (Guarded(n * bits // 8, torch.uint8), Guarded(n // group, torch.float32), Guarded(n, td))
        packed, scales, out = (g.t for g in guards)
        seen = []
        for epoch in (3, (1 << 40) + 3):
            aq.aq_configure(h, aq.AQ_EPOCH, epoch)
            aq.aq_quant_grad(h, grad, n, bits, packed, scales)
            aq.aq_dequant_grad(h, packed, scales, n, bits, out)
            torch.cuda.synchronize()
            check_guards(*guards)
            p_o, s_o = oracle.quant_grad_stochastic(bits16(grad), bits, group, 424242, epoch, DT[dtype][1])
            assert np.array_equal(packed.cpu().numpy(), p_o)
            assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_o.view(np.uint32))
            assert np.array_equal(bits16(out), oracle.dequant_grad(p_o, s_o, n, bits, group, DT[dtype][1]))
            seen.append(p_o)
        assert not np.array_equal(seen[0], seen[1])
    finally:
        aq.aq_destroy(h)


# ----------------------------------------------------------------- limits, overrides and random configurations

def test_largest_batch_of_small_samples():
    """4096 samples in one call (the limit of AQ_BATCH), ids in random order with one repeat and
    one out of range: grid of 4096 samples, the repeat check scans up to 4095 earlier ids."""
    cfg = synth.Boundary("wide", 4096, 4096, 1, 64, "fp16", 4, 64, 2, "normal", 0.1, seed=201)
    gs, gr = GpuSide(cfg, 4096), GpuSide(cfg, 4096)
    os_, or_ = (oracle.Side(4096, 1, 64, 4, 64, oracle.FP16) for _ in range(2))
    try:
        guards = (Guarded((4096, cfg.packed_bytes), torch.uint8), Guarded((4096, cfg.groups), torch.float32), Guarded((4096, 1, 64), torch.float16))
        packed, scales, out = (g.t for g in guards)
        for epoch in range(3):
            ids = synth.epoch_order(cfg, epoch).clone()
            ids[4000] = ids[17]                       # a repeat far into the call
            ids[123] = 5000                           # out of range
            act = synth.activation(cfg, torch.arange(4096), epoch, device="cuda")
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
        with pytest.raises(aq.AqError):
            aq.aq_configure(gs.h, aq.AQ_BATCH, 4097)
    finally:
        gs.close()
        gr.close()


def test_one_large_sample():
    """A single sequence of 2^24 elements (32 MB): 8192 rows, far more CTAs per sample than any workload."""
    cfg = synth.Boundary("long", 2, 1, 8192, 2048, "bf16", 3, 128, 2, "normal", 0.05, seed=202)
    run_boundary(cfg, check_all_m=True)


@pytest.mark.parametrize("rows_per_cta", [1, 3, 7, 1 << 20])
def test_rows_per_cta_override_does_not_change_results(rows_per_cta):
    cfg = synth.Boundary("rows", 4, 2, 21, 1000, "fp16", 4, 8, 2, "outlier", 0.2, seed=203)   # 2625 chunks: 11 rows, ragged
    gs, gr = GpuSide(cfg, 2), GpuSide(cfg, 2)
    os_, or_ = (oracle.Side(4, 21, 1000, 4, 8, oracle.FP16) for _ in range(2))
    try:
        for h in (gs.h, gr.h):
            aq.aq_configure(h, aq.AQ_ROWS_PER_CTA, rows_per_cta)
        guards = (Guarded((2, cfg.packed_bytes), torch.uint8), Guarded((2, cfg.groups), torch.float32), Guarded((2, 21, 1000), torch.float16))
        packed, scales, out = (g.t for g in guards)
        for epoch in range(3):
            ids = torch.tensor([3, 1], dtype=torch.int32)
            act = synth.activation(cfg, ids, epoch, device="cuda")
            aq.aq_encode(gs.h, act, ids.cuda(), packed, scales)
            aq.aq_configure(gr.h, aq.AQ_RAW, act)
            aq.aq_decode(gr.h, packed, scales, ids.cuda(), out)
            torch.cuda.synchronize()
            check_guards(*guards)
            p_o, s_o, _ = os_.encode(bits16(act), ids.numpy())
            out_o, _ = or_.decode(p_o, s_o, ids.numpy(), raw=bits16(act))
            assert np.array_equal(packed.cpu().numpy(), p_o) and np.array_equal(scales.cpu().numpy(), s_o)
            assert np.array_equal(bits16(out), out_o)
        assert aq.aq_state_checksum(gs.h) == os_.checksum() and aq.aq_state_checksum(gr.h) == or_.checksum()
    finally:
        gs.close()
        gr.close()


def test_random_configurations():
    """Seeded random shapes, widths, groups, types, batch sizes and rounding modes."""
    rng = np.random.default_rng(2206)
    for trial in range(24):
        group = int(rng.choice([8, 16, 32, 64, 128, 256]))
        hidden = group * int(rng.integers(1, 9))
        seq = int(rng.integers(1, 70))
        bits = int(rng.integers(1, 9))
        nb = int(rng.choice([1, 2, 3, 5]))
        n_samples = nb * int(rng.integers(1, 4))
        dtype = str(rng.choice(["fp16", "bf16"]))
        kind = str(rng.choice(["normal", "outlier", "student_t3"]))
        cfg = synth.Boundary(f"rnd{trial}", n_samples, nb, seq, hidden, dtype, bits, group, 3, kind,
                             float(rng.choice([0.0, 0.01, 0.5])), seed=300 + trial)
        run_boundary(cfg, stochastic_seed=(int(rng.integers(1 << 40)) if trial % 3 == 0 else None))


# ----------------------------------------------------------------- m in page-locked host memory

def test_hosted_store_gives_the_same_results():
    run_boundary(synth.TINY, hosted=True)
    run_boundary(synth.shrink(synth.GPT2_XL, 8, seq=128, epochs=3), n_batch=4, hosted=True)
    run_boundary(synth.shrink(synth.DEBERTA_XXL, 16, seq=32), hosted=True, stochastic_seed=5)
    cfg = synth.Boundary("hosted-ragged", 6, 3, 37, 136, "bf16", 3, 8, 3, "outlier", 0.3, seed=411)
    run_boundary(cfg, hosted=True)


def test_hosted_store_checkpoint_and_digest():
    cfg = synth.Boundary("hosted-ckpt", 3, 1, 4, 64, "fp16", 4, 64, 1, "normal", 0.1, seed=412)
    a, b = GpuSide(cfg, 1, hosted=True), GpuSide(cfg, 1)
    try:
        ids = torch.tensor([2], dtype=torch.int32, device="cuda")
        act = synth.activation(cfg, [2], 0, device="cuda")
        p = torch.empty((1, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
        s = torch.empty((1, cfg.groups), dtype=torch.float32, device="cuda")
        aq.aq_encode(a.h, act, ids, p, s)
        for i in range(3):
            row, seen = a.m_row(i)
            aq.aq_import_sample(b.h, i, row, seen)
        assert aq.aq_state_checksum(a.h) == aq.aq_state_checksum(b.h) == aq.aq_state_checksum_noalloc(a.h)
    finally:
        a.close()
        b.close()
