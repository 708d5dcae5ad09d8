"""One stage boundary across two processes with the CUDA codec on either side: rank 0 owns the
sender handle, rank 1 the receiver handle, the message crosses through BoundaryLink.  Only one GPU
is at hand, so both ranks use it and the link runs over gloo (host memory); the kernels of the two
ranks never wait for one another on the device -- each side's next step is released by the host
when its message has arrived.  Either rank checks its own side against the CPU oracle bit for bit."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu

N_BATCH, EPOCHS = 4, 3


def _cfg():
    from fixtures import synth
    return synth.Boundary("gpu-link", 16, N_BATCH, 24, 256, "fp16", 3, 64, EPOCHS, "outlier", 0.1, seed=23)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _rank_main(rank, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import oracle
    import paper_2206_01299_b200 as aq
    from fixtures import synth
    from paper_2206_01299_b200.link import BoundaryLink
    cfg = _cfg()
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=2)
    h = aq.aq_create(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group)
    side = oracle.Side(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, oracle.FP16)
    try:
        aq.aq_configure(h, aq.AQ_BATCH, N_BATCH)
        first = torch.zeros(N_BATCH, dtype=torch.uint8, device="cuda")
        aq.aq_configure(h, aq.AQ_FIRST_FLAGS, first)
        link = BoundaryLink(dist, 1 - rank, N_BATCH, cfg.packed_bytes, cfg.groups, cfg.elems, torch.float16, "cpu")
        packed = torch.empty((N_BATCH, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
        scales = torch.empty((N_BATCH, cfg.groups), dtype=torch.float32, device="cuda")
        out = torch.empty((N_BATCH, cfg.seq, cfg.hidden), dtype=torch.float16, device="cuda")
        for epoch in range(EPOCHS):
            order = synth.epoch_order(cfg, epoch)
            for c in range(cfg.n_samples // N_BATCH):
                ids = order[c * N_BATCH:(c + 1) * N_BATCH].contiguous()
                if rank == 0:
                    act = synth.activation(cfg, ids, epoch, device="cuda")
                    aq.aq_encode(h, act, ids.cuda(), packed, scales)
                    torch.cuda.synchronize()
                    link.send(ids, first, packed, scales, act)
                    p_o, s_o, f_o = side.encode(_bits(act), ids.numpy())
                    assert np.array_equal(packed.cpu().numpy(), p_o) and np.array_equal(scales.cpu().numpy(), s_o)
                    assert np.array_equal(first.cpu().numpy(), f_o)
                else:
                    got_ids, flags, p, sc, raw = link.recv(expect_ids=ids)
                    raw_dev = None if raw is None else raw.cuda().reshape(N_BATCH, cfg.seq, cfg.hidden)
                    aq.aq_configure(h, aq.AQ_RAW, raw_dev)
                    aq.aq_decode(h, p.cuda(), sc.cuda(), got_ids.cuda(), out)
                    torch.cuda.synchronize()
                    out_o, f_o = side.decode(p.numpy(), sc.numpy(), got_ids.numpy(), raw=None if raw is None else _bits(raw))
                    assert np.array_equal(_bits(out), out_o)
                    assert np.array_equal(first.cpu().numpy(), f_o) and np.array_equal(flags.numpy(), f_o)
                    assert (raw is not None) == (epoch == 0)
            # the two copies of m agree after every epoch, and with the oracle's
            mine = aq.aq_state_checksum(h)
            assert mine == side.checksum()
            both = [None, None]
            dist.all_gather_object(both, mine)
            assert both[0] == both[1], f"epoch {epoch}: sender and receiver state differ"
        assert aq.aq_status(h) == 0
        np.save(os.path.join(out_dir, f"rank{rank}_ok.npy"), np.array([link.sent + link.received]))
        dist.barrier()
    finally:
        aq.aq_destroy(h)
        side.close()
        dist.destroy_process_group()


def test_boundary_across_two_processes_on_one_gpu(tmp_path):
    mp.spawn(_rank_main, args=(_free_port(), str(tmp_path)), nprocs=2, join=True)
    calls = EPOCHS * (16 // N_BATCH)
    assert int(np.load(tmp_path / "rank0_ok.npy")[0]) == calls
    assert int(np.load(tmp_path / "rank1_ok.npy")[0]) == calls
