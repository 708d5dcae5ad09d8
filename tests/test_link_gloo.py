"""One stage boundary across two ranks, on CPU: rank 0 is the sending stage, rank 1 the receiving
stage, the message travels through BoundaryLink over gloo.  The codec on either side is the CPU
oracle (as the checker: the link itself carries bytes and does no arithmetic), so what is tested is
the protocol around the codec -- which message a first visit sends, how it is framed and unframed,
that both ranks walk the same sample sequence -- and that after every epoch the receiver's state
is the sender's (Algorithm 2: either network keeps its own copy of the previous messages)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from fixtures import synth
from paper_2206_01299_b200.link import BoundaryLink

CFG = synth.Boundary("link", 12, 3, 5, 128, "fp16", 3, 64, 3, "outlier", 0.1, seed=17)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _link(peer):
    return BoundaryLink(dist, peer, CFG.n_batch, CFG.packed_bytes, CFG.groups, CFG.elems, torch.float16)


def _sender(out_dir):
    side = oracle.Side(CFG.n_samples, CFG.seq, CFG.hidden, CFG.bits, CFG.group, oracle.FP16)
    link = _link(1)
    wire_bytes = []
    for epoch in range(CFG.epochs):
        order = synth.epoch_order(CFG, epoch)
        for c in range(CFG.n_samples // CFG.n_batch):
            ids = order[c * CFG.n_batch:(c + 1) * CFG.n_batch].contiguous()
            if epoch == 1 and c == 0:
                ids[1] = ids[0]                                   # a repeated id: skipped on both sides alike
            act = synth.activation(CFG, ids, epoch)
            packed, scales, first = side.encode(_bits(act), ids.numpy())
            parts = link.frame(ids, torch.from_numpy(first), torch.from_numpy(packed), torch.from_numpy(scales), act)
            wire_bytes.append(sum(p.numel() * p.element_size() for p in parts))
            link.send(ids, torch.from_numpy(first), torch.from_numpy(packed), torch.from_numpy(scales), act)
        # the receiver reports its digest after every epoch
        theirs = torch.zeros(1, dtype=torch.int64)
        dist.recv(theirs, src=1)
        assert theirs.item() == np.int64(np.uint64(side.checksum())), f"epoch {epoch}: the two copies of m differ"
    header = 4 * (1 + 2 * CFG.n_batch)
    body = CFG.n_batch * (CFG.packed_bytes + 4 * CFG.groups)
    per_epoch = CFG.n_samples // CFG.n_batch
    # first visits carry the activation itself, later visits b bits per element plus the steps
    assert wire_bytes[:per_epoch] == [header + body + CFG.n_batch * CFG.elems * 2] * per_epoch
    assert wire_bytes[per_epoch + 1:] == [header + body] * (2 * per_epoch - 1)
    np.save(os.path.join(out_dir, "sender_ok.npy"), np.array([link.sent]))


def _receiver(out_dir):
    side = oracle.Side(CFG.n_samples, CFG.seq, CFG.hidden, CFG.bits, CFG.group, oracle.FP16)
    link = _link(0)
    seen_first = 0
    for epoch in range(CFG.epochs):
        order = synth.epoch_order(CFG, epoch)
        for c in range(CFG.n_samples // CFG.n_batch):
            mine = order[c * CFG.n_batch:(c + 1) * CFG.n_batch].clone()
            if epoch == 1 and c == 0:
                mine[1] = mine[0]
            ids, flags, packed, scales, raw = link.recv(expect_ids=mine)
            assert (raw is not None) == (epoch == 0)
            seen_first += int(flags.sum())
            out, first = side.decode(packed.numpy(), scales.numpy(), ids.numpy(), raw=None if raw is None else _bits(raw))
            assert np.array_equal(first, flags.numpy())           # each side decides "first" from its own seen-set
            if epoch == 0:
                assert np.array_equal(out.reshape(CFG.n_batch, -1), _bits(raw))
        dist.send(torch.tensor([np.int64(np.uint64(side.checksum()))]), dst=0)
    assert seen_first == CFG.n_samples
    assert side.status() == oracle.ST_DUP_ID
    np.save(os.path.join(out_dir, "receiver_ok.npy"), np.array([link.received]))


def _rank_main(rank, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=2)
    try:
        (_sender if rank == 0 else _receiver)(out_dir)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_boundary_across_two_gloo_ranks(tmp_path):
    mp.spawn(_rank_main, args=(_free_port(), str(tmp_path)), nprocs=2, join=True)
    calls = CFG.epochs * (CFG.n_samples // CFG.n_batch)
    assert int(np.load(tmp_path / "sender_ok.npy")[0]) == calls
    assert int(np.load(tmp_path / "receiver_ok.npy")[0]) == calls


def test_framing_round_trip_without_communication():
    """frame() and unframe() alone: a mixed call (one first visit among delta visits) keeps the raw
    block of exactly that sample, at that sample's position."""
    link = BoundaryLink(None, 0, 3, 8, 2, 16, torch.float16)
    ids = torch.tensor([7, 2, 9], dtype=torch.int32)
    flags = torch.tensor([0, 1, 0], dtype=torch.uint8)
    packed = torch.arange(24, dtype=torch.uint8).reshape(3, 8)
    scales = torch.arange(6, dtype=torch.float32).reshape(3, 2)
    act = torch.arange(48, dtype=torch.float16).reshape(3, 16)
    parts = link.frame(ids, flags, packed, scales, act)
    assert [tuple(p.shape) for p in parts] == [(7,), (3, 8), (3, 2), (1, 16)]
    assert parts[0].tolist() == [3, 7, 2, 9, 0, 1, 0]
    got_ids, got_flags = link.unframe(parts[0], parts[3])
    assert got_ids.tolist() == [7, 2, 9] and got_flags.tolist() == [0, 1, 0]
    assert torch.equal(link.raw[1], act[1]) and not link.raw[0].any() and not link.raw[2].any()
    assert len(link.frame(ids, torch.zeros(3, dtype=torch.uint8), packed, scales, act)) == 3     # no first visit, no raw part
    other = BoundaryLink(None, 0, 4, 8, 2, 16, torch.float16)
    with pytest.raises(ValueError):
        other.unframe(parts[0], None)
