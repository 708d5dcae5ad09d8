"""aq_state_checksum_noalloc against aq_state_checksum, through the C ABI.

The entry point under test serves callers that cannot allocate device memory at the time
of the call (a process whose memory a caching pool handed out at start-up, a loop that cannot
take an allocator's device-wide synchronisation, a service with a fixed memory budget per
library): its scratch is a fixed array in the library image.  The digest must be the same 64 bits that the allocating entry
point returns -- the tolerance of every other digest test here: bit-exact -- and because the
fixed array keeps the previous call's contents, the check is made on consecutive calls, on
states of different sizes, and after the state changed.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2206_01299_b200 as aq
from fixtures import synth

pytestmark = pytest.mark.gpu


def _visit(h, cfg, ids, epoch):
    act = synth.activation(cfg, ids, epoch, device="cuda")
    packed = torch.empty((len(ids), cfg.packed_bytes), dtype=torch.uint8, device="cuda")
    scales = torch.empty((len(ids), cfg.groups), dtype=torch.float32, device="cuda")
    aq.aq_encode(h, act, torch.tensor(ids, dtype=torch.int32, device="cuda"), packed, scales)


def test_noalloc_digest_equals_the_allocating_one_on_consecutive_calls():
    # 5 x 700 x 1600 x 2 B = 11.2 MB of m: 11 slabs, the last one ragged
    big = synth.Boundary("noalloc-big", 5, 2, 700, 1600, "fp16", 4, 64, 2, "normal", 0.05, seed=91)
    # 3 x 3 x 64 x 2 B: far less than one slab, so the second call reads fewer slots than the first wrote
    small = synth.Boundary("noalloc-small", 3, 1, 3, 64, "bf16", 2, 64, 2, "normal", 0.05, seed=92)
    hb = aq.aq_create(big.n_samples, big.seq, big.hidden, big.bits, big.group)
    hs = aq.aq_create(small.n_samples, small.seq, small.hidden, small.bits, small.group)
    try:
        aq.aq_configure(hb, aq.AQ_BATCH, 2)
        aq.aq_configure(hs, aq.AQ_DTYPE, aq.AQ_BF16)
        empty = aq.aq_state_checksum(hb)
        assert aq.aq_state_checksum_noalloc(hb) == empty            # first call on this device: set-up
        assert aq.aq_state_checksum_noalloc(hb) == empty            # and again, on the array it left
        seen_digests = {empty}
        for epoch, ids in [(0, [4, 1]), (0, [0, 3]), (1, [1, 4])]:
            _visit(hb, big, ids, epoch)
            want = aq.aq_state_checksum(hb)
            assert want not in seen_digests                         # the state did change
            seen_digests.add(want)
            assert aq.aq_state_checksum_noalloc(hb) == want
            assert aq.aq_state_checksum_noalloc(hb) == want
            # a smaller state in between, on the same array
            _visit(hs, small, [epoch % 3], 0)
            want_small = aq.aq_state_checksum(hs)
            assert aq.aq_state_checksum_noalloc(hs) == want_small
            assert aq.aq_state_checksum_noalloc(hb) == want
        assert aq.aq_status(hb) == 0 and aq.aq_status(hs) == 0
    finally:
        aq.aq_destroy(hb)
        aq.aq_destroy(hs)


def test_noalloc_digest_takes_no_device_memory():
    cfg = synth.Boundary("noalloc-mem", 4, 1, 64, 256, "fp16", 4, 64, 1, "normal", 0.05, seed=93)
    h = aq.aq_create(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group)
    try:
        _visit(h, cfg, [2], 0)
        aq.aq_state_checksum_noalloc(h)                             # set-up done
        aq.aq_state_checksum(h)                                     # its kernel is loaded too
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        for _ in range(4):
            assert aq.aq_state_checksum_noalloc(h) == aq.aq_state_checksum(h)
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
    finally:
        aq.aq_destroy(h)


def test_noalloc_digest_rejects_null_output():
    h = aq.aq_create(2, 1, 64, 4, 64)
    try:
        rc = aq.lib().aq_state_checksum_noalloc(h, None)
        assert rc == aq.AQ_EINVAL
        assert "null" in aq.aq_last_error(h)
    finally:
        aq.aq_destroy(h)


def test_noalloc_digest_refuses_the_stores_it_is_not_built_for():
    for create in (lambda: aq.aq_create_lowbit(4, 2, 64, 4, 64, 8), lambda: aq.aq_create_fp32(4, 2, 64, 4, 64)):
        h = create()
        try:
            rc = aq.lib().aq_state_checksum_noalloc(h, ctypes.byref(ctypes.c_uint64(0)))
            assert rc == aq.AQ_EUNSUPPORTED
            assert "store" in aq.aq_last_error(h)
        finally:
            aq.aq_destroy(h)


def test_noalloc_digest_of_a_hosted_store_after_a_staged_call():
    """m in page-locked host memory, visited through aq_prefetch: the digest call has to wait for the rows
    that are still travelling back to the host block, and must then equal the allocating digest and the
    oracle's, on a stream of the caller's own, with a ragged bf16 state."""
    cfg = synth.Boundary("noalloc-hosted", 6, 3, 37, 136, "bf16", 3, 8, 2, "outlier", 0.3, seed=94)
    stream = torch.cuda.Stream()
    h = aq.aq_create_hosted(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group)
    o = oracle.Side(cfg.n_samples, cfg.seq, cfg.hidden, cfg.bits, cfg.group, oracle.BF16)
    try:
        aq.aq_configure(h, aq.AQ_DTYPE, aq.AQ_BF16)
        aq.aq_configure(h, aq.AQ_BATCH, cfg.n_batch)
        aq.aq_configure(h, aq.AQ_STREAM, stream.cuda_stream)
        packed = torch.empty((cfg.n_batch, cfg.packed_bytes), dtype=torch.uint8, device="cuda")
        scales = torch.empty((cfg.n_batch, cfg.groups), dtype=torch.float32, device="cuda")
        for epoch, id_list in [(0, [5, 0, 2]), (1, [2, 5, 0]), (1, [1, 3, 4])]:
            ids = torch.tensor(id_list, dtype=torch.int32)
            act = synth.activation(cfg, ids, epoch, device="cuda")
            torch.cuda.synchronize()
            aq.aq_prefetch(h, ids)
            aq.aq_encode(h, act, ids.cuda(), packed, scales)
            got = aq.aq_state_checksum_noalloc(h)                       # no synchronisation in between: the write-back is in flight
            o.encode(act.view(torch.int16).cpu().numpy().view(np.uint16), ids.numpy())
            assert got == o.checksum() == aq.aq_state_checksum(h) == aq.aq_state_checksum_noalloc(h)
    finally:
        aq.aq_destroy(h)
        o.close()
