"""The wire between two ranks: one stage boundary whose sender handle lives in one process (one
GPU) and whose receiver handle lives in another.

Algorithm 2 splits every visit of a sample between "network a" (the sending stage) and "network
b" (the receiving stage): a forms the message -- the quantized change of the activation, or, on
the first visit of a sample, the activation itself -- and b applies it to its own copy of the
previous messages.  This module carries that message with `torch.distributed` point-to-point
calls (NCCL between GPUs, gloo between CPU processes) into buffers that the receiving rank owns;
the codec call on either side then works on local memory only.  No kernel of the library reads
another GPU's memory.

It does none of the codec's arithmetic: the caller runs aq_encode before `send` and aq_decode
after `recv`.

Message of one call of n_batch samples, in this order:
  header  int32[1 + 2 * n_batch]: n_batch, the sample ids, the sender's first-visit flags
  codes   uint8[n_batch * packed_bytes]
  steps   float32[n_batch * groups]
  raw     16-bit[n_first * elems]: the activations of the first-visit samples, in call order
          (absent when the call has no first visit)
The header is what tells the receiver how long the message is, so it is read on the host of
both ranks (one small device-to-host copy per call).
"""
import torch


class BoundaryLink:
    def __init__(self, dist, peer, n_batch, packed_bytes, groups, elems, act_dtype, device="cpu", group=None):
        """dist: torch.distributed (initialised); peer: the rank at the other end of the boundary;
        sizes per sample as aq_packed_bytes_per_sample / aq_scales_per_sample report them; device: where
        the message travels from and to ("cuda" with NCCL: straight between the GPUs' memories; "cpu"
        with gloo: the sender's parts are copied to the host first, and the receiver copies what
        arrived to its GPU before it decodes)."""
        self.dist, self.peer, self.group = dist, peer, group
        self.n_batch, self.packed_bytes, self.groups, self.elems = n_batch, packed_bytes, groups, elems
        self.act_dtype, self.device = act_dtype, torch.device(device)
        # the receiving end's own buffers; aq_decode reads these
        self.header = torch.zeros(1 + 2 * n_batch, dtype=torch.int32, device=self.device)
        self.packed = torch.empty((n_batch, packed_bytes), dtype=torch.uint8, device=self.device)
        self.scales = torch.empty((n_batch, groups), dtype=torch.float32, device=self.device)
        self.raw = torch.zeros((n_batch, elems), dtype=act_dtype, device=self.device)
        self.sent = self.received = 0

    # ------------------------------------------------------------------ framing (no communication)

    def frame(self, ids, first_flags, packed, scales, act):
        """The tensors that make up one message, in sending order."""
        n = self.n_batch
        ids = ids.to(self.device, torch.int32).reshape(n)
        flags = first_flags.to(self.device).reshape(-1)[:n].to(torch.int32)
        header = torch.cat([torch.tensor([n], dtype=torch.int32, device=self.device), ids, flags])
        parts = [header, packed.reshape(n, self.packed_bytes).to(self.device), scales.reshape(n, self.groups).to(self.device)]
        first = torch.nonzero(flags.cpu(), as_tuple=False).reshape(-1)          # host read: sizes the message
        if first.numel():
            rows = act.reshape(n, self.elems).index_select(0, first.to(act.device))
            parts.append(rows.contiguous().to(self.device))
        return parts

    def unframe(self, header, raw_rows):
        """(ids, first_flags) from a received header; raw_rows (or None) go to their samples' rows of self.raw."""
        n = self.n_batch
        h = header.cpu()
        if int(h[0]) != n:
            raise ValueError(f"message for {int(h[0])} samples, this end expects {n}")
        ids, flags = h[1:1 + n].clone(), h[1 + n:1 + 2 * n].to(torch.uint8)
        first = torch.nonzero(flags, as_tuple=False).reshape(-1)
        if first.numel():
            self.raw.index_copy_(0, first.to(self.device), raw_rows.reshape(first.numel(), self.elems))
        return ids, flags

    # ------------------------------------------------------------------ the two ends

    def send(self, ids, first_flags, packed, scales, act):
        """Sender rank, after aq_encode: ids int32[n_batch], first_flags uint8[n_batch] (what AQ_FIRST_FLAGS
        received), packed, scales as aq_encode wrote them, act the call's activations."""
        for part in self.frame(ids, first_flags, packed, scales, act):
            self.dist.send(part.contiguous(), dst=self.peer, group=self.group)
        self.sent += 1

    def recv(self, expect_ids=None):
        """Receiver rank, before aq_decode.  Returns (ids, first_flags, packed, scales, raw): ids and flags
        on the host; packed, scales in this end's own buffers; raw = the buffer holding the first-visit
        activations at their samples' positions (pass it as AQ_RAW), or None when the call has none.
        expect_ids: this rank's own idea of the call's ids; a message for other ids is refused."""
        self.dist.recv(self.header, src=self.peer, group=self.group)
        n_first = int(self.header[1 + self.n_batch:].sum().item())               # host read: sizes the rest
        self.dist.recv(self.packed, src=self.peer, group=self.group)
        self.dist.recv(self.scales, src=self.peer, group=self.group)
        rows = None
        if n_first:
            rows = torch.empty((n_first, self.elems), dtype=self.act_dtype, device=self.device)
            self.dist.recv(rows, src=self.peer, group=self.group)
        ids, flags = self.unframe(self.header, rows)
        if expect_ids is not None and not torch.equal(ids, expect_ids.cpu().to(torch.int32).reshape(-1)):
            raise ValueError("the two ends of the boundary are not walking the same sample sequence")
        self.received += 1
        return ids, flags, self.packed, self.scales, (self.raw if n_first else None)
