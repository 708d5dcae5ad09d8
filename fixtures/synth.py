"""Seeded synthetic inputs for the boundary codec: activations, gradients, id orders.

This module holds NO codec arithmetic.  It serves the CUDA path, the tests and
the benchmark alike; everything is a pure function of integer counters
(seed, stream, sample id, epoch, element index), so any sample of any epoch can
be regenerated alone, on the CPU or on the GPU, with identical bits: integer
hashing in wrapping int64, one exact int->fp32 conversion, and single fp32
operations (no fused multiply-add can form across separate torch calls).

The workloads mimic the shapes of the paper's fine-tuning runs (Appendix
"Training Task Setup": GPT2-1.5B, sequence length 1024, micro-batch 1;
DeBERTa-1.5B on QNLI, sequence length 256, micro-batch 8) and the structure its
Figure 1(b) reports: across epochs the change of an activation is much smaller
than the activation itself.  The datasets and checkpoints themselves are not
available; these inputs stand in for them.
"""
from dataclasses import dataclass, replace

import torch

_M64 = (1 << 64) - 1
_PHI = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Python int -> the signed 64-bit value with the same low 64 bits."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _fmix_int(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def _srl(x: torch.Tensor, n: int) -> torch.Tensor:
    return (x >> n) & ((1 << (64 - n)) - 1)


def _fmix(z: torch.Tensor) -> torch.Tensor:
    """64-bit avalanche mixer on wrapping int64 tensors."""
    z = (z ^ _srl(z, 30)) * _s64(_C1)
    z = (z ^ _srl(z, 27)) * _s64(_C2)
    return z ^ _srl(z, 31)


# sum of eight independent 16-bit uniforms: mean 8*32767.5, variance 8*(2^32-1)/12
_Z_SCALE = 0.5 / (8.0 * ((1 << 32) - 1) / 12.0) ** 0.5


def _normal(key: torch.Tensor, counter: torch.Tensor, draw: int) -> torch.Tensor:
    """Approximately N(0,1) fp32 (Irwin-Hall, 8 terms), one value per (key, counter).

    key int64 [n,1], counter int64 [1,E]; `draw` separates independent variates
    of the same element.
    """
    total = None
    for t in range(2):
        h = _fmix(key + (counter * 16 + (draw * 2 + t)) * _s64(_PHI))
        part = (h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + ((h >> 48) & 0xFFFF)
        total = part if total is None else total + part
    centred = (2 * total - 8 * 65535).to(torch.float32)     # exact: |value| < 2^24
    return centred * _Z_SCALE


def _sample_keys(seed: int, stream: int, epoch: int, ids: torch.Tensor) -> torch.Tensor:
    k = _fmix_int(_fmix_int(seed * _PHI + stream) + epoch)
    return _fmix(ids.to(torch.int64) * _s64(_PHI) + _s64(k)).reshape(-1, 1)


@dataclass(frozen=True)
class Boundary:
    """One forward stage boundary: shapes, quantizer settings and value recipe."""
    name: str
    n_samples: int
    n_batch: int            # sequences per call (the micro-batch)
    seq: int
    hidden: int
    dtype: str              # "fp16" | "bf16"
    bits: int
    group: int
    epochs: int
    kind: str               # "normal" | "outlier" | "student_t3"
    drift: float            # std of the per-epoch change
    seed: int = 0
    stream: int = 0         # separates independent boundaries of one model

    @property
    def elems(self) -> int:
        return self.seq * self.hidden

    @property
    def torch_dtype(self):
        return torch.float16 if self.dtype == "fp16" else torch.bfloat16

    @property
    def packed_bytes(self) -> int:
        return self.elems * self.bits // 8

    @property
    def groups(self) -> int:
        return self.elems // self.group


@dataclass(frozen=True)
class GradWorkload:
    """Backward path: activation-gradients quantized directly, no buffer."""
    name: str
    n_batch: int
    seq: int
    hidden: int
    dtype: str
    bits: tuple
    group: int
    seed: int = 0

    @property
    def elems(self) -> int:
        return self.n_batch * self.seq * self.hidden

    @property
    def torch_dtype(self):
        return torch.float16 if self.dtype == "fp16" else torch.bfloat16


# The five workloads, at full size.
TINY = Boundary("tiny", 64, 4, 128, 768, "fp16", 2, 128, 3, "outlier", 0.05, seed=0)
GPT2_XL = Boundary("gpt2-1.5b", 4096, 1, 1024, 1600, "fp16", 4, 64, 5, "normal", 0.02, seed=1)
DEBERTA_XXL = Boundary("deberta-1.5b", 32768, 8, 256, 1536, "bf16", 2, 128, 3, "student_t3", 0.02,
                       seed=2)
BACKWARD = GradWorkload("backward", 4, 1024, 1600, "fp16", (8, 4), 64, seed=3)
# pipeline sweep: 8 boundaries, forward 3-bit delta + backward 6-bit direct, 16 micro-batches per macro-batch
SWEEP_FWD = Boundary("sweep-fwd", 8192, 1, 1024, 1600, "fp16", 3, 64, 3, "normal", 0.02, seed=4)
SWEEP_BWD = GradWorkload("sweep-bwd", 1, 1024, 1600, "fp16", (6,), 64, seed=5)
SWEEP_BOUNDARIES = 8
SWEEP_MICRO_BATCHES = 16


def shrink(cfg: Boundary, n_samples: int, seq: int = None, epochs: int = None) -> Boundary:
    """A smaller instance of the same recipe (for element-by-element checks on the CPU)."""
    return replace(cfg, n_samples=n_samples, seq=seq or cfg.seq, epochs=epochs or cfg.epochs)


def outlier_channels(cfg: Boundary, count: int = 4) -> torch.Tensor:
    ch = torch.arange(cfg.hidden, dtype=torch.int64)
    k = _fmix_int(_fmix_int(cfg.seed * _PHI + 0x0C4A) + cfg.stream)
    return torch.argsort(_fmix(ch * _s64(_PHI) + _s64(k)), stable=True)[:count]


def base_f32(cfg: Boundary, ids, device="cpu") -> torch.Tensor:
    """A_0 in fp32 for each id: tensor [len(ids), seq*hidden]."""
    ids = torch.as_tensor(ids, dtype=torch.int64, device=device).reshape(-1)
    ctr = torch.arange(cfg.elems, dtype=torch.int64, device=device).reshape(1, -1)
    key0 = _sample_keys(cfg.seed, cfg.stream, 0, ids)
    if cfg.kind == "student_t3":
        z0 = _normal(key0, ctr, 0)
        acc = None
        for d in (1, 2, 3):
            z = _normal(key0, ctr, d)
            sq = z * z
            acc = sq if acc is None else acc + sq
        a = z0 / torch.sqrt(acc / 3.0)
        return torch.clamp(a, -1.0e4, 1.0e4)
    a = _normal(key0, ctr, 0)
    if cfg.kind == "outlier":
        gain = torch.ones(cfg.hidden, dtype=torch.float32, device=device)
        gain[outlier_channels(cfg).to(device)] = 20.0
        a = (a.reshape(-1, cfg.seq, cfg.hidden) * gain).reshape(-1, cfg.elems)
    return a


def advance_f32(cfg: Boundary, a: torch.Tensor, ids, epoch: int) -> torch.Tensor:
    """A_epoch = A_{epoch-1} + drift * z_epoch, one fp32 multiply and one fp32 add per element."""
    ids = torch.as_tensor(ids, dtype=torch.int64, device=a.device).reshape(-1)
    ctr = torch.arange(cfg.elems, dtype=torch.int64, device=a.device).reshape(1, -1)
    z = _normal(_sample_keys(cfg.seed, cfg.stream, epoch, ids), ctr, 0)
    return a + z * cfg.drift


def activation(cfg: Boundary, ids, epoch: int, device="cpu") -> torch.Tensor:
    """a(xi) at the given epoch for each id: tensor [len(ids), seq, hidden] of cfg's dtype.

    A_0 follows cfg.kind; A_e = A_{e-1} + drift * z_e accumulated in fp32; the
    result is A_epoch rounded to the 16-bit type.
    """
    a = base_f32(cfg, ids, device)
    for e in range(1, epoch + 1):
        a = advance_f32(cfg, a, ids, e)
    return a.to(cfg.torch_dtype).reshape(-1, cfg.seq, cfg.hidden)


def gradient(cfg: GradWorkload, call: int, device="cpu", stream: int = 0) -> torch.Tensor:
    """Activation-gradient of one call: 1e-3 * z, with 1 % of the entries multiplied by 100."""
    ctr = torch.arange(cfg.elems, dtype=torch.int64, device=device).reshape(1, -1)
    key = _sample_keys(cfg.seed, 0x6AD + stream, 0, torch.tensor([call], device=device))
    g = _normal(key, ctr, 0) * 1.0e-3
    h = _fmix(key + (ctr * 16 + 15) * _s64(_PHI))
    spike = (_srl(h, 11) % 100) == 0
    g = torch.where(spike, g * 100.0, g)
    return g.to(cfg.torch_dtype).reshape(cfg.n_batch, cfg.seq, cfg.hidden)


def epoch_order(cfg: Boundary, epoch: int, n_samples: int = None) -> torch.Tensor:
    """Seeded permutation of the sample ids for one epoch (int32, CPU)."""
    n = n_samples or cfg.n_samples
    ids = torch.arange(n, dtype=torch.int64)
    k = _fmix_int(_fmix_int(cfg.seed * _PHI + 0x0E90C4) + epoch * 1315423911 + cfg.stream)
    return torch.argsort(_fmix(ids * _s64(_PHI) + _s64(k)), stable=True).to(torch.int32)
