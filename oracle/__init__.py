"""ctypes front end of the CPU oracle (test infrastructure, never a product path).

Arrays are numpy; 16-bit activations travel as uint16 bit patterns so that no
numpy float16 / bfloat16 conversion can leak into the oracle's arithmetic.
"""
import ctypes as C

import numpy as np

from . import build as _build

FP16, BF16 = 0, 1
ST_BAD_ID, ST_DUP_ID, ST_NO_RAW = 1, 2, 4

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        u16p, u8p, f32p, i32p = (C.POINTER(C.c_uint16), C.POINTER(C.c_uint8),
                                 C.POINTER(C.c_float), C.POINTER(C.c_int32))
        L.aqo_half_to_float.restype = C.c_float
        L.aqo_half_to_float.argtypes = [C.c_uint16]
        L.aqo_float_to_half.restype = C.c_uint16
        L.aqo_float_to_half.argtypes = [C.c_float]
        L.aqo_bf16_to_float.restype = C.c_float
        L.aqo_bf16_to_float.argtypes = [C.c_uint16]
        L.aqo_float_to_bf16.restype = C.c_uint16
        L.aqo_float_to_bf16.argtypes = [C.c_float]
        L.aqo_mix64.restype = C.c_uint64
        L.aqo_mix64.argtypes = [C.c_uint64, C.c_uint64]
        L.aqo_quantize_group.restype = None
        L.aqo_quantize_group.argtypes = [f32p, C.c_int, C.c_int, i32p, f32p]
        L.aqo_reconstruct.restype = C.c_float
        L.aqo_reconstruct.argtypes = [C.c_int32, C.c_float]
        L.aqo_put_code.restype = None
        L.aqo_put_code.argtypes = [u8p, C.c_int64, C.c_int, C.c_int32]
        L.aqo_get_code.restype = C.c_int32
        L.aqo_get_code.argtypes = [u8p, C.c_int64, C.c_int]
        L.aqo_create.restype = C.c_void_p
        L.aqo_create.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]
        L.aqo_destroy.restype = None
        L.aqo_destroy.argtypes = [C.c_void_p]
        L.aqo_m.restype = u16p
        L.aqo_m.argtypes = [C.c_void_p]
        L.aqo_seen.restype = u8p
        L.aqo_seen.argtypes = [C.c_void_p]
        L.aqo_status.restype = C.c_uint32
        L.aqo_status.argtypes = [C.c_void_p]
        L.aqo_encode.restype = None
        L.aqo_encode.argtypes = [C.c_void_p, u16p, i32p, C.c_int, u8p, f32p, u8p]
        L.aqo_decode.restype = None
        L.aqo_decode.argtypes = [C.c_void_p, u8p, f32p, u16p, i32p, C.c_int, u16p, u8p]
        L.aqo_quant_grad.restype = None
        L.aqo_quant_grad.argtypes = [u16p, C.c_int64, C.c_int, C.c_int, C.c_int, u8p, f32p]
        L.aqo_dequant_grad.restype = None
        L.aqo_dequant_grad.argtypes = [u8p, f32p, C.c_int64, C.c_int, C.c_int, C.c_int, u16p]
        u32p = C.POINTER(C.c_uint32)
        L.aqo_philox4x32_10.restype = None
        L.aqo_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.aqo_quantize_group_stochastic.restype = None
        L.aqo_quantize_group_stochastic.argtypes = [f32p, C.c_int, C.c_int, C.c_uint64, C.c_uint64, C.c_uint32,
                                                    C.c_int64, i32p, f32p]
        L.aqo_set_rounding.restype = None
        L.aqo_set_rounding.argtypes = [C.c_void_p, C.c_int, C.c_uint64, C.c_uint64]
        L.aqo_quant_grad_stochastic.restype = None
        L.aqo_quant_grad_stochastic.argtypes = [u16p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_uint64,
                                                u8p, f32p]
        L.aqo_low_create.restype = C.c_void_p
        L.aqo_low_create.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]
        L.aqo_low_set_rounding.restype = None
        L.aqo_low_set_rounding.argtypes = [C.c_void_p, C.c_int, C.c_uint64, C.c_uint64]
        L.aqo_low_destroy.restype = None
        L.aqo_low_destroy.argtypes = [C.c_void_p]
        L.aqo_low_m_codes.restype = u8p
        L.aqo_low_m_codes.argtypes = [C.c_void_p]
        L.aqo_low_m_scales.restype = f32p
        L.aqo_low_m_scales.argtypes = [C.c_void_p]
        L.aqo_low_seen.restype = u8p
        L.aqo_low_seen.argtypes = [C.c_void_p]
        L.aqo_low_status.restype = C.c_uint32
        L.aqo_low_status.argtypes = [C.c_void_p]
        L.aqo_low_encode.restype = None
        L.aqo_low_encode.argtypes = [C.c_void_p, u16p, i32p, C.c_int, u8p, f32p, u8p]
        L.aqo_low_decode.restype = None
        L.aqo_low_decode.argtypes = [C.c_void_p, u8p, f32p, u16p, i32p, C.c_int, u16p, u8p]
        L.aqo_low_state_checksum.restype = C.c_uint64
        L.aqo_low_state_checksum.argtypes = [C.c_void_p]
        L.aqo_state_checksum.restype = C.c_uint64
        L.aqo_state_checksum.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _c(a, dtype):
    a = np.ascontiguousarray(a)
    assert a.dtype == dtype, (a.dtype, dtype)
    return a


def half_to_float(h):
    return lib().aqo_half_to_float(int(h))


def float_to_half(f):
    return lib().aqo_float_to_half(float(f))


def bf16_to_float(h):
    return lib().aqo_bf16_to_float(int(h))


def float_to_bf16(f):
    return lib().aqo_float_to_bf16(float(f))


def mix64(index, word):
    return lib().aqo_mix64(int(index), int(word))


def quantize_group(d, bits):
    """d: float32[G] -> (k int32[G], Delta float)."""
    d = _c(d, np.float32)
    k = np.zeros(d.shape[0], np.int32)
    delta = C.c_float(0)
    lib().aqo_quantize_group(_p(d, C.c_float), d.shape[0], bits, _p(k, C.c_int32),
                             C.byref(delta))
    return k, np.float32(delta.value)


def philox4x32_10(counter, key):
    """counter: 4 uint32, key: 2 uint32 -> 4 uint32 (Philox4x32, 10 rounds)."""
    c = np.array(counter, np.uint32)
    k = np.array(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().aqo_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def quantize_group_stochastic(d, bits, seed, epoch, stream_id, first_elem=0):
    """d: float32[G] (G a multiple of 8) -> (k int32[G], Delta float), unbiased stochastic Q."""
    d = _c(d, np.float32)
    k = np.zeros(d.shape[0], np.int32)
    delta = C.c_float(0)
    lib().aqo_quantize_group_stochastic(_p(d, C.c_float), d.shape[0], bits, seed, epoch, stream_id, first_elem,
                                        _p(k, C.c_int32), C.byref(delta))
    return k, np.float32(delta.value)


def reconstruct(k, delta):
    return np.float32(lib().aqo_reconstruct(int(k), float(delta)))


def put_codes(codes, bits):
    """codes int[n] -> little-endian bitstream uint8[ceil(n*bits/8)]."""
    n = len(codes)
    out = np.zeros((n * bits + 7) // 8, np.uint8)
    for j, k in enumerate(codes):
        lib().aqo_put_code(_p(out, C.c_uint8), j, bits, int(k))
    return out


def get_codes(stream, n, bits):
    stream = _c(stream, np.uint8)
    return np.array([lib().aqo_get_code(_p(stream, C.c_uint8), j, bits) for j in range(n)],
                    np.int32)


class Side:
    """One copy of the previous-message array m: the sender's or the receiver's."""

    def __init__(self, n_samples, seq, hidden, bits, group, dtype=FP16):
        self.n_samples, self.seq, self.hidden = n_samples, seq, hidden
        self.bits, self.group, self.dtype = bits, group, dtype
        self.h = lib().aqo_create(n_samples, seq, hidden, bits, group, dtype)
        if not self.h:
            raise ValueError("aqo_create rejected the configuration")
        self.E = seq * hidden
        self.pbytes = self.E * bits // 8
        self.ngroups = self.E // group

    def close(self):
        if self.h:
            lib().aqo_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def m(self):
        n = self.n_samples * self.E
        return np.ctypeslib.as_array(lib().aqo_m(self.h), shape=(n,)).reshape(
            self.n_samples, self.seq, self.hidden)

    def seen(self):
        return np.ctypeslib.as_array(lib().aqo_seen(self.h), shape=(self.n_samples,))

    def status(self):
        return lib().aqo_status(self.h)

    def set_rounding(self, stochastic, seed=0, epoch=0):
        lib().aqo_set_rounding(self.h, int(bool(stochastic)), seed, epoch)

    def encode(self, act, ids):
        """act uint16[n_batch, seq, hidden], ids int32[n_batch] ->
        (packed uint8[n_batch, pbytes], scales float32[n_batch, ngroups], first uint8[n_batch])"""
        act = _c(act, np.uint16)
        ids = _c(ids, np.int32)
        nb = ids.shape[0]
        assert act.size == nb * self.E
        packed = np.empty((nb, self.pbytes), np.uint8)
        scales = np.empty((nb, self.ngroups), np.float32)
        first = np.zeros(nb, np.uint8)
        lib().aqo_encode(self.h, _p(act, C.c_uint16), _p(ids, C.c_int32), nb,
                         _p(packed, C.c_uint8), _p(scales, C.c_float), _p(first, C.c_uint8))
        return packed, scales, first

    def decode(self, packed, scales, ids, raw=None):
        packed = _c(packed, np.uint8)
        scales = _c(scales, np.float32)
        ids = _c(ids, np.int32)
        nb = ids.shape[0]
        out = np.empty((nb, self.seq, self.hidden), np.uint16)
        first = np.zeros(nb, np.uint8)
        rawp = None
        if raw is not None:
            raw = _c(raw, np.uint16)
            rawp = _p(raw, C.c_uint16)
        lib().aqo_decode(self.h, _p(packed, C.c_uint8), _p(scales, C.c_float), rawp,
                         _p(ids, C.c_int32), nb, _p(out, C.c_uint16), _p(first, C.c_uint8))
        return out, first

    def checksum(self):
        return lib().aqo_state_checksum(self.h)


class SideLow:
    """One copy of m kept in m_bits bits per element (codes + one fp32 step per group)."""

    def __init__(self, n_samples, seq, hidden, bits, group, dtype=FP16, m_bits=8):
        self.n_samples, self.seq, self.hidden = n_samples, seq, hidden
        self.bits, self.group, self.dtype, self.m_bits = bits, group, dtype, m_bits
        self.h = lib().aqo_low_create(n_samples, seq, hidden, bits, group, dtype, m_bits)
        if not self.h:
            raise ValueError("aqo_low_create rejected the configuration")
        self.E = seq * hidden
        self.pbytes = self.E * bits // 8
        self.ngroups = self.E // group
        self.mbytes = self.E * m_bits // 8

    def close(self):
        if self.h:
            lib().aqo_low_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def set_rounding(self, stochastic, seed=0, epoch=0):
        """Rounding of the messages; the store's own re-quantization stays deterministic."""
        lib().aqo_low_set_rounding(self.h, int(bool(stochastic)), seed, epoch)

    def m_codes(self):
        return np.ctypeslib.as_array(lib().aqo_low_m_codes(self.h), shape=(self.n_samples, self.mbytes))

    def m_scales(self):
        if self.m_bits == 32:
            return np.zeros((self.n_samples, 0), np.float32)
        return np.ctypeslib.as_array(lib().aqo_low_m_scales(self.h), shape=(self.n_samples, self.ngroups))

    def m_values(self):
        """The dequantized store as float64 [n_samples, E]."""
        if self.m_bits == 32:
            return self.m_codes().view(np.float32).astype(np.float64)
        out = np.empty((self.n_samples, self.E), np.float64)
        for i in range(self.n_samples):
            k = get_codes(self.m_codes()[i], self.E, self.m_bits).astype(np.float64)
            out[i] = (k + 0.5) * np.repeat(self.m_scales()[i].astype(np.float64), self.group)
        return out

    def seen(self):
        return np.ctypeslib.as_array(lib().aqo_low_seen(self.h), shape=(self.n_samples,))

    def status(self):
        return lib().aqo_low_status(self.h)

    def encode(self, act, ids):
        act = _c(act, np.uint16)
        ids = _c(ids, np.int32)
        nb = ids.shape[0]
        assert act.size == nb * self.E
        packed = np.empty((nb, self.pbytes), np.uint8)
        scales = np.empty((nb, self.ngroups), np.float32)
        first = np.zeros(nb, np.uint8)
        lib().aqo_low_encode(self.h, _p(act, C.c_uint16), _p(ids, C.c_int32), nb,
                             _p(packed, C.c_uint8), _p(scales, C.c_float), _p(first, C.c_uint8))
        return packed, scales, first

    def decode(self, packed, scales, ids, raw=None):
        packed = _c(packed, np.uint8)
        scales = _c(scales, np.float32)
        ids = _c(ids, np.int32)
        nb = ids.shape[0]
        out = np.empty((nb, self.seq, self.hidden), np.uint16)
        first = np.zeros(nb, np.uint8)
        rawp = None
        if raw is not None:
            raw = _c(raw, np.uint16)
            rawp = _p(raw, C.c_uint16)
        lib().aqo_low_decode(self.h, _p(packed, C.c_uint8), _p(scales, C.c_float), rawp,
                             _p(ids, C.c_int32), nb, _p(out, C.c_uint16), _p(first, C.c_uint8))
        return out, first

    def checksum(self):
        return lib().aqo_low_state_checksum(self.h)


def quant_grad(grad, bits, group, dtype=FP16):
    grad = _c(grad, np.uint16).reshape(-1)
    n = grad.shape[0]
    assert n % group == 0 and (n * bits) % 8 == 0
    packed = np.empty(n * bits // 8, np.uint8)
    scales = np.empty(n // group, np.float32)
    lib().aqo_quant_grad(_p(grad, C.c_uint16), n, bits, group, dtype,
                         _p(packed, C.c_uint8), _p(scales, C.c_float))
    return packed, scales


def quant_grad_stochastic(grad, bits, group, seed, epoch, dtype=FP16):
    grad = _c(grad, np.uint16).reshape(-1)
    n = grad.shape[0]
    assert n % group == 0 and (n * bits) % 8 == 0
    packed = np.empty(n * bits // 8, np.uint8)
    scales = np.empty(n // group, np.float32)
    lib().aqo_quant_grad_stochastic(_p(grad, C.c_uint16), n, bits, group, dtype, seed, epoch,
                                    _p(packed, C.c_uint8), _p(scales, C.c_float))
    return packed, scales


def dequant_grad(packed, scales, n, bits, group, dtype=FP16):
    packed = _c(packed, np.uint8)
    scales = _c(scales, np.float32)
    out = np.empty(n, np.uint16)
    lib().aqo_dequant_grad(_p(packed, C.c_uint8), _p(scales, C.c_float), n, bits, group, dtype,
                           _p(out, C.c_uint16))
    return out
