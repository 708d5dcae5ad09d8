"""ctypes binding of libaq_b200.so: the same names as include/aq_b200.h, argument
marshalling only.  Every operation runs in the CUDA library; there is no Python or CPU
implementation behind these calls, and a missing library is an error.

Pointer arguments accept a torch tensor (its data_ptr() is passed; the tensor must be
contiguous), a numpy array (host forms), an int address, or None.
"""
import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libaq_b200.so")

AQ_OK, AQ_EINVAL, AQ_ENOMEM, AQ_ECUDA, AQ_EUNSUPPORTED = 0, -1, -2, -3, -4
AQ_DTYPE, AQ_BATCH, AQ_STREAM, AQ_RAW, AQ_FIRST_FLAGS, AQ_ROWS_PER_CTA = 1, 2, 3, 4, 5, 6
AQ_L2_PREFETCH = 10
AQ_RAW_LIST = 11
AQ_ROUNDING, AQ_SEED, AQ_EPOCH = 7, 8, 9
AQ_FP16, AQ_BF16 = 0, 1
AQ_ROUND_INTERVAL, AQ_ROUND_STOCHASTIC = 0, 1
AQ_ST_BAD_ID, AQ_ST_DUP_ID, AQ_ST_NO_RAW, AQ_ST_STAGED, AQ_ST_BAD_PTR = 1, 2, 4, 8, 16

# name -> (restype, argtypes); the load test checks these against the header
SIGNATURES = {
    "aq_create": (C.c_void_p, [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int]),
    "aq_create_hosted": (C.c_void_p, [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int]),
    "aq_create_fp32": (C.c_void_p, [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int]),
    "aq_create_lowbit": (C.c_void_p, [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]),
    "aq_create_hosted_lowbit": (C.c_void_p, [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]),
    "aq_destroy": (None, [C.c_void_p]),
    "aq_configure": (C.c_int, [C.c_void_p, C.c_int, C.c_int64]),
    "aq_encode": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "aq_decode": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "aq_encode_list": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "aq_decode_list": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "aq_quant_grad": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_void_p]),
    "aq_dequant_grad": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p]),
    "aq_state_checksum": (C.c_int, [C.c_void_p, C.POINTER(C.c_uint64)]),
    "aq_state_checksum_noalloc": (C.c_int, [C.c_void_p, C.POINTER(C.c_uint64)]),
    "aq_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_uint32)]),
    "aq_last_error": (C.c_char_p, [C.c_void_p]),
    "aq_last_error_code": (C.c_int, [C.c_void_p]),
    "aq_packed_bytes_per_sample": (C.c_int64, [C.c_void_p]),
    "aq_scales_per_sample": (C.c_int64, [C.c_void_p]),
    "aq_m_bytes_per_sample": (C.c_int64, [C.c_void_p]),
    "aq_encode_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "aq_decode_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "aq_wire_copy": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                               C.c_void_p]),
    "aq_wire_copy_grad": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int]),
    "aq_prefetch": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int]),
    "aq_export_sample": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]),
    "aq_import_sample": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_uint8]),
}

_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2206_01299_b200.build` "
                "(nvcc, sm_100a).  There is no fallback implementation.")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class AqError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"aq error {code}: {msg}")
        self.code = code


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        assert x.is_contiguous(), "tensor must be contiguous"
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        assert x.flags["C_CONTIGUOUS"], "array must be contiguous"
        return x.ctypes.data
    raise TypeError(type(x))


def _check(h, rc):
    if rc != AQ_OK:
        raise AqError(rc, aq_last_error(h))
    return rc


def _created(h):
    if not h:
        raise AqError(aq_last_error_code(None), aq_last_error(None))
    return h


def aq_create(n_samples, seq, hidden, bits, group):
    return _created(lib().aq_create(n_samples, seq, hidden, bits, group))


def aq_create_hosted(n_samples, seq, hidden, bits, group):
    return _created(lib().aq_create_hosted(n_samples, seq, hidden, bits, group))


def aq_create_fp32(n_samples, seq, hidden, bits, group):
    return _created(lib().aq_create_fp32(n_samples, seq, hidden, bits, group))


def aq_create_lowbit(n_samples, seq, hidden, bits, group, m_bits):
    return _created(lib().aq_create_lowbit(n_samples, seq, hidden, bits, group, m_bits))


def aq_create_hosted_lowbit(n_samples, seq, hidden, bits, group, m_bits):
    return _created(lib().aq_create_hosted_lowbit(n_samples, seq, hidden, bits, group, m_bits))


def aq_destroy(h):
    lib().aq_destroy(h)


def aq_configure(h, key, value):
    """value: an int, or a tensor / None for the pointer-valued keys (AQ_RAW, AQ_FIRST_FLAGS)."""
    val = value if isinstance(value, int) else (_ptr(value) or 0)
    return _check(h, lib().aq_configure(h, key, val))


def aq_encode(h, act, sample_ids, packed, scales):
    return _check(h, lib().aq_encode(h, _ptr(act), _ptr(sample_ids), _ptr(packed), _ptr(scales)))


def aq_decode(h, packed, scales, sample_ids, out):
    return _check(h, lib().aq_decode(h, _ptr(packed), _ptr(scales), _ptr(sample_ids), _ptr(out)))


def aq_encode_list(h, act_list, sample_ids, packed_list, scales_list):
    """The *_list arguments are int64 device tensors holding one device address per sample."""
    return _check(h, lib().aq_encode_list(h, _ptr(act_list), _ptr(sample_ids), _ptr(packed_list), _ptr(scales_list)))


def aq_decode_list(h, packed_list, scales_list, sample_ids, out_list):
    return _check(h, lib().aq_decode_list(h, _ptr(packed_list), _ptr(scales_list), _ptr(sample_ids), _ptr(out_list)))


def aq_quant_grad(h, grad, n_elems, bits, packed, scales):
    return _check(h, lib().aq_quant_grad(h, _ptr(grad), n_elems, bits, _ptr(packed), _ptr(scales)))


def aq_dequant_grad(h, packed, scales, n_elems, bits, out):
    return _check(h, lib().aq_dequant_grad(h, _ptr(packed), _ptr(scales), n_elems, bits, _ptr(out)))


def aq_state_checksum(h):
    v = C.c_uint64(0)
    _check(h, lib().aq_state_checksum(h, C.byref(v)))
    return v.value


def aq_state_checksum_noalloc(h):
    """aq_state_checksum through the library's fixed scratch array: no device allocation."""
    v = C.c_uint64(0)
    _check(h, lib().aq_state_checksum_noalloc(h, C.byref(v)))
    return v.value


def aq_status(h):
    v = C.c_uint32(0)
    _check(h, lib().aq_status(h, C.byref(v)))
    return v.value


def aq_last_error(h):
    return lib().aq_last_error(h).decode()


def aq_last_error_code(h):
    return lib().aq_last_error_code(h)


def aq_packed_bytes_per_sample(h):
    return lib().aq_packed_bytes_per_sample(h)


def aq_scales_per_sample(h):
    return lib().aq_scales_per_sample(h)


def aq_m_bytes_per_sample(h):
    return lib().aq_m_bytes_per_sample(h)


def aq_encode_host(h, act_host, sample_ids_host, packed_host, scales_host):
    return _check(h, lib().aq_encode_host(h, _ptr(act_host), _ptr(sample_ids_host), _ptr(packed_host),
                                          _ptr(scales_host)))


def aq_decode_host(h, packed_host, scales_host, raw_host, sample_ids_host, out_host):
    return _check(h, lib().aq_decode_host(h, _ptr(packed_host), _ptr(scales_host), _ptr(raw_host),
                                          _ptr(sample_ids_host), _ptr(out_host)))


def aq_wire_copy(h, dst_device, packed_dst, scales_dst, raw_dst, packed_src, scales_src, raw_src):
    return _check(h, lib().aq_wire_copy(h, dst_device, _ptr(packed_dst), _ptr(scales_dst), _ptr(raw_dst),
                                        _ptr(packed_src), _ptr(scales_src), _ptr(raw_src)))


def aq_wire_copy_grad(h, dst_device, packed_dst, scales_dst, packed_src, scales_src, n_elems, bits):
    return _check(h, lib().aq_wire_copy_grad(h, dst_device, _ptr(packed_dst), _ptr(scales_dst), _ptr(packed_src),
                                             _ptr(scales_src), n_elems, bits))


def aq_prefetch(h, sample_ids_host):
    """sample_ids_host: int32 CPU tensor / numpy array of AQ_BATCH ids."""
    return _check(h, lib().aq_prefetch(h, _ptr(sample_ids_host), int(sample_ids_host.numel()
                                       if hasattr(sample_ids_host, "numel") else sample_ids_host.size)))


def aq_export_sample(h, sample_id, m_host):
    """Returns the seen flag; fills m_host (numpy / CPU tensor of seq*hidden 16-bit values)."""
    seen = C.c_uint8(0)
    _check(h, lib().aq_export_sample(h, sample_id, _ptr(m_host), C.addressof(seen)))
    return seen.value


def aq_import_sample(h, sample_id, m_host, seen):
    return _check(h, lib().aq_import_sample(h, sample_id, _ptr(m_host), int(bool(seen))))
