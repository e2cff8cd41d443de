"""ctypes front end of the CPU oracle (oracle/llms_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The GPU library and its binding never import
this package, and this package never imports them.

All arrays are numpy arrays on the host.  fp16 data travels as uint16 bit
patterns so that nothing here depends on numpy's own half conversions.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

_lib = None


class KVDesc(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("n_q_heads", C.c_int32), ("head_dim", C.c_int32),
        ("n_tokens", C.c_int32), ("chunk_len", C.c_int32), ("group_size", C.c_int32), ("quant_mode", C.c_int32),
        ("stride_l", C.c_int64), ("stride_s", C.c_int64), ("stride_h", C.c_int64),
    ]


class ChunkMeta(C.Structure):
    _fields_ = [
        ("chunk_id", C.c_uint32), ("bits", C.c_uint32), ("offset", C.c_uint64), ("nbytes", C.c_uint64),
        ("n_groups", C.c_uint32), ("checksum", C.c_uint32),
    ]


class ChunkState(C.Structure):
    _fields_ = [
        ("ctx_id", C.c_uint32), ("chunk_id", C.c_uint32), ("bits", C.c_uint32), ("resident", C.c_uint32),
        ("locked", C.c_uint32), ("pad_", C.c_uint32), ("last_access_step", C.c_uint64),
    ]


META_DTYPE = np.dtype([("chunk_id", "<u4"), ("bits", "<u4"), ("offset", "<u8"), ("nbytes", "<u8"),
                       ("n_groups", "<u4"), ("checksum", "<u4")])
STATE_DTYPE = np.dtype([("ctx_id", "<u4"), ("chunk_id", "<u4"), ("bits", "<u4"), ("resident", "<u4"),
                        ("locked", "<u4"), ("pad_", "<u4"), ("last_access_step", "<u8")])


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.orc_f16_to_f32.restype = C.c_float
        _lib.orc_f16_to_f32.argtypes = [C.c_uint16]
        _lib.orc_f32_to_f16.restype = C.c_uint16
        _lib.orc_f32_to_f16.argtypes = [C.c_float]
        _lib.orc_dequantize_one.restype = C.c_uint16
        _lib.orc_dequantize_one.argtypes = [C.c_uint16, C.c_uint16, C.c_uint8]
        _lib.orc_checksum.restype = C.c_uint32
        _lib.orc_checksum.argtypes = [C.c_void_p, C.c_uint64]
    return _lib


def make_desc(n_layers, n_kv_heads, n_q_heads, head_dim, n_tokens, chunk_len, group_size, quant_mode=0):
    """Descriptor of a contiguous kv[l][s][h][t][c] tensor."""
    d = KVDesc()
    d.n_layers, d.n_kv_heads, d.n_q_heads, d.head_dim = n_layers, n_kv_heads, n_q_heads, head_dim
    d.n_tokens, d.chunk_len, d.group_size, d.quant_mode = n_tokens, chunk_len, group_size, quant_mode
    d.stride_h = n_tokens * head_dim
    d.stride_s = n_kv_heads * d.stride_h
    d.stride_l = 2 * d.stride_s
    return d


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


def _check(rc, what):
    if rc < 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")
    return rc


def f16_to_f32(h):
    return lib().orc_f16_to_f32(int(h))


def f32_to_f16(f):
    return lib().orc_f32_to_f16(C.c_float(f))


def f32_array_to_f16_bits(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    f = lib().orc_f32_to_f16
    flat_in, flat_out = a.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = f(C.c_float(flat_in[i]))
    return out


def record_layout(desc, bits):
    co, nb = C.c_uint64(), C.c_uint64()
    _check(lib().orc_record_layout(C.byref(desc), int(bits), C.byref(co), C.byref(nb)), "record_layout")
    return co.value, nb.value


def record_bytes(desc, bits):
    return record_layout(desc, bits)[1]


def compressed_size(desc, bits):
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    out = C.c_uint64()
    _check(lib().orc_compressed_size(C.byref(desc), _ptr(bits), len(bits), C.byref(out)), "compressed_size")
    return out.value


def quantize_group(x_bits, bits):
    """x_bits: uint16 fp16 bit patterns of one group -> (scale_bits, zero_bits, codes)."""
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    sc, ze = C.c_uint16(), C.c_uint16()
    codes = np.empty(x.size, dtype=np.uint8)
    lib().orc_quantize_group(_ptr(x), C.c_int64(1), int(x.size), int(bits), C.byref(sc), C.byref(ze), _ptr(codes))
    return sc.value, ze.value, codes


def pack_codes(codes, bits):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty((codes.size * bits + 7) // 8, dtype=np.uint8)
    lib().orc_pack_codes(_ptr(codes), C.c_uint64(codes.size), int(bits), _ptr(out))
    return out


def unpack_codes(packed, n, bits):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.empty(n, dtype=np.uint8)
    lib().orc_unpack_codes(_ptr(packed), C.c_uint64(n), int(bits), _ptr(out))
    return out


def dequantize_one(scale_bits, zero_bits, q):
    return lib().orc_dequantize_one(int(scale_bits), int(zero_bits), int(q))


def checksum(buf):
    buf = np.ascontiguousarray(buf, dtype=np.uint8)
    return lib().orc_checksum(_ptr(buf), C.c_uint64(buf.size))


def compress_chunks(desc, kv_bits, chunk_ids, bits):
    """-> (out_buf uint8[total], meta structured array)."""
    kv = np.ascontiguousarray(kv_bits, dtype=np.uint16)
    ids = np.ascontiguousarray(chunk_ids, dtype=np.uint32)
    b = np.ascontiguousarray(bits, dtype=np.uint8)
    total = compressed_size(desc, b)
    out = np.empty(total, dtype=np.uint8)
    meta = np.zeros(len(ids), dtype=META_DTYPE)
    _check(lib().orc_compress_chunks(C.byref(desc), _ptr(kv), _ptr(ids), _ptr(b), len(ids), _ptr(out),
                                     C.c_uint64(total), _ptr(meta)), "compress_chunks")
    return out, meta


def decompress_chunks(desc, buf, meta, kv_out_bits, dst_ids=None):
    buf = np.ascontiguousarray(buf, dtype=np.uint8)
    meta = np.ascontiguousarray(meta, dtype=META_DTYPE)
    assert kv_out_bits.dtype == np.uint16 and kv_out_bits.flags.c_contiguous
    ids = None if dst_ids is None else np.ascontiguousarray(dst_ids, dtype=np.uint32)
    _check(lib().orc_decompress_chunks(C.byref(desc), _ptr(buf), _ptr(meta), None if ids is None else _ptr(ids),
                                       len(meta), _ptr(kv_out_bits)), "decompress_chunks")
    return kv_out_bits


def attention_window(desc, kv_bits, q_win_bits, W):
    kv = np.ascontiguousarray(kv_bits, dtype=np.uint16)
    q = np.ascontiguousarray(q_win_bits, dtype=np.uint16)
    probs = np.empty((desc.n_layers, desc.n_q_heads, W, desc.n_tokens), dtype=np.float64)
    _check(lib().orc_attention_window(C.byref(desc), _ptr(kv), _ptr(q), int(W), _ptr(probs)), "attention_window")
    return probs


def chunk_tolerance_from_probs(desc, probs, W):
    p = np.ascontiguousarray(probs, dtype=np.float64)
    assert p.size == desc.n_layers * desc.n_q_heads * W * desc.n_tokens
    scores = np.empty(desc.n_tokens // desc.chunk_len, dtype=np.float64)
    _check(lib().orc_chunk_tolerance_from_probs(C.byref(desc), _ptr(p), int(W), _ptr(scores)), "tolerance_from_probs")
    return scores


def chunk_tolerance(desc, kv_bits, q_win_bits, W):
    kv = np.ascontiguousarray(kv_bits, dtype=np.uint16)
    q = np.ascontiguousarray(q_win_bits, dtype=np.uint16)
    scores = np.empty(desc.n_tokens // desc.chunk_len, dtype=np.float64)
    _check(lib().orc_chunk_tolerance(C.byref(desc), _ptr(kv), _ptr(q), int(W), _ptr(scores)), "chunk_tolerance")
    return scores


def assign_bits(scores, frac):
    s = np.ascontiguousarray(scores, dtype=np.float32)
    f = (C.c_float * 3)(*[float(x) for x in frac])
    bits = np.empty(s.size, dtype=np.uint8)
    order = np.empty(s.size, dtype=np.uint32)
    _check(lib().orc_assign_bits(_ptr(s), int(s.size), f, _ptr(bits), _ptr(order)), "assign_bits")
    return bits, order


def assign_levels(scores, frac, levels):
    """Eq. 2 for a level set {top, middle, low}, e.g. (8, 4, 2) or (4, 2, 1)."""
    s = np.ascontiguousarray(scores, dtype=np.float32)
    f = (C.c_float * 3)(*[float(x) for x in frac])
    lv = (C.c_uint8 * 3)(*[int(x) for x in levels])
    bits = np.empty(s.size, dtype=np.uint8)
    order = np.empty(s.size, dtype=np.uint32)
    _check(lib().orc_assign_levels(_ptr(s), int(s.size), f, lv, _ptr(bits), _ptr(order)), "assign_levels")
    return bits, order


def optimize_thresholds(scores, ratio_global):
    """-> (frac float32[3], counts int[3]) for the levels 8 / 4 / 2 bits."""
    s = np.ascontiguousarray(scores, dtype=np.float32)
    frac = (C.c_float * 3)()
    counts = (C.c_int * 3)()
    _check(lib().orc_optimize_thresholds(_ptr(s), int(s.size), C.c_float(ratio_global), frac, counts), "optimize_thresholds")
    return np.array(list(frac), dtype=np.float32), list(counts)


def optimize_thresholds_levels(scores, ratio_global, levels):
    """-> (frac float32[3], counts int[3]) for a level set {top, middle, low}."""
    s = np.ascontiguousarray(scores, dtype=np.float32)
    frac = (C.c_float * 3)()
    counts = (C.c_int * 3)()
    lv = (C.c_uint8 * 3)(*[int(x) for x in levels])
    _check(lib().orc_optimize_thresholds_levels(_ptr(s), int(s.size), C.c_float(ratio_global), lv, frac, counts),
           "optimize_thresholds_levels")
    return np.array(list(frac), dtype=np.float32), list(counts)


def lctru_order(table):
    t = np.ascontiguousarray(table, dtype=STATE_DTYPE)
    order = np.empty(max(len(t), 1), dtype=np.uint32)
    m = _check(lib().orc_lctru_order(_ptr(t), len(t), _ptr(order)), "lctru_order")
    return order[:m].copy()


def set_num_threads(n):
    """Threads the oracle's slab loops may use from now on (for timing it single-threaded)."""
    lib().orc_set_num_threads(int(n))


def num_threads():
    return lib().orc_num_threads()
