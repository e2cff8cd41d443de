"""ctypes binding of libllms.so: the same names as include/llms.h, argument marshalling only.

Tensors may be torch tensors (device or pinned host), numpy arrays (host) or raw integer addresses;
nothing here computes anything.  A missing library is an error: there is no fallback path.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# LLMS_LIBRARY names another build of the library to load instead of the in-tree one (the checked build's test uses it)
LIB_PATH = os.environ.get("LLMS_LIBRARY") or os.path.join(_HERE, "libllms.so")
_lib = None

OK = 0
ERR_INVALID_ARG, ERR_BAD_BITS, ERR_MISALIGNED, ERR_BUF_TOO_SMALL = -1, -2, -3, -4
ERR_CUDA, ERR_TIMEOUT, ERR_CORRUPT, ERR_UNSUPPORTED = -5, -6, -7, -8


class LlmsError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        msg = lib().llms_strerror(status).decode()
        if status == ERR_CUDA:
            msg += ": " + lib().llms_last_cuda_error().decode()
        super().__init__(f"{what}: {msg} ({status})")


class KVDesc(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("n_q_heads", C.c_int32), ("head_dim", C.c_int32),
        ("n_tokens", C.c_int32), ("chunk_len", C.c_int32), ("group_size", C.c_int32), ("quant_mode", C.c_int32),
        ("stride_l", C.c_int64), ("stride_s", C.c_int64), ("stride_h", C.c_int64),
    ]


META_DTYPE = np.dtype([("chunk_id", "<u4"), ("bits", "<u4"), ("offset", "<u8"), ("nbytes", "<u8"),
                       ("n_groups", "<u4"), ("checksum", "<u4")])
STATE_DTYPE = np.dtype([("ctx_id", "<u4"), ("chunk_id", "<u4"), ("bits", "<u4"), ("resident", "<u4"),
                        ("locked", "<u4"), ("pad_", "<u4"), ("last_access_step", "<u8")])

_SIGNATURES = {
    "llms_strerror": (C.c_char_p, [C.c_int]),
    "llms_last_cuda_error": (C.c_char_p, []),
    "llms_record_layout": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]),
    "llms_record_bytes": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p]),
    "llms_compressed_size": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]),
    "llms_codec_workspace_bytes": (C.c_int, [C.c_int, C.c_void_p]),
    "llms_compress_chunks": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                       C.c_uint64, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]),
    "llms_compress_chunks_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                              C.c_uint64, C.c_void_p, C.c_void_p]),
    "llms_decompress_chunks": (C.c_int, [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                         C.c_void_p, C.c_uint64, C.c_void_p]),
    "llms_decompress_chunks_ordered": (C.c_int, [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_int,
                                                 C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]),
    "llms_codec_corrupt_count": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "llms_tolerance_workspace_bytes": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p]),
    "llms_chunk_tolerance": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                       C.c_uint64, C.c_void_p]),
    "llms_chunk_tolerance_from_probs": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                                  C.c_uint64, C.c_void_p]),
    "llms_assign_bits": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]),
    "llms_assign_levels": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "llms_optimize_thresholds": (C.c_int, [C.c_void_p, C.c_int, C.c_float, C.c_void_p]),
    "llms_optimize_thresholds_levels": (C.c_int, [C.c_void_p, C.c_int, C.c_float, C.c_void_p, C.c_void_p]),
    "llms_compress_context": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_uint64,
                                        C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p]),
    "llms_lctru_order": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p]),
    "llms_swap_out": (C.c_int, [C.c_void_p, C.c_uint64, C.c_void_p, C.c_int, C.c_void_p, C.c_uint64, C.c_void_p,
                                C.c_void_p, C.c_void_p, C.c_void_p]),
    "llms_swap_in": (C.c_int, [C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_uint64,
                               C.c_void_p, C.c_void_p, C.c_void_p]),
    "llms_wait": (C.c_int, [C.c_void_p, C.c_uint32]),
    "llms_stream_probe": (C.c_int, [C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64, C.c_uint64, C.c_int, C.c_int, C.c_void_p]),
    "llms_debug_bounds": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "llms_stream_probe_split": (C.c_int, [C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64, C.c_uint64, C.c_int, C.c_int, C.c_int,
                                          C.c_void_p]),
}


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2403_11805_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        _lib = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(_lib, name)
            fn.restype, fn.argtypes = res, args
    return _lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        assert x.flags.c_contiguous
        return x.ctypes.data
    if hasattr(x, "data_ptr"):          # torch tensor
        assert x.is_contiguous()
        return x.data_ptr()
    if isinstance(x, C.Structure):
        return C.addressof(x)
    raise TypeError(type(x))


def _nbytes(x):
    if isinstance(x, np.ndarray):
        return x.nbytes
    return x.numel() * x.element_size()


def _stream(s):
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _event(e):
    if e is None:
        return None
    if isinstance(e, int):
        return e
    h = e.cuda_event
    return h.value if hasattr(h, "value") else int(h)


def _check(rc, what):
    if rc < 0:
        raise LlmsError(rc, what)
    return rc


def make_desc(n_layers, n_kv_heads, n_q_heads, head_dim, n_tokens, chunk_len, group_size, quant_mode=0):
    """Descriptor of a contiguous kv[l][s][h][t][c] tensor."""
    d = KVDesc()
    d.n_layers, d.n_kv_heads, d.n_q_heads, d.head_dim = n_layers, n_kv_heads, n_q_heads, head_dim
    d.n_tokens, d.chunk_len, d.group_size, d.quant_mode = n_tokens, chunk_len, group_size, quant_mode
    d.stride_h = n_tokens * head_dim
    d.stride_s = n_kv_heads * d.stride_h
    d.stride_l = 2 * d.stride_s
    return d


def desc_of(shape, quant_mode=0, n_tokens=None):
    """Descriptor for a synth.KVShape (n_tokens overrides the token count, e.g. for a slot pool)."""
    return make_desc(shape.n_layers, shape.n_kv_heads, shape.n_q_heads, shape.head_dim,
                     shape.n_tokens if n_tokens is None else n_tokens, shape.chunk_len, shape.group_size, quant_mode)


def new_meta(n, pinned=False):
    """n zeroed llms_chunk_meta entries as a numpy structured array (optionally over pinned memory)."""
    if not pinned:
        return np.zeros(n, dtype=META_DTYPE)
    import torch
    t = torch.zeros(max(n, 1) * META_DTYPE.itemsize, dtype=torch.uint8).pin_memory()
    return t.numpy()[:n * META_DTYPE.itemsize].view(META_DTYPE)   # the view keeps the pinned storage alive


def new_pinned(n, dtype=np.uint8):
    """n zeroed elements as a numpy array over page-locked memory (e.g. the level array of compress_context)."""
    import torch
    dt = np.dtype(dtype)
    t = torch.zeros(max(n, 1) * dt.itemsize, dtype=torch.uint8).pin_memory()
    return t.numpy()[:n * dt.itemsize].view(dt)                  # the view keeps the pinned storage alive


def new_event(stream=None):
    """A created cudaEvent_t wrapped by torch (recorded once so that the handle exists)."""
    import torch
    ev = torch.cuda.Event()
    ev.record(torch.cuda.current_stream() if stream is None else stream)
    return ev


# ----------------------------------------------------------------------------- sizes

def record_layout(desc, bits):
    co, nb = C.c_uint64(), C.c_uint64()
    _check(lib().llms_record_layout(C.addressof(desc), int(bits), C.addressof(co), C.addressof(nb)), "llms_record_layout")
    return co.value, nb.value


def record_bytes(desc, bits):
    nb = C.c_uint64()
    _check(lib().llms_record_bytes(C.addressof(desc), int(bits), C.addressof(nb)), "llms_record_bytes")
    return nb.value


def compressed_size(desc, bits):
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    nb = C.c_uint64()
    _check(lib().llms_compressed_size(C.addressof(desc), _ptr(bits), len(bits), C.addressof(nb)), "llms_compressed_size")
    return nb.value


def codec_workspace_bytes(n):
    nb = C.c_uint64()
    _check(lib().llms_codec_workspace_bytes(int(n), C.addressof(nb)), "llms_codec_workspace_bytes")
    return nb.value


def tolerance_workspace_bytes(desc, W):
    nb = C.c_uint64()
    _check(lib().llms_tolerance_workspace_bytes(C.addressof(desc), int(W), C.addressof(nb)), "llms_tolerance_workspace_bytes")
    return nb.value


# ----------------------------------------------------------------------------- codec

def codec_launches(desc, bits):
    """Kernels one compress or decompress call launches.  Groups of channels of a token: one codec kernel for the whole
    call (the bit-widths are phases of it, and its last CTA stores or checks the sums; a pageable meta array gets the
    sums by a copy).  Channel-wise mode: one kernel per bit-width present and one small kernel for the sums."""
    return len(set(int(b) for b in bits)) + 1 if desc.quant_mode == 1 else 1


def compress_chunks(desc, kv, chunk_ids, bits, out_buf, meta, workspace, stream=None, out_bytes=None, workspace_bytes=None):
    chunk_ids = np.ascontiguousarray(chunk_ids, dtype=np.uint32)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    assert len(chunk_ids) == len(bits) and len(meta) >= len(bits)
    _check(lib().llms_compress_chunks(
        C.addressof(desc), _ptr(kv), _ptr(chunk_ids), _ptr(bits), len(bits), _ptr(out_buf),
        _nbytes(out_buf) if out_bytes is None else out_bytes, _ptr(meta), _ptr(workspace),
        _nbytes(workspace) if workspace_bytes is None else workspace_bytes, _stream(stream)), "llms_compress_chunks")


STATIC_MAX_CHUNKS = 1024


def compress_chunks_static(desc, kv, chunk_ids, bits, out_buf, meta, stream=None, out_bytes=None):
    """llms_compress_chunks_static: same as compress_chunks, scratch built into the library (<= 1024 chunks)."""
    chunk_ids = np.ascontiguousarray(chunk_ids, dtype=np.uint32)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    assert len(chunk_ids) == len(bits) and len(meta) >= len(bits)
    _check(lib().llms_compress_chunks_static(
        C.addressof(desc), _ptr(kv), _ptr(chunk_ids), _ptr(bits), len(bits), _ptr(out_buf),
        _nbytes(out_buf) if out_bytes is None else out_bytes, _ptr(meta), _stream(stream)), "llms_compress_chunks_static")


def decompress_chunks(desc, buf, meta, dst_chunk_ids, kv_out, workspace, stream=None, n=None, workspace_bytes=None,
                      buf_bytes=None):
    ids = None if dst_chunk_ids is None else np.ascontiguousarray(dst_chunk_ids, dtype=np.uint32)
    n = len(meta) if n is None else n
    _check(lib().llms_decompress_chunks(
        C.addressof(desc), _ptr(buf), _nbytes(buf) if buf_bytes is None else buf_bytes, _ptr(meta), _ptr(ids), n, _ptr(kv_out), _ptr(workspace),
        _nbytes(workspace) if workspace_bytes is None else workspace_bytes, _stream(stream)), "llms_decompress_chunks")


def decompress_chunks_ordered(desc, buf, meta, dst_chunk_ids, kv_out, workspace, stream=None, n=None, workspace_bytes=None,
                              buf_bytes=None):
    """llms_decompress_chunks_ordered: meta pinned; its checksums are read by the device in stream order."""
    ids = None if dst_chunk_ids is None else np.ascontiguousarray(dst_chunk_ids, dtype=np.uint32)
    n = len(meta) if n is None else n
    _check(lib().llms_decompress_chunks_ordered(
        C.addressof(desc), _ptr(buf), _nbytes(buf) if buf_bytes is None else buf_bytes, _ptr(meta), _ptr(ids), n, _ptr(kv_out), _ptr(workspace),
        _nbytes(workspace) if workspace_bytes is None else workspace_bytes, _stream(stream)), "llms_decompress_chunks_ordered")


def codec_corrupt_count(workspace, stream=None):
    """Synchronises the stream; returns the number of records whose checksum did not match."""
    bad = C.c_uint32()
    rc = lib().llms_codec_corrupt_count(_ptr(workspace), C.addressof(bad), _stream(stream))
    if rc not in (OK, ERR_CORRUPT):
        _check(rc, "llms_codec_corrupt_count")
    return bad.value


# ----------------------------------------------------------------------------- tolerance score

def chunk_tolerance(desc, kv, q_win, W, scores, workspace, stream=None):
    _check(lib().llms_chunk_tolerance(C.addressof(desc), _ptr(kv), _ptr(q_win), int(W), _ptr(scores), _ptr(workspace),
                                      _nbytes(workspace), _stream(stream)), "llms_chunk_tolerance")


def chunk_tolerance_from_probs(desc, probs, W, scores, workspace, stream=None):
    _check(lib().llms_chunk_tolerance_from_probs(C.addressof(desc), _ptr(probs), int(W), _ptr(scores), _ptr(workspace),
                                                 _nbytes(workspace), _stream(stream)), "llms_chunk_tolerance_from_probs")


# ----------------------------------------------------------------------------- policy (host)

def assign_bits(scores, frac):
    s = np.ascontiguousarray(scores, dtype=np.float32)
    f = np.asarray(frac, dtype=np.float32)
    bits = np.empty(s.size, dtype=np.uint8)
    order = np.empty(s.size, dtype=np.uint32)
    _check(lib().llms_assign_bits(_ptr(s), int(s.size), _ptr(f), _ptr(bits), _ptr(order)), "llms_assign_bits")
    return bits, order


def assign_levels(scores, frac, levels):
    """Eq. 2 for a level set {top, middle, low}, e.g. (4, 2, 1)."""
    s = np.ascontiguousarray(scores, dtype=np.float32)
    f = np.asarray(frac, dtype=np.float32)
    lv = np.asarray(levels, dtype=np.uint8)
    assert f.size == 3 and lv.size == 3
    bits = np.empty(s.size, dtype=np.uint8)
    order = np.empty(s.size, dtype=np.uint32)
    _check(lib().llms_assign_levels(_ptr(s), int(s.size), _ptr(f), _ptr(lv), _ptr(bits), _ptr(order)), "llms_assign_levels")
    return bits, order


def level_counts(n, frac, levels=(8, 4, 2)):
    """How many of n chunks each level gets under llms_assign_levels (the counts depend on n and frac alone):
    asked of the library itself, on n distinct scores."""
    bits, _ = assign_levels(np.arange(n, 0, -1, dtype=np.float32), frac, levels)
    return tuple(int((bits == b).sum()) for b in levels)


def optimize_thresholds(scores, ratio_global):
    s = np.ascontiguousarray(scores, dtype=np.float32)
    frac = np.zeros(3, dtype=np.float32)
    _check(lib().llms_optimize_thresholds(_ptr(s), int(s.size), float(ratio_global), _ptr(frac)), "llms_optimize_thresholds")
    return frac


def optimize_thresholds_levels(scores, ratio_global, levels):
    s = np.ascontiguousarray(scores, dtype=np.float32)
    lv = np.asarray(levels, dtype=np.uint8)
    assert lv.size == 3
    frac = np.zeros(3, dtype=np.float32)
    _check(lib().llms_optimize_thresholds_levels(_ptr(s), int(s.size), float(ratio_global), _ptr(lv), _ptr(frac)),
           "llms_optimize_thresholds_levels")
    return frac


def lctru_order(table):
    t = np.ascontiguousarray(table, dtype=STATE_DTYPE)
    order = np.empty(max(len(t), 1), dtype=np.uint32)
    m = _check(lib().llms_lctru_order(_ptr(t), len(t), _ptr(order)), "llms_lctru_order")
    return order[:m].copy()


# ----------------------------------------------------------------------------- a whole context

def compress_context(desc, kv, q_win, W, frac, levels, scores_dev, scores_host, bits_out, out_buf, meta,
                     tolerance_workspace, codec_workspace, after_scores=None, stream=None):
    """llms_compress_context: scores, levels and records of every chunk in one call.
    frac: float32[3], levels: uint8[3], bits_out: uint8[n_chunks] numpy arrays; scores_host: fp32 tensor.
    With scores_host, bits_out and meta all in page-locked memory nothing synchronises: the three arrays are valid
    once after_scores has completed.  Otherwise the stream is synchronised once inside the call."""
    assert frac.dtype == np.float32 and levels.dtype == np.uint8 and bits_out.dtype == np.uint8
    _check(lib().llms_compress_context(
        C.addressof(desc), _ptr(kv), _ptr(q_win), int(W), _ptr(frac), _ptr(levels), _ptr(scores_dev), _ptr(scores_host),
        _ptr(bits_out), _ptr(out_buf), _nbytes(out_buf), _ptr(meta), _ptr(tolerance_workspace), _nbytes(tolerance_workspace),
        _ptr(codec_workspace), _nbytes(codec_workspace), _event(after_scores), _stream(stream)), "llms_compress_context")


# ----------------------------------------------------------------------------- swap

def swap_out(dev_buf, meta, pinned_dst, host_offsets=None, side_stream=None, after=None, done=None, n=None,
             dev_bytes=None, host_bytes=None):
    ho = None if host_offsets is None else np.ascontiguousarray(host_offsets, dtype=np.uint64)
    _check(lib().llms_swap_out(_ptr(dev_buf), _nbytes(dev_buf) if dev_bytes is None else dev_bytes, _ptr(meta),
                               len(meta) if n is None else n, _ptr(pinned_dst),
                               _nbytes(pinned_dst) if host_bytes is None else host_bytes, _ptr(ho),
                               _stream(side_stream), _event(after), _event(done)), "llms_swap_out")


def swap_in(pinned_src, meta, dev_buf, host_offsets=None, side_stream=None, after=None, done=None, n=None,
            dev_bytes=None, host_bytes=None):
    ho = None if host_offsets is None else np.ascontiguousarray(host_offsets, dtype=np.uint64)
    _check(lib().llms_swap_in(_ptr(pinned_src), _nbytes(pinned_src) if host_bytes is None else host_bytes, _ptr(ho),
                              _ptr(meta), len(meta) if n is None else n, _ptr(dev_buf),
                              _nbytes(dev_buf) if dev_bytes is None else dev_bytes,
                              _stream(side_stream), _event(after), _event(done)), "llms_swap_in")


def wait(event, timeout_ms=10000):
    _check(lib().llms_wait(_event(event), int(timeout_ms)), "llms_wait")


# ----------------------------------------------------------------------------- checked build

def debug_bounds():
    """llms_debug_bounds: (compiled_in, violations, first_address) of the loaded library."""
    c, v, a = C.c_uint32(0), C.c_uint32(0), C.c_uint64(0)
    _check(lib().llms_debug_bounds(C.byref(c), C.byref(v), C.byref(a)), "llms_debug_bounds")
    return int(c.value), int(v.value), int(a.value)


# ----------------------------------------------------------------------------- measurement aid

def stream_probe(src, dst, iters, read_kib, write_kib, stream=None, split=None):
    """llms_stream_probe: a plain stream of the given read:write mix (KiB per warp iteration) over src / dst.
    split (llms_stream_probe_split): 0 a warp per iteration, 1 resident CTAs with a fixed split, 2 resident CTAs that
    draw their iterations from counters."""
    if split is None:
        _check(lib().llms_stream_probe(_ptr(src), _nbytes(src), _ptr(dst), _nbytes(dst), int(iters), int(read_kib),
                                       int(write_kib), _stream(stream)), "llms_stream_probe")
    else:
        _check(lib().llms_stream_probe_split(_ptr(src), _nbytes(src), _ptr(dst), _nbytes(dst), int(iters), int(read_kib),
                                             int(write_kib), int(split), _stream(stream)), "llms_stream_probe_split")
