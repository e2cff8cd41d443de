"""Shared plumbing of the GPU parity tests: run the library through its binding, run the oracle, compare."""
import numpy as np
import torch

import oracle
from paper_2403_11805_b200 import binding as B

CANARY = 0xA5


def odesc(sh, mode=0, n_tokens=None):
    return oracle.make_desc(sh.n_layers, sh.n_kv_heads, sh.n_q_heads, sh.head_dim,
                            sh.n_tokens if n_tokens is None else n_tokens, sh.chunk_len, sh.group_size, mode)


def bits_view(t):
    """uint16 numpy view of an fp16 tensor (copied to the host if needed)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def gpu_compress(sh, kv_dev, ids, bits, mode=0, stream=None):
    """-> (records uint8 numpy, meta numpy) after synchronising; also checks the canary behind the buffer."""
    d = B.desc_of(sh, mode)
    n = len(ids)
    total = B.compressed_size(d, bits)
    out = torch.full((total + 512,), CANARY, dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    ws = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    B.compress_chunks(d, kv_dev, ids, bits, out, meta, ws, stream=stream, out_bytes=total)
    torch.cuda.synchronize()
    host = out.cpu().numpy()
    assert (host[total:] == CANARY).all(), "wrote past the end of the swap buffer"
    return host[:total].copy(), meta.copy(), out


def gpu_decompress(sh, buf_dev, meta, kv_out_dev, dst_ids=None, mode=0):
    d = B.desc_of(sh, mode)
    ws = torch.empty(B.codec_workspace_bytes(len(meta)), dtype=torch.uint8, device="cuda")
    B.decompress_chunks(d, buf_dev, meta, dst_ids, kv_out_dev, ws)
    return B.codec_corrupt_count(ws)


def assert_meta_equal(got, want):
    for f in ("chunk_id", "bits", "offset", "nbytes", "n_groups", "checksum"):
        assert np.array_equal(got[f], want[f]), f


def first_mismatch(a, b):
    idx = np.flatnonzero(a != b)
    return None if idx.size == 0 else (int(idx[0]), int(a[idx[0]]), int(b[idx[0]]), int(idx.size))
