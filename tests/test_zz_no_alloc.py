"""llms_compress_chunks_static: the compress call for callers that have no device scratch to give.

Some users of this library run inside a serving process whose device memory was handed out completely at
start-up, or in a place where entering the CUDA allocator is off limits because it would stall the GPU; they
cannot provide the workspace that llms_compress_chunks asks for.  This entry point keeps its chunk table in an
array built into the library instead.  The test drives it through the C ABI twice in a row (the second call
finds the first call's leftovers in that array) and wants exactly the bytes the ordinary entry point produces.
This file is named so that pytest collects it after every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import binding as B, synth
from gpu_helpers import assert_meta_equal, bits_view, odesc

pytestmark = pytest.mark.gpu


def run_both(sh, kv_dev, ids, bits):
    d = B.desc_of(sh)
    n = len(ids)
    total = B.compressed_size(d, bits)
    ref = torch.full((total + 256,), 0x11, dtype=torch.uint8, device="cuda")
    got = torch.full((total + 256,), 0x22, dtype=torch.uint8, device="cuda")
    ref_meta, got_meta = B.new_meta(n, pinned=True), B.new_meta(n, pinned=True)
    ws = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    B.compress_chunks(d, kv_dev, ids, bits, ref, ref_meta, ws, out_bytes=total)
    B.compress_chunks_static(d, kv_dev, ids, bits, got, got_meta, out_bytes=total)
    torch.cuda.synchronize()
    assert torch.equal(got[:total], ref[:total])                 # packed records: bit-exact
    assert bool((got[total:] == 0x22).all())                     # nothing written past the end
    for f in B.META_DTYPE.names:
        assert np.array_equal(got_meta[f], ref_meta[f]), f       # offsets, sizes and checksums


def test_static_entry_matches_workspace_entry_twice_in_a_row():
    sh = synth.CONFIGS["tiny"]
    kv_dev = synth.kv_tensor(sh).cuda()
    # first call: the whole context, mixed widths
    run_both(sh, kv_dev, np.arange(sh.n_chunks, dtype=np.uint32), synth.random_bits(sh.n_chunks, 3).numpy())
    # second call right behind it: fewer chunks, other ids and widths - the old table and its checksums must not leak
    run_both(sh, kv_dev, np.array([9, 1, 14], dtype=np.uint32), np.array([2, 8, 4], dtype=np.uint8))
    # and a larger shape, many slabs per chunk
    big = synth.CONFIGS["llama7b"].with_(n_layers=2, n_tokens=1024)
    big_kv = synth.kv_tensor(big, device="cuda")
    bits = np.array([(8, 4, 2)[i % 3] for i in range(big.n_chunks)], dtype=np.uint8)
    run_both(big, big_kv, np.arange(big.n_chunks, dtype=np.uint32), bits)


def test_static_entry_against_the_oracle_without_taking_device_memory():
    """The records and meta of the no-scratch entry point equal the CPU oracle's, call after call, and the device's
    free memory does not move across the calls: whoever could not allocate before the call still has not had to."""
    sh = synth.CONFIGS["tiny"]
    kv = synth.kv_tensor(sh)
    kv_dev = kv.cuda()
    d = B.desc_of(sh)
    cases = [(np.arange(sh.n_chunks, dtype=np.uint32), synth.random_bits(sh.n_chunks, 5).numpy()),
             (np.array([3, 12, 0, 7], dtype=np.uint32), np.array([4, 4, 8, 2], dtype=np.uint8)),
             (np.arange(sh.n_chunks, dtype=np.uint32)[::-1].copy(), np.full(sh.n_chunks, 2, dtype=np.uint8))]
    # every buffer exists before the first measured call; the calls themselves get raw pointers only
    outs = [torch.zeros(B.compressed_size(d, bits), dtype=torch.uint8, device="cuda") for _, bits in cases]
    metas = [B.new_meta(len(ids), pinned=True) for ids, _ in cases]
    B.compress_chunks_static(d, kv_dev, cases[0][0], cases[0][1], outs[0], metas[0])   # first call: looks the array's address up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for (ids, bits), out, meta in zip(cases[1:], outs[1:], metas[1:]):
        B.compress_chunks_static(d, kv_dev, ids, bits, out, meta)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
    for (ids, bits), out, meta in zip(cases, outs, metas):
        want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), ids, bits)
        assert np.array_equal(out.cpu().numpy(), want_buf)
        assert_meta_equal(meta, want_meta)


def test_static_entry_rejects_more_chunks_than_its_table_holds():
    sh = synth.KVShape("many", 1, 1, 1, 16, 16 * (B.STATIC_MAX_CHUNKS + 1), 16, 16)
    d = B.desc_of(sh)
    n = B.STATIC_MAX_CHUNKS + 1
    kv_dev = torch.zeros(sh.n_elements, dtype=torch.float16, device="cuda")
    bits = np.full(n, 2, dtype=np.uint8)
    out = torch.full((B.compressed_size(d, bits),), 0x33, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.LlmsError) as e:
        B.compress_chunks_static(d, kv_dev, np.arange(n, dtype=np.uint32), bits, out, B.new_meta(n))
    assert e.value.status == B.ERR_BUF_TOO_SMALL
    torch.cuda.synchronize()
    assert bool((out == 0x33).all())                             # nothing was launched
    # exactly the maximum is accepted
    B.compress_chunks_static(d, kv_dev, np.arange(n - 1, dtype=np.uint32), bits[:-1], out, B.new_meta(n - 1, pinned=True))
    torch.cuda.synchronize()
