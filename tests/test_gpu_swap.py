"""Swap copies over pinned host memory on a side stream: byte equality, checksums, events, the bounded wait."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import binding as B, synth
from gpu_helpers import bits_view, first_mismatch, odesc

pytestmark = pytest.mark.gpu


def test_round_trip_through_pinned_memory_matches_oracle():
    sh = synth.CONFIGS["llama7b"].with_(n_layers=2, n_tokens=512)
    kv = synth.kv_tensor(sh)
    kv_dev = kv.cuda()
    n = sh.n_chunks
    ids = np.arange(n, dtype=np.uint32)
    bits = np.array([(8, 4, 2)[i % 3] for i in range(n)], dtype=np.uint8)
    d = B.desc_of(sh)
    total = B.compressed_size(d, bits)
    main, side = torch.cuda.current_stream(), torch.cuda.Stream()
    buf = torch.empty(total, dtype=torch.uint8, device="cuda")
    back = torch.zeros(total, dtype=torch.uint8, device="cuda")
    arena = torch.zeros(total, dtype=torch.uint8).pin_memory()
    meta = B.new_meta(n, pinned=True)
    ws = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    compressed, out_done, in_done = B.new_event(), B.new_event(), B.new_event()
    B.compress_chunks(d, kv_dev, ids, bits, buf, meta, ws)
    compressed.record(main)
    torch.cuda.synchronize()     # meta (sizes) is final; checksums too
    B.swap_out(buf, meta, arena, side_stream=side, after=compressed, done=out_done)
    B.swap_in(arena, meta, back, side_stream=side, done=in_done)
    main.wait_event(in_done)
    out = torch.zeros_like(kv_dev)
    B.decompress_chunks(d, back, meta, None, out, ws)
    B.wait(in_done, 10000)
    assert B.codec_corrupt_count(ws) == 0
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), ids, bits)
    assert first_mismatch(arena.numpy(), want_buf) is None
    for i in range(n):
        rec = arena.numpy()[int(meta[i]["offset"]):int(meta[i]["offset"] + meta[i]["nbytes"])]
        assert oracle.checksum(rec) == meta[i]["checksum"] == want_meta[i]["checksum"]
    want = np.zeros(kv.numel(), dtype=np.uint16).reshape(kv.shape)
    oracle.decompress_chunks(odesc(sh), want_buf, want_meta, want)
    assert first_mismatch(bits_view(out).reshape(-1), want.reshape(-1)) is None


def test_scattered_host_offsets():
    sh = synth.CONFIGS["tiny"]
    kv_dev = synth.kv_tensor(sh).cuda()
    ids = np.array([3, 4, 9], dtype=np.uint32)
    bits = np.array([8, 2, 4], dtype=np.uint8)
    d = B.desc_of(sh)
    total = B.compressed_size(d, bits)
    buf = torch.empty(total, dtype=torch.uint8, device="cuda")
    meta = B.new_meta(3, pinned=True)
    ws = torch.empty(B.codec_workspace_bytes(3), dtype=torch.uint8, device="cuda")
    B.compress_chunks(d, kv_dev, ids, bits, buf, meta, ws)
    torch.cuda.synchronize()
    arena = torch.full((65536,), 0x5A, dtype=torch.uint8).pin_memory()
    offs = np.array([40960, 0, 16384], dtype=np.uint64)
    side = torch.cuda.Stream()
    done = B.new_event()
    B.swap_out(buf, meta, arena, host_offsets=offs, side_stream=side, done=done)
    B.wait(done)
    host = buf.cpu().numpy()
    used = np.zeros(65536, dtype=bool)
    for i in range(3):
        o, nb, ho = int(meta[i]["offset"]), int(meta[i]["nbytes"]), int(offs[i])
        assert np.array_equal(arena.numpy()[ho:ho + nb], host[o:o + nb])
        used[ho:ho + nb] = True
    assert (arena.numpy()[~used] == 0x5A).all()
    back = torch.zeros(total, dtype=torch.uint8, device="cuda")
    B.swap_in(arena, meta, back, host_offsets=offs, side_stream=side, done=done)
    B.wait(done)
    assert torch.equal(back, buf)


def test_wait_times_out_and_then_succeeds():
    side = torch.cuda.Stream()
    ev = B.new_event(side)
    with torch.cuda.stream(side):
        torch.cuda._sleep(int(1.0e9))       # a bounded spin of about half a second
        ev.record(side)
    with pytest.raises(B.LlmsError) as e:
        B.wait(ev, 5)
    assert e.value.status == B.ERR_TIMEOUT
    B.wait(ev, 20000)


def test_codec_works_straight_on_mapped_pinned_memory():
    """Swap-out and swap-in without a staging buffer: the encoder writes its records straight into page-locked host
    memory (which the device reaches over the link) and the decoder reads them from there.  The ABI takes such
    pointers as they are; bytes, checksums and decoded values are the oracle's."""
    import oracle
    from gpu_helpers import assert_meta_equal, bits_view, first_mismatch, odesc
    sh = synth.CONFIGS["llama7b"].with_(n_layers=1, n_tokens=512)
    kv = synth.kv_tensor(sh)
    kv_dev = kv.cuda()
    d = B.desc_of(sh)
    n = sh.n_chunks
    ids = np.arange(n, dtype=np.uint32)
    bits = np.array([(8, 4, 2, 1)[i % 4] for i in range(n)], dtype=np.uint8)
    total = B.compressed_size(d, bits)
    arena = torch.full((total + 4096,), 0x5A, dtype=torch.uint8).pin_memory()
    meta = B.new_meta(n, pinned=True)
    ws = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    B.compress_chunks(d, kv_dev, ids, bits, arena, meta, ws, out_bytes=total)
    torch.cuda.synchronize()
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), ids, bits)
    assert first_mismatch(arena.numpy()[:total], want_buf) is None
    assert (arena.numpy()[total:] == 0x5A).all()
    assert_meta_equal(meta, want_meta)
    out = torch.zeros_like(kv_dev)
    B.decompress_chunks(d, arena, meta, None, out, ws, buf_bytes=total)
    assert B.codec_corrupt_count(ws) == 0
    want = np.zeros(kv.numel(), dtype=np.uint16).reshape(kv.shape)
    oracle.decompress_chunks(odesc(sh), want_buf, want_meta, want)
    assert first_mismatch(bits_view(out).reshape(-1), want.reshape(-1)) is None


def test_swap_argument_errors():
    meta = B.new_meta(1)
    meta[0]["nbytes"] = 100          # not a multiple of 256
    assert B.lib().llms_swap_out(4096, 1 << 20, meta.ctypes.data, 1, 8192, 1 << 20, None, None, None, None) == B.ERR_MISALIGNED
    assert B.lib().llms_swap_out(None, 1 << 20, meta.ctypes.data, 1, 8192, 1 << 20, None, None, None, None) == B.ERR_INVALID_ARG
    assert B.lib().llms_swap_in(4096, 0, None, meta.ctypes.data, 0, 8192, 0, None, None, None) == B.OK


def test_stream_probe_stays_inside_its_buffers():
    """The measurement aid: every supported mix runs under every work split, writes every one of its iters * write_kib
    KiB (each iteration stores its own number: a split that skipped an iteration would leave a hole) and nothing
    behind them, and refuses buffers that are too short or mixes it has no kernel for, before anything is launched."""
    src = torch.arange(1 << 20, dtype=torch.int32, device="cuda")              # 4 MiB
    for split in (None, 0, 1, 2):
        for rk, wk in ((4, 0), (0, 4), (4, 1), (1, 4), (2, 2)):
            iters = 1000 if split in (None, 0) else 20011                      # resident CTAs: several draws per warp
            if rk * iters * 1024 > src.numel() * 4:
                iters = src.numel() * 4 // (rk * 1024)
            dst = torch.full((iters * wk * 1024 + 4096,), 0x77, dtype=torch.uint8, device="cuda")
            B.stream_probe(src, dst, iters, rk, wk, split=split)
            torch.cuda.synchronize()
            assert bool((dst[iters * wk * 1024:] == 0x77).all())
            if wk:
                words = dst[:iters * wk * 1024].view(torch.int32).view(iters, wk * 256)
                want = torch.arange(iters, dtype=torch.int32, device="cuda")[:, None].expand(iters, wk * 256)
                assert torch.equal(words, want)
    dst = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    for args, status in (((src, dst, 3, 1, 4), B.ERR_BUF_TOO_SMALL), ((src, dst, 2000, 4, 0), B.ERR_BUF_TOO_SMALL),
                         ((src, dst, 2, 3, 1), B.ERR_UNSUPPORTED), ((src, dst, 0, 4, 1), B.ERR_INVALID_ARG)):
        with pytest.raises(B.LlmsError) as e:
            B.stream_probe(*args)
        assert e.value.status == status
    with pytest.raises(B.LlmsError) as e:
        B.stream_probe(src, dst, 1, 1, 4, split=3)
    assert e.value.status == B.ERR_INVALID_ARG
