"""GPU parity of the chunk codec against the CPU oracle: packed records, scale/zero-point bits, meta and
checksums bit-exact; decoded values bit-exact (and inside the stated tolerance of 1e-3 of each group's range)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import binding as B, synth
from gpu_helpers import (CANARY, assert_meta_equal, bits_view, first_mismatch, gpu_compress, gpu_decompress, odesc)

pytestmark = pytest.mark.gpu


def check_compress(sh, kv_host, ids, bits):
    kv_dev = kv_host.cuda()
    got_buf, got_meta, buf_dev = gpu_compress(sh, kv_dev, ids, bits)
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv_host), ids, bits)
    assert first_mismatch(got_buf, want_buf) is None
    assert_meta_equal(got_meta, want_meta)
    return kv_dev, buf_dev, got_meta, want_buf


def check_decompress(sh, kv_host, buf_dev, meta, want_buf, dst_ids=None):
    out_dev = torch.full(kv_host.shape, float("nan"), dtype=torch.float16, device="cuda")
    assert gpu_decompress(sh, buf_dev, meta, out_dev, dst_ids) == 0
    want = np.full(kv_host.numel(), 0x7E00, dtype=np.uint16).reshape(kv_host.shape)
    oracle.decompress_chunks(odesc(sh), want_buf, meta, want, dst_ids)
    got = bits_view(out_dev)
    # NaN canaries: torch writes 0x7E00 for nan
    assert first_mismatch(got.reshape(-1), want.reshape(-1)) is None
    return out_dev


def group_range_tolerance_ok(sh, kv_host, out_dev, ids, tol=1e-3):
    """max-abs error relative to each group's range, for the 8-bit chunks (|err| <= scale/2 ~ range/510)."""
    x = kv_host.double()
    y = out_dev.cpu().double()
    CL, G = sh.chunk_len, sh.group_size
    for cid in ids:
        xs = x[..., cid * CL:(cid + 1) * CL, :].reshape(-1, G)
        ys = y[..., cid * CL:(cid + 1) * CL, :].reshape(-1, G)
        rng = (xs.max(1).values - xs.min(1).values).clamp_min(1e-30)
        # fp16 rounding of the decoded value adds up to half an ulp of the value itself
        slack = 2.0 ** -11 * xs.abs().max(1).values
        assert bool((((ys - xs).abs().max(1).values - slack) / rng <= 0.5 / 255 + tol).all())


def test_tiny_config_whole_context():
    sh = synth.CONFIGS["tiny"]
    kv = synth.kv_tensor(sh)
    ids = np.arange(sh.n_chunks)
    bits = synth.random_bits(sh.n_chunks, sh.seed).numpy()
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    out = check_decompress(sh, kv, buf_dev, meta, want_buf)
    group_range_tolerance_ok(sh, kv, out, ids[bits == 8])


def test_gemma2b_config_whole_context():
    sh = synth.CONFIGS["gemma2b"]
    kv = synth.kv_tensor(sh)
    ids = np.arange(sh.n_chunks)
    bits = np.array([8] * 43 + [4] * 42 + [2] * 43, dtype=np.uint8)[np.random.default_rng(0).permutation(128)]
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    check_decompress(sh, kv, buf_dev, meta, want_buf)


@pytest.mark.parametrize("name,layers", [("llama7b", 2), ("mistral7b_32k", 1), ("multiapp", 1)])
def test_model_shaped_slices(name, layers):
    # the 7B shapes with fewer layers and tokens: still thousands of slabs per chunk, many chunks
    sh = synth.CONFIGS[name].with_(n_layers=layers, n_tokens=min(synth.CONFIGS[name].n_tokens, 1024))
    kv = synth.kv_tensor(sh)
    rng = np.random.default_rng(1)
    ids = rng.permutation(sh.n_chunks)[: max(3, sh.n_chunks // 2)]
    bits = rng.choice([8, 4, 2], len(ids)).astype(np.uint8)
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    check_decompress(sh, kv, buf_dev, meta, want_buf)


@pytest.mark.parametrize("G", [16, 32, 64, 128, 256, 512])
def test_every_group_size_and_ragged_shapes(G):
    # chunk_len 5 and 24 with head_dim G or 2G: slabs that are not a multiple of a warp pass, tail tokens
    for CL, mult, T in ((5, 1, 23), (24, 2, 100)):
        d = G * mult
        if d > 1024:
            continue
        sh = synth.KVShape(f"g{G}", 2, 3, 3, d, T, CL, G, seed=G + CL)
        kv = synth.kv_tensor(sh)
        ids = np.arange(sh.n_chunks)[::-1].copy()
        bits = np.array([(8, 4, 2)[i % 3] for i in range(sh.n_chunks)], dtype=np.uint8)
        kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
        check_decompress(sh, kv, buf_dev, meta, want_buf)


@pytest.mark.parametrize("CL,d,G,L,H", [
    (1, 64, 64, 1, 1),       # slab of 64 elements, 2 slabs per chunk: one unit, mostly empty
    (1, 128, 32, 3, 5),      # 30 slabs of 128: 1.9 units per chunk, ragged last unit, four groups per slab
    (2, 128, 128, 2, 3),     # slabs of 256
    (4, 128, 64, 2, 5),      # slabs of 512: one load instruction per slab
    (8, 128, 128, 3, 3),     # slabs of 1024: 18 slabs = 9 units
    (16, 64, 16, 1, 3),      # head_dim 64 at the paper's chunk size, groups inside a lane
    (4, 256, 256, 1, 3),     # slabs of 1024 from a wide head
])
def test_slabs_shorter_than_a_warp_pass(CL, d, G, L, H):
    """Short slabs are packed several to a unit; KV addresses then change slab inside a unit."""
    sh = synth.KVShape("short", L, H, H, d, CL * 11 + (CL - 1), CL, G, seed=CL + d + G)   # tail tokens unless CL == 1
    kv = synth.kv_tensor(sh)
    rng = np.random.default_rng(CL * d)
    ids = rng.permutation(sh.n_chunks)[:9].astype(np.uint32)
    bits = np.array([(2, 8, 4)[i % 3] for i in range(len(ids))], dtype=np.uint8)
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    check_decompress(sh, kv, buf_dev, meta, want_buf)
    check_decompress(sh, kv, buf_dev, meta, want_buf, dst_ids=np.arange(2, 11, dtype=np.uint32))


@pytest.mark.parametrize("shape", [
    ("tiny", None),
    ("g128", (2, 3, 3, 128, 100, 16, 128)),     # whole passes
    ("ragged", (2, 3, 3, 96, 50, 24, 32)),      # slab of 2304 elements: ragged second pass
    ("odd", (1, 1, 1, 16, 25, 5, 16)),          # slab of 80 elements: 10-byte code runs, pieces on either half of a word
    ("short", (2, 5, 5, 128, 40, 4, 64)),       # packed units
])
def test_one_bit_level(shape):
    """Level set {4, 2, 1} (Sec. 3.2): records with 1-bit chunks among the others, bit for bit against the oracle."""
    name, dims = shape
    sh = synth.CONFIGS["tiny"] if dims is None else synth.KVShape(name, *dims, seed=17)
    kv = synth.kv_tensor(sh)
    ids = np.arange(sh.n_chunks)
    bits = np.array([(1, 4, 2, 1, 8)[i % 5] for i in range(sh.n_chunks)], dtype=np.uint8)
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    out = check_decompress(sh, kv, buf_dev, meta, want_buf)
    # a 1-bit group decodes to its minimum or (to fp16 accuracy) its maximum
    x, y = kv.double(), out.cpu().double()
    CL, G = sh.chunk_len, sh.group_size
    for cid in ids[bits == 1][:3]:
        xs = x[..., cid * CL:(cid + 1) * CL, :].reshape(-1, G)
        ys = y[..., cid * CL:(cid + 1) * CL, :].reshape(-1, G)
        lo, hi = xs.min(1, keepdim=True).values, xs.max(1, keepdim=True).values
        tol = 2.0 ** -10 * torch.maximum(hi.abs(), hi - lo) + 1e-12
        assert bool((((ys - lo).abs() <= 1e-12) | ((ys - hi).abs() <= tol)).all())
    bits1 = np.ones(sh.n_chunks, dtype=np.uint8)
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits1)
    check_decompress(sh, kv, buf_dev, meta, want_buf)


def test_one_bit_special_values():
    sh = synth.KVShape("special1", 1, 2, 2, 64, 64, 16, 64, seed=9)
    kv = synth.kv_tensor(sh)
    kv[0, 0, 0, 0:16] = 2.5                        # constant: scale 0
    kv[0, 0, 0, 17, :] = torch.linspace(-6e-7, 6e-7, 64).half()   # subnormal scale: the clamped path
    kv[0, 0, 0, 18, 0] = 65504.0                   # range 125504 is beyond fp16: the scale saturates at 65504
    kv[0, 0, 0, 18, 1] = -60000.0
    kv[0, 0, 0, 19, :] = torch.tensor([0.0, 1.0, 0.5, 0.25] * 16).half()      # the tie at one half goes to 0
    ids = np.arange(sh.n_chunks)
    bits = np.ones(sh.n_chunks, dtype=np.uint8)
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    check_decompress(sh, kv, buf_dev, meta, want_buf)


def test_more_chunks_in_a_launch_than_checksum_slots():
    """Above 1024 chunks of one bit-width a launch adds its checksums straight to global memory."""
    sh = synth.KVShape("many", 1, 2, 2, 64, 2 * 1300, 2, 64, seed=23)      # 1300 chunks of 2 tokens
    kv = synth.kv_tensor(sh)
    ids = np.arange(sh.n_chunks)
    bits = np.full(sh.n_chunks, 4, dtype=np.uint8)
    bits[::50] = 8
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    check_decompress(sh, kv, buf_dev, meta, want_buf)


def test_padding_is_written_and_compared():
    # 2 slabs * 3 tokens * 1 group = 6 groups -> 24 parameter bytes -> 8 zero bytes before the codes,
    # and 144/288 code bytes -> tail padding up to 256/512
    sh = synth.KVShape("pad", 1, 1, 1, 16, 9, 3, 16, seed=3)
    kv = synth.kv_tensor(sh)
    for bits in ([8, 8, 8], [2, 4, 8]):
        check_compress(sh, kv, np.arange(3), np.array(bits, dtype=np.uint8))


def test_special_values():
    sh = synth.KVShape("special", 1, 2, 2, 64, 64, 16, 64, seed=9)
    kv = synth.kv_tensor(sh)
    kv[0, 0, 0, 0:16] = 2.5                        # constant chunk slab: scale 0, reproduced exactly
    kv[0, 0, 0, 16, :32] = -0.0                    # -0 / +0 mix, all zero
    kv[0, 0, 0, 16, 32:] = 0.0
    kv[0, 0, 0, 17, :] = torch.linspace(-6e-7, 6e-7, 64).half()   # subnormal values and a subnormal scale
    kv[0, 0, 0, 18, 0] = 65504.0                   # full fp16 range: decode saturates
    kv[0, 0, 0, 18, 1] = -65504.0
    kv[0, 0, 0, 19, :] = torch.arange(64).half() * 0.5 - 8.0     # exact ties in the quantizer
    kv[0, 1, 1, 20, 5] = -0.0
    ids = np.arange(sh.n_chunks)
    for b in (8, 4, 2):
        bits = np.full(sh.n_chunks, b, dtype=np.uint8)
        kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
        out = check_decompress(sh, kv, buf_dev, meta, want_buf)
        assert torch.equal(out[0, 0, 0, 0:16].cpu(), kv[0, 0, 0, 0:16])
        assert bool(torch.isfinite(out.float()).all())


def test_subset_shuffled_ids_and_other_destination_slots():
    sh = synth.CONFIGS["tiny"]
    kv = synth.kv_tensor(sh)
    ids = np.array([11, 2, 7, 0, 15], dtype=np.uint32)
    bits = np.array([4, 8, 2, 2, 8], dtype=np.uint8)
    kv_dev, buf_dev, meta, want_buf = check_compress(sh, kv, ids, bits)
    check_decompress(sh, kv, buf_dev, meta, want_buf)                       # untouched chunks keep the canary
    check_decompress(sh, kv, buf_dev, meta, want_buf, dst_ids=np.array([0, 1, 2, 3, 4], dtype=np.uint32))


def test_empty_list_is_a_no_op():
    sh = synth.CONFIGS["tiny"]
    d = B.desc_of(sh)
    kv_dev = synth.kv_tensor(sh).cuda()
    out = torch.full((1024,), CANARY, dtype=torch.uint8, device="cuda")
    ws = torch.empty(64, dtype=torch.uint8, device="cuda")
    B.compress_chunks(d, kv_dev, np.zeros(0, np.uint32), np.zeros(0, np.uint8), out, B.new_meta(0), ws)
    B.decompress_chunks(d, out, B.new_meta(0), None, kv_dev, ws)
    torch.cuda.synchronize()
    assert bool((out == CANARY).all())


def test_corrupted_record_is_reported():
    sh = synth.CONFIGS["tiny"]
    kv = synth.kv_tensor(sh)
    ids = np.arange(4, dtype=np.uint32)
    bits = np.array([8, 4, 2, 8], dtype=np.uint8)
    _, meta, buf_dev = gpu_compress(sh, kv.cuda(), ids, bits)
    out = torch.zeros_like(kv, device="cuda")
    assert gpu_decompress(sh, buf_dev, meta, out) == 0
    buf_dev[int(meta[2]["offset"]) + 700] ^= 0x10                          # one flipped bit in record 2
    assert gpu_decompress(sh, buf_dev, meta, out) == 1
    d = B.desc_of(sh)
    ws = torch.empty(B.codec_workspace_bytes(4), dtype=torch.uint8, device="cuda")
    B.decompress_chunks(d, buf_dev, meta, None, out, ws)
    assert B.lib().llms_codec_corrupt_count(ws.data_ptr(), None, torch.cuda.current_stream().cuda_stream) == B.ERR_CORRUPT


def test_pinned_meta_gives_stream_ordered_checksums():
    """llms_decompress_chunks_ordered: the expected checksums are read from the pinned meta by the device when the
    check runs, so the decode call may follow the encode call on the same stream with no synchronisation in between."""
    sh = synth.CONFIGS["gemma2b"].with_(n_layers=4)
    kv = synth.kv_tensor(sh)
    kv_dev = kv.cuda()
    d = B.desc_of(sh)
    n = sh.n_chunks
    ids = np.arange(n, dtype=np.uint32)
    bits = np.array([(8, 4, 2, 1)[i % 4] for i in range(n)], dtype=np.uint8)
    buf = torch.empty(B.compressed_size(d, bits), dtype=torch.uint8, device="cuda")
    ws_c = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    ws_d = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    out = torch.full(kv.shape, float("nan"), dtype=torch.float16, device="cuda")
    for _ in range(3):                                   # checksums of the call before never stand in: meta is zeroed
        meta["checksum"] = 0
        B.compress_chunks(d, kv_dev, ids, bits, buf, meta, ws_c)
        B.decompress_chunks_ordered(d, buf, meta, None, out, ws_d)     # no synchronisation: the checksums are still on their way
        assert B.codec_corrupt_count(ws_d) == 0
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), ids, bits)
    assert_meta_equal(meta, want_meta)
    want = np.zeros(kv.numel(), dtype=np.uint16).reshape(kv.shape)
    oracle.decompress_chunks(odesc(sh), want_buf, want_meta, want)
    assert first_mismatch(bits_view(out).reshape(-1), want.reshape(-1)) is None
    # a wrong expectation in the pinned array is reported, and so is a damaged record
    meta["checksum"][5] ^= 1
    B.decompress_chunks_ordered(d, buf, meta, None, out, ws_d)
    assert B.codec_corrupt_count(ws_d) == 1
    meta["checksum"][5] ^= 1
    buf[int(meta[7]["offset"]) + 1000] ^= 0x04
    B.decompress_chunks_ordered(d, buf, meta, None, out, ws_d)
    assert B.codec_corrupt_count(ws_d) == 1
    with pytest.raises(B.LlmsError) as e:                # pageable meta is refused: the device could not read it
        B.decompress_chunks_ordered(d, buf, meta.copy(), None, out, ws_d)
    assert e.value.status == B.ERR_INVALID_ARG


@pytest.mark.parametrize("layers", [1, 2])
def test_back_to_back_encode_calls_share_one_pinned_meta(layers):
    """Encode calls that follow each other on a stream with no synchronisation may all name the same pinned meta
    array: while the host prepares call k+1 the device is still storing call k's checksums into it.  Every call's
    sums must start from zero all the same.  (Launches about as long as the host's part of a call, so that the
    device's stores fall into the host's preparation of the next call.)"""
    sh = synth.CONFIGS["llama7b"].with_(n_layers=layers)
    kv = synth.kv_tensor(sh)
    kv_dev = kv.cuda()
    d = B.desc_of(sh)
    ids = np.arange(0, sh.n_chunks, 3, dtype=np.uint32)
    n = len(ids)
    out = torch.empty(kv.shape, dtype=torch.float16, device="cuda")
    for b in (8, 2):
        bits = np.full(n, b, dtype=np.uint8)
        buf = torch.empty(B.compressed_size(d, bits), dtype=torch.uint8, device="cuda")
        ws_c = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
        ws_d = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
        meta = B.new_meta(n, pinned=True)
        want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), ids, bits)
        for _ in range(10):
            for _ in range(20):
                B.compress_chunks(d, kv_dev, ids, bits, buf, meta, ws_c)
            B.decompress_chunks_ordered(d, buf, meta, None, out, ws_d)
            assert B.codec_corrupt_count(ws_d) == 0      # synchronises
            assert_meta_equal(meta, want_meta)
        assert first_mismatch(buf.cpu().numpy(), want_buf) is None


def test_pageable_meta_takes_the_copy_path():
    """Checksums reach a pageable meta array by a device-to-host copy (into pinned memory a kernel stores them)."""
    sh = synth.CONFIGS["tiny"]
    kv = synth.kv_tensor(sh)
    d = B.desc_of(sh)
    ids = np.arange(sh.n_chunks, dtype=np.uint32)
    bits = synth.random_bits(sh.n_chunks, 4).numpy()
    buf = torch.empty(B.compressed_size(d, bits), dtype=torch.uint8, device="cuda")
    ws = torch.empty(B.codec_workspace_bytes(len(ids)), dtype=torch.uint8, device="cuda")
    meta = B.new_meta(len(ids), pinned=False)
    B.compress_chunks(d, kv.cuda(), ids, bits, buf, meta, ws)
    torch.cuda.synchronize()
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), ids, bits)
    assert first_mismatch(buf.cpu().numpy(), want_buf) is None
    assert_meta_equal(meta, want_meta)


def test_recompression_is_stable():
    # decode(encode(x)) encoded again at the same width gives the same codes whenever the scale is unchanged
    sh = synth.CONFIGS["tiny"]
    kv = synth.kv_tensor(sh)
    ids = np.arange(sh.n_chunks, dtype=np.uint32)
    for b in (8, 4, 2):
        bits = np.full(sh.n_chunks, b, dtype=np.uint8)
        buf1, meta1, buf_dev = gpu_compress(sh, kv.cuda(), ids, bits)
        out = torch.zeros_like(kv, device="cuda")
        gpu_decompress(sh, buf_dev, meta1, out)
        buf2, meta2, _ = gpu_compress(sh, out, ids, bits)
        co, nb = B.record_layout(B.desc_of(sh), b)
        r1, r2 = buf1.reshape(sh.n_chunks, nb), buf2.reshape(sh.n_chunks, nb)
        ng = int(meta1[0]["n_groups"])
        p1, p2 = r1[:, :4 * ng].view("<u2").reshape(-1, 2), r2[:, :4 * ng].view("<u2").reshape(-1, 2)
        same_scale = p1[:, 0] == p2[:, 0]
        assert same_scale.mean() > 0.9
        per = sh.group_size * b // 8
        c1, c2 = r1[:, co:co + ng * per].reshape(-1, per), r2[:, co:co + ng * per].reshape(-1, per)
        assert (c1[same_scale] == c2[same_scale]).all()


@pytest.mark.parametrize("name", ["llama7b", "mistral7b_32k"])
def test_full_size_sampled_chunks(name):
    """The benchmark's launch configuration: the whole context on the device, every chunk compressed by
    tertile-like bit mix; a few chunks (one per bit-width, first/last included) are checked against the oracle
    completely, the rest through their checksums on the way back in."""
    sh = synth.CONFIGS[name]
    kv_dev = synth.kv_tensor(sh, device="cuda")
    n = sh.n_chunks
    f8, f4, _ = sh.frac
    n8, n84 = int(np.floor(f8 * n + 0.5)), int(np.floor((f8 + f4) * n + 0.5))
    bits = np.array([8] * n8 + [4] * (n84 - n8) + [2] * (n - n84), dtype=np.uint8)[np.random.default_rng(2).permutation(n)]
    ids = np.arange(n, dtype=np.uint32)
    d = B.desc_of(sh)
    total = B.compressed_size(d, bits)
    buf = torch.empty(total, dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    ws = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    B.compress_chunks(d, kv_dev, ids, bits, buf, meta, ws)
    torch.cuda.synchronize()
    CL = sh.chunk_len
    one = sh.with_(n_tokens=CL)                       # a one-chunk context holding the sampled chunk
    picks = {0, n - 1}
    for b in (8, 4, 2):
        picks.add(int(np.flatnonzero(bits == b)[len(np.flatnonzero(bits == b)) // 2]))
    for cid in sorted(picks):
        chunk = kv_dev[..., cid * CL:(cid + 1) * CL, :].contiguous().cpu()
        want_buf, want_meta = oracle.compress_chunks(odesc(one), bits_view(chunk), [0], [bits[cid]])
        m = meta[cid]
        got = buf[int(m["offset"]):int(m["offset"] + m["nbytes"])].cpu().numpy()
        assert first_mismatch(got, want_buf) is None, cid
        assert (m["checksum"], m["nbytes"], m["n_groups"], m["bits"]) == \
               (want_meta[0]["checksum"], want_meta[0]["nbytes"], want_meta[0]["n_groups"], bits[cid])
    # offsets are the running sum of the record sizes
    assert np.array_equal(meta["offset"], np.concatenate([[0], np.cumsum(meta["nbytes"])[:-1]]))
    out = torch.empty_like(kv_dev)
    B.decompress_chunks(d, buf, meta, None, out, ws)
    assert B.codec_corrupt_count(ws) == 0
    for cid in sorted(picks):
        chunk_out = out[..., cid * CL:(cid + 1) * CL, :].contiguous().cpu()
        m = meta[cid:cid + 1].copy()
        m["offset"] = 0
        m["chunk_id"] = 0
        rec = buf[int(meta[cid]["offset"]):int(meta[cid]["offset"] + meta[cid]["nbytes"])].cpu().numpy()
        want = np.zeros(chunk_out.numel(), dtype=np.uint16).reshape(chunk_out.shape)
        oracle.decompress_chunks(odesc(one), rec, m, want)
        assert first_mismatch(bits_view(chunk_out).reshape(-1), want.reshape(-1)) is None, cid
    # property that holds at any size: every decoded value lies inside its group's [min, max] (fp16 rounding aside)
    G = sh.group_size
    for l in range(0, sh.n_layers, 8):
        x = kv_dev[l].float().view(-1, G)
        y = out[l].float().view(-1, G)
        lo, hi = x.min(1, keepdim=True).values, x.max(1, keepdim=True).values
        tol = (hi - lo) * 2.0 ** -9 + 1e-7
        assert bool(((y >= lo - tol) & (y <= hi + tol)).all())
        err8 = ((y - x).abs().max(1).values / (hi - lo).squeeze(1).clamp_min(1e-20))
        chunk_bits = torch.from_numpy(bits.astype(np.int64)).cuda()
        # rows of x are (s, h, t, group): map the token to its chunk
        t_idx = torch.arange(x.shape[0], device="cuda") // (sh.head_dim // G) % sh.n_tokens
        qmax = (2 ** chunk_bits[t_idx // CL] - 1).float()
        assert bool((err8 <= 0.5 / qmax * (1 + 2.0 ** -8) + 2.0 ** -10 * x.abs().max(1).values / (hi - lo).squeeze(1).clamp_min(1e-20)).all())


# ----------------------------------------------------------------- channel-wise mode (quant_mode 1)

CW_SHAPES = [
    synth.CONFIGS["tiny"],                                                        # d 64: 4 lanes per column
    synth.CONFIGS["llama7b"].with_(n_layers=1, n_tokens=256),                     # d 128
    synth.CONFIGS["gemma2b"].with_(n_layers=2, n_tokens=160),                     # d 256, MQA
    synth.CONFIGS["multiapp"].with_(n_layers=1, n_kv_heads=4, n_q_heads=4, n_tokens=128),   # chunk_len 32
    synth.KVShape("cw_ragged", 2, 3, 3, 64, 53, 5, 64, seed=21),                  # chunk_len 5, tail tokens
    synth.KVShape("cw_one_token", 1, 2, 2, 64, 4, 1, 64, seed=22),                # fewer tokens than lanes per column
    synth.KVShape("cw_24", 1, 2, 2, 128, 100, 24, 128, seed=23),
]


@pytest.mark.parametrize("sh", CW_SHAPES, ids=[s.name for s in CW_SHAPES])
def test_channel_wise_mode_matches_oracle(sh):
    kv = synth.kv_tensor(sh)
    rng = np.random.default_rng(5)
    ids = rng.permutation(sh.n_chunks).astype(np.uint32)
    bits = np.array([(8, 4, 2, 1)[i % 4] for i in range(sh.n_chunks)], dtype=np.uint8)
    got_buf, got_meta, buf_dev = gpu_compress(sh, kv.cuda(), ids, bits, mode=1)
    want_buf, want_meta = oracle.compress_chunks(odesc(sh, 1), bits_view(kv), ids, bits)
    assert first_mismatch(got_buf, want_buf) is None
    assert_meta_equal(got_meta, want_meta)
    out_dev = torch.full(kv.shape, float("nan"), dtype=torch.float16, device="cuda")
    assert gpu_decompress(sh, buf_dev, got_meta, out_dev, mode=1) == 0
    want = np.full(kv.numel(), 0x7E00, dtype=np.uint16).reshape(kv.shape)
    oracle.decompress_chunks(odesc(sh, 1), want_buf, want_meta, want)
    assert first_mismatch(bits_view(out_dev).reshape(-1), want.reshape(-1)) is None


def test_channel_wise_special_values_and_outliers():
    sh = synth.KVShape("cw_special", 1, 2, 2, 64, 64, 16, 64, seed=9)
    kv = synth.kv_tensor(sh)
    kv[0, 0, 0, 0:16, 3] = 2.5                       # a constant channel: scale 0, reproduced exactly
    kv[0, 0, 0, 0:16, 4] = torch.tensor([-0.0, 0.0] * 8).half()
    kv[0, 0, 0, 0:16, 5] = torch.linspace(-6e-7, 6e-7, 16).half()   # subnormal scale: the clamped path
    kv[0, 0, 0, 0, 6] = 65504.0
    kv[0, 0, 0, 1, 6] = -65504.0                     # decode saturates
    ids = np.arange(sh.n_chunks, dtype=np.uint32)
    for b in (8, 4, 2, 1):
        bits = np.full(sh.n_chunks, b, dtype=np.uint8)
        got_buf, got_meta, buf_dev = gpu_compress(sh, kv.cuda(), ids, bits, mode=1)
        want_buf, want_meta = oracle.compress_chunks(odesc(sh, 1), bits_view(kv), ids, bits)
        assert first_mismatch(got_buf, want_buf) is None
        assert_meta_equal(got_meta, want_meta)
        out_dev = torch.zeros_like(kv, device="cuda")
        assert gpu_decompress(sh, buf_dev, got_meta, out_dev, mode=1) == 0
        want = np.zeros(kv.numel(), dtype=np.uint16).reshape(kv.shape)
        oracle.decompress_chunks(odesc(sh, 1), want_buf, want_meta, want)
        assert first_mismatch(bits_view(out_dev).reshape(-1), want.reshape(-1)) is None
        assert torch.equal(out_dev[0, 0, 0, 0:16, 3].cpu(), kv[0, 0, 0, 0:16, 3])
        assert bool(torch.isfinite(out_dev.float()).all())


def test_channel_wise_outlier_channels_cost_less_error_than_token_groups():
    # the two 10x outlier channels of K stretch every token group's range; channel-wise groups isolate them
    sh = synth.CONFIGS["llama7b"].with_(n_layers=1, n_tokens=256)
    kv = synth.kv_tensor(sh)
    ids = np.arange(sh.n_chunks, dtype=np.uint32)
    bits = np.full(sh.n_chunks, 4, dtype=np.uint8)
    err = {}
    for mode in (0, 1):
        _, meta, buf_dev = gpu_compress(sh, kv.cuda(), ids, bits, mode=mode)
        out_dev = torch.zeros_like(kv, device="cuda")
        assert gpu_decompress(sh, buf_dev, meta, out_dev, mode=mode) == 0
        err[mode] = float((out_dev.cpu().float() - kv.float())[:, 0].pow(2).mean())     # K half
    assert err[1] < err[0]
