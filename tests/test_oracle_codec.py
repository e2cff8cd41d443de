"""Pins for the CPU oracle's codec: fp16 conversion, group quantizer, bit packer, record layout.

Nothing here compares the oracle with itself: expected values are worked by hand in the comments,
come from numpy's independent fp16 conversion, from closed forms, or from invariants.
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2403_11805_b200 import synth
from conftest import read_golden


def h(x):
    """fp16 bit patterns of a list of Python floats (numpy's conversion, independent of the oracle's)."""
    return np.asarray(x, dtype=np.float64).astype(np.float16).view(np.uint16)


def hval(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


# ----------------------------------------------------------------- fp16 <-> fp32

def test_f16_to_f32_matches_numpy_for_every_half():
    halves = np.arange(65536, dtype=np.uint16)
    ref = halves.view(np.float16).astype(np.float32).view(np.uint32)
    for hb in range(65536):
        got = np.float32(oracle.f16_to_f32(hb)).view(np.uint32)
        if (hb & 0x7c00) == 0x7c00 and (hb & 0x3ff):
            assert (got & 0x7f800000) == 0x7f800000 and (got & 0x7fffff)  # NaN stays NaN
        else:
            assert got == ref[hb], hex(hb)


def test_f32_to_f16_ties_subnormals_overflow():
    cases = [
        (1.0 + 2.0 ** -11, 0x3C00),          # tie between 0x3C00 and 0x3C01 -> even
        (1.0 + 3 * 2.0 ** -11, 0x3C02),      # tie between 0x3C01 and 0x3C02 -> even
        (1.0 + 2.0 ** -11 + 2.0 ** -20, 0x3C01),
        (65504.0, 0x7BFF), (65519.99, 0x7BFF), (65520.0, 0x7C00), (1e9, 0x7C00), (-65520.0, 0xFC00),
        (2.0 ** -24, 0x0001), (2.0 ** -25, 0x0000),            # half of the smallest subnormal: tie -> 0
        (2.0 ** -25 * (1 + 2.0 ** -20), 0x0001), (3 * 2.0 ** -25, 0x0002),  # tie between 1 and 2 units -> 2
        (2.0 ** -14, 0x0400), (2.0 ** -14 - 2.0 ** -25, 0x0400),  # just under the smallest normal: tie -> even (0x400)
        (1023.5 * 2.0 ** -24, 0x0400), (1022.5 * 2.0 ** -24, 0x03FE),
        (0.0, 0x0000), (-0.0, 0x8000), (1e-30, 0x0000), (-1e-30, 0x8000),
    ]
    for f, want in cases:
        assert oracle.f32_to_f16(f) == want, (f, hex(want), hex(oracle.f32_to_f16(f)))


def test_f32_to_f16_matches_numpy_on_random_floats():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(30000) * 10.0 ** rng.integers(-9, 6, 30000)).astype(np.float32)
    # and floats sitting exactly on, and one ulp around, every rounding boundary between positive halves
    mids = ((np.arange(1, 0x7BFF, 37, dtype=np.uint16).view(np.float16).astype(np.float64)
             + np.arange(2, 0x7C00, 37, dtype=np.uint16).view(np.float16).astype(np.float64)) / 2).astype(np.float32)
    x = np.concatenate([x, mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(1e9))])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    got = oracle.f32_array_to_f16_bits(x)
    assert np.array_equal(got, ref)


# ----------------------------------------------------------------- hand-worked groups

def test_group_b2_exact_grid():
    # x = [0,1,2,3], b = 2: range 3, scale = 3/3 = 1.0 (0x3C00), zero = 0; codes 0,1,2,3;
    # byte = 0 | 1<<2 | 2<<4 | 3<<6 = 0xE4; every value decodes exactly.
    sc, ze, codes = oracle.quantize_group(h([0, 1, 2, 3]), 2)
    assert (sc, ze) == (0x3C00, 0x0000)
    assert codes.tolist() == [0, 1, 2, 3]
    assert oracle.pack_codes(codes, 2).tolist() == [0xE4]
    assert [oracle.dequantize_one(sc, ze, q) for q in codes] == h([0, 1, 2, 3]).tolist()


def test_group_b2_half_to_even():
    # x = [0, 0.5, 1.5, 3], scale 1: 0.5 -> 0 and 1.5 -> 2 (ties to even); byte = 2<<4 | 3<<6 = 0xE0.
    sc, ze, codes = oracle.quantize_group(h([0, 0.5, 1.5, 3]), 2)
    assert (sc, ze) == (0x3C00, 0x0000)
    assert codes.tolist() == [0, 0, 2, 3]
    assert oracle.pack_codes(codes, 2).tolist() == [0xE0]


def test_group_b4_negative_zero_point():
    # x = [-1.5, 0, 1.5, 6], b = 4: range 7.5, scale = 7.5/15 = 0.5 (0x3800), zero = -1.5 (0xBE00);
    # (x + 1.5) * 2 = 0,3,6,15; bytes 0|3<<4 = 0x30, 6|15<<4 = 0xF6; decode -1.5 + q/2 is exact.
    sc, ze, codes = oracle.quantize_group(h([-1.5, 0, 1.5, 6]), 4)
    assert (sc, ze) == (0x3800, 0xBE00)
    assert codes.tolist() == [0, 3, 6, 15]
    assert oracle.pack_codes(codes, 4).tolist() == [0x30, 0xF6]
    assert [oracle.dequantize_one(sc, ze, q) for q in codes] == h([-1.5, 0, 1.5, 6]).tolist()


def test_group_b2_inexact_scale_and_decode_tie():
    # x = fp16([0, 1, 0.3, 0.7]) = [0, 1, 0x34CD = 0.300048828125, 0x399A = 0.7001953125], b = 2.
    # scale = fp16(1/3): 1/3 = 1.0101010101|0101.. * 2^-2 -> round down -> 0x3555 = 1365/4096.
    # 1/scale = 3.00073..; codes: 0.30005*3.0007 = 0.90 -> 1; 0.70020*3.0007 = 2.10 -> 2; 1*3.0007 -> 3.
    # byte = 0 | 3<<2 | 1<<4 | 2<<6 = 0x9C.
    # decode q=3: 3*1365/4096 = 1 - 2^-12, halfway between 0x3BFF and 0x3C00 -> even -> 0x3C00.
    x = h([0, 1, 0.3, 0.7])
    assert x.tolist() == [0x0000, 0x3C00, 0x34CD, 0x399A]
    sc, ze, codes = oracle.quantize_group(x, 2)
    assert (sc, ze) == (0x3555, 0x0000)
    assert codes.tolist() == [0, 3, 1, 2]
    assert oracle.pack_codes(codes, 2).tolist() == [0x9C]
    assert [oracle.dequantize_one(sc, ze, q) for q in codes] == [0x0000, 0x3C00, 0x3555, 0x3955]


def test_group_b8_ties():
    # x = [0, 25.5, 255, 127.5], b = 8: scale = 255/255 = 1; 25.5 -> 26 and 127.5 -> 128 (ties to even).
    sc, ze, codes = oracle.quantize_group(h([0, 25.5, 255, 127.5]), 8)
    assert (sc, ze) == (0x3C00, 0x0000)
    assert codes.tolist() == [0, 26, 255, 128]
    assert oracle.pack_codes(codes, 8).tolist() == [0, 26, 255, 128]


def test_group_negative_zero_minimum_is_stored_as_plus_zero():
    for x in ([-0.0, 0.0, 1.0, 0.5], [0.0, -0.0, 1.0, 0.5]):
        sc, ze, codes = oracle.quantize_group(h(x), 2)
        assert (sc, ze) == (0x3555, 0x0000)
        assert codes.tolist() == [0, 0, 3, 2]  # 0.5 * 3.0007 = 1.50037 -> 2


def test_constant_group_is_reproduced_exactly():
    for b in (2, 4, 8):
        for v in (2.5, -7.0, 0.0, 6.1e-5, 65504.0):
            x = h([v] * 16)
            sc, ze, codes = oracle.quantize_group(x, b)
            assert sc == 0 and ze == x[0] and not codes.any()
            assert oracle.dequantize_one(sc, ze, 0) == x[0]


def test_decode_saturates_instead_of_overflowing():
    # min -65504, max 65504, b = 8: scale = fp16(131008/255 = 513.76) = 514; 255*514 - 65504 = 65566 > 65520
    # would round to +inf in fp16: finite input must decode to a finite value, so it saturates at 65504.
    sc, ze, codes = oracle.quantize_group(h([-65504.0, 65504.0, 0.0, 1.0]), 8)
    assert hval([sc])[0] == 514.0 and codes[1] == 255
    assert oracle.dequantize_one(sc, ze, 255) == 0x7BFF


def test_subnormal_scale_clamps_codes():
    # range = 300 * 2^-24, b = 8: 300/255 = 1.18 units -> scale = 1 unit (2^-24); (x-min)/scale = 300 -> clamp 255.
    u = 2.0 ** -24
    sc, ze, codes = oracle.quantize_group(h([0.0, 300 * u, 100 * u, 255.4 * u]), 8)
    assert sc == 0x0001 and ze == 0
    assert codes.tolist() == [0, 255, 100, 255]


# ----------------------------------------------------------------- invariants on random groups

@pytest.mark.parametrize("bits", [1, 2, 4, 8])
@pytest.mark.parametrize("G", [16, 64, 128])
def test_quantizer_invariants(bits, G):
    rng = np.random.default_rng(bits * 1000 + G)
    qmax = (1 << bits) - 1
    for trial in range(200):
        scale = 10.0 ** rng.uniform(-1, 3)   # keeps the scale a normal fp16 number (the subnormal case has its own test)
        x = h(rng.standard_normal(G) * scale + rng.uniform(-2, 2) * scale)
        xv = hval(x)
        sc, ze, codes = oracle.quantize_group(x, bits)
        s = hval([sc])[0]
        assert hval([ze])[0] == xv.min()                      # zero-point is the minimum itself
        rng_ = xv.max() - xv.min()
        assert abs(s - rng_ / qmax) <= 2.0 ** -11 * rng_ / qmax + 1e-30  # scale is (max-min)/(2^b-1) to fp16 accuracy
        assert codes[np.argmin(xv)] == 0 and codes[np.argmax(xv)] == qmax
        assert codes.max() <= qmax
        # codes are monotone in the values
        order = np.argsort(xv, kind="stable")
        assert np.all(np.diff(codes[order].astype(int)) >= 0)
        # per-element error: half a step, plus the fp16 rounding of the decoded value
        y = hval([oracle.dequantize_one(sc, ze, q) for q in codes])
        ulp = np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** -14))) - 10), 2.0 ** -24)
        assert np.all(np.abs(y - xv) <= s / 2 + ulp / 2 + 1e-6 * rng_), (bits, G, trial)


def test_pack_unpack_every_byte_value():
    # each byte is b-bit fields, field k at bits [k*b, (k+1)*b): check against the definition, all 256 bytes
    for bits in (1, 2, 4, 8):
        per = 8 // bits
        for byte in range(256):
            fields = [(byte >> (k * bits)) & ((1 << bits) - 1) for k in range(per)]
            assert oracle.pack_codes(np.array(fields, dtype=np.uint8), bits).tolist() == [byte]
            assert oracle.unpack_codes(np.array([byte], dtype=np.uint8), per, bits).tolist() == fields
    rng = np.random.default_rng(0)
    for bits in (1, 2, 4, 8):
        q = rng.integers(0, 1 << bits, 4096).astype(np.uint8)
        assert np.array_equal(oracle.unpack_codes(oracle.pack_codes(q, bits), q.size, bits), q)
    # one bit per code is numpy's own little-endian bit packing
    q = rng.integers(0, 2, 1000).astype(np.uint8)
    assert np.array_equal(oracle.pack_codes(q, 1), np.packbits(q, bitorder="little"))


def test_group_b1_range_beyond_fp16_keeps_a_finite_scale():
    # max - min = 125504 is not an fp16 number: the scale saturates at 65504 instead of becoming infinite,
    # codes are rint((x - min) / 65504) clamped to 1, and both decoded values are finite
    x = h([-60000.0, 65504.0, 0.0, -27000.0, -27500.0, 30000.0])
    sc, ze, codes = oracle.quantize_group(x, 1)
    assert (sc, ze) == (0x7BFF, int(h([-60000.0])[0]))
    assert codes.tolist() == [0, 1, 1, 1, 0, 1]          # (x + 60000) / 65504 = 0, 1.92, 0.916, 0.504, 0.496, 1.37
    assert hval([oracle.dequantize_one(sc, ze, 0)])[0] == -60000.0
    assert hval([oracle.dequantize_one(sc, ze, 1)])[0] == 5504.0


def test_group_b1_is_a_threshold_at_the_midpoint():
    # Sec. 3.2: atop a 4-bit base the levels are 4, 2 and 1 bits.  One bit: scale = max - min, zero = min, and a
    # value becomes 1 when (x - min) / scale rounds to 1: above one half, the tie at exactly one half goes to 0 (even)
    x = h([0.0, 1.0, 0.25, 0.5, 0.75, 0.5009765625, 0.49951171875])
    sc, ze, codes = oracle.quantize_group(x, 1)
    assert (sc, ze) == (0x3C00, 0x0000)
    assert codes.tolist() == [0, 1, 0, 0, 1, 1, 0]
    assert [oracle.dequantize_one(sc, ze, q) for q in (0, 1)] == [0x0000, 0x3C00]
    # shifted and scaled: the two decoded values are the minimum and (to fp16 accuracy) the maximum
    rng = np.random.default_rng(5)
    for _ in range(200):
        x = h(rng.standard_normal(32) * 3 + rng.uniform(-5, 5))
        xv = hval(x)
        sc, ze, codes = oracle.quantize_group(x, 1)
        lo, hi = hval([oracle.dequantize_one(sc, ze, 0)])[0], hval([oracle.dequantize_one(sc, ze, 1)])[0]
        assert lo == xv.min() and abs(hi - xv.max()) <= 2.0 ** -10 * max(abs(xv.max()), xv.max() - xv.min())
        mid = (xv.min() + xv.max()) / 2
        clear = np.abs(xv - mid) > 2.0 ** -9 * (xv.max() - xv.min())     # away from the rounding of the midpoint
        assert np.array_equal(codes[clear], (xv[clear] > mid).astype(np.uint8))


def test_dequantize_closed_form():
    # y = fp16(zero + q*scale), evaluated here in exact rational arithmetic (float64 holds it exactly)
    rng = np.random.default_rng(3)
    for _ in range(3000):
        sc = int(rng.integers(0, 0x7000))
        ze = int(rng.integers(0, 0x7000)) | (int(rng.integers(0, 2)) << 15)
        q = int(rng.integers(0, 256))
        exact = hval([ze])[0] + q * hval([sc])[0]          # exact in float64
        f32 = np.float32(exact)                              # one binary32 rounding
        with np.errstate(over="ignore"):
            want = np.float32(np.clip(f32, -65504.0, 65504.0)).astype(np.float16).view(np.uint16)
        assert oracle.dequantize_one(sc, ze, q) == int(want)


# ----------------------------------------------------------------- record layout and whole-chunk calls

def desc_of(shape, quant_mode=0):
    return oracle.make_desc(shape.n_layers, shape.n_kv_heads, shape.n_q_heads, shape.head_dim, shape.n_tokens,
                            shape.chunk_len, shape.group_size, quant_mode)


def test_record_sizes_closed_form():
    # n_groups * 4 bytes of parameters + n_elements * b / 8 bytes of codes, padded to 256
    want = {
        "tiny": (8704, 4608, 2560),
        "gemma2b": (152064, 78336, 41472),
        "llama7b": (128 * 1024 + 4 * 2 ** 20, 128 * 1024 + 2 * 2 ** 20, 128 * 1024 + 2 ** 20),
    }
    for name, sizes in want.items():
        d = desc_of(synth.CONFIGS[name])
        assert tuple(oracle.record_bytes(d, b) for b in (8, 4, 2)) == sizes
    # one bit per element: 128 KiB of parameters + 2^25 elements / 8 for a 7B-shaped chunk, 1536 + 128 bytes for tiny
    assert oracle.record_bytes(desc_of(synth.CONFIGS["llama7b"]), 1) == 128 * 1024 + 2 ** 19
    assert oracle.record_bytes(desc_of(synth.CONFIGS["tiny"]), 1) == 1536
    # whole 7B-shaped context at 85/86/85 chunks of 8/4/2 bits: 629 MiB against 2048 MiB of fp16
    d = desc_of(synth.CONFIGS["llama7b"])
    total = oracle.compressed_size(d, [8] * 85 + [4] * 86 + [2] * 85)
    assert total == 85 * want["llama7b"][0] + 86 * want["llama7b"][1] + 85 * want["llama7b"][2]
    assert round(total / 2 ** 20) == 629


def test_context_size_matches_paper(golden_dir):
    (L, H, d, T, bpv, want), = read_golden(os.path.join(golden_dir, "context_size.txt"))
    shape = synth.CONFIGS["llama7b"]
    assert (shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.n_tokens) == (L, H, d, T)
    assert shape.n_elements * bpv == want


def test_record_layout_pads_parameter_block_to_16_bytes():
    d = oracle.make_desc(1, 1, 1, 16, 3, 3, 16)   # 2 slabs * 3 tokens * 1 group = 6 groups -> 24 B -> codes at 32
    co, nb = oracle.record_layout(d, 4)
    assert co == 32 and nb == 256


@pytest.mark.parametrize("quant_mode", [0, 1])
def test_compress_chunks_places_groups_where_the_layout_says(quant_mode):
    shape = synth.KVShape("t", 2, 2, 2, 32, 40, 8, 16, seed=5)     # 5 chunks, ragged: T = 40
    kv = synth.kv_tensor(shape).numpy().view(np.uint16)            # [L,2,H,T,d]
    d = desc_of(shape, quant_mode)
    ids = [3, 0, 4, 1]
    bits = [4, 8, 2, 1]
    buf, meta = oracle.compress_chunks(d, kv, ids, bits)
    L, H, CL, D, G = shape.n_layers, shape.n_kv_heads, shape.chunk_len, shape.head_dim, shape.group_size
    off = 0
    for i, (cid, b) in enumerate(zip(ids, bits)):
        n_groups = L * 2 * H * (CL * (D // G) if quant_mode == 0 else D)
        codes_off = (n_groups * 4 + 15) // 16 * 16
        nbytes = (codes_off + L * 2 * H * CL * D * b // 8 + 255) // 256 * 256
        m = meta[i]
        assert (m["chunk_id"], m["bits"], m["offset"], m["nbytes"], m["n_groups"]) == (cid, b, off, nbytes, n_groups)
        rec = buf[off:off + nbytes]
        assert m["checksum"] == int(rec.view("<u4").sum(dtype=np.uint64) & 0xFFFFFFFF)
        params = rec[:n_groups * 4].view("<u2").reshape(n_groups, 2)
        all_codes = oracle.unpack_codes(rec[codes_off:], L * 2 * H * CL * D, b).reshape(L, 2, H, CL, D)
        g = 0
        for l, s, hh in itertools.product(range(L), range(2), range(H)):
            tile = kv[l, s, hh, cid * CL:(cid + 1) * CL, :]          # [CL, D] of this chunk
            if quant_mode == 0:
                groups = [(tile[t, j * G:(j + 1) * G], (t, slice(j * G, (j + 1) * G)))
                          for t in range(CL) for j in range(D // G)]
            else:
                groups = [(tile[:, c], (slice(None), c)) for c in range(D)]
            for x, where in groups:
                sc, ze, codes = oracle.quantize_group(np.ascontiguousarray(x), b)
                assert (params[g, 0], params[g, 1]) == (sc, ze)
                assert np.array_equal(all_codes[l, s, hh][where], codes)
                g += 1
        assert g == n_groups
        tail = rec[codes_off + L * 2 * H * CL * D * b // 8:]
        assert not tail.any() and not rec[n_groups * 4:codes_off].any()   # padding is zero
        off += nbytes
    assert off == buf.size


@pytest.mark.parametrize("quant_mode", [0, 1])
def test_round_trip_error_and_untouched_chunks(quant_mode):
    shape = synth.CONFIGS["tiny"]
    kv_t = synth.kv_tensor(shape)
    kv = kv_t.numpy().view(np.uint16)
    d = desc_of(shape, quant_mode)
    bits = synth.random_bits(shape.n_chunks, 0).numpy()
    ids = np.arange(shape.n_chunks)
    keep = ids != 7                                     # leave chunk 7 out
    buf, meta = oracle.compress_chunks(d, kv, ids[keep], bits[keep])
    out = np.full_like(kv, 0x7E00)                      # NaN canary
    oracle.decompress_chunks(d, buf, meta, out)
    CL = shape.chunk_len
    assert np.all(out[..., 7 * CL:8 * CL, :] == 0x7E00)
    x = kv_t.numpy().astype(np.float64)
    y = out.view(np.float16).astype(np.float64)
    for cid, b in zip(ids[keep], bits[keep]):
        xs, ys = x[..., cid * CL:(cid + 1) * CL, :], y[..., cid * CL:(cid + 1) * CL, :]
        if quant_mode == 0:
            G = shape.group_size
            xg = xs.reshape(*xs.shape[:-1], -1, G)
            rng_ = np.repeat((xg.max(-1) - xg.min(-1))[..., None], G, -1).reshape(xs.shape)
        else:
            rng_ = np.broadcast_to(xs.max(-2, keepdims=True) - xs.min(-2, keepdims=True), xs.shape)
        step = rng_ / ((1 << int(b)) - 1)
        # half a step (+ fp16 rounding of scale and of the result: both below 2^-10 relative)
        assert np.all(np.abs(ys - xs) <= 0.5 * step * (1 + 2.0 ** -9) + 2.0 ** -10 * np.abs(xs) + 1e-7)


def test_decompress_into_other_slots():
    shape = synth.CONFIGS["tiny"]
    kv = synth.kv_tensor(shape).numpy().view(np.uint16)
    d = desc_of(shape)
    buf, meta = oracle.compress_chunks(d, kv, [2, 5], [8, 4])
    a = np.zeros_like(kv)
    oracle.decompress_chunks(d, buf, meta, a)
    b = np.zeros_like(kv)
    oracle.decompress_chunks(d, buf, meta, b, dst_ids=[9, 0])
    CL = shape.chunk_len
    assert np.array_equal(a[..., 2 * CL:3 * CL, :], b[..., 9 * CL:10 * CL, :])
    assert np.array_equal(a[..., 5 * CL:6 * CL, :], b[..., 0:CL, :])


def test_bad_arguments_are_errors():
    d = desc_of(synth.CONFIGS["tiny"])
    with pytest.raises(RuntimeError):
        oracle.record_bytes(d, 3)
    kv = np.zeros(synth.CONFIGS["tiny"].n_elements, dtype=np.uint16)
    with pytest.raises(RuntimeError):
        oracle.compress_chunks(d, kv, [16], [8])       # chunk id out of range
