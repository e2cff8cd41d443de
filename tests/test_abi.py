"""The C-ABI library: it loads, exports every function the header declares, and its host-only entry points
(sizes, rank -> bits, LCTRU order, argument checks) agree with the oracle.  No GPU needed."""
import ctypes
import itertools
import os
import re

import numpy as np
import pytest

import oracle
from paper_2403_11805_b200 import binding as B, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "llms.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(llms_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported():
    names = declared_functions()
    assert len(names) >= 17
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), name
    assert set(B._SIGNATURES) == set(names)


def odesc(sh, mode=0):
    return oracle.make_desc(sh.n_layers, sh.n_kv_heads, sh.n_q_heads, sh.head_dim, sh.n_tokens, sh.chunk_len,
                            sh.group_size, mode)


def test_record_sizes_match_oracle():
    for sh in synth.CONFIGS.values():
        for mode in (0, 1):
            for b in (1, 2, 4, 8):
                assert B.record_layout(B.desc_of(sh, mode), b) == oracle.record_layout(odesc(sh, mode), b)
    odd = synth.KVShape("odd", 1, 1, 1, 16, 3, 3, 16)
    assert B.record_layout(B.desc_of(odd), 4) == oracle.record_layout(odesc(odd), 4) == (32, 256)
    bits = [8, 4, 2, 2, 8]
    sh = synth.CONFIGS["tiny"]
    assert B.compressed_size(B.desc_of(sh), bits) == oracle.compressed_size(odesc(sh), bits)


def test_assign_bits_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(0)
    for n, frac in [(256, (1 / 3, 1 / 3, 1 / 3)), (128, (1 / 3, 1 / 3, 1 / 3)), (32, (1 / 3, 1 / 3, 1 / 3)),
                    (512, (0.1, 0.5, 0.4)), (7, (0.5, 0.25, 0.25)), (1, (0.2, 0.3, 0.5)), (0, (1 / 3, 1 / 3, 1 / 3))]:
        for ties in (False, True):
            s = rng.random(n).astype(np.float32)
            if ties:
                s = np.round(s * 4) / 4
            gb, go = B.assign_bits(s, frac)
            ob, oo = oracle.assign_bits(s, frac)
            assert np.array_equal(gb, ob) and np.array_equal(go, oo)
    for scores in itertools.product([0.1, 0.2, 0.3], repeat=5):
        gb, go = B.assign_bits(scores, (0.4, 0.2, 0.4))
        ob, oo = oracle.assign_bits(scores, (0.4, 0.2, 0.4))
        assert np.array_equal(gb, ob) and np.array_equal(go, oo)


def test_assign_levels_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(1)
    for levels in ((8, 4, 2), (4, 2, 1), (8, 2, 1), (8, 4, 1)):
        for n, frac in [(256, (1 / 3, 1 / 3, 1 / 3)), (37, (0.1, 0.5, 0.4)), (1, (0.2, 0.3, 0.5)), (0, (1 / 3, 1 / 3, 1 / 3))]:
            s = np.round(rng.random(n).astype(np.float32) * 8) / 8
            gb, go = B.assign_levels(s, frac, levels)
            ob, oo = oracle.assign_levels(s, frac, levels)
            assert np.array_equal(gb, ob) and np.array_equal(go, oo)
    for bad, status in (((4, 4, 2), B.ERR_INVALID_ARG), ((2, 4, 8), B.ERR_INVALID_ARG), ((8, 3, 1), B.ERR_BAD_BITS)):
        with pytest.raises(B.LlmsError) as e:
            B.assign_levels([0.5, 0.25], (0.5, 0.25, 0.25), bad)
        assert e.value.status == status


def test_optimize_thresholds_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(2)
    for n in (1, 2, 5, 32, 256, 512):
        for R in (0.5, 0.3, 0.8, 1.0, 0.25):
            for ties in (False, True):
                s = (rng.random(n) ** 3).astype(np.float32)
                if ties:
                    s = np.round(s * 4) / 4
                try:
                    want, _ = oracle.optimize_thresholds(s, R)
                except RuntimeError:                   # no integer split meets the ratio (tiny n): both refuse
                    with pytest.raises(B.LlmsError):
                        B.optimize_thresholds(s, R)
                    continue
                assert np.array_equal(B.optimize_thresholds(s, R).view(np.uint32), want.view(np.uint32))
    with pytest.raises(B.LlmsError):
        B.optimize_thresholds([0.1, 0.2], 0.2)


def test_optimize_thresholds_levels_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(8)
    for levels in ((8, 4, 2), (4, 2, 1), (8, 2, 1), (8, 4, 1)):
        for n in (6, 32, 256, 1000):
            for R in (0.5, 0.35, 0.8, levels[2] / levels[0], 1.0):
                s = (rng.random(n) ** 3).astype(np.float32)
                try:
                    want, _ = oracle.optimize_thresholds_levels(s, R, levels)
                except RuntimeError:
                    with pytest.raises(B.LlmsError):
                        B.optimize_thresholds_levels(s, R, levels)
                    continue
                assert np.array_equal(B.optimize_thresholds_levels(s, R, levels), want)
    with pytest.raises(B.LlmsError):
        B.optimize_thresholds_levels([0.1, 0.2, 0.3], 0.1, (8, 4, 2))       # below the low level's ratio


def test_optimize_thresholds_against_an_exhaustive_search():
    """Eq. 3 by search, in exact rational arithmetic, sharing no formula with the library or the oracle: for every count
    of top-level chunks the count of low-level chunks is the one whose achieved ratio comes closest to the wanted one
    (searched, not solved for; a tie goes to more compression), the objective is the plain weighted sum over the
    density-ordered chunks, the best triple wins, the smaller top count on a tie."""
    from fractions import Fraction as F
    rng = np.random.default_rng(11)
    for levels in ((8, 4, 2), (4, 2, 1), (8, 2, 1), (8, 4, 1)):
        r1, r2 = F(levels[1], levels[0]), F(levels[2], levels[0])
        for n in (1, 2, 3, 5, 8, 12):
            for R in (F(1, 2), F(3, 8), F(3, 4), F(5, 16), F(1), r2):
                if R < r2:
                    continue
                # dyadic scores: every sum below is exact in binary64 too, so ties are ties on both sides
                scores = (rng.integers(1, 64, n) / 64.0).astype(np.float32)
                dens = sorted((F(float(x)) for x in scores), reverse=True)
                best = None
                step = (r1 - r2) / n                       # what one more low-level chunk takes off the achieved ratio
                for n_top in range(n + 1):
                    cands = []
                    for n_low in range(n + 1):
                        achieved = (n_top + r1 * (n - n_top - n_low) + r2 * n_low) / n
                        cands.append((abs(achieved - R), -n_low, achieved))
                    _, neg_low, achieved = min(cands)
                    n_low = -neg_low
                    if not (-step / 2 <= achieved - R < step / 2):    # even the nearest count is more than half a step off
                        continue
                    if n_top + n_low > n:                             # more chunks than there are
                        continue
                    info = sum(dens[:n_top]) + r1 * sum(dens[n_top:n - n_low]) + r2 * sum(dens[n - n_low:])
                    if best is None or info > best[0]:
                        best = (info, n_top, n_low)
                if best is None:
                    with pytest.raises(B.LlmsError):
                        B.optimize_thresholds_levels(scores, float(R), levels)
                    continue
                got = B.optimize_thresholds_levels(scores, float(R), levels)
                want = np.array([best[1], n - best[1] - best[2], best[2]], dtype=np.float64) / n
                assert np.array_equal(got, want.astype(np.float32)), (levels, n, R, scores, got, want)


def test_lctru_order_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(1)
    for n in (0, 1, 5, 64, 2048):
        t = np.zeros(n, dtype=B.STATE_DTYPE)
        t["ctx_id"] = rng.integers(0, 64, n)
        t["chunk_id"] = rng.integers(0, 32, n)
        t["bits"] = rng.choice([8, 4, 2, 1], n)
        t["resident"] = rng.random(n) < 0.7
        t["locked"] = rng.random(n) < 0.2
        t["last_access_step"] = rng.integers(0, 10, n)
        assert np.array_equal(B.lctru_order(t), oracle.lctru_order(t.astype(oracle.STATE_DTYPE)))


def test_argument_errors_on_the_host():
    sh = synth.CONFIGS["tiny"]
    d = B.desc_of(sh)
    with pytest.raises(B.LlmsError) as e:
        B.record_bytes(d, 3)
    assert e.value.status == B.ERR_BAD_BITS
    bad = B.desc_of(sh)
    bad.n_q_heads = 3
    with pytest.raises(B.LlmsError) as e:
        B.record_bytes(bad, 4)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.LlmsError):
        B.assign_bits([0.1, 0.2], (0.5, 0.6, 0.2))
    # the codec entry points check their arguments before touching CUDA: dummy addresses are enough
    meta = B.new_meta(2)
    lib = B.lib()
    ids = np.array([1, 1], dtype=np.uint32)
    bits = np.array([8, 4], dtype=np.uint8)
    call = lambda **kw: lib.llms_compress_chunks(
        ctypes.addressof(kw.get("desc", d)), kw.get("kv", 4096), B._ptr(kw.get("ids", ids)), B._ptr(kw.get("bits", bits)),
        2, kw.get("out", 8192), kw.get("out_bytes", 1 << 20), B._ptr(meta), kw.get("ws", 4096), kw.get("ws_bytes", B.codec_workspace_bytes(2)), None)
    assert call() == B.ERR_INVALID_ARG                                   # duplicate chunk id
    ok_ids = np.array([1, 2], dtype=np.uint32)
    assert call(ids=np.array([1, 16], dtype=np.uint32)) == B.ERR_INVALID_ARG   # id out of range
    assert call(ids=ok_ids, bits=np.array([8, 5], dtype=np.uint8)) == B.ERR_BAD_BITS
    assert call(ids=ok_ids, kv=4098) == B.ERR_MISALIGNED
    assert call(ids=ok_ids, out=8192 + 64) == B.ERR_MISALIGNED
    assert call(ids=ok_ids, out_bytes=8704) == B.ERR_BUF_TOO_SMALL        # needs 8704 + 4608
    assert call(ids=ok_ids, ws_bytes=32) == B.ERR_BUF_TOO_SMALL
    d2 = B.desc_of(sh)
    d2.group_size = 48                                                      # divides 96 but is not a power of two
    d2.head_dim = 96
    assert call(ids=ok_ids, desc=d2) == B.ERR_UNSUPPORTED
    assert B.lib().llms_wait(None, 1) == B.ERR_INVALID_ARG
    assert B.lib().llms_strerror(B.ERR_CORRUPT).decode() == "record checksum mismatch"


def test_records_outside_their_buffers_are_refused_on_the_host():
    """A meta table that points past the end of the swap buffer or of the arena (stale, damaged) is an error code,
    found before anything is enqueued: the addresses here are dummies that no kernel or copy could survive."""
    sh = synth.CONFIGS["tiny"]
    d = B.desc_of(sh)
    lib = B.lib()
    nb8, nb4 = B.record_bytes(d, 8), B.record_bytes(d, 4)
    meta = B.new_meta(2)
    meta["chunk_id"] = [0, 1]
    meta["bits"] = [8, 4]
    meta["offset"] = [0, nb8]
    meta["nbytes"] = [nb8, nb4]
    meta["n_groups"] = sh.n_slabs * sh.chunk_len * (sh.head_dim // sh.group_size)
    for fn in (lib.llms_decompress_chunks,):
        dec = lambda buf_bytes, m=meta: fn(ctypes.addressof(d), 8192, buf_bytes, B._ptr(m), None, 2, 4096, 4096, B.codec_workspace_bytes(2), None)
        assert dec(nb8 + nb4 - 1) == B.ERR_BUF_TOO_SMALL
        assert dec(nb8) == B.ERR_BUF_TOO_SMALL
        assert dec(0) == B.ERR_BUF_TOO_SMALL
        far = meta.copy()
        far["offset"][1] = (1 << 64) - 256                               # offset + nbytes wraps around
        assert dec(1 << 40, far) == B.ERR_BUF_TOO_SMALL
        wrong = meta.copy()
        wrong["nbytes"][1] = nb8                                         # not the size of a 4-bit record
        assert dec(1 << 40, wrong) == B.ERR_INVALID_ARG
    out = lambda dev_bytes, host_bytes, ho=None, m=meta: lib.llms_swap_out(
        8192, dev_bytes, B._ptr(m), 2, 1 << 20, host_bytes, B._ptr(ho), None, None, None)
    inn = lambda dev_bytes, host_bytes, ho=None, m=meta: lib.llms_swap_in(
        1 << 20, host_bytes, B._ptr(ho), B._ptr(m), 2, 8192, dev_bytes, None, None, None)
    for call in (out, inn):
        assert call(nb8 + nb4 - 256, 1 << 30) == B.ERR_BUF_TOO_SMALL     # device buffer too short
        assert call(1 << 30, nb8 + nb4 - 256) == B.ERR_BUF_TOO_SMALL     # arena too short at the same offsets
        ho = np.array([0, 1 << 20], dtype=np.uint64)
        assert call(1 << 30, (1 << 20) + nb4 - 16, ho) == B.ERR_BUF_TOO_SMALL   # arena too short at its own offsets
        ho[1] = (1 << 64) - 16
        assert call(1 << 30, 1 << 40, ho) == B.ERR_BUF_TOO_SMALL         # wraps around
