"""llms_compress_context (scores, levels and records of a whole context in one call): the same bytes as the
three calls made one after the other, and as the oracle run on the scores the GPU produced."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import binding as B, synth
from gpu_helpers import assert_meta_equal, bits_view, first_mismatch, odesc

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("pinned_scores,pinned_bits", [(True, True), (True, False), (False, False)],
                         ids=["stream_ordered", "pinned_scores", "pageable"])
@pytest.mark.parametrize("levels,frac", [((8, 4, 2), (1 / 3, 1 / 3, 1 / 3)), ((4, 2, 1), (0.2, 0.5, 0.3))])
def test_compress_context_equals_the_separate_calls_and_the_oracle(levels, frac, pinned_scores, pinned_bits):
    """With scores, levels and meta all in page-locked memory the ranking and the chunk table are made by a kernel and
    the call does not synchronise; with any of them pageable the ranking is a host step.  Same bytes either way."""
    sh = synth.KVShape("ctx", 3, 2, 4, 64, 208, 16, 64, seed=13)          # 13 chunks, GQA
    W = sh.window
    kv, q = synth.kv_tensor(sh), synth.q_window(sh, W)
    kv_dev, q_dev = kv.cuda(), q.cuda()
    d = B.desc_of(sh)
    n = sh.n_chunks
    frac_a, levels_a = np.asarray(frac, dtype=np.float32), np.asarray(levels, dtype=np.uint8)

    # one call
    scores_dev = torch.empty(n, dtype=torch.float32, device="cuda")
    # into pinned memory the score kernel stores the scores itself, pageable memory gets them by a copy
    scores_host = torch.full((n,), -1.0, dtype=torch.float32)
    if pinned_scores:
        scores_host = scores_host.pin_memory()
    bits = B.new_pinned(n) if pinned_bits else np.zeros(n, dtype=np.uint8)
    total = B.compressed_size(d, np.full(n, levels[0], np.uint8))
    buf = torch.zeros(total, dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    ws_t = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    ws_c = torch.full((B.codec_workspace_bytes(n),), 0xA5, dtype=torch.uint8, device="cuda")   # nothing relies on zeros
    before, after = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    after.record()                                                        # creates the handle the library records
    torch.cuda.synchronize()
    before.record()
    B.compress_context(d, kv_dev, q_dev, W, frac_a, levels_a, scores_dev, scores_host, bits, buf, meta, ws_t, ws_c,
                       after_scores=after)
    B.wait(after)                                                         # scores, levels and meta are on the host now
    early_bits, early_meta = bits.copy(), meta.copy()
    torch.cuda.synchronize()
    assert before.elapsed_time(after) > 0                                 # recorded behind the score kernels
    assert np.array_equal(early_bits, bits)
    for f in ("chunk_id", "bits", "offset", "nbytes", "n_groups"):
        assert np.array_equal(early_meta[f], meta[f]), f

    # the three calls
    scores2 = torch.empty(n, dtype=torch.float32, device="cuda")
    B.chunk_tolerance(d, kv_dev, q_dev, W, scores2, ws_t)
    s2 = scores2.cpu().numpy()
    assert np.array_equal(s2, scores_host.numpy())                        # scores are reproducible bit for bit
    bits2, _ = B.assign_levels(s2, frac, levels)
    assert np.array_equal(bits, bits2)
    buf2 = torch.zeros(total, dtype=torch.uint8, device="cuda")
    meta2 = B.new_meta(n, pinned=True)
    B.compress_chunks(d, kv_dev, np.arange(n, dtype=np.uint32), bits2, buf2, meta2, ws_c)
    torch.cuda.synchronize()
    used = int(meta["offset"][-1] + meta["nbytes"][-1])
    assert torch.equal(buf[:used], buf2[:used])
    assert_meta_equal(meta, meta2)

    # the oracle, on the GPU's scores (fp32 scores can flip near-ties against fp64 ones)
    obits, _ = oracle.assign_levels(s2, frac, levels)
    assert np.array_equal(bits, obits)
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), np.arange(n), obits)
    assert first_mismatch(buf[:used].cpu().numpy(), want_buf) is None
    assert_meta_equal(meta, want_meta)


def test_compress_context_argument_errors():
    sh = synth.CONFIGS["tiny"]
    d = B.desc_of(sh)
    rc = B.lib().llms_compress_context(None, None, None, 8, None, None, None, None, None, None, 0, None, None, 0, None, 0,
                                       None, None)
    assert rc == B.ERR_INVALID_ARG
    # everything is checked before the first launch: nothing of the outputs is touched on an error
    W, n = sh.window, sh.n_chunks
    kv_dev, q_dev = synth.kv_tensor(sh).cuda(), synth.q_window(sh, W).cuda()
    scores_dev = torch.full((n,), -7.0, dtype=torch.float32, device="cuda")
    scores_host = torch.full((n,), -7.0, dtype=torch.float32).pin_memory()
    bits = B.new_pinned(n)
    meta = B.new_meta(n, pinned=True)
    buf = torch.zeros(B.compressed_size(d, np.full(n, 8, np.uint8)), dtype=torch.uint8, device="cuda")
    ws_t = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    ws_c = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    good = dict(frac=np.asarray((1 / 3, 1 / 3, 1 / 3), np.float32), levels=np.asarray((8, 4, 2), np.uint8), out=buf, ws_c=ws_c)

    def call(**kw):
        a = dict(good, **kw)
        with pytest.raises(B.LlmsError) as e:
            B.compress_context(d, kv_dev, q_dev, W, a["frac"], a["levels"], scores_dev, scores_host, bits, a["out"], meta, ws_t,
                               a["ws_c"])
        return e.value.status

    assert call(frac=np.asarray((0.5, 0.6, 0.2), np.float32)) == B.ERR_INVALID_ARG
    assert call(levels=np.asarray((8, 3, 2), np.uint8)) == B.ERR_BAD_BITS
    assert call(levels=np.asarray((2, 4, 8), np.uint8)) == B.ERR_INVALID_ARG
    assert call(out=buf[:B.compressed_size(d, np.full(n, 4, np.uint8))]) == B.ERR_BUF_TOO_SMALL   # 5 or 6 of 16 chunks keep 8 bits
    assert call(ws_c=ws_c[:64]) == B.ERR_BUF_TOO_SMALL
    torch.cuda.synchronize()
    assert (scores_dev.cpu() == -7.0).all() and (scores_host == -7.0).all() and not bits.any() and not meta["nbytes"].any()


@pytest.mark.parametrize("n", [4096, 3001, 700, 200, 2])
def test_device_ranking_with_equal_scores_and_many_chunks(n):
    """The kernel that ranks the chunks (stream-ordered form) against the oracle's rule on the same scores: up to the
    most chunks it takes, chunk counts that are no power of two, and contexts whose second half repeats the first,
    so that whole runs of chunks have bit-equal scores and only their index orders them."""
    sh = synth.KVShape("many", 1, 1, 1, 64, 4 * n, 4, 64, seed=21)
    W = min(sh.window, sh.n_tokens)
    kv = synth.kv_tensor(sh)
    half = (n // 2) * sh.chunk_len
    kv[..., half:2 * half, :] = kv[..., :half, :]
    q = synth.q_window(sh, W)
    d = B.desc_of(sh)
    frac_a, levels_a = np.asarray((0.3, 0.4, 0.3), dtype=np.float32), np.asarray((8, 4, 2), dtype=np.uint8)
    scores_dev = torch.empty(n, dtype=torch.float32, device="cuda")
    scores_host = torch.empty(n, dtype=torch.float32).pin_memory()
    bits = B.new_pinned(n)
    buf = torch.zeros(B.compressed_size(d, np.full(n, 8, np.uint8)), dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    ws_t = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    ws_c = torch.full((B.codec_workspace_bytes(n),), 0x5A, dtype=torch.uint8, device="cuda")
    B.compress_context(d, kv.cuda(), q.cuda(), W, frac_a, levels_a, scores_dev, scores_host, bits, buf, meta, ws_t, ws_c)
    torch.cuda.synchronize()
    s = scores_host.numpy()
    if n >= 200:
        assert np.unique(s).size < n - n // 4                 # many chunks share their score with another one
    obits, _ = oracle.assign_levels(s, (0.3, 0.4, 0.3), (8, 4, 2))
    assert np.array_equal(bits, obits)
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), np.arange(n), obits)
    assert_meta_equal(meta, want_meta)
    assert first_mismatch(buf[:want_buf.size].cpu().numpy(), want_buf) is None


def test_full_size_step_as_the_benchmark_runs_it():
    """The 7B-shaped context through llms_compress_context and llms_decompress_chunks_ordered, back to back without a
    synchronisation in between: levels against the oracle's rule on the GPU's scores, sampled records and their decoded
    chunks against the oracle, every record through its checksum."""
    sh = synth.CONFIGS["llama7b"]
    W, n, CL = sh.window, sh.n_chunks, sh.chunk_len
    kv_dev = synth.kv_tensor(sh, device="cuda")
    q_dev = synth.q_window(sh, W, device="cuda")
    d = B.desc_of(sh)
    frac, levels = np.asarray(sh.frac, dtype=np.float32), np.asarray((8, 4, 2), dtype=np.uint8)
    scores_dev = torch.empty(n, dtype=torch.float32, device="cuda")
    scores_host = torch.empty(n, dtype=torch.float32).pin_memory()
    bits = B.new_pinned(n)
    buf = torch.empty(B.compressed_size(d, np.full(n, 8, np.uint8)), dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    ws_t = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    ws_c = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    ws_d = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(kv_dev)
    planned = B.new_event()
    for _ in range(2):
        B.compress_context(d, kv_dev, q_dev, W, frac, levels, scores_dev, scores_host, bits, buf, meta, ws_t, ws_c,
                           after_scores=planned)
        B.wait(planned)                                   # levels and record offsets are on the host; the encoder still runs
        B.decompress_chunks_ordered(d, buf, meta, None, out, ws_d)
        assert B.codec_corrupt_count(ws_d) == 0
    obits, _ = oracle.assign_levels(scores_host.numpy(), sh.frac, (8, 4, 2))
    assert np.array_equal(bits, obits)
    assert tuple(int((bits == b).sum()) for b in (8, 4, 2)) == (85, 86, 85)
    one = sh.with_(n_tokens=CL)
    picks = {0, n - 1} | {int(np.flatnonzero(bits == b)[40]) for b in (8, 4, 2)}
    for cid in sorted(picks):
        chunk = kv_dev[..., cid * CL:(cid + 1) * CL, :].contiguous().cpu()
        want_buf, want_meta = oracle.compress_chunks(odesc(one), bits_view(chunk), [0], [bits[cid]])
        m = meta[cid]
        got = buf[int(m["offset"]):int(m["offset"] + m["nbytes"])].cpu().numpy()
        assert first_mismatch(got, want_buf) is None, cid
        assert m["checksum"] == want_meta[0]["checksum"]
        want = np.zeros(chunk.numel(), dtype=np.uint16).reshape(chunk.shape)
        oracle.decompress_chunks(odesc(one), want_buf, want_meta, want)
        got_chunk = out[..., cid * CL:(cid + 1) * CL, :].contiguous().cpu()
        assert first_mismatch(bits_view(got_chunk).reshape(-1), want.reshape(-1)) is None, cid
