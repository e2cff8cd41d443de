"""Whole workloads against the oracle at the sizes the throughput is quoted on, in the launch configuration the
benchmark times (llms_compress_context followed by llms_decompress_chunks_ordered on one stream):

  * the 7B-shaped context (32 layers x 32 heads x 4096 tokens, 256 chunks): every score, every level, every record
    byte, every meta field and every decoded value;
  * the 32K-token grouped-query context (512 chunks, levels 10% / 50% / 40% by the GPU's own scores): the same,
    with the score of all 32 query heads over all 32768 tokens against the binary64 oracle;
  * the multi-app driver at its real shape (64 contexts of 1024 tokens, pool of 512 slots, 8 contexts per step):
    every LCTRU order, four contexts replayed operation by operation with the oracle's codec, every record of the
    arena through the oracle's checksum.

The oracle needs a few seconds per workload for the codec and up to a minute for the binary64 attention window of
the 32K context; nothing here is sampled.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import binding as B, synth
from paper_2403_11805_b200.multiapp import MultiApp
from gpu_helpers import assert_meta_equal, bits_view, first_mismatch, odesc

pytestmark = pytest.mark.gpu


def oracle_scores(sh, kv_host, q_host, W, layers_per_pass=8):
    """Eq. 1 in binary64 over the whole context.  The density is a mean over layers, so the oracle is run on blocks
    of layers (its attention window for all 32 layers of the long context would not fit comfortably) and the block
    results are averaged, weighted by their layer counts."""
    total = np.zeros(sh.n_chunks, dtype=np.float64)
    for l0 in range(0, sh.n_layers, layers_per_pass):
        l1 = min(sh.n_layers, l0 + layers_per_pass)
        part = sh.with_(n_layers=l1 - l0)
        total += (l1 - l0) * oracle.chunk_tolerance(odesc(part), kv_host[l0:l1], q_host[l0:l1], W)
    return total / sh.n_layers


def run_whole_context(sh, levels=(8, 4, 2)):
    W, n = sh.window, sh.n_chunks
    kv_dev = synth.kv_tensor(sh, device="cuda")
    q_dev = synth.q_window(sh, W, device="cuda")
    d = B.desc_of(sh)
    frac_a, levels_a = np.asarray(sh.frac, dtype=np.float32), np.asarray(levels, dtype=np.uint8)
    scores_dev = torch.empty(n, dtype=torch.float32, device="cuda")
    scores_host = torch.empty(n, dtype=torch.float32).pin_memory()
    bits = B.new_pinned(n)                  # everything page-locked: the call ranks on the device and does not synchronise
    buf = torch.empty(B.compressed_size(d, np.full(n, levels[0], np.uint8)), dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    ws_t = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    ws_c = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    ws_d = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    out = torch.zeros_like(kv_dev)
    planned = B.new_event()
    for _ in range(2):                      # the second pass reuses every workspace, as the timed loop does
        B.compress_context(d, kv_dev, q_dev, W, frac_a, levels_a, scores_dev, scores_host, bits, buf, meta, ws_t, ws_c,
                           after_scores=planned)
        B.wait(planned)                     # meta is needed on the host by the next call
        B.decompress_chunks_ordered(d, buf, meta, None, out, ws_d)
        assert B.codec_corrupt_count(ws_d) == 0
    kv_host, q_host = bits_view(kv_dev), bits_view(q_dev)
    del kv_dev

    # scores: every chunk within 1e-4 relative of the binary64 oracle
    got_scores = scores_host.numpy().copy()
    assert np.array_equal(got_scores, scores_dev.cpu().numpy())
    want_scores = oracle_scores(sh, kv_host, q_host, W)
    rel = np.abs(got_scores - want_scores) / want_scores
    assert rel.max() < 1e-4, (int(rel.argmax()), float(rel.max()))

    # levels: the oracle's rule on the scores the GPU produced (binary32 scores can flip near-ties against binary64)
    obits, _ = oracle.assign_levels(got_scores, sh.frac, levels)
    assert np.array_equal(bits, obits)

    # every record, every meta field
    ids = np.arange(n, dtype=np.uint32)
    want_buf, want_meta = oracle.compress_chunks(odesc(sh), kv_host, ids, obits)
    used = int(meta["offset"][-1] + meta["nbytes"][-1])
    assert used == want_buf.size
    assert_meta_equal(meta, want_meta)
    got_buf = buf[:used].cpu().numpy()
    assert first_mismatch(got_buf, want_buf) is None
    del got_buf

    # every decoded value, layer by layer
    want = np.zeros(kv_host.shape, dtype=np.uint16)
    oracle.decompress_chunks(odesc(sh), want_buf, want_meta, want)
    for l in range(sh.n_layers):
        assert first_mismatch(bits_view(out[l]).reshape(-1), want[l].reshape(-1)) is None, l
    return bits


def test_llama7b_whole_context_against_the_oracle():
    bits = run_whole_context(synth.CONFIGS["llama7b"])
    assert tuple(int((bits == b).sum()) for b in (8, 4, 2)) == (85, 86, 85)


def test_mistral_32k_whole_context_against_the_oracle():
    bits = run_whole_context(synth.CONFIGS["mistral7b_32k"])
    assert tuple(int((bits == b).sum()) for b in (8, 4, 2)) == (51, 256, 205)


def test_multiapp_real_shape_against_the_oracle():
    sh = synth.CONFIGS["multiapp"]
    n_slots, per_step, steps = 512, 8, 4
    app = MultiApp(sh, n_slots=n_slots, seed=sh.seed, log_ops=True)
    app.build()
    first_op_of_trace = len(app.ops)
    served = [app.step(per_step) for _ in range(steps)]
    app.finish()
    assert all(len(s) == per_step for s in served)
    assert any(op == "evict" for op, _, _ in app.ops[first_op_of_trace:])

    # every eviction order is the oracle's for the same table
    assert len(app.orders) >= steps
    for table, order in app.orders:
        assert np.array_equal(order, oracle.lctru_order(table.astype(oracle.STATE_DTYPE)))
        assert not table["locked"][order].any() and table["resident"][order].all()

    # four contexts in full: one that the trace served and evicted again where there is one, plus fixed picks
    CL, cpc = sh.chunk_len, app.cpc
    touched = [int(r) // cpc for op, r, _ in app.ops[first_op_of_trace:] if op == "evict"]
    picks = sorted(set(touched[:2]) | {0, sh.n_contexts - 1, served[0][0], served[-1][-1]})[:4]
    one = sh.with_(n_tokens=CL)
    od_one, od_ctx = odesc(one), odesc(sh)
    host_arena = app.arena.numpy()
    for c in picks:
        kv_dev = synth.kv_tensor(sh, device="cuda", context=c)
        q_dev = synth.q_window(sh, sh.window, device="cuda", context=c)
        kv, q = bits_view(kv_dev), bits_view(q_dev)
        # scores (reproducible bit for bit, so the ones the driver ranked are these) and the levels made from them
        scores = torch.empty(cpc, dtype=torch.float32, device="cuda")
        ws_t = torch.empty(B.tolerance_workspace_bytes(app.desc_ctx, sh.window), dtype=torch.uint8, device="cuda")
        B.chunk_tolerance(app.desc_ctx, kv_dev, q_dev, sh.window, scores, ws_t)
        got_scores = scores.cpu().numpy()
        del kv_dev, q_dev
        want_scores = oracle.chunk_tolerance(od_ctx, kv, q, sh.window)
        assert (np.abs(got_scores - want_scores) / want_scores).max() < 1e-4
        ob, _ = oracle.assign_bits(got_scores, app.frac)
        assert np.array_equal(app.bits[c], ob)
        assert sorted(ob.tolist()) == [2] * 11 + [4] * 10 + [8] * 11
        rows = range(c * cpc, (c + 1) * cpc)
        arena = {}
        for i, r in enumerate(rows):
            chunk = np.ascontiguousarray(kv[..., i * CL:(i + 1) * CL, :])
            arena[r] = oracle.compress_chunks(od_one, chunk, [0], [app.bits[c][i]])
        pool = {}
        for op, row, slot in app.ops:
            if row not in arena:
                continue
            if op == "load":
                buf, meta = arena[row]
                out = np.zeros((sh.n_layers, 2, sh.n_kv_heads, CL, sh.head_dim), dtype=np.uint16)
                oracle.decompress_chunks(od_one, buf, meta, out)
                pool[row] = (slot, out)
            elif op == "drop":
                pool.pop(row)
            else:
                assert pool[row][0] == slot
                arena[row] = oracle.compress_chunks(od_one, pool[row][1], [0], [int(app.table["bits"][row])])
                if op == "evict":
                    pool.pop(row)
        for r in rows:
            buf, meta = arena[r]
            off = int(app.arena_off[r])
            assert first_mismatch(host_arena[off:off + buf.size], buf) is None, r
            assert app.checksum[r] == meta[0]["checksum"]
            assert (r in pool) == bool(app.table["resident"][r])
        for r, (slot, want) in pool.items():
            assert app.slot[r] == slot
            got = bits_view(app.pool[..., slot * CL:(slot + 1) * CL, :])
            assert first_mismatch(got.reshape(-1), want.reshape(-1)) is None, r

    # every other record: the bytes in the arena carry the checksum the device computed for them
    for r in range(sh.n_contexts * cpc):
        off, nb = int(app.arena_off[r]), app.rec_bytes[int(app.table["bits"][r])]
        assert oracle.checksum(host_arena[off:off + nb]) == app.checksum[r], r
    res = app.slot >= 0
    assert np.array_equal(res, app.table["resident"] != 0)
    assert len(set(app.slot[res].tolist())) == res.sum()
    assert sorted(app.slot[res].tolist() + app.free) == list(range(n_slots))
