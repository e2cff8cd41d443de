"""Multi-app switching on a small pool: every LCTRU order bit-exact against the oracle, and the whole history of
evictions and loads replayed with the oracle's codec: arena records and resident KV must match bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import binding as B, synth
from paper_2403_11805_b200.multiapp import MultiApp
from gpu_helpers import bits_view, odesc

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("aot", [False, True], ids=["reclaim", "aot"])
def test_multiapp_history_matches_oracle_replay(aot):
    sh = synth.KVShape("apps", 2, 4, 4, 64, 128, 32, 64, window=8, seed=1, n_contexts=10)   # 4 chunks per context
    app = MultiApp(sh, n_slots=12, seed=1, log_ops=True, aot=aot)   # room for 3 contexts
    app.keep_sources = True
    app.build()
    served = [app.step(k=2) for _ in range(12)]
    app.finish()                                  # an ahead-of-time write-back of the last step may still be running
    assert all(len(s) == 2 for s in served)
    assert app.bytes_out > 0 and app.bytes_in > 0
    kinds = {op for op, _, _ in app.ops}
    if aot:   # everything that leaves was written back when its call returned: Reclaim never compresses
        assert "aot" in kinds and "drop" in kinds and "evict" not in kinds
    else:
        assert "evict" in kinds and "aot" not in kinds

    # (1) every eviction order is the oracle's order for the same table
    assert len(app.orders) > 5
    for table, order in app.orders:
        want = oracle.lctru_order(table.astype(oracle.STATE_DTYPE))
        assert np.array_equal(order, want)
        assert not table["locked"][order].any() and table["resident"][order].all()

    # (2) scores -> bits per context: same array through both rank -> bits implementations, tertile counts
    od_ctx = odesc(sh)
    for c in range(sh.n_contexts):
        kv = app.sources[c]
        q = synth.q_window(sh, sh.window, context=c)
        s64 = oracle.chunk_tolerance(od_ctx, bits_view(kv), bits_view(q), sh.window)
        ob, _ = oracle.assign_bits(s64.astype(np.float32), app.frac)
        assert sorted(app.bits[c].tolist()) == sorted(ob.tolist())

    # (3) replay the logged history with the oracle's codec
    CL = sh.chunk_len
    one = sh.with_(n_tokens=CL)                                  # a one-chunk tensor, to code chunks one at a time
    od_one = odesc(one)
    arena = {}
    for c in range(sh.n_contexts):
        src = bits_view(app.sources[c])
        for i in range(app.cpc):
            chunk = np.ascontiguousarray(src[..., i * CL:(i + 1) * CL, :])
            arena[c * app.cpc + i] = oracle.compress_chunks(od_one, chunk, [0], [app.bits[c][i]])
    pool = {}
    for op, row, slot in app.ops:
        if op == "load":
            buf, meta = arena[row]
            out = np.zeros((sh.n_layers, 2, sh.n_kv_heads, CL, sh.head_dim), dtype=np.uint16)
            oracle.decompress_chunks(od_one, buf, meta, out)
            pool[slot] = out
        elif op == "drop":
            pool.pop(slot)
        else:   # "evict" frees the slot after writing the record, "aot" writes it and stays
            bits = int(app.table["bits"][row])
            arena[row] = oracle.compress_chunks(od_one, pool[slot], [0], [bits])
            if op == "evict":
                pool.pop(slot)
    host_arena = app.arena.numpy()
    for row, (buf, meta) in arena.items():
        off = int(app.arena_off[row])
        assert np.array_equal(host_arena[off:off + buf.size], buf), row
        assert app.checksum[row] == meta[0]["checksum"]
    got_pool = bits_view(app.pool)
    for slot, want in pool.items():
        assert np.array_equal(got_pool[..., slot * CL:(slot + 1) * CL, :], want), slot
    # bookkeeping is consistent: resident rows own distinct slots, the rest of the pool is free
    res = app.slot >= 0
    assert np.array_equal(res, app.table["resident"] != 0)
    assert len(set(app.slot[res].tolist())) == res.sum() and sorted(app.slot[res].tolist() + app.free) == list(range(12))
    assert sorted(pool) == sorted(app.slot[res].tolist())


def test_multiapp_locked_contexts_are_never_evicted():
    sh = synth.KVShape("apps", 1, 2, 2, 64, 64, 16, 64, window=4, seed=1, n_contexts=6)
    app = MultiApp(sh, n_slots=8, seed=3, log_ops=True)          # 2 contexts of 4 chunks fit
    app.build()
    for _ in range(6):
        before = len(app.ops)
        ctxs = app.step(k=2)
        rows_served = {c * app.cpc + i for c in ctxs for i in range(app.cpc)}
        evicted = {row for op, row, _ in app.ops[before:] if op in ("evict", "drop")}
        assert not (evicted & rows_served)
        for c in ctxs:
            assert app.table["resident"][c * app.cpc:(c + 1) * app.cpc].all()
