"""Multi-app context switching on one GPU: many contexts share a pool of device chunk slots.

Follows Sec. 3.4 of the paper with pinned host memory in the place of the disk: chunks live compressed in a host
arena; a pool of chunk slots on the device holds the working sets.  Serving a context (callLLM) locks it, loads
its missing chunks (Load: host -> device copy, unpack + dequantize) and, when the pool is full, first evicts
chunks of other contexts in LCTRU order (Reclaim: quantize + pack, device -> host copy).  Everything that touches
data goes through the C-ABI calls of the binding; this module is only the bookkeeping of who sits where.

The pool is one KV tensor kv_pool[l][s][h][slot*chunk_len + t][c]: a slot is a chunk id of that tensor, so the
codec calls work on it unchanged.
"""
import numpy as np
import torch

from . import binding as B
from . import synth


class MultiApp:
    def __init__(self, shape, n_slots, frac=(1 / 3, 1 / 3, 1 / 3), seed=1, log_ops=False, aot=False):
        """shape: synth.KVShape of ONE context (n_contexts of them); n_slots: device pool size in chunks.
        aot: swap the served contexts out ahead of time, when the call returns (Sec. 3.4 i), so that a later
        Reclaim of their chunks costs nothing."""
        self.shape, self.n_slots, self.frac, self.seed, self.aot = shape, n_slots, frac, seed, aot
        self.n_ctx, self.cpc = shape.n_contexts, shape.n_chunks       # contexts, chunks per context
        self.desc_ctx = B.desc_of(shape)
        self.desc_pool = B.desc_of(shape, n_tokens=n_slots * shape.chunk_len)
        self.rec_bytes = {b: B.record_bytes(self.desc_pool, b) for b in (8, 4, 2)}
        L, H, d, CL = shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.chunk_len
        self.pool = torch.zeros(L, 2, H, n_slots * CL, d, dtype=torch.float16, device="cuda")
        self.main = torch.cuda.current_stream()
        self.side_out, self.side_in = torch.cuda.Stream(), torch.cuda.Stream()
        # host-side chunk table (rows of llms_chunk_state) and placement
        n = self.n_ctx * self.cpc
        self.table = np.zeros(n, dtype=B.STATE_DTYPE)
        self.table["ctx_id"] = np.repeat(np.arange(self.n_ctx), self.cpc)
        self.table["chunk_id"] = np.tile(np.arange(self.cpc), self.n_ctx)
        self.slot = np.full(n, -1, dtype=np.int64)
        self.free = list(range(n_slots - 1, -1, -1))
        self.checksum = np.zeros(n, dtype=np.uint32)
        self.clean = np.zeros(n, dtype=bool)      # the record in the arena matches what sits in the slot
        self.ready_ms = []                        # per step: time until the served contexts were resident
        self.arena_off = np.zeros(n, dtype=np.uint64)
        self.step_no = 0
        self.ops = [] if log_ops else None        # ("evict"|"load", row, slot) in execution order
        self.orders = [] if log_ops else None     # (table copy, order) of every LCTRU query
        self._pending = []                        # (meta, rows) of compress calls whose checksums are not read yet
        self._draw = 0
        self._aot_rows = None                     # rows whose ahead-of-time write-back may still be in flight
        self._ev_aot = None                       # recorded on the copy-out stream behind that write-back
        self.bytes_out = self.bytes_in = 0
        self.kernel_launches = 0                  # kernels launched by the codec calls

    # ------------------------------------------------------------------ set-up (untimed)
    def build(self):
        """Generate every context, score it, assign bit-widths, compress it into the arena; then make the
        first contexts resident."""
        sh, W = self.shape, self.shape.window
        scores = torch.empty(self.cpc, dtype=torch.float32, device="cuda")
        ws_t = torch.empty(B.tolerance_workspace_bytes(self.desc_ctx, W), dtype=torch.uint8, device="cuda")
        all_bits = np.zeros((self.n_ctx, self.cpc), dtype=np.uint8)
        kvs = []
        for c in range(self.n_ctx):
            kv = synth.kv_tensor(sh, device="cuda", context=c)
            q = synth.q_window(sh, W, device="cuda", context=c)
            B.chunk_tolerance(self.desc_ctx, kv, q, W, scores, ws_t)
            bits, _ = B.assign_bits(scores.cpu().numpy(), self.frac)
            all_bits[c] = bits
            kvs.append(kv.cpu() if self.keep_sources else None)
            self._place_in_arena(c, bits)
            self._first_compress(c, kv, bits)
        torch.cuda.synchronize()
        self._collect_checksums()
        self.sources = kvs
        self.bits = all_bits
        resident = self.n_slots // self.cpc
        for c in range(min(resident, self.n_ctx)):
            self._load(np.arange(c * self.cpc, (c + 1) * self.cpc))
        self._end_of_step()

    keep_sources = False

    def _place_in_arena(self, c, bits):
        """Fix the context's bit-widths and give each of its records a place of its own in the arena."""
        rows = np.arange(c * self.cpc, (c + 1) * self.cpc)
        self.table["bits"][rows] = bits
        cursor = 0 if c == 0 else int(self.arena_off[rows[0] - 1]) + self.rec_bytes[int(self.table["bits"][rows[0] - 1])]
        for r, b in zip(rows, bits):
            self.arena_off[r] = cursor
            cursor += self.rec_bytes[int(b)]

    def _alloc_buffers(self):
        if hasattr(self, "arena"):
            return
        worst = self.cpc * self.rec_bytes[8]
        # staging buffers on the way out: two take turns; with ahead-of-time swap-out one per context of a step, so
        # that all of a step's write-back kernels run at once and only their copies stay behind
        n_out = 8 if self.aot else 2
        self.stage_out = [torch.empty(worst, dtype=torch.uint8, device="cuda") for _ in range(n_out)]
        self.stage_in = [torch.empty(worst, dtype=torch.uint8, device="cuda") for _ in range(2)]
        self.ws = [torch.empty(B.codec_workspace_bytes(self.cpc), dtype=torch.uint8, device="cuda") for _ in range(64)]
        self.metas = [B.new_meta(self.cpc, pinned=True) for _ in range(64)]
        self._ws_next = 0
        self._used_ws = []
        self.ev_stage_out_free = [B.new_event() for _ in range(n_out)]
        self.ev_stage_in_free = [B.new_event() for _ in range(2)]
        self.ev_compressed = [B.new_event() for _ in range(n_out)]
        self.ev_landed = [B.new_event() for _ in range(2)]
        self._out_k = self._in_k = 0
        # the arena: every (context, chunk) record at its own offset, bit-widths fixed at set-up by the tertiles
        n8, n4, n2 = B.level_counts(self.cpc, self.frac)
        total = self.n_ctx * (n8 * self.rec_bytes[8] + n4 * self.rec_bytes[4] + n2 * self.rec_bytes[2])
        self.arena = torch.empty(total, dtype=torch.uint8).pin_memory()

    def _next_ws(self):
        i = self._ws_next % len(self.ws)
        self._ws_next += 1
        return self.ws[i], self.metas[i]

    def _first_compress(self, c, kv, bits):
        self._alloc_buffers()
        rows = np.arange(c * self.cpc, (c + 1) * self.cpc)
        ws, meta = self._next_ws()
        k = self._out_k % len(self.stage_out)
        self._out_k += 1
        self.main.wait_event(self.ev_stage_out_free[k])
        B.compress_chunks(self.desc_ctx, kv, np.arange(self.cpc, dtype=np.uint32), bits, self.stage_out[k], meta, ws)
        self.ev_compressed[k].record(self.main)
        B.swap_out(self.stage_out[k], meta, self.arena, host_offsets=self.arena_off[rows], side_stream=self.side_out,
                   after=self.ev_compressed[k], done=self.ev_stage_out_free[k], n=len(rows))
        self._pending.append((meta, rows))
        if len(self._pending) >= len(self.ws) - 2:
            torch.cuda.synchronize()
            self._collect_checksums()

    def _collect_checksums(self):
        for meta, rows in self._pending:
            self.checksum[rows] = meta["checksum"][:len(rows)]
        self._pending = []

    # ------------------------------------------------------------------ Reclaim and Load
    def _evict(self, rows):
        """Reclaim: chunks whose record in the arena is still valid are simply dropped; the others are
        quantized + packed out of their slots and their records copied to the arena first."""
        rows = np.asarray(rows)
        for r in rows[self.clean[rows]]:
            s = int(self.slot[r])
            if self.ops is not None:
                self.ops.append(("drop", int(r), s))
            self.free.append(s)
            self.slot[r] = -1
            self.table["resident"][r] = 0
        self._write_back(rows[~self.clean[rows]], release=True)

    def _write_back(self, rows, release):
        """Quantize + pack the chunks in `rows` and copy their records to the arena; release=True frees the
        slots (Reclaim), release=False leaves the chunks resident (ahead-of-time swap-out)."""
        for r0 in range(0, len(rows), self.cpc):
            part = rows[r0:r0 + self.cpc]
            slots = self.slot[part].astype(np.uint32)
            bits = self.table["bits"][part].astype(np.uint8)
            ws, meta = self._next_ws()
            k = self._out_k % len(self.stage_out)
            self._out_k += 1
            self.main.wait_event(self.ev_stage_out_free[k])
            B.compress_chunks(self.desc_pool, self.pool, slots, bits, self.stage_out[k], meta, ws)
            self.ev_compressed[k].record(self.main)
            B.swap_out(self.stage_out[k], meta, self.arena, host_offsets=self.arena_off[part], side_stream=self.side_out,
                       after=self.ev_compressed[k], done=self.ev_stage_out_free[k], n=len(part))
            self._pending.append((meta, part))
            self.bytes_out += int(sum(self.rec_bytes[int(b)] for b in bits))
            self.kernel_launches += B.codec_launches(self.desc_pool, bits)
            for r, s in zip(part, slots):
                if self.ops is not None:
                    self.ops.append(("evict" if release else "aot", int(r), int(s)))
                if release:
                    self.free.append(int(s))
            if release:
                self.slot[part] = -1
                self.table["resident"][part] = 0
            else:
                self.clean[part] = True

    def _settle_write_back(self):
        """Wait for the ahead-of-time write-back that was left running and take its checksums."""
        if self._aot_rows is not None:
            self._ev_aot.synchronize()
            self._collect_checksums()
            self._aot_rows = None

    def finish(self):
        """Everything queued has completed and every checksum is known on the host."""
        torch.cuda.synchronize()
        self._collect_checksums()
        self._aot_rows = None

    def _load(self, rows):
        """Load: copy the records of the chunks in `rows` from the arena, unpack + dequantize into free slots."""
        rows = np.asarray(rows)
        if self._aot_rows is not None and np.isin(rows, self._aot_rows).any():
            self._settle_write_back()             # a record still on its way out must land before it is read back
        for r0 in range(0, len(rows), self.cpc):
            part = rows[r0:r0 + self.cpc]
            slots = np.array([self.free.pop() for _ in part], dtype=np.uint32)
            bits = self.table["bits"][part]
            ws, meta = self._next_ws()
            meta = meta[:len(part)]
            sizes = np.array([self.rec_bytes[int(b)] for b in bits], dtype=np.uint64)
            meta["chunk_id"] = slots
            meta["bits"] = bits
            meta["offset"] = np.concatenate([[0], np.cumsum(sizes)[:-1]])
            meta["nbytes"] = sizes
            meta["n_groups"] = self.n_groups
            meta["checksum"] = self.checksum[part]
            k = self._in_k % 2
            self._in_k += 1
            B.swap_in(self.arena, meta, self.stage_in[k], host_offsets=self.arena_off[part], side_stream=self.side_in,
                      after=self.ev_stage_in_free[k], done=self.ev_landed[k])
            self.main.wait_event(self.ev_landed[k])
            B.decompress_chunks(self.desc_pool, self.stage_in[k], meta, None, self.pool, ws)
            self.ev_stage_in_free[k].record(self.main)
            self._used_ws.append(ws)
            self.bytes_in += int(sizes.sum())
            self.kernel_launches += B.codec_launches(self.desc_pool, bits)
            self.slot[part] = slots
            self.table["resident"][part] = 1
            self.clean[part] = True
            if self.ops is not None:
                self.ops.extend(("load", int(r), int(s)) for r, s in zip(part, slots))

    @property
    def n_groups(self):
        sh = self.shape
        return sh.n_slabs * sh.chunk_len * (sh.head_dim // sh.group_size)

    def _end_of_step(self):
        """One synchronisation per step: read back the checksums of this step's records, check the decoded ones."""
        torch.cuda.synchronize()
        self._collect_checksums()
        bad = sum(B.codec_corrupt_count(ws) for ws in self._used_ws)
        self._used_ws = []
        if bad:
            raise RuntimeError(f"{bad} records failed their checksum on the way in")

    # ------------------------------------------------------------------ one step of the trace
    def draw_contexts(self, k):
        """k distinct contexts that are not fully resident, uniformly (splitmix64 stream of the seed)."""
        resident = self.table["resident"].reshape(self.n_ctx, self.cpc).all(axis=1)
        cand = [c for c in range(self.n_ctx) if not resident[c]]
        picks = []
        while len(picks) < k and cand:
            z = synth.splitmix64_int((synth.stream_key(self.seed, 7) + self._draw * 0x9E3779B97F4A7C15) & ((1 << 64) - 1))
            self._draw += 1
            picks.append(cand.pop(z % len(cand)))
        return picks

    def step(self, k=8):
        """Serve k contexts: lock, evict in LCTRU order as far as needed, load, touch, unlock."""
        self.step_no += 1
        if not hasattr(self, "_ev_t0"):
            self._ev_t0, self._ev_ready = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self._ev_t0.record(self.main)
        ctxs = self.draw_contexts(k)
        locked_rows = np.concatenate([np.arange(c * self.cpc, (c + 1) * self.cpc) for c in ctxs])
        self.table["locked"][locked_rows] = 1            # working-set lock
        for c in ctxs:
            rows = np.arange(c * self.cpc, (c + 1) * self.cpc)
            missing = rows[self.table["resident"][rows] == 0]
            need = len(missing) - len(self.free)
            if need > 0:
                order = B.lctru_order(self.table)
                if self.orders is not None:
                    self.orders.append((self.table.copy(), order.copy()))
                if len(order) < need:
                    raise RuntimeError("pool too small for the locked working sets")
                self._evict(order[:need])
            if len(missing):
                self._load(missing)
            self.table["last_access_step"][rows] = self.step_no
        self._ev_ready.record(self.main)                 # the working sets are resident: inference could start
        self.clean[locked_rows] = False                  # a served context counts as modified by its call
        self.table["locked"][locked_rows] = 0
        self._end_of_step()                              # also settles the write-back left running by the step before
        self._aot_rows = None
        if self.aot:
            # ahead-of-time swap-out when the call returns (Sec. 3.4 i): queued now, left running, so that its
            # copies out share the link with the next step's copies in
            self._write_back(locked_rows, release=False)
            if self._ev_aot is None:
                self._ev_aot = B.new_event(self.side_out)
            self._ev_aot.record(self.side_out)
            self._aot_rows = locked_rows
        self.ready_ms.append(self._ev_t0.elapsed_time(self._ev_ready))
        return ctxs

    def context_kv(self, c):
        """The resident KV of context c gathered from its slots: fp16 [L, 2, H, T, d] (device)."""
        sh = self.shape
        rows = np.arange(c * self.cpc, (c + 1) * self.cpc)
        assert (self.slot[rows] >= 0).all()
        CL = sh.chunk_len
        parts = [self.pool[..., int(s) * CL:(int(s) + 1) * CL, :] for s in self.slot[rows]]
        return torch.cat(parts, dim=3)
