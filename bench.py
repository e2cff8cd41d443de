"""Throughput of the context-switching hot path on synthetic KV caches.

One step = one pass of the whole path over one context that is resident in HBM:
tolerance score (Eq. 1) -> rank -> bits on the host (Eq. 2) -> quantize + pack every chunk -> unpack + dequantize
every chunk.  `value` counts the fp16 bytes the codec processed (compress + decompress: 2 x the KV size) per
second of step time.  `e2e` runs compress -> swap-out to pinned host memory -> swap-in -> decompress through
the same C-ABI calls, with the host copies inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama7b] [--impl ours|reference]
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "KV compress+decompress GB/s (fp16 bytes)"
UNIT = "GB/s"


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=200)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="llama7b", help="a key of synth.CONFIGS (single-context workloads)")
    p.add_argument("--layers", type=int, default=0, help="use only this many layers (smaller cases for profiler captures)")
    p.add_argument("--chunk-len", type=int, default=0, help="override the workload's tokens per chunk (chunk-size sweep, Sec. 5.4)")
    p.add_argument("--levels", default="8,4,2", help="bit-widths of the three levels, top first (Sec. 3.2: 8,4,2 or 4,2,1)")
    p.add_argument("--e2e-steps", type=int, default=10)
    p.add_argument("--e2e-batches", type=int, default=16, help="batches of chunks the pipelined round trip is cut into")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-layerwise", dest="layerwise", action="store_false",
                   help="skip the layer-wise swap timing (records split per layer, Sec. 4: first layer ready / all layers ready)")
    p.add_argument("--fused-swap", action="store_true",
                   help="also time swap-out and swap-in without a staging buffer: the encoder writes into, the decoder reads "
                        "from page-locked host memory directly (e2e.fused_swap)")
    p.add_argument("--aot", action="store_true", help="multiapp: swap served contexts out ahead of time (Sec. 3.4 i)")
    p.add_argument("--quant-mode", type=int, default=0, choices=[0, 1],
                   help="0: groups of group_size channels of one token (the metric's setting); 1: one group per channel "
                        "across the chunk's tokens")
    return p.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# dram__bytes_read.sum + dram__bytes_write.sum of one codec launch on the full llama7b workload, from one ncu capture.
# Each figure is tied to the codec source it was taken with: when that source has changed since, the line reports null
# instead of a number that may no longer hold.
CODEC_SOURCES = ("paper_2403_11805_b200/csrc/codec.cu", "paper_2403_11805_b200/csrc/codec_cw.cuh",
                 "paper_2403_11805_b200/csrc/llms_internal.cuh")
NCU_DRAM_TRAFFIC = {
    "codec_sha256_16": "78c2b6ab0867d80c",      # hash of CODEC_SOURCES at the capture
    "source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of one full-size launch, commit 396a81d "
              "(profiles/codec_and_score_kernels_llama7b.md)",
    ("llama7b", 32, "compress_kernel"): 2149846528 + 646908672,
    ("llama7b", 32, "decompress_kernel"): 659665408 + 2085249792,
}


def codec_source_hash():
    import hashlib
    h = hashlib.sha256()
    for rel in CODEC_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_traffic(key):
    """The captured DRAM bytes of a launch, or None when there is no capture for it or the codec has changed since."""
    if codec_source_hash() != NCU_DRAM_TRAFFIC["codec_sha256_16"]:
        return None, "no capture for the codec source as it is now"
    return NCU_DRAM_TRAFFIC.get(key), NCU_DRAM_TRAFFIC["source"]


LEVELS = (8, 4, 2)      # set from --levels


class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons while the timed region runs."""
    FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(gpu_index), "-lms", "100"], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        self.t_begin = self.t_end = None

    def begin(self):
        self.t_begin = time.time()

    def end(self):
        self.t_end = time.time()

    def finish(self):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        rows = [r.strip().split(", ") for r in self.file.read().splitlines() if r.strip()]
        self.file.close()
        os.unlink(self.file.name)
        import datetime
        inside, every = [], []
        for r in rows:
            if len(r) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rec = (float(r[2]), float(r[3]), r[6:10])
            except ValueError:
                continue
            every.append(rec)
            if self.t_begin is not None and self.t_begin - 0.05 <= ts <= self.t_end + 0.05:
                inside.append(rec)
        use = inside if len(inside) >= 2 else every
        if not use:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for rec in use for i, v in enumerate(rec[2]) if v.strip().lower() == "active"})
        return {"sm_mhz": statistics.median(r[0] for r in use), "sm_max_mhz": use[0][1], "reasons": reasons,
                "samples": len(use), "in_timed_region": use is inside}


def run_reference(args):
    """The oracle, as it stands, on the host cores: score, rank -> bits, compress, decompress of a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import torch
    import oracle
    from paper_2403_11805_b200 import synth

    shape = synth.CONFIGS[args.workload]
    sample_layers = min(shape.n_layers, args.layers or 8)
    sh = shape.with_(n_layers=sample_layers)
    W = sh.window
    kv = synth.kv_tensor(sh).view(torch.int16).numpy().view(np.uint16)
    q = synth.q_window(sh, W).view(torch.int16).numpy().view(np.uint16)
    od = oracle.make_desc(sh.n_layers, sh.n_kv_heads, sh.n_q_heads, sh.head_dim, sh.n_tokens, sh.chunk_len, sh.group_size)
    frac = sh.frac if sh.frac is not None else (1 / 3, 1 / 3, 1 / 3)
    ids = np.arange(sh.n_chunks, dtype=np.uint32)
    out = np.zeros(kv.size, dtype=np.uint16).reshape(kv.shape)

    def step():
        scores = oracle.chunk_tolerance(od, kv, q, W)
        bits, _ = oracle.assign_levels(scores.astype(np.float32), frac, LEVELS)
        buf, meta = oracle.compress_chunks(od, kv, ids, bits)
        oracle.decompress_chunks(od, buf, meta, out)

    steps, warmup = max(1, min(args.steps, 5)), max(1, min(args.warmup, 1))
    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    value = 2 * sh.n_elements * 2 / dt / 1e9
    sample = f"{sample_layers} of {shape.n_layers} layers of the {shape.name} context per step, all {sh.n_chunks} chunks"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 codec decisions, f64 score", "data": "synthetic",
        "config": {"workload": shape.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline(shape, kv_dev, q_dev):
    """Oracle timed on this host on a bounded sample of the same workload (rank 0, N = 1)."""
    import numpy as np
    import torch
    import oracle

    sample_layers = min(shape.n_layers, 8)
    sh = shape.with_(n_layers=sample_layers)
    W = sh.window
    kv = kv_dev[:sample_layers].cpu().view(torch.int16).numpy().view(np.uint16)
    q = q_dev[:sample_layers].cpu().view(torch.int16).numpy().view(np.uint16)
    od = oracle.make_desc(sh.n_layers, sh.n_kv_heads, sh.n_q_heads, sh.head_dim, sh.n_tokens, sh.chunk_len, sh.group_size)
    frac = sh.frac if sh.frac is not None else (1 / 3, 1 / 3, 1 / 3)
    ids = np.arange(sh.n_chunks, dtype=np.uint32)
    out = np.zeros(kv.size, dtype=np.uint16).reshape(kv.shape)
    t0 = time.perf_counter()
    scores = oracle.chunk_tolerance(od, kv, q, W)
    bits, _ = oracle.assign_levels(scores.astype(np.float32), frac, LEVELS)
    t1 = time.perf_counter()
    buf, meta = oracle.compress_chunks(od, kv, ids, bits)
    t2 = time.perf_counter()
    oracle.decompress_chunks(od, buf, meta, out)
    t3 = time.perf_counter()
    nbytes = sh.n_elements * 2
    cores = oracle.num_threads()
    # the same on one thread, on a quarter of the sample
    one_layers = max(1, sample_layers // 4)
    sh1 = shape.with_(n_layers=one_layers)
    od1 = oracle.make_desc(sh1.n_layers, sh1.n_kv_heads, sh1.n_q_heads, sh1.head_dim, sh1.n_tokens, sh1.chunk_len, sh1.group_size)
    kv1, q1 = np.ascontiguousarray(kv[:one_layers]), np.ascontiguousarray(q[:one_layers])
    out1 = np.zeros(kv1.size, dtype=np.uint16).reshape(kv1.shape)
    oracle.set_num_threads(1)
    s0 = time.perf_counter()
    scores1 = oracle.chunk_tolerance(od1, kv1, q1, W)
    bits1, _ = oracle.assign_levels(scores1.astype(np.float32), frac, LEVELS)
    buf1, meta1 = oracle.compress_chunks(od1, kv1, ids, bits1)
    oracle.decompress_chunks(od1, buf1, meta1, out1)
    s1 = time.perf_counter()
    oracle.set_num_threads(cores)
    return {
        "value": 2 * nbytes / (t3 - t0) / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
        "sample": f"{sample_layers} of {shape.n_layers} layers, all {sh.n_chunks} chunks, one pass",
        "score_s": t1 - t0, "compress_gbs": nbytes / (t2 - t1) / 1e9, "decompress_gbs": nbytes / (t3 - t2) / 1e9,
        "single_thread": {"value": 2 * sh1.n_elements * 2 / (s1 - s0) / 1e9, "unit": UNIT,
                          "sample": f"{one_layers} of {shape.n_layers} layers, all {sh1.n_chunks} chunks, one pass"},
        "host_cores_available": len(os.sched_getaffinity(0)),
    }


def run_ours(args):
    import numpy as np
    import torch
    from paper_2403_11805_b200 import binding as B, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} was started with WORLD_SIZE={world}: one rank per GPU is expected")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.lib()

    shape = synth.CONFIGS[args.workload]
    if args.layers:
        shape = shape.with_(n_layers=args.layers)
    if args.chunk_len:
        shape = shape.with_(chunk_len=args.chunk_len)
    W = shape.window
    frac = shape.frac if shape.frac is not None else (1 / 3, 1 / 3, 1 / 3)
    # every rank owns one context of the workload (contexts are independent: no data-path collective)
    from paper_2403_11805_b200 import sharding
    my_context = sharding.contexts_of_rank(world, rank, world)[0]
    kv = synth.kv_tensor(shape, device="cuda", context=my_context)
    q_win = synth.q_window(shape, W, device="cuda", context=my_context)
    d = B.desc_of(shape, quant_mode=args.quant_mode)
    n = shape.n_chunks
    ids = np.arange(n, dtype=np.uint32)
    n8, n4, n2 = B.level_counts(n, frac, LEVELS)          # what the rank -> bits rule gives each level
    worst_bits = np.full(n, 8, dtype=np.uint8)
    buf = torch.empty(B.compressed_size(d, worst_bits), dtype=torch.uint8, device="cuda")
    kv_out = torch.empty_like(kv)
    scores = torch.empty(n, dtype=torch.float32, device="cuda")
    scores_host = torch.empty(n, dtype=torch.float32).pin_memory()
    ws_tol = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    ws = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    ws_dec = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    meta = B.new_meta(n, pinned=True)
    stream = torch.cuda.current_stream()
    state = {}

    frac_a = np.asarray(frac, dtype=np.float32)
    levels_a = np.asarray(LEVELS, dtype=np.uint8)
    bits = B.new_pinned(n)
    planned = B.new_event()

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        # score -> rank -> levels -> chunk table -> records, as one library call; scores, levels and meta are
        # page-locked, so a kernel does the ranking and nothing synchronises.  The event sits behind that kernel.
        after = ev[1] if ev else planned
        B.compress_context(d, kv, q_win, W, frac_a, levels_a, scores, scores_host, bits, buf, meta, ws_tol, ws,
                           after_scores=after)
        if ev:
            ev[2].record(stream)
        # the decode call reads sizes and offsets from meta on the host: wait for the ranking (the encoder runs on);
        # the expected checksums are read by the device in stream order
        B.wait(after)
        B.decompress_chunks_ordered(d, buf, meta, None, kv_out, ws_dec)
        if ev:
            ev[3].record(stream)
        state["bits"] = bits

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    assert B.codec_corrupt_count(ws_dec) == 0
    bits = state["bits"]
    assert tuple(int((bits == b).sum()) for b in LEVELS) == (n8, n4, n2)
    record_bytes = B.compressed_size(d, bits)

    sampler = ClockSampler(local_rank) if rank == 0 else None
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    for e in events:
        e[1].record(stream)                      # the library records this one: give it its handle first
    barrier()
    if sampler:
        sampler.begin()
    t_wall = time.perf_counter()
    for k in range(args.steps):
        step(events[k])
    barrier()
    t_wall = time.perf_counter() - t_wall
    if sampler:
        sampler.end()
    span_ms = events[0][0].elapsed_time(events[-1][3])
    tol_ms = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
    comp_ms = sum(e[1].elapsed_time(e[2]) for e in events) / args.steps
    decomp_ms = sum(e[2].elapsed_time(e[3]) for e in events) / args.steps
    ms_per_step = span_ms / args.steps
    step_ms = sorted(e[0].elapsed_time(e[3]) for e in events)       # each step by itself (mean above: the whole span)
    ms_per_step, tol_ms, comp_ms, decomp_ms = sharding.max_over_ranks([ms_per_step, tol_ms, comp_ms, decomp_ms], dist, "cuda")
    kv_bytes = shape.n_elements * 2
    value = world * 2 * kv_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- every codec launch by itself: the chunks of one level go through one compress call and one decompress call
    # (one codec kernel each, plus the few-microsecond checksum kernel), bracketed by events on the launching stream.
    # Each launch reads or writes its level's share of the fp16 KV (a third of 2 GiB on the metric's workload: larger than L2).
    per_launch = []
    reps = max(3, min(20, args.steps))
    for b in LEVELS:
        sel = ids[bits == b]
        if len(sel) == 0:
            continue
        sel_bits = np.full(len(sel), b, dtype=np.uint8)
        sel_meta = B.new_meta(len(sel), pinned=True)
        launch_bytes = len(sel) * shape.n_slabs * shape.chunk_len * shape.head_dim * 2 + B.compressed_size(d, sel_bits)
        for which in ("compress_kernel", "decompress_kernel"):
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps + 3)]
            for e0, e1 in evs:
                e0.record(stream)
                if which == "compress_kernel":
                    B.compress_chunks(d, kv, sel, sel_bits, buf, sel_meta, ws)
                else:
                    B.decompress_chunks_ordered(d, buf, sel_meta, None, kv_out, ws_dec)
                e1.record(stream)
            torch.cuda.synchronize()
            ms = sum(e0.elapsed_time(e1) for e0, e1 in evs[3:]) / reps
            ms = sharding.max_over_ranks([ms], dist, "cuda")[0]
            per_launch.append({"kernel": which, "bits": int(b), "chunks": int(len(sel)), "ms": ms,
                               "algorithmic_bytes": int(launch_bytes), "gbs": launch_bytes / (ms * 1e-3) / 1e9})
        assert B.codec_corrupt_count(ws_dec) == 0

    # ---- what a plain stream of the codec's access shape reaches on this GPU, per read:write mix (the encoder reads
    # about four bytes per byte written, the decoder the reverse): context for the roofline fractions
    def stream_ceiling(read_kib, write_kib, reps=6, split=None):
        per_iter = (read_kib + write_kib) * 1024
        iters = min(kv.numel() * 2 // (max(read_kib, 1) * 1024), kv_out.numel() * 2 // (max(write_kib, 1) * 1024))
        best = None
        for it in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            B.stream_probe(kv, kv_out, iters, read_kib, write_kib, split=split)
            e1.record(stream)
            torch.cuda.synchronize()
            if it >= 2:
                ms = e0.elapsed_time(e1)
                best = ms if best is None else min(best, ms)
        return iters * per_iter / (best * 1e-3) / 1e9

    mix = {"read_only": stream_ceiling(4, 0), "write_only": stream_ceiling(0, 4), "read4_write1": stream_ceiling(4, 1),
           "read1_write4": stream_ceiling(1, 4), "read1_write1": stream_ceiling(2, 2)}
    mix = {k: -sharding.max_over_ranks([-v], dist, "cuda")[0] for k, v in mix.items()}
    # the same two mixes under the work splits a persistent kernel can have: resident CTAs with a fixed split (what the
    # codec kernels had at first) and resident CTAs whose warps draw their iterations from counters (what they have now)
    by_split = {name: {"resident_ctas_fixed_split": stream_ceiling(r, w, split=1),
                       "resident_ctas_drawn_split": stream_ceiling(r, w, split=2)}
                for name, (r, w) in (("read4_write1", (4, 1)), ("read1_write4", (1, 4)))}
    by_split = {m: {k: -sharding.max_over_ranks([-v], dist, "cuda")[0] for k, v in d.items()} for m, d in by_split.items()}

    # ---- end to end: compress -> swap-out -> swap-in -> decompress with the pinned arena in the loop.
    # The chunks go in batches: while batch j travels to the host, batch j-1 is already on its way back and batch
    # j-2 is being decoded (the two copy directions and the kernels overlap); "serial" does one batch of everything.
    arena = torch.empty(record_bytes, dtype=torch.uint8).pin_memory()
    back = torch.empty(record_bytes, dtype=torch.uint8, device="cuda")
    side_out, side_in = torch.cuda.Stream(), torch.cuda.Stream()

    def make_plan(batch):
        plan, off = [], 0
        for j0 in range(0, n, batch):
            sl = slice(j0, min(n, j0 + batch))
            nbytes = B.compressed_size(d, bits[sl])
            plan.append({"ids": ids[sl], "bits": bits[sl], "off": off, "nbytes": nbytes,
                         "meta": B.new_meta(sl.stop - sl.start, pinned=True),
                         "ws": torch.empty(B.codec_workspace_bytes(sl.stop - sl.start), dtype=torch.uint8, device="cuda"),
                         "ev_c": B.new_event(), "ev_out": B.new_event(), "ev_in": B.new_event()})
            off += nbytes
        return plan

    def e2e_step(plan):
        for p_ in plan:
            sl = slice(p_["off"], p_["off"] + p_["nbytes"])
            B.compress_chunks(d, kv, p_["ids"], p_["bits"], buf[sl], p_["meta"], p_["ws"])
            p_["ev_c"].record(stream)
            B.swap_out(buf[sl], p_["meta"], arena[sl], side_stream=side_out, after=p_["ev_c"], done=p_["ev_out"], n=len(p_["ids"]))
            # sizes and offsets are already in the host meta; the checksums arrive with ev_c
            B.swap_in(arena[sl], p_["meta"], back[sl], side_stream=side_in, after=p_["ev_out"], done=p_["ev_in"], n=len(p_["ids"]))
        for p_ in plan:
            sl = slice(p_["off"], p_["off"] + p_["nbytes"])
            stream.wait_event(p_["ev_in"])
            # the pinned meta's checksums are read by the device in stream order: no host wait per batch
            B.decompress_chunks_ordered(d, back[sl], p_["meta"], None, kv_out, p_["ws"])
        stream.synchronize()                     # the next step's compress calls rewrite the meta arrays

    def time_e2e(plan):
        for _ in range(3):
            e2e_step(plan)
        for p_ in plan:
            assert B.codec_corrupt_count(p_["ws"]) == 0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step(plan)
        e1.record(stream)
        barrier()
        return sharding.max_over_ranks([e0.elapsed_time(e1) / args.e2e_steps], dist, "cuda")[0]

    # ---- what the host link gives a bare copy of the same bytes: one way each, then both ways at once
    def time_copies(pairs):
        streams = [side_out, side_in][:len(pairs)]
        best = None
        for it in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for st, (dst, src) in zip(streams, pairs):
                st.wait_event(e0)
                with torch.cuda.stream(st):
                    dst.copy_(src, non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(st)
                stream.wait_event(ev)
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            if it >= 2:
                best = ms if best is None else min(best, ms)
        return record_bytes / (best * 1e-3) / 1e9

    arena2 = torch.empty(record_bytes, dtype=torch.uint8).pin_memory()
    link = {"d2h_gbs": time_copies([(arena, buf[:record_bytes])]), "h2d_gbs": time_copies([(back, arena2)]),
            "both_at_once_gbs_each_way": time_copies([(arena, buf[:record_bytes]), (back, arena2)]),
            "what": "bare cudaMemcpyAsync of the records' bytes between device and pinned host memory, best of 4"}
    del arena2
    # the slowest rank's link counts
    link = {k: (-sharding.max_over_ranks([-v], dist, "cuda")[0] if isinstance(v, float) else v) for k, v in link.items()}

    e2e_batch = max(1, n // max(1, args.e2e_batches))
    e2e_serial_ms = time_e2e(make_plan(n))
    e2e_ms = time_e2e(make_plan(e2e_batch))
    e2e_value = world * 2 * kv_bytes / (e2e_ms * 1e-3) / 1e9

    # ---- swap without a staging buffer: the kernels work straight on the page-locked arena, against kernel + copy engine
    fused_swap = None
    if args.fused_swap:
        p_ = make_plan(n)[0]
        def timed(fn, reps=5):
            ts = []
            for it in range(reps + 2):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record(stream)
                fn()
                e1.record(stream)
                torch.cuda.synchronize()
                if it >= 2:
                    ts.append(e0.elapsed_time(e1))
            return statistics.median(ts)

        def staged_out():
            B.compress_chunks(d, kv, p_["ids"], p_["bits"], buf, p_["meta"], p_["ws"])
            p_["ev_c"].record(stream)
            B.swap_out(buf[:record_bytes], p_["meta"], arena, side_stream=side_out, after=p_["ev_c"], done=p_["ev_out"], n=n)
            stream.wait_event(p_["ev_out"])

        def staged_in():
            p_["ev_out"].record(stream)
            B.swap_in(arena, p_["meta"], back, side_stream=side_in, after=p_["ev_out"], done=p_["ev_in"], n=n)
            stream.wait_event(p_["ev_in"])
            B.decompress_chunks(d, back, p_["meta"], None, kv_out, p_["ws"])

        fused_swap = {
            "swap_out_staged_ms": timed(staged_out),
            "swap_out_fused_ms": timed(lambda: B.compress_chunks(d, kv, p_["ids"], p_["bits"], arena, p_["meta"], p_["ws"])),
            "swap_in_staged_ms": timed(staged_in),
            "swap_in_fused_ms": timed(lambda: B.decompress_chunks(d, arena, p_["meta"], None, kv_out, p_["ws"])),
            "what": "whole context in one call; staged = codec kernel on a device buffer + copy engine, fused = the codec "
                    "kernel reads or writes the page-locked arena itself"}
        assert B.codec_corrupt_count(p_["ws"]) == 0

    # ---- layer-wise load (Sec. 4): records split per layer; how soon is the first layer usable, when the last
    layerwise = None
    if args.e2e_steps > 0 and args.layerwise:
        from paper_2403_11805_b200.layerwise import LayerwiseContext
        p_ = make_plan(n)[0]                         # the whole context as one batch, for comparison
        B.compress_chunks(d, kv, p_["ids"], p_["bits"], buf, p_["meta"], p_["ws"])
        arena.copy_(buf[:record_bytes], non_blocking=True)
        torch.cuda.synchronize()
        whole = []
        for it in range(3 + args.e2e_steps):
            w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            w0.record(stream)
            p_["ev_out"].record(stream)
            B.swap_in(arena, p_["meta"], back, side_stream=side_in, after=p_["ev_out"], done=p_["ev_in"], n=n)
            stream.wait_event(p_["ev_in"])
            B.decompress_chunks(d, back, p_["meta"], None, kv_out, p_["ws"])
            w1.record(stream)
            torch.cuda.synchronize()
            if it >= 3:
                whole.append(w0.elapsed_time(w1))
        del back, arena
        lw = LayerwiseContext(shape, bits, quant_mode=args.quant_mode)
        first, last, out_ms = [], [], []
        for it in range(3 + args.e2e_steps):
            o0, o1, i0 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            o0.record(stream)
            lw.swap_out(kv)
            lw.side_out.synchronize()
            o1.record(stream)
            torch.cuda.synchronize()
            i0.record(stream)
            lw.swap_in(kv_out)
            torch.cuda.synchronize()
            if it >= 3:
                out_ms.append(o0.elapsed_time(o1))
                first.append(i0.elapsed_time(lw.ready[0]))
                last.append(i0.elapsed_time(lw.ready[-1]))
        assert lw.corrupt_count() == 0
        layerwise = {"first_layer_ready_ms": sharding.max_over_ranks([statistics.median(first)], dist, "cuda")[0],
                     "all_layers_ready_ms": sharding.max_over_ranks([statistics.median(last)], dist, "cuda")[0],
                     "swap_out_ms": sharding.max_over_ranks([statistics.median(out_ms)], dist, "cuda")[0],
                     "records": "one per (layer, chunk); a layer's records travel as one copy",
                     "whole_context_load_ms": sharding.max_over_ranks([statistics.median(whole)], dist, "cuda")[0]}
    clocks = sampler.finish() if sampler else None

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant codec kernel (algorithmic bytes per launch / measured launch time)
    peak, peak_kind = measured_peaks()
    algo_bytes = kv_bytes + record_bytes             # compress: fp16 read + record written; decompress: the reverse
    k_ms = {"compress_kernel": comp_ms, "decompress_kernel": decomp_ms}
    dominant = max(k_ms, key=k_ms.get)
    achieved = algo_bytes / (k_ms[dominant] * 1e-3) / 1e9
    if args.quant_mode == 0 and LEVELS == (8, 4, 2) and not args.chunk_len:
        traffic, traffic_source = measured_traffic((shape.name, shape.n_layers, dominant))
    else:
        traffic, traffic_source = None, "no capture for this workload"
    # the score stage: K read once, one float of softmax statistics per (segment, row) written by the logits kernel
    # and read back once by the column kernel (a pass over them for the row sums, where one is needed, is not counted)
    rows = shape.n_layers * shape.n_q_heads * W
    seg = 1
    while seg < 32 and shape.chunk_len % (seg * 2) == 0:
        seg *= 2
    stat_bytes = rows * ((shape.n_tokens + seg - 1) // seg) * 4
    score_bytes = kv_bytes // 2 + 2 * stat_bytes
    roofline = {
        "kernel": dominant, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "peak_source": f"{peak_kind} copy bandwidth", "launches_per_stage": B.codec_launches(d, bits) - (1 if args.quant_mode == 1 else 0),
        "traffic": traffic, "traffic_source": traffic_source,
        "algorithmic_bytes_per_launch": algo_bytes,
        # plain streams with the codec's access shape, GB/s of bytes read + written, best of 4 launches over this
        # workload's buffers; the dominant kernel's own mix beside it
        "stream_ceilings_gbs": mix, "stream_by_work_split_gbs": by_split,
        "frac_of_stream_with_its_mix": achieved / mix["read4_write1" if dominant == "compress_kernel" else "read1_write4"],
        "frac_of_nominal_8000": achieved / 8000.0,
        # each codec launch timed alone (events around one call = one codec kernel + its checksum kernel)
        "per_launch": [dict(pl, frac=pl["gbs"] / peak) for pl in per_launch],
        "score": {"what": "score stage: K read once + softmax statistics written and read back; stage time includes the ranking kernel",
                  "bytes": score_bytes, "k_bytes": kv_bytes // 2, "ms": tol_ms,
                  "achieved": score_bytes / (tol_ms * 1e-3) / 1e9, "frac": score_bytes / (tol_ms * 1e-3) / 1e9 / peak,
                  "frac_k_only": (kv_bytes // 2) / (tol_ms * 1e-3) / 1e9 / peak},
        "per_stage": {
            "tolerance_ms": tol_ms, "compress_ms": comp_ms, "decompress_ms": decomp_ms,
            "tolerance_gbs_of_K_read": (kv_bytes / 2) / (tol_ms * 1e-3) / 1e9,
            "compress_algorithmic_gbs": algo_bytes / (comp_ms * 1e-3) / 1e9,
            "decompress_algorithmic_gbs": algo_bytes / (decomp_ms * 1e-3) / 1e9,
            "compress_fp16_gbs": kv_bytes / (comp_ms * 1e-3) / 1e9,
            "decompress_fp16_gbs": kv_bytes / (decomp_ms * 1e-3) / 1e9,
            "codec_only_fp16_gbs": 2 * kv_bytes / ((comp_ms + decomp_ms) * 1e-3) / 1e9,
        },
    }
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 (fp16 in/out, integer codes)", "data": "synthetic",
        "config": {"workload": shape.name, "layers": shape.n_layers, "kv_heads": shape.n_kv_heads, "head_dim": shape.head_dim,
                   "tokens": shape.n_tokens, "chunk_len": shape.chunk_len, "group_size": shape.group_size,
                   "window": W, "levels": list(LEVELS), "chunks_per_level": [n8, n4, n2], "contexts_per_gpu": 1, "quant_mode": args.quant_mode,
                   "l2": "inputs larger than L2 (fp16 KV %.0f MiB per context)" % (kv_bytes / 2 ** 20),
                   "step": "score + rank->bits + compress + decompress of one context"},
        "contexts_per_s": world / (ms_per_step * 1e-3),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": record_bytes, "d2h_bytes_per_step": record_bytes,
                "ms_per_step": e2e_ms, "context_switches_per_s": world / (e2e_ms * 1e-3),
                "host_copy_gbs_each_way": record_bytes / (e2e_ms * 1e-3) / 1e9,
                "link_gbs": link,
                "frac_of_link": record_bytes / (e2e_ms * 1e-3) / 1e9 / link["both_at_once_gbs_each_way"],
                "serial_ms_per_step": e2e_serial_ms, "batch_chunks": e2e_batch,
                "what": "compress -> swap-out to pinned host -> swap-in -> decompress, pipelined in batches of chunks",
                "layerwise_load": layerwise, "fused_swap": fused_swap},
        # score kernels (logits, column sums + chunk means; a row pass in between for more than 16 rows per KV head),
        # the ranking kernel, then one codec kernel per call (channel-wise mode: one per bit-width and one for the sums)
        "gpu_launches": args.steps * ((2 if shape.n_q_heads // shape.n_kv_heads * W <= 16 and shape.chunk_len % 16 == 0 else 3)
                                      + 1 + 2 * B.codec_launches(d, bits)),
        "roofline": roofline, "clocks": clocks,
        "wall_ms_per_step": t_wall * 1e3 / args.steps,
        "step_ms_median_best": [statistics.median(step_ms), step_ms[0]],
    }
    if world == 1 and not args.no_cpu_baseline and args.quant_mode == 0:
        line["cpu_baseline"] = cpu_baseline(shape, kv, q_win)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_multiapp(args):
    """Config 4: 64 contexts of 1024 tokens share a device pool of 512 chunk slots; every step serves 8 contexts that
    are not resident (LCTRU eviction with compress + copy out, copy in + decompress).  Metric: context switches/s."""
    import torch
    from paper_2403_11805_b200 import binding as B, synth
    from paper_2403_11805_b200.multiapp import MultiApp

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    B.lib()
    shape = synth.CONFIGS["multiapp"]
    if args.layers:
        shape = shape.with_(n_layers=args.layers)
    per_step, n_slots = 8, 512
    app = MultiApp(shape, n_slots=n_slots, seed=shape.seed, aot=args.aot)
    app.build()
    for _ in range(max(args.warmup, 3)):
        app.step(per_step)
    steps = min(args.steps, 100)
    sampler = ClockSampler(0)
    out0, in0, launches0 = app.bytes_out, app.bytes_in, app.kernel_launches
    torch.cuda.synchronize()
    sampler.begin()
    t0 = time.perf_counter()
    for _ in range(steps):
        app.step(per_step)              # ends with a device synchronisation (an ahead-of-time write-back runs on)
    app.finish()
    dt = time.perf_counter() - t0
    sampler.end()
    clocks = sampler.finish()
    chunk_bytes = shape.n_slabs * shape.chunk_len * shape.head_dim * 2
    chunks_moved = (app.bytes_in - in0) / (sum(app.rec_bytes.values()) / 3)
    line = {
        "metric": "context switches/sec", "value": per_step * steps / dt, "unit": "contexts/s", "n_gpus": 1, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": dt * 1e3 / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 (fp16 in/out, integer codes)", "data": "synthetic",
        "config": {"workload": shape.name, "contexts": shape.n_contexts, "tokens_per_context": shape.n_tokens,
                   "chunk_len": shape.chunk_len, "layers": shape.n_layers, "pool_slots": n_slots, "contexts_per_step": per_step,
                   "l2": "pool of %.0f MiB, far larger than L2" % (n_slots * chunk_bytes / 2 ** 20)},
        "e2e": {"value": per_step * steps / dt, "unit": "contexts/s",
                "h2d_bytes_per_step": (app.bytes_in - in0) // steps, "d2h_bytes_per_step": (app.bytes_out - out0) // steps,
                "h2d_gbs": (app.bytes_in - in0) / dt / 1e9, "d2h_gbs": (app.bytes_out - out0) / dt / 1e9,
                "what": "LCTRU eviction (compress + copy out) and load (copy in + decompress) per step, wall clock"},
        "fp16_gbs_through_codec": 2 * chunks_moved * chunk_bytes / dt / 1e9,
        "aot_swap_out": bool(args.aot),
        "switch_latency_ms": statistics.mean(app.ready_ms[-steps:]),   # step start until the 8 working sets are resident
        "gpu_launches": app.kernel_launches - launches0, "clocks": clocks,
    }
    print(json.dumps(line))


def main():
    global LEVELS
    args = parse_args()
    LEVELS = tuple(int(x) for x in args.levels.split(","))
    assert len(LEVELS) == 3
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as one plain process: become the launcher of args.gpus ranks, one per GPU, and relay their exit code
        import torch
        from paper_2403_11805_b200 import sharding
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"bench.py --gpus {args.gpus}: only {torch.cuda.device_count()} CUDA devices are visible")
        sys.exit(sharding.launch_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    elif args.workload == "multiapp":
        run_multiapp(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
