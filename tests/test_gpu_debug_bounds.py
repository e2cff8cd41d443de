"""The checked build of the library (a bounds check in front of every access the group-wise codec kernels make to the KV
tensor and the swap buffer): contexts of several shapes go through compress and decompress in a process of its own
that loads that build, the records equal the oracle's, and no access fell outside its call's buffers; then the swap
buffer is declared shorter than it is and the check has to catch the stores into its end.

The checked build is made by `python -m paper_2403_11805_b200.build --debug-bounds` (the build entry point of the
repository makes it too); where it is missing or older than the sources the test is skipped."""
import json
import os
import subprocess
import sys

import pytest

from paper_2403_11805_b200 import build as gpu_build

pytestmark = pytest.mark.gpu

CHILD = r"""
import json, sys
import numpy as np, torch
import oracle
from paper_2403_11805_b200 import binding as B, synth
sys.path.insert(0, "tests")
from gpu_helpers import bits_view, odesc

assert B.debug_bounds()[0] == 1, "not the checked build"
shapes = [synth.CONFIGS["tiny"],
          synth.KVShape("short_slabs", 2, 2, 2, 64, 96, 4, 64, seed=3),        # several slabs per unit
          synth.KVShape("ragged", 1, 2, 2, 64, 600, 40, 32, seed=4),           # a pass and a tail per slab
          synth.CONFIGS["llama7b"].with_(n_layers=1, n_tokens=512)]
cases = 0
for sh in shapes:
    kv = synth.kv_tensor(sh)
    kv_dev = kv.cuda()
    d = B.desc_of(sh)
    n = sh.n_chunks
    for levels in ((8, 4, 2), (1, 1, 1)):
        bits = np.array([levels[i % 3] for i in range(n)], dtype=np.uint8)
        ids = np.arange(n, dtype=np.uint32)
        total = B.compressed_size(d, bits)
        buf = torch.zeros(total, dtype=torch.uint8, device="cuda")          # exactly as long as the records
        meta = B.new_meta(n, pinned=True)
        ws = torch.empty(B.codec_workspace_bytes(n), dtype=torch.uint8, device="cuda")
        out = torch.zeros_like(kv_dev)
        B.compress_chunks(d, kv_dev, ids, bits, buf, meta, ws, out_bytes=total)
        torch.cuda.synchronize()
        B.decompress_chunks(d, buf, meta, None, out, ws)
        assert B.codec_corrupt_count(ws) == 0
        want_buf, want_meta = oracle.compress_chunks(odesc(sh), bits_view(kv), ids, bits)
        assert np.array_equal(buf.cpu().numpy(), want_buf)
        want = np.zeros(bits_view(kv).shape, dtype=np.uint16)
        oracle.decompress_chunks(odesc(sh), want_buf, want_meta, want)
        assert np.array_equal(bits_view(out), want)
        cases += 1
compiled_in, violations, first = B.debug_bounds()
# the check itself: with the swap buffer declared 1 KiB shorter than it is, the stores into its last KiB are counted
# (and skipped: every address involved is valid memory either way)
import ctypes
B.lib().llms_debug_shrink_swap_range.argtypes = [ctypes.c_uint64]
B.lib().llms_debug_shrink_swap_range.restype = None
B.lib().llms_debug_shrink_swap_range(1024)
B.compress_chunks(d, kv_dev, ids, bits, buf, meta, ws, out_bytes=total)
torch.cuda.synchronize()
B.lib().llms_debug_shrink_swap_range(0)
_, caught, caught_at = B.debug_bounds()
end = buf.data_ptr() + total
print(json.dumps({"compiled_in": compiled_in, "violations": violations, "first_address": first, "cases": cases,
                  "caught": caught - violations, "caught_inside_last_kib": end - 1024 <= caught_at < end}))
"""


def test_codec_kernels_stay_inside_their_buffers():
    lib = gpu_build.DEBUG_LIB
    if not os.path.exists(lib) or os.path.getmtime(lib) < gpu_build._newest_input():
        pytest.skip("the checked build is missing or stale: python -m paper_2403_11805_b200.build --debug-bounds")
    env = dict(os.environ, LLMS_LIBRARY=lib)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    done = subprocess.run([sys.executable, "-c", CHILD], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert done.returncode == 0, done.stderr[-2000:]
    report = json.loads(done.stdout.strip().splitlines()[-1])
    assert report["compiled_in"] == 1 and report["cases"] == 8
    assert report["violations"] == 0, hex(report["first_address"])
    assert report["caught"] > 0 and report["caught_inside_last_kib"]
