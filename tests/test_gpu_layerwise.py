"""Layer-wise swap (Sec. 4, I/O half of the layer-wise pipeline): every layer's records in the arena, their
checksums and the reloaded KV against the CPU oracle run on one-layer views of the same tensor, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import synth
from paper_2403_11805_b200.layerwise import LayerwiseContext
from gpu_helpers import assert_meta_equal, bits_view, first_mismatch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [0, 1])
def test_layerwise_round_trip_matches_oracle_per_layer(mode):
    sh = synth.KVShape("lw", 5, 2, 4, 64, 160, 16, 64, seed=21)     # odd layer count: both staging buffers wrap
    kv = synth.kv_tensor(sh)
    bits = synth.random_bits(sh.n_chunks, 3).numpy()
    kv_dev = kv.cuda()
    ctx = LayerwiseContext(sh, bits, quant_mode=mode)
    ctx.swap_out(kv_dev)
    torch.cuda.synchronize()
    out = torch.full(kv.shape, float("nan"), dtype=torch.float16, device="cuda")
    ctx.swap_in(out)
    assert ctx.corrupt_count() == 0
    d1 = oracle.make_desc(1, sh.n_kv_heads, sh.n_q_heads, sh.head_dim, sh.n_tokens, sh.chunk_len, sh.group_size, mode)
    ids = np.arange(sh.n_chunks)
    got = bits_view(out)
    for l in range(sh.n_layers):
        want_buf, want_meta = oracle.compress_chunks(d1, bits_view(kv[l]), ids, bits)
        assert first_mismatch(ctx.layer_arena(l).numpy(), want_buf) is None, f"layer {l}"
        assert_meta_equal(ctx.meta[l], want_meta)
        want = np.full(kv[l].numel(), 0x7E00, dtype=np.uint16).reshape(kv[l].shape)
        oracle.decompress_chunks(d1, want_buf, want_meta, want)
        assert first_mismatch(got[l].reshape(-1), want.reshape(-1)) is None, f"layer {l}"
    # the per-layer events fire in layer order
    times = [ctx.ready[0].elapsed_time(ctx.ready[l]) for l in range(1, sh.n_layers)]
    assert all(t >= 0 for t in times)


def test_layerwise_decodes_the_same_values_as_whole_context_records():
    """Groups never cross a layer, so splitting the records by layer changes where bytes sit, not what is decoded."""
    from paper_2403_11805_b200 import binding as B
    from gpu_helpers import gpu_compress, gpu_decompress
    sh = synth.KVShape("lw2", 3, 2, 2, 64, 96, 32, 32, seed=5)
    kv = synth.kv_tensor(sh).cuda()
    bits = synth.random_bits(sh.n_chunks, 9).numpy()
    _, meta, buf_dev = gpu_compress(sh, kv, np.arange(sh.n_chunks), bits)
    whole = torch.zeros_like(kv)
    assert gpu_decompress(sh, buf_dev, meta, whole) == 0
    ctx = LayerwiseContext(sh, bits)
    ctx.swap_out(kv)
    torch.cuda.synchronize()
    split = torch.zeros_like(kv)
    ctx.swap_in(split)
    assert ctx.corrupt_count() == 0
    assert torch.equal(whole.view(torch.int16), split.view(torch.int16))
    assert ctx.kernel_launches == sh.n_layers * 2        # per layer one codec kernel each way
