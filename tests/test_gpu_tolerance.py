"""GPU parity of the tolerance score (Eq. 1) against the float64 oracle: scores within 1e-4 relative;
the rankings taken from the same score array are identical bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_11805_b200 import binding as B, synth
from gpu_helpers import bits_view, odesc

pytestmark = pytest.mark.gpu
REL = 1e-4


def gpu_scores(sh, kv_dev, q_dev, W):
    d = B.desc_of(sh)
    scores = torch.full((sh.n_chunks,), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    B.chunk_tolerance(d, kv_dev, q_dev, W, scores, ws)
    torch.cuda.synchronize()
    return scores.cpu().numpy()


def gpu_scores_from_probs(sh, probs_dev, W):
    d = B.desc_of(sh)
    scores = torch.full((sh.n_chunks,), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(B.tolerance_workspace_bytes(d, W), dtype=torch.uint8, device="cuda")
    B.chunk_tolerance_from_probs(d, probs_dev, W, scores, ws)
    torch.cuda.synchronize()
    return scores.cpu().numpy()


def check_scores(sh, W):
    kv = synth.kv_tensor(sh)
    q = synth.q_window(sh, W)
    got = gpu_scores(sh, kv.cuda(), q.cuda(), W)
    want = oracle.chunk_tolerance(odesc(sh), bits_view(kv), bits_view(q), W)
    assert np.all(np.isfinite(got))
    assert np.max(np.abs(got - want) / want) < REL, np.max(np.abs(got - want) / want)
    return got, want


SHAPES = [
    ("tiny", synth.CONFIGS["tiny"], 8),
    ("gemma2b", synth.CONFIGS["gemma2b"], 8),
    ("llama7b_2layers", synth.CONFIGS["llama7b"].with_(n_layers=2), 8),
    ("mistral_gqa_slice", synth.CONFIGS["mistral7b_32k"].with_(n_layers=1, n_tokens=4096), 8),
    ("multiapp_1layer", synth.CONFIGS["multiapp"].with_(n_layers=1), 8),
    ("full_matrix", synth.KVShape("full", 2, 2, 4, 64, 96, 16, 64, seed=5), 96),           # W = T: the paper's matrix
    ("ragged_tail", synth.KVShape("rag", 2, 2, 2, 32, 1000, 24, 32, seed=6), 5),          # SEG 8, tail of 16 tokens
    ("odd_chunk", synth.KVShape("odd", 1, 1, 3, 16, 77, 7, 16, seed=7), 3),              # SEG 1
    ("one_row", synth.KVShape("w1", 1, 2, 2, 64, 300, 4, 64, seed=8), 1),
    ("window_longer_than_chunk", synth.KVShape("wl", 1, 1, 2, 32, 128, 8, 32, seed=9), 20),
    # the tcgen05 kernel with its running row sums: at least as many (layer, KV head) pairs as SMs, so that a pair's
    # tiles fall to one or two CTAs.  Pairs of three tiles (fewer than accumulators: some statistics threads see no tile
    # of a pair), 40 rows per pair in a 64-row operand (padding rows), 128 rows per pair
    ("tc_short_pairs", synth.KVShape("tcs", 20, 8, 32, 64, 272, 16, 64, seed=31), 8),
    ("tc_padded_rows", synth.KVShape("tcp", 20, 8, 40, 128, 400, 32, 128, seed=32), 8),
    ("tc_128_rows", synth.KVShape("tcr", 16, 10, 160, 64, 300, 16, 64, seed=33), 8),
]


@pytest.mark.parametrize("name,sh,W", SHAPES, ids=[s[0] for s in SHAPES])
def test_chunk_tolerance_matches_oracle(name, sh, W):
    check_scores(sh, W)


@pytest.mark.parametrize("name,sh,W", SHAPES[:2] + SHAPES[5:], ids=[s[0] for s in SHAPES[:2] + SHAPES[5:]])
def test_from_probs_matches_oracle(name, sh, W):
    probs = synth.attention_probs(sh, W)
    got = gpu_scores_from_probs(sh, probs.cuda(), W)
    want = oracle.chunk_tolerance_from_probs(odesc(sh), probs.double().numpy(), W)
    assert np.max(np.abs(got - want) / want) < REL


def test_from_probs_ignores_masked_entries():
    sh, W = SHAPES[6][1], 5
    probs = synth.attention_probs(sh, W)
    want = gpu_scores_from_probs(sh, probs.cuda(), W)
    dirty = probs.clone()
    for r in range(W):
        dirty[:, :, r, sh.n_tokens - W + r + 1:] = 7.0
    assert np.array_equal(gpu_scores_from_probs(sh, dirty.cuda(), W), want)


def test_two_paths_agree_and_scores_are_reproducible():
    # the oracle's attention window fed to the probability path must give what the K/q path gives
    sh, W = synth.CONFIGS["tiny"], 8
    kv, q = synth.kv_tensor(sh), synth.q_window(sh, W)
    a = gpu_scores(sh, kv.cuda(), q.cuda(), W)
    probs = oracle.attention_window(odesc(sh), bits_view(kv), bits_view(q), W)
    b = gpu_scores_from_probs(sh, torch.from_numpy(probs).float().cuda(), W)
    assert np.max(np.abs(a - b) / b) < REL
    assert np.array_equal(a, gpu_scores(sh, kv.cuda(), q.cuda(), W))       # fixed summation order


def test_scores_drive_the_same_bit_assignment():
    # rank -> bits is taken from the same fp32 score array on both sides: identical orderings
    sh, W = synth.CONFIGS["gemma2b"], 8
    got, want = check_scores(sh, W)
    gb, go = B.assign_bits(got, sh.frac)
    ob, oo = oracle.assign_bits(got, sh.frac)
    assert np.array_equal(gb, ob) and np.array_equal(go, oo)
    assert tuple(int((gb == b).sum()) for b in (8, 4, 2)) == (43, 42, 43)
    # how fragile is the ranking against the float64 scores: adjacent pairs closer than the tolerance
    srt = np.sort(want)[::-1]
    close = int(np.sum((srt[:-1] - srt[1:]) / srt[:-1] < REL))
    ob64, _ = oracle.assign_bits(want.astype(np.float32), sh.frac)
    assert int((ob64 != gb).sum()) <= 2 * close


def test_full_size_llama7b_scores():
    sh, W = synth.CONFIGS["llama7b"], 8
    kv_dev = synth.kv_tensor(sh, device="cuda")
    q_dev = synth.q_window(sh, W, device="cuda")
    got = gpu_scores(sh, kv_dev, q_dev, W)
    assert np.all(np.isfinite(got)) and np.all(got > 0)
    # every row sums to 1: sum over chunks of chunk_len * D_i * n_vis-weights equals W rows ... for the columns
    # all W rows see (col <= T - W) n_vis = W, so sum_i CL * D_i is 1 up to the last W - 1 columns' reweighting
    total = float(np.sum(got.astype(np.float64)) * sh.chunk_len)
    assert 1.0 - 1e-4 <= total < 1.5
    # the K half only: the oracle on the K planes (V is never read) - whole config, threads of the host
    k_only = kv_dev[:, :1].cpu()
    small = oracle.make_desc(sh.n_layers, sh.n_kv_heads, sh.n_q_heads, sh.head_dim, sh.n_tokens, sh.chunk_len, sh.group_size)
    small.stride_s = 0
    small.stride_l = sh.n_kv_heads * sh.n_tokens * sh.head_dim
    want = oracle.chunk_tolerance(small, bits_view(k_only), bits_view(q_dev), W)
    assert np.max(np.abs(got - want) / want) < REL
