"""Seeded synthetic inputs: KV tensors, query windows, attention windows, bit draws.

This module serves both the GPU library's tests/benchmarks and the CPU oracle's
tests.  It contains no step of the codec or of the score: only shapes and a
counter-based random number generator (splitmix64 -> uniform -> Box-Muller),
written with device-agnostic torch ops so that the same code fills a host
tensor for small cases and a device tensor for full-size ones.  Whoever needs
the other side's copy of an input copies the tensor; nothing is generated twice.

Value recipe (the workloads stand in for Llama-2 / OPT KV caches, which are not
available here): element = z * sigma_c * o_c with z ~ N(0,1),
sigma_c = exp(0.5 * N(0,1)) drawn once per channel (layer, K/V, head, channel),
o_c = `outlier` for two fixed K channels per (layer, head) and 1 elsewhere;
rounded to fp16.  Query windows are N(0,1) in fp16.
"""
from dataclasses import dataclass, replace
import math

import torch

_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def splitmix64_int(x: int) -> int:
    """One splitmix64 output for state x (pure Python, for keys and for testing the tensor version)."""
    z = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    return (z >> k) & ((1 << (64 - k)) - 1)


def splitmix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on an int64 tensor of states (bit pattern of the uint64 result)."""
    z = x + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def stream_key(seed: int, *tags: int) -> int:
    k = splitmix64_int(seed)
    for t in tags:
        k = splitmix64_int(k ^ (t & _MASK64))
    return k


def _draw_u64(key: int, start: int, count: int, device) -> torch.Tensor:
    """Outputs number start .. start+count-1 of the splitmix64 stream seeded with `key`."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return splitmix64(idx * _GOLDEN + _s64(key))


def _uniform(z: torch.Tensor) -> torch.Tensor:
    return (_lsr(z, 11).to(torch.float64) + 0.5) * (2.0 ** -53)


def normal(key: int, start: int, count: int, device) -> torch.Tensor:
    """count N(0,1) float64 draws; draw i uses stream outputs 2i and 2i+1 (Box-Muller, cosine branch)."""
    z = _draw_u64(key, 2 * start, 2 * count, device).view(count, 2)
    u1, u2 = _uniform(z[:, 0]), _uniform(z[:, 1])
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


@dataclass(frozen=True)
class KVShape:
    name: str
    n_layers: int
    n_kv_heads: int
    n_q_heads: int
    head_dim: int
    n_tokens: int
    chunk_len: int
    group_size: int
    window: int = 8
    outlier: float = 10.0
    seed: int = 0
    frac: tuple = (1.0 / 3.0, 1.0 / 3.0, 1.0 / 3.0)  # share of chunks kept at 8 / 4 / 2 bits; None = uniform random draw
    n_contexts: int = 1

    @property
    def n_chunks(self) -> int:
        return self.n_tokens // self.chunk_len

    @property
    def n_slabs(self) -> int:
        return self.n_layers * 2 * self.n_kv_heads

    @property
    def n_elements(self) -> int:
        return self.n_slabs * self.n_tokens * self.head_dim

    def with_(self, **kw) -> "KVShape":
        return replace(self, **kw)


# The five workloads.  The first is the small case; the third is the one the
# throughput metric is quoted on.
CONFIGS = {
    "tiny": KVShape("tiny", 1, 4, 4, 64, 256, 16, 64, frac=None),
    "gemma2b": KVShape("gemma2b", 18, 1, 8, 256, 2048, 16, 128),
    "llama7b": KVShape("llama7b", 32, 32, 32, 128, 4096, 16, 128),
    "multiapp": KVShape("multiapp", 32, 32, 32, 128, 1024, 32, 128, seed=1, n_contexts=64),
    "mistral7b_32k": KVShape("mistral7b_32k", 32, 8, 32, 128, 32768, 64, 128, outlier=20.0, frac=(0.1, 0.5, 0.4)),
}

_TAG_VALUES, _TAG_SIGMA, _TAG_OUTLIER, _TAG_QWIN, _TAG_BITS, _TAG_PROBS = 1, 2, 3, 4, 5, 6


def channel_scales(shape: KVShape, device="cpu", context: int = 0) -> torch.Tensor:
    """float64 [L, 2, Hkv, d]: sigma_c * o_c."""
    L, H, d = shape.n_layers, shape.n_kv_heads, shape.head_dim
    n = L * 2 * H * d
    sig = torch.exp(0.5 * normal(stream_key(shape.seed, _TAG_SIGMA, context), 0, n, device)).view(L, 2, H, d)
    z = _draw_u64(stream_key(shape.seed, _TAG_OUTLIER, context), 0, 2 * L * H, device).view(L, H, 2)
    c1 = _lsr(z[..., 0], 33) % d
    c2 = (c1 + 1 + _lsr(z[..., 1], 33) % (d - 1)) % d
    boost = torch.ones(L, H, d, dtype=torch.float64, device=device)
    boost.scatter_(2, c1.unsqueeze(-1), shape.outlier)
    boost.scatter_(2, c2.unsqueeze(-1), shape.outlier)
    sig[:, 0] = sig[:, 0] * boost
    return sig


def kv_tensor(shape: KVShape, device="cpu", context: int = 0) -> torch.Tensor:
    """fp16 [L, 2, Hkv, T, d], contiguous."""
    L, H, T, d = shape.n_layers, shape.n_kv_heads, shape.n_tokens, shape.head_dim
    out = torch.empty(L, 2, H, T, d, dtype=torch.float16, device=device)
    scales = channel_scales(shape, device, context)
    key = stream_key(shape.seed, _TAG_VALUES, context)
    plane = H * T * d
    piece = max(1, min(H, (1 << 24) // (T * d)))  # heads per piece: bounds the float64 temporaries
    for l in range(L):
        for s in range(2):
            for h0 in range(0, H, piece):
                h1 = min(H, h0 + piece)
                start = (l * 2 + s) * plane + h0 * T * d
                z = normal(key, start, (h1 - h0) * T * d, device).view(h1 - h0, T, d)
                out[l, s, h0:h1] = (z * scales[l, s, h0:h1].unsqueeze(1)).to(torch.float16)
    return out


def q_window(shape: KVShape, W: int = None, device="cpu", context: int = 0) -> torch.Tensor:
    """fp16 [L, Hq, W, d]: the last W query vectors of every layer and head."""
    W = shape.window if W is None else W
    n = shape.n_layers * shape.n_q_heads * W * shape.head_dim
    z = normal(stream_key(shape.seed, _TAG_QWIN, context), 0, n, device)
    return z.to(torch.float16).view(shape.n_layers, shape.n_q_heads, W, shape.head_dim)


def random_bits(n: int, seed: int = 0) -> torch.Tensor:
    """uint8 [n]: each chunk's bit-width drawn uniformly from {8, 4, 2}."""
    z = _draw_u64(stream_key(seed, _TAG_BITS), 0, n, "cpu")
    levels = torch.tensor([8, 4, 2], dtype=torch.uint8)
    return levels[(_lsr(z, 33) % 3)]


def attention_probs(shape: KVShape, W: int = None, device="cpu", sharpness: float = 8.0) -> torch.Tensor:
    """fp32 [L, Hq, W, T]: a valid causal attention window (row r sits at position T-W+r, sees columns
    0..T-W+r, sums to 1, masked entries are 0).  Rows are heavy-tailed positive draws (a uniform number raised to
    the power `sharpness`: a few columns carry most of a row) divided by their sum over the visible columns."""
    W = shape.window if W is None else W
    L, H, T = shape.n_layers, shape.n_q_heads, shape.n_tokens
    out = torch.empty(L, H, W, T, dtype=torch.float32, device=device)
    key = stream_key(shape.seed, _TAG_PROBS)
    col = torch.arange(T, device=device).view(1, 1, T)
    pos = (T - W + torch.arange(W, device=device)).view(1, W, 1)
    for l in range(L):
        weights = _uniform(_draw_u64(key, l * H * W * T, H * W * T, device)).view(H, W, T) ** sharpness
        weights = weights.masked_fill(col > pos, 0.0)
        out[l] = (weights / weights.sum(dim=-1, keepdim=True)).to(torch.float32)
    return out
