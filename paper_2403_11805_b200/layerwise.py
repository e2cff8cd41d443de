"""Layer-wise swap of one context (the I/O half of the layer-wise pipeline of Sec. 4).

A record of the plain path holds one chunk over all layers, so nothing of a context can be used before all
of it has been loaded.  Here every (layer, chunk) pair is a record of its own: the codec is called with a
one-layer view of the KV tensor, the records of a layer sit next to each other in the pinned arena, and a
load moves and decodes one layer at a time.  While layer l is decoded, layer l+1 is already on its way over
PCIe, and an event per layer tells a consumer (the inference of that layer) when its KV is in place.

Everything here is orchestration of library calls on CUDA streams; the arithmetic is the library's.
"""
import numpy as np
import torch

from . import binding as B


class LayerwiseContext:
    def __init__(self, shape, bits, quant_mode=0):
        """shape: synth.KVShape of the context; bits: one bit-width per chunk (all chunks are swapped)."""
        self.shape = shape
        self.L = shape.n_layers
        self.n = shape.n_chunks
        self.bits = np.ascontiguousarray(bits, dtype=np.uint8)
        assert len(self.bits) == self.n
        self.ids = np.arange(self.n, dtype=np.uint32)
        # one layer of the same tensor: the strides inside a layer do not change
        self.desc = B.make_desc(1, shape.n_kv_heads, shape.n_q_heads, shape.head_dim, shape.n_tokens, shape.chunk_len,
                                shape.group_size, quant_mode)
        self.layer_bytes = B.compressed_size(self.desc, self.bits)
        self.arena = torch.empty(self.L * self.layer_bytes, dtype=torch.uint8).pin_memory()
        self.meta = [B.new_meta(self.n, pinned=True) for _ in range(self.L)]
        ws_bytes = B.codec_workspace_bytes(self.n)
        self.ws_out = [torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") for _ in range(2)]
        self.ws_in = [torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") for _ in range(self.L)]
        self.stage_out = [torch.empty(self.layer_bytes, dtype=torch.uint8, device="cuda") for _ in range(2)]
        self.stage_in = [torch.empty(self.layer_bytes, dtype=torch.uint8, device="cuda") for _ in range(2)]
        self.main = torch.cuda.current_stream()
        self.side_out, self.side_in = torch.cuda.Stream(), torch.cuda.Stream()
        self.ev_packed = [B.new_event() for _ in range(2)]
        self.ev_out_free = [B.new_event() for _ in range(2)]
        self.ev_in_free = [B.new_event() for _ in range(2)]
        self.ev_landed = [B.new_event() for _ in range(2)]
        self.ready = [torch.cuda.Event(enable_timing=True) for _ in range(self.L)]
        self.kernel_launches = 0
        self._launches = B.codec_launches(self.desc, self.bits)      # kernels per codec call

    def layer_arena(self, l):
        return self.arena[l * self.layer_bytes:(l + 1) * self.layer_bytes]

    def swap_out(self, kv):
        """Quantize + pack layer after layer and copy each layer's records to the arena while the next is packed."""
        for l in range(self.L):
            k = l % 2
            self.main.wait_event(self.ev_out_free[k])          # the copy of layer l-2 has left this staging buffer
            B.compress_chunks(self.desc, kv[l], self.ids, self.bits, self.stage_out[k], self.meta[l], self.ws_out[k])
            self.ev_packed[k].record(self.main)
            B.swap_out(self.stage_out[k], self.meta[l], self.layer_arena(l), side_stream=self.side_out,
                       after=self.ev_packed[k], done=self.ev_out_free[k], n=self.n)
            self.kernel_launches += self._launches

    def swap_in(self, kv_out):
        """Load layer after layer; self.ready[l] is recorded on the main stream when layer l of kv_out is complete.
        The checksums in self.meta must have reached the host (synchronise after swap_out)."""
        for l in range(self.L):
            k = l % 2
            B.swap_in(self.layer_arena(l), self.meta[l], self.stage_in[k], side_stream=self.side_in,
                      after=self.ev_in_free[k], done=self.ev_landed[k], n=self.n)
            self.main.wait_event(self.ev_landed[k])
            B.decompress_chunks(self.desc, self.stage_in[k], self.meta[l], None, kv_out[l], self.ws_in[l])
            self.ev_in_free[k].record(self.main)
            self.ready[l].record(self.main)
            self.kernel_launches += self._launches

    def corrupt_count(self):
        """Synchronises; number of records of the last swap_in whose checksum did not match."""
        return sum(B.codec_corrupt_count(w) for w in self.ws_in)
