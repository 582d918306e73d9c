"""Block-sparse attention with inputs and outputs in pinned host memory.

The copies are the expensive part of such a call (2.1 GB per 64k/32-head layer), so the layer is
processed in chunks of heads on a few CUDA streams: while one chunk's kernel runs, the next chunk's
Q, K, V are on their way to the device and the previous chunk's O is on its way back (host-to-device
and device-to-host copies use different copy engines). Every chunk is an ordinary
sparsed_attn_sparse call on views of the device tensors; only the row_ptr pointer moves, since
row_ptr holds absolute offsets into col_idx. Torch provides memory, streams and copies only.
"""
from __future__ import annotations

from typing import Sequence

import torch

from . import binding as sd


class HostSparseAttention:
    """Reusable plan: device staging buffers, streams and per-chunk pattern descriptors."""

    def __init__(self, q_host: torch.Tensor, k_host: torch.Tensor, row_ptr: torch.Tensor, col_idx: torch.Tensor,
                 block_size: int, device, kv_heads_per_chunk: int = 4, n_streams: int = 3):
        B, Hq, L, D = q_host.shape
        Hkv = k_host.shape[1]
        if B != 1:
            raise ValueError("HostSparseAttention handles batch 1 (loop over the batch outside)")
        self.shape = (B, Hq, Hkv, L, D)
        self.group = Hq // Hkv
        self.block_size = block_size
        self.nb = L // block_size
        self.dev = torch.device(device)
        self.q = torch.empty(B, Hq, L, D, dtype=torch.bfloat16, device=self.dev)
        self.k = torch.empty(B, Hkv, L, D, dtype=torch.bfloat16, device=self.dev)
        self.v = torch.empty_like(self.k)
        self.o = torch.empty_like(self.q)
        self.row_ptr, self.col_idx = row_ptr, col_idx
        self.streams = [torch.cuda.Stream(device=self.dev) for _ in range(n_streams)]
        self.ws = [sd.new_workspace(sd.STATUS_BYTES, self.dev) for _ in range(n_streams)]
        self.chunks = []
        for kv0 in range(0, Hkv, kv_heads_per_chunk):
            kv1 = min(Hkv, kv0 + kv_heads_per_chunk)
            h0, h1 = kv0 * self.group, kv1 * self.group
            pat = sd.Pattern(row_ptr.data_ptr() + 4 * h0 * self.nb, col_idx.data_ptr(), col_idx.numel(),
                             int(col_idx.numel()), block_size, self.nb, 1, h1 - h0)
            self.chunks.append((kv0, kv1, h0, h1, pat))

    def run(self, q_host, k_host, v_host, o_host) -> None:
        """Enqueues the whole layer; returns when everything has been issued (not finished)."""
        cur = torch.cuda.current_stream(self.dev)
        for s in self.streams:
            s.wait_stream(cur)
        for i, (kv0, kv1, h0, h1, pat) in enumerate(self.chunks):
            s = self.streams[i % len(self.streams)]
            with torch.cuda.stream(s):
                qd, kd, vd, od = self.q[:, h0:h1], self.k[:, kv0:kv1], self.v[:, kv0:kv1], self.o[:, h0:h1]
                qd.copy_(q_host[:, h0:h1], non_blocking=True)
                kd.copy_(k_host[:, kv0:kv1], non_blocking=True)
                vd.copy_(v_host[:, kv0:kv1], non_blocking=True)
                sd.sparsed_attn_sparse(qd, kd, vd, od, pat, self.ws[i % len(self.ws)])
                o_host[:, h0:h1].copy_(od, non_blocking=True)
        for s in self.streams:
            cur.wait_stream(s)

    def device_status(self) -> Sequence:
        return [sd.sparsed_last_device_status(w) for w in self.ws]
