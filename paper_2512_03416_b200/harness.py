"""Loads a synthetic StepBatch into a Decoder: tables, cached context, step tensors.

Used by the benchmark, the smoke check and the GPU tests. No oracle code is imported here.
"""
from __future__ import annotations

import numpy as np
import torch

from . import workloads as wl
from .decoder import Decoder


def to_dev(a_u16: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy uint16 bf16 bit patterns -> int16 CUDA tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(a_u16).view(np.int16)).to(device)


def from_dev(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint16)


class LoadedBatch:
    """A Decoder whose pool already holds the batch's cached context (via ts_kv_append)."""

    def __init__(self, batch: wl.StepBatch, decode_split_tokens: int = 0, chunk_size=None,
                 max_requests=None, extra_pages: int = 0, device: int = 0, nan_fill: bool = True,
                 mixed_prefill_ctas: int = 0, wait_limit_cycles: int = 0, debug_flags: int = 0):
        s = batch.shape
        width = max([len(t) for t in batch.tables] + [1]) + extra_pages
        cs = batch.chunk_size if chunk_size is None else chunk_size
        self.batch = batch
        self.device = torch.device("cuda", device)
        self.dec = Decoder(s.Hq, s.Hkv, s.D, batch.n_pages, max_requests or max(batch.n_rows, 1), width,
                           chunk_size=cs, decode_split_tokens=decode_split_tokens, device=device,
                           nan_fill=nan_fill, mixed_prefill_ctas=mixed_prefill_ctas,
                           wait_limit_cycles=wait_limit_cycles, debug_flags=debug_flags)
        self.slots = []
        for r in range(batch.n_rows):
            slot = self.dec.request_add(1000 + r, int(batch.ctx_len[r]) + int(batch.q_len[r]))
            self.dec.block_table_set(slot, batch.tables[r])
            self.slots.append(slot)
        with torch.cuda.device(self.device):
            self._load_context()
            self.q = to_dev(batch.q, self.device)
            self.k_new = to_dev(batch.k_new, self.device)
            self.v_new = to_dev(batch.v_new, self.device)
            self.out = torch.full((batch.n_tokens, s.Hq, s.D), 0x7FC0, dtype=torch.int16, device=self.device)
        self._prepared = None

    def _load_context(self, rows_per_call: int = 16) -> None:
        b = self.batch
        rows = [r for r in range(b.n_rows) if b.ctx_len[r] > 0]
        starts = np.concatenate([[0], np.cumsum(b.ctx_len)]).astype(np.int64)
        for i in range(0, len(rows), rows_per_call):        # bounded staging memory
            grp = rows[i:i + rows_per_call]
            ck = np.concatenate([b.context_k[starts[r]:starts[r + 1]] for r in grp])
            cv = np.concatenate([b.context_v[starts[r]:starts[r + 1]] for r in grp])
            self.dec.kv_append([self.slots[r] for r in grp], [int(b.ctx_len[r]) for r in grp],
                               [0] * len(grp), to_dev(ck, self.device), to_dev(cv, self.device))
            torch.cuda.synchronize(self.device)

    def step(self, keep_len: bool = False) -> None:
        """Enqueue the batch's step on the current stream (no synchronisation)."""
        b = self.batch
        with torch.cuda.device(self.device):
            self.dec.mixed_step(self.slots, b.q_len.tolist(), b.ctx_len.tolist(), self.q, self.k_new,
                                self.v_new, self.out, keep_len=keep_len)

    def step_repeatable(self) -> None:
        """Same step with TS_STEP_KEEP_LEN, marshalled once: for timing loops."""
        b = self.batch
        if self._prepared is None:
            self._prepared = self.dec.make_step(self.slots, b.q_len.tolist(), b.ctx_len.tolist(), self.q,
                                                self.k_new, self.v_new, self.out, keep_len=True)
        self.dec.mixed_step_prepared(self._prepared[0])

    def output(self) -> np.ndarray:
        torch.cuda.synchronize(self.device)
        return wl.bf16_bits_to_f32(from_dev(self.out))

    def pool(self) -> np.ndarray:
        torch.cuda.synchronize(self.device)
        return from_dev(self.dec.pool)
