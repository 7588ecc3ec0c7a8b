"""A decoder instance's KV pool and step calls, with PyTorch supplying device memory and the
stream. All computation happens inside libtokenscale.so; this file only marshals arguments.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class TsError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {B.ts_strerror(code)} ({code})")
        self.code = code


def _check(code: int, what: str) -> None:
    if code != B.TS_OK:
        raise TsError(code, what)


def _addr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous()
        return t.data_ptr()
    raise TypeError("expected a torch tensor")


class Decoder:
    """One attention layer's paged KV pool plus the step entry points."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, n_pages: int, max_requests: int,
                 max_pages_per_req: int, chunk_size: int = 0, reserved_pages: int = 0,
                 decode_split_tokens: int = 0, softmax_scale: float = 0.0, device: int = 0,
                 alloc_shuffle_seed: int = 0, page_size: int = 16, nan_fill: bool = False,
                 mixed_prefill_ctas: int = 0, wait_limit_cycles: int = 0, debug_flags: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required; there is no CPU implementation")
        self.device = torch.device("cuda", device)
        cfg = B.ts_config(n_q_heads, n_kv_heads, head_dim, page_size, n_pages, max_requests,
                          max_pages_per_req, chunk_size, reserved_pages, decode_split_tokens,
                          mixed_prefill_ctas, softmax_scale, device, alloc_shuffle_seed, None, 0, None, 0,
                          wait_limit_cycles, debug_flags)
        pool_bytes, ws_bytes = B.ts_pool_bytes(cfg), B.ts_workspace_bytes(cfg)
        if pool_bytes == 0:
            raise TsError(B.TS_ERR_UNSUPPORTED, "ts_pool_bytes")
        self.pool = torch.empty(pool_bytes // 2, dtype=torch.int16, device=self.device)
        if nan_fill:
            self.pool.fill_(0x7FC0)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        cfg.kv_pool, cfg.kv_pool_bytes = self.pool.data_ptr(), pool_bytes
        cfg.workspace, cfg.workspace_bytes = self.workspace.data_ptr(), ws_bytes
        self.cfg = cfg
        rc, self.ctx = B.ts_create(cfg)
        _check(rc, "ts_create")

    def close(self) -> None:
        if getattr(self, "ctx", None):
            torch.cuda.synchronize(self.device)
            B.ts_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ requests and pages
    def request_add(self, req_id: int, prompt_len: int, expected_output_len: int = 0) -> int:
        rc, slot = B.ts_request_add(self.ctx, req_id, prompt_len, expected_output_len)
        _check(rc, "ts_request_add")
        return slot

    def alloc_pages(self, slot: int, total_tokens: int, for_prefill: bool = False) -> None:
        _check(B.ts_alloc_pages(self.ctx, slot, total_tokens, int(for_prefill)), "ts_alloc_pages")

    def block_table(self, slot: int):
        rc, pages, n_tokens = B.ts_block_table(self.ctx, slot)
        _check(rc, "ts_block_table")
        return np.asarray(pages, dtype=np.int32), n_tokens

    def block_table_set(self, slot: int, pages) -> None:
        _check(B.ts_block_table_set(self.ctx, slot, list(pages)), "ts_block_table_set")

    def request_free(self, slot: int) -> None:
        _check(B.ts_request_free(self.ctx, slot), "ts_request_free")

    def request_set_len(self, slot: int, n_tokens: int) -> None:
        _check(B.ts_request_set_len(self.ctx, slot, n_tokens), "ts_request_set_len")

    # ------------------------------------------------------------------------------- steps
    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    def make_step(self, slots, q_len, ctx_len, q=None, k_new=None, v_new=None, out=None,
                  keep_len: bool = False, flags: int = 0):
        return B.make_step(slots, q_len, ctx_len, _addr(q), _addr(k_new), _addr(v_new), _addr(out),
                           (B.TS_STEP_KEEP_LEN if keep_len else 0) | flags)

    def kv_append(self, slots, q_len, ctx_len, k_new, v_new, keep_len: bool = False) -> None:
        st, _keep = self.make_step(slots, q_len, ctx_len, None, k_new, v_new, None, keep_len)
        _check(B.ts_kv_append(self.ctx, st, self._stream()), "ts_kv_append")

    def mixed_step(self, slots, q_len, ctx_len, q, k_new, v_new, out, keep_len: bool = False) -> None:
        st, _keep = self.make_step(slots, q_len, ctx_len, q, k_new, v_new, out, keep_len)
        _check(B.ts_mixed_step(self.ctx, st, self._stream()), "ts_mixed_step")

    def mixed_step_prepared(self, st) -> None:
        """Issue a step marshalled earlier with make_step (keeps the per-call host cost low)."""
        _check(B.ts_mixed_step(self.ctx, st, self._stream()), "ts_mixed_step")

    def mixed_step_host(self, slots, q_len, ctx_len, q, k_new, v_new, out, keep_len: bool = False,
                        wait: bool = True) -> None:
        """q, k_new, v_new, out are HOST tensors (pinned for asynchronous copies). With
        wait=False the call only enqueues (TS_STEP_HOST_ASYNC): consecutive calls overlap their
        copies and kernels, and out is valid once the current stream has passed a later
        host_fence()."""
        st, _keep = self.make_step(slots, q_len, ctx_len, q, k_new, v_new, out, keep_len,
                                   0 if wait else B.TS_STEP_HOST_ASYNC)
        _check(B.ts_mixed_step_host(self.ctx, st, self._stream()), "ts_mixed_step_host")

    def host_fence(self) -> None:
        """Order the current stream behind the downloads of all host steps issued so far."""
        _check(B.ts_host_fence(self.ctx, self._stream()), "ts_host_fence")

    def step_np(self, slots, q_len, ctx_len, q, k_new, v_new, out, alloc: bool = True) -> None:
        """One iteration from numpy int32 row arrays: grow the tables (ts_alloc_step), then
        ts_mixed_step. The cheap path for per-step callers such as the trace replay."""
        st, _keep = B.make_step_np(slots, q_len, ctx_len, _addr(q), _addr(k_new), _addr(v_new), _addr(out))
        if alloc:
            _check(B.ts_alloc_step(self.ctx, st), "ts_alloc_step")
        _check(B.ts_mixed_step(self.ctx, st, self._stream()), "ts_mixed_step")

    def plan_step(self, slots, q_len, ctx_len):
        st, _keep = B.make_step(slots, q_len, ctx_len)
        rc, items = B.ts_plan_step(self.ctx, st)
        _check(rc, "ts_plan_step")
        return items

    def velocity(self) -> dict:
        rc, d = B.ts_velocity(self.ctx)
        _check(rc, "ts_velocity")
        return d

    def profile_enable(self, enable: bool) -> None:
        _check(B.ts_profile_enable(self.ctx, int(enable)), "ts_profile_enable")

    def profile_read(self) -> dict:
        rc, d = B.ts_profile_read(self.ctx, self._stream())
        _check(rc, "ts_profile_read")
        return d

    def device_status(self) -> int:
        rc, bits = B.ts_last_device_status(self.ctx, self._stream())
        if rc not in (B.TS_OK, B.TS_ERR_DEVICE_TIMEOUT):
            _check(rc, "ts_last_device_status")
        return bits
