"""The decoder layer around the attention step (ts_layer_*), with PyTorch supplying device memory
and the stream. All computation happens inside libtokenscale.so; this file only marshals arguments.
"""
from __future__ import annotations

import torch

from . import binding as B
from .decoder import Decoder, TsError, _check


class DecoderLayer:
    """RMSNorm, fused QKV projection with rotary embedding, the decoder's paged attention step,
    output projection and gated MLP, bound to a Decoder (its pool, block tables and counters).

    Weights are int16 CUDA tensors holding bf16 bit patterns, [out features, in features]:
    w_norm1 [hidden], w_qkv [(Hq + 2 Hkv) D, hidden], w_o [hidden, Hq D], w_norm2 [hidden],
    w_gate, w_up [intermediate, hidden], w_down [hidden, intermediate]."""

    def __init__(self, dec: Decoder, w_norm1, w_qkv, w_o, w_norm2, w_gate, w_up, w_down, max_position: int,
                 rms_eps: float = 0.0, rope_theta: float = 0.0):
        self.dec = dec
        hidden = int(w_norm1.numel())
        inter = int(w_gate.shape[0])
        stream = torch.cuda.current_stream(dec.device).cuda_stream
        self.w_gate_up = torch.empty((2 * inter, hidden), dtype=torch.int16, device=dec.device)
        _check(B.ts_pack_gate_up(w_gate.data_ptr(), w_up.data_ptr(), self.w_gate_up.data_ptr(), inter, hidden, stream),
               "ts_pack_gate_up")
        self.weights = (w_norm1, w_qkv, w_o, w_norm2, w_down)          # keep the caller's tensors alive
        cfg = B.ts_layer_config(hidden, inter, max_position, rms_eps, rope_theta, w_norm1.data_ptr(), w_qkv.data_ptr(),
                                w_o.data_ptr(), w_norm2.data_ptr(), self.w_gate_up.data_ptr(), w_down.data_ptr(), None, 0)
        nbytes = B.ts_layer_workspace_bytes(dec.cfg, cfg)
        if nbytes == 0:
            raise TsError(B.TS_ERR_UNSUPPORTED, "ts_layer_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=dec.device)
        cfg.workspace, cfg.workspace_bytes = self.workspace.data_ptr(), nbytes
        self.cfg = cfg
        rc, self.handle = B.ts_layer_create(dec.ctx, cfg, stream)
        _check(rc, "ts_layer_create")

    def close(self) -> None:
        if getattr(self, "handle", None):
            torch.cuda.synchronize(self.dec.device)
            B.ts_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def make_step(self, slots, q_len, ctx_len, keep_len: bool = False):
        return B.make_step(slots, q_len, ctx_len, 0, 0, 0, 0, B.TS_STEP_KEEP_LEN if keep_len else 0)

    def step_prepared(self, st, x_in, x_out) -> None:
        _check(B.ts_layer_step(self.handle, st, x_in.data_ptr(), x_out.data_ptr(),
                               torch.cuda.current_stream(self.dec.device).cuda_stream), "ts_layer_step")

    def step(self, slots, q_len, ctx_len, x_in, x_out, keep_len: bool = False) -> None:
        st, _keep = self.make_step(slots, q_len, ctx_len, keep_len)
        self.step_prepared(st, x_in, x_out)
