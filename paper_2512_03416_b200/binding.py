"""ctypes binding of libtokenscale.so: the same names as include/tokenscale.h, argument
marshalling only. Every function returns the library's integer code unchanged unless noted.

The library is CUDA-only. If it has not been built, importing symbols from here raises: there
is no fallback implementation.
"""
from __future__ import annotations

import ctypes
import os

from . import build as _build

TS_OK = 0
TS_ERR_INVALID = -1
TS_ERR_NO_PAGES = -2
TS_ERR_NO_SLOT = -3
TS_ERR_TABLE_SHORT = -4
TS_ERR_BUDGET = -5
TS_ERR_CUDA = -6
TS_ERR_DEVICE_TIMEOUT = -7
TS_ERR_UNSUPPORTED = -8
TS_ERR_WORKSPACE = -9
TS_STEP_KEEP_LEN = 1
TS_STEP_HOST_ASYNC = 2
TS_DEV_BAD_PAGE = 1
TS_DEV_TIMEOUT = 2
TS_DEV_BAD_INDEX = 4
TS_DEBUG_LOSE_APPEND_ARRIVAL = 1

_i32p = ctypes.POINTER(ctypes.c_int32)


class ts_config(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("n_pages", ctypes.c_int32), ("max_requests", ctypes.c_int32),
                ("max_pages_per_req", ctypes.c_int32), ("chunk_size", ctypes.c_int32),
                ("reserved_pages", ctypes.c_int32), ("decode_split_tokens", ctypes.c_int32),
                ("mixed_prefill_ctas", ctypes.c_int32), ("softmax_scale", ctypes.c_float), ("device", ctypes.c_int32),
                ("alloc_shuffle_seed", ctypes.c_uint64),
                ("kv_pool", ctypes.c_void_p), ("kv_pool_bytes", ctypes.c_size_t),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("wait_limit_cycles", ctypes.c_int64), ("debug_flags", ctypes.c_int32)]


class ts_layer_config(ctypes.Structure):
    _fields_ = [("hidden", ctypes.c_int32), ("intermediate", ctypes.c_int32), ("max_position", ctypes.c_int32),
                ("rms_eps", ctypes.c_float), ("rope_theta", ctypes.c_float),
                ("w_norm1", ctypes.c_void_p), ("w_qkv", ctypes.c_void_p), ("w_o", ctypes.c_void_p),
                ("w_norm2", ctypes.c_void_p), ("w_gate_up", ctypes.c_void_p), ("w_down", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


class ts_step(ctypes.Structure):
    _fields_ = [("n_rows", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("slot", _i32p), ("q_len", _i32p), ("ctx_len", _i32p),
                ("q", ctypes.c_void_p), ("k_new", ctypes.c_void_p), ("v_new", ctypes.c_void_p),
                ("out", ctypes.c_void_p)]


class ts_velocity_counters(ctypes.Structure):
    _fields_ = [("steps", ctypes.c_uint64), ("prefill_tokens", ctypes.c_uint64),
                ("decode_tokens", ctypes.c_uint64), ("released_tokens", ctypes.c_uint64),
                ("released_requests", ctypes.c_uint64), ("pages_in_use", ctypes.c_uint64),
                ("pages_free", ctypes.c_uint64), ("kernel_launches", ctypes.c_uint64),
                ("busy_seconds", ctypes.c_double)]


class ts_profile(ctypes.Structure):
    _fields_ = [("append_ms", ctypes.c_double), ("prefill_ms", ctypes.c_double),
                ("decode_ms", ctypes.c_double), ("combine_ms", ctypes.c_double), ("steps", ctypes.c_int64),
                ("mixed_ms", ctypes.c_double), ("mixed_steps", ctypes.c_int64)]


EXPORTS = ["ts_pool_bytes", "ts_workspace_bytes", "ts_create", "ts_destroy", "ts_request_add",
           "ts_alloc_pages", "ts_block_table", "ts_block_table_set", "ts_request_free",
           "ts_request_set_len", "ts_kv_append", "ts_mixed_step", "ts_mixed_step_host", "ts_host_fence",
           "ts_velocity", "ts_report_step_time", "ts_prefill_budget", "ts_plan_step",
           "ts_last_device_status", "ts_last_cuda_error", "ts_strerror", "ts_profile_enable",
           "ts_profile_read", "ts_decode_attention_static", "ts_alloc_step", "ts_pick_chunk_size",
           "ts_convertible_prefill_velocity", "ts_reserved_memory", "ts_reserved_pages",
           "ts_prefiller_instances", "ts_decoder_demand", "ts_regular_decoders", "ts_route_prefill",
           "ts_layer_workspace_bytes", "ts_pack_gate_up", "ts_layer_create", "ts_layer_destroy", "ts_layer_step",
           "ts_layer_last_cuda_error", "ts_gemm_bf16"]

_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2512_03416_b200.build` "
                "(needs nvcc); this package has no other implementation")
        L = ctypes.CDLL(path)
        cfgp, stepp, vp = ctypes.POINTER(ts_config), ctypes.POINTER(ts_step), ctypes.c_void_p
        L.ts_pool_bytes.restype = ctypes.c_size_t
        L.ts_pool_bytes.argtypes = [cfgp]
        L.ts_workspace_bytes.restype = ctypes.c_size_t
        L.ts_workspace_bytes.argtypes = [cfgp]
        L.ts_create.argtypes = [cfgp, ctypes.POINTER(vp)]
        L.ts_destroy.argtypes = [vp]
        L.ts_request_add.argtypes = [vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, _i32p]
        L.ts_alloc_pages.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        L.ts_block_table.argtypes = [vp, ctypes.c_int32, ctypes.POINTER(_i32p), _i32p, _i32p]
        L.ts_block_table_set.argtypes = [vp, ctypes.c_int32, _i32p, ctypes.c_int32]
        L.ts_request_free.argtypes = [vp, ctypes.c_int32]
        L.ts_request_set_len.argtypes = [vp, ctypes.c_int32, ctypes.c_int32]
        L.ts_alloc_step.argtypes = [vp, stepp]
        L.ts_kv_append.argtypes = [vp, stepp, vp]
        L.ts_mixed_step.argtypes = [vp, stepp, vp]
        L.ts_mixed_step_host.argtypes = [vp, stepp, vp]
        L.ts_host_fence.argtypes = [vp, vp]
        L.ts_velocity.argtypes = [vp, ctypes.POINTER(ts_velocity_counters)]
        L.ts_report_step_time.argtypes = [vp, ctypes.c_double]
        L.ts_prefill_budget.restype = ctypes.c_int32
        L.ts_prefill_budget.argtypes = [vp, ctypes.c_int32]
        L.ts_plan_step.argtypes = [vp, stepp, _i32p, ctypes.c_int32, _i32p]
        L.ts_pick_chunk_size.restype = ctypes.c_int32
        L.ts_pick_chunk_size.argtypes = [_i32p, ctypes.POINTER(ctypes.c_double), ctypes.c_int32, ctypes.c_int32,
                                         ctypes.c_double]
        L.ts_convertible_prefill_velocity.restype = ctypes.c_double
        L.ts_convertible_prefill_velocity.argtypes = [ctypes.c_int32, ctypes.c_double, ctypes.c_double]
        L.ts_reserved_memory.restype = ctypes.c_double
        L.ts_reserved_memory.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double]
        L.ts_reserved_pages.restype = ctypes.c_int32
        L.ts_reserved_pages.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_int32]
        dp = ctypes.POINTER(ctypes.c_double)
        L.ts_prefiller_instances.restype = ctypes.c_int32
        L.ts_prefiller_instances.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double]
        L.ts_decoder_demand.restype = ctypes.c_double
        L.ts_decoder_demand.argtypes = [dp, dp, ctypes.c_int32]
        L.ts_regular_decoders.restype = ctypes.c_int32
        L.ts_regular_decoders.argtypes = [ctypes.c_double, ctypes.c_int32]
        L.ts_route_prefill.restype = ctypes.c_int32
        L.ts_route_prefill.argtypes = [dp, dp, ctypes.c_int32, dp, dp, ctypes.c_int32, ctypes.c_double, _i32p]
        L.ts_last_device_status.argtypes = [vp, vp, _i32p]
        L.ts_last_cuda_error.argtypes = [vp]
        L.ts_profile_enable.argtypes = [vp, ctypes.c_int]
        L.ts_profile_read.argtypes = [vp, vp, ctypes.POINTER(ts_profile)]
        L.ts_decode_attention_static.argtypes = [
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp,
            ctypes.c_int32, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_float, vp, vp, vp]
        lcfgp = ctypes.POINTER(ts_layer_config)
        L.ts_layer_workspace_bytes.restype = ctypes.c_size_t
        L.ts_layer_workspace_bytes.argtypes = [cfgp, lcfgp]
        L.ts_pack_gate_up.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, vp]
        L.ts_layer_create.argtypes = [vp, lcfgp, vp, ctypes.POINTER(vp)]
        L.ts_layer_destroy.argtypes = [vp]
        L.ts_layer_step.argtypes = [vp, stepp, vp, vp, vp]
        L.ts_layer_last_cuda_error.argtypes = [vp]
        L.ts_gemm_bf16.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, vp,
                                   ctypes.c_int32, vp, vp]
        L.ts_strerror.restype = ctypes.c_char_p
        L.ts_strerror.argtypes = [ctypes.c_int]
        for name in EXPORTS:
            getattr(L, name)  # AttributeError here means the library is older than the header
        _lib = L
    return _lib


def ts_pool_bytes(cfg: ts_config) -> int:
    return lib().ts_pool_bytes(ctypes.byref(cfg))


def ts_workspace_bytes(cfg: ts_config) -> int:
    return lib().ts_workspace_bytes(ctypes.byref(cfg))


def ts_create(cfg: ts_config):
    """Returns (code, handle)."""
    h = ctypes.c_void_p()
    rc = lib().ts_create(ctypes.byref(cfg), ctypes.byref(h))
    return rc, h


def ts_destroy(ctx) -> int:
    return lib().ts_destroy(ctx)


def ts_request_add(ctx, req_id: int, prompt_len: int, expected_output_len: int):
    """Returns (code, slot)."""
    slot = ctypes.c_int32(-1)
    rc = lib().ts_request_add(ctx, req_id, prompt_len, expected_output_len, ctypes.byref(slot))
    return rc, slot.value


def ts_alloc_pages(ctx, slot: int, total_tokens: int, for_prefill: int = 0) -> int:
    return lib().ts_alloc_pages(ctx, slot, total_tokens, for_prefill)


def ts_block_table(ctx, slot: int):
    """Returns (code, pages as a list copy, n_tokens)."""
    pages = _i32p()
    n_pages, n_tokens = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = lib().ts_block_table(ctx, slot, ctypes.byref(pages), ctypes.byref(n_pages), ctypes.byref(n_tokens))
    if rc != TS_OK:
        return rc, [], 0
    return rc, [pages[i] for i in range(n_pages.value)], n_tokens.value


def ts_block_table_set(ctx, slot: int, pages) -> int:
    arr = (ctypes.c_int32 * len(pages))(*[int(p) for p in pages])
    return lib().ts_block_table_set(ctx, slot, arr, len(pages))


def ts_request_free(ctx, slot: int) -> int:
    return lib().ts_request_free(ctx, slot)


def ts_request_set_len(ctx, slot: int, n_tokens: int) -> int:
    return lib().ts_request_set_len(ctx, slot, n_tokens)


def make_step(slots, q_len, ctx_len, q=0, k_new=0, v_new=0, out=0, flags: int = 0):
    """Marshal host int arrays and raw addresses into a ts_step. Returns (step, keepalive)."""
    n = len(slots)
    a_slot = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in slots])
    a_q = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in q_len])
    a_c = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in ctx_len])
    st = ts_step(n, flags, a_slot, a_q, a_c, q or None, k_new or None, v_new or None, out or None)
    return st, (a_slot, a_q, a_c)


def make_step_np(slots, q_len, ctx_len, q=0, k_new=0, v_new=0, out=0, flags: int = 0):
    """Like make_step, for contiguous numpy int32 arrays: no per-element conversion.
    Returns (step, keepalive); the arrays must stay alive while the step is used."""
    import numpy as np
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in (slots, q_len, ctx_len)]
    ptrs = [a.ctypes.data_as(_i32p) for a in arrs]
    st = ts_step(len(arrs[0]), flags, ptrs[0], ptrs[1], ptrs[2], q or None, k_new or None, v_new or None,
                 out or None)
    return st, arrs


def ts_alloc_step(ctx, step: ts_step) -> int:
    return lib().ts_alloc_step(ctx, ctypes.byref(step))


def ts_kv_append(ctx, step: ts_step, cuda_stream: int = 0) -> int:
    return lib().ts_kv_append(ctx, ctypes.byref(step), ctypes.c_void_p(cuda_stream))


def ts_mixed_step(ctx, step: ts_step, cuda_stream: int = 0) -> int:
    return lib().ts_mixed_step(ctx, ctypes.byref(step), ctypes.c_void_p(cuda_stream))


def ts_mixed_step_host(ctx, step: ts_step, cuda_stream: int = 0) -> int:
    return lib().ts_mixed_step_host(ctx, ctypes.byref(step), ctypes.c_void_p(cuda_stream))


def ts_host_fence(ctx, cuda_stream: int = 0) -> int:
    return lib().ts_host_fence(ctx, ctypes.c_void_p(cuda_stream))


def ts_velocity(ctx):
    """Returns (code, dict of counters)."""
    c = ts_velocity_counters()
    rc = lib().ts_velocity(ctx, ctypes.byref(c))
    return rc, {name: getattr(c, name) for name, _ in ts_velocity_counters._fields_}


def ts_report_step_time(ctx, seconds: float) -> int:
    return lib().ts_report_step_time(ctx, seconds)


def ts_prefill_budget(ctx, decode_batch_size: int) -> int:
    return lib().ts_prefill_budget(ctx, decode_batch_size)


def ts_pick_chunk_size(prefill_tokens, iteration_seconds, decode_batch_size: int, tpot_slo_s: float) -> int:
    n = len(prefill_tokens)
    a = (ctypes.c_int32 * max(n, 1))(*[int(t) for t in prefill_tokens])
    b = (ctypes.c_double * max(n, 1))(*[float(t) for t in iteration_seconds])
    return lib().ts_pick_chunk_size(a, b, n, decode_batch_size, tpot_slo_s)


def ts_convertible_prefill_velocity(chunk_size: int, decode_batch_size: float, tpot_slo_s: float) -> float:
    return lib().ts_convertible_prefill_velocity(chunk_size, decode_batch_size, tpot_slo_s)


def ts_reserved_memory(prefill_velocity: float, mem_per_token: float, ttft_slo_s: float) -> float:
    return lib().ts_reserved_memory(prefill_velocity, mem_per_token, ttft_slo_s)


def ts_reserved_pages(prefill_velocity: float, ttft_slo_s: float, page_size: int = 16) -> int:
    return lib().ts_reserved_pages(prefill_velocity, ttft_slo_s, page_size)


TS_ROUTE_PREFILLER, TS_ROUTE_CONVERTIBLE, TS_ROUTE_QUEUE = 0, 1, 2


def _doubles(values):
    n = len(values)
    return (ctypes.c_double * max(n, 1))(*[float(v) for v in values]), n


def ts_prefiller_instances(token_rate: float, prefill_velocity: float, network_velocity: float) -> int:
    return lib().ts_prefiller_instances(token_rate, prefill_velocity, network_velocity)


def ts_decoder_demand(token_rate, velocity) -> float:
    a, n = _doubles(token_rate)
    b, _ = _doubles(velocity)
    return lib().ts_decoder_demand(a, b, n)


def ts_regular_decoders(decoder_demand: float, convertible_decoders: int) -> int:
    return lib().ts_regular_decoders(decoder_demand, convertible_decoders)


def ts_route_prefill(prefiller_inflight, prefiller_velocity, convertible_inflight, convertible_velocity, slo_s: float):
    """Returns (index or error code, kind)."""
    pa, np_ = _doubles(prefiller_inflight)
    pv, _ = _doubles(prefiller_velocity)
    ca, nc = _doubles(convertible_inflight)
    cv, _ = _doubles(convertible_velocity)
    kind = ctypes.c_int32(-1)
    idx = lib().ts_route_prefill(pa, pv, np_, ca, cv, nc, slo_s, ctypes.byref(kind))
    return idx, kind.value


def ts_plan_step(ctx, step: ts_step):
    """Returns (code, list of 8-int records)."""
    n = ctypes.c_int32(0)
    rc = lib().ts_plan_step(ctx, ctypes.byref(step), None, 0, ctypes.byref(n))
    if rc != TS_OK or n.value == 0:
        return rc, []
    buf = (ctypes.c_int32 * (8 * n.value))()
    rc = lib().ts_plan_step(ctx, ctypes.byref(step), buf, n.value, ctypes.byref(n))
    return rc, [tuple(buf[8 * i:8 * i + 8]) for i in range(n.value)]


def ts_last_device_status(ctx, cuda_stream: int = 0):
    """Returns (code, status bits)."""
    s = ctypes.c_int32(0)
    rc = lib().ts_last_device_status(ctx, ctypes.c_void_p(cuda_stream), ctypes.byref(s))
    return rc, s.value


def ts_profile_enable(ctx, enable: int) -> int:
    return lib().ts_profile_enable(ctx, enable)


def ts_profile_read(ctx, cuda_stream: int = 0):
    """Returns (code, dict)."""
    p = ts_profile()
    rc = lib().ts_profile_read(ctx, ctypes.c_void_p(cuda_stream), ctypes.byref(p))
    return rc, {name: getattr(p, name) for name, _ in ts_profile._fields_}


def ts_decode_attention_static(device: int, n_q_heads: int, n_kv_heads: int, head_dim: int, n_pages: int,
                               kv_pool: int, block_tables: int, table_width: int, kv_len: int,
                               n_rows: int, n_splits: int, softmax_scale: float, q: int, out: int,
                               cuda_stream: int = 0) -> int:
    """Decode attention that uses the library's built-in scratch; pointers are raw device addresses."""
    return lib().ts_decode_attention_static(device, n_q_heads, n_kv_heads, head_dim, n_pages,
                                            ctypes.c_void_p(kv_pool), ctypes.c_void_p(block_tables),
                                            table_width, ctypes.c_void_p(kv_len), n_rows, n_splits,
                                            softmax_scale, ctypes.c_void_p(q), ctypes.c_void_p(out),
                                            ctypes.c_void_p(cuda_stream))


def ts_last_cuda_error(ctx) -> int:
    return lib().ts_last_cuda_error(ctx)


def ts_strerror(code: int) -> str:
    return lib().ts_strerror(code).decode()


# ------------------------------------------------------------------- the decoder layer around attention
def ts_layer_workspace_bytes(cfg: ts_config, layer: ts_layer_config) -> int:
    return lib().ts_layer_workspace_bytes(ctypes.byref(cfg), ctypes.byref(layer))


def ts_pack_gate_up(w_gate: int, w_up: int, w_gate_up: int, intermediate: int, hidden: int, stream: int) -> int:
    return lib().ts_pack_gate_up(w_gate, w_up, w_gate_up, intermediate, hidden, stream)


def ts_layer_create(ctx, layer: ts_layer_config, stream: int):
    """Returns (code, handle)."""
    h = ctypes.c_void_p()
    rc = lib().ts_layer_create(ctx, ctypes.byref(layer), stream, ctypes.byref(h))
    return rc, h


def ts_layer_destroy(layer) -> int:
    return lib().ts_layer_destroy(layer)


def ts_layer_step(layer, step: ts_step, x_in: int, x_out: int, stream: int) -> int:
    return lib().ts_layer_step(layer, ctypes.byref(step), x_in, x_out, stream)


def ts_gemm_bf16(device: int, M: int, N: int, K: int, A: int, B: int, R: int, C: int, tile_m: int, status: int,
                 stream: int) -> int:
    return lib().ts_gemm_bf16(device, M, N, K, A, B, R or None, C, tile_m, status, stream)
