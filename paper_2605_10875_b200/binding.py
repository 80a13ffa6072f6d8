"""ctypes binding of libsol.so: the same names as include/sol.h, argument
marshalling only.  Every step of the decode path runs in the CUDA library;
there is no Python or CPU fallback: if the library is missing, loading fails.

Pointer arguments accept anything with a ``data_ptr()`` method (a torch
tensor), a raw integer address, or None for optional pointers.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsol.so")

SOL_OK = 0
SOL_ERR_INVALID_ARG = 1
SOL_ERR_UNSUPPORTED = 2
SOL_ERR_WORKSPACE_TOO_SMALL = 3
SOL_ERR_CUDA = 4
SOL_ERR_DEVICE_TIMEOUT = 5

EXPORTS = [
    "sol_status_string", "sol_last_cuda_error", "sol_workspace_bytes", "sol_workspace_init", "sol_quant_act",
    "sol_packed_weight_bytes", "sol_pack_weights", "sol_quant_act_wide", "sol_quest_meta_bytes", "sol_quest_build_meta",
    "sol_sparse_decode_attn", "sol_sparse_decode_attn_static", "sol_pruned_swiglu_mlp", "sol_decode_layer", "sol_decode_step",
    "sol_decode_step_traced", "sol_kv_refresh", "sol_decode_step_host", "sol_read_device_status", "sol_selftest_wait_timeout", "sol_timing_enable", "sol_timing_collect",
    "sol_launch_count",
]


class SolShape(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("page_size", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("n_sink", C.c_int32), ("n_window", C.c_int32),
                ("quant_placement", C.c_int32), ("mlp_prune", C.c_int32), ("token_select", C.c_int32),
                ("quest_page_size", C.c_int32)]


class SolKV(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("page_table", C.c_void_p),
                ("seq_lens", C.c_void_p), ("max_pages_per_seq", C.c_int32), ("num_pages", C.c_int32),
                ("quest_meta", C.c_void_p)]


class SolLayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_qkv", "w_o", "w_gate_up", "w_down", "gamma1", "gamma2")]


TRACE_FIELDS = ("xn1", "codes1", "scales1", "q_rot", "kept_idx", "kept_cnt", "attn_out", "h_mid", "xn2", "codes2",
                "scales2", "t", "kept_ch", "kept_ch_cnt", "h_out", "z", "z_codes", "z_scales", "xm2")


class SolLayerTrace(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in TRACE_FIELDS]


class SolKernelTime(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_int32), ("total_ms", C.c_float)]


class SolError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status} ({status_string(status)}) {last_cuda_error()}".strip())
        self.status = status


_lib = None


def lib() -> C.CDLL:
    """Loads libsol.so on first use; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_10875_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        P, I, S = C.c_void_p, C.c_int32, C.c_size_t
        L.sol_status_string.restype = C.c_char_p
        L.sol_status_string.argtypes = [I]
        L.sol_last_cuda_error.restype = C.c_char_p
        L.sol_last_cuda_error.argtypes = []
        L.sol_workspace_bytes.restype = S
        L.sol_workspace_bytes.argtypes = [C.POINTER(SolShape), I, I]
        L.sol_workspace_init.restype = I
        L.sol_workspace_init.argtypes = [P, S, P]
        L.sol_quant_act.restype = I
        L.sol_quant_act.argtypes = [P, I, I, P, P, P, P, P]
        L.sol_quant_act_wide.restype = I
        L.sol_quant_act_wide.argtypes = [P, I, I, P, P, P, P]
        L.sol_sparse_decode_attn.restype = I
        L.sol_sparse_decode_attn.argtypes = [C.POINTER(SolShape), P, C.POINTER(SolKV), I, P, P, P, P, P, S, P]
        L.sol_sparse_decode_attn_static.restype = I
        L.sol_sparse_decode_attn_static.argtypes = [C.POINTER(SolShape), P, C.POINTER(SolKV), I, P, P, P, P, P, P]
        L.sol_pruned_swiglu_mlp.restype = I
        L.sol_pruned_swiglu_mlp.argtypes = [C.POINTER(SolShape), P, P, P, I, P, P, P, P, P, S, P]
        L.sol_packed_weight_bytes.restype = S
        L.sol_packed_weight_bytes.argtypes = [C.POINTER(SolShape), I]
        L.sol_quest_meta_bytes.restype = S
        L.sol_quest_meta_bytes.argtypes = [C.POINTER(SolShape), I]
        L.sol_quest_build_meta.restype = I
        L.sol_quest_build_meta.argtypes = [C.POINTER(SolShape), C.POINTER(SolKV), I, P]
        L.sol_pack_weights.restype = I
        L.sol_pack_weights.argtypes = [C.POINTER(SolShape), I, P, P, P, S, P]
        L.sol_decode_layer.restype = I
        L.sol_decode_layer.argtypes = [C.POINTER(SolShape), C.POINTER(SolLayerWeights), C.POINTER(SolKV), I, P, P, P,
                                       P, P, C.POINTER(SolLayerTrace), P, S, P]
        L.sol_decode_step.restype = I
        L.sol_decode_step.argtypes = [C.POINTER(SolShape), I, C.POINTER(SolLayerWeights), C.POINTER(SolKV), I, P, P,
                                      P, P, P, P, P, S, P]
        L.sol_decode_step_traced.restype = I
        L.sol_decode_step_traced.argtypes = [C.POINTER(SolShape), I, C.POINTER(SolLayerWeights), C.POINTER(SolKV), I,
                                             P, P, P, P, P, P, C.POINTER(SolLayerTrace), P, S, P]
        L.sol_kv_refresh.restype = I
        L.sol_kv_refresh.argtypes = [C.POINTER(SolShape), I, C.POINTER(SolLayerWeights), C.POINTER(SolKV), I, I, P, P,
                                     P, S, P]
        L.sol_selftest_wait_timeout.restype = I
        L.sol_selftest_wait_timeout.argtypes = [P, P]
        L.sol_decode_step_host.restype = I
        L.sol_decode_step_host.argtypes = [C.POINTER(SolShape), I, C.POINTER(SolLayerWeights), C.POINTER(SolKV), I,
                                           P, P, P, P, P, P, P, S, P]
        L.sol_read_device_status.restype = I
        L.sol_read_device_status.argtypes = [P, C.POINTER(C.c_int32), P]
        L.sol_timing_enable.restype = None
        L.sol_timing_enable.argtypes = [I]
        L.sol_timing_collect.restype = I
        L.sol_timing_collect.argtypes = [C.POINTER(SolKernelTime), I]
        L.sol_launch_count.restype = C.c_int64
        L.sol_launch_count.argtypes = [I]
        _lib = L
    return _lib


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):  # numpy array (host pointer)
        return x.ctypes.data
    return int(x)


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    return getattr(stream, "cuda_stream", stream)


def _check(status: int, what: str) -> None:
    if status != SOL_OK:
        raise SolError(status, what)


def status_string(status: int) -> str:
    return lib().sol_status_string(status).decode()


def last_cuda_error() -> str:
    return lib().sol_last_cuda_error().decode()


def make_shape(d_model, n_q_heads, n_kv_heads, head_dim, d_ff, page_size=64, rms_eps=1e-5, rope_theta=0.0,
               n_sink=0, n_window=1, quant_placement=0, mlp_prune=0, token_select=0, quest_page_size=0) -> SolShape:
    return SolShape(d_model, n_q_heads, n_kv_heads, head_dim, d_ff, page_size, rms_eps, rope_theta, n_sink, n_window,
                    quant_placement, mlp_prune, token_select, quest_page_size)


def make_kv(k_pool, v_pool, page_table, seq_lens, max_pages_per_seq: int, num_pages: int, quest_meta=None) -> SolKV:
    return SolKV(_ptr(k_pool), _ptr(v_pool), _ptr(page_table), _ptr(seq_lens), max_pages_per_seq, num_pages,
                 _ptr(quest_meta))


SELECT_TOKENS, SELECT_QUEST_PAGES = 0, 1


def quest_meta_bytes(shape: SolShape, num_pages: int) -> int:
    return int(lib().sol_quest_meta_bytes(C.byref(shape), num_pages))


def quest_build_meta(shape: SolShape, kv: SolKV, B: int, stream=None, check=True) -> int:
    """Page extrema of every token the B sequences hold, into kv.quest_meta."""
    s = lib().sol_quest_build_meta(C.byref(shape), C.byref(kv), B, _stream(stream))
    if check:
        _check(s, "sol_quest_build_meta")
    return s


W_QKV, W_O, W_GATE_UP, W_DOWN = 0, 1, 2, 3


def packed_weight_bytes(shape: SolShape, kind: int) -> int:
    return int(lib().sol_packed_weight_bytes(C.byref(shape), kind))


def pack_weights(shape: SolShape, kind: int, src0, src1, dst, dst_bytes: int, stream=None, check=True) -> int:
    """One-time packing of a row-major bf16 weight matrix (src1: the up matrix of the gate/up pair)."""
    s = lib().sol_pack_weights(C.byref(shape), kind, _ptr(src0), _ptr(src1), _ptr(dst), dst_bytes, _stream(stream))
    if check:
        _check(s, "sol_pack_weights")
    return s


def make_weights(w_qkv, w_o, w_gate_up, w_down, gamma1, gamma2) -> SolLayerWeights:
    """The four matrices are the PACKED buffers (pack_weights)."""
    return SolLayerWeights(*[_ptr(x) for x in (w_qkv, w_o, w_gate_up, w_down, gamma1, gamma2)])


def make_trace(**taps) -> SolLayerTrace:
    return SolLayerTrace(*[_ptr(taps.get(n)) for n in TRACE_FIELDS])


def workspace_bytes(shape: SolShape, max_batch: int, max_pages_per_seq: int) -> int:
    return int(lib().sol_workspace_bytes(C.byref(shape), max_batch, max_pages_per_seq))


def workspace_init(ws, ws_bytes: int, stream=None) -> None:
    _check(lib().sol_workspace_init(_ptr(ws), ws_bytes, _stream(stream)), "sol_workspace_init")


def quant_act(x_bf16, B: int, d: int, bits, codes, scales, xhat_bf16=None, stream=None, check=True) -> int:
    s = lib().sol_quant_act(_ptr(x_bf16), B, d, _ptr(bits), _ptr(codes), _ptr(scales), _ptr(xhat_bf16),
                            _stream(stream))
    if check:
        _check(s, "sol_quant_act")
    return s


QUANT_PROJ_INPUTS, QUANT_MLP_OUTPUT = 0, 1
PRUNE_INTERMEDIATE, PRUNE_MLP_INPUT = 0, 1


def quant_act_wide(x_bf16, B: int, d: int, bits, codes_i16, scales, stream=None, check=True) -> int:
    s = lib().sol_quant_act_wide(_ptr(x_bf16), B, d, _ptr(bits), _ptr(codes_i16), _ptr(scales), _stream(stream))
    if check:
        _check(s, "sol_quant_act_wide")
    return s


def sparse_decode_attn(shape, q_bf16, kv: SolKV, B: int, r_permille, out_bf16, kept_idx, kept_cnt, ws,
                       ws_bytes: int, stream=None, check=True) -> int:
    s = lib().sol_sparse_decode_attn(C.byref(shape), _ptr(q_bf16), C.byref(kv), B, _ptr(r_permille), _ptr(out_bf16),
                                     _ptr(kept_idx), _ptr(kept_cnt), _ptr(ws), ws_bytes, _stream(stream))
    if check:
        _check(s, "sol_sparse_decode_attn")
    return s


STATIC_SCRATCH_BYTES = 4 << 20


def sparse_decode_attn_static(shape, q_bf16, kv: SolKV, B: int, r_permille, out_bf16, kept_idx=None, kept_cnt=None,
                              status_out=None, stream=None, check=True) -> int:
    """sol_sparse_decode_attn for a caller with no workspace to give: the scratch is a fixed array
    inside the library (STATIC_SCRATCH_BYTES per GPU), nothing is allocated.  Problems that do not
    fit are refused with SOL_ERR_WORKSPACE_TOO_SMALL.  Calls share the array: do not overlap them."""
    s = lib().sol_sparse_decode_attn_static(C.byref(shape), _ptr(q_bf16), C.byref(kv), B, _ptr(r_permille),
                                            _ptr(out_bf16), _ptr(kept_idx), _ptr(kept_cnt), _ptr(status_out),
                                            _stream(stream))
    if check:
        _check(s, "sol_sparse_decode_attn_static")
    return s


def pruned_swiglu_mlp(shape, x_bf16, w_gate_up, w_down, B: int, p_permille, out_bf16, kept_ch, kept_ch_cnt,
                      ws, ws_bytes: int, stream=None, check=True) -> int:
    s = lib().sol_pruned_swiglu_mlp(C.byref(shape), _ptr(x_bf16), _ptr(w_gate_up), _ptr(w_down), B,
                                    _ptr(p_permille), _ptr(out_bf16), _ptr(kept_ch), _ptr(kept_ch_cnt), _ptr(ws),
                                    ws_bytes, _stream(stream))
    if check:
        _check(s, "sol_pruned_swiglu_mlp")
    return s


def decode_layer(shape, weights: SolLayerWeights, kv: SolKV, B: int, h_in_bf16, h_out_bf16, r_permille,
                 p_permille, bits, trace: Optional[SolLayerTrace], ws, ws_bytes: int, stream=None, check=True) -> int:
    s = lib().sol_decode_layer(C.byref(shape), C.byref(weights), C.byref(kv), B, _ptr(h_in_bf16), _ptr(h_out_bf16),
                               _ptr(r_permille), _ptr(p_permille), _ptr(bits),
                               C.byref(trace) if trace is not None else None, _ptr(ws), ws_bytes, _stream(stream))
    if check:
        _check(s, "sol_decode_layer")
    return s


def _arrays(layers: Sequence[SolLayerWeights], kvs: Sequence[SolKV]):
    n = len(layers)
    return (SolLayerWeights * n)(*layers), (SolKV * n)(*kvs)


def decode_step(shape, layers, kvs, B: int, h_in_bf16, h_out_bf16, h_out_f32, r_permille, p_permille, bits, ws,
                ws_bytes: int, stream=None, check=True) -> int:
    la, ka = _arrays(layers, kvs)
    s = lib().sol_decode_step(C.byref(shape), len(layers), la, ka, B, _ptr(h_in_bf16), _ptr(h_out_bf16),
                              _ptr(h_out_f32), _ptr(r_permille), _ptr(p_permille), _ptr(bits), _ptr(ws), ws_bytes,
                              _stream(stream))
    if check:
        _check(s, "sol_decode_step")
    return s


def decode_step_traced(shape, layers, kvs, B: int, h_in_bf16, h_out_bf16, h_out_f32, r_permille, p_permille, bits,
                       traces: Optional[Sequence[SolLayerTrace]], ws, ws_bytes: int, stream=None, check=True) -> int:
    la, ka = _arrays(layers, kvs)
    ta = (SolLayerTrace * len(layers))(*traces) if traces is not None else None
    s = lib().sol_decode_step_traced(C.byref(shape), len(layers), la, ka, B, _ptr(h_in_bf16), _ptr(h_out_bf16),
                                     _ptr(h_out_f32), _ptr(r_permille), _ptr(p_permille), _ptr(bits), ta, _ptr(ws),
                                     ws_bytes, _stream(stream))
    if check:
        _check(s, "sol_decode_step_traced")
    return s


def kv_refresh(shape, layers, kvs, B: int, n_tokens: int, h_in_bf16, h_out_bf16, ws, ws_bytes: int, stream=None,
               check=True) -> int:
    la, ka = _arrays(layers, kvs)
    s = lib().sol_kv_refresh(C.byref(shape), len(layers), la, ka, B, n_tokens, _ptr(h_in_bf16), _ptr(h_out_bf16),
                             _ptr(ws), ws_bytes, _stream(stream))
    if check:
        _check(s, "sol_kv_refresh")
    return s


def selftest_wait_timeout(ws, stream=None) -> None:
    _check(lib().sol_selftest_wait_timeout(_ptr(ws), _stream(stream)), "sol_selftest_wait_timeout")


def decode_step_host(shape, layers, kvs, B: int, h_in_host, h_out_host, r_host, p_host, bits_host, seq_lens_host,
                     ws, ws_bytes: int, stream=None, check=True) -> int:
    la, ka = _arrays(layers, kvs)
    s = lib().sol_decode_step_host(C.byref(shape), len(layers), la, ka, B, _ptr(h_in_host), _ptr(h_out_host),
                                   _ptr(r_host), _ptr(p_host), _ptr(bits_host), _ptr(seq_lens_host), _ptr(ws),
                                   ws_bytes, _stream(stream))
    if check:
        _check(s, "sol_decode_step_host")
    return s


def read_device_status(ws, stream=None, check=True):
    out = (C.c_int32 * 8)()
    s = lib().sol_read_device_status(_ptr(ws), out, _stream(stream))
    if check:
        _check(s, "sol_read_device_status")
    return list(out)


def timing_enable(on: bool) -> None:
    lib().sol_timing_enable(1 if on else 0)


def timing_collect(max_entries: int = 64):
    buf = (SolKernelTime * max_entries)()
    n = lib().sol_timing_collect(buf, max_entries)
    return [(buf[i].name.decode(), int(buf[i].launches), float(buf[i].total_ms)) for i in range(n)]


def launch_count(reset: bool = False) -> int:
    return int(lib().sol_launch_count(1 if reset else 0))
