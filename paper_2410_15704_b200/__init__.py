"""Python binding of the B200 residual-VQ KV-cache library.

Argument marshalling only: every function below forwards to the C entry point
of the same name in ``librvq_b200.so`` (declared in ``include/rvq.h``).  PyTorch
supplies device memory and streams; all arithmetic runs in the CUDA kernels.
There is no CPU fallback: if the library is missing or fails to load, importing
this package raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librvq_b200.so")

F32, BF16, F16 = 0, 1, 2
CONTIGUOUS, STRIDED = 0, 1
TORCH_DTYPE = {F32: torch.float32, BF16: torch.bfloat16, F16: torch.float16}
DTYPE_OF = {v: k for k, v in TORCH_DTYPE.items()}


class RvqError(RuntimeError):
    pass


class rvq_config(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in
                ("dim", "group_dim", "layout", "depth", "codebook_size", "code_bits", "x_dtype", "std_ddof")]


STATUS_FIELDS = ("degenerate_vectors", "std_out_of_half", "rescored_rows", "exhaustive_rows",
                 "wait_timeouts", "bad_codes", "reserved0", "reserved1")


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python paper_2410_15704_b200/build.py` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
    cfgp = ctypes.POINTER(rvq_config)
    lib.rvq_status_string.restype = ctypes.c_char_p
    lib.rvq_status_string.argtypes = [ctypes.c_int]
    lib.rvq_version.restype = ctypes.c_int
    lib.rvq_code_bytes.restype = sz
    lib.rvq_code_bytes.argtypes = [cfgp]
    lib.rvq_prepared_bytes.restype = sz
    lib.rvq_prepared_bytes.argtypes = [cfgp]
    lib.rvq_workspace_bytes.restype = sz
    lib.rvq_workspace_bytes.argtypes = [cfgp, i64]
    lib.rvq_prepare_codebooks.restype = ctypes.c_int
    lib.rvq_prepare_codebooks.argtypes = [cfgp, vp, vp, vp]
    lib.rvq_encode.restype = ctypes.c_int
    lib.rvq_encode.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.rvq_selftest_encode_timeout.restype = ctypes.c_int
    lib.rvq_selftest_encode_timeout.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, ctypes.c_uint32, vp, vp]
    lib.rvq_encode_exact.restype = ctypes.c_int
    lib.rvq_encode_exact.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp]
    lib.rvq_encode_stats.restype = ctypes.c_int
    lib.rvq_encode_stats.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.rvq_decode.restype = ctypes.c_int
    lib.rvq_decode.argtypes = [cfgp, vp, vp, i64, vp, vp, vp, i64, vp, vp]
    lib.rvq_ema_update.restype = ctypes.c_int
    lib.rvq_ema_update.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, vp, ctypes.c_float,
                                   ctypes.c_float, vp, sz, vp, vp]
    lib.rvq_launch_count.restype = ctypes.c_uint64
    lib.rvq_ema_stats.restype = ctypes.c_int
    lib.rvq_ema_stats.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.rvq_ema_apply.restype = ctypes.c_int
    lib.rvq_ema_apply.argtypes = [cfgp, vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp]
    lib.rvq_ema_update_static.restype = ctypes.c_int
    lib.rvq_ema_update_static.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, vp, ctypes.c_float,
                                          ctypes.c_float, vp, vp]
    lib.rvq_ema_static_scratch_bytes.restype = sz
    lib.rvq_rope_table.restype = ctypes.c_int
    lib.rvq_rope_table.argtypes = [ctypes.c_int32, ctypes.c_double, ctypes.c_int32, vp, vp]
    lib.rvq_decode_rope.restype = ctypes.c_int
    lib.rvq_decode_rope.argtypes = [cfgp, vp, vp, i64, vp, vp, vp, ctypes.c_int32, vp, ctypes.c_int32,
                                    ctypes.c_int32, vp, i64, vp, vp]
    lib.rvq_attention_workspace_bytes.restype = sz
    lib.rvq_attention_workspace_bytes.argtypes = [i64, ctypes.c_int32]
    lib.rvq_attention_decode.restype = ctypes.c_int
    lib.rvq_attention_decode.argtypes = [cfgp, cfgp, vp, ctypes.c_int32, vp, vp, vp, vp, i64, ctypes.c_int32, vp, vp,
                                         vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_float, vp, vp, sz, vp, vp]
    lib.rvq_learn_step.restype = ctypes.c_int
    lib.rvq_learn_step.argtypes = [cfgp, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float,
                                   vp, sz, vp, vp]
    lib.rvq_kmeans_workspace_bytes.restype = sz
    lib.rvq_kmeans_workspace_bytes.argtypes = [cfgp, i64]
    lib.rvq_kmeans_init.restype = ctypes.c_int
    lib.rvq_kmeans_init.argtypes = [cfgp, vp, i64, i64, vp, ctypes.c_int32, vp, vp, vp, sz, vp, vp]
    return lib


lib = _load()

EXPORTS = ("rvq_attention_workspace_bytes", "rvq_attention_decode", "rvq_selftest_encode_timeout", "rvq_rope_table", "rvq_decode_rope", "rvq_learn_step", "rvq_kmeans_workspace_bytes", "rvq_kmeans_init", "rvq_encode_stats", "rvq_ema_update_static", "rvq_ema_static_scratch_bytes", "rvq_encode_exact", "rvq_status_string", "rvq_version", "rvq_launch_count", "rvq_ema_stats", "rvq_ema_apply", "rvq_code_bytes", "rvq_prepared_bytes",
           "rvq_prepare_codebooks", "rvq_workspace_bytes", "rvq_encode", "rvq_decode",
           "rvq_ema_update")


def make_config(dim=128, group_dim=32, layout=CONTIGUOUS, depth=8, codebook_size=2048,
                code_bits=16, x_dtype=BF16, std_ddof=0) -> rvq_config:
    return rvq_config(dim, group_dim, layout, depth, codebook_size, code_bits, x_dtype, std_ddof)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(rc: int, what: str):
    if rc != 0:
        raise RvqError(f"{what}: {lib.rvq_status_string(rc).decode()} ({rc})")


def rvq_status_string(code: int) -> str:
    return lib.rvq_status_string(code).decode()


def rvq_version() -> int:
    return lib.rvq_version()


def rvq_code_bytes(cfg: rvq_config) -> int:
    return lib.rvq_code_bytes(ctypes.byref(cfg))


def rvq_prepared_bytes(cfg: rvq_config) -> int:
    return lib.rvq_prepared_bytes(ctypes.byref(cfg))


def rvq_workspace_bytes(cfg: rvq_config, n: int) -> int:
    return lib.rvq_workspace_bytes(ctypes.byref(cfg), n)


def rvq_prepare_codebooks(cfg, codebooks, prepared, stream=None, check=True) -> int:
    rc = lib.rvq_prepare_codebooks(ctypes.byref(cfg), _ptr(codebooks), _ptr(prepared), _stream(stream))
    if check:
        _check(rc, "rvq_prepare_codebooks")
    return rc


def rvq_encode(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, workspace=None,
               workspace_bytes=0, status=None, stream=None, check=True, stage_energy=None) -> int:
    rc = lib.rvq_encode(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codebooks), _ptr(prepared),
                        _ptr(codes), _ptr(std_f16), _ptr(stage_energy), _ptr(workspace), workspace_bytes,
                        _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_encode")
    return rc


def rvq_encode_stats(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, batch_count, batch_sum,
                     workspace, workspace_bytes, status=None, stream=None, check=True, stage_energy=None) -> int:
    rc = lib.rvq_encode_stats(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codebooks), _ptr(prepared),
                              _ptr(codes), _ptr(std_f16), _ptr(stage_energy), _ptr(batch_count), _ptr(batch_sum),
                              _ptr(workspace), workspace_bytes, _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_encode_stats")
    return rc


def rvq_selftest_encode_timeout(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, wait_polls, status,
                                stream=None, check=True) -> int:
    """rvq_encode with one MMA chain left out per CTA: its wait gives up (include/rvq_selftest.h)."""
    rc = lib.rvq_selftest_encode_timeout(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codebooks), _ptr(prepared),
                                         _ptr(codes), _ptr(std_f16), wait_polls, _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_selftest_encode_timeout")
    return rc


def rvq_encode_exact(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, status=None,
                     stream=None, check=True, stage_energy=None) -> int:
    rc = lib.rvq_encode_exact(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codebooks), _ptr(prepared),
                              _ptr(codes), _ptr(std_f16), _ptr(stage_energy), _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_encode_exact")
    return rc


def rvq_decode(cfg, codes, std_f16, n, codebooks, prepared, x_out, out_row_stride, status=None,
               stream=None, check=True) -> int:
    rc = lib.rvq_decode(ctypes.byref(cfg), _ptr(codes), _ptr(std_f16), n, _ptr(codebooks),
                        _ptr(prepared), _ptr(x_out), out_row_stride, _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_decode")
    return rc


def rvq_ema_update(cfg, x, n, x_row_stride, codes, codebooks, ema_count, ema_sum, batch_count,
                   decay, eps, workspace, workspace_bytes, status=None, stream=None, check=True) -> int:
    rc = lib.rvq_ema_update(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codes), _ptr(codebooks),
                            _ptr(ema_count), _ptr(ema_sum), _ptr(batch_count), decay, eps,
                            _ptr(workspace), workspace_bytes, _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_ema_update")
    return rc


def rvq_ema_stats(cfg, x, n, x_row_stride, codes, codebooks, batch_count, batch_sum, workspace,
                  workspace_bytes, status=None, stream=None, check=True) -> int:
    rc = lib.rvq_ema_stats(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codes), _ptr(codebooks),
                           _ptr(batch_count), _ptr(batch_sum), _ptr(workspace), workspace_bytes,
                           _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_ema_stats")
    return rc


def rvq_ema_apply(cfg, batch_count, batch_sum, codebooks, ema_count, ema_sum, decay, eps,
                  stream=None, check=True) -> int:
    rc = lib.rvq_ema_apply(ctypes.byref(cfg), _ptr(batch_count), _ptr(batch_sum), _ptr(codebooks),
                           _ptr(ema_count), _ptr(ema_sum), decay, eps, _stream(stream))
    if check:
        _check(rc, "rvq_ema_apply")
    return rc


def rvq_ema_update_static(cfg, x, n, x_row_stride, codes, codebooks, ema_count, ema_sum, batch_count,
                          decay, eps, status=None, stream=None, check=True) -> int:
    """rvq_ema_update with the library's own fixed scratch: no workspace to pass, nothing
    allocated.  For callers that cannot obtain device memory themselves; see include/rvq.h
    for the size limit and for why overlapping calls must be ordered."""
    rc = lib.rvq_ema_update_static(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codes), _ptr(codebooks),
                                   _ptr(ema_count), _ptr(ema_sum), _ptr(batch_count), decay, eps,
                                   _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_ema_update_static")
    return rc


ROPE_HALVES, ROPE_ADJACENT = 0, 1


def rvq_rope_table(dim, base, positions, cos_sin, stream=None, check=True) -> int:
    """Fill cos_sin (float32 [positions][dim/2][2]) with the rotary embedding's cosines and sines."""
    rc = lib.rvq_rope_table(dim, float(base), positions, _ptr(cos_sin), _stream(stream))
    if check:
        _check(rc, "rvq_rope_table")
    return rc


def rvq_decode_rope(cfg, codes, std_f16, n, codebooks, prepared, position, vectors_per_position, cos_sin,
                    positions, pairing, x_out, out_row_stride, status=None, stream=None, check=True) -> int:
    """Decode and rotate: x_out = RoPE(decode(codes)) at the given positions (prepared may be None)."""
    rc = lib.rvq_decode_rope(ctypes.byref(cfg), _ptr(codes), _ptr(std_f16), n, _ptr(codebooks), _ptr(prepared),
                             _ptr(position),
                             vectors_per_position, _ptr(cos_sin), positions, pairing, _ptr(x_out), out_row_stride,
                             _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_decode_rope")
    return rc


def rvq_attention_workspace_bytes(tokens: int, q_heads: int) -> int:
    return int(lib.rvq_attention_workspace_bytes(tokens, q_heads))


def rvq_attention_decode(cfg_k, cfg_v, q, q_heads, codes_k, std_k, codes_v, std_v, tokens, kv_heads, codebooks_k,
                         codebooks_v, position, cos_sin, positions, pairing, scale, out, workspace, workspace_bytes,
                         status=None, stream=None, check=True) -> int:
    """out = attention of the query heads q over the compressed cache (keys rotated as they are read)."""
    rc = lib.rvq_attention_decode(ctypes.byref(cfg_k), ctypes.byref(cfg_v), _ptr(q), q_heads, _ptr(codes_k), _ptr(std_k),
                                  _ptr(codes_v), _ptr(std_v), tokens, kv_heads, _ptr(codebooks_k), _ptr(codebooks_v),
                                  _ptr(position), _ptr(cos_sin), positions, pairing, scale, _ptr(out), _ptr(workspace),
                                  workspace_bytes, _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_attention_decode")
    return rc


def rvq_learn_step(cfg, x, n, x_row_stride, codebooks, prepared, ema_count, ema_sum, codes, std_f16,
                   decay, eps, workspace, workspace_bytes, status=None, stream=None, check=True,
                   stage_energy=None) -> int:
    """Encode the batch, update N, M and the codebooks from its assignments, rebuild the prepared block."""
    rc = lib.rvq_learn_step(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(codebooks), _ptr(prepared),
                            _ptr(ema_count), _ptr(ema_sum), _ptr(codes), _ptr(std_f16), _ptr(stage_energy), decay, eps,
                            _ptr(workspace), workspace_bytes, _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_learn_step")
    return rc


def rvq_kmeans_workspace_bytes(cfg: rvq_config, n: int) -> int:
    return int(lib.rvq_kmeans_workspace_bytes(ctypes.byref(cfg), n))


def rvq_kmeans_init(cfg, x, n, x_row_stride, seed_rows, iterations, codebooks, prepared, workspace,
                    workspace_bytes, status=None, stream=None, check=True) -> int:
    """Stage-wise k-means initialisation of the codebooks from the int64 [R][K] seed rows."""
    rc = lib.rvq_kmeans_init(ctypes.byref(cfg), _ptr(x), n, x_row_stride, _ptr(seed_rows), iterations,
                             _ptr(codebooks), _ptr(prepared), _ptr(workspace), workspace_bytes,
                             _ptr(status), _stream(stream))
    if check:
        _check(rc, "rvq_kmeans_init")
    return rc


def rvq_ema_static_scratch_bytes() -> int:
    return int(lib.rvq_ema_static_scratch_bytes())


def rvq_launch_count() -> int:
    return int(lib.rvq_launch_count())


# --------------------------------------------------------------------------
# buffer helpers (device memory only; no arithmetic)
# --------------------------------------------------------------------------

def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(8, dtype=torch.int32, device=device)


def read_status(status: torch.Tensor) -> dict:
    vals = status.cpu().tolist()
    return {k: int(v) & 0xFFFFFFFF for k, v in zip(STATUS_FIELDS, vals)}


@dataclass
class Buffers:
    """Device buffers of one quantizer for up to ``n`` head vectors."""
    cfg: rvq_config
    n: int
    codebooks: torch.Tensor
    prepared: torch.Tensor
    codes: torch.Tensor
    std: torch.Tensor
    workspace: torch.Tensor
    status: torch.Tensor

    @property
    def workspace_bytes(self) -> int:
        return self.workspace.numel()


def alloc_buffers(cfg: rvq_config, n: int, codebooks, device="cuda") -> Buffers:
    """Allocate the caller-owned buffers the C entry points expect and run
    rvq_prepare_codebooks on them."""
    cb = torch.as_tensor(codebooks, dtype=torch.float32).to(device).contiguous()
    prepared = torch.empty(max(256, rvq_prepared_bytes(cfg)), dtype=torch.uint8, device=device)
    codes = torch.empty(max(1, n) * rvq_code_bytes(cfg), dtype=torch.uint8, device=device)
    std = torch.empty(max(1, n), dtype=torch.int16, device=device)
    ws = torch.empty(max(256, rvq_workspace_bytes(cfg, n)), dtype=torch.uint8, device=device)
    b = Buffers(cfg, n, cb, prepared, codes, std, ws, new_status(device))
    rvq_prepare_codebooks(cfg, b.codebooks, b.prepared)
    return b
