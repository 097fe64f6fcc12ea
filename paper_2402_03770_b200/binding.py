"""Thin ctypes binding of libcvlc (same names as include/cvlc.h).

Argument marshalling only: every step of the compression path runs in the CUDA
kernels of libcvlc.so.  torch provides device memory and the stream handle.
There is no CPU fallback: if the library is missing, importing the entry points
raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcvlc.so")

CVLC_OK = 0
CVLC_ERR_INVALID_ARG = 1
CVLC_ERR_BUDGET_TOO_SMALL = 2
CVLC_ERR_BUDGET_TOO_LARGE = 3
CVLC_ERR_PACKET_TOO_SMALL = 4
CVLC_ERR_NONFINITE_INPUT = 5
CVLC_ERR_WORKSPACE_TOO_SMALL = 6
CVLC_ERR_OUTPUT_TOO_SMALL = 7
CVLC_ERR_BAD_STREAM = 8
CVLC_ERR_DEVICE_TIMEOUT = 9
CVLC_ERR_CUDA = 10
CVLC_ERR_NOT_IMPLEMENTED = 11
CVLC_ERR_SCALE_TOO_SMALL = 12
CVLC_ERR_PLAN_MISMATCH = 13

CVLC_QUANT_PQ = 0
CVLC_QUANT_QSGD = 1

MAX_CODE_BITS = 32
MAX_BATCH = 512
HIST_BINS = 4096
PLAN_BYTES = 512
PLAN_WS_HIST_OFFSET = 256

EXPORTS = [
    "cvlc_version", "cvlc_status_string", "cvlc_set_device", "cvlc_stream_bytes", "cvlc_default_scale",
    "cvlc_plan_workspace_bytes", "cvlc_encode_workspace_bytes", "cvlc_decode_workspace_bytes",
    "cvlc_plan", "cvlc_plan_fixed", "cvlc_encode", "cvlc_plan_batch_workspace_bytes",
    "cvlc_encode_batch_workspace_bytes", "cvlc_plan_batch", "cvlc_encode_batch", "cvlc_decode_aggregate", "cvlc_read_status",
    "cvlc_selftest_philox", "cvlc_selftest_math", "cvlc_histogram_batch", "cvlc_plan_from_histogram_batch", "cvlc_decode_apply",
    "cvlc_decode_aggregate_noalloc", "cvlc_compress_batch", "cvlc_selftest_wait", "cvlc_plan_literal",
    "cvlc_plan_literal_workspace_bytes", "cvlc_ec_accumulate_batch", "cvlc_encode_batch_ec",
    "cvlc_unframed_stream_capacity", "cvlc_unframed_workspace_bytes", "cvlc_encode_unframed_batch", "cvlc_decode_aggregate_unframed", "cvlc_launch_count", "cvlc_profile_select", "cvlc_profile_reset", "cvlc_profile_read",
]


class CvlcParams(C.Structure):
    _fields_ = [
        ("d", C.c_uint64), ("budget_bits", C.c_uint64),
        ("packet_bits", C.c_uint32), ("header_bits", C.c_uint32),
        ("quantizer", C.c_uint32), ("max_code_bits", C.c_uint32),
        ("scale_B", C.c_double), ("seed", C.c_uint64),
        ("client_id", C.c_uint32), ("round", C.c_uint32),
    ]


class CvlcPlan(C.Structure):
    _fields_ = [
        ("status", C.c_int32), ("s", C.c_uint32), ("R", C.c_uint32), ("y_min", C.c_uint32),
        ("n_lengths", C.c_uint32), ("thresh_bin", C.c_uint32),
        ("k", C.c_uint64), ("n_candidates", C.c_uint64),
        ("alpha", C.c_double), ("alpha_q", C.c_double), ("beta", C.c_double),
        ("gamma", C.c_double), ("B_next", C.c_double),
        ("n_y", C.c_uint32 * (MAX_CODE_BITS + 1)), ("cap", C.c_uint32 * (MAX_CODE_BITS + 1)),
        ("top_bin", C.c_uint32), ("reserved0", C.c_uint32),
        ("reserved", C.c_uint8 * (512 - 88 - 2 * 4 * (MAX_CODE_BITS + 1))),
    ]


assert C.sizeof(CvlcPlan) == PLAN_BYTES


class CvlcError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: status {code} ({status_string(code)})")
        self.code = code


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Loads libcvlc.so; raises if it has not been built (there is nothing to fall back to)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2402_03770_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, u32, u64, f64, sz = C.c_void_p, C.c_uint32, C.c_uint64, C.c_double, C.c_size_t
    PP = C.POINTER(CvlcParams)
    L.cvlc_version.restype = C.c_int
    L.cvlc_version.argtypes = []
    L.cvlc_status_string.restype = C.c_char_p
    L.cvlc_status_string.argtypes = [C.c_int]
    L.cvlc_set_device.restype = C.c_int
    L.cvlc_set_device.argtypes = [C.c_int]
    L.cvlc_stream_bytes.restype = sz
    L.cvlc_stream_bytes.argtypes = [PP]
    L.cvlc_default_scale.restype = f64
    L.cvlc_default_scale.argtypes = [PP]
    L.cvlc_plan_workspace_bytes.restype = sz
    L.cvlc_plan_workspace_bytes.argtypes = [PP]
    L.cvlc_encode_workspace_bytes.restype = sz
    L.cvlc_encode_workspace_bytes.argtypes = [PP]
    L.cvlc_decode_workspace_bytes.restype = sz
    L.cvlc_decode_workspace_bytes.argtypes = [u32]
    L.cvlc_plan.restype = C.c_int
    L.cvlc_plan.argtypes = [vp, PP, vp, vp, sz, vp]
    L.cvlc_plan_fixed.restype = C.c_int
    L.cvlc_plan_fixed.argtypes = [vp, PP, u32, vp, vp, sz, vp]
    L.cvlc_encode.restype = C.c_int
    L.cvlc_encode.argtypes = [vp, PP, vp, vp, vp, sz, vp, sz, vp]
    L.cvlc_plan_batch_workspace_bytes.restype = sz
    L.cvlc_plan_batch_workspace_bytes.argtypes = [PP, u32]
    L.cvlc_encode_batch_workspace_bytes.restype = sz
    L.cvlc_encode_batch_workspace_bytes.argtypes = [PP, u32, u64]
    L.cvlc_plan_batch.restype = C.c_int
    L.cvlc_plan_batch.argtypes = [vp, PP, u32, u32, vp, vp, sz, vp]
    L.cvlc_encode_batch.restype = C.c_int
    L.cvlc_encode_batch.argtypes = [vp, PP, u32, vp, vp, vp, sz, u64, vp, sz, vp]
    L.cvlc_compress_batch.restype = C.c_int
    L.cvlc_compress_batch.argtypes = [vp, PP, u32, u32, vp, vp, sz, u64, vp, sz, vp, sz, vp, vp]
    L.cvlc_plan_literal_workspace_bytes.restype = sz
    L.cvlc_plan_literal_workspace_bytes.argtypes = [PP, u32]
    L.cvlc_plan_literal.restype = C.c_int
    L.cvlc_plan_literal.argtypes = [PP, f64, u32, u32, vp, vp, vp, sz, vp]
    L.cvlc_ec_accumulate_batch.restype = C.c_int
    L.cvlc_ec_accumulate_batch.argtypes = [vp, vp, u32, u64, vp]
    L.cvlc_encode_batch_ec.restype = C.c_int
    L.cvlc_encode_batch_ec.argtypes = [vp, PP, u32, vp, vp, vp, sz, u64, vp, sz, vp]
    L.cvlc_unframed_stream_capacity.restype = sz
    L.cvlc_unframed_stream_capacity.argtypes = [PP]
    L.cvlc_unframed_workspace_bytes.restype = sz
    L.cvlc_unframed_workspace_bytes.argtypes = [PP, u32]
    L.cvlc_encode_unframed_batch.restype = C.c_int
    L.cvlc_encode_unframed_batch.argtypes = [vp, PP, u32, vp, vp, vp, sz, vp, u64, vp, sz, vp, sz, vp]
    L.cvlc_decode_aggregate_unframed.restype = C.c_int
    L.cvlc_decode_aggregate_unframed.argtypes = [vp, vp, vp, u32, f64, u64, vp, C.c_int, vp, sz, vp]
    L.cvlc_selftest_wait.restype = C.c_int
    L.cvlc_selftest_wait.argtypes = [vp, vp, u32, vp]
    L.cvlc_decode_aggregate.restype = C.c_int
    L.cvlc_decode_aggregate.argtypes = [vp, vp, vp, u32, f64, u64, vp, C.c_int, vp, sz, vp]
    L.cvlc_histogram_batch.restype = C.c_int
    L.cvlc_histogram_batch.argtypes = [vp, PP, u32, vp, vp, sz, vp]
    L.cvlc_plan_from_histogram_batch.restype = C.c_int
    L.cvlc_plan_from_histogram_batch.argtypes = [vp, PP, u32, vp, vp, sz, vp]
    L.cvlc_decode_apply.restype = C.c_int
    L.cvlc_decode_apply.argtypes = [vp, vp, vp, u32, f64, u64, vp, vp, vp, sz, vp]
    L.cvlc_decode_aggregate_noalloc.restype = C.c_int
    L.cvlc_decode_aggregate_noalloc.argtypes = [vp, vp, vp, u32, f64, u64, vp, C.c_int, vp, vp]
    L.cvlc_read_status.restype = C.c_int
    L.cvlc_read_status.argtypes = [vp, vp]
    L.cvlc_selftest_philox.restype = C.c_int
    L.cvlc_selftest_philox.argtypes = [u64, u32, u32, u64, u64, vp, vp]
    L.cvlc_selftest_math.restype = C.c_int
    L.cvlc_selftest_math.argtypes = [vp, u64, vp, vp, vp, vp, vp]
    L.cvlc_launch_count.restype = C.c_ulonglong
    L.cvlc_launch_count.argtypes = [C.c_char_p]
    L.cvlc_profile_select.restype = C.c_int
    L.cvlc_profile_select.argtypes = [C.c_char_p, u32]
    L.cvlc_profile_reset.restype = C.c_int
    L.cvlc_profile_reset.argtypes = []
    L.cvlc_profile_read.restype = C.c_int
    L.cvlc_profile_read.argtypes = [C.c_char_p, C.POINTER(u32), C.POINTER(f64)]
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().cvlc_status_string(int(code)).decode()


def make_params(d: int, budget_bits: int, *, packet_bits: int = 12000, header_bits: int = 80,
                quantizer: int = 0, max_code_bits: int = 32, scale_B: Optional[float] = None,
                seed: int = 0, client_id: int = 0, round: int = 0) -> CvlcParams:
    p = CvlcParams(d, budget_bits, packet_bits, header_bits, quantizer, max_code_bits, 1.0, seed,
                   client_id, round)
    p.scale_B = cvlc_default_scale(p) if scale_B is None else float(scale_B)
    return p


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> int:
    st = torch.cuda.current_stream() if stream is None else stream
    return int(st.cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


def _check(rc: int, where: str) -> None:
    if rc != CVLC_OK:
        raise CvlcError(rc, where)


# ---- host-only helpers -------------------------------------------------------------

def cvlc_set_device(device: int) -> None:
    _check(lib().cvlc_set_device(int(device)), "cvlc_set_device")


def cvlc_stream_bytes(p: CvlcParams) -> int:
    return int(lib().cvlc_stream_bytes(C.byref(p)))


def cvlc_default_scale(p: CvlcParams) -> float:
    return float(lib().cvlc_default_scale(C.byref(p)))


def cvlc_plan_workspace_bytes(p: CvlcParams) -> int:
    return int(lib().cvlc_plan_workspace_bytes(C.byref(p)))


def cvlc_encode_workspace_bytes(p: CvlcParams) -> int:
    return int(lib().cvlc_encode_workspace_bytes(C.byref(p)))


def cvlc_decode_workspace_bytes(n_clients: int) -> int:
    return int(lib().cvlc_decode_workspace_bytes(int(n_clients)))


# ---- the hot path (device tensors in, kernels enqueued on the stream) ----------------

def cvlc_plan(x: torch.Tensor, p: CvlcParams, plan: torch.Tensor, ws: torch.Tensor,
              stream: Optional[torch.cuda.Stream] = None) -> None:
    assert x.dtype == torch.float32 and x.numel() == p.d
    assert plan.dtype == torch.uint8 and plan.numel() >= PLAN_BYTES
    _check(lib().cvlc_plan(_ptr(x), C.byref(p), _ptr(plan), _ptr(ws), ws.numel() * ws.element_size(),
                           _stream_handle(stream)), "cvlc_plan")


def cvlc_plan_fixed(x: torch.Tensor, p: CvlcParams, y: int, plan: torch.Tensor, ws: torch.Tensor,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
    assert x.dtype == torch.float32 and x.numel() == p.d
    _check(lib().cvlc_plan_fixed(_ptr(x), C.byref(p), int(y), _ptr(plan), _ptr(ws),
                                 ws.numel() * ws.element_size(), _stream_handle(stream)), "cvlc_plan_fixed")


def cvlc_encode(x: torch.Tensor, p: CvlcParams, plan: torch.Tensor, out_stream: torch.Tensor,
                ws: torch.Tensor, stream: Optional[torch.cuda.Stream] = None,
                plan_ws: Optional[torch.Tensor] = None) -> None:
    """plan_ws: the workspace cvlc_plan used for this plan (fast selection) or None (look-back selection)."""
    assert x.dtype == torch.float32 and x.numel() == p.d
    assert out_stream.dtype == torch.uint8
    _check(lib().cvlc_encode(_ptr(x), C.byref(p), _ptr(plan), _ptr(plan_ws), _ptr(out_stream), out_stream.numel(),
                             _ptr(ws), ws.numel() * ws.element_size(), _stream_handle(stream)), "cvlc_encode")


def cvlc_plan_batch_workspace_bytes(p: CvlcParams, n: int) -> int:
    return int(lib().cvlc_plan_batch_workspace_bytes(C.byref(p), int(n)))


def cvlc_encode_batch_workspace_bytes(p: CvlcParams, n: int, max_candidates: int = 0) -> int:
    return int(lib().cvlc_encode_batch_workspace_bytes(C.byref(p), int(n), int(max_candidates)))


def _ptr_array(tensors: Sequence[torch.Tensor]):
    return (C.c_void_p * len(tensors))(*[_ptr(t) for t in tensors])


def _params_array(params: Sequence[CvlcParams]):
    return (CvlcParams * len(params))(*params)


def cvlc_plan_batch(xs: Sequence[torch.Tensor], params: Sequence[CvlcParams], plans: torch.Tensor, ws: torch.Tensor,
                    fixed_y: int = 0, stream: Optional[torch.cuda.Stream] = None, _cache=None) -> None:
    """xs: n device tensors; params: n CvlcParams; plans: device uint8 tensor of n * 512 bytes."""
    n = len(xs)
    assert len(params) == n and plans.dtype == torch.uint8 and plans.numel() >= n * PLAN_BYTES
    xa, pa = _cache if _cache is not None else (_ptr_array(xs), _params_array(params))
    _check(lib().cvlc_plan_batch(xa, pa, n, int(fixed_y), _ptr(plans), _ptr(ws), ws.numel() * ws.element_size(),
                                 _stream_handle(stream)), "cvlc_plan_batch")


def cvlc_encode_batch(xs: Sequence[torch.Tensor], params: Sequence[CvlcParams], plans: torch.Tensor,
                      outs: Sequence[torch.Tensor], ws: torch.Tensor, max_candidates: int = 0,
                      stream: Optional[torch.cuda.Stream] = None, _cache=None,
                      plan_ws: Optional[torch.Tensor] = None) -> None:
    """outs: n device uint8 tensors of cvlc_stream_bytes(params[0]) bytes each."""
    n = len(xs)
    assert len(params) == n and len(outs) == n
    xa, pa, oa = _cache if _cache is not None else (_ptr_array(xs), _params_array(params), _ptr_array(outs))
    cap = min(o.numel() for o in outs)
    _check(lib().cvlc_encode_batch(xa, pa, n, _ptr(plans), _ptr(plan_ws), oa, cap, int(max_candidates), _ptr(ws),
                                   ws.numel() * ws.element_size(), _stream_handle(stream)), "cvlc_encode_batch")


def cvlc_compress_batch(xs: Sequence[torch.Tensor], params: Sequence[CvlcParams], plans: torch.Tensor,
                        outs: Sequence[torch.Tensor], plan_ws: torch.Tensor, enc_ws: torch.Tensor, max_candidates: int = 0,
                        fixed_y: int = 0, stream: Optional[torch.cuda.Stream] = None,
                        side_stream: Optional[torch.cuda.Stream] = None, _cache=None) -> None:
    """plan + encode of n clients in one call; with side_stream the length tuning runs next to selection and ranking."""
    n = len(xs)
    assert len(params) == n and len(outs) == n and plans.numel() >= n * PLAN_BYTES
    xa, pa, oa = _cache if _cache is not None else (_ptr_array(xs), _params_array(params), _ptr_array(outs))
    cap = min(o.numel() for o in outs)
    side = None if side_stream is None else int(side_stream.cuda_stream)
    _check(lib().cvlc_compress_batch(xa, pa, n, int(fixed_y), _ptr(plans), oa, cap, int(max_candidates), _ptr(plan_ws),
                                     plan_ws.numel() * plan_ws.element_size(), _ptr(enc_ws),
                                     enc_ws.numel() * enc_ws.element_size(), _stream_handle(stream), side),
           "cvlc_compress_batch")


def cvlc_ec_accumulate_batch(memories: Sequence[torch.Tensor], updates: Sequence[torch.Tensor],
                             stream: Optional[torch.cuda.Stream] = None) -> None:
    """memory <- memory + update for every client (error compensation, first step of a round)"""
    n = len(memories)
    assert len(updates) == n and all(m.dtype == torch.float32 and u.dtype == torch.float32 and m.numel() == u.numel()
                                     for m, u in zip(memories, updates))
    _check(lib().cvlc_ec_accumulate_batch(_ptr_array(memories), _ptr_array(updates), n, memories[0].numel(),
                                          _stream_handle(stream)), "cvlc_ec_accumulate_batch")


def cvlc_encode_batch_ec(memories: Sequence[torch.Tensor], params: Sequence[CvlcParams], plans: torch.Tensor,
                         outs: Sequence[torch.Tensor], ws: torch.Tensor, max_candidates: int = 0,
                         stream: Optional[torch.cuda.Stream] = None, plan_ws: Optional[torch.Tensor] = None) -> None:
    """cvlc_encode_batch on the compensated updates; on return they hold the new error-compensation memories"""
    n = len(memories)
    assert len(params) == n and len(outs) == n
    cap = min(o.numel() for o in outs)
    _check(lib().cvlc_encode_batch_ec(_ptr_array(memories), _params_array(params), n, _ptr(plans), _ptr(plan_ws),
                                      _ptr_array(outs), cap, int(max_candidates), _ptr(ws), ws.numel() * ws.element_size(),
                                      _stream_handle(stream)), "cvlc_encode_batch_ec")


def cvlc_unframed_stream_capacity(p: CvlcParams) -> int:
    return int(lib().cvlc_unframed_stream_capacity(C.byref(p)))


def cvlc_unframed_workspace_bytes(p: CvlcParams, n: int) -> int:
    return int(lib().cvlc_unframed_workspace_bytes(C.byref(p), int(n)))


def cvlc_encode_unframed_batch(xs: Sequence[torch.Tensor], params: Sequence[CvlcParams], plans: torch.Tensor,
                               outs: Sequence[torch.Tensor], sizes: Optional[torch.Tensor], enc_ws: torch.Tensor,
                               uf_ws: torch.Tensor, max_candidates: int = 0, stream: Optional[torch.cuda.Stream] = None,
                               plan_ws: Optional[torch.Tensor] = None) -> None:
    """the unframed (version 2) streams of n planned clients; sizes: device int64[n] that receives their lengths"""
    n = len(xs)
    assert len(params) == n and len(outs) == n
    cap = min(o.numel() for o in outs)
    _check(lib().cvlc_encode_unframed_batch(_ptr_array(xs), _params_array(params), n, _ptr(plans), _ptr(plan_ws),
                                            _ptr_array(outs), cap, _ptr(sizes), int(max_candidates), _ptr(enc_ws),
                                            enc_ws.numel() * enc_ws.element_size(), _ptr(uf_ws),
                                            uf_ws.numel() * uf_ws.element_size(), _stream_handle(stream)),
           "cvlc_encode_unframed_batch")


def cvlc_decode_aggregate_unframed(stream_ptrs: torch.Tensor, stream_bytes: torch.Tensor, weights: torch.Tensor,
                                   n_clients: int, weight_total: float, d: int, out: torch.Tensor, accumulate: bool,
                                   ws: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    assert weights.dtype == torch.float32 and out.dtype == torch.float32 and out.numel() == d
    _check(lib().cvlc_decode_aggregate_unframed(_ptr(stream_ptrs), _ptr(stream_bytes), _ptr(weights), int(n_clients),
                                                float(weight_total), int(d), _ptr(out), 1 if accumulate else 0, _ptr(ws),
                                                ws.numel() * ws.element_size(), _stream_handle(stream)),
           "cvlc_decode_aggregate_unframed")


class CvlcLiteralPlan(C.Structure):
    _fields_ = [("status", C.c_int32), ("R", C.c_uint32), ("n_k", C.c_uint32), ("sweeps", C.c_uint32),
                ("k_star", C.c_uint64), ("gamma_star", C.c_double), ("alpha_q", C.c_double), ("beta", C.c_double),
                ("reserved", C.c_uint8 * 16)]


assert C.sizeof(CvlcLiteralPlan) == 64


def cvlc_plan_literal(p: CvlcParams, alpha_q: float, n_k: int, max_sweeps: int, device: torch.device,
                      stream: Optional[torch.cuda.Stream] = None):
    """Problem P2 with real-valued packet sizes (plan only).  Returns (CvlcLiteralPlan, P_star, k_grid, gamma_of_k,
    sweeps_of_k) as host copies; allocates its buffers itself (marshalling and allocation only)."""
    nbytes = int(lib().cvlc_plan_literal_workspace_bytes(C.byref(p), int(n_k)))
    R = int(p.budget_bits // p.packet_bits)
    ws = alloc_bytes(max(nbytes, 256), device)
    out = alloc_bytes(64, device)
    P_star = torch.zeros(max(R, 1), dtype=torch.float64, device=device)
    _check(lib().cvlc_plan_literal(C.byref(p), float(alpha_q), int(n_k), int(max_sweeps), _ptr(out), _ptr(P_star), _ptr(ws),
                                   ws.numel(), _stream_handle(stream)), "cvlc_plan_literal")
    head = CvlcLiteralPlan.from_buffer_copy(bytes(out.cpu().numpy().tobytes()))
    raw = ws.cpu().numpy()
    a256 = lambda v: (v + 255) & ~255
    off_k = 256
    off_g = a256(off_k + 8 * n_k)
    off_s = a256(off_g + 8 * n_k)
    import numpy as np
    k_grid = raw[off_k:off_k + 8 * n_k].view(np.uint64).copy()
    gamma = raw[off_g:off_g + 8 * n_k].view(np.float64).copy()
    sweeps = raw[off_s:off_s + 4 * n_k].view(np.uint32).copy()
    return head, P_star.cpu().numpy(), k_grid, gamma, sweeps


def cvlc_selftest_wait(word: torch.Tensor, status: torch.Tensor, max_polls: int,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    assert word.element_size() == 8 and status.dtype == torch.int32
    _check(lib().cvlc_selftest_wait(_ptr(word), _ptr(status), int(max_polls), _stream_handle(stream)), "cvlc_selftest_wait")


def cvlc_decode_aggregate(stream_ptrs: torch.Tensor, stream_bytes: torch.Tensor, weights: torch.Tensor,
                          n_clients: int, weight_total: float, d: int, out: torch.Tensor, accumulate: bool,
                          ws: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    assert stream_ptrs.dtype in (torch.int64, torch.uint64) and stream_ptrs.numel() >= n_clients
    assert stream_bytes.dtype in (torch.int64, torch.uint64) and stream_bytes.numel() >= n_clients
    assert weights.dtype == torch.float32 and out.dtype == torch.float32 and out.numel() == d
    _check(lib().cvlc_decode_aggregate(_ptr(stream_ptrs), _ptr(stream_bytes), _ptr(weights), int(n_clients),
                                       float(weight_total), int(d), _ptr(out), 1 if accumulate else 0,
                                       _ptr(ws), ws.numel() * ws.element_size(), _stream_handle(stream)),
           "cvlc_decode_aggregate")


def cvlc_histogram_batch(xs: Sequence[torch.Tensor], params: Sequence[CvlcParams], hist: torch.Tensor, ws: torch.Tensor,
                         stream: Optional[torch.cuda.Stream] = None) -> None:
    """hist: device int64/uint64 tensor of n * HIST_BINS counts (what a client sends when the server plans)."""
    n = len(xs)
    assert len(params) == n and hist.element_size() == 8 and hist.numel() >= n * HIST_BINS
    _check(lib().cvlc_histogram_batch(_ptr_array(xs), _params_array(params), n, _ptr(hist), _ptr(ws),
                                      ws.numel() * ws.element_size(), _stream_handle(stream)), "cvlc_histogram_batch")


def cvlc_plan_from_histogram_batch(hist: torch.Tensor, params: Sequence[CvlcParams], plans: torch.Tensor,
                                   ws: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    n = len(params)
    assert hist.element_size() == 8 and hist.numel() >= n * HIST_BINS
    assert plans.dtype == torch.uint8 and plans.numel() >= n * PLAN_BYTES
    _check(lib().cvlc_plan_from_histogram_batch(_ptr(hist), _params_array(params), n, _ptr(plans), _ptr(ws),
                                                ws.numel() * ws.element_size(), _stream_handle(stream)),
           "cvlc_plan_from_histogram_batch")


def cvlc_decode_apply(stream_ptrs: torch.Tensor, stream_bytes: torch.Tensor, weights: torch.Tensor, n_clients: int,
                      weight_total: float, d: int, model: torch.Tensor, aggregate: torch.Tensor, ws: torch.Tensor,
                      stream: Optional[torch.cuda.Stream] = None) -> None:
    """model <- model - aggregate of the decoded streams; `aggregate` (d fp32) receives the aggregate."""
    assert model.dtype == torch.float32 and model.numel() == d
    assert aggregate.dtype == torch.float32 and aggregate.numel() == d
    _check(lib().cvlc_decode_apply(_ptr(stream_ptrs), _ptr(stream_bytes), _ptr(weights), int(n_clients),
                                   float(weight_total), int(d), _ptr(model), _ptr(aggregate), _ptr(ws),
                                   ws.numel() * ws.element_size(), _stream_handle(stream)), "cvlc_decode_apply")


NOALLOC_MAX_CLIENTS = 256


def cvlc_decode_aggregate_noalloc(stream_ptrs: torch.Tensor, stream_bytes: torch.Tensor, weights: torch.Tensor,
                                  n_clients: int, weight_total: float, d: int, out: torch.Tensor,
                                  accumulate: bool, status: torch.Tensor,
                                  stream: Optional[torch.cuda.Stream] = None) -> None:
    """cvlc_decode_aggregate without a workspace argument: for callers that may not allocate
    device memory.  Uses the library's built-in scratch (at most NOALLOC_MAX_CLIENTS clients);
    `status` is one int32 device word that receives the device status.  Calls on one device
    must not overlap on the GPU."""
    assert status.dtype == torch.int32 and status.numel() >= 1
    assert weights.dtype == torch.float32 and out.dtype == torch.float32 and out.numel() == d
    _check(lib().cvlc_decode_aggregate_noalloc(_ptr(stream_ptrs), _ptr(stream_bytes), _ptr(weights), int(n_clients),
                                               float(weight_total), int(d), _ptr(out), 1 if accumulate else 0,
                                               _ptr(status), _stream_handle(stream)),
           "cvlc_decode_aggregate_noalloc")


def cvlc_read_status(plan_or_ws: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
    return int(lib().cvlc_read_status(_ptr(plan_or_ws), _stream_handle(stream)))


def cvlc_selftest_philox(seed: int, client_id: int, round: int, first: int, n: int, out: torch.Tensor,
                         stream: Optional[torch.cuda.Stream] = None) -> None:
    assert out.dtype in (torch.int32, torch.uint32) and out.numel() >= 4 * n
    _check(lib().cvlc_selftest_philox(seed, client_id, round, first, n, _ptr(out), _stream_handle(stream)),
           "cvlc_selftest_philox")


def cvlc_selftest_math(inp: torch.Tensor, log2_out: Optional[torch.Tensor], exp2_out: Optional[torch.Tensor],
                       div_out: Optional[torch.Tensor], div_ref: Optional[torch.Tensor],
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    assert inp.dtype == torch.float64
    _check(lib().cvlc_selftest_math(_ptr(inp), inp.numel(), _ptr(log2_out), _ptr(exp2_out), _ptr(div_out),
                                    _ptr(div_ref), _stream_handle(stream)), "cvlc_selftest_math")


def cvlc_launch_count(kernel_name: str = "") -> int:
    return int(lib().cvlc_launch_count(kernel_name.encode()))


def cvlc_profile_select(kernel_name: Optional[str], max_launches: int) -> None:
    _check(lib().cvlc_profile_select((kernel_name or "").encode(), int(max_launches)), "cvlc_profile_select")


def cvlc_profile_reset() -> None:
    _check(lib().cvlc_profile_reset(), "cvlc_profile_reset")


KERNEL_NAMES = ["k_zero_words", "k_hist", "k_plan_fit", "k_plan_tune", "k_plan_finish", "k_encode_init", "k_select",
                "k_select_lookback", "k_sort_hist", "k_sort_scan", "k_sort_pass", "k_pack", "k_decode_prepare", "k_fill_zero",
                "k_prefetch_l2", "k_decode", "k_noalloc_publish_status", "k_selftest", "k_hist_check", "k_apply", "k_plan_literal", "k_ec_accumulate", "k_pack_unframed", "k_decode_unframed"]


def cvlc_profile_read(kernel_name: str = "*"):
    n, ms = C.c_uint32(), C.c_double()
    _check(lib().cvlc_profile_read(kernel_name.encode(), C.byref(n), C.byref(ms)), "cvlc_profile_read")
    return int(n.value), float(ms.value)


# ---- buffer helpers (allocation only) ---------------------------------------------------

def alloc_bytes(n: int, device: torch.device) -> torch.Tensor:
    """Device byte buffer; torch's caching allocator returns 512-byte aligned blocks."""
    return torch.empty(max(int(n), 1), dtype=torch.uint8, device=device)


def read_plan(plan: torch.Tensor) -> CvlcPlan:
    """Copies a device plan to the host (synchronises the current stream)."""
    raw = bytes(plan[:PLAN_BYTES].cpu().numpy().tobytes())
    return CvlcPlan.from_buffer_copy(raw)


class ClientEncoder:
    """Owns the buffers one client's plan + encode needs; all work is enqueued on `stream`."""

    def __init__(self, p: CvlcParams, device: torch.device):
        self.p = p
        self.device = device
        self.plan = alloc_bytes(PLAN_BYTES, device)
        self.plan_ws = alloc_bytes(cvlc_plan_workspace_bytes(p), device)
        self.enc_ws = alloc_bytes(cvlc_encode_workspace_bytes(p), device)
        self.out = alloc_bytes(cvlc_stream_bytes(p), device)

    def run(self, x: torch.Tensor, p: Optional[CvlcParams] = None, out: Optional[torch.Tensor] = None,
            stream: Optional[torch.cuda.Stream] = None, fixed_y: int = 0, use_plan_ws: bool = True) -> torch.Tensor:
        p = self.p if p is None else p
        out = self.out if out is None else out
        if fixed_y:
            cvlc_plan_fixed(x, p, fixed_y, self.plan, self.plan_ws, stream)
        else:
            cvlc_plan(x, p, self.plan, self.plan_ws, stream)
        cvlc_encode(x, p, self.plan, out, self.enc_ws, stream, plan_ws=self.plan_ws if use_plan_ws else None)
        return out

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        rc = cvlc_read_status(self.plan, stream)
        return rc if rc != CVLC_OK else cvlc_read_status(self.enc_ws, stream)


class BatchEncoder:
    """Buffers for plan + encode of a batch of n clients that share a problem shape."""

    def __init__(self, params: Sequence[CvlcParams], device: torch.device, max_candidates: int = 0):
        self.params = list(params)
        self.n = len(self.params)
        self.device = device
        self.max_candidates = max_candidates
        p0 = self.params[0]
        self.plans = alloc_bytes(PLAN_BYTES * self.n, device)
        self.plan_ws = alloc_bytes(cvlc_plan_batch_workspace_bytes(p0, self.n), device)
        self.enc_ws = alloc_bytes(cvlc_encode_batch_workspace_bytes(p0, self.n, max_candidates), device)
        self.outs = [alloc_bytes(cvlc_stream_bytes(p0), device) for _ in range(self.n)]
        self._pa = _params_array(self.params)
        self._oa = _ptr_array(self.outs)

    def plan(self, xs: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None, fixed_y: int = 0):
        self._xa = _ptr_array(xs)
        cvlc_plan_batch(xs, self.params, self.plans, self.plan_ws, fixed_y, stream, _cache=(self._xa, self._pa))

    def encode(self, xs: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None, use_plan_ws: bool = True):
        cvlc_encode_batch(xs, self.params, self.plans, self.outs, self.enc_ws, self.max_candidates, stream,
                          _cache=(self._xa, self._pa, self._oa), plan_ws=self.plan_ws if use_plan_ws else None)
        return self.outs

    def run(self, xs: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None, fixed_y: int = 0,
            use_plan_ws: bool = True):
        self.plan(xs, stream, fixed_y)
        return self.encode(xs, stream, use_plan_ws)

    def compress(self, xs: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None,
                 side_stream: Optional[torch.cuda.Stream] = None, fixed_y: int = 0):
        """plan + encode in one call (cvlc_compress_batch)"""
        self._xa = _ptr_array(xs)
        cvlc_compress_batch(xs, self.params, self.plans, self.outs, self.plan_ws, self.enc_ws, self.max_candidates,
                            fixed_y, stream, side_stream, _cache=(self._xa, self._pa, self._oa))
        return self.outs

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        rc = cvlc_read_status(self.plan_ws, stream)
        return rc if rc != CVLC_OK else cvlc_read_status(self.enc_ws, stream)

    def read_plan(self, i: int) -> CvlcPlan:
        return read_plan(self.plans[i * PLAN_BYTES:(i + 1) * PLAN_BYTES])


class Aggregator:
    """Owns the pointer tables and workspace of cvlc_decode_aggregate for up to n_max clients."""

    def __init__(self, n_max: int, d: int, device: torch.device):
        self.n_max, self.d, self.device = n_max, d, device
        self.ptrs = torch.zeros(n_max, dtype=torch.int64, device=device)
        self.sizes = torch.zeros(n_max, dtype=torch.int64, device=device)
        self.weights = torch.zeros(n_max, dtype=torch.float32, device=device)
        self.ws = alloc_bytes(cvlc_decode_workspace_bytes(n_max), device)
        self._keep: List[torch.Tensor] = []

    def set_clients(self, streams: Sequence[torch.Tensor], weights: torch.Tensor) -> int:
        n = len(streams)
        assert n <= self.n_max
        self._keep = list(streams)
        self.ptrs[:n] = torch.tensor([s.data_ptr() for s in streams], dtype=torch.int64)
        self.sizes[:n] = torch.tensor([s.numel() for s in streams], dtype=torch.int64)
        self.weights[:n] = weights.to(self.device, dtype=torch.float32)
        return n

    def run(self, n: int, out: torch.Tensor, *, weight_total: float = 0.0, accumulate: bool = False,
            stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        cvlc_decode_aggregate(self.ptrs, self.sizes, self.weights, n, weight_total, self.d, out, accumulate,
                              self.ws, stream)
        return out

    def apply(self, n: int, model: torch.Tensor, aggregate: torch.Tensor, *, weight_total: float = 0.0,
              stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        cvlc_decode_apply(self.ptrs, self.sizes, self.weights, n, weight_total, self.d, model, aggregate, self.ws, stream)
        return model

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        return cvlc_read_status(self.ws, stream)
