"""ctypes access to the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

from .build import build as _build

ORC_OK = 0
ORC_ERR_INVALID_ARG = 1
ORC_ERR_BUDGET_TOO_SMALL = 2
ORC_ERR_BUDGET_TOO_LARGE = 3
ORC_ERR_PACKET_TOO_SMALL = 4
ORC_ERR_NONFINITE_INPUT = 5
ORC_ERR_OUTPUT_TOO_SMALL = 7
ORC_ERR_BAD_STREAM = 8
ORC_ERR_SCALE_TOO_SMALL = 12

HIST_BINS = 4096
MAX_Y = 32


class OrcParams(C.Structure):
    _fields_ = [
        ("d", C.c_uint64), ("budget_bits", C.c_uint64),
        ("packet_bits", C.c_uint32), ("header_bits", C.c_uint32),
        ("quantizer", C.c_uint32), ("max_code_bits", C.c_uint32),
        ("scale_B", C.c_double), ("seed", C.c_uint64),
        ("client_id", C.c_uint32), ("round", C.c_uint32),
    ]


class OrcPlan(C.Structure):
    _fields_ = [
        ("s", C.c_uint32), ("R", C.c_uint32), ("y_min", C.c_uint32), ("n_lengths", C.c_uint32),
        ("k", C.c_uint64),
        ("alpha", C.c_double), ("alpha_q", C.c_double), ("beta", C.c_double),
        ("gamma", C.c_double), ("B_next", C.c_double),
        ("n_y", C.c_uint32 * (MAX_Y + 1)), ("cap", C.c_uint32 * (MAX_Y + 1)),
        ("n_evals", C.c_uint64),
    ]


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"oracle {where} failed with status {code}")
        self.code = code


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        f64, u32, u64 = C.c_double, C.c_uint32, C.c_uint64
        P = C.POINTER
        L.cvlc_log2_oracle.restype = f64
        L.cvlc_log2_oracle.argtypes = [f64]
        L.cvlc_exp2_oracle.restype = f64
        L.cvlc_exp2_oracle.argtypes = [f64]
        L.cvlc_powr_oracle.restype = f64
        L.cvlc_powr_oracle.argtypes = [f64, f64]
        L.cvlc_philox4x32_10_oracle.restype = None
        L.cvlc_philox4x32_10_oracle.argtypes = [P(u32), P(u32), P(u32)]
        L.cvlc_philox_coord_oracle.restype = u32
        L.cvlc_philox_coord_oracle.argtypes = [u64, u32, u32, u64]
        L.cvlc_histogram_oracle.restype = C.c_int
        L.cvlc_histogram_oracle.argtypes = [C.c_void_p, u64, C.c_void_p]
        L.cvlc_alpha_fit_oracle.restype = None
        L.cvlc_alpha_fit_oracle.argtypes = [C.c_void_p, u64, P(f64), P(f64)]
        L.cvlc_derive_oracle.restype = C.c_int
        L.cvlc_derive_oracle.argtypes = [P(OrcParams), P(u32), P(u32), P(u32)]
        L.cvlc_default_scale_oracle.restype = f64
        L.cvlc_default_scale_oracle.argtypes = [P(OrcParams)]
        L.cvlc_stream_bytes_oracle.restype = C.c_size_t
        L.cvlc_stream_bytes_oracle.argtypes = [P(OrcParams)]
        L.cvlc_coeff_g_oracle.restype = f64
        L.cvlc_coeff_g_oracle.argtypes = [P(OrcParams), u32]
        L.cvlc_quant_error_Q_oracle.restype = f64
        L.cvlc_quant_error_Q_oracle.argtypes = [P(OrcParams), u32]
        L.cvlc_objective_oracle.restype = f64
        L.cvlc_objective_oracle.argtypes = [P(OrcParams), f64, P(u32)]
        L.cvlc_candidates_oracle.restype = C.c_int
        L.cvlc_candidates_oracle.argtypes = [P(OrcParams), P(u32)]
        L.cvlc_plan_from_alpha_oracle.restype = C.c_int
        L.cvlc_plan_from_alpha_oracle.argtypes = [P(OrcParams), f64, P(OrcPlan)]
        L.cvlc_plan_oracle.restype = C.c_int
        L.cvlc_plan_oracle.argtypes = [C.c_void_p, P(OrcParams), P(OrcPlan)]
        L.cvlc_plan_from_histogram_oracle.restype = C.c_int
        L.cvlc_plan_from_histogram_oracle.argtypes = [C.c_void_p, P(OrcParams), P(OrcPlan)]
        L.cvlc_decode_apply_oracle.restype = C.c_int
        L.cvlc_decode_apply_oracle.argtypes = [P(C.c_void_p), P(u64), C.c_void_p, u32, f64, u64, C.c_void_p]
        L.cvlc_plan_literal_oracle.restype = C.c_int
        L.cvlc_plan_literal_oracle.argtypes = [P(OrcParams), f64, u32, u32, C.c_void_p, C.c_void_p, C.c_void_p,
                                               P(u64), P(f64), C.c_void_p]
        L.cvlc_ec_accumulate_oracle.restype = None
        L.cvlc_ec_accumulate_oracle.argtypes = [C.c_void_p, C.c_void_p, u64]
        L.cvlc_ec_residual_oracle.restype = C.c_int
        L.cvlc_ec_residual_oracle.argtypes = [C.c_void_p, C.c_void_p, u64, u64, C.c_void_p]
        L.cvlc_unframed_header_bytes_oracle.restype = C.c_size_t
        L.cvlc_unframed_header_bytes_oracle.argtypes = [u32]
        L.cvlc_unframed_capacity_oracle.restype = C.c_size_t
        L.cvlc_unframed_capacity_oracle.argtypes = [P(OrcParams)]
        L.cvlc_encode_unframed_oracle.restype = C.c_int
        L.cvlc_encode_unframed_oracle.argtypes = [C.c_void_p, P(OrcParams), P(OrcPlan), C.c_void_p, C.c_size_t, P(C.c_size_t)]
        L.cvlc_decode_aggregate_unframed_oracle.restype = C.c_int
        L.cvlc_decode_aggregate_unframed_oracle.argtypes = [P(C.c_void_p), P(u64), C.c_void_p, u32, f64, u64, C.c_void_p, C.c_int]
        L.cvlc_plan_fixed_oracle.restype = C.c_int
        L.cvlc_plan_fixed_oracle.argtypes = [P(OrcParams), u32, P(OrcPlan)]
        L.cvlc_rank_oracle.restype = C.c_int
        L.cvlc_rank_oracle.argtypes = [C.c_void_p, u64, u64, C.c_void_p]
        L.cvlc_pq_quantize_oracle.restype = u32
        L.cvlc_pq_quantize_oracle.argtypes = [C.c_float, C.c_float, C.c_float, u32, u32]
        L.cvlc_pq_dequantize_oracle.restype = C.c_float
        L.cvlc_pq_dequantize_oracle.argtypes = [u32, C.c_float, C.c_float, u32]
        L.cvlc_qsgd_norm_oracle.restype = C.c_float
        L.cvlc_qsgd_norm_oracle.argtypes = [C.POINTER(C.c_float), u32]
        L.cvlc_qsgd_quantize_oracle.restype = u32
        L.cvlc_qsgd_quantize_oracle.argtypes = [C.c_float, C.c_float, u32, u32]
        L.cvlc_qsgd_dequantize_oracle.restype = C.c_float
        L.cvlc_qsgd_dequantize_oracle.argtypes = [u32, C.c_float, u32]
        L.cvlc_encode_oracle.restype = C.c_int
        L.cvlc_encode_oracle.argtypes = [C.c_void_p, P(OrcParams), P(OrcPlan), C.c_void_p, C.c_size_t,
                                         C.c_void_p]
        L.cvlc_decode_aggregate_oracle.restype = C.c_int
        L.cvlc_decode_aggregate_oracle.argtypes = [P(C.c_void_p), P(u64), C.c_void_p, u32, f64, u64,
                                                   C.c_void_p, C.c_int]
        _lib = L
    return _lib


def make_params(d: int, budget_bits: int, *, packet_bits: int = 12000, header_bits: int = 80,
                quantizer: int = 0, max_code_bits: int = 32, scale_B: Optional[float] = None,
                seed: int = 0, client_id: int = 0, round: int = 0) -> OrcParams:
    p = OrcParams(d, budget_bits, packet_bits, header_bits, quantizer, max_code_bits, 1.0, seed,
                  client_id, round)
    p.scale_B = default_scale(p) if scale_B is None else float(scale_B)
    return p


def default_scale(p: OrcParams) -> float:
    return lib().cvlc_default_scale_oracle(C.byref(p))


def stream_bytes(p: OrcParams) -> int:
    return int(lib().cvlc_stream_bytes_oracle(C.byref(p)))


def log2(v: float) -> float:
    return lib().cvlc_log2_oracle(v)


def exp2(v: float) -> float:
    return lib().cvlc_exp2_oracle(v)


def powr(a: float, beta: float) -> float:
    return lib().cvlc_powr_oracle(a, beta)


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().cvlc_philox4x32_10_oracle(c, k, o)
    return tuple(int(v) for v in o)


def philox_coord(seed: int, client_id: int, round: int, coord: int) -> int:
    return int(lib().cvlc_philox_coord_oracle(seed, client_id, round, coord))


def _f32(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return x


def histogram(x: np.ndarray) -> Tuple[int, np.ndarray]:
    x = _f32(x)
    h = np.zeros(HIST_BINS, dtype=np.uint64)
    rc = lib().cvlc_histogram_oracle(x.ctypes.data, x.size, h.ctypes.data)
    return rc, h


def alpha_fit(h: np.ndarray, d: int) -> Tuple[float, float]:
    h = np.ascontiguousarray(h, dtype=np.uint64)
    a, aq = C.c_double(), C.c_double()
    lib().cvlc_alpha_fit_oracle(h.ctypes.data, d, C.byref(a), C.byref(aq))
    return a.value, aq.value


def derive(p: OrcParams) -> Tuple[int, int, int, List[int]]:
    s, R = C.c_uint32(), C.c_uint32()
    cap = (C.c_uint32 * (MAX_Y + 1))()
    rc = lib().cvlc_derive_oracle(C.byref(p), C.byref(s), C.byref(R), cap)
    return rc, s.value, R.value, [int(c) for c in cap]


def coeff_g(p: OrcParams, y: int) -> float:
    return lib().cvlc_coeff_g_oracle(C.byref(p), y)


def quant_error_Q(p: OrcParams, y: int) -> float:
    return lib().cvlc_quant_error_Q_oracle(C.byref(p), y)


def candidates(p: OrcParams) -> List[int]:
    Y = (C.c_uint32 * (MAX_Y + 1))()
    n = lib().cvlc_candidates_oracle(C.byref(p), Y)
    return [int(Y[i]) for i in range(n)]


def objective(p: OrcParams, beta: float, n_y: Sequence[int]) -> float:
    n = (C.c_uint32 * (MAX_Y + 1))(*[int(v) for v in n_y])
    return lib().cvlc_objective_oracle(C.byref(p), beta, n)


def plan_from_alpha(p: OrcParams, alpha_q: float) -> OrcPlan:
    plan = OrcPlan()
    rc = lib().cvlc_plan_from_alpha_oracle(C.byref(p), alpha_q, C.byref(plan))
    if rc != ORC_OK:
        raise OracleError(rc, "plan_from_alpha")
    return plan


def plan_from_histogram(h: np.ndarray, p: OrcParams) -> OrcPlan:
    h = np.ascontiguousarray(h, dtype=np.uint64)
    assert h.size == HIST_BINS
    pl = OrcPlan()
    rc = lib().cvlc_plan_from_histogram_oracle(h.ctypes.data, C.byref(p), C.byref(pl))
    if rc != ORC_OK:
        raise OracleError(rc, "plan_from_histogram")
    return pl


def plan(x: np.ndarray, p: OrcParams) -> OrcPlan:
    x = _f32(x)
    assert x.size == p.d
    pl = OrcPlan()
    rc = lib().cvlc_plan_oracle(x.ctypes.data, C.byref(p), C.byref(pl))
    if rc != ORC_OK:
        raise OracleError(rc, "plan")
    return pl


def plan_fixed(p: OrcParams, y: int) -> OrcPlan:
    pl = OrcPlan()
    rc = lib().cvlc_plan_fixed_oracle(C.byref(p), y, C.byref(pl))
    if rc != ORC_OK:
        raise OracleError(rc, "plan_fixed")
    return pl


@dataclass
class LiteralPlan:
    k_star: int
    gamma_star: float
    P_star: np.ndarray        # R real-valued packet sizes at k_star
    k_grid: np.ndarray        # the values of k that were tried
    gamma_of_k: np.ndarray    # Eq. (5) after tuning, per value of k
    sweeps_of_k: np.ndarray


def plan_literal(p: OrcParams, alpha_q: float, n_k: int, max_sweeps: int = 1 << 20) -> LiteralPlan:
    """problem P2 with real-valued packet sizes: k on an equidistant grid, pairwise tuning of consecutive packets"""
    rc0, s, R, cap = derive(p)
    if rc0 != ORC_OK:
        raise OracleError(rc0, "plan_literal")
    k_grid = np.zeros(n_k, dtype=np.uint64)
    gam = np.zeros(n_k, dtype=np.float64)
    sw = np.zeros(n_k, dtype=np.uint32)
    P_star = np.zeros(R, dtype=np.float64)
    k_star, g_star = C.c_uint64(), C.c_double()
    rc = lib().cvlc_plan_literal_oracle(C.byref(p), float(alpha_q), int(n_k), int(max_sweeps), k_grid.ctypes.data,
                                        gam.ctypes.data, sw.ctypes.data, C.byref(k_star), C.byref(g_star),
                                        P_star.ctypes.data)
    if rc != ORC_OK:
        raise OracleError(rc, "plan_literal")
    return LiteralPlan(int(k_star.value), float(g_star.value), P_star, k_grid, gam, sw)


def rank(x: np.ndarray, k: int) -> np.ndarray:
    x = _f32(x)
    idx = np.empty(max(k, 1), dtype=np.uint32)
    rc = lib().cvlc_rank_oracle(x.ctypes.data, x.size, k, idx.ctypes.data)
    if rc != ORC_OK:
        raise OracleError(rc, "rank")
    return idx[:k]


def pq_quantize(x: float, lo: float, hi: float, y: int, rnd: int) -> int:
    return int(lib().cvlc_pq_quantize_oracle(x, lo, hi, y, rnd))


def pq_dequantize(code: int, lo: float, hi: float, y: int) -> float:
    return float(lib().cvlc_pq_dequantize_oracle(code, lo, hi, y))


def qsgd_norm(v: np.ndarray) -> float:
    v = _f32(v)
    return float(lib().cvlc_qsgd_norm_oracle(v.ctypes.data_as(C.POINTER(C.c_float)), v.size))


def qsgd_quantize(x: float, norm: float, y: int, rnd: int) -> int:
    return int(lib().cvlc_qsgd_quantize_oracle(x, norm, y, rnd))


def qsgd_dequantize(code: int, norm: float, y: int) -> float:
    return float(lib().cvlc_qsgd_dequantize_oracle(code, norm, y))


def encode(x: np.ndarray, p: OrcParams, pl: OrcPlan, want_rank: bool = False):
    x = _f32(x)
    assert x.size == p.d
    nbytes = stream_bytes(p)
    st = np.zeros(nbytes, dtype=np.uint8)
    ranked = np.empty(max(int(pl.k), 1), dtype=np.uint32) if want_rank else None
    rc = lib().cvlc_encode_oracle(x.ctypes.data, C.byref(p), C.byref(pl), st.ctypes.data, nbytes,
                                  ranked.ctypes.data if want_rank else None)
    if rc != ORC_OK:
        raise OracleError(rc, "encode")
    if want_rank:
        return st, ranked[: int(pl.k)]
    return st


def decode_aggregate(streams: Sequence[np.ndarray], weights: np.ndarray, d: int, *,
                     weight_total: float = 0.0, out: Optional[np.ndarray] = None,
                     accumulate: bool = False) -> np.ndarray:
    n = len(streams)
    streams = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    ptrs = (C.c_void_p * n)(*[s.ctypes.data for s in streams])
    sizes = (C.c_uint64 * n)(*[s.size for s in streams])
    w = np.ascontiguousarray(weights, dtype=np.float32)
    assert w.size == n
    if out is None:
        out = np.zeros(d, dtype=np.float32)
    assert out.dtype == np.float32 and out.size == d
    rc = lib().cvlc_decode_aggregate_oracle(ptrs, sizes, w.ctypes.data, n, float(weight_total), d,
                                            out.ctypes.data, 1 if accumulate else 0)
    if rc != ORC_OK:
        raise OracleError(rc, "decode_aggregate")
    return out


def encode_unframed(x: np.ndarray, p: OrcParams, plan: OrcPlan) -> np.ndarray:
    """the unframed (version 2) stream of the same records: returns its bytes"""
    x = _f32(x)
    capacity = int(lib().cvlc_unframed_capacity_oracle(C.byref(p)))
    buf = np.zeros(capacity, dtype=np.uint8)
    n = C.c_size_t()
    rc = lib().cvlc_encode_unframed_oracle(x.ctypes.data, C.byref(p), C.byref(plan), buf.ctypes.data, capacity, C.byref(n))
    if rc != ORC_OK:
        raise OracleError(rc, "encode_unframed")
    return buf[:n.value].copy()


def unframed_capacity(p: OrcParams) -> int:
    return int(lib().cvlc_unframed_capacity_oracle(C.byref(p)))


def decode_aggregate_unframed(streams: Sequence[np.ndarray], weights: np.ndarray, d: int, *, weight_total: float = 0.0,
                              out: Optional[np.ndarray] = None, accumulate: bool = False) -> np.ndarray:
    n = len(streams)
    streams = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    ptrs = (C.c_void_p * n)(*[s.ctypes.data for s in streams])
    sizes = (C.c_uint64 * n)(*[s.size for s in streams])
    w = np.ascontiguousarray(weights, dtype=np.float32)
    if out is None:
        out = np.zeros(d, dtype=np.float32)
    rc = lib().cvlc_decode_aggregate_unframed_oracle(ptrs, sizes, w.ctypes.data, n, float(weight_total), d,
                                                     out.ctypes.data, 1 if accumulate else 0)
    if rc != ORC_OK:
        raise OracleError(rc, "decode_aggregate_unframed")
    return out


def ec_accumulate(memory: np.ndarray, update: np.ndarray) -> np.ndarray:
    """memory <- memory + update in fp32, in place; returns memory (the compensated update to compress)"""
    assert memory.dtype == np.float32 and memory.flags.c_contiguous
    u = _f32(update)
    assert u.size == memory.size
    lib().cvlc_ec_accumulate_oracle(memory.ctypes.data, u.ctypes.data, memory.size)
    return memory


def ec_residual(compensated: np.ndarray, stream: np.ndarray) -> np.ndarray:
    """the new memory: compensated minus what the parameter server rebuilds from the stream"""
    a = _f32(compensated)
    st = np.ascontiguousarray(stream, dtype=np.uint8)
    out = np.empty_like(a)
    rc = lib().cvlc_ec_residual_oracle(a.ctypes.data, st.ctypes.data, st.size, a.size, out.ctypes.data)
    if rc != ORC_OK:
        raise OracleError(rc, "ec_residual")
    return out


def decode_apply(streams: Sequence[np.ndarray], weights: np.ndarray, model: np.ndarray, *,
                 weight_total: float = 0.0) -> np.ndarray:
    """model <- model - aggregate, in place; returns model"""
    n = len(streams)
    streams = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    ptrs = (C.c_void_p * n)(*[s.ctypes.data for s in streams])
    sizes = (C.c_uint64 * n)(*[s.size for s in streams])
    w = np.ascontiguousarray(weights, dtype=np.float32)
    assert w.size == n and model.dtype == np.float32 and model.flags.c_contiguous
    rc = lib().cvlc_decode_apply_oracle(ptrs, sizes, w.ctypes.data, n, float(weight_total), model.size,
                                        model.ctypes.data)
    if rc != ORC_OK:
        raise OracleError(rc, "decode_apply")
    return model
