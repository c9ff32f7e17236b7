"""CPU oracle for the ZGR step: ctypes front end of ``zgr_oracle.cpp``.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; it exists so that the
tests, the smoke check and the benchmark's CPU-baseline leg have an independent, slow,
double-precision statement of Eq. (ZOO), Eq. (perturbation), Eq. (grad), Algorithm 1 and the DTC
dequantisation to compare the CUDA library against.

All of the arithmetic lives in the C++ file; this module only builds it (g++, OpenMP), marshals numpy
arrays, and keeps the per-seed bookkeeping of the call sequence
``perturb(+eps) -> perturb(-2 eps) -> restore_update`` (class :class:`OracleZGR`).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zgr_oracle.cpp")
_LIB = os.path.join(_HERE, "libzgr_oracle.so")

F32, F16, BF16, F64 = 0, 1, 2, 3
SCALE_PAPER, SCALE_UNIT = 0, 1
_NP_STORAGE = {F32: np.float32, F16: np.uint16, BF16: np.uint16, F64: np.float64}


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source (idempotent)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-o", tmp, _SRC]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.zgro_projected_grad.restype = ctypes.c_double
        _lib.zgro_projected_grad.argtypes = [ctypes.c_double] * 3
        _lib.zgro_num_threads.restype = ctypes.c_int
        _lib.zgro_update_coefficient.restype = ctypes.c_double
        _lib.zgro_adapt_alpha.restype = ctypes.c_double
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u64(x):
    return ctypes.c_uint64(int(x) & 0xFFFFFFFFFFFFFFFF)


def _i64(x):
    return ctypes.c_int64(int(x))


def num_threads() -> int:
    return int(lib().zgro_num_threads())


# ----------------------------------------------------------------------------- generator
def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().zgro_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def blocks(seed: int, tensor: int, tag: int, first_block: int, n_blocks: int) -> np.ndarray:
    out = np.zeros((n_blocks, 4), dtype=np.uint32)
    lib().zgro_blocks(_u64(seed), ctypes.c_uint32(tensor), ctypes.c_uint32(tag), _u64(first_block), _i64(n_blocks), _p(out))
    return out


def normals(seed: int, tensor: int, tag: int, bits: int, e0: int, count: int) -> np.ndarray:
    out = np.zeros(count, dtype=np.float64)
    lib().zgro_normals(_u64(seed), ctypes.c_uint32(tensor), ctypes.c_uint32(tag), ctypes.c_int(bits), _u64(e0), _i64(count), _p(out))
    return out


# ----------------------------------------------------------------------------- scalars
def mix_scalars(alpha: float, d: int, K: int, scale_mode: int):
    a, b = ctypes.c_double(), ctypes.c_double()
    lib().zgro_mix_scalars(ctypes.c_double(alpha), _i64(d), _i64(K), ctypes.c_int(scale_mode), ctypes.byref(a), ctypes.byref(b))
    return a.value, b.value


def projected_grad(loss_plus: float, loss_minus: float, eps: float) -> float:
    return float(lib().zgro_projected_grad(loss_plus, loss_minus, eps))


# ----------------------------------------------------------------------------- rounding / storage
def round_to(x: np.ndarray, dtype: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty_like(x)
    lib().zgro_round(_p(x), _i64(x.size), ctypes.c_int(dtype), _p(out))
    return out


def decode(storage: np.ndarray, dtype: int) -> np.ndarray:
    """Storage array (float32 / uint16 bit patterns / float64) -> exact doubles."""
    s = np.ascontiguousarray(storage, dtype=_NP_STORAGE[dtype])
    out = np.empty(s.shape, dtype=np.float64)
    lib().zgro_decode(_p(s), ctypes.c_int(dtype), _i64(s.size), _p(out))
    return out


def encode(values: np.ndarray, dtype: int) -> np.ndarray:
    """Doubles -> storage array, rounding to nearest even."""
    v = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty(v.shape, dtype=_NP_STORAGE[dtype])
    lib().zgro_encode(_p(v), ctypes.c_int(dtype), _i64(v.size), _p(out))
    return out


# ----------------------------------------------------------------------------- tensors
@dataclass
class OracleTensor:
    """One model tensor as the oracle sees it: storage array plus its subspace and coefficient source."""

    theta: np.ndarray                 # storage: float32, uint16 (f16/bf16 bit patterns) or float64; rows*cols
    rows: int
    cols: int
    dtype: int
    U: Optional[np.ndarray] = None    # rows x rank float32, orthonormal columns
    q: Optional[np.ndarray] = None    # qrows x cols int8  (DTC codes) or None -> coefficients from the seed
    scale: Optional[np.ndarray] = None
    zero: Optional[np.ndarray] = None
    # (Sec. 3.4, proportion omega: the codes may cover only the first q.shape[0] rows of G_l; the other rows
    #  are drawn from the seed)

    @property
    def rank(self) -> int:
        return 0 if self.U is None else int(self.U.shape[1])

    def _args(self):
        U = None if self.U is None else np.ascontiguousarray(self.U, dtype=np.float32)
        q = None if self.q is None else np.ascontiguousarray(self.q, dtype=np.int8)
        sc = None if self.scale is None else np.ascontiguousarray(self.scale, dtype=np.float32)
        ze = None if self.zero is None else np.ascontiguousarray(self.zero, dtype=np.float32)
        return U, q, sc, ze

    @property
    def qrows(self) -> int:
        """Rows of G_l taken from the codes."""
        return 0 if self.q is None else int(np.asarray(self.q).shape[0])


def coeffs(seed, tensor_id, bits, rank, cols, q=None, scale=None, zero=None) -> np.ndarray:
    out = np.zeros((rank, cols), dtype=np.float64)
    qrows = 0 if q is None else int(np.asarray(q).shape[0])
    lib().zgro_coeffs(_u64(seed), ctypes.c_uint32(tensor_id), ctypes.c_int(bits), _i64(rank), _i64(cols), _p(q), _p(scale), _p(zero), _i64(qrows), _p(out))
    return out


def z_tensor(t: OracleTensor, seed: int, tensor_id: int, bits: int, a: float, b: float, parts: bool = False):
    U, q, sc, ze = t._args()
    n = t.rows * t.cols
    z = np.zeros(n, dtype=np.float64)
    iso = np.zeros(n, dtype=np.float64) if parts else None
    gd = np.zeros(n, dtype=np.float64) if parts else None
    lib().zgro_z_tensor(_u64(seed), ctypes.c_uint32(tensor_id), ctypes.c_int(bits), _i64(t.rows), _i64(t.cols), _p(U), _i64(t.rank),
                        _p(q), _p(sc), _p(ze), _i64(t.qrows), ctypes.c_double(a), ctypes.c_double(b), _p(z), _p(iso), _p(gd))
    z = z.reshape(t.rows, t.cols)
    if parts:
        return z, iso.reshape(t.rows, t.cols), gd.reshape(t.rows, t.cols)
    return z


def z_elements(t: OracleTensor, seed: int, tensor_id: int, bits: int, a: float, b: float, idx: np.ndarray) -> np.ndarray:
    U, q, sc, ze = t._args()
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    out = np.zeros(idx.size, dtype=np.float64)
    lib().zgro_z_elements(_u64(seed), ctypes.c_uint32(tensor_id), ctypes.c_int(bits), _i64(t.rows), _i64(t.cols), _p(U), _i64(t.rank),
                          _p(q), _p(sc), _p(ze), _i64(t.qrows), ctypes.c_double(a), ctypes.c_double(b), _i64(idx.size), _p(idx), _p(out))
    return out


def sweep_tensor(t: OracleTensor, seed: int, tensor_id: int, bits: int, a: float, b: float, c: float) -> None:
    """theta <- rnd(theta + c z), in place on ``t.theta``."""
    U, q, sc, ze = t._args()
    assert t.theta.flags["C_CONTIGUOUS"] and t.theta.dtype == _NP_STORAGE[t.dtype] and t.theta.size == t.rows * t.cols
    lib().zgro_sweep_tensor(_p(t.theta), ctypes.c_int(t.dtype), _u64(seed), ctypes.c_uint32(tensor_id), ctypes.c_int(bits),
                            _i64(t.rows), _i64(t.cols), _p(U), _i64(t.rank), _p(q), _p(sc), _p(ze), _i64(t.qrows),
                            ctypes.c_double(a), ctypes.c_double(b), ctypes.c_double(c))


def sweep_elements(t: OracleTensor, theta_in: np.ndarray, seed: int, tensor_id: int, bits: int, a: float, b: float, c: float,
                   idx: np.ndarray) -> np.ndarray:
    """Sweep result at selected elements; ``theta_in`` holds their current stored values as doubles."""
    U, q, sc, ze = t._args()
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    th = np.ascontiguousarray(theta_in, dtype=np.float64)
    out = np.zeros(idx.size, dtype=np.float64)
    lib().zgro_sweep_elements(_p(th), ctypes.c_int(t.dtype), _u64(seed), ctypes.c_uint32(tensor_id), ctypes.c_int(bits), _i64(t.rows),
                              _i64(t.cols), _p(U), _i64(t.rank), _p(q), _p(sc), _p(ze), _i64(t.qrows), ctypes.c_double(a), ctypes.c_double(b),
                              ctypes.c_double(c), _i64(idx.size), _p(idx), _p(out))
    return out


def _terms(seeds, coeffs):
    n = len(seeds)
    assert n == len(coeffs) and n >= 1
    return n, np.asarray([int(x) & 0xFFFFFFFFFFFFFFFF for x in seeds], dtype=np.uint64), np.asarray(coeffs, dtype=np.float64)


def sweep_multi_tensor(t: OracleTensor, seeds: Sequence[int], coeffs: Sequence[float], tensor_id: int, bits: int, a: float, b: float) -> None:
    """theta <- rnd(theta + sum_q c_q z(seed_q)), in place: the sum over seeds of Algorithm 1
    ("Recover gradient": sum_t g_t z_t; "Update") applied with a single rounding to the storage type."""
    U, q, sc, ze = t._args()
    n, sd, cf = _terms(seeds, coeffs)
    assert t.theta.flags["C_CONTIGUOUS"] and t.theta.dtype == _NP_STORAGE[t.dtype] and t.theta.size == t.rows * t.cols
    lib().zgro_sweep_multi_tensor(_p(t.theta), ctypes.c_int(t.dtype), ctypes.c_int(n), _p(sd), _p(cf), ctypes.c_uint32(tensor_id),
                                  ctypes.c_int(bits), _i64(t.rows), _i64(t.cols), _p(U), _i64(t.rank), _p(q), _p(sc), _p(ze), _i64(t.qrows),
                                  ctypes.c_double(a), ctypes.c_double(b))


def sweep_multi_elements(t: OracleTensor, theta_in: np.ndarray, seeds: Sequence[int], coeffs: Sequence[float], tensor_id: int, bits: int,
                         a: float, b: float, idx: np.ndarray) -> np.ndarray:
    """The same at selected elements; ``theta_in`` holds their current stored values as doubles."""
    U, q, sc, ze = t._args()
    n, sd, cf = _terms(seeds, coeffs)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    th = np.ascontiguousarray(theta_in, dtype=np.float64)
    out = np.zeros(idx.size, dtype=np.float64)
    lib().zgro_sweep_multi_elements(_p(th), ctypes.c_int(t.dtype), ctypes.c_int(n), _p(sd), _p(cf), ctypes.c_uint32(tensor_id), ctypes.c_int(bits),
                                    _i64(t.rows), _i64(t.cols), _p(U), _i64(t.rank), _p(q), _p(sc), _p(ze), _i64(t.qrows), ctypes.c_double(a), ctypes.c_double(b),
                                    _i64(idx.size), _p(idx), _p(out))
    return out


def update_coefficient(net: float, loss_plus: float, loss_minus: float, eps: float, lr: float) -> float:
    """Coefficient of the fused restore + update sweep: -net - lr (L+ - L-)/(2 eps)  (Eq. (grad), Algorithm 1 "Update")."""
    return float(lib().zgro_update_coefficient(ctypes.c_double(net), ctypes.c_double(loss_plus), ctypes.c_double(loss_minus),
                                               ctypes.c_double(eps), ctypes.c_double(lr)))


def adapt_alpha(stats: np.ndarray, a0: float, b0: float, d: int, K: int, alpha_old: float, alpha_min: float = 0.05, alpha_max: float = 0.95,
                eta: float = 1.0) -> float:
    """The energy-balancing candidate for the adaptive mixing ratio announced in Sec. 1 (see zgro_adapt_alpha)."""
    st = np.ascontiguousarray(stats, dtype=np.float64).reshape(-1, 3)
    return float(lib().zgro_adapt_alpha(_p(st), _i64(st.shape[0]), ctypes.c_double(a0), ctypes.c_double(b0), _i64(d), _i64(K),
                                        ctypes.c_double(alpha_old), ctypes.c_double(alpha_min), ctypes.c_double(alpha_max), ctypes.c_double(eta)))


def householder_qr(A: np.ndarray, with_r: bool = False):
    """Orthonormal basis of the span of the columns of A (rows x r; Algorithm 1 "build basis V_r"): thin Q of a
    Householder QR in double with R_kk > 0."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    rows, r = A.shape
    Q = np.zeros((rows, r), dtype=np.float64)
    R = np.zeros((r, r), dtype=np.float64) if with_r else None
    lib().zgro_householder_qr(_p(A), _i64(rows), _i64(r), _p(Q), _p(R))
    return (Q, R) if with_r else Q


def stats_tensor(t: OracleTensor, seed: int, tensor_id: int, bits: int, a: float, b: float) -> np.ndarray:
    U, q, sc, ze = t._args()
    out = np.zeros(3, dtype=np.float64)
    lib().zgro_stats_tensor(_u64(seed), ctypes.c_uint32(tensor_id), ctypes.c_int(bits), _i64(t.rows), _i64(t.cols), _p(U), _i64(t.rank),
                            _p(q), _p(sc), _p(ze), _i64(t.qrows), ctypes.c_double(a), ctypes.c_double(b), _p(out))
    return out


# ----------------------------------------------------------------------------- DTC
def dtc_quantise(G: np.ndarray, bits: int = 8, symmetric: bool = True):
    """Row-wise quantiser of Sec. 3.4: returns (codes int8, scale float32, zero float32)."""
    G = np.ascontiguousarray(G, dtype=np.float64)
    r, n = G.shape
    q = np.zeros((r, n), dtype=np.int8)
    sc = np.zeros(r, dtype=np.float32)
    ze = np.zeros(r, dtype=np.float32)
    for k in range(r):
        lib().zgro_dtc_quantise_row(_p(G[k]), _i64(n), ctypes.c_int(bits), ctypes.c_int(1 if symmetric else 0),
                                    ctypes.c_void_p(q[k].ctypes.data), ctypes.c_void_p(sc[k:].ctypes.data), ctypes.c_void_p(ze[k:].ctypes.data))
    return q, sc, ze


def dtc_dequantise(q: np.ndarray, scale: np.ndarray, zero: Optional[np.ndarray] = None) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    r, n = q.shape
    out = np.zeros((r, n), dtype=np.float64)
    for k in range(r):
        z = 0.0 if zero is None else float(zero[k])
        lib().zgro_dtc_dequantise_row(ctypes.c_void_p(q[k].ctypes.data), _i64(n), ctypes.c_float(float(scale[k])), ctypes.c_float(z),
                                      ctypes.c_void_p(out[k].ctypes.data))
    return out


def dtc_quantise_int4(G: np.ndarray):
    """The paper's INT4 form of Sec. 3.4: unsigned codes x_q in [0, 15], lambda = (max - min)/15 and a zero
    point delta per row, x = lambda (x_q - delta)  (zgro_dtc_quantise_row_int4)."""
    G = np.ascontiguousarray(G, dtype=np.float64)
    r, n = G.shape
    q = np.zeros((r, n), dtype=np.int8)
    sc = np.zeros(r, dtype=np.float32)
    ze = np.zeros(r, dtype=np.float32)
    for k in range(r):
        lib().zgro_dtc_quantise_row_int4(_p(G[k]), _i64(n), ctypes.c_void_p(q[k].ctypes.data), ctypes.c_void_p(sc[k:].ctypes.data),
                                         ctypes.c_void_p(ze[k:].ctypes.data))
    return q, sc, ze


def dtc_pack4(codes: np.ndarray) -> np.ndarray:
    """Transmission layout of 4-bit codes: each row becomes (cols + 1)//2 bytes, column 2j in the low nibble
    of byte j and column 2j + 1 in its high nibble (a missing last column is stored as 0)."""
    codes = np.asarray(codes)
    assert codes.ndim == 2 and codes.min() >= 0 and codes.max() <= 15
    c8 = np.ascontiguousarray(codes, dtype=np.int8)
    r, n = c8.shape
    out = np.zeros((r, (n + 1) // 2), dtype=np.uint8)
    lib().zgro_dtc_pack4(_p(c8), _i64(r), _i64(n), _p(out))
    return out


def dtc_unpack4(packed: np.ndarray, cols: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.zeros((packed.shape[0], cols), dtype=np.int8)
    lib().zgro_dtc_unpack4(_p(packed), _i64(packed.shape[0]), _i64(cols), _p(out))
    return out


# ----------------------------------------------------------------------------- the call sequence
class OracleZGR:
    """Mirror of the library's call sequence over a list of :class:`OracleTensor`.

    ``perturb(seed, c)`` applies ``theta <- rnd(theta + c z(seed))`` to every tensor and records the
    net coefficient applied under that seed; ``restore_update(seed, L+, L-, lr)`` applies
    ``c = -net - lr (L+ - L-)/(2 eps)`` (Eq. (grad) and the update line of Algorithm 1), which undoes
    the perturbation and takes the projected-gradient step in the same sweep.
    """

    def __init__(self, tensors: Sequence[OracleTensor], alpha: float, eps: float, scale_mode: int = SCALE_UNIT, bits: int = 32):
        self.tensors = list(tensors)
        self.alpha, self.eps, self.scale_mode, self.bits = float(alpha), float(eps), int(scale_mode), int(bits)
        self.d = sum(t.rows * t.cols for t in self.tensors)
        self.K = sum(t.rank * t.cols for t in self.tensors)
        self.a, self.b = mix_scalars(self.alpha, self.d, self.K, self.scale_mode)
        self.active_seed: Optional[int] = None
        self.net = 0.0
        self.nets = {}                # ledger of the multi-seed calls: seed -> net coefficient applied

    def perturb(self, seed: int, c: float) -> None:
        if self.active_seed is not None and self.active_seed != seed:
            raise RuntimeError("another seed is active")
        for l, t in enumerate(self.tensors):
            sweep_tensor(t, seed, l, self.bits, self.a, self.b, c)
        self.active_seed = seed
        self.net += c

    def update_coefficient(self, loss_plus: float, loss_minus: float, lr: float) -> float:
        return update_coefficient(self.net, loss_plus, loss_minus, self.eps, lr)

    def sweep_multi(self, seeds: Sequence[int], coeffs: Sequence[float]) -> None:
        """One pass applying several seeds; the ledger ``self.nets`` records what stays applied per seed."""
        for l, t in enumerate(self.tensors):
            sweep_multi_tensor(t, seeds, coeffs, l, self.bits, self.a, self.b)
        for seed, c in zip(seeds, coeffs):
            self.nets[seed] = self.nets.get(seed, 0.0) + float(c)
            if self.nets[seed] == 0.0:
                del self.nets[seed]

    def restore_update_multi(self, seeds: Sequence[int], loss_plus: Sequence[float], loss_minus: Sequence[float], lr: float):
        """Eq. (grad) per seed, then theta <- rnd(theta + sum_i (-net_i - lr g_i) z_i) in one pass."""
        coeffs = [update_coefficient(self.nets.get(s, 0.0), lp, lm, self.eps, lr) for s, lp, lm in zip(seeds, loss_plus, loss_minus)]
        for l, t in enumerate(self.tensors):
            sweep_multi_tensor(t, seeds, coeffs, l, self.bits, self.a, self.b)
        for s in seeds:
            self.nets.pop(s, None)
        return coeffs

    def restore_update(self, seed: int, loss_plus: float, loss_minus: float, lr: float) -> float:
        if self.active_seed != seed:
            raise RuntimeError("restore_update without a matching perturb")
        c = self.update_coefficient(loss_plus, loss_minus, lr)
        for l, t in enumerate(self.tensors):
            sweep_tensor(t, seed, l, self.bits, self.a, self.b, c)
        self.active_seed = None
        self.net = 0.0
        return c
