"""Python driver of the CPU oracle for ConEF (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It orchestrates the scalar C routines of ``conef_oracle.c`` in
the order of the paper's Algorithm 2 (lines 5-9), per worker and per tensor,
and keeps the per-worker compressed error state between steps.  It imports
nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conef_oracle.c")
_LIB = os.path.join(_HERE, "libconef_oracle.so")
CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", *CFLAGS, "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _declare(_lib)
    return _lib


_f32p = np.ctypeslib.ndpointer(dtype=np.float32, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(dtype=np.uint8, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(dtype=np.uint32, flags="C_CONTIGUOUS")
_i16p = np.ctypeslib.ndpointer(dtype=np.int16, flags="C_CONTIGUOUS")
_u16p = np.ctypeslib.ndpointer(dtype=np.uint16, flags="C_CONTIGUOUS")


def _declare(L: C.CDLL) -> None:
    i64, u64, f32, i32 = C.c_int64, C.c_uint64, C.c_float, C.c_int
    L.orc_mix64.restype = u64
    L.orc_mix64.argtypes = [u64]
    L.orc_stream.restype = u64
    L.orc_stream.argtypes = [u64, u64, u64]
    L.orc_h64.restype = u64
    L.orc_h64.argtypes = [u64, u64]
    L.orc_f32_to_f16.restype = C.c_uint16
    L.orc_f32_to_f16.argtypes = [f32]
    L.orc_f16_to_f32.restype = f32
    L.orc_f16_to_f32.argtypes = [C.c_uint16]
    L.orc_form_p.restype = None
    L.orc_form_p.argtypes = [f32, _f32p, _f32p, i64, _f32p]
    L.orc_passthrough.restype = None
    L.orc_passthrough.argtypes = [f32, _f32p, i64, _f32p]
    L.orc_randk_indices.restype = i32
    L.orc_randk_indices.argtypes = [u64, i64, i64, i64, i64, _u32p]
    L.orc_randk_apply.restype = None
    L.orc_randk_apply.argtypes = [_f32p, i64, _u32p, i64, _f32p, _f32p]
    L.orc_quant_encode.restype = None
    L.orc_quant_encode.argtypes = [_f32p, i64, i32, i32, i32, _u8p, _f32p, C.c_void_p]
    L.orc_quant_decode.restype = None
    L.orc_quant_decode.argtypes = [_u8p, _f32p, i64, i32, i32, _f32p]
    L.orc_sketch_bucket.restype = None
    L.orc_sketch_bucket.argtypes = [u64, i64, i32, i64, i64, C.POINTER(i64), C.POINTER(i32)]
    L.orc_sketch_encode.restype = i32
    L.orc_sketch_encode.argtypes = [_f32p, i64, i32, i64, u64, i64, _f32p]
    L.orc_sketch_decode.restype = None
    L.orc_sketch_decode.argtypes = [_f32p, i64, i32, i64, u64, i64, _f32p]
    L.orc_lowrank_project_rows.restype = None
    L.orc_lowrank_project_rows.argtypes = [_f32p, i64, i64, _f32p, i32, _f32p]
    L.orc_gram_schmidt.restype = None
    L.orc_gram_schmidt.argtypes = [_f32p, i64, i32]
    L.orc_lowrank_project_cols.restype = None
    L.orc_lowrank_project_cols.argtypes = [_f32p, i64, i64, _f32p, i32, _f32p]
    L.orc_lowrank_residual.restype = None
    L.orc_lowrank_residual.argtypes = [_f32p, i64, i64, _f32p, _f32p, i32, _f32p, C.c_void_p]
    L.orc_sum_workers.restype = None
    L.orc_sum_workers.argtypes = [C.POINTER(C.c_void_p), i32, i64, _f32p]
    L.orc_divide.restype = None
    L.orc_divide.argtypes = [_f32p, f32, i64, _f32p]
    L.orc_randblock_start.restype = i64
    L.orc_randblock_start.argtypes = [u64, i64, i64, i64, i64]
    L.orc_error_reset.restype = None
    L.orc_error_reset.argtypes = [C.POINTER(C.c_void_p), i32, i64]
    L.orc_apply_dense.restype = None
    L.orc_apply_dense.argtypes = [_f32p, _f32p, f32, i64]
    L.orc_apply_sparse.restype = None
    L.orc_apply_sparse.argtypes = [_f32p, _u32p, _f32p, f32, i64]
    L.orc_apply_lowrank.restype = None
    L.orc_apply_lowrank.argtypes = [_f32p, i64, i64, _f32p, _f32p, i32]
    L.orc_stochquant_encode.restype = None
    L.orc_stochquant_encode.argtypes = [_f32p, _f32p, i64, i32, i32, _i16p, _f32p]
    L.orc_stochquant_decode.restype = None
    L.orc_stochquant_decode.argtypes = [_i16p, _f32p, i64, i32, _f32p]
    L.orc_uniform24.restype = None
    L.orc_uniform24.argtypes = [u64, i32, i64, i64, i64, _f32p]
    L.orc_form_p_partial.restype = None
    L.orc_form_p_partial.argtypes = [f32, f32, _f32p, _f32p, i64, _f32p]
    L.orc_partial_keep.restype = None
    L.orc_partial_keep.argtypes = [f32, _f32p, _f32p, i64, _f32p]
    L.orc_chunk_window.restype = None
    L.orc_chunk_window.argtypes = [i64, i64, i64, i64, C.POINTER(i64), C.POINTER(i64)]
    L.orc_sketch_encode_chunked.restype = i32
    L.orc_sketch_encode_chunked.argtypes = [_f32p, i64, i32, i64, i64, u64, i64, _f32p]
    L.orc_sketch_decode_chunked.restype = None
    L.orc_sketch_decode_chunked.argtypes = [_f32p, i64, i32, i64, i64, u64, i64, _f32p]
    L.orc_rowsketch_update.restype = i32
    L.orc_rowsketch_update.argtypes = [f32, _f32p, i64, i64, i32, i64, u64, i64, _f32p]
    L.orc_rowsketch_update_f16.restype = i32
    L.orc_rowsketch_update_f16.argtypes = [f32, _f32p, i64, i64, i32, i64, u64, i64, _u16p]
    L.orc_rowsketch_decode_f16.restype = None
    L.orc_rowsketch_decode_f16.argtypes = [_u16p, i64, i64, i32, i64, u64, i64, _f32p]
    L.orc_error_reset_f16.restype = None
    L.orc_error_reset_f16.argtypes = [C.POINTER(C.c_void_p), i32, i64]
    L.orc_rowsketch_decode.restype = None
    L.orc_rowsketch_decode.argtypes = [_f32p, i64, i64, i32, i64, u64, i64, _f32p]


# ------------------------------------------------------------------ thin wrappers


def mix64(z: int) -> int:
    return lib().orc_mix64(z & (2**64 - 1))


def h64(seed: int, a: int, b: int, j: int) -> int:
    return lib().orc_h64(lib().orc_stream(seed, a, b), j)


def f32_to_f16_bits(x: float) -> int:
    return lib().orc_f32_to_f16(x)


def f16_bits_to_f32(h: int) -> float:
    return lib().orc_f16_to_f32(h)


def form_p(lr: float, g: np.ndarray, e: np.ndarray) -> np.ndarray:
    p = np.empty_like(g)
    lib().orc_form_p(lr, g, e, g.size, p)
    return p


def passthrough(lr: float, g: np.ndarray) -> np.ndarray:
    out = np.empty_like(g)
    lib().orc_passthrough(lr, g, g.size, out)
    return out


def randk_indices(seed: int, tensor: int, step: int, d: int, k: int) -> np.ndarray:
    idx = np.empty(k, dtype=np.uint32)
    rc = lib().orc_randk_indices(seed, tensor, step, d, k, idx)
    if rc != 0:
        raise ValueError(f"orc_randk_indices failed: {rc}")
    return idx


def randblock_indices(seed: int, tensor: int, step: int, d: int, k: int) -> np.ndarray:
    """Random-block-k: the k consecutive indices from the shared random start."""
    start = lib().orc_randblock_start(seed, tensor, step, d, k)
    return np.arange(start, start + k, dtype=np.uint32)


def randk_apply(p: np.ndarray, idx: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    msg = np.empty(idx.size, dtype=np.float32)
    r = np.empty_like(p)
    lib().orc_randk_apply(p, p.size, idx, idx.size, msg, r)
    return msg, r


def quant_encode(r: np.ndarray, block: int, bits: int, scale_half: bool):
    d = r.size
    nb = (d + block - 1) // block
    codes = np.zeros(d if bits == 8 else (d + 1) // 2, dtype=np.uint8)
    s32 = np.empty(nb, dtype=np.float32)
    s16 = np.zeros(nb, dtype=np.uint16)
    lib().orc_quant_encode(r, d, block, bits, int(scale_half), codes, s32,
                           s16.ctypes.data_as(C.c_void_p) if scale_half else None)
    return codes, s32, (s16 if scale_half else None)


def quant_decode(codes: np.ndarray, s32: np.ndarray, d: int, block: int, bits: int) -> np.ndarray:
    e = np.empty(d, dtype=np.float32)
    lib().orc_quant_decode(codes, s32, d, block, bits, e)
    return e


def sketch_bucket(seed: int, tensor: int, row: int, j: int, w: int) -> Tuple[int, int]:
    b, s = C.c_int64(), C.c_int()
    lib().orc_sketch_bucket(seed, tensor, row, j, w, C.byref(b), C.byref(s))
    return b.value, s.value


def sketch_encode(r: np.ndarray, v: int, w: int, seed: int, tensor: int) -> np.ndarray:
    S = np.empty(v * w, dtype=np.float32)
    rc = lib().orc_sketch_encode(r, r.size, v, w, seed, tensor, S)
    if rc != 0:
        raise MemoryError
    return S


def sketch_decode(S: np.ndarray, d: int, v: int, w: int, seed: int, tensor: int) -> np.ndarray:
    e = np.empty(d, dtype=np.float32)
    lib().orc_sketch_decode(S, d, v, w, seed, tensor, e)
    return e


def chunk_window(d: int, w: int, chunk: int, j: int) -> Tuple[int, int]:
    """(first bucket, width) of the window that element j's run owns in every sketch row."""
    lo, width = C.c_int64(), C.c_int64()
    lib().orc_chunk_window(d, w, chunk, j, C.byref(lo), C.byref(width))
    return lo.value, width.value


def sketch_encode_chunked(r: np.ndarray, v: int, w: int, chunk: int, seed: int, tensor: int) -> np.ndarray:
    S = np.empty(v * w, dtype=np.float32)
    rc = lib().orc_sketch_encode_chunked(r, r.size, v, w, chunk, seed, tensor, S)
    if rc != 0:
        raise MemoryError
    return S


def sketch_decode_chunked(S: np.ndarray, d: int, v: int, w: int, chunk: int, seed: int, tensor: int) -> np.ndarray:
    e = np.empty(d, dtype=np.float32)
    lib().orc_sketch_decode_chunked(S, d, v, w, chunk, seed, tensor, e)
    return e


def stochquant_encode(r: np.ndarray, rnd: np.ndarray, block: int, levels: int):
    """Eq. 6 with the max-norm, block-wise: (signed levels int16[d], scales fp32[nblocks])."""
    d = r.size
    codes = np.empty(d, np.int16)
    scales = np.empty((d + block - 1) // block, np.float32)
    lib().orc_stochquant_encode(r, rnd, d, block, levels, codes, scales)
    return codes, scales


def stochquant_decode(codes: np.ndarray, scales: np.ndarray, block: int) -> np.ndarray:
    e = np.empty(codes.size, np.float32)
    lib().orc_stochquant_decode(codes, scales, codes.size, block, e)
    return e


def uniform24(seed: int, worker: int, tensor: int, step: int, d: int) -> np.ndarray:
    """The quantiser's uniform variates in [0, 1): a pure function of (seed, worker, tensor, step, j)."""
    out = np.empty(d, np.float32)
    lib().orc_uniform24(seed, worker, tensor, step, d, out)
    return out


def form_p_partial(lr: float, one_minus_beta: float, g: np.ndarray, e: np.ndarray) -> np.ndarray:
    """Alg. 4 line 5: p = eta g + (1 - beta) e."""
    p = np.empty_like(g)
    lib().orc_form_p_partial(lr, one_minus_beta, g, e, g.size, p)
    return p


def partial_keep(beta: float, e: np.ndarray, r: np.ndarray) -> np.ndarray:
    """Alg. 4 line 9, the argument of a non-linear C: beta e + (p - Delta)."""
    x = np.empty_like(r)
    lib().orc_partial_keep(beta, e, r, r.size, x)
    return x


def rowsketch_update(beta: float, R: np.ndarray, T: np.ndarray, v: int, w: int, seed: int,
                     tensor: int) -> np.ndarray:
    """T <- beta T + sketch(R) for the row-wise count sketch (R is n x m); returns the new T."""
    n, m = R.shape
    T = np.ascontiguousarray(T, dtype=np.float32).copy()
    assert T.size == v * w * m
    rc = lib().orc_rowsketch_update(beta, np.ascontiguousarray(R, dtype=np.float32).reshape(-1), n, m, v, w,
                                    seed, tensor, T)
    if rc != 0:
        raise MemoryError
    return T


def rowsketch_update_f16(beta: float, R: np.ndarray, T16: np.ndarray, v: int, w: int, seed: int,
                         tensor: int) -> np.ndarray:
    """The same update on a sketch stored as binary16 bit patterns (uint16); returns the new one."""
    n, m = R.shape
    T16 = np.ascontiguousarray(T16, dtype=np.uint16).copy()
    assert T16.size == v * w * m
    rc = lib().orc_rowsketch_update_f16(beta, np.ascontiguousarray(R, dtype=np.float32).reshape(-1), n, m, v, w,
                                        seed, tensor, T16)
    if rc != 0:
        raise MemoryError
    return T16


def rowsketch_decode_f16(T16: np.ndarray, n: int, m: int, v: int, w: int, seed: int, tensor: int) -> np.ndarray:
    e = np.empty(n * m, dtype=np.float32)
    lib().orc_rowsketch_decode_f16(T16, n, m, v, w, seed, tensor, e)
    return e


def rowsketch_decode(T: np.ndarray, n: int, m: int, v: int, w: int, seed: int, tensor: int) -> np.ndarray:
    e = np.empty(n * m, dtype=np.float32)
    lib().orc_rowsketch_decode(T, n, m, v, w, seed, tensor, e)
    return e


def lowrank_project_rows(M: np.ndarray, Q: np.ndarray) -> np.ndarray:
    n, m = M.shape
    r = Q.shape[1]
    P = np.empty((n, r), dtype=np.float32)
    lib().orc_lowrank_project_rows(M, n, m, Q, r, P)
    return P


def gram_schmidt(P: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(P, dtype=np.float32).copy()
    lib().orc_gram_schmidt(out, out.shape[0], out.shape[1])
    return out


def lowrank_project_cols(M: np.ndarray, Phat: np.ndarray) -> np.ndarray:
    n, m = M.shape
    r = Phat.shape[1]
    Qi = np.empty((m, r), dtype=np.float32)
    lib().orc_lowrank_project_cols(M, n, m, Phat, r, Qi)
    return Qi


def lowrank_residual(M: np.ndarray, Phat: np.ndarray, Qi: np.ndarray, want_delta: bool = False):
    n, m = M.shape
    res = np.empty((n, m), dtype=np.float32)
    delta = np.empty((n, m), dtype=np.float32) if want_delta else None
    lib().orc_lowrank_residual(M, n, m, Phat, Qi, Phat.shape[1], res,
                               delta.ctypes.data_as(C.c_void_p) if want_delta else None)
    return (res, delta) if want_delta else res


def sum_workers(msgs: Sequence[np.ndarray]) -> np.ndarray:
    n = len(msgs)
    ln = msgs[0].size
    arr = (C.c_void_p * n)(*[m.ctypes.data for m in msgs])
    out = np.empty(ln, dtype=np.float32)
    lib().orc_sum_workers(arr, n, ln, out)
    return out.reshape(msgs[0].shape)


def divide(x: np.ndarray, denom: float) -> np.ndarray:
    out = np.empty_like(x)
    lib().orc_divide(x, denom, x.size, out)
    return out


# ------------------------------------------------------------------ configuration


@dataclass
class QCfg:
    """Gradient compressor Q (Alg. 2 line 6)."""
    kind: str = "randk"            # 'identity' | 'randk' | 'randblock' | 'lowrank'
    k_num: int = 1                 # random-k: k = max(1, floor(d * k_num / k_den))
    k_den: int = 100
    rank: int = 4                  # low-rank: r = min(rank, rows, cols)
    q_init: Optional[np.ndarray] = None  # concat over compressed tensors of (cols x r) row-major
    seed: int = 0


@dataclass
class CCfg:
    """Error compressor C (Alg. 2 line 9)."""
    kind: str = "int8"             # 'identity' | 'int8' | 'int4' | 'countsketch' | 'rowsketch' | 'stochquant'
    block: int = 256
    scale_dtype: str = "fp32"      # 'fp32' | 'fp16'
    cs_rows: int = 5               # v
    cs_col_div: int = 10           # w = max(1, floor(d / cs_col_div)); rowsketch: floor(rows / cs_col_div)
    seed: int = 0
    beta: float = 0.0              # partial error feedback (Alg. 4); 0 is Alg. 2
    levels: int = 16               # stochastic quantiser: s (Eq. 6)
    iconef: int = 0                # 1: iConEF-v1 (Alg. 3): a second stored state q = C(r - e~);
                                   # 2: iConEF-v2: e~ = Q(r) kept as the k values of a second draw of Q, q = C(r - e~)
    cs_chunk: int = 0              # count sketch: > 0 sketches runs of this many elements on their own


SECOND_DRAW = 1 << 62     # step offset of the stream that the second application of Q draws from (iConEF-v2)


@dataclass
class LayerStep:
    """Everything the oracle produced for one tensor in one step."""
    idx: Optional[np.ndarray] = None            # random-k index set (shared)
    idx2: Optional[np.ndarray] = None           # iConEF-v2: index set of e~ = Q(r)
    msg: List[np.ndarray] = field(default_factory=list)   # per worker: values / dense 1-D
    P: List[np.ndarray] = field(default_factory=list)     # per worker n x r
    Pbar: Optional[np.ndarray] = None
    Phat: Optional[np.ndarray] = None
    Qi: List[np.ndarray] = field(default_factory=list)    # per worker m x r
    Qsum: Optional[np.ndarray] = None
    p: List[np.ndarray] = field(default_factory=list)     # per worker, when record=True
    r: List[np.ndarray] = field(default_factory=list)     # per worker, when record=True


class ConEFOracle:
    """Algorithm 2 for N simulated workers on a list of tensors.

    ``tensors`` is a list of (rows, cols, compress).  A tensor with cols == 1
    or compress == 0 passes through: its message is eta * g and it keeps no
    error state.  Gradients are given per worker as one flat fp32 array, the
    concatenation of all tensors in table order.
    """

    def __init__(self, tensors: Sequence[Tuple[int, int, int]], n_workers: int, q: QCfg, c: CCfg,
                 lr: float):
        self.tensors = [(int(a), int(b), int(cc)) for a, b, cc in tensors]
        self.N = int(n_workers)
        self.q, self.c = q, c
        self.lr = np.float32(lr)
        self.offsets = np.concatenate([[0], np.cumsum([a * b for a, b, _ in self.tensors])]).astype(np.int64)
        self.compressed = [l for l, (a, b, cc) in enumerate(self.tensors) if cc and b > 1]
        # e_0 = 0 (Alg. 2 line 1)
        self.state: List[Dict[int, dict]] = [dict() for _ in range(self.N)]
        for i in range(self.N):
            for l in self.compressed:
                self.state[i][l] = self._zero_state(l)
        # iConEF-v1 (Alg. 3 line 1): q_0 = 0, a second state of the same kind
        self.state2: List[Dict[int, dict]] = [dict() for _ in range(self.N)]
        if c.iconef:
            if c.kind not in ("identity", "int8", "int4") or c.beta != 0:
                raise ValueError("iConEF is defined here for the deterministic quantisers and identity, beta = 0")
        if c.iconef == 1:
            for i in range(self.N):
                for l in self.compressed:
                    self.state2[i][l] = self._zero_state(l)
        # iConEF-v2 (Alg. 3 line 12): e~ = Q(r) is sparse; kept as (indices, values) of the second
        # draw of Q at the step that stored it; `state` holds q.  e~_0 = 0.
        self.ev: List[Dict[int, Optional[Tuple[np.ndarray, np.ndarray]]]] = [dict() for _ in range(self.N)]
        if c.iconef == 2:
            if q.kind not in ("randk", "randblock"):
                raise ValueError("iConEF-v2 is defined here for random-k and random-block-k")
            for i in range(self.N):
                for l in self.compressed:
                    self.ev[i][l] = None
        # shared warm start of the low-rank compressor
        self.Qprev: Dict[int, np.ndarray] = {}
        if q.kind == "lowrank":
            off = 0
            for l in self.compressed:
                n, m, _ = self.tensors[l]
                r = self.rank_of(l)
                self.Qprev[l] = np.ascontiguousarray(
                    np.asarray(q.q_init[off:off + m * r], dtype=np.float32).reshape(m, r))
                off += m * r

    # -- per-tensor derived sizes
    def d_of(self, l: int) -> int:
        return self.tensors[l][0] * self.tensors[l][1]

    def k_of(self, l: int) -> int:
        return max(1, self.d_of(l) * self.q.k_num // self.q.k_den)

    def rank_of(self, l: int) -> int:
        return min(self.q.rank, self.tensors[l][0], self.tensors[l][1])

    def w_of(self, l: int) -> int:
        if self.c.kind == "rowsketch":
            return max(1, self.tensors[l][0] // self.c.cs_col_div)
        return max(1, self.d_of(l) // self.c.cs_col_div)

    def _bits(self) -> int:
        return 8 if self.c.kind == "int8" else 4

    def _zero_state(self, l: int) -> dict:
        d = self.d_of(l)
        k = self.c.kind
        if k == "identity":
            return {"e": np.zeros(d, np.float32)}
        if k in ("int8", "int4"):
            nb = (d + self.c.block - 1) // self.c.block
            return {"codes": np.zeros(d if k == "int8" else (d + 1) // 2, np.uint8),
                    "scales": np.zeros(nb, np.float32),
                    "scales16": np.zeros(nb, np.uint16) if self.c.scale_dtype == "fp16" else None}
        if k == "countsketch":
            return {"S": np.zeros(self.c.cs_rows * self.w_of(l), np.float32)}
        if k == "stochquant":
            return {"levels": np.zeros(d, np.int16),
                    "scales": np.zeros((d + self.c.block - 1) // self.c.block, np.float32)}
        if k == "rowsketch":
            size = self.c.cs_rows * self.w_of(l) * self.tensors[l][1]
            if self.c.scale_dtype == "fp16":     # the sketch itself in binary16
                return {"T16": np.zeros(size, np.uint16)}
            return {"T": np.zeros(size, np.float32)}
        raise ValueError(k)

    # -- Alg. 2 line 5 (decode of the stored error); second=True: the state q of Alg. 3
    def decode(self, i: int, l: int, second: bool = False) -> np.ndarray:
        st = (self.state2 if second else self.state)[i][l]
        k = self.c.kind
        if k == "identity":
            return st["e"].copy()
        if k in ("int8", "int4"):
            return quant_decode(st["codes"], st["scales"], self.d_of(l), self.c.block, self._bits())
        if k == "stochquant":
            return stochquant_decode(st["levels"], st["scales"], self.c.block)
        if k == "rowsketch":
            n, m, _ = self.tensors[l]
            if "T16" in st:
                return rowsketch_decode_f16(st["T16"], n, m, self.c.cs_rows, self.w_of(l), self.c.seed, l)
            return rowsketch_decode(st["T"], n, m, self.c.cs_rows, self.w_of(l), self.c.seed, l)
        if self.c.cs_chunk > 0:
            return sketch_decode_chunked(st["S"], self.d_of(l), self.c.cs_rows, self.w_of(l), self.c.cs_chunk,
                                         self.c.seed, l)
        return sketch_decode(st["S"], self.d_of(l), self.c.cs_rows, self.w_of(l), self.c.seed, l)

    # iConEF-v2: the stored e~ of (worker, tensor) as a dense vector
    def ev_dense(self, i: int, l: int) -> np.ndarray:
        e = np.zeros(self.d_of(l), np.float32)
        if self.ev[i][l] is not None:
            idx, val = self.ev[i][l]
            e[idx] = val
        return e

    # -- Alg. 2 line 9 / Alg. 4 line 9 (store through C); e is the decoded old error, used when beta != 0
    def encode(self, i: int, l: int, r: np.ndarray, e: Optional[np.ndarray] = None, t: int = 0) -> None:
        if self.c.iconef == 1:
            # Alg. 3 lines 10 and 14: e~ = C(r); q = C(r - e~), elementwise fp32 difference
            self._encode_into(self.state, i, l, r, e, t)
            r2 = (np.ascontiguousarray(r.reshape(-1), dtype=np.float32) - self.decode(i, l)).astype(np.float32)
            self._encode_into(self.state2, i, l, r2, e, t)
            return
        self._encode_into(self.state, i, l, r, e, t)

    def _encode_into(self, store, i: int, l: int, r: np.ndarray, e: Optional[np.ndarray], t: int) -> None:
        k = self.c.kind
        r = np.ascontiguousarray(r.reshape(-1), dtype=np.float32)
        beta = np.float32(self.c.beta)
        if k == "rowsketch":
            # linear C: T <- beta T + sketch(r), no decode needed
            n, m, _ = self.tensors[l]
            if "T16" in store[i][l]:
                store[i][l] = {"T16": rowsketch_update_f16(beta, r.reshape(n, m), store[i][l]["T16"],
                                                           self.c.cs_rows, self.w_of(l), self.c.seed, l)}
            else:
                store[i][l] = {"T": rowsketch_update(beta, r.reshape(n, m), store[i][l]["T"],
                                                     self.c.cs_rows, self.w_of(l), self.c.seed, l)}
            return
        if beta != 0:
            r = partial_keep(beta, e, r)
        if k == "stochquant":
            rnd = uniform24(self.c.seed, i, l, t, r.size)
            lv, sc = stochquant_encode(r, rnd, self.c.block, self.c.levels)
            store[i][l] = {"levels": lv, "scales": sc}
        elif k == "identity":
            store[i][l] = {"e": r.copy()}
        elif k in ("int8", "int4"):
            codes, s32, s16 = quant_encode(r, self.c.block, self._bits(), self.c.scale_dtype == "fp16")
            store[i][l] = {"codes": codes, "scales": s32, "scales16": s16}
        else:
            if self.c.cs_chunk > 0:
                store[i][l] = {"S": sketch_encode_chunked(r, self.c.cs_rows, self.w_of(l), self.c.cs_chunk,
                                                          self.c.seed, l)}
            else:
                store[i][l] = {"S": sketch_encode(r, self.c.cs_rows, self.w_of(l), self.c.seed, l)}

    def decompress_error(self, i: int) -> np.ndarray:
        """e of worker i, concatenated over the compressed tensors in table order."""
        if not self.compressed:
            return np.zeros(0, np.float32)
        if self.c.iconef == 1:   # the error carried to the next step is e~ + q
            return np.concatenate([(self.decode(i, l) + self.decode(i, l, True)).astype(np.float32) for l in self.compressed])
        if self.c.iconef == 2:
            return np.concatenate([(self.ev_dense(i, l) + self.decode(i, l)).astype(np.float32) for l in self.compressed])
        return np.concatenate([self.decode(i, l) for l in self.compressed])

    def _grad(self, grads, i: int, l: int) -> np.ndarray:
        return np.ascontiguousarray(grads[i][self.offsets[l]:self.offsets[l + 1]], dtype=np.float32)

    def step(self, t: int, grads: Sequence[np.ndarray], record: bool = False,
             layers: Optional[Sequence[int]] = None) -> Dict[int, LayerStep]:
        """One iteration of Alg. 2 for all workers; returns per-tensor results.

        ``layers`` restricts the work to a subset of tensors (used to time a
        bounded sample); the others keep their state.
        """
        out: Dict[int, LayerStep] = {}
        todo = range(len(self.tensors)) if layers is None else layers
        for l in todo:
            n, m, cc = self.tensors[l]
            d = n * m
            ls = LayerStep()
            out[l] = ls
            if l not in self.compressed:
                ls.msg = [passthrough(self.lr, self._grad(grads, i, l)) for i in range(self.N)]
                continue
            # line 5: p = eta g + e  (Alg. 4: eta g + (1 - beta) e)
            if self.c.iconef == 2:
                es = [self.ev_dense(i, l) for i in range(self.N)]
            else:
                es = [self.decode(i, l) for i in range(self.N)]
            if self.c.beta != 0:
                omb = np.float32(1.0) - np.float32(self.c.beta)
                ps = [form_p_partial(self.lr, omb, self._grad(grads, i, l), es[i]) for i in range(self.N)]
            else:
                ps = [form_p(self.lr, self._grad(grads, i, l), es[i]) for i in range(self.N)]
            if self.c.iconef == 1:   # Alg. 3 line 5: p = (eta g + e~) + q
                ps = [(ps[i] + self.decode(i, l, True)).astype(np.float32) for i in range(self.N)]
            elif self.c.iconef == 2:   # the same line; q is what `state` holds
                ps = [(ps[i] + self.decode(i, l)).astype(np.float32) for i in range(self.N)]
            if record:
                ls.p = [p.copy() for p in ps]
            # line 6: Delta = Q(p); line 9: r = p - Delta
            if self.q.kind == "identity":
                ls.msg = ps
                rs = [p - p for p in ps]
            elif self.q.kind in ("randk", "randblock"):
                pick = randk_indices if self.q.kind == "randk" else randblock_indices
                ls.idx = pick(self.q.seed, l, t, d, self.k_of(l))
                rs = []
                for p in ps:
                    msg, r = randk_apply(p, ls.idx)
                    ls.msg.append(msg)
                    rs.append(r)
            elif self.q.kind == "lowrank":
                Ms = [p.reshape(n, m) for p in ps]
                ls.P = [lowrank_project_rows(M, self.Qprev[l]) for M in Ms]
                ls.Pbar = sum_workers(ls.P)            # first all-reduce
                ls.Phat = gram_schmidt(ls.Pbar)
                ls.Qi = [lowrank_project_cols(M, ls.Phat) for M in Ms]
                rs = [lowrank_residual(M, ls.Phat, Qi).reshape(-1) for M, Qi in zip(Ms, ls.Qi)]
                ls.Qsum = sum_workers(ls.Qi)           # second all-reduce
                self.Qprev[l] = divide(ls.Qsum, np.float32(self.N))
            else:
                raise ValueError(self.q.kind)
            if record:
                ls.r = [r.copy() for r in rs]
            if self.c.iconef == 2:
                # Alg. 3 line 12: e~ = Q(p - Delta), a second draw of Q in the same step (its stream is
                # that of step t + 2^62); line 14: q = C(p - Delta - e~), and r - e~ is exactly 0 on
                # the coordinates e~ keeps
                pick = randk_indices if self.q.kind == "randk" else randblock_indices
                ls.idx2 = pick(self.q.seed, l, t + SECOND_DRAW, d, self.k_of(l))
                for i in range(self.N):
                    self.ev[i][l] = (ls.idx2, rs[i][ls.idx2].copy())
                    rs[i] = rs[i].copy()
                    rs[i][ls.idx2] = 0.0
            for i in range(self.N):
                self.encode(i, l, rs[i], es[i], t)
        return out

    # -- error reset (linear C only)
    def error_reset(self) -> None:
        key = {"identity": "e", "countsketch": "S", "rowsketch": "T"}.get(self.c.kind)
        if key is None:
            raise ValueError("error reset needs a linear error compressor")
        for l in self.compressed:
            half = "T16" in self.state[0][l]
            arrs = [self.state[i][l]["T16" if half else key] for i in range(self.N)]
            ptrs = (C.c_void_p * self.N)(*[a.ctypes.data for a in arrs])
            (lib().orc_error_reset_f16 if half else lib().orc_error_reset)(ptrs, self.N, arrs[0].size)

    # -- Alg. 2 lines 7-8
    def apply_update(self, x: np.ndarray, res: Dict[int, LayerStep]) -> None:
        """x <- x - Delta_t in place; x is the flat parameter vector (all tensors, table order)
        and res the result of this step."""
        L = lib()
        N = np.float32(self.N)
        for l in sorted(res):
            ls = res[l]
            n, m, _ = self.tensors[l]
            xs = x[self.offsets[l]:self.offsets[l + 1]]
            assert xs.flags["C_CONTIGUOUS"] and xs.dtype == np.float32
            if l not in self.compressed or self.q.kind == "identity":
                L.orc_apply_dense(xs, sum_workers(ls.msg), N, xs.size)
            elif self.q.kind in ("randk", "randblock"):
                L.orc_apply_sparse(xs, ls.idx, sum_workers(ls.msg), N, ls.idx.size)
            else:
                qmean = divide(ls.Qsum, N)
                L.orc_apply_lowrank(xs, n, m, np.ascontiguousarray(ls.Phat), qmean, self.rank_of(l))

    # -- message concatenations, in the layout the library's reduce call returns
    def reduced(self, res: Dict[int, LayerStep], which: str) -> np.ndarray:
        """Sum over workers (Alg. 2 line 7, before the division by N) of one
        message kind, concatenated over tensors in table order.
        which: 'values' | 'P' | 'Q' | 'dense1d'."""
        parts = []
        for l in sorted(res):
            ls = res[l]
            if which == "dense1d":
                if l not in self.compressed:
                    parts.append(sum_workers(ls.msg))
            elif l in self.compressed:
                if which == "values" and ls.msg:
                    parts.append(sum_workers(ls.msg))
                elif which == "P" and ls.Pbar is not None:
                    parts.append(ls.Pbar.reshape(-1))
                elif which == "Q" and ls.Qsum is not None:
                    parts.append(ls.Qsum.reshape(-1))
        return np.concatenate(parts) if parts else np.zeros(0, np.float32)
