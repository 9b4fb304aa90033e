"""ctypes binding of libconef.so: the same entry points as include/conef.h.

Argument marshalling only.  Every step of the path runs in the library's CUDA
kernels; PyTorch supplies device memory and the stream.  Importing this module
fails loudly when the library is missing or cannot be loaded: there is no CPU
fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libconef.so")

OK = 0
ERR_INVALID_ARG, ERR_BAD_PHASE, ERR_WORKSPACE_TOO_SMALL, ERR_UNSUPPORTED, ERR_CUDA, ERR_DEVICE_STATUS, \
    ERR_TOO_LARGE = -1, -2, -3, -4, -5, -6, -7
NOALLOC_MAX_ELEMS = 1 << 24
Q_IDENTITY, Q_RANDK, Q_LOWRANK, Q_RANDBLOCK = 0, 1, 2, 3
C_IDENTITY, C_INT8, C_INT4, C_COUNTSKETCH, C_ROWSKETCH, C_STOCHQUANT = 0, 1, 2, 3, 4, 5
SCALE_FP32, SCALE_FP16 = 0, 1
MSG_VALUES, MSG_P, MSG_Q, MSG_DENSE1D = 0, 1, 2, 3
MAX_WORKERS, MAX_RANK = 64, 8

EXPORTS = ["conef_workspace_bytes", "conef_init", "conef_step", "conef_reduce_messages",
           "conef_decompress_error", "conef_apply_update", "conef_error_reset", "conef_destroy", "conef_message_elems", "conef_error_elems",
           "conef_state_bytes_per_worker", "conef_get_message", "conef_get_state", "conef_get_state2",
           "conef_get_indices", "conef_get_factors", "conef_last_status", "conef_launch_count",
           "conef_set_fast_path", "conef_set_total_workers", "conef_error_string", "conef_randk_indices_noalloc",
           "conef_get_error_step", "conef_set_error_step", "conef_set_fused", "conef_fused_info",
           "conef_get_fused_q"]


class conef_tensor(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("compress", C.c_int32), ("reserved", C.c_int32)]


class conef_q_cfg(C.Structure):
    _fields_ = [("kind", C.c_int32), ("rank", C.c_int32), ("k_num", C.c_int64), ("k_den", C.c_int64),
                ("q_init", C.c_void_p), ("seed", C.c_uint64)]


class conef_c_cfg(C.Structure):
    _fields_ = [("kind", C.c_int32), ("block", C.c_int32), ("scale_dtype", C.c_int32),
                ("cs_rows", C.c_int32), ("cs_col_div", C.c_int64), ("seed", C.c_uint64),
                ("beta", C.c_float), ("levels", C.c_int32), ("iconef", C.c_int32), ("cs_chunk", C.c_int32)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2312_08538_b200.build` "
            "(nvcc, sm_100a). There is no CPU fallback.")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int, C.c_int64
    L.conef_workspace_bytes.argtypes = [C.POINTER(conef_tensor), i32, i32, C.POINTER(conef_q_cfg),
                                        C.POINTER(conef_c_cfg), C.POINTER(C.c_size_t)]
    L.conef_init.argtypes = [C.POINTER(vp), C.POINTER(conef_tensor), i32, i32, C.POINTER(conef_q_cfg),
                             C.POINTER(conef_c_cfg), C.c_float, vp, C.c_size_t, vp]
    L.conef_step.argtypes = [vp, i64, C.POINTER(vp), i32, vp]
    L.conef_reduce_messages.argtypes = [vp, i32, vp, vp]
    L.conef_decompress_error.argtypes = [vp, i32, vp, vp]
    L.conef_apply_update.argtypes = [vp, vp, vp, vp, vp]
    L.conef_error_reset.argtypes = [vp, vp]
    L.conef_destroy.argtypes = [vp]
    L.conef_destroy.restype = None
    for name in ("conef_message_elems",):
        getattr(L, name).argtypes = [vp, i32]
        getattr(L, name).restype = i64
    L.conef_set_error_step.argtypes = [vp, i64]
    for name in ("conef_error_elems", "conef_state_bytes_per_worker", "conef_launch_count", "conef_get_error_step"):
        getattr(L, name).argtypes = [vp]
        getattr(L, name).restype = i64
    L.conef_get_message.argtypes = [vp, i32, i32, C.POINTER(vp)]
    L.conef_get_state.argtypes = [vp, i32, i32, C.POINTER(vp), C.POINTER(C.c_size_t), C.POINTER(vp),
                                  C.POINTER(C.c_size_t)]
    L.conef_get_state2.argtypes = L.conef_get_state.argtypes
    L.conef_get_indices.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(i64)]
    L.conef_get_factors.argtypes = [vp, i32, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                    C.POINTER(vp), C.POINTER(i32)]
    L.conef_last_status.argtypes = [vp, vp, C.POINTER(i32)]
    L.conef_set_fast_path.argtypes = [vp, i32]
    L.conef_set_total_workers.argtypes = [vp, i32]
    L.conef_set_fused.argtypes = [vp, i32, i32, i32]
    L.conef_fused_info.argtypes = [vp] + [C.POINTER(i32)] * 5
    L.conef_get_fused_q.argtypes = [vp, i32, i32, C.POINTER(vp)]
    L.conef_randk_indices_noalloc.argtypes = [C.c_uint64, i64, i64, i64, i64, vp, vp]
    L.conef_error_string.argtypes = [i32]
    L.conef_error_string.restype = C.c_char_p
    return L


lib = _load()


class ConEFError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib.conef_error_string(code).decode()} ({code})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise ConEFError(code, where)


_QK = {"identity": Q_IDENTITY, "randk": Q_RANDK, "lowrank": Q_LOWRANK, "randblock": Q_RANDBLOCK}
_CK = {"identity": C_IDENTITY, "int8": C_INT8, "int4": C_INT4, "countsketch": C_COUNTSKETCH,
       "rowsketch": C_ROWSKETCH, "stochquant": C_STOCHQUANT}


def make_tensors(tensors: Sequence[Tuple[int, int, int]]):
    arr = (conef_tensor * len(tensors))()
    for i, (r, c, k) in enumerate(tensors):
        arr[i] = conef_tensor(int(r), int(c), int(k), 0)
    return arr


def make_q(q: Dict, q_init: Optional[torch.Tensor]) -> conef_q_cfg:
    return conef_q_cfg(_QK[q["kind"]], int(q.get("rank", 0)), int(q.get("k_num", 1)),
                       int(q.get("k_den", 100)), q_init.data_ptr() if q_init is not None else None,
                       int(q.get("seed", 0)))


def make_c(c: Dict) -> conef_c_cfg:
    return conef_c_cfg(_CK[c["kind"]], int(c.get("block", 256)),
                       SCALE_FP16 if c.get("scale_dtype", "fp32") == "fp16" else SCALE_FP32,
                       int(c.get("cs_rows", 5)), int(c.get("cs_col_div", 10)), int(c.get("seed", 0)),
                       float(c.get("beta", 0.0)), int(c.get("levels", 16)), int(c.get("iconef", 0)), int(c.get("cs_chunk", 0)))


def conef_workspace_bytes(tensors, n_workers: int, q: Dict, c: Dict) -> int:
    out = C.c_size_t()
    t = make_tensors(tensors)
    qc, cc = make_q(q, None), make_c(c)
    _check(lib.conef_workspace_bytes(t, len(tensors), n_workers, C.byref(qc), C.byref(cc), C.byref(out)),
           "conef_workspace_bytes")
    return out.value


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def conef_randk_indices_noalloc(seed: int, tensor: int, step: int, d: int, k: int, idx_out: torch.Tensor,
                                stream=None) -> None:
    """The shared random-k index set of (seed, tensor, step), written into the caller's
    int32/uint32 device tensor of k entries.  For callers that hold no context and may not
    allocate device memory (the receiving side of a random-k message): the library's scratch
    for this call is a fixed array in its device image, so d is limited to NOALLOC_MAX_ELEMS."""
    assert idx_out.is_cuda and idx_out.element_size() == 4 and idx_out.numel() >= k and idx_out.is_contiguous()
    _check(lib.conef_randk_indices_noalloc(int(seed), int(tensor), int(step), int(d), int(k), idx_out.data_ptr(),
                                           _stream_handle(stream)), "conef_randk_indices_noalloc")


class ConEF:
    """One context of the library: N simulated workers on the current device."""

    def __init__(self, tensors, n_workers: int, q: Dict, c: Dict, lr: float,
                 q_init: Optional[torch.Tensor] = None, device="cuda", stream=None):
        self.tensors = [(int(a), int(b), int(k)) for a, b, k in tensors]
        self.n_workers = int(n_workers)
        self.device = torch.device(device)
        self.q, self.c = dict(q), dict(c)
        nbytes = conef_workspace_bytes(self.tensors, self.n_workers, q, c)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_off = (-base) % 256
        self._ws_ptr = base + self._ws_off
        self._ws_bytes = nbytes
        if q_init is not None:
            q_init = q_init.to(self.device, torch.float32).contiguous()
        self._q_init = q_init
        self._t = make_tensors(self.tensors)
        qc, cc = make_q(q, q_init), make_c(c)
        h = C.c_void_p()
        _check(lib.conef_init(C.byref(h), self._t, len(self.tensors), self.n_workers, C.byref(qc),
                              C.byref(cc), float(lr), self._ws_ptr, nbytes, _stream_handle(stream)),
               "conef_init")
        self.h = h

    def close(self):
        if getattr(self, "h", None) and lib is not None:
            lib.conef_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    # ---- the four calls
    def step(self, t: int, grads: Sequence[torch.Tensor], phase: int = 0, stream=None) -> None:
        arr = (C.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
        _check(lib.conef_step(self.h, int(t), arr, int(phase), _stream_handle(stream)), "conef_step")

    def reduce_messages(self, which: int, out: Optional[torch.Tensor] = None, stream=None,
                        want_output: bool = True) -> Optional[torch.Tensor]:
        if out is None and want_output:
            out = torch.empty(self.message_elems(which), dtype=torch.float32, device=self.device)
        _check(lib.conef_reduce_messages(self.h, which, out.data_ptr() if out is not None else None,
                                         _stream_handle(stream)), "conef_reduce_messages")
        return out

    def error_reset(self, stream=None) -> None:
        """Every worker's (linear) error state becomes the mean over workers (Sec. 4.2.2)."""
        _check(lib.conef_error_reset(self.h, _stream_handle(stream)), "conef_error_reset")

    def apply_update(self, x: torch.Tensor, sums: Dict[int, torch.Tensor], stream=None) -> None:
        """x <- x - Delta_t in place (Alg. 2 lines 7-8) from this step's reduced messages."""
        assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
        sv, s1 = sums.get(MSG_VALUES), sums.get(MSG_DENSE1D)
        _check(lib.conef_apply_update(self.h, x.data_ptr(), sv.data_ptr() if sv is not None and sv.numel() else None,
                                      s1.data_ptr() if s1 is not None and s1.numel() else None,
                                      _stream_handle(stream)), "conef_apply_update")

    def decompress_error(self, worker: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        if out is None:
            out = torch.empty(self.error_elems(), dtype=torch.float32, device=self.device)
        _check(lib.conef_decompress_error(self.h, worker, out.data_ptr(), _stream_handle(stream)),
               "conef_decompress_error")
        return out

    def full_step(self, t: int, grads: Sequence[torch.Tensor], outs: Optional[Dict[int, torch.Tensor]] = None,
                  stream=None) -> Dict[int, torch.Tensor]:
        """The call sequence of one whole step: every phase and every reduce."""
        outs = {} if outs is None else outs
        res = {}
        self.step(t, grads, 0, stream)
        if self.q["kind"] == "lowrank":
            res[MSG_P] = self.reduce_messages(MSG_P, outs.get(MSG_P), stream)
            self.step(t, grads, 1, stream)
            res[MSG_Q] = self.reduce_messages(MSG_Q, outs.get(MSG_Q), stream)
        else:
            res[MSG_VALUES] = self.reduce_messages(MSG_VALUES, outs.get(MSG_VALUES), stream)
        if self.message_elems(MSG_DENSE1D) > 0:
            res[MSG_DENSE1D] = self.reduce_messages(MSG_DENSE1D, outs.get(MSG_DENSE1D), stream)
        return res

    # ---- sizes
    def message_elems(self, which: int) -> int:
        return lib.conef_message_elems(self.h, which)

    def error_elems(self) -> int:
        return lib.conef_error_elems(self.h)

    def state_bytes_per_worker(self) -> int:
        return lib.conef_state_bytes_per_worker(self.h)

    def launch_count(self) -> int:
        return lib.conef_launch_count(self.h)

    def set_total_workers(self, total: int) -> None:
        """The N of the means when messages are all-reduced across processes (see multirank.ShardedConEF)."""
        _check(lib.conef_set_total_workers(self.h, int(total)), "conef_set_total_workers")

    def set_fast_path(self, enable: bool) -> None:
        _check(lib.conef_set_fast_path(self.h, int(enable)), "conef_set_fast_path")

    def set_fused(self, enable: bool, tile_periods: int = 0, ctas_per_sm: int = 0) -> None:
        """Low-rank phase 1 in one persistent kernel (default on); tile_periods = 0: default tile
        length; ctas_per_sm 0 (default) or 2..4."""
        _check(lib.conef_set_fused(self.h, int(enable), int(tile_periods), int(ctas_per_sm)), "conef_set_fused")

    def fused_info(self) -> Dict[str, int]:
        v = [C.c_int() for _ in range(5)]
        _check(lib.conef_fused_info(self.h, *[C.byref(x) for x in v]), "conef_fused_info")
        return dict(zip(("active", "ctas", "tile_periods", "ring", "tasks"), (x.value for x in v)))

    def fused_q(self, tensor: int, worker: int) -> torch.Tensor:
        """The Q_i the fused kernel computed during a phase-4 call (tests)."""
        p = C.c_void_p()
        _check(lib.conef_get_fused_q(self.h, tensor, worker, C.byref(p)), "conef_get_fused_q")
        n, m, _ = self.tensors[tensor]
        rr = min(int(self.q.get("rank", 0)), n, m)
        return self._view(p.value, m * rr * 4, torch.float32).view(m, rr)

    def last_status(self, stream=None) -> int:
        st = C.c_int()
        rc = lib.conef_last_status(self.h, _stream_handle(stream), C.byref(st))
        if rc not in (OK, ERR_DEVICE_STATUS):
            _check(rc, "conef_last_status")
        return st.value

    # ---- views into the workspace (inspection)
    def _view(self, ptr: int, nbytes: int, dtype) -> torch.Tensor:
        off = ptr - self.workspace.data_ptr()
        assert 0 <= off and off + nbytes <= self.workspace.numel()
        return self.workspace[off:off + nbytes].view(dtype)

    def message(self, which: int, worker: int) -> torch.Tensor:
        p = C.c_void_p()
        _check(lib.conef_get_message(self.h, which, worker, C.byref(p)), "conef_get_message")
        n = self.message_elems(which)
        return self._view(p.value, n * 4, torch.float32) if n else torch.empty(0, device=self.device)

    def state(self, worker: int, tensor: int, second: bool = False):
        """Views of the stored error of (worker, tensor); second=True: the state q of iConEF-v1."""
        a, b = C.c_void_p(), C.c_void_p()
        na, nb = C.c_size_t(), C.c_size_t()
        fn = lib.conef_get_state2 if second else lib.conef_get_state
        _check(fn(self.h, worker, tensor, C.byref(a), C.byref(na), C.byref(b), C.byref(nb)),
               "conef_get_state2" if second else "conef_get_state")
        ta = self._view(a.value, na.value, torch.uint8)
        tb = self._view(b.value, nb.value, torch.uint8) if b.value else None
        return ta, tb

    def error_step(self) -> int:
        """iConEF-v2: the step whose second draw of Q stored the current e~ (-1: none yet)."""
        return int(lib.conef_get_error_step(self.h))

    def set_error_step(self, step: int) -> None:
        _check(lib.conef_set_error_step(self.h, int(step)), "conef_set_error_step")

    def indices(self, tensor: int) -> torch.Tensor:
        p, k = C.c_void_p(), C.c_int64()
        _check(lib.conef_get_indices(self.h, tensor, C.byref(p), C.byref(k)), "conef_get_indices")
        return self._view(p.value, k.value * 4, torch.int32)

    # -- checkpoints: everything that carries over from one step to the next
    def _compressed(self):
        return [l for l, (r, c, k) in enumerate(self.tensors) if k and c > 1]

    def state_dict(self) -> Dict[str, torch.Tensor]:
        """Host copies of the workers' compressed errors (both states with iConEF) and, for the
        low-rank compressor, of the warm start Q_t.  Messages and scratch are not part of it."""
        out = {}
        for l in self._compressed():
            for i in range(self.n_workers):
                for second in ((False, True) if self.c.get("iconef", 0) else (False,)):
                    a, b = self.state(i, l, second)
                    tag = f"w{i}.t{l}" + (".q" if second else "")
                    out[tag + ".a"] = a.cpu().clone()
                    if b is not None:
                        out[tag + ".b"] = b.cpu().clone()
            if self.q["kind"] == "lowrank":
                out[f"t{l}.q_prev"] = self.factors(l, 0)["q_prev"].cpu().clone()
        if self.c.get("iconef", 0) == 2:
            out["error_step"] = torch.tensor(self.error_step(), dtype=torch.int64)
        return out

    def load_state_dict(self, sd: Dict[str, torch.Tensor]) -> None:
        """Restore what state_dict saved into a context of the same configuration (between steps)."""
        for l in self._compressed():
            for i in range(self.n_workers):
                for second in ((False, True) if self.c.get("iconef", 0) else (False,)):
                    a, b = self.state(i, l, second)
                    tag = f"w{i}.t{l}" + (".q" if second else "")
                    a.copy_(sd[tag + ".a"].to(a.device))
                    if b is not None:
                        b.copy_(sd[tag + ".b"].to(b.device))
            if self.q["kind"] == "lowrank":
                self.factors(l, 0)["q_prev"].copy_(sd[f"t{l}.q_prev"].to(self.device))
        if self.c.get("iconef", 0) == 2:
            self.set_error_step(int(sd["error_step"]))

    def factors(self, tensor: int, worker: int = 0):
        ph, qp, qi, pi = C.c_void_p(), C.c_void_p(), C.c_void_p(), C.c_void_p()
        r = C.c_int()
        _check(lib.conef_get_factors(self.h, tensor, worker, C.byref(ph), C.byref(qp), C.byref(qi),
                                     C.byref(pi), C.byref(r)), "conef_get_factors")
        n, m, _ = self.tensors[tensor]
        rr = r.value
        f32 = torch.float32
        return dict(rank=rr,
                    p_hat=self._view(ph.value, n * rr * 4, f32).view(n, rr),
                    q_prev=self._view(qp.value, m * rr * 4, f32).view(m, rr),
                    q_i=self._view(qi.value, m * rr * 4, f32).view(m, rr),
                    p_i=self._view(pi.value, n * rr * 4, f32).view(n, rr))
