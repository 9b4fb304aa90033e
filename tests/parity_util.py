"""Helpers shared by the GPU parity tests: build both sides from one workload
configuration, move state between them, and compare with the stated tolerances.

Tolerances (from the benchmark spec of the target):
  * integer outputs (indices, codes, bucket positions) bit-exact, except that a
    code may differ by +-1 at an exact rounding tie in at most 1e-6 of elements;
  * floating-point outputs within 1e-5 relative, elementwise.  For sums of
    terms of random sign (message sums, sketch buckets, factors) the
    denominator is max(|a|, |b|, rho) with rho the RMS of the reference array:
    a purely elementwise relative error is ill-posed where a sum cancels;
  * low-rank factors within 1e-4 relative in Frobenius norm.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import conef_oracle as orc
from paper_2312_08538_b200 import workloads as wl

REL = 1e-5
FROB = 1e-4
TIE_FRACTION = 1e-6


def make_oracle(cfg, q_init=None):
    q, c = cfg["q"], cfg["c"]
    qc = orc.QCfg(kind=q["kind"], k_num=q.get("k_num", 1), k_den=q.get("k_den", 100),
                  rank=q.get("rank", 0), q_init=q_init, seed=q.get("seed", 0))
    cc = orc.CCfg(kind=c["kind"], block=c.get("block", 256), scale_dtype=c.get("scale_dtype", "fp32"),
                  cs_rows=c.get("cs_rows", 5), cs_col_div=c.get("cs_col_div", 10), seed=c.get("seed", 0),
                  beta=c.get("beta", 0.0), levels=c.get("levels", 16), iconef=c.get("iconef", 0), cs_chunk=c.get("cs_chunk", 0))
    return orc.ConEFOracle(cfg["tensors"], cfg["n_workers"], qc, cc, cfg["lr"])


def make_gpu(cfg, q_init=None, fast=True):
    from paper_2312_08538_b200 import binding
    eng = binding.ConEF(cfg["tensors"], cfg["n_workers"], cfg["q"], cfg["c"], cfg["lr"], q_init=q_init)
    eng.set_fast_path(fast)
    return eng


def grads_both(cfg, t):
    """Per-worker gradients on the device and the same bits on the host."""
    dev = [wl.gradient(cfg, i, t, device="cuda") for i in range(cfg["n_workers"])]
    host = [g.cpu().numpy() for g in dev]
    return dev, host


def rel_err(a: np.ndarray, b: np.ndarray) -> float:
    """max |a-b| / max(|a|, |b|, rms(b)) over the array (b is the reference)."""
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    if a.size == 0:
        return 0.0
    rho = float(np.sqrt(np.mean(b * b)))
    den = np.maximum(np.maximum(np.abs(a), np.abs(b)), max(rho, 1e-300))
    return float(np.max(np.abs(a - b) / den))


def rel_err_large(a: np.ndarray, b: np.ndarray) -> float:
    """Plain elementwise relative error max |a-b| / |b|, over the elements with |b| >= rms(b) only
    (no floor on the denominator: these elements are not the result of a cancellation)."""
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    if a.size == 0:
        return 0.0
    rho = float(np.sqrt(np.mean(b * b)))
    big = np.abs(b) >= max(rho, 1e-300)
    if not big.any():
        return 0.0
    return float(np.max(np.abs(a[big] - b[big]) / np.abs(b[big])))


def frob_err(a: np.ndarray, b: np.ndarray) -> float:
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    nb = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / nb if nb > 0 else float(np.linalg.norm(a))


def unpack_codes(raw: np.ndarray, d: int, bits: int) -> np.ndarray:
    if bits == 8:
        return raw.view(np.int8).astype(np.int32)[:d]
    lo = (raw & 0xF).astype(np.int32)
    hi = (raw >> 4).astype(np.int32)
    both = np.stack([lo, hi], axis=1).reshape(-1)[:d]
    return np.where(both >= 8, both - 16, both)


def gpu_state_arrays(eng, oracle, i, l, second=False):
    """(codes int32[d], scales fp32[nb]) or the raw fp32 state of (worker, tensor)."""
    a, b = eng.state(i, l, second)
    kind = oracle.c.kind
    d = oracle.d_of(l)
    if kind in ("int8", "int4"):
        codes = unpack_codes(a.cpu().numpy(), d, 8 if kind == "int8" else 4)
        if oracle.c.scale_dtype == "fp16":
            scales = b.view(torch.float16).cpu().numpy().astype(np.float32)
        else:
            scales = b.view(torch.float32).cpu().numpy()
        return codes, scales
    if kind == "rowsketch" and oracle.c.scale_dtype == "fp16":
        return a.view(torch.int16).cpu().numpy().view(np.uint16), None
    if kind == "stochquant":
        lv = a.view(torch.int16 if oracle.c.levels > 127 else torch.int8).cpu().numpy().astype(np.int32)[:d]
        return lv, b.view(torch.float32).cpu().numpy()
    return a.view(torch.float32).cpu().numpy(), None


def oracle_state_arrays(oracle, i, l, second=False):
    st = (oracle.state2 if second else oracle.state)[i][l]
    kind = oracle.c.kind
    if kind == "stochquant":
        return st["levels"].astype(np.int32), st["scales"]
    if kind in ("int8", "int4"):
        return unpack_codes(st["codes"], oracle.d_of(l), 8 if kind == "int8" else 4), st["scales"]
    if kind == "rowsketch":
        return (st["T16"] if "T16" in st else st["T"]), None
    return (st["e"] if kind == "identity" else st["S"]), None


def load_state_from_oracle(eng, oracle):
    """Teacher forcing: overwrite the GPU's stored error with the oracle's."""
    for i in range(oracle.N):
        for l in oracle.compressed:
            a, b = eng.state(i, l)
            st = oracle.state[i][l]
            kind = oracle.c.kind
            if kind in ("int8", "int4"):
                a.copy_(torch.from_numpy(st["codes"]).cuda())
                if oracle.c.scale_dtype == "fp16":
                    b.view(torch.int16).copy_(torch.from_numpy(st["scales16"].view(np.int16)).cuda())
                else:
                    b.view(torch.float32).copy_(torch.from_numpy(st["scales"]).cuda())
            elif kind == "identity":
                a.view(torch.float32).copy_(torch.from_numpy(st["e"]).cuda())
            elif kind == "stochquant":
                dt = torch.int16 if oracle.c.levels > 127 else torch.int8
                a.view(dt).copy_(torch.from_numpy(st["levels"].astype(np.int16 if oracle.c.levels > 127 else np.int8)).cuda())
                b.view(torch.float32).copy_(torch.from_numpy(st["scales"]).cuda())
            elif kind == "rowsketch" and "T16" in st:
                a.view(torch.int16).copy_(torch.from_numpy(st["T16"].view(np.int16)).cuda())
            elif kind == "rowsketch":
                a.view(torch.float32).copy_(torch.from_numpy(st["T"]).cuda())
            else:
                a.view(torch.float32).copy_(torch.from_numpy(st["S"]).cuda())


def compare_codes(gc, gs, oc, os_, exact_scales=True):
    """Returns (mismatch fraction, max |delta code|); asserts the scales."""
    if exact_scales:
        assert np.array_equal(gs, os_), "block scales differ"
    diff = np.abs(gc - oc)
    return float(np.count_nonzero(diff)) / max(1, diff.size), int(diff.max()) if diff.size else 0
