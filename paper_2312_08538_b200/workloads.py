"""Synthetic workloads: parameter-list shapes and seeded gradient generators.

This module holds no arithmetic of the method.  It is the one piece that the
tests hand to both the CUDA library and the CPU oracle, so that both see
bit-identical inputs: every array is drawn once with a seeded
``torch.Generator`` on the requested device and, for the oracle, copied to the
host.

The shapes are architecture hyper-parameters only (ResNet-50, GPT-2 small/XL,
a 6+6-layer "big" translation transformer); they stand in for the training
gradients of the paper's image-classification, language-model and translation
tasks, whose datasets are not needed to time or check one ConEF step.
"""
from __future__ import annotations

import math
from typing import Dict, List, Tuple

import torch

BASE_SEED = 231208538
Tensor3 = Tuple[int, int, int]  # (rows, cols, compress)


# ------------------------------------------------------------------ shape lists

def _t(rows: int, cols: int = 1) -> Tensor3:
    return (rows, cols, 1 if cols > 1 else 0)


def resnet50() -> List[Tensor3]:
    """Conv weights viewed as out x (in*kh*kw); BN weights/biases and the fc bias are 1-D."""
    L: List[Tensor3] = []

    def conv(o, i, k):
        L.append(_t(o, i * k * k))

    def bn(c):
        L.extend([_t(c), _t(c)])

    conv(64, 3, 7)
    bn(64)
    inpl = 64
    for planes, blocks in [(64, 3), (128, 4), (256, 6), (512, 3)]:
        for b in range(blocks):
            conv(planes, inpl, 1); bn(planes)
            conv(planes, planes, 3); bn(planes)
            conv(planes * 4, planes, 1); bn(planes * 4)
            if b == 0:
                conv(planes * 4, inpl, 1); bn(planes * 4)
            inpl = planes * 4
    L.append(_t(1000, 2048))
    L.append(_t(1000))
    return L


def gpt2(n_layer: int, d_model: int, vocab: int = 50257, ctx: int = 1024) -> List[Tensor3]:
    D = d_model
    L: List[Tensor3] = [_t(vocab, D), _t(ctx, D)]
    for _ in range(n_layer):
        L += [_t(D), _t(D), _t(D, 3 * D), _t(3 * D), _t(D, D), _t(D), _t(D), _t(D),
              _t(D, 4 * D), _t(4 * D), _t(4 * D, D), _t(D)]
    L += [_t(D), _t(D)]
    return L


def transformer_big(d: int = 1024, ff: int = 4096, vocab: int = 32768, n_enc: int = 6,
                    n_dec: int = 6) -> List[Tensor3]:
    L: List[Tensor3] = [_t(vocab, d)]

    def attn():
        r = []
        for _ in range(4):
            r += [_t(d, d), _t(d)]
        return r

    def ffn():
        return [_t(ff, d), _t(ff), _t(d, ff), _t(d)]

    def ln():
        return [_t(d), _t(d)]

    for _ in range(n_enc):
        L += attn() + ln() + ffn() + ln()
    for _ in range(n_dec):
        L += attn() + ln() + attn() + ln() + ffn() + ln()
    return L


# ------------------------------------------------------------------ configurations
# q / c are plain dicts so that the CUDA binding and the oracle can each build
# their own configuration objects from them.

def _cfg(idx, tensors, n_workers, q, c, lr, steps, grad):
    return dict(index=idx, tensors=tensors, n_workers=n_workers, q=q, c=c, lr=lr, steps=steps,
                grad=grad)


def config(name: str) -> Dict:
    """The five benchmark configurations and scaled-down variants of each
    (same compressor settings, smaller shapes) that the CPU oracle finishes in
    seconds."""
    randk = dict(kind="randk", k_num=1, k_den=100, seed=BASE_SEED + 13)
    int8 = dict(kind="int8", block=256, scale_dtype="fp32")
    int4 = dict(kind="int4", block=128, scale_dtype="fp16")
    # 5 x floor(d / 10) buckets per tensor, every element hashed over the whole row of the sketch
    # (Sec. 4.2.2): the error compressor of configuration 4.  "-chunksketch" is a DIFFERENT error
    # compressor, not a reading of the same one: the sketch applied to runs of 8192 elements, each
    # run with its own window of the 5 rows (other collision statistics, faster on a GPU)
    flatsketch = dict(kind="countsketch", cs_rows=5, cs_col_div=10, seed=BASE_SEED + 17)
    sketch = dict(flatsketch, cs_chunk=8192)
    # the setting of Sec. 5.4: one sketch row over matrix rows, a tenth of the rows as buckets,
    # partial error feedback with beta = 0.9
    rowsketch = dict(kind="rowsketch", cs_rows=1, cs_col_div=10, seed=BASE_SEED + 17, beta=0.9)

    def lowrank(r):
        return dict(kind="lowrank", rank=r, seed=BASE_SEED + 13)

    if name == "tiny":
        return _cfg(1, [_t(256, 512)], 2, randk, int8, 0.1, 10, "normal1e-2")
    if name == "resnet50":
        return _cfg(2, resnet50(), 4, lowrank(4), int8, 0.1, 20, "layerscaled")
    if name == "gpt2-small":
        return _cfg(3, gpt2(12, 768), 4, lowrank(8), int4, 0.05, 20, "student")
    if name in ("transformer-big", "transformer-big-flatsketch"):
        return _cfg(4, transformer_big(), 8, randk, flatsketch, 0.1, 10, "normal1e-3")
    if name == "gpt2-xl":
        return _cfg(5, gpt2(48, 1600), 8, lowrank(4), int4, 0.05, 5, "student")
    if name == "transformer-big-slice-chunksketch":
        # one encoder and one decoder layer with a small embedding: a case for profiler captures
        return _cfg(4, transformer_big(vocab=4096, n_enc=1, n_dec=1), 8, randk, dict(sketch, cs_chunk=8192), 0.1, 10,
                    "normal1e-3")
    if name.startswith("transformer-big-chunksketch") and not name.endswith("-mini"):
        # "transformer-big-chunksketch-16384" and the like choose another run length
        chunk = int(name.rsplit("-", 1)[1]) if name[-1].isdigit() else 8192
        return _cfg(4, transformer_big(), 8, randk, dict(sketch, cs_chunk=chunk), 0.1, 10, "normal1e-3")
    if name == "transformer-big-stochquant":
        # the unbiased quantiser of Eq. 6 as C, 16 levels (one byte per element here)
        stoch = dict(kind="stochquant", block=256, levels=16, seed=BASE_SEED + 19)
        return _cfg(4, transformer_big(), 8, randk, stoch, 0.1, 10, "normal1e-3")
    if name in ("transformer-big-iconef1", "transformer-big-iconef2"):
        # Alg. 3 on top of the int8 state: version 1 keeps a second int8 state, version 2 the k
        # values of a second random-k draw
        return _cfg(4, transformer_big(), 8, randk, dict(int8, iconef=int(name[-1])), 0.1, 10, "normal1e-3")
    if name == "transformer-big-slice-int8":
        # one encoder and one decoder layer with a small embedding: a case for profiler captures
        return _cfg(4, transformer_big(vocab=4096, n_enc=1, n_dec=1), 8, randk, int8, 0.1, 10, "normal1e-3")
    if name == "transformer-big-int8":
        return _cfg(4, transformer_big(), 8, randk, int8, 0.1, 10, "normal1e-3")
    if name == "transformer-big-int4":
        return _cfg(4, transformer_big(), 8, randk, int4, 0.1, 10, "normal1e-3")
    if name == "transformer-big-rowsketch":
        return _cfg(4, transformer_big(), 8, randk, rowsketch, 0.1, 10, "normal1e-3")
    if name == "gpt2-xl-rowsketch":
        return _cfg(5, gpt2(48, 1600), 8, lowrank(4), rowsketch, 0.05, 5, "student")
    if name == "gpt2-xl-slice-rowsketch":
        return _cfg(5, gpt2(2, 1600, vocab=2048, ctx=1024), 8, lowrank(4), rowsketch, 0.05, 5, "student")
    if name == "transformer-big-rowsketch-mini":
        ts = [_t(512, 1024), _t(128, 1024), _t(1024), _t(64, 4096), _t(4096), _t(1024, 64), _t(33, 77)]
        return _cfg(4, ts, 8, randk, rowsketch, 0.1, 3, "normal1e-3")
    if name == "gpt2-xl-partial":
        # partial error feedback (Alg. 4, beta = 0.9) on the int4 state of configuration 5
        return _cfg(5, gpt2(48, 1600), 8, lowrank(4), dict(int4, beta=0.9), 0.05, 5, "student")
    if name == "gpt2-xl-slice":
        # two transformer blocks of the GPT-2-XL list (about 2 GB of gradients for 8 workers):
        # larger than L2, small enough for a profiler capture
        return _cfg(5, gpt2(2, 1600, vocab=2048, ctx=1024), 8, lowrank(4), int4, 0.05, 5, "student")
    # scaled-down variants: several tiles, ragged tails, blocks that straddle
    # rows, odd shapes, tensors thinner than the rank, 1-D pass-through
    if name == "resnet50-mini":
        ts = [_t(64, 147), _t(64), _t(64), _t(64, 64), _t(64), _t(64, 576), _t(256, 64), _t(256),
              _t(128, 1152), _t(3, 4608), _t(100, 2048), _t(100), _t(37, 3), _t(5, 700)]
        return _cfg(2, ts, 4, lowrank(4), int8, 0.1, 4, "layerscaled")
    if name == "gpt2-small-mini":
        ts = [_t(1031, 768), _t(64, 768), _t(768), _t(768), _t(768, 2304), _t(2304), _t(96, 768),
              _t(768), _t(48, 3072), _t(3072), _t(384, 768), _t(6, 1000), _t(129, 129)]
        return _cfg(3, ts, 4, lowrank(8), int4, 0.05, 4, "student")
    if name in ("transformer-big-mini", "transformer-big-chunksketch-mini"):
        ts = [_t(512, 1024), _t(128, 1024), _t(1024), _t(64, 4096), _t(4096), _t(1024, 64), _t(33, 77)]
        return _cfg(4, ts, 8, randk, sketch if "chunk" in name else flatsketch, 0.1, 3, "normal1e-3")
    if name == "gpt2-xl-mini":
        ts = [_t(257, 1600), _t(32, 1600), _t(1600), _t(80, 4800), _t(4800), _t(64, 1600), _t(1600),
              _t(40, 6400), _t(6400), _t(160, 1600), _t(1600), _t(7, 1601)]
        return _cfg(5, ts, 8, lowrank(4), int4, 0.05, 3, "student")
    raise KeyError(name)


FULL = ["tiny", "resnet50", "gpt2-small", "transformer-big", "gpt2-xl"]
MINI = ["tiny", "resnet50-mini", "gpt2-small-mini", "transformer-big-mini", "gpt2-xl-mini"]


def total_elems(tensors: List[Tensor3]) -> int:
    return sum(r * c for r, c, _ in tensors)


def compressed_elems(tensors: List[Tensor3]) -> int:
    return sum(r * c for r, c, k in tensors if k and c > 1)


# ------------------------------------------------------------------ seeded arrays

def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def layer_scales(cfg: Dict, device="cpu") -> torch.Tensor:
    """Per-tensor gradient scale, log-uniform in [0.1, 10], drawn once per configuration."""
    g = _gen(BASE_SEED + 7, "cpu")
    u = torch.rand(len(cfg["tensors"]), generator=g, dtype=torch.float64)
    return (10.0 ** (2.0 * u - 1.0)).to(torch.float32).to(device)


def gradient(cfg: Dict, worker: int, step: int, device="cpu", chunk: int = 1 << 26) -> torch.Tensor:
    """Flat fp32 gradient of one worker at one step: the concatenation of all
    tensors in table order.  Distribution per configuration:
    normal1e-2 / normal1e-3: N(0, sigma^2); layerscaled: sigma_l * N(0, 1e-6);
    student: 1e-3 * Student-t(3), drawn as Z0 / sqrt((Z1^2+Z2^2+Z3^2)/3); planted: a few
    fixed directions per tensor with a spectral gap, plus small noise."""
    seed = BASE_SEED + 1_000_003 * cfg["index"] + 1_009 * worker + step
    gen = _gen(seed, device)
    total = total_elems(cfg["tensors"])
    out = torch.empty(total, dtype=torch.float32, device=device)
    kind = cfg["grad"]
    if kind == "layerscaled":
        scales = layer_scales(cfg, "cpu").tolist()
        off = 0
        for (r, c, _), s in zip(cfg["tensors"], scales):
            n = r * c
            out[off:off + n] = torch.randn(n, generator=gen, dtype=torch.float32, device=device) * (s * 1e-3)
            off += n
        return out
    if kind == "planted":
        # A spectrum with a gap: per 2-D tensor the same few directions at every worker and step
        # (seeded by the tensor alone), with amplitudes 1, 0.7, 0.5, ... times a per-(worker, step)
        # factor in [0.75, 1.25], entries of size 1e-3, plus noise a hundred times smaller.  The
        # power iteration of a rank-r compressor then has a subspace to converge to.
        off = 0
        for l, (r, c, k) in enumerate(cfg["tensors"]):
            n = r * c
            noise = torch.randn(n, generator=gen, dtype=torch.float32, device=device) * 1e-5
            if k and c > 1:
                gl = _gen(BASE_SEED + 23 + 7919 * l, device)
                nd = min(int(cfg["q"].get("rank", 4)) or 4, r, c)   # as many dominant directions as the compressor keeps
                U = torch.randn(r, nd, generator=gl, dtype=torch.float32, device=device)
                Vt = torch.randn(nd, c, generator=gl, dtype=torch.float32, device=device)
                amp = torch.tensor([0.7 ** j for j in range(nd)], dtype=torch.float32, device=device)
                jit = 0.75 + 0.5 * torch.rand(nd, generator=gen, dtype=torch.float32, device=device)
                sig = (U * (amp * jit * (1e-3 / nd ** 0.5))) @ Vt
                noise = noise + sig.reshape(-1)
            out[off:off + n] = noise
            off += n
        return out
    for lo in range(0, total, chunk):
        n = min(chunk, total - lo)
        z = torch.randn(n, generator=gen, dtype=torch.float32, device=device)
        if kind == "normal1e-2":
            out[lo:lo + n] = z * 1e-2
        elif kind == "normal1e-3":
            out[lo:lo + n] = z * 1e-3
        elif kind == "student":
            chi = torch.zeros(n, dtype=torch.float32, device=device)
            for _ in range(3):
                w = torch.randn(n, generator=gen, dtype=torch.float32, device=device)
                chi += w * w
            out[lo:lo + n] = z / torch.sqrt(chi / 3.0) * 1e-3
        else:
            raise KeyError(kind)
    return out


def q_init(cfg: Dict, device="cpu") -> torch.Tensor:
    """Warm start Q_0 ~ N(0,1) of the low-rank compressor: the concatenation,
    over compressed tensors in table order, of (cols x r_l) row-major blocks
    with r_l = min(rank, rows, cols)."""
    rank = cfg["q"].get("rank", 0)
    n = sum(c * min(rank, r, c) for r, c, k in cfg["tensors"] if k and c > 1)
    gen = _gen(BASE_SEED + 11, device)
    return torch.randn(n, generator=gen, dtype=torch.float32, device=device)


def checksum(x: torch.Tensor) -> int:
    """64-bit sum of the bit patterns, to confirm that two sides saw the same array."""
    v = x.detach().reshape(-1).view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    return int(v.sum().item()) & (2**64 - 1)
