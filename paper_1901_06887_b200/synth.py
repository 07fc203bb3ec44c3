"""Seeded synthetic multi-tenant workloads (numpy only).

This module only *draws inputs*: tenant model descriptions (layer shapes, bf16
weights, fp32 biases), request tags (model ids) and request payloads.  It holds
none of the arithmetic of the inference path itself, so the CPU oracle and the
CUDA library can both be fed from it without sharing any code of the method.

The paper (Sec. 3, "Workers host DNNs for many tenants simultaneously") gives
no dataset for a mixed-tenant batch; the five workloads below stand in for a
worker hosting many tenants with skewed, sporadic demand (Sec. 1.3, Sec. 3.3):
a few heavy tenants and a long tail, drawn from a finite Zipf law.

Conventions
-----------
* bf16 values travel as ``uint16`` bit patterns (numpy has no bf16 dtype).
* Dense weights are ``[out, in]`` row-major; conv weights ``[out, 3, 3, in]``;
  images are NHWC.
* He-uniform weights ``U(-sqrt(6/fan_in), +sqrt(6/fan_in))`` rounded to bf16
  (round-to-nearest-even); biases ``N(0, 0.01**2)`` fp32; payloads ``N(0, 1)``
  rounded to bf16.
* ``P(rank k) ~ k**-s`` over the T tenants (``s = 0`` is uniform); ranks are
  mapped to model ids through a seeded permutation; ids are i.i.d. per request.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

BASE_SEED = 190106887

DENSE = 0
CONV3X3 = 1
GLOBAL_AVG_POOL = 2
CONV1X1 = 3

_PURPOSE = {"widths": 1, "weights": 2, "biases": 3, "ids": 4, "rankperm": 5, "inputs": 6}


def stream(config: int, purpose: str, *extra: int) -> np.random.Generator:
    """Independent Philox stream for (config, purpose, extra...)."""
    ss = np.random.SeedSequence([BASE_SEED, int(config), _PURPOSE[purpose], *map(int, extra)])
    return np.random.Generator(np.random.Philox(ss))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns uint16 bit patterns.

    Inputs are finite here, so NaN handling is not needed.
    """
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Layer:
    kind: int
    in_ch: int
    out_ch: int
    h: int = 0
    w: int = 0
    relu: int = 0
    weight: Optional[np.ndarray] = None  # uint16 bf16 bits; None for pooling
    bias: Optional[np.ndarray] = None    # float32 [out_ch]; None for pooling
    residual: int = 0                    # conv only, 1: the previous layer's input is added before the activation

    @property
    def in_elems(self) -> int:
        return self.in_ch * (self.h * self.w if self.kind != DENSE else 1)

    @property
    def out_elems(self) -> int:
        return self.out_ch * (self.h * self.w if self.kind in (CONV3X3, CONV1X1) else 1)


@dataclass
class Workload:
    name: str
    config: int
    models: List[List[Layer]]
    model_ids: np.ndarray   # int32 [n], arrival order, values index ``models``
    inputs: np.ndarray      # uint16 bf16 bits [n, in_elems]
    zipf_s: float = 0.0
    notes: dict = field(default_factory=dict)

    @property
    def n(self) -> int:
        return int(self.model_ids.shape[0])

    @property
    def in_elems(self) -> int:
        return self.models[0][0].in_elems

    @property
    def out_elems(self) -> int:
        return self.models[0][-1].out_elems


def _he_uniform_bf16(rng: np.random.Generator, shape: Sequence[int], fan_in: int) -> np.ndarray:
    bound = np.float32(np.sqrt(6.0 / fan_in))
    w = rng.random(size=tuple(shape), dtype=np.float32)
    w *= np.float32(2.0) * bound
    w -= bound
    return f32_to_bf16_bits(w)


def _bias(rng: np.random.Generator, n: int) -> np.ndarray:
    return (rng.standard_normal(n, dtype=np.float32) * np.float32(0.01)).astype(np.float32)


def make_mlp(config: int, tenant: int, widths: Sequence[int]) -> List[Layer]:
    """MLP widths[0] -> ... -> widths[-1]; ReLU after every layer but the last."""
    layers = []
    for li in range(len(widths) - 1):
        k, n = int(widths[li]), int(widths[li + 1])
        layers.append(Layer(
            kind=DENSE, in_ch=k, out_ch=n, relu=int(li < len(widths) - 2),
            weight=_he_uniform_bf16(stream(config, "weights", tenant, li), (n, k), k),
            bias=_bias(stream(config, "biases", tenant, li), n)))
    return layers


def make_conv_stack(config: int, tenant: int, n_conv: int, ch: int, h: int, w: int, n_out: int,
                    shortcuts: Sequence[int] = ()) -> List[Layer]:
    """n_conv x (3x3 conv ch->ch, stride 1, pad 1, ReLU) -> global avg pool -> dense ch->n_out.
    shortcuts: indices (>= 1) of conv layers that close a two-layer residual block (identity shortcut)."""
    layers = []
    for li in range(n_conv):
        layers.append(Layer(
            kind=CONV3X3, in_ch=ch, out_ch=ch, h=h, w=w, relu=1, residual=int(li in shortcuts),
            weight=_he_uniform_bf16(stream(config, "weights", tenant, li), (ch, 3, 3, ch), 9 * ch),
            bias=_bias(stream(config, "biases", tenant, li), ch)))
    layers.append(Layer(kind=GLOBAL_AVG_POOL, in_ch=ch, out_ch=ch, h=h, w=w))
    layers.append(Layer(
        kind=DENSE, in_ch=ch, out_ch=n_out, relu=0,
        weight=_he_uniform_bf16(stream(config, "weights", tenant, n_conv + 1), (n_out, ch), ch),
        bias=_bias(stream(config, "biases", tenant, n_conv + 1), n_out)))
    return layers


def make_pointwise_stack(config: int, tenant: int, mid_ch: int, h: int, w: int, n_out: int) -> List[Layer]:
    """conv3x3 64->64 -> conv1x1 64->mid_ch -> conv1x1 mid_ch->64 -> conv3x3 64->64 -> global avg pool -> dense 64->n_out,
    ReLU after every conv: 3x3 layers around a pair of pointwise ones."""
    def conv(li, kind, cin, cout):
        taps = 9 if kind == CONV3X3 else 1
        shape = (cout, 3, 3, cin) if kind == CONV3X3 else (cout, cin)
        return Layer(kind=kind, in_ch=cin, out_ch=cout, h=h, w=w, relu=1,
                     weight=_he_uniform_bf16(stream(config, "weights", tenant, li), shape, taps * cin),
                     bias=_bias(stream(config, "biases", tenant, li), cout))
    layers = [conv(0, CONV3X3, 64, 64), conv(1, CONV1X1, 64, mid_ch), conv(2, CONV1X1, mid_ch, 64), conv(3, CONV3X3, 64, 64)]
    layers.append(Layer(kind=GLOBAL_AVG_POOL, in_ch=64, out_ch=64, h=h, w=w))
    layers.append(Layer(kind=DENSE, in_ch=64, out_ch=n_out, relu=0,
                        weight=_he_uniform_bf16(stream(config, "weights", tenant, 5), (n_out, 64), 64),
                        bias=_bias(stream(config, "biases", tenant, 5), n_out)))
    return layers


def zipf_ids(config: int, n: int, n_tenants: int, s: float, salt: int = 0) -> np.ndarray:
    """i.i.d. model ids with P(rank k) ~ k**-s, ranks shuffled onto ids by a seeded permutation."""
    ranks = np.arange(1, n_tenants + 1, dtype=np.float64)
    p = ranks ** (-float(s))
    p /= p.sum()
    rank_to_id = stream(config, "rankperm", salt).permutation(n_tenants)
    drawn = stream(config, "ids", salt).choice(n_tenants, size=n, p=p)
    return rank_to_id[drawn].astype(np.int32)


def normal_inputs_bf16(config: int, n: int, in_elems: int, salt: int = 0) -> np.ndarray:
    x = stream(config, "inputs", salt).standard_normal((n, in_elems), dtype=np.float32)
    return f32_to_bf16_bits(x)


# --------------------------------------------------------------------------
# The five workloads.  Every size can be overridden to get a reduced case of
# the same shape family (used by parity tests the CPU oracle must finish fast).
# --------------------------------------------------------------------------

CONFIG_NAMES = {
    1: "c1: 4 x MLP 256-256-256-10, 64 req, uniform",
    2: "c2: 64 x MLP 1024-4096-4096-1024, 4096 req, Zipf 1.1",
    3: "c3: 1000 x MLP 512-h1-h2-64 (h in {128,256,512,1024}), 16384 req, Zipf 0.9",
    4: "c4: 16 x (4 conv3x3 64->64 @56x56 + GAP + dense 64->10), 256 req, Zipf 1.0",
    5: "c5: 8 x MLP 4096-16384-4096, 65536 req, uniform",
}

_DEFAULTS = {
    1: dict(n_tenants=4, n=64, widths=(256, 256, 256, 10), s=0.0),
    2: dict(n_tenants=64, n=4096, widths=(1024, 4096, 4096, 1024), s=1.1),
    3: dict(n_tenants=1000, n=16384, widths=(512, None, None, 64), s=0.9,
            hidden_choices=(128, 256, 512, 1024)),
    4: dict(n_tenants=16, n=256, s=1.0, n_conv=4, ch=64, h=56, w=56, n_out=10),
    5: dict(n_tenants=8, n=65536, widths=(4096, 16384, 4096), s=0.0),
}


def make_models(config: int, **over) -> List[List[Layer]]:
    d = dict(_DEFAULTS[config]); d.update(over)
    T = d["n_tenants"]
    if config == 4:
        return [make_conv_stack(config, t, d["n_conv"], d["ch"], d["h"], d["w"], d["n_out"],
                                shortcuts=tuple(d.get("shortcuts", ()))) for t in range(T)]
    models = []
    wrng = stream(config, "widths")
    for t in range(T):
        widths = list(d["widths"])
        for i, wv in enumerate(widths):
            if wv is None:  # heterogeneous hidden width: one independent uniform draw per hidden layer
                widths[i] = int(wrng.choice(d["hidden_choices"]))
        models.append(make_mlp(config, t, widths))
    return models


def make_requests(config: int, models: List[List[Layer]], n: Optional[int] = None,
                  s: Optional[float] = None, salt: int = 0):
    d = _DEFAULTS[config]
    n = d["n"] if n is None else int(n)
    s = d["s"] if s is None else float(s)
    ids = zipf_ids(config, n, len(models), s, salt)
    x = normal_inputs_bf16(config, n, models[0][0].in_elems, salt)
    return ids, x


def make_workload(config: int, n: Optional[int] = None, salt: int = 0, **over) -> Workload:
    """Build workload ``config`` (1..5); keyword overrides shrink it (e.g. n_tenants=3, widths=(64,128,10))."""
    d = dict(_DEFAULTS[config]); d.update(over)
    models = make_models(config, **over)
    ids, x = make_requests(config, models, n=n if n is not None else d["n"], s=d["s"], salt=salt)
    return Workload(name=CONFIG_NAMES[config], config=config, models=models, model_ids=ids, inputs=x,
                    zipf_s=d["s"])


# --------------------------------------------------------------------------
# Closed-form work counts (the paper, Sec. 3.2: the flops of each layer are
# known a priori).  Real rows and features only.
# --------------------------------------------------------------------------

def layer_flops(layer: Layer) -> int:
    if layer.kind == DENSE:
        return 2 * layer.in_ch * layer.out_ch
    if layer.kind == CONV3X3:
        return 2 * 9 * layer.in_ch * layer.out_ch * layer.h * layer.w
    if layer.kind == CONV1X1:
        return 2 * layer.in_ch * layer.out_ch * layer.h * layer.w
    return 0


def workload_flops(models: List[List[Layer]], model_ids: np.ndarray) -> int:
    counts = np.bincount(model_ids, minlength=len(models))
    return int(sum(int(c) * sum(layer_flops(l) for l in m) for c, m in zip(counts, models)))


def workload_bytes(models: List[List[Layer]], model_ids: np.ndarray, per_layer: bool = False):
    """Algorithmic bytes of one pass of the executor: weights+bias of tenants that have at least one
    request, read once; the input read once (bf16); every hidden activation written and read once
    (bf16); the final output written once (fp32).  Bucketing gather / un-permute traffic excluded."""
    counts = np.bincount(model_ids, minlength=len(models))
    n_layers = len(models[0])
    per = [0] * n_layers
    for c, m in zip(counts, models):
        c = int(c)
        if c == 0:
            continue
        for li, l in enumerate(m):
            b = 0
            if l.weight is not None:
                b += l.weight.size * 2 + l.bias.size * 4
            b += c * l.in_elems * 2                                   # read input activation (bf16)
            if getattr(l, "residual", 0):
                b += c * l.out_elems * 2                              # read the block's input once more (identity shortcut)
            b += c * l.out_elems * (4 if li == n_layers - 1 else 2)   # write output
            per[li] += b
    return per if per_layer else int(sum(per))
