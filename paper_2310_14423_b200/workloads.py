"""Seeded synthetic workloads: parameter-set shapes, run configurations and input arrays.

This module holds no arithmetic of the method itself (no optimizer step, no learning-rate
schedule, no round-length rule, no noise generator).  It only describes *what* a run looks
like -- how many replicas, how many parameters, which hyper-parameters -- and draws the two
input vectors of the synthetic loss, so that the CUDA library and the CPU oracle can be fed
the very same numbers without sharing any code of their own.

The synthetic loss stands in for ImageNet training of ResNet-152 / ViT-B (paper, Sec. 4 and
App. C): per replica k the gradient of coordinate i is lambda_i * (theta_i - theta*_i) plus
Gaussian noise, with lambda log-uniform in [1e-3, 1] and theta* standard normal.  The
parameter sets keep the tensor shapes of the two models so that the flattened [K, P] slabs
have the sizes, the tensor count and the ragged tensor boundaries of the paper's workloads.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

# Optimizer / schedule / rule identifiers.  Plain strings here; each side maps them to its own enum.
OPT_SGDM = "sgdm"
OPT_ADAMW = "adamw"
SCHED_COSINE = "cosine"
SCHED_STEP_POW2 = "step_pow2"
SCHED_LINEAR = "linear"
SCHED_CONST = "const"
SCHED_HALVING = "halving"          # peak until t_hold, then halved every t_period steps (App. G)
SCHED_COSINE_HELD = "cosine_held"  # cosine that stops decaying at t_hold (App. G)
RULE_QSR = "qsr"
RULE_CONST_H = "const_h"
RULE_POWER = "power"               # H = max(H_base, floor((alpha/eta)^gamma))
RULE_POST_LOCAL = "post_local"     # H = 1 until t_switch, then H_base
RULE_SWAP = "swap"                 # H_base until t_switch, then a single round to T
STATE_KEEP = "keep"
STATE_AVERAGE = "average"
STATE_RESET = "reset"

NOISE_SEED_BASE = 0x231014423000


@dataclass(frozen=True)
class TensorSpec:
    name: str
    shape: Tuple[int, ...]

    @property
    def numel(self) -> int:
        n = 1
        for d in self.shape:
            n *= d
        return n


@dataclass(frozen=True)
class Layout:
    """Flattened parameter set: tensor t occupies [offset[t], offset[t] + numel[t]) of a row.

    Every tensor starts on a multiple of `pad` elements; the gap elements are ordinary
    coordinates of the slab (they get their own lambda / theta* and are updated like any other).
    """
    names: Tuple[str, ...]
    offset: np.ndarray  # int64 [n_tensors]
    numel: np.ndarray   # int64 [n_tensors]
    P: int              # row length including padding
    P_model: int        # sum of numel (the model's own parameter count)


def resnet152_tensors() -> List[TensorSpec]:
    """Conv / BatchNorm / fc tensors of ResNet-152 (bottleneck stages of 3, 8, 36, 3 blocks)."""
    specs: List[TensorSpec] = []

    def conv(name, cout, cin, k):
        specs.append(TensorSpec(name + ".weight", (cout, cin, k, k)))

    def bn(name, c):
        specs.append(TensorSpec(name + ".weight", (c,)))
        specs.append(TensorSpec(name + ".bias", (c,)))

    conv("conv1", 64, 3, 7)
    bn("bn1", 64)
    inplanes = 64
    for stage, (planes, blocks) in enumerate(zip((64, 128, 256, 512), (3, 8, 36, 3)), start=1):
        for b in range(blocks):
            p = f"layer{stage}.{b}"
            conv(p + ".conv1", planes, inplanes, 1)
            bn(p + ".bn1", planes)
            conv(p + ".conv2", planes, planes, 3)
            bn(p + ".bn2", planes)
            conv(p + ".conv3", planes * 4, planes, 1)
            bn(p + ".bn3", planes * 4)
            if b == 0:
                conv(p + ".downsample.0", planes * 4, inplanes, 1)
                bn(p + ".downsample.1", planes * 4)
            inplanes = planes * 4
    specs.append(TensorSpec("fc.weight", (1000, 2048)))
    specs.append(TensorSpec("fc.bias", (1000,)))
    return specs


def vit_b16_tensors() -> List[TensorSpec]:
    """ViT-B/16 with global average pooling and fixed sin-cos positions (paper, App. C.2):
    no class token and no learned position table, so only the tensors below are trained."""
    d, mlp, classes, patch = 768, 3072, 1000, 16 * 16 * 3
    specs: List[TensorSpec] = [TensorSpec("patch_embed.weight", (d, patch)),
                               TensorSpec("patch_embed.bias", (d,))]
    for b in range(12):
        p = f"blocks.{b}"
        specs += [
            TensorSpec(p + ".norm1.weight", (d,)), TensorSpec(p + ".norm1.bias", (d,)),
            TensorSpec(p + ".attn.qkv.weight", (3 * d, d)), TensorSpec(p + ".attn.qkv.bias", (3 * d,)),
            TensorSpec(p + ".attn.proj.weight", (d, d)), TensorSpec(p + ".attn.proj.bias", (d,)),
            TensorSpec(p + ".norm2.weight", (d,)), TensorSpec(p + ".norm2.bias", (d,)),
            TensorSpec(p + ".mlp.fc1.weight", (mlp, d)), TensorSpec(p + ".mlp.fc1.bias", (mlp,)),
            TensorSpec(p + ".mlp.fc2.weight", (d, mlp)), TensorSpec(p + ".mlp.fc2.bias", (d,)),
        ]
    specs += [TensorSpec("norm.weight", (d,)), TensorSpec("norm.bias", (d,)),
              TensorSpec("head.weight", (classes, d)), TensorSpec("head.bias", (classes,))]
    return specs


def make_layout(specs: Sequence[TensorSpec], pad: int = 4) -> Layout:
    offs, nums = [], []
    cur = 0
    for s in specs:
        cur = (cur + pad - 1) // pad * pad
        offs.append(cur)
        nums.append(s.numel)
        cur += s.numel
    P = (cur + pad - 1) // pad * pad
    return Layout(tuple(s.name for s in specs), np.asarray(offs, np.int64), np.asarray(nums, np.int64),
                  int(P), int(sum(nums)))


def flat_layout(P: int) -> Layout:
    return Layout(("flat",), np.zeros(1, np.int64), np.asarray([P], np.int64), int(P), int(P))


@dataclass(frozen=True)
class Workload:
    """One run configuration.  Field names follow the paper's notation where it has one."""
    name: str
    K: int                      # replicas (workers)
    layout: Layout
    opt: str
    T: int                      # total iterations
    T_warmup: int               # linear warm-up iterations
    eta_max: float              # peak learning rate
    eta_min: float = 0.0
    sched: str = SCHED_COSINE
    rule: str = RULE_QSR
    alpha: float = 0.0          # growth coefficient of the Quadratic Synchronization Rule
    H_base: int = 1             # minimum (or constant) synchronization period
    momentum: float = 0.0
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    noise_std: float = 0.0
    state_sync: str = STATE_KEEP
    data_seed: int = 1          # seed of lambda / theta*
    noise_seed: int = NOISE_SEED_BASE
    worker_offset: int = 0      # global index of this process's first replica (multi-GPU sharding)
    gamma: float = 2.0          # exponent of the power rule
    t_switch: int = 0           # switching step of the post-local and SWAP schedules
    t_hold: int = 0             # halving / held-cosine schedules: last step at the regular value
    t_period: int = 1           # halving schedule: steps between halvings
    clip_norm: float = 0.0      # > 0: per-worker global-norm gradient clipping threshold (App. C.2); 0: off

    @property
    def P(self) -> int:
        return self.layout.P

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _shaped(name: str) -> Layout:
    if name == "resnet152":
        return make_layout(resnet152_tensors())
    if name == "vit_b16":
        return make_layout(vit_b16_tensors())
    raise KeyError(name)


def workload(name: str) -> Workload:
    """The run configurations, by short name.

    c1  K=4,  P=65,536     Local SGD(momentum)  cosine, QSR alpha=0.2 H_base=2, T=2000
    c2  K=8,  P=1,048,576  Local AdamW          warm-up 100 + cosine, QSR alpha=0.0175 H_base=4, T=5000
    c3  K=16, ResNet-152 shapes, Local SGD(momentum, wd 1e-4), peak lr 0.8, T=10,000
    c4  K=16, ViT-B/16 shapes, Local AdamW, peak lr 8e-4, T=10,000
    c4p as c4 with the paper's peak lr 0.008 (App. C.2), so that H_base shapes the schedule
    c5  K=32, ViT-B/16 shapes (sweep base: alpha, H_base and the rule are overridden by the caller)
    """
    if name == "c4u":
        # c4s with eight more parameters: rows of 2^25 + 32 bytes, so that rows packed at P start at unrelated offsets
        # of every power-of-two address unit, as the rows of the full-size shaped sets do.
        return workload("c4").replace(name=name, layout=flat_layout((1 << 23) + 8))
    if name in ("c3s", "c4s", "c4ps"):
        # The same runs on a flat 2^23-parameter set: slabs of 512 MiB, larger than L2 but small enough for
        # profiler captures that replay each launch many times.
        return workload(name[:-1]).replace(name=name, layout=flat_layout(1 << 23))
    if name == "c1":
        return Workload("c1", 4, flat_layout(65536), OPT_SGDM, T=2000, T_warmup=0, eta_max=0.1,
                        alpha=0.2, H_base=2, momentum=0.9, noise_std=0.1,
                        data_seed=1, noise_seed=NOISE_SEED_BASE + 0)
    if name == "c2":
        return Workload("c2", 8, flat_layout(1 << 20), OPT_ADAMW, T=5000, T_warmup=100, eta_max=1e-3,
                        alpha=0.0175, H_base=4, weight_decay=0.05, noise_std=0.05,
                        data_seed=2, noise_seed=NOISE_SEED_BASE + 1)
    if name == "c3":
        return Workload("c3", 16, _shaped("resnet152"), OPT_SGDM, T=10000, T_warmup=0, eta_max=0.8,
                        alpha=0.2, H_base=2, momentum=0.9, weight_decay=1e-4, noise_std=0.1,
                        data_seed=3, noise_seed=NOISE_SEED_BASE + 2)
    if name in ("c4", "c4p", "c5"):
        w = Workload("c4", 16, _shaped("vit_b16"), OPT_ADAMW, T=10000, T_warmup=100, eta_max=8e-4,
                     alpha=0.0175, H_base=4, weight_decay=0.05, noise_std=0.05,
                     data_seed=4, noise_seed=NOISE_SEED_BASE + 3)
        if name == "c4p":
            w = w.replace(name="c4p", eta_max=8e-3)
        if name == "c5":
            w = w.replace(name="c5", K=32, data_seed=5, noise_seed=NOISE_SEED_BASE + 4)
        return w
    raise KeyError(name)


def tiny_workload(opt: str = OPT_SGDM, K: int = 3, P: int = 1000, T: int = 60, **kw) -> Workload:
    """A small ragged case for tests: P not a multiple of the vector width, K not a power of two."""
    base = dict(name="tiny", K=K, layout=flat_layout(P), opt=opt, T=T, T_warmup=0,
                eta_max=0.1 if opt == OPT_SGDM else 1e-2, alpha=0.25 if opt == OPT_SGDM else 0.03,
                H_base=2, momentum=0.9, weight_decay=0.01, noise_std=0.1, data_seed=11,
                noise_seed=NOISE_SEED_BASE + 99)
    base.update(kw)
    return Workload(**base)


def draw_inputs(P: int, data_seed: int, lo: int = 0, hi: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """lambda (log-uniform in [1e-3, 1]) and theta* (standard normal) as fp32 [P], or their slice [lo, hi).

    Drawn in fixed blocks so that a slice of a large parameter set costs only the blocks it touches
    and equals the same slice of the full draw."""
    hi = P if hi is None else hi
    blk = 1 << 20
    lam = np.empty(hi - lo, np.float32)
    ths = np.empty(hi - lo, np.float32)
    for b in range(lo // blk, (max(hi, lo + 1) - 1) // blk + 1):
        b0, b1 = b * blk, min((b + 1) * blk, P)
        rng = np.random.default_rng([data_seed, b])
        lam_b = np.power(10.0, rng.uniform(-3.0, 0.0, b1 - b0)).astype(np.float32)
        ths_b = rng.standard_normal(b1 - b0).astype(np.float32)
        s0, s1 = max(lo, b0), min(hi, b1)
        if s1 > s0:
            lam[s0 - lo:s1 - lo] = lam_b[s0 - b0:s1 - b0]
            ths[s0 - lo:s1 - lo] = ths_b[s0 - b0:s1 - b0]
    return lam, ths


def draw_inputs_at(P: int, data_seed: int, idx: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """lambda / theta* at the given coordinates only (same values as draw_inputs(P, seed)[idx])."""
    idx = np.asarray(idx, np.int64)
    lam = np.empty(idx.size, np.float32)
    ths = np.empty(idx.size, np.float32)
    blk = 1 << 20
    blocks = idx // blk
    for b in np.unique(blocks):
        sel = np.nonzero(blocks == b)[0]
        b0, b1 = int(b) * blk, min((int(b) + 1) * blk, P)
        l, s = draw_inputs(P, data_seed, b0, b1)
        lam[sel] = l[idx[sel] - b0]
        ths[sel] = s[idx[sel] - b0]
    return lam, ths


def coordinate_subset(layout: Layout, n: int, seed: int = 0) -> np.ndarray:
    """A sorted subset of about n coordinates of a row: the first and last element of every tensor,
    their neighbours across the padding, the row's first and last elements, and seeded random fill."""
    P = layout.P
    must = [np.asarray([0, 1, 2, 3, P - 4, P - 3, P - 2, P - 1], np.int64)]
    ends = layout.offset + layout.numel - 1
    for d in (-1, 0, 1):
        must.append(layout.offset + d)
        must.append(ends + d)
    must = np.unique(np.clip(np.concatenate(must), 0, P - 1))
    if must.size > n:
        rng = np.random.default_rng([seed, 1])
        keep = np.sort(rng.choice(must.size, n, replace=False))
        return must[keep]
    rng = np.random.default_rng([seed, 2])
    extra = rng.integers(0, P, size=max(0, n - must.size), dtype=np.int64)
    return np.unique(np.concatenate([must, extra]))
