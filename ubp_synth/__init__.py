"""Seeded synthetic inputs for unaligned block-wise pruned (UBP) layers.

This module only draws random data: masks whose ones form non-overlapping
vertical runs of ``Nb`` output channels inside one input-channel column
(the 1xN block of Section 3.1), dense weights, activations and biases.
It performs none of the method's arithmetic (no packing, no products), so
both the CPU oracle's tests and the CUDA path's tests can take their
inputs from here without sharing any code of the method itself.

Everything is a pure function of the integer seed (numpy PCG64).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

__all__ = [
    "block_budget", "random_block_starts", "mask_from_starts", "random_mask",
    "Layer", "make_layer", "CONFIGS", "MBV1_CHAIN", "config_layers", "selection_weights",
]


def block_budget(M: int, C: int, sparsity_pct: int, Nb: int) -> int:
    """Number of kept blocks m = floor(M*C*(1-p)/Nb) (Section 3.1), with the
    pruning rate given as an integer percentage so the floor is exact."""
    return (M * C * (100 - sparsity_pct)) // (100 * Nb)


def random_block_starts(M: int, C: int, Nb: int, m: int,
                        rng: np.random.Generator,
                        aligned: bool = False) -> List[np.ndarray]:
    """Draw ``m`` block start rows spread over the ``C`` columns.

    Column loads: ``m`` balls thrown uniformly at the columns, a ball that
    lands on a column already holding floor(M/Nb) blocks is thrown again.
    Inside a column holding ``c`` blocks the placement is uniform over all
    non-overlapping placements: draw ``c`` distinct integers q_0<...<q_{c-1}
    from [0, M - c*(Nb-1)) and start block t at q_t + t*(Nb-1).
    With ``aligned`` the starts are instead distinct multiples of ``Nb``
    (the aligned pattern the paper calls ABP).
    Returns one sorted int64 array of start rows per column.
    """
    cap = M // Nb
    if m > cap * C:
        raise ValueError("more blocks requested than fit")
    cnt = np.zeros(C, dtype=np.int64)
    left = m
    while left > 0:
        js = rng.integers(0, C, size=left)
        for j in js:
            if cnt[j] < cap:
                cnt[j] += 1
                left -= 1
    starts = []
    for j in range(C):
        c = int(cnt[j])
        if aligned:
            q = np.sort(rng.choice(cap, size=c, replace=False)).astype(np.int64)
            starts.append(q * Nb)
        else:
            q = np.sort(rng.choice(M - c * (Nb - 1), size=c, replace=False)).astype(np.int64)
            starts.append(q + np.arange(c, dtype=np.int64) * (Nb - 1))
    return starts


def mask_from_starts(M: int, C: int, Nb: int, starts: List[np.ndarray]) -> np.ndarray:
    """0/1 mask [M][C] (uint8) with ones on rows i..i+Nb-1 of column j for
    every start row i listed for column j."""
    mask = np.zeros((M, C), dtype=np.uint8)
    for j, s in enumerate(starts):
        for i in s:
            mask[int(i):int(i) + Nb, j] = 1
    return mask


def random_mask(M: int, C: int, Nb: int, sparsity_pct: int, seed: int,
                aligned: bool = False) -> Tuple[np.ndarray, List[np.ndarray]]:
    rng = np.random.Generator(np.random.PCG64(seed))
    m = block_budget(M, C, sparsity_pct, Nb)
    starts = random_block_starts(M, C, Nb, m, rng, aligned=aligned)
    return mask_from_starts(M, C, Nb, starts), starts


@dataclass
class Layer:
    """One synthetic UBP layer. ``W`` is [M][C][R] (R = taps: 1 or 9),
    ``mask`` is [M][C]; ``X`` is [C][Nc] when the layer was made with an explicit
    column count and [C][B][H][Wd] otherwise (channel-major activations,
    columns n = (b, y, x))."""
    name: str
    M: int
    C: int
    R: int
    Nb: int
    sparsity_pct: int
    m: int
    W: np.ndarray
    mask: np.ndarray
    X: np.ndarray
    bias: Optional[np.ndarray]
    relu: bool
    B: int = 1
    H: int = 1
    Wd: int = 1
    starts: List[np.ndarray] = field(default_factory=list, repr=False)
    stride: int = 1          # convolution stride (the strided workloads only)
    src: Optional[int] = None   # chained workloads: index of the layer whose output this one reads (-1 = the block
                                # input, None = the layer before it)

    @property
    def Nc(self) -> int:
        if self.X.size:
            return int(self.X.size // self.C)
        return self.B * self.H * self.Wd        # made without activations: the conv view's column count

    @property
    def Nc_out(self) -> int:
        """Output columns: Nc, or batch x the strided output plane for a strided layer."""
        if self.stride == 1:
            return self.Nc
        return self.B * ((self.H - 1) // self.stride + 1) * ((self.Wd - 1) // self.stride + 1)

    @property
    def surviving_macs(self) -> int:
        return self.m * self.Nb * self.R * self.Nc_out


def make_layer(name: str, M: int, C: int, Nb: int, sparsity_pct: int, seed: int, *,
               Nc: Optional[int] = None, B: int = 1, H: int = 1, Wd: int = 1,
               R: int = 1, w_dist: str = "normal", w_scale: float = 0.05,
               x_dist: str = "absnormal", bias: bool = True, relu: bool = True,
               aligned: bool = False, make_x: bool = True) -> Layer:
    """Build one seeded layer. ``w_dist``: 'uniform' -> U[-w_scale, w_scale],
    'normal' -> N(0, w_scale). ``x_dist``: 'normal' -> N(0,1),
    'absnormal' -> |N(0,1)| (post-ReLU-like). Bias ~ N(0, 0.1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    m = block_budget(M, C, sparsity_pct, Nb)
    starts = random_block_starts(M, C, Nb, m, rng, aligned=aligned)
    mask = mask_from_starts(M, C, Nb, starts)
    if w_dist == "uniform":
        W = rng.uniform(-w_scale, w_scale, size=(M, C, R)).astype(np.float32)
    else:
        W = (rng.standard_normal(size=(M, C, R), dtype=np.float32) * np.float32(w_scale)).astype(np.float32)
    if Nc is not None:
        xshape = (C, Nc)
    else:
        xshape = (C, B, H, Wd)
    if make_x:
        X = rng.standard_normal(size=xshape, dtype=np.float32)
        if x_dist == "absnormal":
            np.abs(X, out=X)
    else:
        X = np.zeros((C, 0), dtype=np.float32)
    b = (rng.standard_normal(size=(M,), dtype=np.float32) * np.float32(0.1)).astype(np.float32) if bias else None
    return Layer(name, M, C, R, Nb, sparsity_pct, m, W, mask, X, b, relu, B, H, Wd, starts)


# (C_in, C_out, spatial) of the 13 pointwise layers of a MobileNetV1-shaped
# network at 224x224 input.
MBV1_CHAIN = [(32, 64, 112), (64, 128, 56), (128, 128, 56), (128, 256, 28),
              (256, 256, 28), (256, 512, 14)] + [(512, 512, 14)] * 5 + \
             [(512, 1024, 7), (1024, 1024, 7)]

CONFIGS = {
    "fc64": "FC 64x64, 1x4 blocks, 50 % sparsity, X 64x256 ~ N(0,1), bias, no ReLU",
    "mbv1_pw512": "pointwise 512->512 at 14x14, batch 32 (M=K=512, Nc=6272), 1x4, 70 %, bias+ReLU",
    "r50_3x3": "3x3 conv 256->256 at 14x14, batch 64, pad 1, blocks 8x1x3x3, 80 %",
    "sweep": "M=K=2048, Nc=8192; Nb in {2,4,8,16} x sparsity in {50,70,80,90} (and 95: where the sparse kernel takes over)",
    "mbv1_chain": "13 pointwise layers of MobileNetV1, batch 64, 1x4, 80 %, bias+ReLU",
    "r50_bottleneck": "1x1 1024->256, 3x3 256->256, 1x1 256->1024 at 14x14, batch 32, blocks of 4, 80 %, chained",
    "r50_downsample": "downsampling bottleneck 28x28 -> 14x14: 1x1 512->256, 3x3 256->256 stride 2, 1x1 256->1024, and "
                      "the shortcut 1x1 512->1024 stride 2 on the block input; batch 32, blocks of 4, 80 %",
}

# r50_downsample: (output channels, input channels, taps, stride, relu, index of the layer whose output it reads;
# -1 = the block input)
R50_DOWNSAMPLE = [(256, 512, 1, 1, True, -1), (256, 256, 9, 2, True, 0), (1024, 256, 1, 1, False, 1),
                  (1024, 512, 1, 2, False, -1)]


def config_layers(cfg: str, *, batch: Optional[int] = None, Nb: Optional[int] = None,
                  sparsity_pct: Optional[int] = None, index: int = 0,
                  make_x: bool = True) -> List[Layer]:
    """Layers of one named configuration; seed = 1000*config_number + index."""
    if cfg == "fc64":
        return [make_layer("fc64", 64, 64, 4, 50, 1000 + index, Nc=256, w_dist="uniform",
                           w_scale=1.0, x_dist="normal", bias=True, relu=False, make_x=make_x)]
    if cfg == "mbv1_pw512":
        b = 32 if batch is None else batch
        return [make_layer("mbv1_pw512", 512, 512, 4, 70, 2000 + index, B=b, H=14, Wd=14,
                           w_scale=0.05, bias=True, relu=True, make_x=make_x)]
    if cfg == "r50_3x3":
        b = 64 if batch is None else batch
        return [make_layer("r50_3x3", 256, 256, 8, 80, 3000 + index, B=b, H=14, Wd=14, R=9,
                           w_scale=0.02, bias=True, relu=True, make_x=make_x)]
    if cfg == "sweep":
        nb = 4 if Nb is None else Nb
        sp = 70 if sparsity_pct is None else sparsity_pct
        # (the 95 % points were added after the 4 x 4 grid: their seeds follow it)
        idx = [2, 4, 8, 16].index(nb) * 4 + [50, 70, 80, 90].index(sp) if sp != 95 else 16 + [2, 4, 8, 16].index(nb)
        return [make_layer(f"sweep_nb{nb}_p{sp}", 2048, 2048, nb, sp, 4000 + idx, Nc=8192,
                           w_scale=0.02, x_dist="normal", bias=False, relu=False, make_x=make_x)]
    if cfg == "mbv1_chain":
        b = 64 if batch is None else batch
        out = []
        for li, (ci, co, hw) in enumerate(MBV1_CHAIN):
            out.append(make_layer(f"mbv1_L{li + 1}", co, ci, 4, 80, 5000 + li, B=b, H=hw, Wd=hw,
                                  w_scale=0.05, bias=True, relu=True, make_x=make_x))
        return out
    if cfg == "r50_bottleneck":
        # a ResNet-50-shaped bottleneck of the 14x14 stage: 1x1 1024->256, 3x3 256->256, 1x1 256->1024;
        # only the first layer's activations are an input, the other two read their predecessor's output
        b = 32 if batch is None else batch
        shapes = [(256, 1024, 1, True), (256, 256, 9, True), (1024, 256, 1, False)]
        return [make_layer(f"r50_bn_{li + 1}", co, ci, 4, 80, 6000 + 10 * index + li, B=b, H=14, Wd=14, R=r,
                           w_scale=0.03, bias=True, relu=relu, make_x=make_x and li == 0)
                for li, (co, ci, r, relu) in enumerate(shapes)]
    if cfg == "r50_downsample":
        b = 32 if batch is None else batch
        out = []
        for li, (co, ci, r, stride, relu, src) in enumerate(R50_DOWNSAMPLE):
            hw = 28 if src == -1 or li == 1 else 14          # spatial size of the tensor the layer READS
            L = make_layer(f"r50_ds_{li + 1}", co, ci, 4, 80, 6500 + 10 * index + li, B=b, H=hw, Wd=hw, R=r, w_scale=0.03,
                           bias=True, relu=relu, make_x=make_x and li == 0)
            L.stride, L.src = stride, src
            out.append(L)
        return out
    raise KeyError(cfg)


def selection_weights(M: int, C: int, R: int, seed: int, kind: str = "trained") -> np.ndarray:
    """Dense weights [M][C][R] for block-selection experiments (stand-ins for
    trained layers, which are not available). ``kind``:
    'trained'  N(0, 0.05) scaled by a log-normal gain per output channel and per
               input channel (sigma 0.5 each), so that important kernels cluster
               along rows and columns the way trained layers do;
    'normal'   plain N(0, 0.05);
    'integer'  integers in [-3, 3]: many equal scores, every sum exact."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if kind == "integer":
        return rng.integers(-3, 4, size=(M, C, R)).astype(np.float32)
    W = rng.standard_normal(size=(M, C, R), dtype=np.float32) * np.float32(0.05)
    if kind == "trained":
        go = np.exp(rng.standard_normal(M) * 0.5).astype(np.float32)
        gc = np.exp(rng.standard_normal(C) * 0.5).astype(np.float32)
        W = W * go[:, None, None] * gc[None, :, None]
    elif kind != "normal":
        raise ValueError(kind)
    return np.ascontiguousarray(W, dtype=np.float32)
