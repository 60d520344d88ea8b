"""Seeded synthetic inputs for pattern-pruned 3x3 convolution layers.

This module only *draws data*: tensors, pattern ids and the pattern library
that callers hand to a convolution.  It holds none of the convolution's own
arithmetic, so the CPU oracle and the CUDA path can both be fed from it while
sharing no code with each other.  It needs numpy only.

Every element is a pure function of (seed, tensor tag, layer index, element
index): a counter-based scheme, so a tensor can be regenerated anywhere, in any
order, and a sub-range costs only that sub-range.

The paper (Sec. 2.1, "Pattern-Based Pruning") shows its pattern shapes only in
a figure; the shapes below are this repository's own, defined by rule.  Taps
are numbered row-major, t = 3*dy + dx, so tap 4 is the centre and bit t of a
mask marks tap t as kept.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

BASE_SEED = 20620

# --- the repository's pattern library (12 shapes, each keeps 4 of 9 taps) ---
# four 2x2 blocks that contain the centre
_BLOCKS = [(0, 1, 3, 4), (1, 2, 4, 5), (3, 4, 6, 7), (4, 5, 7, 8)]
# four "T" shapes: the centre and three of its four edge neighbours
_TEES = [(1, 3, 4, 5), (1, 3, 4, 7), (1, 4, 5, 7), (3, 4, 5, 7)]
# four "edge row / column plus centre"
_EDGES = [(0, 1, 2, 4), (4, 6, 7, 8), (0, 3, 4, 6), (2, 4, 5, 8)]


def _mask(taps) -> int:
    m = 0
    for t in taps:
        m |= 1 << t
    return m


PATTERN_LIBRARY_12 = np.array(
    [_mask(t) for t in _BLOCKS + _TEES + _EDGES], dtype=np.uint16
)


def pattern_library(size: int) -> np.ndarray:
    """First `size` masks of the 12-shape library (sizes 4, 8 and 12 are the
    ones the workloads use; any 1..12 is allowed)."""
    if not 1 <= size <= 12:
        raise ValueError("library size must be in 1..12")
    return PATTERN_LIBRARY_12[:size].copy()


# --- counter-based random numbers -------------------------------------------
_TAGS = {"W": 1, "PID": 2, "CONN": 3, "B": 4, "X": 5, "AUX": 6}
_M64 = (1 << 64) - 1


def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser (Steele, Lea, Flood 2014) applied elementwise."""
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(30)
    z *= np.uint64(0xBF58476D1CE4E5B9)
    z ^= z >> np.uint64(27)
    z *= np.uint64(0x94D049BB133111EB)
    z ^= z >> np.uint64(31)
    return z


def _stream_key(seed: int, tag: str, layer: int, sub: int = 0) -> int:
    k = (seed * 0x9E3779B97F4A7C15) & _M64
    k ^= (_TAGS[tag] * 0xD1B54A32D192ED03) & _M64
    k ^= ((layer + 1) * 0x8CB92BA72F3D8DD7) & _M64
    k ^= ((sub + 1) * 0xDB4F0B9175AE2165) & _M64
    return k


def raw_u64(seed: int, tag: str, layer: int, n: int, sub: int = 0, start: int = 0) -> np.ndarray:
    """n 64-bit words; word i depends only on (seed, tag, layer, sub, start+i)."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + n, dtype=np.uint64)
        key = np.uint64(_stream_key(seed, tag, layer, sub))
        return _mix64(_mix64(idx * np.uint64(0x9E3779B97F4A7C15) + key) ^ key)


def uniform01(seed, tag, layer, n, sub=0, start=0) -> np.ndarray:
    """float64 uniform on [0, 1) with 53 random bits."""
    return (raw_u64(seed, tag, layer, n, sub, start) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normal(seed, tag, layer, n, sub=0, start=0) -> np.ndarray:
    """float64 standard normal by Box-Muller on two independent streams."""
    u1 = 1.0 - uniform01(seed, tag, layer, n, 2 * sub + 10, start)  # (0, 1]
    u2 = uniform01(seed, tag, layer, n, 2 * sub + 11, start)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)


def integers(seed, tag, layer, n, lo, hi, sub=0, start=0) -> np.ndarray:
    """int64 uniform on [lo, hi] inclusive (multiply-shift on the top 32 bits;
    the bias of at most (hi-lo+1)/2^32 is irrelevant for test data)."""
    span = hi - lo + 1
    top = raw_u64(seed, tag, layer, n, sub, start) >> np.uint64(32)
    return ((top * np.uint64(span)) >> np.uint64(32)).astype(np.int64) + lo


# --- one layer's problem -----------------------------------------------------
@dataclasses.dataclass
class LayerSpec:
    """Shape and pruning recipe of one pattern-pruned 3x3 convolution layer."""
    name: str
    n: int
    c_in: int
    c_out: int
    h: int
    w: int
    stride: int = 1
    dtype: str = "f32"            # "f32" | "f16" | "i8"
    prune: float = 0.5            # connectivity-pruning rate (whole kernels removed)
    lib_size: int = 8
    w_dist: str = "he"            # "he" -> N(0, sqrt(2/(9*c_in))); float -> N(0, that sigma)
    x_dist: str = "u01"           # "u01" | "upm1" | "relu_normal"
    bias_sigma: float = 0.01
    relu: bool = True
    index: int = 0                # layer index mixed into every stream

    @property
    def ho(self) -> int:
        return (self.h + 2 - 3) // self.stride + 1

    @property
    def wo(self) -> int:
        return (self.w + 2 - 3) // self.stride + 1

    @property
    def k_surv(self) -> int:
        return self.c_in * self.c_out - int(round(self.prune * self.c_in * self.c_out))

    def useful_macs(self) -> int:
        return 4 * self.k_surv * self.n * self.ho * self.wo

    def dense_macs(self) -> int:
        return 9 * self.c_in * self.c_out * self.n * self.ho * self.wo

    def elem_bytes(self):
        """(activation-in, weight, activation-out) bytes per element."""
        return {"f32": (4, 4, 4), "f16": (2, 2, 2), "i8": (1, 1, 4)}[self.dtype]

    def compulsory_bytes(self) -> int:
        bx, bw, by = self.elem_bytes()
        return (self.n * self.h * self.w * self.c_in * bx
                + self.n * self.ho * self.wo * self.c_out * by
                + self.k_surv * (4 * bw + 2) + 4 * self.c_out)


@dataclasses.dataclass
class LayerData:
    spec: LayerSpec
    masks: np.ndarray     # uint16 [P]
    pid: np.ndarray       # int16  [c_out, c_in], -1 = kernel removed
    w: np.ndarray         # [c_out, c_in, 3, 3] float32 | float16 | int8 (dense, unmasked)
    bias: np.ndarray      # [c_out] float32 (f32, f16) | int32 (i8)
    x: np.ndarray         # [n, h, w, c_in] float32 | float16 | uint8


def make_pattern_ids(seed: int, layer: int, c_out: int, c_in: int, lib_size: int, prune: float) -> np.ndarray:
    """Pattern id per kernel, uniform over the library; exactly
    round(prune*c_in*c_out) kernels, chosen by ranking one random key per
    kernel, are removed (id -1)."""
    nk = c_out * c_in
    pid = integers(seed, "PID", layer, nk, 0, lib_size - 1).astype(np.int16)
    n_pruned = int(round(prune * nk))
    if n_pruned > 0:
        keys = raw_u64(seed, "CONN", layer, nk)
        order = np.argsort(keys, kind="stable")
        pid[order[:n_pruned]] = -1
    return pid.reshape(c_out, c_in)


def make_layer(spec: LayerSpec, seed: int = BASE_SEED, n_override: int | None = None) -> LayerData:
    """Draw every tensor of one layer.  `n_override` draws only the first
    images of the batch (same values as the full batch's leading images)."""
    L = spec.index
    n = spec.n if n_override is None else n_override
    masks = pattern_library(spec.lib_size)
    pid = make_pattern_ids(seed, L, spec.c_out, spec.c_in, spec.lib_size, spec.prune)
    nw = spec.c_out * spec.c_in * 9
    nx = n * spec.h * spec.w * spec.c_in
    if spec.dtype == "i8":
        w = integers(seed, "W", L, nw, -127, 127).astype(np.int8)
        x = integers(seed, "X", L, nx, 0, 255).astype(np.uint8)
        bias = integers(seed, "B", L, spec.c_out, -(1 << 20), 1 << 20).astype(np.int32)
    else:
        sigma = math.sqrt(2.0 / (9.0 * spec.c_in)) if spec.w_dist == "he" else float(spec.w_dist)
        w64 = normal(seed, "W", L, nw) * sigma
        if spec.x_dist == "u01":
            x64 = uniform01(seed, "X", L, nx)
        elif spec.x_dist == "upm1":
            x64 = 2.0 * uniform01(seed, "X", L, nx) - 1.0
        elif spec.x_dist == "relu_normal":
            x64 = np.maximum(normal(seed, "X", L, nx), 0.0)
        else:
            raise ValueError(spec.x_dist)
        ft = np.float32 if spec.dtype == "f32" else np.float16
        w = w64.astype(ft)
        x = x64.astype(ft)
        bias = (normal(seed, "B", L, spec.c_out) * spec.bias_sigma).astype(np.float32)
    return LayerData(
        spec=spec, masks=masks, pid=pid,
        w=w.reshape(spec.c_out, spec.c_in, 3, 3),
        bias=bias,
        x=x.reshape(n, spec.h, spec.w, spec.c_in),
    )


# --- the named workloads -----------------------------------------------------
def config_single_layer() -> list[LayerSpec]:
    """One small fp32 layer: 16 -> 32 channels at 32x32, half the kernels removed."""
    return [LayerSpec("single", 1, 16, 32, 32, 32, 1, "f32", 0.5, 8, 0.1, "upm1", 0.01, True, 0)]


def config_vgg16(batch: int = 1) -> list[LayerSpec]:
    """The thirteen 3x3 layers of VGG-16, fp32; 70 % of kernels removed except
    in the first layer."""
    shapes = [(3, 64, 224), (64, 64, 224), (64, 128, 112), (128, 128, 112),
              (128, 256, 56), (256, 256, 56), (256, 256, 56),
              (256, 512, 28), (512, 512, 28), (512, 512, 28),
              (512, 512, 14), (512, 512, 14), (512, 512, 14)]
    return [LayerSpec(f"conv{i + 1}", batch, ci, co, hw, hw, 1, "f32",
                      0.0 if i == 0 else 0.7, 8, "he", "u01", 0.01, True, i)
            for i, (ci, co, hw) in enumerate(shapes)]


def _resnet_3x3(blocks, batch, dtype, prune, x_dist) -> list[LayerSpec]:
    out, i = [], 0
    for (ci, co, hw, stride, reps) in blocks:
        for _ in range(reps):
            out.append(LayerSpec(f"l{i + 1}_{ci}to{co}_{hw}s{stride}", batch, ci, co, hw, hw,
                                 stride, dtype, prune, 8, "he", x_dist, 0.01, True, i))
            i += 1
    return out


def config_resnet50(batch: int = 32) -> list[LayerSpec]:
    """The sixteen 3x3 layers of ResNet-50 (one per bottleneck), fp16 storage."""
    blocks = [(64, 64, 56, 1, 3), (128, 128, 56, 2, 1), (128, 128, 28, 1, 3),
              (256, 256, 28, 2, 1), (256, 256, 14, 1, 5), (512, 512, 14, 2, 1),
              (512, 512, 7, 1, 2)]
    return _resnet_3x3(blocks, batch, "f16", 0.6, "relu_normal")


def config_resnet18(batch: int = 64) -> list[LayerSpec]:
    """The sixteen 3x3 layers of ResNet-18 after the stem, int8."""
    blocks = [(64, 64, 56, 1, 4), (64, 128, 56, 2, 1), (128, 128, 28, 1, 3),
              (128, 256, 28, 2, 1), (256, 256, 14, 1, 3), (256, 512, 14, 2, 1),
              (512, 512, 7, 1, 3)]
    return _resnet_3x3(blocks, batch, "i8", 0.5, "u01")


def config_sweep() -> list[LayerSpec]:
    """256 -> 256 channels at 28x28, fp16 storage: batch x pruning rate x library size."""
    out, i = [], 0
    for lib in (4, 8, 12):
        for p in (0.0, 0.5, 0.75, 0.875):
            for n in (1, 8, 64, 256):
                out.append(LayerSpec(f"sweep_n{n}_p{p}_lib{lib}", n, 256, 256, 28, 28, 1, "f16",
                                     p, lib, 0.1, "upm1", 0.01, True, i))
                i += 1
    return out


CONFIGS = {
    "single": config_single_layer,
    "vgg16": config_vgg16,
    "resnet50": config_resnet50,
    "resnet18": config_resnet18,
    "sweep": config_sweep,
}


# --- block-pruned matrix products (fully connected layers, 1x1 convolutions) ---
@dataclasses.dataclass
class GemmSpec:
    """Shape and pruning recipe of one block-pruned matrix product
    y[m, c_out] = x[m, k] . W[c_out, k]^T: W is cut into blocks of br rows x bc
    columns, and every block keeps round(row_keep * rows) of its rows and
    round(col_keep * columns) of its columns."""
    name: str
    m: int                        # rows of x: pixels of an NHWC tensor (n*h*w) or tokens
    k: int                        # input features
    c_out: int
    br: int = 32
    bc: int = 32
    row_keep: float = 0.5
    col_keep: float = 0.5
    dtype: str = "f32"            # "f32" | "f16"
    x_dist: str = "relu_normal"
    bias_sigma: float = 0.01
    relu: bool = True
    index: int = 0

    @property
    def nbr(self) -> int:
        return (self.c_out + self.br - 1) // self.br

    @property
    def nbc(self) -> int:
        return (self.k + self.bc - 1) // self.bc

    def elem_bytes(self):
        return {"f32": (4, 4, 4), "f16": (2, 2, 2)}[self.dtype]


@dataclasses.dataclass
class GemmData:
    spec: GemmSpec
    w: np.ndarray          # [c_out, k] float32 | float16 (dense, unmasked)
    row_keep: np.ndarray   # uint8 [nbr, nbc, br]
    col_keep: np.ndarray   # uint8 [nbr, nbc, bc]
    bias: np.ndarray       # [c_out] float32
    x: np.ndarray          # [m, k] float32 | float16

    def kept_weights(self) -> int:
        """Weights that survive (edge blocks count only the rows and columns that exist)."""
        s = self.spec
        total = 0
        for i in range(s.nbr):
            rows = min(s.br, s.c_out - i * s.br)
            for j in range(s.nbc):
                cols = min(s.bc, s.k - j * s.bc)
                total += int(self.row_keep[i, j, :rows].sum()) * int(self.col_keep[i, j, :cols].sum())
        return total

    def useful_macs(self) -> int:
        return self.kept_weights() * self.spec.m

    def dense_macs(self) -> int:
        return self.spec.m * self.spec.k * self.spec.c_out

    def compulsory_bytes(self) -> int:
        bx, bw, by = self.spec.elem_bytes()
        s = self.spec
        return s.m * s.k * bx + s.m * s.c_out * by + self.kept_weights() * bw + 4 * s.c_out


def _keep_exact(keys: np.ndarray, count: int) -> np.ndarray:
    """uint8 flags keeping the `count` entries with the smallest keys."""
    flags = np.zeros(len(keys), dtype=np.uint8)
    flags[np.argsort(keys, kind="stable")[:count]] = 1
    return flags


def make_block_gemm(spec: GemmSpec, seed: int = BASE_SEED, m_override: int | None = None) -> GemmData:
    """Draw every tensor of one block-pruned matrix product.  `m_override` draws
    only the first rows of x (same values as the full tensor's leading rows)."""
    L = 1000 + spec.index                         # streams apart from the convolution layers'
    m = spec.m if m_override is None else m_override
    ft = np.float32 if spec.dtype == "f32" else np.float16
    sigma = math.sqrt(2.0 / max(1.0, spec.k * spec.col_keep))
    w = (normal(seed, "W", L, spec.c_out * spec.k) * sigma).astype(ft).reshape(spec.c_out, spec.k)
    if spec.x_dist == "relu_normal":
        x64 = np.maximum(normal(seed, "X", L, m * spec.k), 0.0)
    elif spec.x_dist == "upm1":
        x64 = 2.0 * uniform01(seed, "X", L, m * spec.k) - 1.0
    else:
        x64 = uniform01(seed, "X", L, m * spec.k)
    x = x64.astype(ft).reshape(m, spec.k)
    bias = (normal(seed, "B", L, spec.c_out) * spec.bias_sigma).astype(np.float32)
    nbr, nbc = spec.nbr, spec.nbc
    rkeys = raw_u64(seed, "CONN", L, nbr * nbc * spec.br, sub=1).reshape(nbr, nbc, spec.br)
    ckeys = raw_u64(seed, "CONN", L, nbr * nbc * spec.bc, sub=2).reshape(nbr, nbc, spec.bc)
    row_keep = np.zeros((nbr, nbc, spec.br), dtype=np.uint8)
    col_keep = np.zeros((nbr, nbc, spec.bc), dtype=np.uint8)
    for i in range(nbr):
        rows = min(spec.br, spec.c_out - i * spec.br)
        for j in range(nbc):
            cols = min(spec.bc, spec.k - j * spec.bc)
            row_keep[i, j, :rows] = _keep_exact(rkeys[i, j, :rows], int(round(spec.row_keep * rows)))
            col_keep[i, j, :cols] = _keep_exact(ckeys[i, j, :cols], int(round(spec.col_keep * cols)))
    return GemmData(spec=spec, w=w, row_keep=row_keep, col_keep=col_keep, bias=bias, x=x)


def config_resnet50_1x1(batch: int = 32, dtype: str = "f16", row_keep: float = 0.4,
                        col_keep: float = 0.4, br: int = 32, bc: int = 32) -> list[GemmSpec]:
    """The distinct 1x1 convolutions of ResNet-50's bottleneck blocks in matrix form
    (rows of x = batch * pixels), block-pruned to about one sixth of the weights."""
    shapes = [(64, 64, 56), (64, 256, 56), (256, 64, 56), (256, 128, 56), (128, 512, 28),
              (512, 128, 28), (512, 256, 28), (256, 1024, 14), (1024, 256, 14),
              (1024, 512, 14), (512, 2048, 7), (2048, 512, 7)]
    return [GemmSpec(f"pw{i + 1}_{k}to{co}_{hw}", batch * hw * hw, k, co, br, bc, row_keep, col_keep,
                     dtype, "relu_normal", 0.01, True, i)
            for i, (k, co, hw) in enumerate(shapes)]


# --- depthwise pattern-pruned 3x3 layers ---------------------------------------
@dataclasses.dataclass
class DepthwiseSpec:
    """One depthwise 3x3 layer: every channel has one kernel, which keeps the 4 weights
    of a pattern; a fraction `prune` of the channels loses its kernel altogether."""
    name: str
    n: int
    c: int
    h: int
    w: int
    stride: int = 1
    dtype: str = "f32"            # "f32" | "f16"
    prune: float = 0.0
    lib_size: int = 8
    x_dist: str = "relu_normal"
    bias_sigma: float = 0.01
    relu: bool = True
    index: int = 0

    @property
    def ho(self) -> int:
        return (self.h + 2 - 3) // self.stride + 1

    @property
    def wo(self) -> int:
        return (self.w + 2 - 3) // self.stride + 1

    @property
    def k_surv(self) -> int:
        return self.c - int(round(self.prune * self.c))

    def useful_macs(self) -> int:
        return 4 * self.k_surv * self.n * self.ho * self.wo

    def compulsory_bytes(self) -> int:
        b = 4 if self.dtype == "f32" else 2
        return (self.n * self.h * self.w * self.c + self.n * self.ho * self.wo * self.c) * b + self.k_surv * (4 * b + 2) + 4 * self.c


@dataclasses.dataclass
class DepthwiseData:
    spec: DepthwiseSpec
    masks: np.ndarray     # uint16 [P]
    pid: np.ndarray       # int16 [c], -1 = kernel removed
    w: np.ndarray         # [c, 3, 3] (dense, unmasked)
    bias: np.ndarray      # [c] float32
    x: np.ndarray         # [n, h, w, c]


def make_depthwise(spec: DepthwiseSpec, seed: int = BASE_SEED, n_override: int | None = None) -> DepthwiseData:
    L = 2000 + spec.index                         # streams apart from the other layer kinds
    n = spec.n if n_override is None else n_override
    masks = pattern_library(spec.lib_size)
    pid = integers(seed, "PID", L, spec.c, 0, spec.lib_size - 1).astype(np.int16)
    n_pruned = int(round(spec.prune * spec.c))
    if n_pruned:
        pid[np.argsort(raw_u64(seed, "CONN", L, spec.c), kind="stable")[:n_pruned]] = -1
    ft = np.float32 if spec.dtype == "f32" else np.float16
    w = (normal(seed, "W", L, spec.c * 9) * math.sqrt(2.0 / 9.0)).astype(ft).reshape(spec.c, 3, 3)
    nx = n * spec.h * spec.w * spec.c
    if spec.x_dist == "relu_normal":
        x64 = np.maximum(normal(seed, "X", L, nx), 0.0)
    elif spec.x_dist == "upm1":
        x64 = 2.0 * uniform01(seed, "X", L, nx) - 1.0
    else:
        x64 = uniform01(seed, "X", L, nx)
    bias = (normal(seed, "B", L, spec.c) * spec.bias_sigma).astype(np.float32)
    return DepthwiseData(spec, masks, pid, w, bias, x64.astype(ft).reshape(n, spec.h, spec.w, spec.c))


def config_mobilenet_depthwise(batch: int = 32, dtype: str = "f16") -> list[DepthwiseSpec]:
    """The distinct depthwise 3x3 layers of a MobileNet-v1-shaped network (channels x extent, stride)."""
    shapes = [(32, 112, 1), (64, 112, 2), (128, 56, 1), (128, 56, 2), (256, 28, 1), (256, 28, 2),
              (512, 14, 1), (512, 14, 2), (1024, 7, 1)]
    return [DepthwiseSpec(f"dw{i + 1}_{c}_{hw}s{s}", batch, c, hw, hw, s, dtype, 0.0, 8, "relu_normal", 0.01, True, i)
            for i, (c, hw, s) in enumerate(shapes)]
