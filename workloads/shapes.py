"""Problem shapes of the workloads: square sweeps, non-squarish shapes and im2row-lowered
convolution layers.

The im2row shapes are derived from convolution-layer descriptors (C_in, C_out, kernel, output
size): lowering a layer gives a GEMM with one row per output pixel, one column per output
channel and k = C_in*kh*kw.  At batch 1 the descriptors below give the GEMM dimensions of the
paper's Table "resnet50" (ResNet50 v1.5) and Table "vgg16"; tests check that against the
table rows stored under tests/golden/.
"""
from __future__ import annotations

from dataclasses import dataclass, field

from .generators import DTYPE_F32, DTYPE_F16, DTYPE_BF16, Matrix, make_matrix


@dataclass(frozen=True)
class ConvLayer:
    cin: int
    cout: int
    ksize: int     # square kernel
    out_hw: int    # output height == width for a 224x224 input

    def im2row_mnk(self, batch: int = 1) -> tuple[int, int, int]:
        """(m, n, k) in the paper's orientation: m = batch*Ho*Wo, n = C_out, k = C_in*kh*kw."""
        return (batch * self.out_hw * self.out_hw, self.cout, self.cin * self.ksize * self.ksize)


# the 20 distinct convolution shapes of ResNet50 v1.5, in the order of Table "resnet50"
RESNET50_V15_BATCH1 = (
    ConvLayer(3, 64, 7, 112),
    ConvLayer(64, 64, 1, 56),
    ConvLayer(64, 64, 3, 56),
    ConvLayer(64, 256, 1, 56),
    ConvLayer(256, 64, 1, 56),
    ConvLayer(256, 128, 1, 56),
    ConvLayer(128, 128, 3, 28),
    ConvLayer(128, 512, 1, 28),
    ConvLayer(256, 512, 1, 28),
    ConvLayer(512, 128, 1, 28),
    ConvLayer(512, 256, 1, 28),
    ConvLayer(256, 256, 3, 14),
    ConvLayer(256, 1024, 1, 14),
    ConvLayer(512, 1024, 1, 14),
    ConvLayer(1024, 256, 1, 14),
    ConvLayer(1024, 512, 1, 14),
    ConvLayer(512, 512, 3, 7),
    ConvLayer(512, 2048, 1, 7),
    ConvLayer(1024, 2048, 1, 7),
    ConvLayer(2048, 512, 1, 7),
)

# the 9 distinct shapes of Table "vgg16"; row 7 is kept as the table prints it (n = 256)
VGG16_BATCH1 = (
    ConvLayer(3, 64, 3, 224),
    ConvLayer(64, 64, 3, 224),
    ConvLayer(64, 128, 3, 112),
    ConvLayer(128, 128, 3, 112),
    ConvLayer(128, 256, 3, 56),
    ConvLayer(256, 256, 3, 56),
    ConvLayer(256, 256, 3, 28),
    ConvLayer(512, 512, 3, 28),
    ConvLayer(512, 512, 3, 14),
)


def im2row_shapes(layers=RESNET50_V15_BATCH1, batch: int = 32, weights_as_A: bool = True):
    """GEMM dimensions of the lowered layers.

    weights_as_A=True gives C[C_out x batch*Ho*Wo] = W[C_out x k] * X[k x batch*Ho*Wo]
    (weights are operand A, activations operand B): the paper's problem transposed.
    weights_as_A=False keeps the paper's orientation (m = pixels, n = channels).
    """
    out = []
    for L in layers:
        m, n, k = L.im2row_mnk(batch)
        out.append((n, m, k) if weights_as_A else (m, n, k))
    return out


def square_fp32_sweep():
    return [(s, s, s) for s in (1024, 2048, 4096, 8192)]


def nonsquarish_fp32():
    return [(65536, 64, 512), (64, 65536, 512), (8192, 8192, 32), (256, 256, 65536)]


def square_half_sweep():
    return [(s, s, s) for s in (4096, 8192, 16384)]


@dataclass(frozen=True)
class Problem:
    """One GEMM call of a workload: shape, scalars and the recipe of its synthetic operands."""
    name: str
    dtype: int
    m: int
    n: int
    k: int
    alpha: float = 1.0
    beta: float = 0.0
    transA: str = "N"
    transB: str = "N"
    kindA: str = "uniform"
    kindB: str = "uniform"
    kindC: str = "uniform"
    scaleA: float = 1.0
    scaleB: float = 1.0
    seed: int = 0
    pad: tuple = field(default=(0, 0, 0))   # extra leading-dimension rows for A, B, C
    c16: bool = False                       # C in the 16-bit type of A and B (the library's *_C16 data types)
    tc3: bool = False                       # fp32 data multiplied on the tensor cores as three bfloat16 pieces (GEMM_F32_TC)
    acc16: bool = False                     # binary16 data, binary16 accumulator (GEMM_F16_ACC16; set together with c16)

    @property
    def flops(self) -> float:
        return 2.0 * self.m * self.n * self.k

    @property
    def api_dtype(self) -> int:
        """Data-type code of the library call: dtype, or its all-16-bit form (3 = f16, 4 = bf16) when C is 16-bit."""
        if self.tc3:
            return 5
        if self.acc16:
            return 6
        return self.dtype + 2 if self.c16 else self.dtype

    def algorithmic_bytes(self) -> float:
        es = 4 if self.dtype == DTYPE_F32 else 2
        c_passes = 1 + (1 if self.beta != 0.0 else 0)
        return es * (self.m * self.k + self.k * self.n) + (2.0 if self.c16 else 4.0) * self.m * self.n * c_passes

    def stored_dims(self):
        a = (self.m, self.k) if self.transA in "Nn" else (self.k, self.m)
        b = (self.k, self.n) if self.transB in "Nn" else (self.n, self.k)
        return a, b

    def operands(self, need_c0: bool = True) -> tuple[Matrix, Matrix, Matrix]:
        """(A, B, C0) as stored matrices; C0 is fp32 unless c16.  need_c0=False (callers that never read C0, beta = 0)
        fills C0 with zeros instead of generating it."""
        (ar, ac), (br, bc) = self.stored_dims()
        A = make_matrix(ar, ac, kind=self.kindA, seed=self.seed, matrix_id=0, dtype=self.dtype,
                        ld=max(1, ar) + self.pad[0], scale=self.scaleA)
        B = make_matrix(br, bc, kind=self.kindB, seed=self.seed, matrix_id=1, dtype=self.dtype,
                        ld=max(1, br) + self.pad[1], scale=self.scaleB)
        C = make_matrix(self.m, self.n, kind=self.kindC if need_c0 else "zeros", seed=self.seed, matrix_id=2,
                        dtype=self.dtype if self.c16 else DTYPE_F32, ld=max(1, self.m) + self.pad[2])
        return A, B, C


def config_problems(config: int, *, integer: bool = False, dtype: int | None = None, c16: bool = False) -> list[Problem]:
    """The problems of workload `config` (1..5).

    1: single fp32 512^3, seed 0, alpha=1, beta=0 (integer=True: entries in [-4,4])
    2: square fp32 sweep, alpha=1.5, beta=0.5, C pre-filled
    3: im2row-lowered ResNet-50-style layers, batch 32, fp32; weights N(0, 2/k), activations |N(0,1)|
    4: non-squarish fp32 shapes
    5: fp16/bf16 inputs (dtype argument), squares with N(0,1) entries plus the shapes of 3
    Seeds: the first problem of config c uses seed c-1, the following ones 1000*c + index.
    """
    def seed(i):
        return config - 1 if i == 0 else 1000 * config + i

    kind = "int" if integer else None
    probs: list[Problem] = []
    if config == 1:
        probs.append(Problem("sq512", DTYPE_F32, 512, 512, 512, 1.0, 0.0,
                             kindA=kind or "uniform", kindB=kind or "uniform",
                             kindC=kind or "uniform", seed=seed(0)))
    elif config == 2:
        for i, (m, n, k) in enumerate(square_fp32_sweep()):
            probs.append(Problem(f"sq{m}", DTYPE_F32, m, n, k, 1.5, 0.5,
                                 kindA=kind or "uniform", kindB=kind or "uniform",
                                 kindC=kind or "uniform", seed=seed(i)))
    elif config == 3:
        for i, (m, n, k) in enumerate(im2row_shapes()):
            probs.append(Problem(f"rn50_{i + 1:02d}", DTYPE_F32, m, n, k, 1.0, 0.0,
                                 kindA=kind or "normal", kindB=kind or "absnormal",
                                 kindC=kind or "uniform", scaleA=(2.0 / k) ** 0.5, seed=seed(i)))
    elif config == 4:
        for i, (m, n, k) in enumerate(nonsquarish_fp32()):
            probs.append(Problem(f"ns_{m}x{n}x{k}", DTYPE_F32, m, n, k, 1.0, 0.0,
                                 kindA=kind or "uniform", kindB=kind or "uniform",
                                 kindC=kind or "uniform", seed=seed(i)))
    elif config == 5:
        dt = DTYPE_F16 if dtype is None else dtype
        tag = "h" if dt == DTYPE_F16 else "b"
        i = 0
        for (m, n, k) in square_half_sweep():
            probs.append(Problem(f"{tag}sq{m}", dt, m, n, k, 1.0, 0.0,
                                 kindA=kind or "normal", kindB=kind or "normal",
                                 kindC=kind or "uniform", seed=seed(i)))
            i += 1
        for j, (m, n, k) in enumerate(im2row_shapes()):
            probs.append(Problem(f"{tag}rn50_{j + 1:02d}", dt, m, n, k, 1.0, 0.0,
                                 kindA=kind or "normal", kindB=kind or "absnormal",
                                 kindC=kind or "uniform", scaleA=(2.0 / k) ** 0.5, seed=seed(i)))
            i += 1
    else:
        raise ValueError("config must be 1..5")
    if c16:      # the same problems with C in the 16-bit type of the operands (config 5 only)
        if config != 5:
            raise ValueError("c16 needs 16-bit operands")
        import dataclasses
        probs = [dataclasses.replace(p, name=p.name + "_c16", c16=True) for p in probs]
    return probs


def im2row_problems(network: str = "vgg16", *, batch: int = 32, weights_as_A: bool = True,
                    dtype: int = DTYPE_F32) -> list[Problem]:
    """The second workload and the paper's own orientation of both networks.

    network: 'resnet50' or 'vgg16' (Tables "resnet50" / "vgg16").  weights_as_A=False keeps the paper's roles
    (m = batch*pixels, n = output channels: activations are operand A, weights operand B), the tall-and-skinny
    mirror of the config-3 problems.  Seeds 6000 + index (vgg16) / 7000 + index (resnet50), +500 in the paper's
    orientation.
    """
    layers = {"vgg16": VGG16_BATCH1, "resnet50": RESNET50_V15_BATCH1}[network]
    base = (6000 if network == "vgg16" else 7000) + (0 if weights_as_A else 500)
    tag = ("h" if dtype == DTYPE_F16 else "b" if dtype == DTYPE_BF16 else "") + network[:3] + ("" if weights_as_A else "_px")
    probs = []
    for i, (m, n, k) in enumerate(im2row_shapes(layers, batch, weights_as_A)):
        w_std = (2.0 / k) ** 0.5
        if weights_as_A:
            kinds = dict(kindA="normal", kindB="absnormal", scaleA=w_std)
        else:
            kinds = dict(kindA="absnormal", kindB="normal", scaleB=w_std)
        probs.append(Problem(f"{tag}_{i + 1:02d}", dtype, m, n, k, 1.0, 0.0, seed=base + i, **kinds))
    return probs


# ---------------------------------------------------------------- convolution layers (the step before the lowering)

@dataclass(frozen=True)
class ConvProblem:
    """One convolution layer whose im2row lowering is a GEMM of the workloads: geometry, scalars and the recipe of
    its synthetic tensors.  Activations are NHWC, filters a column-major C_out x (kh*kw*C_in) matrix with the k index
    in (r, s, c) order, the result NHWC (as a column-major matrix: C_out x pixels)."""
    name: str
    dtype: int
    batch: int
    h: int
    w: int
    c_in: int
    c_out: int
    kh: int
    kw: int
    stride: int = 1
    pad: int = 0
    alpha: float = 1.0
    beta: float = 0.0
    kindX: str = "absnormal"
    kindW: str = "normal"
    kindY: str = "uniform"
    seed: int = 0
    ld_pad: tuple = field(default=(0, 0))     # extra leading-dimension rows for the filter matrix and for Y
    c16: bool = False                         # result in the 16-bit type of the activations (the library's *_C16 types)

    @property
    def api_dtype(self) -> int:
        return self.dtype + 2 if self.c16 else self.dtype

    @property
    def out_hw(self):
        return ((self.h + 2 * self.pad - self.kh) // self.stride + 1, (self.w + 2 * self.pad - self.kw) // self.stride + 1)

    @property
    def gemm_mnk(self):
        """(m, n, k) of the lowered GEMM with the filters as operand A: m = C_out, n = batch*Ho*Wo, k = kh*kw*C_in."""
        ho, wo = self.out_hw
        return self.c_out, self.batch * ho * wo, self.kh * self.kw * self.c_in

    @property
    def flops(self) -> float:
        m, n, k = self.gemm_mnk
        return 2.0 * m * n * k

    def algorithmic_bytes(self) -> float:
        """Activations and filters read once, result written once (read once more if beta != 0): what a fused
        lowering has to move.  The lowered matrix itself (k x pixels) is never counted."""
        es = 4 if self.dtype == DTYPE_F32 else 2
        m, n, k = self.gemm_mnk
        return es * (self.batch * self.h * self.w * self.c_in + m * k) + (2.0 if self.c16 else 4.0) * m * n * (2 if self.beta != 0.0 else 1)

    def operands(self) -> tuple[Matrix, Matrix, Matrix]:
        """(X, W, Y0): X as the C_in x (batch*H*W) column-major matrix that an NHWC tensor is, W as C_out x k,
        Y0 (fp32) as C_out x pixels."""
        m, n, k = self.gemm_mnk
        scale_w = 1.0 if self.kindW == "int" else (2.0 / k) ** 0.5
        X = make_matrix(self.c_in, self.batch * self.h * self.w, kind=self.kindX, seed=self.seed, matrix_id=1, dtype=self.dtype)
        W = make_matrix(m, k, kind=self.kindW, seed=self.seed, matrix_id=0, dtype=self.dtype, ld=m + self.ld_pad[0], scale=scale_w)
        Y0 = make_matrix(m, n, kind=self.kindY, seed=self.seed, matrix_id=2, dtype=self.dtype if self.c16 else DTYPE_F32,
                         ld=m + self.ld_pad[1])
        return X, W, Y0


def conv_layer_problems(network: str = "resnet50", *, batch: int = 32, dtype: int = DTYPE_F32, integer: bool = False,
                        c16: bool = False) -> list[ConvProblem]:
    """The convolution layers behind the rows of Tables "resnet50" / "vgg16", with the usual geometry of those
    networks: 7 x 7 stride 2 pad 3 on a 224 x 224 image for the ResNet stem, 3 x 3 stride 1 pad 1 and 1 x 1 layers on
    an input of the output's size.  Their lowered GEMM dimensions equal im2row_shapes(..., weights_as_A=True).
    Seeds 8000 + index (resnet50) / 9000 + index (vgg16)."""
    layers = {"vgg16": VGG16_BATCH1, "resnet50": RESNET50_V15_BATCH1}[network]
    base = 8000 if network == "resnet50" else 9000
    tag = ("h" if dtype == DTYPE_F16 else "b" if dtype == DTYPE_BF16 else "") + network[:3] + "_conv"
    kinds = dict(kindX="int", kindW="int", kindY="int") if integer else {}
    out = []
    for i, L in enumerate(layers):
        if L.ksize == 7:
            geo = dict(h=2 * L.out_hw, w=2 * L.out_hw, stride=2, pad=3)
        else:
            geo = dict(h=L.out_hw, w=L.out_hw, stride=1, pad=L.ksize // 2)
        out.append(ConvProblem(f"{tag}_{i + 1:02d}" + ("_c16" if c16 else ""), dtype, batch, c_in=L.cin, c_out=L.cout,
                               kh=L.ksize, kw=L.ksize, seed=base + i, c16=c16, **geo, **kinds))
    return out
