"""Declarative descriptions of fused operator chains and their seeded synthetic inputs.

A ``Chain`` is data only (producer kind, sizes, ordered epilogue ops, reduction); the CPU oracle
and the CUDA binding each interpret it with their own code.  ``make_inputs`` draws the tensors.

The five benchmark workloads C1..C5 stand in for composed-operator problems of the kind the paper
evaluates (Level-2 style chains: a contraction or a memory-bound pass, an elementwise epilogue and
an optional row / channel reduction); the paper prints no shapes, so the shapes are the fixed
synthetic configurations of this repository.  Dense random data; no sparsity or structure.

Reading of "N(0, s)": ``s`` is the standard deviation (primary).  ``variant="var"`` re-reads it as a
variance, which makes GEMM outputs O(1) so that clamps fire and softmax rows are far from uniform.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Tuple

import numpy as np

from . import rng


@dataclass(frozen=True)
class Chain:
    name: str
    producer: str                 # "elementwise" | "gemm_nt" | "conv2d_nhwc" | "conv2d_nchw"
    in_dtype: str                 # "f32" | "bf16"  storage of inputs[0] (and inputs[1] for contractions)
    out_dtype: str                # storage of the main output (reductions other than softmax are f32)
    M: int = 0                    # elementwise: rows; gemm: rows of A
    N: int = 0                    # elementwise: cols; gemm: rows of B
    K: int = 0
    batch: int = 0                # conv only from here
    H: int = 0
    W: int = 0
    Cin: int = 0
    Cout: int = 0
    R: int = 3
    S: int = 3
    stride: int = 1
    pad: int = 1
    # ops: ("bias_n", i) ("affine_n", i, j) ("relu",) ("gelu_tanh",) ("scale", f) ("clamp", lo, hi)
    #      ("add_tensor", i) ("linear", i)   -- i, j index the input list
    ops: Tuple[tuple, ...] = ()
    reduce: str = "none"          # "none" | "row_logsumexp" | "row_softmax" | "global_avgpool" | "row_sum" | "row_max" | "row_mean" | "maxpool_2x2"
    store_main: bool = True
    # (tag, dtype, shape, dist, p0, p1) per input, in input order
    input_recipe: Tuple[tuple, ...] = field(default=(), compare=False)

    @property
    def pooled_dtype(self) -> str:
        """Storage of a 2x2 max-pool's output: the chain's out_dtype when that is a 16-bit type, else f32."""
        return self.out_dtype if self.out_dtype in ("bf16", "f16") else "f32"

    @property
    def OH(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def OW(self) -> int:
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    @property
    def widths(self):
        """Output width after the producer and after every ("linear", i) op (gemm / elementwise chains)."""
        w = [self.N]
        for op in self.ops:
            if op[0] == "linear":
                w.append(self.input_recipe[op[1]][2][0])
        return w

    @property
    def is_conv(self) -> bool:
        return self.producer in ("conv2d_nhwc", "conv2d_nchw")

    @property
    def N_out(self) -> int:
        return self.widths[-1]

    def flops(self) -> float:
        if self.producer == "gemm_nt":
            w = self.widths
            return 2.0 * self.M * (self.N * self.K + sum(a * b for a, b in zip(w[:-1], w[1:])))
        if self.is_conv:
            return 2.0 * self.batch * self.OH * self.OW * self.Cout * self.R * self.S * self.Cin
        return 0.0


def _size(dtype: str) -> int:
    if dtype in ("f8e4m3", "mxf8e4m3", "e8m0"):
        return 1
    return 4 if dtype == "f32" else 2


def gemm_bias_relu_f32(M=256, N=256, K=256, variant="std") -> Chain:
    s = 1.0 / K if variant == "std" else (1.0 / K) ** 0.5
    return Chain("gemm_f32_bias_relu", "gemm_nt", "f32", "f32", M=M, N=N, K=K,
                 ops=(("bias_n", 2), ("relu",)),
                 input_recipe=(("X", "f32", (M, K), "normal", 0.0, s),
                               ("W", "f32", (N, K), "normal", 0.0, s),
                               ("b", "f32", (N,), "uniform", -0.1, 0.1)))


def affine_gelu_residual_lse(M=16384, N=4096) -> Chain:
    return Chain("ew_affine_gelu_add_lse", "elementwise", "bf16", "bf16", M=M, N=N,
                 ops=(("affine_n", 1, 2), ("gelu_tanh",), ("add_tensor", 3)),
                 reduce="row_logsumexp", store_main=True,
                 input_recipe=(("x", "bf16", (M, N), "normal", 0.0, 1.0),
                               ("gamma", "bf16", (N,), "normal", 1.0, 0.1),
                               ("beta", "bf16", (N,), "normal", 0.0, 0.1),
                               ("r", "bf16", (M, N), "normal", 0.0, 1.0)))


def scale_add_softmax(M=16384, N=4096, scale=0.125, dtype="bf16") -> Chain:
    """x * scale + t -> row softmax: the memory-bound softmax of a score matrix with an additive term."""
    return Chain("ew_scale_add_softmax", "elementwise", dtype, dtype, M=M, N=N,
                 ops=(("scale", scale), ("add_tensor", 1)), reduce="row_softmax", store_main=False,
                 input_recipe=(("x", dtype, (M, N), "normal", 0.0, 4.0),
                               ("t", dtype, (M, N), "normal", 0.0, 1.0)))


def gemm_bias_gelu_scale_clamp(M=8192, N=8192, K=4096, variant="std") -> Chain:
    s = K ** -0.5 if variant == "std" else K ** -0.25
    return Chain("gemm_bf16_bias_gelu_scale_clamp", "gemm_nt", "bf16", "bf16", M=M, N=N, K=K,
                 ops=(("bias_n", 2), ("gelu_tanh",), ("scale", 0.5), ("clamp", -1.0, 1.0)),
                 input_recipe=(("A", "bf16", (M, K), "normal", 0.0, s),
                               ("B", "bf16", (N, K), "normal", 0.0, s),
                               ("bias", "bf16", (N,), "uniform", -0.1, 0.1)))


def gemm_f8_bias_gelu_scale_clamp(M=8192, N=8192, K=4096, out_dtype="bf16") -> Chain:
    """C3's chain with both GEMM operands stored as 8-bit E4M3 floats (per-tensor scaling is the caller's: a
    SCALE op in the epilogue undoes it).  Operand magnitudes sit in the middle of the E4M3 range."""
    return Chain("gemm_f8e4m3_bias_gelu_scale_clamp", "gemm_nt", "f8e4m3", out_dtype, M=M, N=N, K=K,
                 ops=(("scale", 1.0 / K ** 0.5), ("bias_n", 2), ("gelu_tanh",), ("scale", 0.5), ("clamp", -1.0, 1.0)),
                 input_recipe=(("A", "f8e4m3", (M, K), "normal", 0.0, 1.0),
                               ("B", "f8e4m3", (N, K), "normal", 0.0, 1.0),
                               ("bias", "bf16", (N,), "uniform", -0.1, 0.1)))


def gemm_softmax(M=4096, N=4096, K=4096, variant="std") -> Chain:
    s = K ** -0.5 if variant == "std" else K ** -0.25
    return Chain("gemm_bf16_row_softmax", "gemm_nt", "bf16", "bf16", M=M, N=N, K=K,
                 ops=(), reduce="row_softmax", store_main=False,
                 input_recipe=(("A", "bf16", (M, K), "normal", 0.0, s),
                               ("B", "bf16", (N, K), "normal", 0.0, s)))


def gemm_bias_scale_lse(M=1024, N=4096, K=1024, variant="var", store_main=False) -> Chain:
    """A linear layer followed by a row reduction to one value per row (the shape of the paper's
    appendix example: linear -> reduction -> logsumexp), here: logsumexp_n((A B^T + bias) * 0.5)."""
    s = K ** -0.5 if variant == "std" else K ** -0.25
    return Chain("gemm_bf16_bias_scale_lse", "gemm_nt", "bf16", "bf16", M=M, N=N, K=K,
                 ops=(("bias_n", 2), ("scale", 0.5)), reduce="row_logsumexp", store_main=store_main,
                 input_recipe=(("A", "bf16", (M, K), "normal", 0.0, s),
                               ("B", "bf16", (N, K), "normal", 0.0, s),
                               ("bias", "bf16", (N,), "uniform", -0.1, 0.1)))


def linear_row_reduce(M=1024, N=8192, K=8192, reduce="row_sum", ops=None, variant="std", store_main=False) -> Chain:
    """A linear layer reduced over its output features to one value per row (the first steps of the
    paper's showcase chain: linear -> sum over features).  Default ops: bias only, which leaves the chain
    linear; pass ops with a ("relu",) to keep the contraction."""
    s = K ** -0.5 if variant == "std" else K ** -0.25
    if ops is None:
        ops = (("bias_n", 2),)
    return Chain(f"linear_bf16_{reduce}", "gemm_nt", "bf16", "bf16", M=M, N=N, K=K,
                 ops=tuple(ops), reduce=reduce, store_main=store_main,
                 input_recipe=(("A", "bf16", (M, K), "normal", 0.0, s),
                               ("B", "bf16", (N, K), "normal", 0.0, s),
                               ("bias", "bf16", (N,), "uniform", -0.1, 0.1),
                               ("gamma", "bf16", (N,), "normal", 1.0, 0.1),
                               ("beta", "bf16", (N,), "normal", 0.0, 0.1)))


def mlp(M=4096, dims=(1024, 256, 256, 64), variant="std", act="relu", out_dtype="bf16") -> Chain:
    """Back-to-back linear layers, x -> act(x W1^T + b1) -> act(. W2^T + b2) -> ... -> . WL^T + bL, with every
    hidden width at most 256 so that a block of rows stays on chip from the first layer to the last (the
    cross-layer fusion of the paper's Level-3 discussion; its appendix network ends in three such layers)."""
    assert len(dims) >= 3
    rec = [("x", "bf16", (M, dims[0]), "normal", 0.0, 1.0)]
    ops = []
    s0 = dims[0] ** -0.5 if variant == "std" else dims[0] ** -0.25
    rec.append(("W1", "bf16", (dims[1], dims[0]), "normal", 0.0, s0))
    rec.append(("b1", "bf16", (dims[1],), "uniform", -0.1, 0.1))
    ops.append(("bias_n", 2))
    for l in range(2, len(dims)):
        ops.append((act,))
        sl = (2.0 / dims[l - 1]) ** 0.5
        rec.append((f"W{l}", "bf16", (dims[l], dims[l - 1]), "normal", 0.0, sl))
        rec.append((f"b{l}", "bf16", (dims[l],), "uniform", -0.1, 0.1))
        ops.append(("linear", len(rec) - 2))
        ops.append(("bias_n", len(rec) - 1))
    return Chain("mlp_bf16", "gemm_nt", "bf16", out_dtype, M=M, N=dims[1], K=dims[0], ops=tuple(ops), reduce="none",
                 store_main=True, input_recipe=tuple(rec))


def conv_bias_relu_avgpool(batch=32, H=56, W=56, Cin=256, Cout=256, R=3, S=3, stride=1, pad=1) -> Chain:
    s = (R * S * Cin) ** -0.5
    return Chain("conv_bf16_bias_relu_avgpool", "conv2d_nhwc", "bf16", "f32",
                 batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, stride=stride, pad=pad,
                 ops=(("bias_n", 2), ("relu",)), reduce="global_avgpool", store_main=False,
                 input_recipe=(("in", "bf16", (batch, H, W, Cin), "normal", 0.0, 1.0),
                               ("Wt", "bf16", (Cout, R, S, Cin), "normal", 0.0, s),
                               ("bias", "bf16", (Cout,), "uniform", -0.1, 0.1)))


def conv_bias_relu_maxpool(batch=8, H=32, W=32, Cin=64, Cout=128, R=5, S=5, stride=1, pad=2) -> Chain:
    """Convolution -> bias -> ReLU -> 2x2 max-pool (the conv / ReLU / max-pool stage of the paper's
    Level-3 LeNet-shaped example, at tensor-core-sized channel counts)."""
    base = conv_bias_relu_avgpool(batch, H, W, Cin, Cout, R, S, stride, pad)
    return replace(base, name="conv_bf16_bias_relu_maxpool", reduce="maxpool_2x2")


def cast(M: int, N: int, in_dtype="f32", out_dtype="bf16") -> Chain:
    """Elementwise chain with an empty op list: re-store a tensor in another type (what joins a pooled fp32
    output to the 16-bit operand of the next contraction)."""
    return Chain(f"cast_{in_dtype}_{out_dtype}", "elementwise", in_dtype, out_dtype, M=M, N=N, ops=(), reduce="none",
                 store_main=True, input_recipe=(("x", in_dtype, (M, N), "normal", 0.0, 1.0),))


def lenet_shaped(batch=64, C0=8, C1=64, C2=128, widths=(120, 88, 10), pooled="bf16"):
    """The shape of the paper's Level-3 example network (LeNet-5) as a sequence of chains, at tensor-core-sized channel counts:
    conv 5x5 -> ReLU -> 2x2 max-pool, twice (32x32 -> 28 -> 14 -> 10 -> 5), then three linear layers kept on chip.
    The first input of every stage after the first is the previous stage's output (same bytes, reshaped).
    pooled="bf16": the pooled outputs are stored in the next layer's operand type (three chains); "f32": they are
    fp32 and a cast chain behind each re-stores them (five chains)."""
    s1 = conv_bias_relu_maxpool(batch=batch, H=32, W=32, Cin=C0, Cout=C1, R=5, S=5, pad=0)
    s2 = conv_bias_relu_maxpool(batch=batch, H=14, W=14, Cin=C1, Cout=C2, R=5, S=5, pad=0)
    flat = 5 * 5 * C2
    fc3 = replace(mlp(batch, (flat,) + tuple(widths)), name="lenet_fc")
    if pooled == "f32":
        return [replace(s1, name="lenet_conv1"), cast(batch, 14 * 14 * C1), replace(s2, name="lenet_conv2"), cast(batch, flat), fc3]
    return [replace(s1, name="lenet_conv1", out_dtype=pooled), replace(s2, name="lenet_conv2", out_dtype=pooled), fc3]


def conv_nchw(base: Chain) -> Chain:
    """The same convolution chain with the image stored [batch, Cin, H, W] and the weights [Cout, Cin, R, S]
    (the layouts of the paper's appendix listings); outputs are unchanged."""
    (n0, d0, (b, H, W, Ci), *r0), (n1, d1, (Co, R, S, _), *r1) = base.input_recipe[0], base.input_recipe[1]
    rec = ((n0, d0, (b, Ci, H, W), *r0), (n1, d1, (Co, Ci, R, S), *r1)) + tuple(base.input_recipe[2:])
    return replace(base, name=base.name + "_nchw", producer="conv2d_nchw", input_recipe=rec)


def gemm_mxf8_bias_gelu_scale_clamp(M=8192, N=8192, K=4096, out_dtype="bf16", exp_lo=-2, exp_hi=2) -> Chain:
    """C3's chain on block-scaled 8-bit operands (MXFP8): E4M3 elements, and per row and block of 32 elements along K
    one power-of-two scale stored as an E8M0 byte (inputs 2 and 3, shapes [M, K/32] and [N, K/32]).  The block
    exponents are uniform in [exp_lo, exp_hi]; the SCALE op brings the accumulator back to unit variance."""
    span = np.arange(exp_lo, exp_hi + 1, dtype=np.float64)
    var = K * float(np.mean(4.0 ** span)) ** 2         # unit-variance elements: variance of the scaled dot product
    return Chain("gemm_mxf8e4m3_bias_gelu_scale_clamp", "gemm_nt", "mxf8e4m3", out_dtype, M=M, N=N, K=K,
                 ops=(("scale", var ** -0.5), ("bias_n", 4), ("gelu_tanh",), ("scale", 0.5), ("clamp", -1.0, 1.0)),
                 input_recipe=(("A", "f8e4m3", (M, K), "normal", 0.0, 1.0),
                               ("B", "f8e4m3", (N, K), "normal", 0.0, 1.0),
                               ("SA", "e8m0", (M, K // 32), "int", exp_lo, exp_hi),
                               ("SB", "e8m0", (N, K // 32), "int", exp_lo, exp_hi),
                               ("bias", "bf16", (N,), "uniform", -0.1, 0.1)))


#: The five benchmark configurations, in the order the benchmark numbers them.
CONFIGS = {
    "C1": gemm_bias_relu_f32,
    "C2": affine_gelu_residual_lse,
    "C3": gemm_bias_gelu_scale_clamp,
    "C4": gemm_softmax,
    "C5": conv_bias_relu_avgpool,
}

#: Further measured workloads beyond the five configurations (rows marked "next" in the scope table).
EXTRA = {
    "F1": lambda **kw: gemm_bias_scale_lse(**{"M": 4096, "N": 8192, "K": 4096, **kw}),
    "F2": lambda **kw: linear_row_reduce(**{"M": 1024, "N": 8192, "K": 8192, **kw}),
    "F5": lambda **kw: gemm_f8_bias_gelu_scale_clamp(**kw),
    "F4": lambda **kw: mlp(**{"M": 16384, "dims": (1024, 256, 256, 64), **kw}),
    "F3": lambda **kw: conv_bias_relu_maxpool(**{"batch": 32, "H": 56, "W": 56, "Cin": 256, "Cout": 256, "R": 3, "S": 3, "pad": 1, **kw}),
    "F6": lambda **kw: conv_nchw(conv_bias_relu_avgpool(**kw)),
    "F7": lambda **kw: scale_add_softmax(**kw),
    "F8": lambda **kw: gemm_softmax(**{"M": 2048, "N": 50264, "K": 4096, **kw}),   # a vocabulary-wide softmax: two kernels
    "F9": lambda **kw: gemm_bias_relu_f32(**{"M": 2048, "N": 2048, "K": 2048, **kw}),   # C1's chain at a size where fp32 operands go to the tensor cores (three tf32 products per product)
    "F10": lambda **kw: gemm_mxf8_bias_gelu_scale_clamp(**kw),   # C3's chain on block-scaled 8-bit operands
    # an image layer (the network N1's first): 5 x 5 on 8 channels -> 64, ReLU, 2x2 max-pool stored in bf16 for the next layer
    "F11": lambda **kw: replace(conv_bias_relu_maxpool(**{"batch": 4096, "H": 32, "W": 32, "Cin": 8, "Cout": 64, "R": 5, "S": 5, "pad": 0, **kw}), out_dtype="bf16"),
}
ALL = {**CONFIGS, **EXTRA}


def make_inputs(chain: Chain, seed: int = 0) -> List[np.ndarray]:
    """Draw every input of ``chain`` (float32 arrays, or uint16 bf16 bit patterns)."""
    out = []
    for tag, dtype, shape, dist, p0, p1 in chain.input_recipe:
        key = f"{chain.name}/{tag}"
        if dist == "normal":
            a = rng.normal_f32(seed, key, shape, p0, p1)
        elif dist == "uniform":
            a = rng.uniform_f32(seed, key, shape, p0, p1)
        elif dist == "int":
            a = rng.integers_f32(seed, key, shape, int(p0), int(p1))
        else:
            raise ValueError(dist)
        out.append(rng.store(a, dtype))
    return out


def with_integer_inputs(chain: Chain, lo: int = -4, hi: int = 4) -> Chain:
    """Same chain with the two contraction operands drawn as small integers (exact in bf16 and in
    fp32 accumulation), which makes every correct contraction agree bit for bit."""
    rec = list(chain.input_recipe)
    for i in range(min(2, len(rec))):
        tag, dtype, shape, _, _, _ = rec[i]
        rec[i] = (tag, dtype, shape, "int", lo, hi)   # (block scales, inputs 2 and 3 of an MX chain, stay as they are)
    return replace(chain, input_recipe=tuple(rec))


def collapses(chain: Chain) -> bool:
    """True for a 16-bit linear layer whose ops are all linear in the accumulator and whose only output is
    the row sum / mean: the reduction then commutes with the contraction and the chain is bound by reading
    its operands once, not by the M x N x K flops."""
    return (chain.producer == "gemm_nt" and chain.in_dtype != "f32" and chain.reduce in ("row_sum", "row_mean")
            and not chain.store_main and all(op[0] in ("bias_n", "affine_n", "scale") for op in chain.ops))


def input_bytes(chain: Chain) -> int:
    return sum(int(np.prod(shape)) * _size(dtype) for _, dtype, shape, *_ in chain.input_recipe)


def output_shapes(chain: Chain):
    """[(role, dtype, shape)] of the outputs, in output order: main first (if stored), then the reduction."""
    outs = []
    if chain.is_conv:
        main_shape = (chain.batch, chain.OH, chain.OW, chain.Cout)
    else:
        main_shape = (chain.M, chain.N_out)
    if chain.reduce == "row_softmax":
        outs.append(("reduce", chain.out_dtype, main_shape))
        return outs
    if chain.store_main:
        outs.append(("main", chain.out_dtype, main_shape))
    if chain.reduce in ("row_logsumexp", "row_sum", "row_max", "row_mean"):
        outs.append(("reduce", "f32", (chain.M,)))
    elif chain.reduce == "global_avgpool":
        outs.append(("reduce", "f32", (chain.batch, chain.Cout)))
    elif chain.reduce == "maxpool_2x2":
        outs.append(("reduce", chain.pooled_dtype, (chain.batch, chain.OH // 2, chain.OW // 2, chain.Cout)))
    return outs


def algorithmic_bytes(chain: Chain) -> int:
    """Each input read once plus each output written once."""
    return input_bytes(chain) + sum(int(np.prod(s)) * _size(d) for _, d, s in output_shapes(chain))
