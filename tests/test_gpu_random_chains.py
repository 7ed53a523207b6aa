"""Seeded random chains against the oracle: random producer, sizes (ragged on purpose), op lists
(fused-shape and arbitrary orders) and reductions, through the C ABI."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from fc_inputs import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fc():
    import __graft_entry__ as entry
    entry.build()
    import paper_2602_14293_b200 as fc
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    torch.cuda.set_device(0)
    return fc


def _random_ops(r, vec_idx, tensor_idx, max_vecs):
    """A random op list: half the time of the fused shape, else any order; operands by input index."""
    pool = [("relu",), ("gelu_tanh",), ("scale", float(r.choice([0.5, -0.75, 1.25]))), ("clamp", -0.75, 0.9)]
    if r.random() < 0.5:
        ops = []
        if vec_idx and r.random() < 0.7:
            ops.append(("bias_n", vec_idx[0]) if len(vec_idx) < 2 or r.random() < 0.5 else ("affine_n", vec_idx[0], vec_idx[1]))
        if r.random() < 0.7:
            ops.append(pool[int(r.integers(0, 2))])
        if r.random() < 0.5:
            ops.append(pool[2])
        if r.random() < 0.5:
            ops.append(pool[3])
        if tensor_idx is not None and r.random() < 0.5:
            ops.append(("add_tensor", tensor_idx))
        return tuple(ops)
    ops, vecs = [], 0
    for _ in range(int(r.integers(0, 6))):
        k = int(r.integers(0, 7))
        if k < 4:
            ops.append(pool[k])
        elif k == 4 and vec_idx and vecs + 1 <= max_vecs:
            ops.append(("bias_n", vec_idx[0])); vecs += 1
        elif k == 5 and len(vec_idx) >= 2 and vecs + 2 <= max_vecs:
            ops.append(("affine_n", vec_idx[1], vec_idx[0])); vecs += 2
        elif k == 6 and tensor_idx is not None:
            ops.append(("add_tensor", tensor_idx))
    return tuple(ops)


def _random_chain(r):
    kind = r.choice(["ew", "gemm", "gemm", "conv", "gemm_f32"])
    if kind == "ew":
        M, N = int(r.integers(1, 70)), int(r.choice([8, 24, 64, 200, 256, 264, 1000, 1024, 4096, 333, 10240, 12296, 30000]))
        dt = str(r.choice(["bf16", "f32", "f16"]))
        rec = (("x", dt, (M, N), "normal", 0.0, 1.0), ("v0", dt, (N,), "normal", 1.0, 0.1), ("v1", "bf16", (N,), "normal", 0.0, 0.1),
               ("t", dt, (M, N), "normal", 0.0, 1.0))
        red = str(r.choice(["none", "row_logsumexp", "row_softmax", "row_sum", "row_max", "row_mean"]))
        if red == "row_softmax":
            return wl.Chain("rand_ew", "elementwise", dt, dt, M=M, N=N, ops=_random_ops(r, [1, 2], 3, 8), reduce=red,
                            store_main=False, input_recipe=rec)
        return wl.Chain("rand_ew", "elementwise", dt, dt, M=M, N=N, ops=_random_ops(r, [1, 2], 3, 8), reduce=red,
                        store_main=bool(red == "none" or r.random() < 0.7), input_recipe=rec)
    if kind == "gemm_f32":
        M, N, K = int(r.integers(1, 150)), int(r.integers(1, 150)), int(r.integers(1, 200))
        rec = (("A", "f32", (M, K), "normal", 0.0, K ** -0.25), ("B", "f32", (N, K), "normal", 0.0, K ** -0.25),
               ("v0", "f32", (N,), "uniform", -0.1, 0.1), ("v1", "f32", (N,), "normal", 1.0, 0.1), ("t", "f32", (M, N), "normal", 0.0, 1.0))
        return wl.Chain("rand_gemm_f32", "gemm_nt", "f32", "f32", M=M, N=N, K=K, ops=_random_ops(r, [2, 3], 4, 8), input_recipe=rec)
    if kind == "gemm":
        M, N, K = int(r.integers(1, 600)), int(r.choice([8, 40, 128, 264, 520, 1000])), int(r.choice([8, 64, 72, 136, 512]))
        out_dt = str(r.choice(["bf16", "f32"]))
        rec = (("A", "bf16", (M, K), "normal", 0.0, K ** -0.25), ("B", "bf16", (N, K), "normal", 0.0, K ** -0.25),
               ("v0", "bf16", (N,), "uniform", -0.1, 0.1), ("v1", "f32", (N,), "normal", 1.0, 0.1), ("t", "bf16", (M, N), "normal", 0.0, 0.5))
        red = str(r.choice(["none", "none", "row_softmax", "row_logsumexp"]))
        ops = _random_ops(r, [2, 3], 4, 3)
        if red == "row_softmax":
            out_dt = "bf16"
        return wl.Chain("rand_gemm", "gemm_nt", "bf16", out_dt, M=M, N=N, K=K, ops=ops, reduce=red,
                        store_main=bool(red != "row_logsumexp" or r.random() < 0.5) and red != "row_softmax", input_recipe=rec)
    R, S = int(r.choice([1, 3, 5])), int(r.choice([1, 3]))
    pad, stride = int(r.integers(0, min(R, S))), int(r.choice([1, 1, 2]))
    H, W = int(r.integers(max(R, 4), 20)), int(r.integers(max(S, 4), 24))
    Cin, Cout, batch = int(r.choice([8, 64, 72])), int(r.choice([8, 64, 136])), int(r.integers(1, 4))
    base = wl.conv_bias_relu_avgpool(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, stride=stride, pad=pad)
    rec = base.input_recipe + (("v1", "bf16", (Cout,), "normal", 1.0, 0.1),)
    ops = tuple(o for o in _random_ops(r, [2, 3], None, 3))
    return replace(base, ops=ops, input_recipe=rec)


@pytest.mark.parametrize("seed", range(96))
def test_random_chain(fc, orc, seed):
    r = np.random.default_rng(1000 + seed)
    ch = _random_chain(r)
    ins = wl.make_inputs(ch, seed)
    ref = orc.run_chain(ch, ins)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    for (name, _, _), t in zip(wl.output_shapes(ch), outs):
        got, want = util.to_f64(t), ref[name]
        what = f"seed {seed}: {ch.producer} {[o[0] for o in ch.ops]} reduce={ch.reduce} {name}"
        if t.dtype in (torch.bfloat16, torch.float16):
            # magnitudes are not O(1) for every random op list: scale the absolute mean bound with the output's rms
            scale = max(1.0, float(np.sqrt(np.mean(want * want))))
            (util.check_bf16 if t.dtype == torch.bfloat16 else util.check_f16)(got / scale, want / scale, what)
        else:
            util.check_f32(got, want, what)


def _random_maxpool_chain(r):
    """Convolution -> random ops ending in ReLU -> 2x2 max-pool, every filter / stride / padding / channel mix of the
    generator above; the pooled output in 16 bits wherever the library takes it (even row count, at most 64 columns)."""
    for _ in range(100):
        R, S = int(r.choice([1, 3, 5])), int(r.choice([1, 3, 5]))
        pad, stride = int(r.integers(0, min(R, S))), int(r.choice([1, 1, 2]))
        H, W = int(r.integers(max(R, 4), 40)), int(r.integers(max(S, 4), 72))
        Cin, Cout, batch = int(r.choice([8, 16, 64, 72])), int(r.choice([8, 40, 64, 128, 136])), int(r.integers(1, 9))
        base = wl.conv_bias_relu_maxpool(batch=batch, H=H, W=W, Cin=Cin, Cout=Cout, R=R, S=S, stride=stride, pad=pad)
        if base.OH >= 2 and base.OW >= 2:
            break
    rec = base.input_recipe + (("v1", "bf16", (Cout,), "normal", 1.0, 0.1),)
    ops = tuple(o for o in _random_ops(r, [2, 3], None, 3) if o[0] != "relu") + (("relu",),)
    out_dt = "f32"
    if base.OH % 2 == 0 and base.OW <= 64:
        out_dt = str(r.choice(["f32", "bf16", "f16"]))
    in_dt = "f16" if out_dt == "f16" else "bf16"
    rec = tuple((t, in_dt if d == "bf16" else d, sh, dist, a, b) for t, d, sh, dist, a, b in rec)
    return replace(base, ops=ops, input_recipe=rec, in_dtype=in_dt, out_dtype=out_dt)


@pytest.mark.parametrize("seed", range(64))
def test_random_maxpool_chain(fc, orc, seed):
    r = np.random.default_rng(5000 + seed)
    ch = _random_maxpool_chain(r)
    ins = wl.make_inputs(ch, seed)
    ref = orc.run_chain(ch, ins)
    outs = util.poison_(fc.binding.output_tensors(ch, "cuda"))
    fc.run_chain(ch, [fc.to_device(a) for a in ins], outs)
    fc.fc_get_async_status()
    t = outs[0]
    assert t.dtype == {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[ch.out_dtype]
    what = f"seed {seed}: {ch.batch}x{ch.H}x{ch.W}x{ch.Cin}->{ch.Cout} {ch.R}x{ch.S} s{ch.stride} p{ch.pad} {[o[0] for o in ch.ops]} -> {ch.out_dtype}"
    got, want = util.to_f64(t), ref["reduce"]
    scale = max(1.0, float(np.sqrt(np.mean(want * want))))
    check = {"f32": util.check_f32, "bf16": util.check_bf16, "f16": util.check_f16}[ch.out_dtype]
    check(got / scale, want / scale, what)
