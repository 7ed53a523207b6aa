"""Which kernel a chain takes (fc_last_plan): a chain that silently fell back to the interpreter, or a GEMM that
stopped splitting, would still pass the parity tests and be several times slower."""
from dataclasses import replace

import pytest
import torch

from fc_inputs import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fc():
    import __graft_entry__ as entry
    entry.build()
    import paper_2602_14293_b200 as fc
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    torch.cuda.set_device(0)
    return fc


def _plan(fc, ch):
    ins = [fc.to_device(a) for a in wl.make_inputs(ch, 0)]
    fc.run_chain(ch, ins)
    fc.fc_get_async_status()
    return fc.fc_last_plan()


def test_elementwise_routing(fc):
    base = wl.affine_gelu_residual_lse(64, 4096)
    assert _plan(fc, base) == "ew_rows"
    assert _plan(fc, replace(base, reduce="none")) == "ew_rows"
    assert _plan(fc, replace(base, ops=(("bias_n", 2), ("relu",), ("scale", 0.5), ("clamp", -1.0, 1.0), ("add_tensor", 3)))) == "ew_rows"
    assert _plan(fc, wl.scale_add_softmax(64, 4096)) == "ew_rows_softmax_stash"
    assert _plan(fc, replace(wl.affine_gelu_residual_lse(64, 8192), reduce="row_softmax", store_main=False)) == "ew_rows_softmax"   # vectors + stash do not fit
    assert _plan(fc, wl.affine_gelu_residual_lse(64, 64)) == "ew_narrow"
    assert _plan(fc, wl.scale_add_softmax(1000, 256)) == "ew_narrow"
    assert _plan(fc, replace(wl.affine_gelu_residual_lse(64, 64), reduce="none")) == "ew_interpreter_flat"
    assert _plan(fc, wl.affine_gelu_residual_lse(8, 12288)) == "ew_longrow"
    assert _plan(fc, wl.scale_add_softmax(8, 50264)) == "ew_longrow"
    assert _plan(fc, wl.scale_add_softmax(8, 50257)) == "ew_longrow_ragged"
    assert _plan(fc, wl.affine_gelu_residual_lse(8, 50257)) == "ew_interpreter_rows"   # vectors on ragged rows
    assert _plan(fc, wl.cast(100, 640)) == "ew_interpreter_flat"
    assert _plan(fc, replace(base, ops=(("add_tensor", 3), ("clamp", -1.0, 1.0)))) == "ew_interpreter_rows"


def test_contraction_routing(fc):
    assert _plan(fc, wl.gemm_bias_relu_f32(256, 256, 256)) == "gemm_f32"
    assert _plan(fc, wl.gemm_bias_relu_f32(1024, 1024, 64)) == "gemm_f32_mid"
    assert _plan(fc, wl.gemm_bias_relu_f32(2048, 1024, 64)) == "gemm_f32_big"
    # rounds of tiles: 240-column tiles where rounds x width is smaller (256 tiles = 4 rounds x 256 against 288 = 4 rounds x 240)
    assert _plan(fc, wl.gemm_bias_gelu_scale_clamp(4096, 4096, 256)) == "gemm_tc_mode0_bn240"
    assert _plan(fc, wl.gemm_bias_gelu_scale_clamp(8192, 8192, 256)) == "gemm_tc_mode0_bn256"     # 14 rounds x 256 against 16 x 240
    # few tiles: 128-wide ones where the cost model prefers twice the tiles with half the epilogue each ...
    assert _plan(fc, wl.gemm_bias_gelu_scale_clamp(512, 512, 256)) == "gemm_tc_mode0_bn128"
    assert _plan(fc, wl.gemm_bias_gelu_scale_clamp(128, 256, 4096)) == "gemm_tc_mode0_bn128_split"
    # ... and 256-wide ones cut along K where the main loop dominates
    assert _plan(fc, wl.gemm_bias_gelu_scale_clamp(16, 8192, 8192)) == "gemm_tc_mode0_bn256_split"
    assert _plan(fc, wl.gemm_bias_gelu_scale_clamp(512, 128, 256)) == "gemm_tc_mode0_bn128"
    assert _plan(fc, wl.gemm_softmax(256, 1024, 4096)) == "gemm_tc_mode1_bn256_split"      # 4 tiles: cut along K as well
    assert _plan(fc, wl.gemm_softmax(4096, 4096, 4096)) == "gemm_tc_mode1_bn240"
    assert _plan(fc, wl.gemm_softmax(4096, 1024, 4096)) == "gemm_tc_mode1_bn256"      # one round of 64 tiles against two of 240-column ones
    assert _plan(fc, wl.gemm_softmax(256, 1024, 256)) == "gemm_tc_mode1_bn256"                # rows of up to 16 tiles: one pass at any depth
    assert _plan(fc, wl.gemm_softmax(256, 8192, 4096)) == "gemm_tc_mode1_bn256_split"         # up to 32 tiles from K = 2048 on (few enough to be cut along K)
    assert _plan(fc, wl.gemm_softmax(256, 8192, 1024)) == "gemm_tc_mode1_bn256_two_pass softmax_rescale"         # 32 tiles behind a short contraction (too short to be cut)
    assert _plan(fc, wl.gemm_softmax(256, 8448, 4096)) == "gemm_tc_mode1_bn256_split_two_pass softmax_rescale"   # 33 tiles per panel
    assert _plan(fc, wl.gemm_softmax(64, 20000, 64)) == "gemm_tc_mode1_bn256_two_pass softmax_rescale"
    assert _plan(fc, wl.gemm_bias_scale_lse(256, 1024, 256)) == "gemm_tc_mode3_bn128"       # few tiles: as the plain GEMM
    assert _plan(fc, wl.gemm_bias_scale_lse(2048, 4096, 256)) == "gemm_tc_mode3_bn240"
    assert _plan(fc, wl.gemm_bias_scale_lse(4096, 8192, 256)) == "gemm_tc_mode3_bn256"
    assert _plan(fc, wl.linear_row_reduce(96, 512, 256)) == "weight_colsum colsum_finish row_dot"
    assert _plan(fc, wl.mlp(300, (64, 64, 32))) == "mlp_tc"
    conv = wl.conv_bias_relu_avgpool(batch=2, H=14, W=14, Cin=64, Cout=128)
    assert _plan(fc, conv) == "zero_fill gemm_tc_mode2_bn128"
    # max-pool: tiles of whole row pairs (no zeros in front) where they pay or where the output is 16 bits wide
    padded8 = wl.conv_bias_relu_maxpool(batch=2, H=14, W=14, Cin=8, Cout=264, R=5, S=5, pad=2)
    assert _plan(fc, padded8) == "pad_image gemm_tc_mode2_bn256_rowtaps"           # bordered copy in the workspace, filter rows
    # ... by the library's own rule only from some eight rounds of tiles on (the border pass is a launch of its own)
    fc.binding.fc_testing_set(fc.binding.FC_TESTING_BORDER_PASS, 0)
    try:
        assert _plan(fc, padded8) == "gemm_tc_mode4_bn256"
        big = wl.conv_bias_relu_maxpool(batch=1024, H=32, W=32, Cin=8, Cout=32, R=3, S=3, pad=1)     # 4096 tiles
        assert _plan(fc, big) == "pad_image gemm_tc_mode2_bn64_rowtaps"
        small = wl.conv_bias_relu_maxpool(batch=64, H=32, W=32, Cin=8, Cout=32, R=3, S=3, pad=1)      # 256 tiles
        assert _plan(fc, small) == "gemm_tc_mode4_bn64"
    finally:
        fc.binding.fc_testing_set(fc.binding.FC_TESTING_BORDER_PASS, 1)
    fc.binding.fc_set_workspace(None)
    fc.binding.fc_run(fc.make_spec(padded8), [fc.to_device(a) for a in wl.make_inputs(padded8, 0)], fc.binding.output_tensors(padded8, "cuda"))
    assert fc.fc_last_plan() == "gemm_tc_mode4_bn256"                              # no workspace: eight taps per k-block
    assert _plan(fc, wl.conv_bias_relu_maxpool(batch=2, H=14, W=14, Cin=8, Cout=264, R=5, S=5, pad=0)) == "gemm_tc_mode2_bn256_rowtaps"
    deep = wl.conv_bias_relu_maxpool(batch=2, H=14, W=14, Cin=64, Cout=128, R=5, S=5, pad=0)          # 25 k-blocks, row pairs of 20
    assert _plan(fc, deep) == "zero_fill gemm_tc_mode2_bn128"
    assert _plan(fc, replace(deep, out_dtype="bf16")) == "gemm_tc_mode2_bn128"
    assert _plan(fc, wl.conv_bias_relu_maxpool(batch=2, H=15, W=14, Cin=8, Cout=64, R=5, S=5, pad=0)) == "zero_fill gemm_tc_mode2_bn64_rowtaps"   # 11 rows
    assert _plan(fc, wl.conv_bias_relu_maxpool(batch=2, H=16, W=16, Cin=64, Cout=128, R=3, S=3, pad=1)) == "gemm_tc_mode2_bn128"   # row pairs of 32
    assert _plan(fc, wl.conv_nchw(conv)) == "cfirst_to_clast cfirst_to_clast zero_fill gemm_tc_mode2_bn128"
