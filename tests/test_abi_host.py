"""Host-side checks that need no GPU: the library loads, exports every symbol the header declares,
and rejects malformed chains before touching a device."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from fc_inputs import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fc():
    entry.build()
    import paper_2602_14293_b200 as fc
    return fc


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(fc_[a-z_0-9]+)\s*\(", src))
    return names


def test_library_exports_every_declared_symbol(fc):
    L = fc.lib()
    names = _declared_symbols()
    assert {"fc_run", "fc_run_host", "fc_workspace_size", "fc_set_workspace", "fc_get_async_status"} <= names
    for n in names:
        assert hasattr(L, n), n
    assert fc.fc_version() == 2


def test_spec_struct_matches_header_size(fc):
    # 4 + 4 + 4*4 + 12*8 + 4 (+4 pad?) ... the library checks struct_size itself; a mismatch is INVALID_SPEC
    spec = fc.make_spec(wl.CONFIGS["C3"]())
    n = ctypes.c_size_t(0)
    assert fc.lib().fc_workspace_size(ctypes.byref(spec), ctypes.byref(n)) == 0 and n.value == 0


def test_workspace_size_softmax(fc):
    spec = fc.make_spec(wl.CONFIGS["C4"]())
    # 32 arrival + 32 departure panel counters (each padded to 256 B) + 4096 rows x 16 tiles x (max, sum) fp32
    assert fc.fc_workspace_size(spec) == 2 * 256 + 4096 * 16 * 8 * 2      # a (max, sum) pair per row, tile and column half
    # the other row reductions: the same room, for a pair per row and 128-column tile
    lse = fc.make_spec(wl.gemm_bias_scale_lse(4096, 4096, 512))
    assert fc.fc_workspace_size(lse) == 2 * 256 + 4096 * 32 * 8


def _status(fc, spec, ins=None, outs=None):
    pi = ctypes.cast(ins, ctypes.POINTER(type(ins[0]))) if ins is not None else None
    po = ctypes.cast(outs, ctypes.POINTER(type(outs[0]))) if outs is not None else None
    return fc.lib().fc_run(ctypes.byref(spec) if spec is not None else None, pi, len(ins) if ins is not None else 0,
                           po, len(outs) if outs is not None else 0, None)


def _fake_tensor(fc, shape, dtype, ptr=0x1000):
    from paper_2602_14293_b200.binding import fc_tensor
    t = fc_tensor()
    t.ptr = ptr
    t.dtype = dtype
    t.rank = len(shape)
    st = 1
    for i in reversed(range(len(shape))):
        t.shape[i] = shape[i]
        t.stride[i] = st
        st *= shape[i]
    return t


def _arr(fc, ts):
    from paper_2602_14293_b200.binding import fc_tensor
    a = (fc_tensor * len(ts))()
    for i, t in enumerate(ts):
        a[i] = t
    return a


def test_rejections_happen_before_any_device_access(fc):
    L = fc.lib()
    launches_before = fc.fc_launch_count()
    ch = wl.gemm_bias_gelu_scale_clamp(256, 256, 64)
    good_in = _arr(fc, [_fake_tensor(fc, (256, 64), 1), _fake_tensor(fc, (256, 64), 1), _fake_tensor(fc, (256,), 1)])
    good_out = _arr(fc, [_fake_tensor(fc, (256, 256), 1)])
    FC_ERR_NULL, INVALID, UNSUP, SHAPE, ALIGN = 1, 2, 3, 4, 5

    assert L.fc_run(None, None, 0, None, 0, None) == FC_ERR_NULL
    s = fc.make_spec(ch); s.struct_size = 8
    assert _status(fc, s, good_in, good_out) == INVALID
    s = fc.make_spec(ch); s.version = 99
    assert _status(fc, s, good_in, good_out) == INVALID
    s = fc.make_spec(ch); s.producer = 7
    assert _status(fc, s, good_in, good_out) == INVALID
    s = fc.make_spec(ch); s.ops[0].kind = 42
    assert _status(fc, s, good_in, good_out) == INVALID
    s = fc.make_spec(ch); s.ops[0].in0 = 9          # operand index out of range
    assert _status(fc, s, good_in, good_out) == INVALID
    s = fc.make_spec(ch); s.ops[3].f0, s.ops[3].f1 = 1.0, -1.0   # clamp lo > hi
    assert _status(fc, s, good_in, good_out) == INVALID
    s = fc.make_spec(ch); s.K = 0
    assert _status(fc, s, good_in, good_out) == SHAPE
    s = fc.make_spec(ch)
    bad_in = _arr(fc, [_fake_tensor(fc, (256, 64), 1), _fake_tensor(fc, (128, 64), 1), _fake_tensor(fc, (256,), 1)])
    assert _status(fc, s, bad_in, good_out) == SHAPE
    null_in = _arr(fc, [_fake_tensor(fc, (256, 64), 1, ptr=0), _fake_tensor(fc, (256, 64), 1), _fake_tensor(fc, (256,), 1)])
    assert _status(fc, s, null_in, good_out) == FC_ERR_NULL
    mis_in = _arr(fc, [_fake_tensor(fc, (256, 64), 1, ptr=0x1008), _fake_tensor(fc, (256, 64), 1), _fake_tensor(fc, (256,), 1)])
    assert _status(fc, s, mis_in, good_out) == ALIGN
    ch_k = wl.gemm_bias_gelu_scale_clamp(256, 256, 60)     # K % 8 != 0
    k_in = _arr(fc, [_fake_tensor(fc, (256, 60), 1), _fake_tensor(fc, (256, 60), 1), _fake_tensor(fc, (256,), 1)])
    assert _status(fc, fc.make_spec(ch_k), k_in, good_out) == ALIGN
    # well-formed but not implemented: average pool after a GEMM, conv stride > 8, pooling on an elementwise producer
    s = fc.make_spec(ch); s.reduce = 3          # global average pool after a GEMM
    assert _status(fc, s, good_in, good_out) == UNSUP
    s = fc.make_spec(wl.conv_bias_relu_avgpool(stride=9))
    assert _status(fc, s, good_in, good_out) == UNSUP
    s = fc.make_spec(wl.affine_gelu_residual_lse(8, 8)); s.reduce = 3
    assert _status(fc, s, good_in, good_out) == UNSUP
    assert "FC_ERR_UNSUPPORTED" == L.fc_status_string(UNSUP).decode()
    assert len(fc.fc_last_error()) > 0
    # nothing above reached a launch
    assert fc.fc_launch_count() == launches_before


def test_non_contiguous_tensor_is_rejected(fc):
    ch = wl.affine_gelu_residual_lse(8, 16)
    s = fc.make_spec(ch)
    x = _fake_tensor(fc, (8, 16), 1); x.stride[0] = 32
    ins = _arr(fc, [x, _fake_tensor(fc, (16,), 1), _fake_tensor(fc, (16,), 1), _fake_tensor(fc, (8, 16), 1)])
    outs = _arr(fc, [_fake_tensor(fc, (8, 16), 1), _fake_tensor(fc, (8,), 0)])
    assert _status(fc, s, ins, outs) == 3


def test_workspace_sizes_of_split_and_collapsed_chains(fc):
    """Sizes are host arithmetic: the optional split scratch is a fixed region behind the required part,
    and a collapsing chain needs its slabs of fp64 column sums plus the fp32 vector."""
    b = fc.binding
    plain = fc.make_spec(wl.gemm_bias_gelu_scale_clamp(256, 1024, 4096))
    assert b.fc_workspace_size(plain) == 0
    split_region = b.fc_workspace_size_split(plain)
    assert split_region == 1024 + 80 * 2 * 128 * 256 * 4
    soft = fc.make_spec(wl.CONFIGS["C4"]())
    assert b.fc_workspace_size_split(soft) == b.fc_workspace_size(soft) + split_region
    ew = fc.make_spec(wl.CONFIGS["C2"]())
    assert b.fc_workspace_size_split(ew) == 0
    # collapse: 640 target blocks / 32 column blocks = 20 slabs for K = 8192
    col = fc.make_spec(wl.linear_row_reduce(1024, 8192, 8192))
    slabs = 20
    doubles = slabs * 8192 + slabs + 1
    assert b.fc_workspace_size(col) == (doubles * 8 + 255) // 256 * 256 + 8192 * 4
    assert b.fc_workspace_size_split(col) == 0


def test_workspace_size_of_channel_first_convolution(fc):
    """CONV2D_NCHW keeps a channels-last copy of the image and of the weights, each rounded up to 256 bytes;
    the optional split scratch follows them."""
    b = fc.binding
    base = wl.conv_bias_relu_avgpool(batch=3, H=7, W=9, Cin=8, Cout=24)
    ch = wl.conv_nchw(base)
    assert [r[2] for r in ch.input_recipe[:2]] == [(3, 8, 7, 9), (24, 8, 3, 3)]
    assert wl.output_shapes(ch) == wl.output_shapes(base)
    img = (3 * 7 * 9 * 8 * 2 + 255) // 256 * 256
    wts = (24 * 3 * 3 * 8 * 2 + 255) // 256 * 256
    spec = fc.make_spec(ch)
    assert b.fc_workspace_size(spec) == img + wts
    scratch = b.fc_workspace_size_split(fc.make_spec(wl.conv_bias_relu_avgpool(batch=3, H=7, W=9, Cin=64, Cout=24)))   # split scratch alone
    # few channels with padding: room (optional) for the image with its zero border written out, behind the channels-last copies
    bordered = (3 * 9 * 11 * 8 * 2 + 255) // 256 * 256
    assert b.fc_workspace_size_split(spec) == img + wts + bordered + scratch
    assert b.fc_workspace_size(fc.make_spec(base)) == 0
    assert b.fc_workspace_size_split(fc.make_spec(base)) == bordered + scratch
    wide = wl.conv_nchw(wl.conv_bias_relu_avgpool(batch=3, H=7, W=9, Cin=64, Cout=24))
    assert b.fc_workspace_size_split(fc.make_spec(wide)) == b.fc_workspace_size(fc.make_spec(wide)) + scratch
    assert b.fc_describe_plan is not None


def test_network_stages_fit_together_and_validate(fc):
    """The LeNet-shaped sequence: every stage's first input has exactly the bytes of the previous stage's
    output, and every stage's spec passes the library's validation (fc_workspace_size validates without a GPU)."""
    import numpy as np
    size = {"f32": 4, "bf16": 2, "f16": 2}
    for pooled, n_stages in (("bf16", 3), ("f32", 5)):
        stages = wl.lenet_shaped(batch=12, pooled=pooled)
        assert len(stages) == n_stages
        prev_bytes = None
        for ch in stages:
            spec = fc.make_spec(ch)
            assert fc.binding.fc_workspace_size(spec) == 0
            _, in_dt, in_shape, *_ = ch.input_recipe[0]
            if prev_bytes is not None:
                assert int(np.prod(in_shape)) * size[in_dt] == prev_bytes, ch.name
            _, out_dt, out_shape = wl.output_shapes(ch)[0]
            prev_bytes = int(np.prod(out_shape)) * size[out_dt]
        assert wl.output_shapes(stages[-1])[0][2] == (12, 10)
    # a 16-bit pooled output is stored by the tile that holds the whole window: odd row counts and outputs wider
    # than 64 columns are turned away with a message that names the way out
    from dataclasses import replace
    for H, W in ((9, 8), (8, 130)):
        odd = replace(wl.conv_bias_relu_maxpool(batch=1, H=H, W=W, Cin=8, Cout=8, R=3, S=3, pad=1), out_dtype="bf16")
        with pytest.raises(fc.FcError, match="16-bit out_dtype"):
            fc.binding.fc_workspace_size(fc.make_spec(odd))
    assert fc.binding.fc_describe_plan is not None
    # an 8-channel first layer is legal; 4 channels are not (rows of the image must be multiples of 16 bytes)
    bad = wl.conv_bias_relu_maxpool(batch=1, H=8, W=8, Cin=4, Cout=8, R=3, S=3, pad=1)
    assert fc.binding.fc_workspace_size(fc.make_spec(bad)) == 0   # the channel rule is checked with the tensors


def test_collapse_is_chosen_only_for_linear_epilogues_without_main_output():
    assert wl.collapses(wl.linear_row_reduce(64, 64, 64))
    assert wl.collapses(wl.linear_row_reduce(64, 64, 64, "row_mean", ops=(("affine_n", 3, 4), ("scale", 2.0))))
    assert not wl.collapses(wl.linear_row_reduce(64, 64, 64, "row_max"))
    assert not wl.collapses(wl.linear_row_reduce(64, 64, 64, ops=(("bias_n", 2), ("relu",))))
    assert not wl.collapses(wl.linear_row_reduce(64, 64, 64, store_main=True))
    assert not wl.collapses(wl.gemm_bias_scale_lse(64, 64, 64))


def test_two_host_threads_keep_their_own_errors(fc):
    """fc_run may be called from several host threads: the error text and the plan record are per thread, and the
    shared state (device table, launch counter, per-device launcher state) is atomic or lock-guarded.  Two threads
    hammer the entry points with different rejected chains and each must always read back its own message."""
    import threading
    L = fc.lib()
    ch = wl.gemm_bias_gelu_scale_clamp(256, 256, 64)
    good_in = _arr(fc, [_fake_tensor(fc, (256, 64), 1), _fake_tensor(fc, (256, 64), 1), _fake_tensor(fc, (256,), 1)])
    good_out = _arr(fc, [_fake_tensor(fc, (256, 256), 1)])
    errors = []

    def worker(kind):
        s = fc.make_spec(ch)
        if kind == 0:
            s.version = 99
            want_status, want_text = 2, "version 99"
        else:
            s.K = 0
            want_status, want_text = 4, "M, N, K must be >= 1"
        for _ in range(3000):
            st = _status(fc, s, good_in, good_out)
            msg = L.fc_last_error().decode()
            if st != want_status or want_text not in msg:
                errors.append((kind, st, msg))
                return
            n = ctypes.c_size_t(0)
            if L.fc_workspace_size(ctypes.byref(fc.make_spec(wl.CONFIGS["C4"]())), ctypes.byref(n)) != 0 or n.value == 0:
                errors.append((kind, "workspace", n.value))
                return

    threads = [threading.Thread(target=worker, args=(k,)) for k in (0, 1)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors[:3]


def test_block_scaled_spec_is_validated_on_the_host(fc):
    """FC_MXF8E4M3: four producer inputs (elements and scales), K a multiple of 128, reduce NONE, workspace for the
    scale tiles."""
    ch = wl.gemm_mxf8_bias_gelu_scale_clamp(256, 384, 512)
    s = fc.make_spec(ch)
    assert fc.fc_workspace_size(s) == (2 + 2 * 2) * 4 * 512     # A: two 128-row tiles; B: two 240-column tiles of two 512-byte parts each
    F8, E8 = 3, 5
    ins = [_fake_tensor(fc, (256, 512), F8), _fake_tensor(fc, (384, 512), F8), _fake_tensor(fc, (256, 16), E8), _fake_tensor(fc, (384, 16), E8),
           _fake_tensor(fc, (384,), 1)]
    out = _arr(fc, [_fake_tensor(fc, (256, 384), 1)])
    bad = list(ins); bad[2] = _fake_tensor(fc, (256, 16), F8)              # scales must be FC_E8M0
    assert _status(fc, s, _arr(fc, bad), out) == 2
    bad = list(ins); bad[3] = _fake_tensor(fc, (384, 8), E8)               # one scale per 32 elements
    assert _status(fc, s, _arr(fc, bad), out) == 4
    assert _status(fc, s, _arr(fc, ins[:3]), out) == 2                      # too few inputs
    s2 = fc.make_spec(wl.gemm_mxf8_bias_gelu_scale_clamp(256, 384, 96))
    ins96 = [_fake_tensor(fc, (256, 96), F8), _fake_tensor(fc, (384, 96), F8), _fake_tensor(fc, (256, 3), E8), _fake_tensor(fc, (384, 3), E8),
             _fake_tensor(fc, (384,), 1)]
    assert _status(fc, s2, _arr(fc, ins96), out) == 5                       # K % 128
    s3 = fc.make_spec(ch); s3.reduce = 2
    assert _status(fc, s3, _arr(fc, ins), out) == 3
