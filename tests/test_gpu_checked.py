"""The checked build of the library (-DQCONV_CHECKED: every computed global access of the CUDA-core kernels
tests its index against the tensor's extent, counts a failure, skips the access and goes on) run over small, odd
and ragged shapes of every such kernel: results must equal the oracle's and no test may have failed.  It stands
in for a memory checker.  Runs in a process of its own because a process loads one build of the library."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r'''
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from oracle import ref, fpconv_ref
from paper_1805_07941_b200 import binding
binding.LIB_PATH = binding.CHECKED_LIB_PATH
from tests.helpers import gpu_conv, oracle_conv, rand_layer
assert binding.qconv_checked_faults()[0] == 0                 # a checked build answers 0, a normal one -1
rng = np.random.default_rng(4)
def same(a, kw, algo=0):
    got, desc = gpu_conv(*a, algo=algo, **kw)
    assert (got == oracle_conv(*a, **kw)).all(), desc
    return desc
# direct kernel: groups, strides, odd sizes, residual, concat window
for (N, H, W, C, K, R, S, g, st, pad) in [(2, 7, 9, 6, 4, 3, 3, 2, (1, 1), (1, 1)), (1, 9, 5, 8, 8, 2, 3, 8, (2, 1), (0, 1)),
                                            (3, 5, 5, 5, 7, 1, 1, 1, (1, 1), (0, 0))]:
    x, w, b, s, r, t = rand_layer(rng, N, H, W, C, K, R, S, groups=g, with_res=True, stride=st, pad=pad)
    assert "direct" in same((x, w, b, s, r, t), dict(R=R, S=S, stride=st, pad=pad, groups=g, relu=1), 1)
    same((x, w, b, s), dict(R=R, S=S, stride=st, pad=pad, groups=g, out_c_offset=3, out_c_pitch=K + 5), 1)
# depthwise: general dp4a kernel, tap-packed with register loads, tap-packed with TMA rows
for (N, H, W, C, st) in [(2, 9, 11, 8, 1), (1, 13, 10, 20, 2), (2, 17, 15, 64, 1), (1, 16, 16, 96, 2), (3, 7, 7, 32, 1)]:
    x, w, b, s, _, _ = rand_layer(rng, N, H, W, C, C, 3, 3, groups=C, stride=(st, st), pad=(1, 1))
    b = (b // 64).astype(np.int32)
    kw = dict(R=3, S=3, stride=(st, st), pad=(1, 1), groups=C, relu=1)
    same((x, w, b, s), kw, 3)
    same((x, w, b, s), dict(kw, rounding=1), 3)               # other rounding mode: the general kernel
    with binding.plan_hints(depthwise_form=1):
        same((x, w, b, s), kw, 3)
# stems: patch rows (both packers), space-to-depth, window rows
for (N, H, W, C, K, R, st, pad) in [(2, 20, 24, 3, 32, 3, (1, 1), (1, 1)), (1, 9, 9, 1, 16, 5, (1, 1), (2, 2)), (1, 8, 8, 4, 24, 3, (1, 2), (1, 0)),
                                     (2, 33, 31, 3, 32, 7, (2, 2), (3, 3)), (1, 17, 19, 2, 16, 3, (2, 2), (0, 0)), (1, 11, 40, 3, 16, 7, (1, 1), (3, 3))]:
    x, w, b, s, _, _ = rand_layer(rng, N, H, W, C, K, R, R, stride=st, pad=pad)
    same((x, w, b, s), dict(R=R, S=R, stride=st, pad=pad, relu=1))
    with binding.plan_hints(window_rows=0, space_to_depth=0):      # the patch-matrix packers
        same((x, w, b, s), dict(R=R, S=R, stride=st, pad=pad, relu=1))
    if st[0] == st[1]:                                             # the float image through the packing kernel
        xf = (rng.standard_normal(x.shape) * 3).astype(np.float32)
        cv = binding.QConv(w, b, s, N=N, H=H, W=W, C=C, K=K, R=R, S=R, stride_h=st[0], stride_w=st[1], pad_h=pad[0], pad_w=pad[1], relu=1)
        want = ref.qconv(ref.quantize_f32(xf, -4), w, b, s, R=R, S=R, stride=st, pad=pad, relu=1)
        yy = torch.zeros(want.shape, dtype=torch.int8, device="cuda")
        cv.run_f32(torch.from_numpy(xf).cuda(), -4, yy)
        assert cv.status() == 0 and (yy.cpu().numpy() == want).all()
        cv.destroy()
x, w, b, s, _, _ = rand_layer(rng, 2, 13, 17, 32, 48, 5, 5, pad=(2, 2))
assert "wrow" in same((x, w, b, s), dict(R=5, S=5, pad=(2, 2), relu=1))
# pooling (strip, vector, scalar forms), input conversion, eltwise add, float-input stem
for (N, H, W, C, R, st, pad) in [(2, 9, 7, 32, 3, 2, 1), (1, 8, 8, 16, 2, 2, 0), (2, 6, 6, 48, 3, 1, 1), (1, 7, 10, 5, 3, 2, 0), (2, 19, 19, 32, 5, 1, 2)]:
    x = rng.integers(-128, 128, size=(N, H, W, C), dtype=np.int8)
    assert (binding.qmaxpool_i8(torch.from_numpy(x).cuda(), R, R, st, pad).cpu().numpy() == ref.maxpool_i8(x, R, R, st, pad)).all()
for count in (1, 17, 4099):
    xf = (rng.standard_normal(count) * 4).astype(np.float32)
    assert (binding.qquantize_f32(torch.from_numpy(xf).cuda(), -4).cpu().numpy() == ref.quantize_f32(xf, -4)).all()
    a, bb = (rng.integers(-128, 128, size=count, dtype=np.int8) for _ in range(2))
    got = binding.qeltwise_add_i8([torch.from_numpy(a).cuda(), torch.from_numpy(bb).cuda()], [0, 2], 3, relu=1).cpu().numpy()
    assert (got == ref.eltwise_add([a, bb], [0, 2], 3, relu=1)).all()
# digit planes and recombination of the (n, p) convolution
xc = rng.integers(0, 128, size=(2, 7, 9, 16)).astype(np.uint8)
wc = rng.integers(0, 128, size=(24, 3, 3, 16)).astype(np.uint8)
conv = binding.QConvNP(wc, None, np.full(24, 9, np.int32), N=2, H=7, W=9, C=16, K=24, R=3, S=3, pad_h=1, pad_w=1,
                       n_in=8, p_in=4, n_w=8, p_w=4, n_out=8, p_out=4, relu=1)
y = torch.zeros((2, 7, 9, 24), dtype=torch.uint8, device="cuda")
conv.run(torch.from_numpy(xc).cuda(), y)
assert conv.status() == 0
assert (y.cpu().numpy() == fpconv_ref.qconv_np(xc, wc, None, np.full(24, 9), (8, 4), (8, 4), (8, 4), R=3, S=3, pad=(1, 1), relu=1)).all()
n, line = binding.qconv_checked_faults()
assert n == 0, "index test failed at kernels line %%d (%%d failures)" %% (line, n)
print("checked build: no index test failed")
''' % ROOT


@pytest.mark.gpu
def test_checked_build_sees_no_out_of_range_access():
    from paper_1805_07941_b200 import binding
    binding.build_library(checked=True)
    r = subprocess.run([sys.executable, "-c", SCRIPT], capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "no index test failed" in r.stdout
