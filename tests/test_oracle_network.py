"""The offline procedure of Section 3 on a small stack: the quantized network must
track the float network it was calibrated against, and its bookkeeping must obey the
scheme's rules (factors in (0, 1], joins share a scale)."""
import numpy as np
import torch

from oracle import network_ref, ref
from paper_1805_07941_b200 import workloads as wl


def _float_forward(net, x, weights):
    acts = {"input": torch.from_numpy(x).permute(0, 3, 1, 2).double()}
    for nd in net["nodes"]:
        src = acts[nd["src"]]
        if nd["op"] == "maxpool":
            acts[nd["dst"]] = torch.nn.functional.max_pool2d(src, nd["R"], nd["stride"], nd["pad"])
            continue
        w, b = weights[nd["name"]]
        y = torch.nn.functional.conv2d(src[:, :nd["C"]], torch.from_numpy(w).permute(0, 3, 1, 2).double(),
                                       torch.from_numpy(b).double(), stride=nd["stride"],
                                       padding=nd["pad"], groups=nd["groups"])
        if nd["residual"]:
            y = y + acts[nd["residual"]][:, :nd["K"]]
        if nd["relu"]:
            y = torch.relu(y)
        h, w_, pitch = net["buffers"][nd["dst"]]
        if nd["dst"] not in acts:
            acts[nd["dst"]] = torch.zeros(x.shape[0], pitch, h, w_, dtype=torch.float64)
        acts[nd["dst"]][:, nd["dst_c_offset"]:nd["dst_c_offset"] + nd["K"]] = y
    return {k: v.permute(0, 2, 3, 1).numpy() for k, v in acts.items()}


def _check(net, tol):
    x = wl.gen_input(net, seed=0)
    weights = {nd["name"]: wl.gen_weights(nd, 0) for nd in net["nodes"] if nd["op"] == "conv"}
    params, e_buf, _, acts = network_ref.calibrate(net, x, weights)
    fl = _float_forward(net, x, weights)
    for nd in net["nodes"]:
        if nd["op"] != "conv":
            assert e_buf[nd["dst"]] == e_buf[nd["src"]]
            continue
        p = params[nd["name"]]
        assert (p["shift"] >= 0).all() and (p["shift"] <= 31).all()          # factors in (0, 1]
        assert (p["shift"] == e_buf[nd["dst"]] - e_buf[nd["src"]] - p["e_w"]).all()
        assert (np.abs(p["wq"]).reshape(nd["K"], -1).max(axis=1) <= 127).all()
    last = net["nodes"][-1]["dst"]
    deq = acts[last].astype(np.float64) * 2.0 ** e_buf[last]
    ref_f = fl[last]
    err = np.abs(deq - ref_f).max() / np.abs(ref_f).max()
    assert err < tol, err
    assert np.abs(acts[last]).max() >= 32                                    # uses the int8 range
    # inference with the stored parameters reproduces the calibration pass on the same batch
    again = network_ref.run(net, x, params, e_buf)
    assert (again[last] == acts[last]).all()
    return params, e_buf


def test_small_vgg_tracks_float_model():
    _check(wl.vgg16(batch=2, res=16, widths=(8, 16), reps=(2, 2)), 0.08)


def test_small_resnet_tracks_float_model():
    _check(wl.resnet50(batch=2, res=32, width=8, blocks=(2, 1)), 0.12)


def test_small_inception_block_shares_scale_across_branches():
    blocks = (("3a", 16, 24, 32, 8, 16, 16), ("pool", 0, 0, 0, 0, 0, 0), ("4a", 32, 24, 48, 8, 16, 16))
    net = wl.inception(batch=2, res=12, cin=32, blocks=blocks)
    params, e_buf = _check(net, 0.12)
    for tag in ("3a", "4a"):
        ez = {int(params[tag + b]["shift"][0] + params[tag + b]["acc_exp"][0])
              for b in ("_1x1", "_3x3", "_5x5", "_pp")}
        assert ez == {e_buf["i" + tag]}


def test_small_mobilenet_per_channel_scales():
    net = wl.mobilenet(batch=2, res=32, width=8, blocks=((16, 1), (32, 2), (32, 1)))
    params, _ = _check(net, 0.15)
    assert len(set(params["dw2"]["e_w"].tolist())) > 1                       # genuinely per channel
