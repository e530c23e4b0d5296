"""GPU parity of the whole procedure: bootstrap calibration (chosen exponents and shifts must be
identical to the oracle's), int8 inference of the four network-shaped workloads, at reduced
sizes element by element and at the benchmark's full sizes on the images the oracle can afford."""
import numpy as np
import pytest

from oracle import network_ref, ref
from paper_1805_07941_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _weights(net, seed=0):
    return {nd["name"]: wl.gen_weights(nd, seed) for nd in net["nodes"] if nd["op"] == "conv"}


def _assert_same_params(qn, params, e_buf):
    assert qn.e_buf == e_buf
    for name, p in params.items():
        g = qn.params[name]
        for key in ("wq", "e_w", "bias_q", "acc_exp", "shift"):
            assert (g[key] == p[key]).all(), (name, key)
        assert (g["res_lshift"] is None) == (p["res_lshift"] is None)
        if p["res_lshift"] is not None:
            assert (g["res_lshift"] == p["res_lshift"]).all()


def _small_nets():
    inc_blocks = (("3a", 16, 24, 32, 8, 16, 16), ("pool", 0, 0, 0, 0, 0, 0), ("4a", 32, 24, 48, 8, 16, 16))
    return [wl.vgg16(batch=3, res=32, widths=(16, 32, 64), reps=(2, 2, 3)),
            wl.resnet50(batch=3, res=64, width=16, blocks=(2, 2, 1, 1)),
            wl.inception(batch=3, res=14, cin=32, blocks=inc_blocks),
            wl.mobilenet(batch=3, res=64, width=8, blocks=((16, 1), (32, 2), (32, 1), (64, 2), (64, 1)))]


@pytest.mark.parametrize("idx", range(4))
def test_small_network_calibration_and_inference(idx):
    import torch
    from paper_1805_07941_b200.network import QNetwork
    net = _small_nets()[idx]
    w = _weights(net)
    x = wl.gen_input(net, seed=0)
    params, e_buf, stats, acts = network_ref.calibrate(net, x, w, keep_stats=True)
    qn = QNetwork(net, w).calibrate(torch.from_numpy(x).cuda(), keep_stats=True)
    qn.check_status()
    _assert_same_params(qn, params, e_buf)
    # a layer that takes the 2x2 max-pool behind it inside its epilogue never writes its un-pooled output
    unwritten = {nd["src"] for nd in net["nodes"] if nd["name"] in qn._pooled}
    assert (len(unwritten) > 0) == (idx == 0), unwritten      # the VGG-shaped net has such pools, the others none
    for name, a in acts.items():
        if name not in unwritten:
            assert (qn.bufs[name].cpu().numpy() == a).all(), name
    if unwritten:                                             # and with the pools as calls of their own: every buffer
        qn0 = QNetwork(net, w, fuse_pool=False).calibrate(torch.from_numpy(x).cuda())
        assert not qn0._pooled
        for name, a in acts.items():
            assert (qn0.bufs[name].cpu().numpy() == a).all(), name
        qn0.destroy()
    for name, st in stats.items():
        g = qn.stats[name]
        assert g["maxabs"] == st["maxabs"] and (g["hist"] == st["hist"]).all(), name
        assert g["count"] == st["count"] and g["nonfinite"] == st["nonfinite"] == 0
        assert abs(g["sum"] - st["sum"]) <= 1e-6 * max(1.0, abs(st["sum"]))
        assert abs(g["sumsq"] - st["sumsq"]) <= 1e-6 * max(1.0, st["sumsq"])
    # a different batch through plain launches and through the captured graph
    x2 = wl.gen_input(net, seed=5)
    want = network_ref.run(net, x2, params, e_buf)[qn.last]
    got = qn.run(torch.from_numpy(x2).cuda()).cpu().numpy()
    assert (got == want).all()
    qn.capture()
    got = qn.run(torch.from_numpy(x2).cuda())
    torch.cuda.synchronize()
    assert (got.cpu().numpy() == want).all()
    # the pipelined end-to-end call: three different batches in pinned host memory
    xs = [wl.gen_input(net, seed=s_) for s_ in (5, 6, 7)]
    outs = [torch.empty(qn.bufs[qn.last].shape, dtype=torch.int8).pin_memory() for _ in xs]
    qn.run_pipelined([torch.from_numpy(a).pin_memory() for a in xs], outs)
    torch.cuda.synchronize()
    for a, o in zip(xs, outs):
        assert (o.numpy() == network_ref.run(net, a, params, e_buf)[qn.last]).all()
    # a smaller batch than the maximum
    got = qn.run(torch.from_numpy(x2[:2]).cuda()).cpu().numpy()
    assert (got == want[:2]).all()
    # parameters chosen by the oracle, loaded as they are
    qn2 = QNetwork(net, w).load_params(params, e_buf)
    assert (qn2.run(torch.from_numpy(x2).cuda()).cpu().numpy() == want).all()
    qn.destroy()
    qn2.destroy()


def test_resnet_with_the_stride_on_the_3x3_layer_runs_on_the_tensor_cores():
    """The later variant of the network strides in the 3x3 layer of a stage's first block: those layers
    take the strided-box form of the tensor-core kernel (no CUDA-core plan anywhere), bit-exact."""
    import torch
    from paper_1805_07941_b200.network import QNetwork
    net = wl.resnet50(batch=3, res=64, width=16, blocks=(2, 2, 1, 1), stride_on_3x3=True)
    w = _weights(net)
    x = wl.gen_input(net, seed=0)
    params, e_buf, _, acts = network_ref.calibrate(net, x, w)
    qn = QNetwork(net, w).calibrate(torch.from_numpy(x).cuda())
    qn.check_status()
    _assert_same_params(qn, params, e_buf)
    for name, a in acts.items():
        assert (qn.bufs[name].cpu().numpy() == a).all(), name
    plans = {name: h.describe() for name, h in qn.handles.items()}
    assert all(p.startswith("igemm") for p in plans.values()), plans
    strided = [nd["name"] for nd in net["nodes"] if nd["op"] == "conv" and nd["R"] == 3 and nd["stride"] == 2]
    assert len(strided) == 3 and all("igemm/box" in plans[n] for n in strided)
    qn.destroy()


@pytest.mark.parametrize("idx,measure", [(0, "ks"), (1, "cvm"), (3, "kl"), (3, "l1")])
def test_small_network_with_searched_thresholds(idx, measure):
    """gamma from Algorithm 1 instead of the maximum: both sides must pick the same exponents (the
    exponent only moves when gamma crosses 127 * 2^e, far coarser than the search's tolerance)."""
    import torch
    from paper_1805_07941_b200.network import QNetwork
    net = _small_nets()[idx]
    w = _weights(net)
    x = wl.gen_input(net, seed=0)
    params, e_buf, _, acts = network_ref.calibrate(net, x, w, threshold=measure)
    _, e_max, _, _ = network_ref.calibrate(net, x, w)
    assert any(e_buf[k] < e_max[k] for k in e_buf), "the search never clipped anything: test is vacuous"
    qn = QNetwork(net, w).calibrate(torch.from_numpy(x).cuda(), threshold=measure)
    qn.check_status()
    _assert_same_params(qn, params, e_buf)
    unwritten = {nd["src"] for nd in net["nodes"] if nd["name"] in qn._pooled}     # pools taken inside a layer
    for name, a in acts.items():
        if name not in unwritten:
            assert (qn.bufs[name].cpu().numpy() == a).all(), name
    qn.destroy()


FULL = [("resnet50", lambda: wl.resnet50(batch=32), 2, (0, 1, 31)),
        ("vgg16", lambda: wl.vgg16(batch=64), 1, (0, 63)),
        ("inception", lambda: wl.inception(batch=128), 2, (0, 1, 127)),
        ("mobilenet", lambda: wl.mobilenet(batch=256), 2, (0, 1, 255))]


@pytest.mark.parametrize("name,make,ncal,check", FULL, ids=[f[0] for f in FULL])
def test_full_size_network(name, make, ncal, check):
    """Calibrate on the first `ncal` images (the paper calibrates on a handful of images and deploys
    on everything), on both sides; then run the full benchmark batch through the captured graph and
    compare every buffer-final value of the images the oracle recomputes."""
    import torch
    from paper_1805_07941_b200.network import QNetwork
    net = make()
    w = _weights(net)
    x = wl.gen_input(net, seed=0)
    params, e_buf, _, acts = network_ref.calibrate(net, x[:ncal], w)
    qn = QNetwork(net, w).calibrate(torch.from_numpy(x[:ncal]).cuda())
    qn.check_status()
    _assert_same_params(qn, params, e_buf)
    assert (qn.bufs[qn.last][:ncal].cpu().numpy() == acts[qn.last]).all()
    qn.capture()
    got = qn.run(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    qn.check_status()
    got = got.cpu().numpy()
    for i in check:
        want = acts[qn.last][i] if i < ncal else network_ref.run(net, x[i:i + 1], params, e_buf)[qn.last][0]
        assert (got[i] == want).all(), (name, i)
    assert np.abs(got).max() >= 32 and (got != 0).mean() > 0.02          # not a degenerate all-zero output
    qn.destroy()


def _sample_points(rng, N, P, Q, K, count):
    pts = np.stack([rng.integers(0, N, count), rng.integers(0, P, count), rng.integers(0, Q, count),
                    rng.integers(0, K, count)], axis=1).astype(np.int32)
    # always include the corners and the last image / channel
    pts[:8] = [[0, 0, 0, 0], [N - 1, P - 1, Q - 1, K - 1], [N - 1, 0, Q - 1, 0], [0, P - 1, 0, K - 1],
               [N // 2, P // 2, Q // 2, K // 2], [N - 1, P - 1, 0, 0], [0, 0, Q - 1, K - 1], [N - 1, 0, 0, K - 1]]
    return pts


LAYER_PICKS = [("vgg16", lambda: wl.vgg16(batch=64), ("conv1_1", "conv1_2", "conv3_2", "conv5_3")),
               ("resnet50", lambda: wl.resnet50(batch=32), ("stem", "s0b0_a", "s0b0_c", "s1b0_a", "s2b0_b",
                                                            "s3b0_prj", "s3b2_c")),
               ("inception", lambda: wl.inception(batch=128), ("3a_5x5", "4d_3x3", "4b_5r", "5b_1x1")),
               ("mobilenet", lambda: wl.mobilenet(batch=256), ("stem", "dw1", "dw2", "pw1", "dw12", "pw13"))]


@pytest.mark.parametrize("name,make,layers", LAYER_PICKS, ids=[f[0] for f in LAYER_PICKS])
def test_full_size_layers_on_sampled_outputs(name, make, layers):
    """Stand-alone layers at the benchmark's batch and launch shape, fed seeded int8 activations;
    the oracle recomputes a few thousand sampled outputs one by one."""
    import torch
    from paper_1805_07941_b200 import binding
    net = make()
    N = net["input"][0]
    for nd in net["nodes"]:
        if nd["op"] != "conv" or nd["name"] not in layers:
            continue
        rng = np.random.default_rng(nd["tid"])
        x = wl.gen_activation_i8((N, nd["H"], nd["W"], nd["C"]), 0, nd["tid"] + 2, relu_like=nd["name"] != "stem")
        cg = nd["C"] // nd["groups"]
        wq = rng.integers(-128, 128, size=(nd["K"], nd["R"], nd["S"], cg), dtype=np.int8)
        bias = rng.integers(-2**12, 2**12, size=nd["K"]).astype(np.int32)
        kg = nd["R"] * nd["S"] * cg
        shift = (int(np.log2(max(2.0, np.sqrt(kg) * 74 * 26 / 48))) + rng.integers(0, 2, nd["K"])).astype(np.int32)
        res = t = None
        if nd["residual"]:
            res = wl.gen_activation_i8((N, nd["P"], nd["Q"], nd["K"]), 0, nd["tid"] + 3)
            t = (shift - 1).clip(0, 23).astype(np.int32)
        pitch = net["buffers"][nd["dst"]][2]
        conv = binding.QConv(wq, bias, shift, t, None, N=N, H=nd["H"], W=nd["W"], C=nd["C"], K=nd["K"], R=nd["R"],
                             S=nd["S"], stride_h=nd["stride"], stride_w=nd["stride"], pad_h=nd["pad"],
                             pad_w=nd["pad"], groups=nd["groups"], relu=nd["relu"], symmetric=nd["symmetric"],
                             out_c_offset=nd["dst_c_offset"], out_c_pitch=pitch, has_residual=int(res is not None))
        y = torch.full((N, nd["P"], nd["Q"], pitch), 99, dtype=torch.int8, device="cuda")
        conv.run(torch.from_numpy(x).cuda(), y, None if res is None else torch.from_numpy(res).cuda())
        assert conv.status() == 0
        pts = _sample_points(rng, N, nd["P"], nd["Q"], nd["K"], 4000)
        want = ref.qconv_points(x, wq, pts, bias, shift, res, t, R=nd["R"], S=nd["S"], stride=(nd["stride"],) * 2,
                                pad=(nd["pad"],) * 2, groups=nd["groups"], relu=nd["relu"],
                                symmetric=nd["symmetric"])
        yc = y.cpu().numpy()
        got = yc[pts[:, 0], pts[:, 1], pts[:, 2], nd["dst_c_offset"] + pts[:, 3]]
        assert (got == want).all(), (nd["name"], conv.describe())
        assert 0.02 < (want != 0).mean() and (want == 127).mean() < 0.9, nd["name"]
        # channels of the concat buffer that belong to other branches are untouched
        if pitch > nd["K"]:
            other = np.ones(pitch, bool)
            other[nd["dst_c_offset"]:nd["dst_c_offset"] + nd["K"]] = False
            assert (yc[..., other] == 99).all()
        conv.destroy()
        del y


@pytest.mark.parametrize("idx", [1, 2])
def test_branches_on_streams_give_the_same_activations(idx):
    """Residual and inception networks: the pass with independent branches on streams of their own
    (plain launches, and captured) must leave every buffer exactly as the one-stream pass does."""
    import torch
    from paper_1805_07941_b200.network import QNetwork
    net = _small_nets()[idx]
    w = _weights(net)
    qn = QNetwork(net, w).calibrate(torch.from_numpy(wl.gen_input(net, seed=0)).cuda())
    deps = qn._dependencies()
    assert any(len(d) > 1 for d in deps)                       # there are joins, hence branches
    x2 = torch.from_numpy(wl.gen_input(net, seed=9)).cuda()
    qn.x_static.copy_(x2)
    qn.forward_static()
    torch.cuda.synchronize()
    serial = {k: v.clone() for k, v in qn.bufs.items()}
    for mode in ("plain", "plain split", "branches", "chain", "split2", None):
        for v in qn.bufs.values():
            v.zero_()                        # nothing stale can pass (padding channels must stay zero)
        if mode == "plain":
            qn.forward_branches()
        elif mode == "plain split":
            qn.forward_split(3)              # batch 3: one image per chain
        else:
            if mode == "split2":
                continue                     # needs an even batch: covered by the benchmark-size test
            qn.capture(mode)
            qn.graph.replay()
        torch.cuda.synchronize()
        qn.check_status()
        for k, v in serial.items():
            if k == "input":
                continue                     # a stem that converts the float input itself leaves it unwritten
            assert torch.equal(qn.bufs[k], v), (mode, k)


def test_two_half_batch_chains_match_the_oracle():
    """The "split2" graph form (two half-batches, each a chain on its own stream with its own layer
    handles) on an even batch: same output as the oracle, and as the single chain."""
    import torch
    from paper_1805_07941_b200.network import QNetwork
    net = wl.resnet50(batch=4, res=64, width=16, blocks=(2, 1, 1, 1))
    w = _weights(net)
    x = wl.gen_input(net, seed=0)
    params, e_buf, _, _ = network_ref.calibrate(net, x, w)
    qn = QNetwork(net, w).calibrate(torch.from_numpy(x).cuda())
    _assert_same_params(qn, params, e_buf)
    x2 = wl.gen_input(net, seed=3)
    want = network_ref.run(net, x2, params, e_buf)[qn.last]
    for form in ("split2", "chain", None):
        qn.capture(form)
        for v in qn.bufs.values():
            v.zero_()
        got = qn.run(torch.from_numpy(x2).cuda())
        torch.cuda.synchronize()
        qn.check_status()
        assert (got.cpu().numpy() == want).all(), form
    assert set(qn.graph_timings) == {"chain", "branches", "split2"}
    qn.destroy()


def _sync_worker(rank, world, port, threshold, q):
    """One of two ranks that share GPU 0 and exchange statistics over gloo (host tensors): each
    calibrates on its shard of the batch with sync=True."""
    import os
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    import torch
    import torch.distributed as dist
    from paper_1805_07941_b200 import dist as qd, workloads as wl_
    from paper_1805_07941_b200.network import QNetwork
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    net = wl_.resnet50(batch=4, res=64, width=16, blocks=(2, 1, 1, 1))
    w = {nd["name"]: wl_.gen_weights(nd, 0) for nd in net["nodes"] if nd["op"] == "conv"}
    x = wl_.gen_input(net, seed=0)
    lo, hi = qd.shard_range(x.shape[0], rank, world)
    qn = QNetwork(net, w).calibrate(torch.from_numpy(x[lo:hi]).cuda(), sync=True, threshold=threshold)
    qn.check_status()
    out = (rank, dict(qn.e_buf), {k: {kk: (None if vv is None else vv.tolist()) for kk, vv in v.items() if kk != "wq"}
                                  for k, v in qn.params.items()})
    qn.destroy()
    dist.destroy_process_group()
    q.put(out)


@pytest.mark.parametrize("threshold", [None, "l1"])
def test_calibration_batch_split_over_two_ranks(threshold):
    """The calibration batch split over two ranks (statistics combined before every exponent is chosen)
    must give both ranks the network the oracle derives from the whole batch."""
    import socket
    import torch.multiprocessing as mp
    net = wl.resnet50(batch=4, res=64, width=16, blocks=(2, 1, 1, 1))
    w = _weights(net)
    x = wl.gen_input(net, seed=0)
    params, e_buf, _, _ = network_ref.calibrate(net, x, w, threshold=threshold)
    with socket.socket() as s_:
        s_.bind(("127.0.0.1", 0))
        port = s_.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_sync_worker, args=(r, 2, port, threshold, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=600) for _ in range(2)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for _, got_e, got_p in res:
        assert got_e == e_buf
        for name, p in params.items():
            for key in ("e_w", "bias_q", "acc_exp", "shift", "res_lshift"):
                want = None if p[key] is None else np.asarray(p[key]).tolist()
                assert got_p[name][key] == want, (name, key)
