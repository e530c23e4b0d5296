"""TEST INFRASTRUCTURE, NOT PRODUCT CODE.

The paper's offline quantization procedure (Section 3) for a feed-forward list
of layers, written with the plain oracle operations of ref.py:

  * weights: threshold = max |w| per output channel (or per layer), power-of-two
    scale, round to int8;
  * activations, bootstrap fashion: layer l is measured on the output of the
    already-quantized layers before it.  Its wide integer result (after bias,
    residual and ReLU -- the threshold is taken after the ReLU) is turned back to
    float by multiplying with its scale, the maximum |value| over the calibration
    batch is the threshold gamma (or, when asked, the gamma Algorithm 1 finds on
    the histogram of abs(x)), and the output exponent is the smallest e with
    beta_max * 2^e >= gamma;
  * joins: layers concatenated into one buffer share the largest exponent of the
    group (scales of inputs to a join must match, Eq. 10); a residual input
    enters the accumulator shifted left by its scale ratio;
  * requantization factors are kept in (0, 1]: the right shift
    s[k] = e_z - e_x - e_w[k] is never negative.

The network description (a dict with "nodes" and "buffers") and the float
tensors are passed in by the caller; this module imports nothing from the CUDA
package.
"""
import numpy as np

from . import ref, threshold_ref


def _stages(nodes):
    """Consecutive nodes writing the same destination buffer form one stage."""
    out = []
    for nd in nodes:
        if out and out[-1][0]["dst"] == nd["dst"] and nd["op"] == "conv" and out[-1][0]["op"] == "conv":
            out[-1].append(nd)
        else:
            out.append([nd])
    return out


def calibrate(net, x_calib, weights, n_bits=8, rounding=0, keep_stats=False, threshold=None):
    """Returns (params, e_buf, stats): per conv node name -> dict(wq, e_w, bias_q, shift,
    res_lshift, acc_exp); per buffer name -> exponent; per node -> calibration statistics."""
    def gamma_of(st_):
        # gamma = max |x| (Section 3), or the result of Algorithm 1 on the histogram of abs(x)
        if threshold is None or not st_["maxabs"] > 0:
            return st_["maxabs"]
        return threshold_ref.threshold(st_["hist"], st_["maxabs"], n_bits, n_bits - 1, threshold)[0]

    e_buf = {}
    acts = {}
    params = {}
    stats = {}
    st_in = ref.calib_stats(x_calib)
    e_buf["input"] = ref.scale_exponent(gamma_of(st_in), n_bits)
    acts["input"] = ref.quantize_f32(x_calib, e_buf["input"], n_bits)
    if keep_stats:
        stats["input"] = st_in
    N = x_calib.shape[0]
    for stage in _stages(net["nodes"]):
        if stage[0]["op"] == "maxpool":
            nd = stage[0]
            acts[nd["dst"]] = ref.maxpool_i8(acts[nd["src"]], nd["R"], nd["S"], nd["stride"], nd["pad"])
            e_buf[nd["dst"]] = e_buf[nd["src"]]
            continue
        cands = []
        for nd in stage:
            w, b = weights[nd["name"]]
            cg = nd["C"] // nd["groups"]
            wq, e_w = ref.quantize_weights(w, K=nd["K"], R=nd["R"], S=nd["S"], Cg=cg, layout=0,
                                           per_channel=net["per_channel"], n=n_bits)
            e_x = e_buf[nd["src"]]
            bias_q = ref.quantize_bias(b, e_x, e_w)
            acc_exp = (e_x + e_w).astype(np.int32)
            res = res_lshift = None
            if nd["residual"]:
                res = acts[nd["residual"]][..., :nd["K"]]
                res_lshift = (e_buf[nd["residual"]] - acc_exp).astype(np.int32)
                assert (res_lshift >= 0).all(), "residual scale below accumulator scale"
            f = ref.qconv(acts[nd["src"]], wq, bias_q, None, res, res_lshift, acc_exp,
                          R=nd["R"], S=nd["S"], stride=(nd["stride"],) * 2, pad=(nd["pad"],) * 2,
                          groups=nd["groups"], relu=nd["relu"], out_mode=2, K=nd["K"])
            st = ref.calib_stats(f)
            if keep_stats:
                stats[nd["name"]] = st
            e_own = ref.scale_exponent(gamma_of(st), n_bits)
            cands.append(max(e_own, int(acc_exp.max())))
            params[nd["name"]] = dict(wq=wq, e_w=e_w, bias_q=bias_q, acc_exp=acc_exp,
                                      res_lshift=res_lshift)
        e_z = max(cands)
        h, w_, pitch = net["buffers"][stage[0]["dst"]]
        y = np.zeros((N, h, w_, pitch), dtype=np.int8)
        for nd in stage:
            p = params[nd["name"]]
            p["shift"] = (e_z - p["acc_exp"]).astype(np.int32)
            assert (p["shift"] >= 0).all() and (p["shift"] <= 31).all()
            res = acts[nd["residual"]][..., :nd["K"]] if nd["residual"] else None
            ref.qconv(acts[nd["src"]], p["wq"], p["bias_q"], p["shift"], res, p["res_lshift"], None,
                      R=nd["R"], S=nd["S"], stride=(nd["stride"],) * 2, pad=(nd["pad"],) * 2,
                      groups=nd["groups"], n_out=n_bits, symmetric=nd["symmetric"], relu=nd["relu"],
                      rounding=rounding, out_mode=0, K=nd["K"], out=y, out_c_offset=nd["dst_c_offset"])
        acts[stage[0]["dst"]] = y
        e_buf[stage[0]["dst"]] = e_z
    return params, e_buf, (stats if keep_stats else None), acts


def run(net, x, params, e_buf, n_bits=8, rounding=0, keep=None):
    """int8 inference with fixed parameters.  Returns {buffer name: int8 array} for
    the buffers named in `keep` (default: the last one written)."""
    acts = {"input": ref.quantize_f32(x, e_buf["input"], n_bits)}
    N = x.shape[0]
    last = "input"
    for stage in _stages(net["nodes"]):
        nd0 = stage[0]
        if nd0["op"] == "maxpool":
            acts[nd0["dst"]] = ref.maxpool_i8(acts[nd0["src"]], nd0["R"], nd0["S"], nd0["stride"],
                                              nd0["pad"])
            last = nd0["dst"]
            continue
        h, w_, pitch = net["buffers"][nd0["dst"]]
        y = np.zeros((N, h, w_, pitch), dtype=np.int8)
        for nd in stage:
            p = params[nd["name"]]
            res = acts[nd["residual"]][..., :nd["K"]] if nd["residual"] else None
            ref.qconv(acts[nd["src"]], p["wq"], p["bias_q"], p["shift"], res, p["res_lshift"], None,
                      R=nd["R"], S=nd["S"], stride=(nd["stride"],) * 2, pad=(nd["pad"],) * 2,
                      groups=nd["groups"], n_out=n_bits, symmetric=nd["symmetric"], relu=nd["relu"],
                      rounding=rounding, out_mode=0, K=nd["K"], out=y, out_c_offset=nd["dst_c_offset"])
        acts[nd0["dst"]] = y
        last = nd0["dst"]
    if keep is None:
        return {last: acts[last]}
    return {k: acts[k] for k in keep}
