"""Shared helpers of the GPU parity tests: run one layer through the C ABI and through the
oracle on the same numpy inputs."""
import numpy as np

from oracle import ref

_NP_OUT = {0: np.int8, 1: np.int32, 2: np.float32}


def gpu_conv(x, w, bias=None, shift=None, res=None, res_lshift=None, acc_exp=None, *, R, S, stride=(1, 1),
             pad=(0, 0), groups=1, n_out=8, symmetric=1, relu=0, rounding=0, out_mode=0, weight_layout=0,
             K=None, out_c_offset=0, out_c_pitch=0, algo=0, canary=77, want_handle=False, pool=0):
    import torch
    from paper_1805_07941_b200 import binding
    N, H, W, C = x.shape
    if K is None:
        K = w.shape[0] if weight_layout == 0 else w.shape[3]
    conv = binding.QConv(w, bias, shift, res_lshift, acc_exp, N=N, H=H, W=W, C=C, K=K, R=R, S=S,
                         stride_h=stride[0], stride_w=stride[1], pad_h=pad[0], pad_w=pad[1], groups=groups,
                         n_out=n_out, symmetric=symmetric, relu=relu, rounding=rounding, out_mode=out_mode,
                         out_c_offset=out_c_offset, out_c_pitch=out_c_pitch, has_residual=int(res is not None),
                         weight_layout=weight_layout, algo=algo, pool=pool)
    tdt = {0: torch.int8, 1: torch.int32, 2: torch.float32}[out_mode]
    pitch = out_c_pitch or K
    guard = 64
    Po, Qo = (conv.P // 2, conv.Q // 2) if pool else (conv.P, conv.Q)      # the layer writes the pooled tensor
    flat = torch.full((N * Po * Qo * pitch + guard,), canary, dtype=tdt, device="cuda")
    y = flat[:N * Po * Qo * pitch].view(N, Po, Qo, pitch)
    xd = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    rd = torch.from_numpy(np.ascontiguousarray(res)).cuda() if res is not None else None
    conv.run(xd, y, rd)
    st = conv.status()
    assert st == 0, (st, conv.describe())
    out = y.cpu().numpy()
    assert (flat[-guard:].cpu().numpy() == canary).all(), "write past the end of the output"
    if want_handle:
        return out, conv
    desc = conv.describe()
    conv.destroy()
    return out, desc


def oracle_conv(x, w, bias=None, shift=None, res=None, res_lshift=None, acc_exp=None, *, out_c_pitch=0,
                out_c_offset=0, canary=77, **kw):
    kw.pop("algo", None)
    if out_c_pitch:
        N, H, W, C = x.shape
        P, Q = ref.out_hw(H, W, kw["R"], kw["S"], *kw.get("stride", (1, 1)), *kw.get("pad", (0, 0)))
        out = np.full((N, P, Q, out_c_pitch), canary, dtype=_NP_OUT[kw.get("out_mode", 0)])
        return ref.qconv(x, w, bias, shift, res, res_lshift, acc_exp, out=out, out_c_offset=out_c_offset, **kw)
    return ref.qconv(x, w, bias, shift, res, res_lshift, acc_exp, **kw)


def rand_layer(rng, N, H, W, C, K, R, S, groups=1, with_bias=True, with_res=False, stride=(1, 1), pad=(0, 0),
               per_channel_shift=True, relu_like_input=False):
    x = rng.integers(0 if relu_like_input else -128, 128, size=(N, H, W, C), dtype=np.int8)
    w = rng.integers(-128, 128, size=(K, R, S, C // groups), dtype=np.int8)
    bias = rng.integers(-2**14, 2**14, size=(K,), dtype=np.int32) if with_bias else None
    kg = R * S * (C // groups)
    base = max(0, int(np.log2(max(1.0, np.sqrt(kg) * 74 * 74 / 64))))
    shift = (base + rng.integers(-1, 3, size=K)).clip(0, 31).astype(np.int32) if per_channel_shift \
        else np.full(K, base, np.int32)
    res = res_lshift = None
    if with_res:
        P, Q = ref.out_hw(H, W, R, S, stride[0], stride[1], pad[0], pad[1])
        res = rng.integers(-128, 128, size=(N, P, Q, K), dtype=np.int8)
        res_lshift = rng.integers(max(0, base - 3), base + 2, size=K).astype(np.int32)
    return x, w, bias, shift, res, res_lshift
