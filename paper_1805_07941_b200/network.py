"""Driver of the offline quantization procedure (Section 3 of the paper) and of int8
inference for a feed-forward list of layers, on the GPU through the C ABI.

This file only sequences library calls: every arithmetic step -- weight/bias conversion
(`qquantize_weights`, `qquantize_bias`), float-out convolution, statistics
(`qcalib_collect`), exponent choice (`qscale_exponent`), int8 convolution, pooling, input
conversion -- runs inside the library.  The bookkeeping it does is the paper's:
  * bootstrap calibration: a layer is measured on the output of the already-quantized layers
    before it, after its ReLU;
  * layers concatenated into one buffer share the largest output exponent of the group;
  * a residual input enters the accumulator shifted left by e_res - (e_x + e_w[k]);
  * right shifts s[k] = e_z - e_x - e_w[k] are never negative (factors in (0, 1]).
"""
import numpy as np
import torch

from . import binding
from . import dist as qdist


def _stages(nodes):
    """Runs of consecutive nodes that are calibrated together: convolutions writing into one buffer
    (the branches of a concatenation) form one run, everything else stands alone."""
    import itertools
    runs, serial = [], itertools.count()
    key = lambda nd: ("join", nd["dst"]) if nd["op"] == "conv" else ("single", next(serial))
    for _, grp in itertools.groupby(nodes, key=key):
        runs.append(list(grp))
    return runs


class QNetwork:
    def __init__(self, net, weights, n_bits=8, rounding=0, device="cuda", fuse_pool=True):
        """net: description from workloads.py; weights: {conv name: (w [K,R,S,C/g] float32, bias [K])}."""
        self.net = net
        self.weights = weights
        self.n_bits = n_bits
        self.rounding = rounding
        self.device = torch.device(device)
        self.N = net["input"][0]
        self.e_buf = {}
        self.params = {}
        self.stats = {}
        self.handles = {}
        self.bufs = {}
        self.graph = None
        self.stages = _stages(net["nodes"])
        for name, (h, w, pitch) in net["buffers"].items():
            if name == "input":
                continue
            self.bufs[name] = torch.zeros((self.N, h, w, pitch), dtype=torch.int8, device=self.device)
        n, h, w, c = net["input"]
        self.bufs["input"] = torch.zeros((n, h, w, c), dtype=torch.int8, device=self.device)
        self.x_static = torch.zeros((n, h, w, c), dtype=torch.float32, device=self.device)
        self.last = net["nodes"][-1]["dst"]
        # A 2x2 / stride-2 max-pool that is the only reader of a convolution's own output buffer can be taken
        # inside that layer (qconv_desc.pool): candidates here, the library decides when the handle is built.
        self.fuse_pool = fuse_pool
        self._pool_after = {}
        nodes = net["nodes"]
        for nd in nodes:
            if nd["op"] != "maxpool" or (nd["R"], nd["S"], nd["stride"], nd["pad"]) != (2, 2, 2, 0):
                continue
            writers = [c for c in nodes if c["dst"] == nd["src"]]
            readers = [c for c in nodes if c["src"] == nd["src"] or c.get("residual") == nd["src"]]
            if len(writers) == 1 and writers[0]["op"] == "conv" and readers == [nd] and nd["src"] != self.last and \
                    not writers[0]["residual"] and net["buffers"][nd["src"]][2] == writers[0]["K"]:
                self._pool_after[writers[0]["name"]] = nd
        self._pooled = set()                       # names of the pool nodes whose work a convolution has taken over

    # ------------------------------------------------------------------ helpers
    def _geom(self, nd, N=None):
        return dict(N=self.N if N is None else N, H=nd["H"], W=nd["W"], C=nd["C"], K=nd["K"], R=nd["R"], S=nd["S"],
                    stride_h=nd["stride"], stride_w=nd["stride"], pad_h=nd["pad"], pad_w=nd["pad"],
                    groups=nd["groups"], relu=nd["relu"], n_in=self.n_bits, n_w=self.n_bits,
                    n_out=self.n_bits, rounding=self.rounding)

    def _make_handle(self, nd, N=None, register=True):
        """The int8 handle of a convolution from self.params; with a fusable pool behind it, the handle that pools
        inside the layer and writes the pool's buffer (when the library takes the shape)."""
        p = self.params[nd["name"]]
        common = dict(symmetric=nd["symmetric"], has_residual=int(p["res_lshift"] is not None), **self._geom(nd, N))
        args = (p["wq"], p["bias_q"], p["shift"], p["res_lshift"], None)
        pool = self._pool_after.get(nd["name"]) if self.fuse_pool else None
        if pool is not None:
            try:
                h = binding.QConv(*args, pool=2, out_c_offset=pool.get("dst_c_offset", 0),
                                  out_c_pitch=self.net["buffers"][pool["dst"]][2], **common)
                if register:
                    self._pooled.add(pool["name"])
                return h
            except binding.QconvError as err:
                if err.code != binding.ERR_UNSUPPORTED_SHAPE:
                    raise
        if register and pool is not None:
            self._pooled.discard(pool["name"])
        return binding.QConv(*args, out_c_offset=nd["dst_c_offset"], out_c_pitch=self.net["buffers"][nd["dst"]][2], **common)

    def _conv_dst(self, nd):
        """Buffer a convolution writes: its own, or the pool's when it pools inside the layer."""
        pool = self._pool_after.get(nd["name"])
        return self.bufs[pool["dst"] if pool is not None and pool["name"] in self._pooled else nd["dst"]]

    def _residual(self, nd):
        if not nd["residual"]:
            return None
        r = self.bufs[nd["residual"]]
        assert r.shape[3] == nd["K"], "residual buffer pitch must equal K"
        return r

    # ------------------------------------------------------------------ calibration
    def calibrate(self, x_calib, nbins=2048, keep_stats=False, group=None, sync=False, threshold=None):
        """x_calib: float32 [n, H, W, C] CUDA tensor, n <= N.  Chooses every exponent and builds the
        int8 layer handles; leaves the int8 activations of the calibration batch in self.bufs.
        With sync=True under torch.distributed, x_calib is this rank's shard of the calibration batch:
        the statistics of every tensor are combined over the ranks before its exponent is chosen, so
        all ranks end up with the same network.
        threshold: None takes gamma = max |x| for every activation tensor; "l1", "ks", "cvm" or "kl"
        takes the gamma that Algorithm 1 finds on the tensor's histogram with that measure."""
        n = x_calib.shape[0]

        def gamma_of(st_):
            if threshold is None or not st_["maxabs"] > 0:
                return st_["maxabs"]
            return binding.qthreshold_search(st_["hist"], st_["maxabs"], self.n_bits, self.n_bits - 1, threshold)[0]

        # the few bytes that are exchanged travel as device tensors under NCCL, as host tensors otherwise
        red_dev = "cpu"
        if sync and torch.distributed.is_initialized() and torch.distributed.get_backend(group) == "nccl":
            red_dev = self.device

        def collect(t):
            if not sync:
                return binding.qcalib_collect(t, nbins)
            if threshold is None:                            # only the maximum matters: one pass, no histogram sum
                return qdist.allreduce_calib(binding.qcalib_collect(t, nbins), group, device=red_dev)
            return qdist.collect_synced(lambda hi: binding.qcalib_collect(t, nbins, hi), group, device=red_dev)

        st = collect(x_calib)
        if keep_stats:
            self.stats["input"] = st
        self.e_buf["input"] = binding.qscale_exponent(gamma_of(st), self.n_bits)
        binding.qquantize_f32(x_calib, self.e_buf["input"], self.n_bits, out=self.bufs["input"][:n])
        fbuf = None
        for stage in self.stages:
            nd0 = stage[0]
            if nd0["op"] == "maxpool":
                if nd0["name"] not in self._pooled:
                    binding.qmaxpool_i8(self.bufs[nd0["src"]][:n], nd0["R"], nd0["S"], nd0["stride"], nd0["pad"],
                                        out=self.bufs[nd0["dst"]][:n])
                self.e_buf[nd0["dst"]] = self.e_buf[nd0["src"]]
                continue
            cands = []
            for nd in stage:
                w, b = self.weights[nd["name"]]
                cg = nd["C"] // nd["groups"]
                wq, e_w = binding.qquantize_weights(w, nd["K"], nd["R"], nd["S"], cg, 0,
                                                    self.net["per_channel"], self.n_bits)
                e_x = self.e_buf[nd["src"]]
                bias_q = binding.qquantize_bias(b, e_x, e_w)
                acc_exp = binding.qacc_exponents(e_x, e_w)
                res_lshift = None
                if nd["residual"]:
                    res_lshift = binding.qresidual_shifts(self.e_buf[nd["residual"]], acc_exp)
                need = n * nd["P"] * nd["Q"] * nd["K"]
                if fbuf is None or fbuf.numel() < need:
                    fbuf = None
                    fbuf = torch.empty(need, dtype=torch.float32, device=self.device)
                fl = binding.QConv(wq, bias_q, None, res_lshift, acc_exp, out_mode=binding.OUT_FLOAT,
                                   has_residual=int(res_lshift is not None), **self._geom(nd))
                res = self._residual(nd)
                fl.run(self.bufs[nd["src"]], fbuf, None if res is None else res, n_run=n)
                st = collect(fbuf[:need])
                fl.destroy()
                if keep_stats:
                    self.stats[nd["name"]] = st
                cands.append(binding.qscale_exponent(gamma_of(st), self.n_bits))
                self.params[nd["name"]] = dict(wq=wq, e_w=e_w, bias_q=bias_q, acc_exp=acc_exp,
                                               res_lshift=res_lshift)
            e_z = binding.qjoin_exponent(cands, [self.params[nd["name"]]["acc_exp"] for nd in stage])
            for nd in stage:
                p = self.params[nd["name"]]
                p["shift"] = binding.qrequant_shifts(e_z, p["acc_exp"])
                if nd["name"] in self.handles:
                    self.handles[nd["name"]].destroy()
                hnd = self._make_handle(nd)
                self.handles[nd["name"]] = hnd
                hnd.run(self.bufs[nd["src"]], self._conv_dst(nd), self._residual(nd), n_run=n)
            self.e_buf[nd0["dst"]] = e_z
        torch.cuda.synchronize()
        self.graph = None
        if hasattr(self, "_fused_name"):
            del self._fused_name
        return self

    def load_params(self, params, e_buf):
        """Build the int8 handles from parameters chosen elsewhere (same keys as self.params)."""
        self.params = params
        self.e_buf = dict(e_buf)
        for nd in self.net["nodes"]:
            if nd["op"] != "conv":
                continue
            self.handles[nd["name"]] = self._make_handle(nd)
        self.graph = None
        if hasattr(self, "_fused_name"):
            del self._fused_name
        return self

    # ------------------------------------------------------------------ inference
    def _fused_input(self):
        """Name of the layer that takes the float input itself (its packing kernel converts on the
        way, `qconv_run_f32`), or None: the only reader of the input must be a stem that repacks its
        input (space-to-depth at stride 2, padded rows at stride 1)."""
        if not hasattr(self, "_fused_name"):
            readers = [nd for nd in self.net["nodes"] if nd["src"] == "input" or nd.get("residual") == "input"]
            self._fused_name = None
            if len(readers) == 1 and readers[0]["op"] == "conv" and readers[0]["src"] == "input":
                plan = self.handles[readers[0]["name"]].describe()
                if "igemm/s2d" in plan or ("igemm/wrow" in plan and readers[0]["C"] <= 4):
                    self._fused_name = readers[0]["name"]
        return self._fused_name

    def _convert_input(self, sl):
        if self._fused_input() is None:
            binding.qquantize_f32(self.x_static[sl], self.e_buf["input"], self.n_bits, out=self.bufs["input"][sl])

    def _run_node(self, nd, sl, handles=None):
        """One layer on the images of slice sl, with the given set of handles (default: the full-batch set)."""
        n = sl.stop - sl.start
        if nd["op"] == "maxpool":
            if nd["name"] not in self._pooled:
                binding.qmaxpool_i8(self.bufs[nd["src"]][sl], nd["R"], nd["S"], nd["stride"], nd["pad"],
                                    out=self.bufs[nd["dst"]][sl])
            return
        h = (self.handles if handles is None else handles)[nd["name"]]
        res = self._residual(nd)
        res = None if res is None else res[sl]
        dst = self._conv_dst(nd)[sl]
        if nd["name"] == self._fused_input():
            h.run_f32(self.x_static[sl], self.e_buf["input"], dst, res, n_run=n)
        else:
            h.run(self.bufs[nd["src"]][sl], dst, res, n_run=n)

    def _forward_layers(self, n):
        for nd in self.net["nodes"]:
            self._run_node(nd, slice(0, n))

    def _dependencies(self):
        """For every node, the earlier nodes it must follow: writers of what it reads (input or
        residual buffer), and, for the buffer it writes, earlier readers and earlier writers of an
        overlapping channel window (layers of a concat group write disjoint windows and stay
        independent).  -1 stands for the input conversion."""
        nodes = self.net["nodes"]
        writers, readers, deps = {"input": [(-1, 0, 1 << 30)]}, {}, []
        for i, nd in enumerate(nodes):
            d = set()
            reads = [nd["src"]] + ([nd["residual"]] if nd.get("residual") else [])
            for b in reads:
                d.update(w for w, _, _ in writers.get(b, []))
            lo = nd.get("dst_c_offset", 0)
            hi = lo + (nd["K"] if nd["op"] == "conv" else 1 << 30)
            d.update(readers.get(nd["dst"], []))
            d.update(w for w, wl, wh in writers.get(nd["dst"], []) if wl < hi and lo < wh)
            for b in reads:
                readers.setdefault(b, []).append(i)
            writers.setdefault(nd["dst"], []).append((i, lo, hi))
            d.discard(i)
            deps.append(sorted(d))
        return deps

    def forward_branches(self, n=None, max_streams=4):
        """The same pass as forward_static with independent branches (the projection shortcut beside
        the main path of a residual block, the four branches of an inception block) on streams of
        their own: most layers here fill the GPU for less than two waves of tiles, so branches that
        run side by side hide each other's latency.  A layer continues on the stream of the latest
        layer it depends on when that stream has not moved on (consecutive launches of one stream
        keep their programmatic dependency); other dependencies become event waits.  Everything
        joins the current stream at the end, so the call can be captured into a CUDA graph."""
        n = self.N if n is None else n
        main = torch.cuda.current_stream()
        if not hasattr(self, "_side"):
            self._side = [torch.cuda.Stream() for _ in range(max(0, max_streams - 1))]
        streams = [main] + self._side[:max(0, max_streams - 1)]
        deps = self._dependencies()
        self._convert_input(slice(0, n))
        tail = [-1] + [None] * (len(streams) - 1)          # last node launched on each stream
        where, done = {-1: 0}, {}
        done[-1] = torch.cuda.Event()
        done[-1].record(main)
        nodes = self.net["nodes"]
        last_use = {}
        for i, d in enumerate(deps):
            for j in d:
                last_use[j] = i
        for i, nd in enumerate(nodes):
            d = deps[i]
            # continue the stream whose tail is the latest of my dependencies, else take a stream
            # whose tail nobody waits for any more (or that was never used), else stay on the main one
            cont = [si for si in range(len(streams)) if tail[si] is not None and tail[si] in d]
            if cont:
                si = max(cont, key=lambda k: tail[k])
            else:
                free = [k for k in range(1, len(streams)) if tail[k] is None or last_use.get(tail[k], -1) < i]
                si = free[0] if free else 0
            st = streams[si]
            for j in d:
                if where[j] != si:
                    st.wait_event(done[j])
            with torch.cuda.stream(st):
                self._run_node(nd, slice(0, n))
                done[i] = torch.cuda.Event()
                done[i].record(st)
            tail[si], where[i] = i, si
        for si in range(1, len(streams)):
            if tail[si] is not None:
                main.wait_event(done[tail[si]])
        return self.bufs[self.last][:n]

    def _part_handles(self, parts):
        """Layer handles for a batch cut into `parts` equal slices: one set per slice (a handle owns
        scratch and cached tensor maps, so slices that run side by side cannot share one)."""
        if not hasattr(self, "_parts"):
            self._parts = {}
        if parts not in self._parts:
            n_sub = self.N // parts
            sets = []
            for _ in range(parts):
                hs = {}
                for nd in self.net["nodes"]:
                    if nd["op"] != "conv":
                        continue
                    hs[nd["name"]] = self._make_handle(nd, n_sub, register=False)
                sets.append(hs)
            self._parts[parts] = sets
        return self._parts[parts]

    def forward_split(self, parts=2):
        """The full batch as `parts` slices of images, each slice a chain of its own on its own stream.
        Images are independent, so the chains need no synchronisation until the end; while one chain
        sits in a layer's launch, set-up or tail, the other one's layer has the SMs.  Pays when the
        layers of the full batch fill the GPU for only a wave or two of tiles."""
        assert self.N % parts == 0
        n_sub = self.N // parts
        sets = self._part_handles(parts)
        main = torch.cuda.current_stream()
        if not hasattr(self, "_side"):
            self._side = []
        while len(self._side) < parts - 1:
            self._side.append(torch.cuda.Stream())
        start = torch.cuda.Event()
        start.record(main)
        ends = []
        for k in range(parts):
            st = main if k == 0 else self._side[k - 1]
            sl = slice(k * n_sub, (k + 1) * n_sub)
            if k:
                st.wait_event(start)
            with torch.cuda.stream(st):
                self._convert_input(sl)
                for nd in self.net["nodes"]:
                    self._run_node(nd, sl, sets[k])
                if k:
                    ev = torch.cuda.Event()
                    ev.record(st)
                    ends.append(ev)
        for ev in ends:
            main.wait_event(ev)
        return self.bufs[self.last]

    def forward_static(self, n=None):
        """Input conversion + every layer on self.x_static[:n]; asynchronous on the current stream."""
        n = self.N if n is None else n
        self._convert_input(slice(0, n))
        self._forward_layers(n)
        return self.bufs[self.last][:n]

    def _capture_one(self, how):
        fwd = {"chain": self.forward_static, "branches": self.forward_branches,
               "split2": lambda: self.forward_split(2)}[how]
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            fwd()                                       # warm-up outside capture: tensor maps get cached
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fwd()
        return g

    def capture(self, how=None):
        """Record one pass over the full batch into a CUDA graph (launch overhead of the few dozen
        small kernels otherwise dominates).  how = "chain": one stream, layer after layer; "branches":
        independent branches on streams of their own (forward_branches), parallel paths of the graph;
        "split2": the batch as two half-batches, two independent chains side by side (forward_split).
        None (default) records every form that applies, replays each a few times and keeps the fastest:
        side-by-side work pays when layers leave SMs idle and costs a little when every layer fills the
        GPU anyway."""
        if how is None:
            cands = ["chain"]
            if any(len(d) > 1 for d in self._dependencies()):
                cands.append("branches")
            if self.N % 2 == 0 and self.N >= 2:
                cands.append("split2")
            timed = []
            for c in cands:
                g = self._capture_one(c)
                for _ in range(3):
                    g.replay()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(10):
                    g.replay()
                e1.record()
                torch.cuda.synchronize()
                timed.append((e0.elapsed_time(e1), c, g))
            timed.sort(key=lambda t: t[0])
            self.graph, self.graph_form = timed[0][2], timed[0][1]
            self.graph_timings = {c: t / 10 for t, c, _ in timed}
            return self.graph
        self.graph = self._capture_one(how)
        self.graph_form = how
        return self.graph

    def run(self, x):
        """x: float32 [n, H, W, C] CUDA tensor.  Returns the int8 output buffer (a view)."""
        n = x.shape[0]
        self.x_static[:n].copy_(x)
        if self.graph is not None and n == self.N:
            self.graph.replay()
            return self.bufs[self.last]
        return self.forward_static(n)

    def run_pipelined(self, host_batches, host_outputs):
        """End-to-end inference of a sequence of batches that live in pinned host memory.
        host_batches: list of pinned float32 CPU tensors [N, H, W, C]; host_outputs: list of pinned int8
        CPU tensors shaped like the network output, one per batch.  Host-to-device copies, compute and
        device-to-host copies run on three streams with double buffers, so the copy of batch i+1 and
        the read-back of batch i-1 overlap the layers of batch i.  Returns after everything finished."""
        assert self.graph is not None, "capture() first"
        if not hasattr(self, "_pipe"):
            self._pipe = dict(
                h2d=torch.cuda.Stream(), d2h=torch.cuda.Stream(),
                xin=[torch.empty_like(self.x_static) for _ in range(2)],
                yout=[torch.empty_like(self.bufs[self.last]) for _ in range(2)])
        pp = self._pipe
        comp = torch.cuda.current_stream()
        in_ready = [None, None]      # H2D of the batch in slot s finished
        in_free = [None, None]       # compute has consumed slot s
        out_ready = [None, None]     # result sits in yout[s]
        out_free = [None, None]      # D2H has drained yout[s]
        pp["h2d"].wait_stream(comp)
        pp["d2h"].wait_stream(comp)
        for i, (xb, yb) in enumerate(zip(host_batches, host_outputs)):
            s = i & 1
            with torch.cuda.stream(pp["h2d"]):
                if in_free[s] is not None:
                    pp["h2d"].wait_event(in_free[s])
                pp["xin"][s].copy_(xb, non_blocking=True)
                in_ready[s] = torch.cuda.Event()
                in_ready[s].record(pp["h2d"])
            comp.wait_event(in_ready[s])
            self.x_static.copy_(pp["xin"][s], non_blocking=True)
            in_free[s] = torch.cuda.Event()
            in_free[s].record(comp)
            self.graph.replay()
            if out_free[s] is not None:
                comp.wait_event(out_free[s])
            pp["yout"][s].copy_(self.bufs[self.last], non_blocking=True)
            out_ready[s] = torch.cuda.Event()
            out_ready[s].record(comp)
            with torch.cuda.stream(pp["d2h"]):
                pp["d2h"].wait_event(out_ready[s])
                yb.copy_(pp["yout"][s], non_blocking=True)
                out_free[s] = torch.cuda.Event()
                out_free[s].record(pp["d2h"])
        comp.wait_stream(pp["d2h"])
        comp.wait_stream(pp["h2d"])

    def check_status(self):
        for name, h in self.handles.items():
            st = h.status()
            if st != 0:
                raise binding.QconvError(st, "layer %s" % name)

    def num_launches(self):
        """Kernels launched by one forward pass (input conversion + one per layer, two for a layer that
        packs its input first)."""
        n = 0 if self._fused_input() else 1
        for nd in self.net["nodes"]:
            if nd["name"] in self._pooled:                   # a pool taken inside the layer before it
                continue
            n += 1
            if nd["op"] == "conv" and any(m in self.handles[nd["name"]].describe() for m in ("igemm/stem", "igemm/s2d", "igemm/wrow")):
                n += 1
        return n * (2 if getattr(self, "graph_form", None) == "split2" and self.graph is not None else 1)

    def destroy(self):
        for h in self.handles.values():
            h.destroy()
        self.handles = {}
        for sets in getattr(self, "_parts", {}).values():
            for hs in sets:
                for h in hs.values():
                    h.destroy()
        self._parts = {}
