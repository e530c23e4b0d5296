"""The N > 1 plumbing on CPU: two gloo ranks shard a calibration batch, combine their statistics and
must arrive at the statistics (and hence the scale exponent) of the whole batch; timing is reduced
with MAX over ranks."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from oracle import ref
    from paper_1805_07941_b200 import dist as qd, workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x = wl.rng_for(3, 7).standard_normal(size=(9, 6, 5, 4), dtype=np.float32) * 3      # 9 images over 2 ranks
    x[8, 0, 0, 0] = 40.0                                                                 # the maximum sits on rank 1
    x[1, 0, 0, 1] = np.nan
    lo, hi = qd.shard_range(x.shape[0], rank, world)
    whole_auto = ref.calib_stats(x, 64)
    part_auto = ref.calib_stats(x[lo:hi], 64)
    part_auto["range_hi"] = part_auto["maxabs"]
    red_auto = qd.allreduce_calib(part_auto)
    whole_fix = ref.calib_stats(x, 64, 50.0)
    part_fix = ref.calib_stats(x[lo:hi], 64, 50.0)
    part_fix["range_hi"] = np.float32(50.0)
    red_fix = qd.allreduce_calib(part_fix)
    # two-pass collection on the agreed range: the combined histogram equals the whole batch's
    synced = qd.collect_synced(lambda hi_: ref.calib_stats(x[lo:hi], 64, hi_))
    slowest = qd.max_over_ranks(10.0 + rank)
    rate = qd.whole_job_rate(32, 5, 10.0 + rank)
    dist.destroy_process_group()
    q.put((rank, (lo, hi), float(red_auto["maxabs"]), red_auto["hist"] is None, red_auto["count"], red_auto["nonfinite"],
           red_auto["sum"], float(whole_auto["maxabs"]), whole_auto["count"], whole_auto["sum"],
           red_fix["hist"].tolist(), whole_fix["hist"].tolist(), ref.scale_exponent(float(red_auto["maxabs"])),
           ref.scale_exponent(float(whole_auto["maxabs"])), slowest, rate,
           synced["hist"].tolist(), whole_auto["hist"].tolist(), float(synced["maxabs"]), synced["count"]))


def test_two_ranks_agree_with_the_whole_batch():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [(0, 5), (5, 9)]
    for r in res:
        (_, _, mx, hist_dropped, cnt, nonf, sm, w_mx, w_cnt, w_sum, h_red, h_whole, e_red, e_whole, slowest, rate,
         h_sync, h_auto, mx_sync, cnt_sync) = r
        assert h_sync == h_auto and mx_sync == 40.0 and cnt_sync == w_cnt
        assert mx == w_mx == 40.0 and e_red == e_whole
        assert hist_dropped                      # per-rank automatic ranges differ: no combined histogram
        assert cnt == w_cnt and nonf == 1
        assert abs(sm - w_sum) <= 1e-9 * max(1.0, abs(w_sum))
        assert h_red == h_whole                  # fixed common range: bins add up exactly
        assert slowest == 11.0 and abs(rate - 2 * 32 * 5 / 11e-3) < 1e-6
