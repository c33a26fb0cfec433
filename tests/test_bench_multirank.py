"""The multi-GPU mode of bench.py is replicas only: images are independent, the path has no exchange
step, and the only collective is the max-over-ranks of the device timings.  That bookkeeping is
checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, ms_e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 20.0 - 3.0 * rank], world, torch.device("cpu"))
    out[rank] = (ms, ms_e2e, bench.whole_job_rate(8, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_two_gloo_ranks():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29653, out), nprocs=world, join=True)
    for rank in range(world):
        ms, ms_e2e, rate = out[rank]
        assert ms == 15.0 and ms_e2e == 20.0            # the slowest rank decides, on every rank
        assert abs(rate - 8 * 2 / 15e-3) < 1e-9         # units of all ranks over that time


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1, None) == [1.5, 2.5]
    assert bench.whole_job_rate(4, 1, 40.0) == 100.0


def test_attention_pair_count_matches_golden_closed_forms():
    """bench.py counts useful attention pairs from block histograms; pin it to the closed forms."""
    import bench
    p, g = bench.attention_pairs(28, 28, 7, 1, 1)
    assert p + g == 241669                               # 490^2 + 784 + 785
    p, g = bench.attention_pairs(64, 64, 8, 1, 1)
    assert p + g == 1990657                              # 1408^2 + 4096 + 4097
    # a filtered token set: brute force over blocks
    import numpy as np
    rng = np.random.default_rng(0)
    pos = np.sort(rng.choice(20 * 12, size=90, replace=False))
    by, bx = (pos // 12) // 8, (pos % 12) // 8
    brute = int(((np.abs(by[:, None] - by[None]) <= 1) & (np.abs(bx[:, None] - bx[None]) <= 1)).sum())
    p, g = bench.attention_pairs(20, 12, 8, 1, 2, pos)
    assert p == brute + 90 * 2 and g == 2 * 92


def test_kept_set_generators_and_config_line():
    """The benchmark's kept-set generators (inputs of the coherent-set measurements) and the config object
    shared by the two arms."""
    import numpy as np
    import bench
    import synth
    k = bench.coherent_kept(7, 64, 0.5)
    assert k.dtype == np.int32 and k.size == 2048 and (np.diff(k) > 0).all() and k.min() >= 0 and k.max() < 4096
    # coherent: far more allowed pairs than a scattered set of the same size
    rng = np.random.default_rng(0)
    sc = np.sort(rng.choice(4096, size=2048, replace=False))
    assert bench.attention_pairs(64, 64, 8, 1, 1, k)[0] > 1.2 * bench.attention_pairs(64, 64, 8, 1, 1, sc)[0]
    bm = bench.block_major(k, 64, 8)
    blk = (bm // 64) // 8 * 8 + (bm % 64) // 8
    assert (np.diff(blk) >= 0).all() and sorted(bm.tolist()) == k.tolist()
    img = synth.tissue_batch(3, 2, 64, 64, background=0.5)
    tk = bench.tissue_kept(img, 4, 100)
    assert tk.shape == (2, 100) and (np.diff(tk, axis=1) > 0).all()
    mean = img[:, 1].reshape(2, 16, 4, 16, 4).mean(axis=(2, 4)).reshape(2, 256)
    for b in range(2):
        assert mean[b][tk[b]].max() <= np.sort(mean[b])[100 - 1] + 1e-6          # the darkest 100
    wl = bench.workload_config(bench.DEFAULT_WORKLOAD)
    c = bench.config_of(wl, 1)
    assert c["workload"] == bench.DEFAULT_WORKLOAD and c["kept"] == 8192 and c["tokens"] == 16385
    assert bench.config_of(wl, 2)["parallelism"] == "replicas"
