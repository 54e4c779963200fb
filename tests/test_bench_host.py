"""Host-side logic of bench.py: rank aggregation over gloo (world size 2) and roofline arithmetic."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, torch.device("cpu"))     # the slowest rank counts
    out[rank] = (ms, bench.whole_job_tokens_per_s(16, 5, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks():
    world, port = 2, _free_port()
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for r in range(world):
        ms, val = out[r]
        assert ms == 20.0
        assert abs(val - 16 * 2 * 5 / 0.020) < 1e-6


def test_roofline_arithmetic():
    import bench
    import workloads as wl
    c = wl.get_config(3)
    full = bench.attention_bytes_per_launch(c, c.capacity)
    # all 513 key rows + 256 kept value rows + q/out + admit rows, 256 B each, + 513 weights, per (b, h)
    per_bh = (513 + 256 + 2 + 2) * 256 + 513 * 4
    assert full == c.batch * c.n_heads * per_bh
    flops, nbytes = bench.rebuild_flops_bytes_per_launch(c, 16384)
    assert flops == 2.0 * 16384 * 4096 * 8192
    assert nbytes == (8192 * 4096 + 16384 * 4096 + 16384 * 8192) * 2
    peaks, kind = bench.measured_peaks()
    assert kind in ("measured", "fallback") and peaks["hbm_gbs"] > 1000


def test_workload_for_a_few_sequences_and_layers_draws_the_same_numbers_as_the_full_one():
    """The parity tests of the large configurations check some sequences and some layers of a run in which the GPU
    holds all of them: the reduced workload must hand out exactly the rows, flags and weights of the full one."""
    import numpy as np
    import workloads as wl
    from oracle.harness import Workload
    cfg = wl.WorkloadConfig(name="sub", dtype="bf16", n_layers=4, batch=6, n_heads=2, head_dim=64, hidden=64, capacity=16,
                            topk=8, rebuild_max=4, prompt=5, steps=9, rope_theta=1.0e4, rebuild_mode="explicit",
                            rebuild_p=0.3, seed=5, per_layer_inputs=True)
    full = Workload(cfg)
    part = Workload(cfg, batch=2, layers=[0, 3])
    assert part.cfg.n_layers == 2 and part.r_in == full.r_in
    assert np.array_equal(part.prompt(1), full.prompt(3)[:2]) and np.array_equal(part.prompt(0), full.prompt(0)[:2])
    assert np.array_equal(part.x_new(7, 1), full.x_new(7, 3)[:2])
    assert np.array_equal(part.w_kv[1], full.w_kv[3]) and np.array_equal(part.w_q[1], full.w_q[3])
    for a, b in zip(part.explicit(4, 9), full.explicit(4, 9)):
        assert np.array_equal(a, b[:2])
    x = full.x_new(6, 3)
    for a, b in zip(part.qkv(6, 1, x[:2]), full.qkv(6, 3, x)):
        assert np.allclose(a, b[:2], rtol=0, atol=1e-6)
