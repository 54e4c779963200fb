"""The allocation-free controller scoring entry point against the cache-based path.

Collected last on purpose (file name), so that a run that stops at the first failure has already
gone through every other test. Some callers of this library may not allocate device memory (a
thread working next to CUDA-graph capture, a process whose device memory belongs to another
allocator); for them adore_controller_score_static keeps its scratch in a fixed array inside the
library. Here it must reproduce, on two calls in a row that share that array, the scores the
cache-based path computes for the same tokens, and the scores the CPU oracle's controller gives.
"""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu

CFG = wl.WorkloadConfig(name="no_alloc", dtype="bf16", n_layers=1, batch=5, n_heads=2, head_dim=128, hidden=512,
                        capacity=16, topk=8, rebuild_max=2, prompt=0, steps=4, rope_theta=1.0e4,
                        rebuild_mode="policy", rebuild_p=0.0, seed=77, ctrl_hidden=128, pos_scale=64.0)


@pytest.mark.parametrize("cfg", [CFG, CFG.scaled(name="no_alloc_f32", dtype="f32", batch=3, ctrl_hidden=96, seed=78),
                                 CFG.scaled(name="no_alloc_wide", batch=4, ctrl_hidden=256, hidden=256, seed=79)],
                         ids=lambda c: c.name)
def test_static_scoring_matches_cache_path_on_two_calls_in_a_row(cfg):
    import torch
    from oracle.harness import Workload
    from paper_2407_02328_b200 import adore as lib
    from tests.gpu_driver import GpuCache, to_dev

    w = Workload(cfg)
    g = GpuCache(w)
    try:
        xs = []
        for n in range(2):                                   # existing entry point: two decode steps
            x = w.x_new(n)
            q, k, v = w.qkv(n, 0, x)
            xs.append(to_dev(x, cfg))
            lib.adore_decode_step(g.handle, 0, to_dev(q, cfg), to_dev(k, cfg), to_dev(v, cfg), xs[-1], None, None, 0,
                                  g.out, g.weights)
            lib.adore_rebuild(g.handle, 0, None)
        lib.adore_cache_sync_status(g.handle)
        ref_score, ref_sigma = g.scores(2)
    finally:
        g.close()

    wdev = {k: torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).cuda() for k, v in w.ctrl.items()}
    z = torch.zeros((cfg.batch, cfg.ctrl_hidden), dtype=torch.float64, device="cuda")
    score = torch.full((2, cfg.batch), float("nan"), dtype=torch.float32, device="cuda")
    sigma = torch.full((2, cfg.batch), float("nan"), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for n in range(2):                                       # two calls in a row share the static scratch
        lib.adore_controller_score_static(wdev, cfg.dtype, cfg.batch, cfg.hidden, cfg.ctrl_hidden, xs[n], z, n,
                                          cfg.pos_scale, score[n], sigma[n], stream)
    torch.cuda.synchronize()
    assert np.allclose(score.cpu().numpy().T, ref_score, rtol=1e-6, atol=1e-9)
    assert np.allclose(sigma.cpu().numpy().T, ref_sigma, rtol=1e-6, atol=1e-9)
    # and against the oracle's controller (Section 2.2 Eq. 2 in float64, rounded once to float32): equal, or one unit in
    # the last place where the float64 sums were split differently
    from oracle import adore_oracle as ao
    zo = np.zeros((cfg.batch, cfg.ctrl_hidden), np.float64)
    for n in range(2):
        zo = ao.gru_step(w.x_new(n), zo, w.ctrl)
        so = ao.controller_score(zo, n, cfg.pos_scale, w.ctrl).astype(np.float32)
        got = score[n].cpu().numpy()
        assert (np.abs(got - so) <= np.spacing(np.abs(so))).all(), f"scores of call {n} differ from the oracle's"
        sig = (1.0 / (1.0 + np.exp(-ao.controller_score(zo, n, cfg.pos_scale, w.ctrl)))).astype(np.float32)
        assert np.allclose(sigma[n].cpu().numpy(), sig, rtol=1e-6, atol=0)
    assert np.allclose(z.cpu().numpy(), zo, rtol=1e-12, atol=1e-15)


def test_static_scoring_rejects_oversized_requests():
    import torch
    from paper_2407_02328_b200 import adore as lib
    dummy = torch.zeros(16, dtype=torch.float32, device="cuda")
    wdev = {k: dummy for k, _ in lib.adore_controller_weights_t._fields_}
    with pytest.raises(lib.AdoreError) as e:                 # 700 * 3 * 128 doubles exceed the 2 MiB array
        lib.adore_controller_score_static(wdev, "bf16", 700, 4096, 128, dummy, dummy, 0, 4096.0, dummy, dummy)
    assert e.value.status == 8


def test_static_scoring_rejects_rows_it_cannot_read_in_16_byte_pieces():
    """Refused on the host, nothing launched: a hidden size that is not a multiple of 64, and an input that does not
    start on a 16-byte boundary."""
    import torch
    from paper_2407_02328_b200 import adore as lib
    dummy = torch.zeros(4096, dtype=torch.float32, device="cuda")
    wdev = {k: dummy for k, _ in lib.adore_controller_weights_t._fields_}
    for hidden, x in ((100, dummy), (128, dummy[1:])):
        with pytest.raises(lib.AdoreError) as e:
            lib.adore_controller_score_static(wdev, "f32", 2, hidden, 64, x.data_ptr(), dummy, 0, 64.0, dummy, dummy)
        assert e.value.status == 8
    torch.cuda.synchronize()
