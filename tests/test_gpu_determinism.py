"""Run-twice determinism: the same workload through fresh caches, with no host wait between the steps, must give
bit-identical outputs, weights, maps, scores and cache rows, and the same as a run that waits after every call. Nothing in the path may depend on timing: the split-K
rebuild adds its parts in a fixed order, the controller's partial sums likewise, and the rebuilds that run on the
library's own stream are ordered against the next step by events only."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu

BASE = wl.WorkloadConfig(name="det", dtype="bf16", n_layers=3, batch=4, n_heads=8, head_dim=128, hidden=1024, capacity=64,
                         topk=24, rebuild_max=24, prompt=100, steps=24, rope_theta=1.0e4, rebuild_mode="explicit",
                         rebuild_p=0.5, seed=161, ctrl_hidden=128, per_layer_inputs=True)


def _free_run(cfg, wait_after_every_call=False, table_at_layer0=False):
    """All steps queued back to back on the device (or, for comparison, with a host wait after every call); returns
    everything observable at the end."""
    import torch
    from paper_2407_02328_b200 import adore as lib
    from oracle.harness import Workload
    from tests.gpu_driver import GpuCache, to_dev, torch_dtype
    w = Workload(cfg, None)
    g = GpuCache(w)
    L, S = cfg.n_layers, cfg.steps
    try:
        tables = None
        lib.adore_cache_append_tokens(g.handle, to_dev(w.prompt(), cfg), cfg.prompt)
        if cfg.per_layer_inputs:
            tables = []
            for l in range(L):
                t = torch.zeros((g.B, cfg.max_tokens, cfg.hidden), dtype=torch_dtype(cfg), device="cuda")
                t[:, : cfg.max_tokens] = to_dev(wl.hidden_rows(cfg, 0, cfg.max_tokens, l, g.B), cfg)
                tables.append(t)
                if l > 0:
                    lib.adore_cache_fill_layer(g.handle, l, t)
        # inputs of every step on the device before the first step is issued
        steps = []
        for s in range(S):
            n = cfg.prompt + s
            lists, counts = w.explicit(s, n)
            dl = torch.from_numpy(lists).cuda() if lists is not None else None
            dc = torch.from_numpy(counts).cuda() if counts is not None else None
            per_layer = []
            for l in range(L):
                x = w.x_new(n, l if cfg.per_layer_inputs else 0)
                q, k, v = w.qkv(n, l, x)
                per_layer.append(tuple(to_dev(a, cfg) for a in (q, k, v, x)))
            steps.append((dl, dc, per_layer))
        outs = torch.zeros((S, L, g.B, cfg.n_heads, cfg.head_dim), dtype=torch_dtype(cfg), device="cuda")
        wts = torch.zeros((S, L, g.B, cfg.n_heads, cfg.capacity + 1), dtype=torch.float32, device="cuda")
        lib.adore_cache_sync_status(g.handle)
        for s, (dl, dc, per_layer) in enumerate(steps):
            for l, (q, k, v, x) in enumerate(per_layer):
                lib.adore_decode_step(g.handle, l, q, k, v, x if l == 0 else None, dl if l == 0 else None,
                                      dc if l == 0 else None, w.r_in if l == 0 else 0, outs[s, l], wts[s, l])
                if wait_after_every_call:
                    lib.adore_cache_sync_status(g.handle)
                lib.adore_rebuild(g.handle, l, tables[l] if (tables is not None and (l > 0 or table_at_layer0)) else None)
                if wait_after_every_call:
                    lib.adore_cache_sync_status(g.handle)
        lib.adore_cache_sync_status(g.handle)
        st, sr = g.slot_map()
        sc, sg = g.scores(cfg.max_tokens)
        kv = [g.kv(l) for l in range(L)]
        occ = st >= 0
        return dict(out=outs.float().cpu().numpy(), w=wts.cpu().numpy(), slot_tok=st, slot_role=sr, score=sc, sigma=sg,
                    k=[np.where(occ[:, None, :, None], a, 0) for a, _ in kv], v=[np.where(occ[:, None, :, None], b, 0) for _, b in kv])
    finally:
        g.close()


@pytest.mark.parametrize("cfg", [BASE, BASE.scaled(name="det_policy_one_layer", n_layers=1, per_layer_inputs=False, rebuild_mode="policy",
                                                   rebuild_max=8, hidden=256, seed=162),
                                 BASE.scaled(name="det_relative", ctrl_relative_position=True, pos_scale=32.0, ctrl_weight_std=0.3,
                                             n_layers=2, seed=163)], ids=lambda c: c.name)
def test_two_free_running_runs_are_bit_identical(cfg):
    a = _free_run(cfg)
    # a second free run, and a run in which the host waits after every call (no two launches of the library overlap):
    # if the free run depended on how its streams interleave, it would differ from one of them
    for other, what in ((_free_run(cfg), "two free runs"), (_free_run(cfg, wait_after_every_call=True), "a free and a serial run")):
        for key in ("out", "w", "slot_tok", "slot_role", "score", "sigma"):
            assert np.array_equal(a[key], other[key]), f"{key} differs between {what}"
        for key in ("k", "v"):
            for l, (x, y) in enumerate(zip(a[key], other[key])):
                assert np.array_equal(x, y), f"{key} rows of layer {l} differ between {what}"
    assert np.isfinite(a["out"]).all() and (a["slot_tok"] >= 0).any()


def test_rebuild_from_a_caller_table_at_layer_0_equals_rebuild_from_the_store():
    """Layer 0 rebuilt from the caller's table (the same rows the library keeps in its token store) instead of from the
    store: the launch then gathers its rows itself, into the buffer that the step's early gather (selection stream) has
    just filled, so it has to wait for that gather. Everything observable must equal the run that rebuilds from the store."""
    a = _free_run(BASE)
    b = _free_run(BASE, table_at_layer0=True)
    for key in a:
        if isinstance(a[key], list):
            for x, y in zip(a[key], b[key]):
                assert np.array_equal(x, y), key
        else:
            assert np.array_equal(a[key], b[key]), key

