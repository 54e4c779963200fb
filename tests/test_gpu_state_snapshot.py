"""Small-state snapshot: export, keep going, import, replay; the replay must repeat the first run bit for bit."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu

CFG = wl.WorkloadConfig(name="snapshot_bf16", dtype="bf16", n_layers=1, batch=3, n_heads=4, head_dim=128,
                        hidden=256, capacity=48, topk=20, rebuild_max=12, prompt=70, steps=16,
                        rope_theta=1.0e4, rebuild_mode="explicit", rebuild_p=0.3, seed=131, ctrl_hidden=128)


def _steps(g, w, lib, torch, to_dev, first, count):
    """Runs `count` decode steps starting at step index `first`; returns what each step produced."""
    cfg = w.cfg
    seen = []
    for s in range(first, first + count):
        n = lib.adore_cache_num_tokens(g.handle)
        lists, counts = w.explicit(s, n)
        dl = torch.from_numpy(lists).cuda() if lists is not None else None
        dc = torch.from_numpy(counts).cuda() if counts is not None else None
        x = w.x_new(n, 0)
        q, k, v = w.qkv(n, 0, x)
        lib.adore_decode_step(g.handle, 0, to_dev(q, cfg), to_dev(k, cfg), to_dev(v, cfg), to_dev(x, cfg), dl, dc, w.r_in,
                              g.out, g.weights)
        lib.adore_rebuild(g.handle, 0, None)
        lib.adore_cache_sync_status(g.handle)
        st, sr = g.slot_map()
        rt, rs, rc = g.rebuild_list()
        seen.append((g.out.float().cpu().numpy().copy(), g.weights.cpu().numpy().copy(), st, sr, rt, rs, rc))
    return seen


@pytest.mark.parametrize("CFG", [CFG, CFG.scaled(name="snapshot_relative", ctrl_relative_position=True, pos_scale=32.0,
                                                 ctrl_weight_std=0.3)], ids=["absolute", "relative"])
def test_export_import_rewinds_the_cache(CFG):
    import torch
    from paper_2407_02328_b200 import adore as lib
    from oracle.harness import Workload
    from tests.gpu_driver import GpuCache, to_dev, torch_dtype
    w = Workload(CFG, None)
    g = GpuCache(w)
    try:
        lib.adore_cache_append_tokens(g.handle, to_dev(w.prompt(), CFG), CFG.prompt)
        _steps(g, w, lib, torch, to_dev, 0, 6)
        need = lib.adore_cache_export_state(g.handle, None)
        assert need > 64
        small = np.zeros(need - 8, np.uint8)
        with pytest.raises(lib.AdoreError) as e:
            lib.adore_cache_export_state(g.handle, small)
        assert e.value.status == 1
        snap = np.zeros(need, np.uint8)
        assert lib.adore_cache_export_state(g.handle, snap) == need
        n0 = lib.adore_cache_num_tokens(g.handle)
        kp, vp = lib.adore_cache_kv(g.handle, 0)
        shape = (g.B, CFG.n_heads, CFG.capacity, CFG.head_dim)
        k_view, v_view = lib.device_view(kp, shape, torch_dtype(CFG)), lib.device_view(vp, shape, torch_dtype(CFG))
        k_keep, v_keep = k_view.clone(), v_view.clone()

        first = _steps(g, w, lib, torch, to_dev, 6, 5)
        assert lib.adore_cache_num_tokens(g.handle) == n0 + 5

        bad = snap.copy()
        bad[0] ^= 0xFF                                    # wrong magic: rejected, nothing changes
        with pytest.raises(lib.AdoreError) as e:
            lib.adore_cache_import_state(g.handle, bad)
        assert e.value.status == 1
        assert lib.adore_cache_num_tokens(g.handle) == n0 + 5

        lib.adore_cache_import_state(g.handle, snap)
        assert lib.adore_cache_num_tokens(g.handle) == n0
        k_view.copy_(k_keep)
        v_view.copy_(v_keep)
        torch.cuda.synchronize()
        again = np.zeros(need, np.uint8)
        lib.adore_cache_export_state(g.handle, again)
        assert (again == snap).all()

        second = _steps(g, w, lib, torch, to_dev, 6, 5)
        for a, b in zip(first, second):
            for x, y in zip(a, b):
                assert np.array_equal(x, y)
    finally:
        g.close()


def test_import_refuses_a_snapshot_whose_indices_do_not_fit_the_cache():
    """A truncated or damaged snapshot must not turn into out-of-range device accesses: every integer section is checked
    on the host, and a snapshot that fails is refused with the cache unchanged and still working."""
    import torch
    from paper_2407_02328_b200 import adore as lib
    from oracle.harness import Workload
    from tests.gpu_driver import GpuCache, to_dev, parse_snapshot
    w = Workload(CFG, None)
    g = GpuCache(w)
    try:
        lib.adore_cache_append_tokens(g.handle, to_dev(w.prompt(), CFG), CFG.prompt)
        _steps(g, w, lib, torch, to_dev, 0, 3)
        snap = np.zeros(lib.adore_cache_export_state(g.handle, None), np.uint8)
        lib.adore_cache_export_state(g.handle, snap)
        fields = parse_snapshot(snap, CFG, g.B)
        B, C, MT, R = g.B, CFG.capacity, CFG.max_tokens, CFG.rebuild_max
        off_slot_tok0 = 64
        off_role0 = off_slot_tok0 + 2 * B * C * 4
        off_tok_slot = off_role0 + 2 * ((B * C + 7) & ~7)
        off_z = off_tok_slot + 3 * B * MT * 4
        off_admit = off_z + B * CFG.ctrl_hidden * 8
        off_count = off_admit + 2 * ((B * 4 + 7) & ~7) + 2 * ((B * R * 4 + 7) & ~7)
        off_row_b = off_count + ((B * 4 + 7) & ~7)
        assert np.array_equal(snap[off_tok_slot: off_tok_slot + B * MT * 4].view(np.int32).reshape(B, MT), fields["tok_slot"])
        assert np.array_equal(snap[off_count: off_count + B * 4].view(np.int32), fields["rebuild_count"])

        def tampered(offset, value, dtype=np.int32):
            bad = snap.copy()
            bad[offset: offset + np.dtype(dtype).itemsize] = np.array([value], dtype).view(np.uint8)
            return bad

        n = int(fields["n"])
        cases = [tampered(off_slot_tok0, 10 ** 6), tampered(off_slot_tok0, n), tampered(off_role0, 7, np.uint8),
                 tampered(off_tok_slot + 4, C), tampered(off_admit, -2), tampered(off_count, R + 1),
                 tampered(40, 3)]                                              # header word 10: step_open
        if int(fields["row_total"][0]) > 0:
            cases.append(tampered(off_row_b, B))
        for bad in cases:
            with pytest.raises(lib.AdoreError) as e:
                lib.adore_cache_import_state(g.handle, bad)
            assert e.value.status == 1
        again = np.zeros_like(snap)
        lib.adore_cache_export_state(g.handle, again)
        assert (again == snap).all(), "a refused import changed the cache"
        lib.adore_cache_import_state(g.handle, snap)                             # the untouched snapshot is accepted
        _steps(g, w, lib, torch, to_dev, 3, 2)
    finally:
        g.close()


def test_import_rejects_a_snapshot_of_another_shape():
    from paper_2407_02328_b200 import adore as lib
    from oracle.harness import Workload
    from tests.gpu_driver import GpuCache
    g1 = GpuCache(Workload(CFG, None))
    g2 = GpuCache(Workload(CFG.scaled(name="snapshot_c40", capacity=40), None))
    try:
        snap = np.zeros(lib.adore_cache_export_state(g1.handle, None), np.uint8)
        lib.adore_cache_export_state(g1.handle, snap)
        with pytest.raises(lib.AdoreError) as e:
            lib.adore_cache_import_state(g2.handle, snap)
        assert e.value.status == 1
    finally:
        g1.close()
        g2.close()
    # and of another reading of the position: the relative one carries a section more
    g1 = GpuCache(Workload(CFG, None))
    g3 = GpuCache(Workload(CFG.scaled(name="snapshot_rel", ctrl_relative_position=True), None))
    try:
        for src, dst in ((g1, g3), (g3, g1)):
            snap = np.zeros(lib.adore_cache_export_state(src.handle, None), np.uint8)
            lib.adore_cache_export_state(src.handle, snap)
            with pytest.raises(lib.AdoreError) as e:
                lib.adore_cache_import_state(dst.handle, snap)
            assert e.value.status == 1
    finally:
        g1.close()
        g3.close()
