"""Error reporting of the C ABI on a GPU: call order, a full token table, a bad explicit entry (device error word),
bad arguments, a cache that cannot fit. None of these cases faults or hangs the device: every one is caught on the host or turned into a no-op."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu

CFG = wl.WorkloadConfig(name="errors_bf16", dtype="bf16", n_layers=2, batch=2, n_heads=2, head_dim=128,
                        hidden=256, capacity=24, topk=8, rebuild_max=4, prompt=10, steps=3,
                        rope_theta=1.0e4, rebuild_mode="explicit", rebuild_p=0.3, seed=141, ctrl_hidden=128)


def _setup():
    import torch
    from paper_2407_02328_b200 import adore as lib
    from oracle.harness import Workload
    from tests.gpu_driver import GpuCache, to_dev
    w = Workload(CFG, None)
    g = GpuCache(w)
    lib.adore_cache_append_tokens(g.handle, to_dev(w.prompt(), CFG), CFG.prompt)
    return torch, lib, w, g, to_dev


def _inputs(w, to_dev, n, layer=0):
    x = w.x_new(n, 0)
    q, k, v = w.qkv(n, layer, x)
    return to_dev(q, CFG), to_dev(k, CFG), to_dev(v, CFG), to_dev(x, CFG)


def test_call_order_is_checked_on_the_host():
    torch, lib, w, g, to_dev = _setup()
    try:
        n = lib.adore_cache_num_tokens(g.handle)
        q, k, v, x = _inputs(w, to_dev, n)
        q_rows = torch.zeros((g.B, CFG.n_heads, CFG.rebuild_max + 1, CFG.head_dim), dtype=torch.bfloat16, device="cuda")
        out_rows = torch.zeros_like(q_rows)
        for call in (lambda: lib.adore_decode_step(g.handle, 1, q, k, v, None, None, None, 0, g.out, None),   # layer 1 first
                     lambda: lib.adore_rebuild(g.handle, 0, None),                                           # no step open
                     lambda: lib.adore_attend_rows(g.handle, 0, q_rows, k, v, out_rows, None)):              # no step_begin
            with pytest.raises(lib.AdoreError) as e:
                call()
            assert e.value.status == 4
        lib.adore_step_begin(g.handle, x, None, None, 0)
        with pytest.raises(lib.AdoreError) as e:                 # a step opened by step_begin is not continued by decode_step
            lib.adore_decode_step(g.handle, 1, q, k, v, None, None, None, 0, g.out, None)
        assert e.value.status == 4
        for l in range(CFG.n_layers):                            # ... but by rebuild + attend_rows, and the cache stays healthy
            lib.adore_rebuild(g.handle, l, None)
            lib.adore_attend_rows(g.handle, l, q_rows, k, v, out_rows, None)
        lib.adore_cache_sync_status(g.handle)
        assert lib.adore_cache_num_tokens(g.handle) == n + 1
    finally:
        g.close()


def test_full_token_table_and_bad_arguments():
    torch, lib, w, g, to_dev = _setup()
    try:
        for s in range(CFG.steps):
            n = lib.adore_cache_num_tokens(g.handle)
            q, k, v, x = _inputs(w, to_dev, n)
            lib.adore_decode_step(g.handle, 0, q, k, v, x, None, None, 0, g.out, None)
            lib.adore_decode_step(g.handle, 1, q, k, v, None, None, None, 0, g.out, None)
        lib.adore_cache_sync_status(g.handle)
        assert lib.adore_cache_num_tokens(g.handle) == CFG.max_tokens
        with pytest.raises(lib.AdoreError) as e:
            lib.adore_decode_step(g.handle, 0, q, k, v, x, None, None, 0, g.out, None)
        assert e.value.status == 3
        for call in (lambda: lib.adore_decode_step(g.handle, 0, None, k, v, x, None, None, 0, g.out, None),
                     lambda: lib.adore_decode_step(g.handle, 5, q, k, v, x, None, None, 0, g.out, None),
                     lambda: lib.adore_cache_set_projection(g.handle, 7, g.w_kv_dev[0])):
            with pytest.raises(lib.AdoreError) as e:
                call()
            assert e.value.status == 1
        lib.adore_cache_sync_status(g.handle)
        # device pointers off the 16-byte boundary the kernels' loads need: refused on the host, nothing is launched
        n_elems = g.B * CFG.n_heads * CFG.head_dim
        skew = torch.zeros(n_elems + 8, dtype=torch.bfloat16, device="cuda")[1:n_elems + 1]     # 2 bytes off
        xskew = torch.zeros(g.B * CFG.hidden + 8, dtype=torch.bfloat16, device="cuda")[3:g.B * CFG.hidden + 3]
        launches = lib.adore_cache_launch_count(g.handle)
        for call in (lambda: lib.adore_decode_step(g.handle, 1, skew, k, v, None, None, None, 0, g.out, None),
                     lambda: lib.adore_decode_step(g.handle, 1, q, k, skew, None, None, None, 0, g.out, None),
                     lambda: lib.adore_decode_step(g.handle, 1, q, k, v, None, None, None, 0, skew, None),
                     lambda: lib.adore_step_begin(g.handle, xskew, None, None, 0),
                     lambda: lib.adore_rebuild(g.handle, 0, xskew),
                     lambda: lib.adore_cache_fill_layer(g.handle, 1, xskew)):
            with pytest.raises(lib.AdoreError) as e:
                call()
            assert e.value.status == 1
        assert lib.adore_cache_launch_count(g.handle) == launches
        lib.adore_cache_sync_status(g.handle)
        # flags that exclude each other, and a flag bit that does not exist
        for flags in (lib.ADORE_FLAG_SCORE_FROM_ATTENTION | lib.ADORE_FLAG_RELATIVE_POSITION, 1 << 9):
            with pytest.raises(lib.AdoreError) as e:
                lib.adore_cache_create(
                    lib.make_config(batch=2, n_layers=1, n_heads=2, head_dim=64, hidden=128, capacity=16, rebuild_max=2, topk=4,
                                    max_tokens=32, ctrl_hidden=32, dtype="f32", rebuild_mode="policy", rope_theta=0.0,
                                    pos_scale=64.0, flags=flags),
                    w.ctrl, torch.cuda.current_stream().cuda_stream)
            assert e.value.status == 1
    finally:
        g.close()


def test_bad_explicit_entry_sets_the_device_error_word_and_is_ignored():
    torch, lib, w, g, to_dev = _setup()
    try:
        n = lib.adore_cache_num_tokens(g.handle)
        q, k, v, x = _inputs(w, to_dev, n)
        lists = torch.tensor([[0, 10 ** 6, 1], [2, -5, 3]], dtype=torch.int32, device="cuda")    # one entry out of range each
        counts = torch.tensor([3, 3], dtype=torch.int32, device="cuda")
        lib.adore_decode_step(g.handle, 0, q, k, v, x, lists, counts, 3, g.out, None)
        lib.adore_rebuild(g.handle, 0, None)
        with pytest.raises(lib.AdoreError) as e:
            lib.adore_cache_sync_status(g.handle)
        assert e.value.status == 6
        tok, _, cnt = g.rebuild_list()
        for b in range(g.B):                                  # the good entries were used, the bad ones dropped
            assert set(tok[b, : cnt[b]]) <= {0, 1, 2, 3}
        lib.adore_cache_sync_status(g.handle)                 # the word was cleared; the cache goes on working
        lib.adore_decode_step(g.handle, 1, q, k, v, None, None, None, 0, g.out, None)
        lib.adore_cache_sync_status(g.handle)
        with pytest.raises(lib.AdoreError) as e:              # more candidates than the selection kernel sorts
            lib.adore_decode_step(g.handle, 0, q, k, v, x, lists, counts, 9000, g.out, None)
        assert e.value.status == 8
    finally:
        g.close()


def test_a_cache_that_cannot_fit_is_refused_with_out_of_memory_and_leaves_the_device_usable():
    """One request far beyond the device's memory (several terabytes of K/V rows): the allocation itself is refused by
    the driver, create reports OOM, frees what it had taken, and a normal cache can be made and used right after."""
    torch, lib, w, g, to_dev = _setup()
    try:
        free0, _ = torch.cuda.mem_get_info()
        with pytest.raises(lib.AdoreError) as e:
            lib.adore_cache_create(
                lib.make_config(batch=1024, n_layers=64, n_heads=128, head_dim=128, hidden=CFG.hidden, capacity=4096, rebuild_max=8,
                                topk=64, max_tokens=4100, ctrl_hidden=CFG.ctrl_hidden, dtype="bf16", rebuild_mode="policy",
                                rope_theta=1.0e4, pos_scale=4096.0),
                w.ctrl, torch.cuda.current_stream().cuda_stream)
        assert e.value.status == 2
        free1, _ = torch.cuda.mem_get_info()
        assert free1 >= free0 - (64 << 20), "the failed create kept device memory"
        n = lib.adore_cache_num_tokens(g.handle)
        q, k, v, x = _inputs(w, to_dev, n)
        lib.adore_decode_step(g.handle, 0, q, k, v, x, None, None, 0, g.out, None)     # the existing cache still works
        lib.adore_cache_sync_status(g.handle)
    finally:
        g.close()


def test_a_bounded_device_wait_that_runs_out_sets_the_timeout_bit_and_returns():
    """Every mbarrier wait of the library is bounded (mbar_wait_bounded): on expiry the kernel sets the timeout bit of an
    error word and leaves through its ordinary exit. Here that path is taken in the safe form: a test-only kernel built
    from the library's own mbarrier header waits on a barrier nobody arrives on, with nothing in flight. The kernel must
    return, the word must carry the timeout bit (the one adore_cache_sync_status reports as ADORE_ERR_TIMEOUT), and a
    cache must work as usual afterwards."""
    import ctypes
    from tests.native import build_wait_probe
    torch, lib, w, g, to_dev = _setup()
    try:
        probe = ctypes.CDLL(build_wait_probe())
        probe.wait_probe_run.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        probe.wait_probe_timeout_bit.restype = ctypes.c_uint
        words = torch.zeros(2, dtype=torch.int32, device="cuda")
        ctas = 4
        rc = probe.wait_probe_run(words.data_ptr(), words.data_ptr() + 4, ctas, torch.cuda.current_stream().cuda_stream)
        assert rc == 0
        torch.cuda.synchronize()                              # the kernel came back: the wait is bounded
        err_word, reached = (int(v) for v in words.cpu())
        assert err_word == probe.wait_probe_timeout_bit() == 1
        assert reached == ctas, "every CTA must leave through the common exit"
        assert lib.STATUS_NAMES[7] == "TIMEOUT"
        n = lib.adore_cache_num_tokens(g.handle)
        q, k, v, x = _inputs(w, to_dev, n)
        lib.adore_decode_step(g.handle, 0, q, k, v, x, None, None, 0, g.out, None)    # the device and the cache are fine
        lib.adore_rebuild(g.handle, 0, None)
        lib.adore_cache_sync_status(g.handle)
    finally:
        g.close()
