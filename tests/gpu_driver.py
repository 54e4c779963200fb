"""Runs the CUDA library and the oracle side by side on one workload and compares them.

Bit-exact: slot maps, roles, admitted slot, evicted token, rebuild lists. Floating point:
attention output and weights within the dtype's tolerance, cache rows within one unit in the
last place of the cache type. Attention top-K sets must be equal except where the oracle's own
logits of the swapped entries differ by less than 1e-6 of the row's largest |logit| (the GPU
ranks float32 logits, the oracle float64 ones); such near-ties are counted and reported.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

import workloads as wl
from oracle import adore_oracle as ao
from paper_2407_02328_b200 import adore as lib
from oracle.harness import Workload, make_oracle, explicit_as_lists

TOL = {"bf16": dict(out_abs=2e-2, out_rel=1e-2, w_abs=1e-3), "f32": dict(out_abs=1e-4, out_rel=1e-4, w_abs=1e-5)}
NEAR_TIE_REL = 1e-6


def torch_dtype(cfg: wl.WorkloadConfig):
    return torch.float32 if cfg.dtype == "f32" else torch.bfloat16


def to_dev(a: np.ndarray, cfg: wl.WorkloadConfig) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(torch_dtype(cfg)).contiguous()


@dataclass
class Report:
    steps: int = 0
    near_ties: int = 0
    rounding_ties: int = 0
    topk_rows: int = 0
    max_out_err: float = 0.0
    max_w_err: float = 0.0
    max_kv_ulp: float = 0.0
    score_mismatch: int = 0
    notes: List[str] = field(default_factory=list)


class GpuCache:
    """The library's cache for a workload, with torch-owned device buffers for the per-step I/O."""

    def __init__(self, w: Workload):
        c = self.cfg = w.cfg
        self.w = w
        self.B = w.batch
        self.handle = lib.adore_cache_create(
            lib.make_config(batch=self.B, n_layers=c.n_layers, n_heads=c.n_heads, head_dim=c.head_dim,
                            hidden=c.hidden, capacity=c.capacity, rebuild_max=c.rebuild_max, topk=c.topk,
                            max_tokens=c.max_tokens, ctrl_hidden=c.ctrl_hidden, dtype=c.dtype,
                            rebuild_mode=c.rebuild_mode, rope_theta=c.rope_theta, pos_scale=c.pos_scale,
                            flags=(lib.ADORE_FLAG_NO_RECURRENCE if c.ctrl_no_recurrence else 0) |
                            (lib.ADORE_FLAG_SCORE_FROM_ATTENTION if c.score_from_attention else 0) |
                            (lib.ADORE_FLAG_RELATIVE_POSITION if c.ctrl_relative_position else 0)),
            w.ctrl, torch.cuda.current_stream().cuda_stream)
        self.w_kv_dev = [to_dev(m, c) for m in w.w_kv]
        for l, m in enumerate(self.w_kv_dev):
            lib.adore_cache_set_projection(self.handle, l, m)
        self.out = torch.empty((self.B, c.n_heads, c.head_dim), dtype=torch_dtype(c), device="cuda")
        self.weights = torch.empty((self.B, c.n_heads, c.capacity + 1), dtype=torch.float32, device="cuda")

    def close(self):
        if self.handle:
            lib.adore_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()

    # ---- views ----
    def slot_map(self):
        st, sr = lib.adore_cache_slot_map(self.handle)
        c = self.cfg
        return (lib.device_view(st, (self.B, c.capacity), torch.int32).cpu().numpy(),
                lib.device_view(sr, (self.B, c.capacity), torch.uint8).cpu().numpy())

    def step_info(self):
        a, e = lib.adore_cache_step_info(self.handle)
        return (lib.device_view(a, (self.B,), torch.int32).cpu().numpy(),
                lib.device_view(e, (self.B,), torch.int32).cpu().numpy())

    def rebuild_list(self):
        c = self.cfg
        if c.rebuild_max == 0:
            z = np.zeros((self.B, 0), np.int32)
            return z, z, np.zeros(self.B, np.int32)
        t, s, n = lib.adore_cache_rebuild_list(self.handle)
        return (lib.device_view(t, (self.B, c.rebuild_max), torch.int32).cpu().numpy(),
                lib.device_view(s, (self.B, c.rebuild_max), torch.int32).cpu().numpy(),
                lib.device_view(n, (self.B,), torch.int32).cpu().numpy())

    def scores(self, n):
        s, g = lib.adore_cache_scores(self.handle)
        c = self.cfg
        return (lib.device_view(s, (self.B, c.max_tokens), torch.float32)[:, :n].cpu().numpy(),
                lib.device_view(g, (self.B, c.max_tokens), torch.float32)[:, :n].cpu().numpy())

    def kv(self, layer):
        k, v = lib.adore_cache_kv(self.handle, layer)
        c = self.cfg
        shape = (self.B, c.n_heads, c.capacity, c.head_dim)
        return (lib.device_view(k, shape, torch_dtype(c)).float().cpu().numpy(),
                lib.device_view(v, shape, torch_dtype(c)).float().cpu().numpy())


def _ulp(ref: np.ndarray, dtype: str) -> np.ndarray:
    """Size of one unit in the last place of the cache type at |ref| (floor at the smallest normal scale used)."""
    mant = 8 if dtype == "bf16" else 24
    e = np.floor(np.log2(np.maximum(np.abs(ref), 1e-30)))
    return np.exp2(e - (mant - 1))


def compare_attention(rep: Report, cfg, q, orc: ao.AdoreOracle, layer, k_new, attn_map, out_g, w_g, out_o, w_o,
                      Kc_before, gpu_k=None, admit_slot=None, own_row=True):
    tol = TOL[cfg.dtype]
    err = np.abs(out_g - out_o)
    bound = tol["out_abs"] + tol["out_rel"] * np.abs(out_o)
    keep_g, keep_o = w_g > 0, w_o > 0
    rep.topk_rows += keep_o.shape[0] * keep_o.shape[1]
    bad = np.argwhere((keep_g != keep_o).any(-1))
    # Where the two kept sets differ by a tie (each case is classified below), the outputs differ by the weight that moved
    # times the value rows it moved between: |out_g - out_o| <= sum_s |w_g - w_o|_s * max|v|. Everywhere else the plain
    # bound holds.
    if len(bad):
        vmax = float(np.abs(orc.Vc[layer]).max())
        for b, h in bad:
            bound[b, h] = bound[b, h] + np.abs(w_g[b, h] - w_o[b, h]).sum() * vmax
    assert (err <= bound).all(), f"attention output off by {err.max():.3e} (step {rep.steps}, layer {layer})"
    rep.max_out_err = max(rep.max_out_err, float(err.max()))
    w_ok = np.ones_like(keep_o)
    for b, h in bad:
        Kall = np.concatenate([Kc_before[b, h].astype(np.float64), k_new[b, h][None].astype(np.float64)])
        logit = Kall @ q[b, h].astype(np.float64) / np.sqrt(cfg.head_dim)
        valid = np.concatenate([attn_map[b] >= 0, [own_row]])
        scale = max(1.0, float(np.abs(logit[valid]).max()))
        diff = np.nonzero(keep_g[b, h] != keep_o[b, h])[0]
        assert keep_g[b, h].sum() == keep_o[b, h].sum(), "kept count differs"
        assert valid[diff].all(), "an empty slot was kept"
        thr = logit[keep_o[b, h]].min()
        gap = np.abs(logit[diff] - thr).max()
        if gap <= NEAR_TIE_REL * scale:
            rep.near_ties += 1
        else:
            # Rebuilt cache rows may differ from the oracle's by one unit in the last place (float32
            # against float64 accumulation before the rounding; checked by compare_state). Such a row
            # moves its logit by far more than 1e-6, so the GPU's choice is checked on the rows it
            # actually holds: with float64 logits of ITS cache bytes the kept set must be the top K.
            assert gpu_k is not None, f"top-K sets differ beyond a near-tie: gap {gap:.3e} scale {scale:.3e}"
            Kg = gpu_k()[b, h].astype(np.float64)
            a = int(admit_slot[b])
            Kg[a] = Kc_before[b, h, a]            # that slot already holds the new token's row
            lg = np.concatenate([Kg, k_new[b, h][None].astype(np.float64)]) @ q[b, h].astype(np.float64) / np.sqrt(cfg.head_dim)
            lowest_kept = lg[keep_g[b, h]].min()
            highest_dropped = lg[valid & ~keep_g[b, h]].max()
            assert lowest_kept >= highest_dropped - NEAR_TIE_REL * scale, \
                f"top-K set is not the top K of the GPU's own cache rows: {lowest_kept:.6e} < {highest_dropped:.6e}"
            assert np.abs(lg - logit)[valid].max() <= 0.05 * scale
            rep.rounding_ties += 1
        w_ok[b, h, diff] = False
    # A cache row that sits one unit in the last place away from the oracle's (allowed by the row check in
    # compare_state) moves its logit by |q_e| ulp(k_e) / sqrt(dh), up to ~2e-3 per element in bfloat16, and a weight w
    # by that factor times w: the bound has a part relative to the weight, the same 1e-2 (1e-4) as for the output.
    werr = np.abs(w_g - w_o)
    wbound = tol["w_abs"] + tol["out_rel"] * np.abs(w_o)
    assert (werr <= wbound)[w_ok].all(), f"attention weights off by {werr[w_ok].max():.3e}"
    werr = werr[w_ok]
    rep.max_w_err = max(rep.max_w_err, float(werr.max()))
    s = w_g.sum(-1)
    assert np.allclose(s, 1.0, atol=1e-4), "weights do not sum to one"


def compare_state(rep: Report, g: GpuCache, orc: ao.AdoreOracle, layers, check_scores=True, score_rtol=1e-6):
    cfg = g.cfg
    st, sr = g.slot_map()
    assert np.array_equal(st, orc.slot_tok), f"slot map differs at step {rep.steps}"
    assert np.array_equal(sr, orc.slot_role), f"slot roles differ at step {rep.steps}"
    adm, ev = g.step_info()
    assert np.array_equal(adm, orc.info.admit_slot) and np.array_equal(ev, orc.info.evicted_tok)
    lt, ls, ln = g.rebuild_list()
    for b in range(g.B):
        k = len(orc.info.rebuild_tok[b])
        assert ln[b] == k, f"rebuild count differs (b={b}): {ln[b]} vs {k}"
        assert np.array_equal(lt[b, :k], orc.info.rebuild_tok[b]) and np.array_equal(ls[b, :k], orc.info.rebuild_slot[b])
    if check_scores:
        sc, sg = g.scores(orc.n)
        mism = int((sc != orc.score[:, : orc.n]).sum())
        rep.score_mismatch += mism
        assert np.allclose(sc, orc.score[:, : orc.n], rtol=score_rtol, atol=1e-9)
        assert np.allclose(sg, orc.sigma[:, : orc.n], rtol=1e-6, atol=1e-9)
    occ = orc.slot_tok >= 0
    for l in layers:
        Kg, Vg = g.kv(l)
        for name, G, O in (("K", Kg, orc.Kc[l]), ("V", Vg, orc.Vc[l])):
            m = np.broadcast_to(occ[:, None, :, None], G.shape)
            d = np.abs(G - O)[m]
            u = _ulp(O, cfg.dtype)[m]
            lim = 1.0 if cfg.dtype == "bf16" else 64.0      # f32: float32 accumulation over d terms
            # float32 accumulation of the d-long dot products leaves an absolute error that one unit
            # in the last place cannot cover for outputs that nearly cancel to zero
            floor = 1e-4 if cfg.dtype == "bf16" else 1e-5
            worst = float((d / u).max()) if d.size else 0.0
            assert (d <= lim * u + floor).all(), f"{name} cache rows off by {worst:.2f} ulp at step {rep.steps}"
            rep.max_kv_ulp = max(rep.max_kv_ulp, worst)


def run_parity(cfg: wl.WorkloadConfig, batch: Optional[int] = None, steps: Optional[int] = None,
               state_every: int = 1, host_entry: bool = False) -> Report:
    """Free-running parity: both sides consume the same inputs and must agree at every step."""
    w = Workload(cfg, batch)
    orc = make_oracle(w)
    g = GpuCache(w)
    rep = Report()
    L = cfg.n_layers
    tables = None
    try:
        if cfg.prompt:
            xp = w.prompt()
            orc.append_tokens(xp)
            lib.adore_cache_append_tokens(g.handle, to_dev(xp, cfg), cfg.prompt)
            if cfg.per_layer_inputs:
                tables = [torch.zeros((g.B, cfg.max_tokens, cfg.hidden), dtype=torch_dtype(cfg), device="cuda")
                          for _ in range(L)]
                otab = [np.zeros((g.B, cfg.max_tokens, cfg.hidden), np.float32) for _ in range(L)]
                for l in range(L):
                    xl = xp if l == 0 else w.prompt(l)
                    otab[l][:, : cfg.prompt] = xl
                    tables[l][:, : cfg.prompt] = to_dev(xl, cfg)
                    if l > 0:
                        orc.fill_layer(l, otab[l])
                        lib.adore_cache_fill_layer(g.handle, l, tables[l])
            lib.adore_cache_sync_status(g.handle)
            compare_state(rep, g, orc, range(L))
        elif cfg.per_layer_inputs:
            tables = [torch.zeros((g.B, cfg.max_tokens, cfg.hidden), dtype=torch_dtype(cfg), device="cuda") for _ in range(L)]
            otab = [np.zeros((g.B, cfg.max_tokens, cfg.hidden), np.float32) for _ in range(L)]
        n_steps = cfg.steps if steps is None else steps
        for s in range(n_steps):
            n = orc.n
            lists, counts = w.explicit(s, n)
            ex = explicit_as_lists(lists, counts)
            dl = torch.from_numpy(lists).cuda() if lists is not None else None
            dc = torch.from_numpy(counts).cuda() if counts is not None else None
            for l in range(L):
                x = w.x_new(n, l if cfg.per_layer_inputs else 0)
                q, k, v = w.qkv(n, l, x)
                if cfg.per_layer_inputs:
                    otab[l][:, n] = x
                    tables[l][:, n] = to_dev(x, cfg)
                attn_map = orc.slot_tok.copy() if l == 0 else orc.attn_slot_tok.copy()
                K_before = orc.Kc[l].copy()
                out_o, w_o = orc.decode_step(l, q, k, v, x if l == 0 else None, ex if l == 0 else None)
                if host_entry:
                    ho = np.zeros((g.B, cfg.n_heads, cfg.head_dim), np.float32)
                    hq, hk, hv, hx = (to_dev(a, cfg).cpu() for a in (q, k, v, x))
                    hout = torch.zeros((g.B, cfg.n_heads, cfg.head_dim), dtype=torch_dtype(cfg))
                    if host_entry == "with_rebuild":     # the call that also queues the layer's rebuild
                        lib.adore_decode_rebuild_host(g.handle, l, hq, hk, hv, hx, lists if l == 0 else None,
                                                      counts if l == 0 else None, w.r_in if l == 0 else 0,
                                                      tables[l] if (cfg.per_layer_inputs and l > 0) else None, hout, g.weights)
                    else:
                        lib.adore_decode_step_host(g.handle, l, hq, hk, hv, hx, lists if l == 0 else None,
                                                   counts if l == 0 else None, w.r_in if l == 0 else 0, hout, g.weights)
                    out_g, w_g = hout.float().numpy(), g.weights.cpu().numpy()
                else:
                    lib.adore_decode_step(g.handle, l, to_dev(q, cfg), to_dev(k, cfg), to_dev(v, cfg), to_dev(x, cfg),
                                          dl if l == 0 else None, dc if l == 0 else None, w.r_in if l == 0 else 0,
                                          g.out, g.weights)
                    out_g, w_g = g.out.float().cpu().numpy(), g.weights.cpu().numpy()
                compare_attention(rep, cfg, q, orc, l, k, attn_map, out_g, w_g, out_o, w_o, K_before,
                                  gpu_k=lambda l=l: g.kv(l)[0], admit_slot=orc.info.admit_slot)
                orc.rebuild(l, otab[l] if (cfg.per_layer_inputs and l > 0) else None)
                if host_entry != "with_rebuild":
                    lib.adore_rebuild(g.handle, l, tables[l] if (cfg.per_layer_inputs and l > 0) else None)
            rep.steps += 1
            if cfg.score_from_attention:
                # The values that rank the tokens are float32 sums of attention weights, which the two sides compute to
                # within a few units in the last place of each other. They are compared every step, and once they agree
                # to 1e-5 the oracle continues from the library's values, so that a difference in the last bits
                # cannot grow into a different eviction many steps later.
                lib.adore_cache_sync_status(g.handle)
                orc.check_invariants()
                compare_state(rep, g, orc, range(L), score_rtol=1e-5)
                orc.score[:, : orc.n] = g.scores(orc.n)[0]
            elif (s + 1) % state_every == 0 or s == n_steps - 1:
                lib.adore_cache_sync_status(g.handle)
                orc.check_invariants()
                compare_state(rep, g, orc, range(L))
        lib.adore_cache_sync_status(g.handle)
    finally:
        g.close()
    return rep


def run_parity_queued_host(cfg: wl.WorkloadConfig, steps: Optional[int] = None, sync_every: int = 1) -> Report:
    """Parity of adore_decode_rebuild_host_queued: per step the calls of ALL layers are issued back to back from pinned
    host buffers, the host waits once every `sync_every` steps, and only then are the outputs of those steps compared
    with the oracle's, layer by layer (every call in flight has `out`, `weights` and input buffers of its own)."""
    w = Workload(cfg, None)
    orc = make_oracle(w)
    g = GpuCache(w)
    rep = Report()
    L = cfg.n_layers
    pin = lambda a: to_dev(a, cfg).cpu().pin_memory()
    try:
        tables = otab = None
        if cfg.prompt:
            xp = w.prompt()
            orc.append_tokens(xp)
            lib.adore_cache_append_tokens(g.handle, to_dev(xp, cfg), cfg.prompt)
        if cfg.per_layer_inputs:
            tables = [torch.zeros((g.B, cfg.max_tokens, cfg.hidden), dtype=torch_dtype(cfg), device="cuda") for _ in range(L)]
            otab = [np.zeros((g.B, cfg.max_tokens, cfg.hidden), np.float32) for _ in range(L)]
            # the tables hold every row of the run from the start: a queued rebuild reads them while later steps are issued
            n_all = cfg.prompt + (cfg.steps if steps is None else steps)
            for l in range(L):
                for t0 in range(0, n_all, 64):
                    rows = wl.hidden_rows(cfg, t0, min(64, n_all - t0), l, g.B)
                    otab[l][:, t0:t0 + rows.shape[1]] = rows
                tables[l].copy_(to_dev(otab[l], cfg))
                if l > 0 and cfg.prompt:
                    orc.fill_layer(l, otab[l])
                    lib.adore_cache_fill_layer(g.handle, l, tables[l])
        lib.adore_cache_sync_status(g.handle)
        n_steps = cfg.steps if steps is None else steps
        pending = []
        for s in range(n_steps):
            n = cfg.prompt + s
            lists, counts = w.explicit(s, n)
            hl = None if lists is None else torch.from_numpy(lists).pin_memory()
            hc = None if counts is None else torch.from_numpy(counts).pin_memory()
            calls = []
            for l in range(L):
                x = w.x_new(n, l if cfg.per_layer_inputs else 0)
                q, k, v = w.qkv(n, l, x)
                hq, hk, hv, hx = pin(q), pin(k), pin(v), pin(x)
                hout = torch.zeros((g.B, cfg.n_heads, cfg.head_dim), dtype=torch_dtype(cfg)).pin_memory()
                wts = torch.empty((g.B, cfg.n_heads, cfg.capacity + 1), dtype=torch.float32, device="cuda")
                lib.adore_decode_rebuild_host_queued(g.handle, l, hq, hk, hv, hx if l == 0 else None, hl if l == 0 else None,
                                                     hc if l == 0 else None, w.r_in if l == 0 else 0,
                                                     tables[l] if (cfg.per_layer_inputs and l > 0) else None, hout, wts)
                calls.append((q, k, v, x, hout, wts, (hq, hk, hv, hx, hl, hc)))
            pending.append((lists, counts, calls))
            if (s + 1) % sync_every and s != n_steps - 1:
                continue
            lib.adore_cache_wait_outputs(g.handle)      # the outputs are in; the rebuilds may still be running
            for lists_p, counts_p, calls_p in pending:
                ex = explicit_as_lists(lists_p, counts_p)
                for l, (q, k, v, x, hout, wts, _keep) in enumerate(calls_p):
                    attn_map = orc.slot_tok.copy() if l == 0 else orc.attn_slot_tok.copy()
                    K_before = orc.Kc[l].copy()
                    out_o, w_o = orc.decode_step(l, q, k, v, x if l == 0 else None, ex if l == 0 else None)
                    compare_attention(rep, cfg, q, orc, l, k, attn_map, hout.float().numpy(), wts.cpu().numpy(), out_o, w_o,
                                      K_before, gpu_k=None, admit_slot=orc.info.admit_slot)
                    orc.rebuild(l, otab[l] if (cfg.per_layer_inputs and l > 0) else None)
                rep.steps += 1
            pending = []
            orc.check_invariants()
            compare_state(rep, g, orc, range(L))
        lib.adore_cache_sync_status(g.handle)
    finally:
        g.close()
    return rep


def run_parity_rebuild_first(cfg: wl.WorkloadConfig, steps: Optional[int] = None) -> Report:
    """Free-running parity of the step in the order Section 2.3 prints it: adore_step_begin, then per layer
    adore_rebuild and adore_attend_rows (R_max + 1 query rows per sequence), against the oracle's same three calls.
    Every layer rebuilds from the token store."""
    assert not cfg.per_layer_inputs
    w = Workload(cfg, None)
    orc = make_oracle(w)
    g = GpuCache(w)
    rep = Report()
    L, R1 = cfg.n_layers, cfg.rebuild_max + 1
    out_dev = torch.empty((g.B, cfg.n_heads, R1, cfg.head_dim), dtype=torch_dtype(cfg), device="cuda")
    w_dev = torch.empty((g.B, cfg.n_heads, R1, cfg.capacity + 1), dtype=torch.float32, device="cuda")
    try:
        if cfg.prompt:
            xp = w.prompt()
            orc.append_tokens(xp)
            lib.adore_cache_append_tokens(g.handle, to_dev(xp, cfg), cfg.prompt)
            lib.adore_cache_sync_status(g.handle)
            compare_state(rep, g, orc, range(L))
        n_steps = cfg.steps if steps is None else steps
        for s in range(n_steps):
            n = orc.n
            lists, counts = w.explicit(s, n)
            dl = torch.from_numpy(lists).cuda() if lists is not None else None
            dc = torch.from_numpy(counts).cuda() if counts is not None else None
            x = w.x_new(n, 0)
            orc.step_begin(x, explicit_as_lists(lists, counts))
            lib.adore_step_begin(g.handle, to_dev(x, cfg), dl, dc, w.r_in)
            for l in range(L):
                _, k, v = w.qkv(n, l, x)
                orc.rebuild(l)
                lib.adore_rebuild(g.handle, l, None)
                q_rows = w.q_rows(n, l, orc.x, orc.info.rebuild_tok)
                K_before = orc.Kc[l].copy()
                st = orc.slot_tok.copy()
                out_o, w_o = orc.attend_rows(l, q_rows, k, v)
                lib.adore_attend_rows(g.handle, l, to_dev(q_rows, cfg), to_dev(k, cfg), to_dev(v, cfg), out_dev, w_dev)
                out_g, w_g = out_dev.float().cpu().numpy(), w_dev.cpu().numpy()
                for i in range(R1):
                    toks = np.array([n if i == R1 - 1 else (int(orc.info.rebuild_tok[b][i]) if i < len(orc.info.rebuild_tok[b]) else -1)
                                     for b in range(g.B)])
                    pad = toks < 0
                    assert not out_g[pad, :, i].any() and not w_g[pad, :, i].any(), "padding rows must be zero"
                    idx = np.nonzero(~pad)[0]
                    if idx.size == 0:
                        continue
                    seen = np.where((st[idx] >= 0) & (st[idx] <= toks[idx, None]) & (st[idx] != n), st[idx], -1)
                    compare_attention(rep, cfg, q_rows[idx, :, i], orc, l, k[idx], seen, out_g[idx, :, i], w_g[idx, :, i],
                                      out_o[idx, :, i], w_o[idx, :, i], K_before[idx],
                                      gpu_k=lambda l=l, idx=idx: g.kv(l)[0][idx], admit_slot=orc.info.admit_slot[idx],
                                      own_row=(i == R1 - 1))
            rep.steps += 1
            lib.adore_cache_sync_status(g.handle)
            orc.check_invariants()
            compare_state(rep, g, orc, range(L))
        lib.adore_cache_sync_status(g.handle)
    finally:
        g.close()
    return rep
