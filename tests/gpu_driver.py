"""Runs the CUDA library and the oracle side by side on one workload and compares them.

Both sides attend over IDENTICAL cache bytes. A row that the library recomputes (prompt fill, rebuild) may sit one
unit in the last place away from the oracle's, because the library accumulates the projection in float32 and the
oracle in float64 before the same rounding. So every such row is first checked against the oracle's (at most one
unit apart) and then copied into the oracle's cache, before any attention reads it: from there on the two attend
over the same numbers, and the comparison can be strict.

Bit-exact: slot maps, roles, admitted slot, evicted token, rebuild lists, and (after the copy) every occupied cache
row. Attention top-K sets must be equal except where the oracle's own logits of the swapped entries differ by less
than 1e-6 of the row's largest |logit| (the GPU ranks float32 logits, the oracle float64 ones); such near-ties are
counted and reported, and there is no other exemption. Attention output and weights within the dtype's tolerance.

Runs without a host wait between the steps (several steps in flight, the queued host-buffer entry point) cannot hand
their rebuilt rows over step by step; they are checked by running the same workload in lockstep first and requiring
the free run to repeat its outputs bit for bit.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

import workloads as wl
from oracle import adore_oracle as ao
from paper_2407_02328_b200 import adore as lib
from oracle.harness import Workload, make_oracle, explicit_as_lists, oracle_config

TOL = {"bf16": dict(out_abs=2e-2, out_rel=1e-2, w_abs=1e-3), "f32": dict(out_abs=1e-4, out_rel=1e-4, w_abs=1e-5)}
NEAR_TIE_REL = 1e-6


def torch_dtype(cfg: wl.WorkloadConfig):
    return torch.float32 if cfg.dtype == "f32" else torch.bfloat16


def to_dev(a: np.ndarray, cfg: wl.WorkloadConfig) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(torch_dtype(cfg)).contiguous()


def cache_flags(c: wl.WorkloadConfig) -> int:
    return ((lib.ADORE_FLAG_NO_RECURRENCE if c.ctrl_no_recurrence else 0) |
            (lib.ADORE_FLAG_SCORE_FROM_ATTENTION if c.score_from_attention else 0) |
            (lib.ADORE_FLAG_RELATIVE_POSITION if c.ctrl_relative_position else 0))


@dataclass
class Report:
    steps: int = 0
    near_ties: int = 0
    topk_rows: int = 0
    max_out_err: float = 0.0
    max_w_err: float = 0.0
    max_kv_ulp: float = 0.0
    rows_adopted: int = 0
    score_mismatch: int = 0
    record: List[List[tuple]] = field(default_factory=list)     # per step, per layer: (out, weights) of the library
    final: Optional[Dict[str, np.ndarray]] = None

    def line(self, name: str) -> str:
        return (f"[{name}] steps={self.steps} near_ties={self.near_ties}/{self.topk_rows} rows "
                f"max_out_err={self.max_out_err:.3e} max_w_err={self.max_w_err:.3e} max_kv_ulp={self.max_kv_ulp:.2f} "
                f"rows_adopted={self.rows_adopted} score_mismatch={self.score_mismatch}")


class GpuCache:
    """The library's cache with torch-owned device buffers for the per-step I/O. `w` gives the controller and (when
    `batch`/`cfg` are not given) the shape; `seqs` sequences and the layers `layers` are the ones a test compares."""

    def __init__(self, w: Workload, cfg: Optional[wl.WorkloadConfig] = None, batch: Optional[int] = None,
                 layers: Optional[Sequence[int]] = None, w_kv_dev: Optional[list] = None):
        c = self.cfg = w.cfg if cfg is None else cfg
        self.w = w
        self.B = w.batch if batch is None else batch
        self.seqs = w.batch                       # sequences the oracle follows (the first ones)
        self.layers = list(range(c.n_layers)) if layers is None else list(layers)
        self.handle = lib.adore_cache_create(
            lib.make_config(batch=self.B, n_layers=c.n_layers, n_heads=c.n_heads, head_dim=c.head_dim,
                            hidden=c.hidden, capacity=c.capacity, rebuild_max=c.rebuild_max, topk=c.topk,
                            max_tokens=c.max_tokens, ctrl_hidden=c.ctrl_hidden, dtype=c.dtype,
                            rebuild_mode=c.rebuild_mode, rope_theta=c.rope_theta, pos_scale=c.pos_scale,
                            flags=cache_flags(c)),
            w.ctrl, torch.cuda.current_stream().cuda_stream)
        self.w_kv_dev = [to_dev(m, c) for m in w.w_kv] if w_kv_dev is None else w_kv_dev
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

    # ---- views (restricted to the sequences the oracle follows) ----
    def slot_map(self):
        st, sr = lib.adore_cache_slot_map(self.handle)
        c = self.cfg
        return (lib.device_view(st, (self.B, c.capacity), torch.int32)[: self.seqs].cpu().numpy(),
                lib.device_view(sr, (self.B, c.capacity), torch.uint8)[: self.seqs].cpu().numpy())

    def step_info(self):
        a, e = lib.adore_cache_step_info(self.handle)
        return (lib.device_view(a, (self.B,), torch.int32)[: self.seqs].cpu().numpy(),
                lib.device_view(e, (self.B,), torch.int32)[: self.seqs].cpu().numpy())

    def rebuild_list(self):
        c = self.cfg
        if c.rebuild_max == 0:
            z = np.zeros((self.seqs, 0), np.int32)
            return z, z, np.zeros(self.seqs, np.int32)
        t, s, n = lib.adore_cache_rebuild_list(self.handle)
        return (lib.device_view(t, (self.B, c.rebuild_max), torch.int32)[: self.seqs].cpu().numpy(),
                lib.device_view(s, (self.B, c.rebuild_max), torch.int32)[: self.seqs].cpu().numpy(),
                lib.device_view(n, (self.B,), torch.int32)[: self.seqs].cpu().numpy())

    def scores(self, n):
        s, g = lib.adore_cache_scores(self.handle)
        c = self.cfg
        return (lib.device_view(s, (self.B, c.max_tokens), torch.float32)[: self.seqs, :n].cpu().numpy(),
                lib.device_view(g, (self.B, c.max_tokens), torch.float32)[: self.seqs, :n].cpu().numpy())

    def kv_views(self, layer):
        k, v = lib.adore_cache_kv(self.handle, layer)
        c = self.cfg
        shape = (self.B, c.n_heads, c.capacity, c.head_dim)
        return lib.device_view(k, shape, torch_dtype(c)), lib.device_view(v, shape, torch_dtype(c))

    def kv(self, layer):
        k, v = self.kv_views(layer)
        return k[: self.seqs].float().cpu().numpy(), v[: self.seqs].float().cpu().numpy()

    def kv_rows(self, layer, b_idx, s_idx):
        """K and V rows [n, H, dh] (float32 values of the stored elements) of the (sequence, slot) pairs given."""
        k, v = self.kv_views(layer)
        bi = torch.as_tensor(np.asarray(b_idx, np.int64), device="cuda")
        si = torch.as_tensor(np.asarray(s_idx, np.int64), device="cuda")
        return k[bi, :, si, :].float().cpu().numpy(), v[bi, :, si, :].float().cpu().numpy()

    def snapshot(self) -> Dict[str, np.ndarray]:
        """The library's exported small state, split into its sections (layout: include/adore.h)."""
        buf = np.zeros(lib.adore_cache_export_state(self.handle, None), np.uint8)
        lib.adore_cache_export_state(self.handle, buf)
        return parse_snapshot(buf, self.cfg, self.B)


def parse_snapshot(buf: np.ndarray, cfg: wl.WorkloadConfig, B: int) -> Dict[str, np.ndarray]:
    """Splits a buffer written by adore_cache_export_state into named arrays, following the layout the header documents:
    a 64-byte header, then the sections in a fixed order, each padded to 8 bytes."""
    hd = buf[:64].view(np.int32)
    assert hd[0] == 0x54534441 and hd[1] == 1, "not a version-1 snapshot"
    batch, capacity, rebuild_max, max_tokens, ctrl_hidden, n, cur, attn, step_open = (int(v) for v in hd[2:11])
    assert (batch, capacity, rebuild_max, max_tokens, ctrl_hidden) == (B, cfg.capacity, cfg.rebuild_max, cfg.max_tokens, cfg.ctrl_hidden)
    C, MT, h, r1 = capacity, max_tokens, ctrl_hidden, max(rebuild_max, 1)
    layout = [("slot_tok0", np.int32, (B, C)), ("slot_tok1", np.int32, (B, C)), ("slot_role0", np.uint8, (B, C)),
              ("slot_role1", np.uint8, (B, C)), ("tok_slot", np.int32, (B, MT)), ("score", np.float32, (B, MT)),
              ("sigma", np.float32, (B, MT)), ("z", np.float64, (B, h)), ("admit_slot", np.int32, (B,)),
              ("evicted_tok", np.int32, (B,)), ("rebuild_tok", np.int32, (B, r1)), ("rebuild_slot", np.int32, (B, r1)),
              ("rebuild_count", np.int32, (B,)), ("row_b", np.int32, (B * r1,)), ("row_tok", np.int32, (B * r1,)),
              ("row_slot", np.int32, (B * r1,)), ("row_total", np.int32, (1,))]
    if cfg.ctrl_relative_position:
        layout.append(("a_tab", np.float64, (B, MT, h)))
    out: Dict[str, np.ndarray] = {"n": np.int64(n), "cur": np.int64(cur), "attn": np.int64(attn), "step_open": np.int64(step_open)}
    off = 64
    for name, dt, shape in layout:
        nbytes = int(np.prod(shape)) * np.dtype(dt).itemsize
        out[name] = buf[off: off + nbytes].view(dt).reshape(shape).copy()
        off += (nbytes + 7) & ~7
    assert off == buf.nbytes, "snapshot size does not match its layout"
    out["slot_tok"] = out[f"slot_tok{cur}"]
    out["slot_role"] = out[f"slot_role{cur}"]
    return out


def _ulp(ref: np.ndarray, dtype: str) -> np.ndarray:
    """Size of one unit in the last place of the cache type at |ref| (floor at the smallest normal scale used)."""
    mant = 8 if dtype == "bf16" else 24
    e = np.floor(np.log2(np.maximum(np.abs(ref), 1e-30)))
    return np.exp2(e - (mant - 1))


def adopt_rows(rep: Report, g: GpuCache, orc: ao.AdoreOracle, layer: int, b_idx, s_idx, gpu_layer: Optional[int] = None) -> None:
    """The library's K/V rows of the given (sequence, slot) pairs: each element within one unit in the last place of the
    oracle's (float32 against float64 accumulation before the same rounding; sums that cancel to ~0 get a small
    absolute floor), then copied into the oracle's cache so that both sides attend over the same bytes."""
    if len(b_idx) == 0:
        return
    cfg = g.cfg
    b_idx, s_idx = np.asarray(b_idx, np.int64), np.asarray(s_idx, np.int64)
    Kg, Vg = g.kv_rows(layer if gpu_layer is None else gpu_layer, b_idx, s_idx)
    lim = 1.0 if cfg.dtype == "bf16" else 64.0          # f32: float32 accumulation over d terms
    floor = 1e-4 if cfg.dtype == "bf16" else 1e-5
    for name, G, O in (("K", Kg, orc.Kc[layer]), ("V", Vg, orc.Vc[layer])):
        ref = O[b_idx, :, s_idx, :]
        d = np.abs(G - ref)
        u = _ulp(ref, cfg.dtype)
        worst = float((d / u).max())
        assert (d <= lim * u + floor).all(), f"{name} cache rows off by {worst:.2f} ulp at step {rep.steps} (layer {layer})"
        rep.max_kv_ulp = max(rep.max_kv_ulp, worst)
        O[b_idx, :, s_idx, :] = G
    rep.rows_adopted += len(b_idx)


def adopt_rebuilt(rep: Report, g: GpuCache, orc: ao.AdoreOracle, layer: int, gpu_layer: Optional[int] = None) -> None:
    """After both sides rebuilt `layer`: hand the library's rebuilt rows to the oracle (see adopt_rows)."""
    bi, si = [], []
    for b in range(orc.cfg.batch):
        for s in orc.info.rebuild_slot[b]:
            bi.append(b)
            si.append(int(s))
    adopt_rows(rep, g, orc, layer, bi, si, gpu_layer)


def adopt_residents(rep: Report, g: GpuCache, orc: ao.AdoreOracle, layer: int, gpu_layer: Optional[int] = None) -> None:
    bi, si = np.nonzero(orc.slot_tok >= 0)
    adopt_rows(rep, g, orc, layer, bi, si, gpu_layer)


def compare_attention(rep: Report, cfg, q, k_new, Kc_before, Vc_before, attn_map, out_g, w_g, out_o, w_o, own_row=True):
    """out/weights of one attention launch for the compared sequences. Kc_before/Vc_before: the oracle's cache rows the
    attention read (the same bytes the library read); attn_map [B, C]: which slots it saw (< 0: not visible)."""
    tol = TOL[cfg.dtype]
    err = np.abs(out_g - out_o)
    bound = tol["out_abs"] + tol["out_rel"] * np.abs(out_o)
    keep_g, keep_o = w_g > 0, w_o > 0
    rep.topk_rows += keep_o.shape[0] * keep_o.shape[1]
    w_ok = np.ones_like(keep_o)
    for b, h in np.argwhere((keep_g != keep_o).any(-1)):
        # the only exemption: the swapped entries' float64 logits lie within 1e-6 (relative to the row's logit scale) of
        # the threshold, so float32 ranking may order them either way
        Kall = np.concatenate([Kc_before[b, h].astype(np.float64), k_new[b, h][None].astype(np.float64)])
        logit = Kall @ q[b, h].astype(np.float64) / np.sqrt(cfg.head_dim)
        valid = np.concatenate([attn_map[b] >= 0, [own_row]])
        scale = max(1.0, float(np.abs(logit[valid]).max()))
        diff = np.nonzero(keep_g[b, h] != keep_o[b, h])[0]
        assert keep_g[b, h].sum() == keep_o[b, h].sum(), "kept count differs"
        assert valid[diff].all(), "an empty slot was kept"
        thr = logit[keep_o[b, h]].min()
        gap = np.abs(logit[diff] - thr).max()
        assert gap <= NEAR_TIE_REL * scale, \
            f"top-K sets differ beyond a near-tie: gap {gap:.3e}, scale {scale:.3e} (step {rep.steps}, b {b}, h {h})"
        rep.near_ties += 1
        w_ok[b, h, diff] = False
        # equal logits carry equal weights: the outputs differ by that weight times the difference of the swapped value rows
        moved = 0.5 * (np.abs(w_g[b, h, diff]).sum() + np.abs(w_o[b, h, diff]).sum())
        bound[b, h] = bound[b, h] + moved * 2.0 * float(np.abs(Vc_before[b, h]).max())
    assert (err <= bound).all(), f"attention output off by {err.max():.3e} (step {rep.steps})"
    rep.max_out_err = max(rep.max_out_err, float(err.max()))
    werr = np.abs(w_g - w_o)
    assert (werr <= tol["w_abs"])[w_ok].all(), f"attention weights off by {werr[w_ok].max():.3e} (step {rep.steps})"
    rep.max_w_err = max(rep.max_w_err, float(werr[w_ok].max()))
    assert np.allclose(w_g.sum(-1), 1.0, atol=1e-4), "weights do not sum to one"


def compare_state(rep: Report, g: GpuCache, orc: ao.AdoreOracle, layers, check_scores=True, score_rtol=1e-6,
                  kv: str = "equal", gpu_layers: Optional[Sequence[int]] = None):
    """Small state bit for bit; cache rows of the occupied slots: kv="adopt" checks them to one unit in the last place
    and hands them to the oracle (after a prompt fill), kv="equal" requires the bytes both sides hold to be the same."""
    cfg = g.cfg
    st, sr = g.slot_map()
    assert np.array_equal(st, orc.slot_tok), f"slot map differs at step {rep.steps}"
    assert np.array_equal(sr, orc.slot_role), f"slot roles differ at step {rep.steps}"
    adm, ev = g.step_info()
    assert np.array_equal(adm, orc.info.admit_slot) and np.array_equal(ev, orc.info.evicted_tok)
    lt, ls, ln = g.rebuild_list()
    for b in range(g.seqs):
        k = len(orc.info.rebuild_tok[b])
        assert ln[b] == k, f"rebuild count differs (b={b}): {ln[b]} vs {k}"
        assert np.array_equal(lt[b, :k], orc.info.rebuild_tok[b]) and np.array_equal(ls[b, :k], orc.info.rebuild_slot[b])
    if check_scores:
        sc, sg = g.scores(orc.n)
        rep.score_mismatch += int((sc != orc.score[:, : orc.n]).sum())
        assert np.allclose(sc, orc.score[:, : orc.n], rtol=score_rtol, atol=1e-9)
        assert np.allclose(sg, orc.sigma[:, : orc.n], rtol=1e-6, atol=1e-9)
    occ = orc.slot_tok >= 0
    for l in layers:
        gl = l if gpu_layers is None else gpu_layers[l]
        if kv == "adopt":
            adopt_residents(rep, g, orc, l, gl)
            continue
        Kg, Vg = g.kv(gl)
        m = np.broadcast_to(occ[:, None, :, None], Kg.shape)
        assert np.array_equal(Kg[m], orc.Kc[l][m]), f"K rows of layer {gl} differ at step {rep.steps}"
        assert np.array_equal(Vg[m], orc.Vc[l][m]), f"V rows of layer {gl} differ at step {rep.steps}"


def final_state(g: GpuCache, n: int) -> Dict[str, np.ndarray]:
    """Everything observable at the end of a run (cache rows of empty slots zeroed: they hold stale bytes)."""
    lib.adore_cache_sync_status(g.handle)
    st, sr = g.slot_map()
    sc, sg = g.scores(n)
    occ = (st >= 0)[:, None, :, None]
    out = dict(slot_tok=st, slot_role=sr, score=sc, sigma=sg)
    for l in range(g.cfg.n_layers):
        k, v = g.kv(l)
        out[f"k{l}"], out[f"v{l}"] = np.where(occ, k, 0), np.where(occ, v, 0)
    return out


def _tables(cfg, w: Workload, g: GpuCache, orc: Optional[ao.AdoreOracle], all_rows: bool, n_steps: int):
    """Per-layer input tables (device for the library, host for the oracle) and the prompt fill of layers > 0."""
    L = cfg.n_layers
    if not cfg.per_layer_inputs:
        return None, None
    tables = [torch.zeros((g.B, cfg.max_tokens, cfg.hidden), dtype=torch_dtype(cfg), device="cuda") for _ in range(L)]
    otab = [np.zeros((g.B, cfg.max_tokens, cfg.hidden), np.float32) for _ in range(L)]
    upto = cfg.prompt + n_steps if all_rows else cfg.prompt      # a free run's tables hold every row from the start
    for l in range(L):
        for t0 in range(0, upto, 64):
            otab[l][:, t0: min(upto, t0 + 64)] = w.rows(t0, min(64, upto - t0), l)
        if upto:
            tables[l][:, :upto] = to_dev(otab[l][:, :upto], cfg)
        if l > 0 and cfg.prompt:
            if orc is not None:
                orc.fill_layer(l, otab[l])
            lib.adore_cache_fill_layer(g.handle, l, tables[l])
    return tables, otab


def run_parity(cfg: wl.WorkloadConfig, batch: Optional[int] = None, steps: Optional[int] = None,
               state_every: int = 1, host_entry=False, record: bool = False) -> Report:
    """Lockstep parity of the attend-first step: both sides consume the same inputs and must agree at every step; the
    library's recomputed rows are handed to the oracle before the next attention reads them (see the module text)."""
    w = Workload(cfg, batch)
    orc = make_oracle(w)
    g = GpuCache(w)
    rep = Report()
    L = cfg.n_layers
    n_steps = cfg.steps if steps is None else steps
    try:
        tables = otab = None
        if cfg.prompt:
            xp = w.prompt()
            orc.append_tokens(xp)
            lib.adore_cache_append_tokens(g.handle, to_dev(xp, cfg), cfg.prompt)
        tables, otab = _tables(cfg, w, g, orc, False, n_steps)
        if cfg.prompt:
            lib.adore_cache_sync_status(g.handle)
            compare_state(rep, g, orc, range(L), kv="adopt")
        for s in range(n_steps):
            n = orc.n
            lists, counts = w.explicit(s, n)
            ex = explicit_as_lists(lists, counts)
            dl = torch.from_numpy(lists).cuda() if lists is not None else None
            dc = torch.from_numpy(counts).cuda() if counts is not None else None
            rec = []
            for l in range(L):
                x = w.x_new(n, l)
                q, k, v = w.qkv(n, l, x)
                if cfg.per_layer_inputs:
                    otab[l][:, n] = x
                    tables[l][:, n] = to_dev(x, cfg)
                attn_map = orc.slot_tok.copy() if l == 0 else orc.attn_slot_tok.copy()
                K_before, V_before = orc.Kc[l].copy(), orc.Vc[l].copy()
                out_o, w_o = orc.decode_step(l, q, k, v, x if l == 0 else None, ex if l == 0 else None)
                x_tab = tables[l] if (cfg.per_layer_inputs and l > 0) else None
                if host_entry:
                    hq, hk, hv, hx = (to_dev(a, cfg).cpu() for a in (q, k, v, x))
                    hout = torch.zeros((g.B, cfg.n_heads, cfg.head_dim), dtype=torch_dtype(cfg))
                    if host_entry == "with_rebuild":     # the call that also queues the layer's rebuild
                        lib.adore_decode_rebuild_host(g.handle, l, hq, hk, hv, hx, lists if l == 0 else None,
                                                      counts if l == 0 else None, w.r_in if l == 0 else 0, x_tab, hout, g.weights)
                    else:
                        lib.adore_decode_step_host(g.handle, l, hq, hk, hv, hx, lists if l == 0 else None,
                                                   counts if l == 0 else None, w.r_in if l == 0 else 0, hout, g.weights)
                    out_g, w_g = hout.float().numpy(), g.weights.cpu().numpy()
                else:
                    lib.adore_decode_step(g.handle, l, to_dev(q, cfg), to_dev(k, cfg), to_dev(v, cfg), to_dev(x, cfg),
                                          dl if l == 0 else None, dc if l == 0 else None, w.r_in if l == 0 else 0,
                                          g.out, g.weights)
                    out_g, w_g = g.out.float().cpu().numpy(), g.weights.cpu().numpy()
                if record:
                    rec.append((out_g.copy(), w_g.copy()))
                compare_attention(rep, cfg, q, k, K_before, V_before, attn_map, out_g, w_g, out_o, w_o)
                orc.rebuild(l, otab[l] if (cfg.per_layer_inputs and l > 0) else None)
                if host_entry != "with_rebuild":
                    lib.adore_rebuild(g.handle, l, x_tab)
                adopt_rebuilt(rep, g, orc, l)
            rep.record.append(rec)
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
        if record:
            rep.final = final_state(g, orc.n)
    finally:
        g.close()
    return rep


def run_free(cfg: wl.WorkloadConfig, batch: Optional[int] = None, steps: Optional[int] = None, mode: str = "device",
             sync_every: int = 0):
    """The library alone, with no host wait between the calls: every step's inputs are on the device (or, for the queued
    host-buffer entry point, in pinned host memory) before the first call; outputs go to per-step buffers.
    mode "device": adore_decode_step + adore_rebuild; "queued_host": adore_decode_rebuild_host_queued, the host waiting
    with adore_cache_wait_outputs every `sync_every` steps (0: only at the end).
    Returns (record, final) in the shape of Report.record / Report.final."""
    w = Workload(cfg, batch)
    g = GpuCache(w)
    L = cfg.n_layers
    n_steps = cfg.steps if steps is None else steps
    host = mode == "queued_host"
    place = (lambda a: to_dev(a, cfg).cpu().pin_memory()) if host else (lambda a: to_dev(a, cfg))
    try:
        if cfg.prompt:
            lib.adore_cache_append_tokens(g.handle, to_dev(w.prompt(), cfg), cfg.prompt)
        tables, _ = _tables(cfg, w, g, None, True, n_steps)
        plan = []
        for s in range(n_steps):
            n = cfg.prompt + s
            lists, counts = w.explicit(s, n)
            if host:
                dl = None if lists is None else torch.from_numpy(lists).pin_memory()
                dc = None if counts is None else torch.from_numpy(counts).pin_memory()
            else:
                dl = None if lists is None else torch.from_numpy(lists).cuda()
                dc = None if counts is None else torch.from_numpy(counts).cuda()
            per_layer = []
            for l in range(L):
                x = w.x_new(n, l)
                q, k, v = w.qkv(n, l, x)
                per_layer.append(tuple(place(a) for a in (q, k, v, x)))
            plan.append((dl, dc, per_layer))
        shape_o = (n_steps, L, g.B, cfg.n_heads, cfg.head_dim)
        outs = torch.zeros(shape_o, dtype=torch_dtype(cfg)).pin_memory() if host else torch.zeros(shape_o, dtype=torch_dtype(cfg), device="cuda")
        wts = torch.zeros((n_steps, L, g.B, cfg.n_heads, cfg.capacity + 1), dtype=torch.float32, device="cuda")
        lib.adore_cache_sync_status(g.handle)
        for s, (dl, dc, per_layer) in enumerate(plan):
            for l, (q, k, v, x) in enumerate(per_layer):
                x_tab = tables[l] if (tables is not None and l > 0) else None
                first = l == 0
                if host:
                    lib.adore_decode_rebuild_host_queued(g.handle, l, q, k, v, x if first else None, dl if first else None,
                                                         dc if first else None, w.r_in if first else 0, x_tab, outs[s, l], wts[s, l])
                else:
                    lib.adore_decode_step(g.handle, l, q, k, v, x if first else None, dl if first else None,
                                          dc if first else None, w.r_in if first else 0, outs[s, l], wts[s, l])
                    lib.adore_rebuild(g.handle, l, x_tab)
            if host and sync_every and (s + 1) % sync_every == 0:
                lib.adore_cache_wait_outputs(g.handle)      # the outputs are in; the rebuilds may still be running
        final = final_state(g, cfg.prompt + n_steps)
        o, ww = outs.float().cpu().numpy(), wts.cpu().numpy()
        record = [[(o[s, l], ww[s, l]) for l in range(L)] for s in range(n_steps)]
        return record, final
    finally:
        g.close()


def assert_same_run(rep: Report, record, final, what: str) -> None:
    """A free run must repeat the lockstep run's outputs, weights and final state bit for bit."""
    assert len(record) == len(rep.record)
    for s, (a, b) in enumerate(zip(rep.record, record)):
        for l, ((o1, w1), (o2, w2)) in enumerate(zip(a, b)):
            assert np.array_equal(o1, o2), f"{what}: out differs at step {s}, layer {l}"
            assert np.array_equal(w1, w2), f"{what}: weights differ at step {s}, layer {l}"
    for key, val in rep.final.items():
        assert np.array_equal(val, final[key]), f"{what}: {key} differs at the end"


def run_parity_rebuild_first(cfg: wl.WorkloadConfig, steps: Optional[int] = None) -> Report:
    """Lockstep parity of the step in the order Section 2.3 prints it: adore_step_begin, then per layer adore_rebuild
    and adore_attend_rows (R_max + 1 query rows per sequence), against the oracle's same three calls. Every layer
    rebuilds from the token store; the rebuilt rows are handed to the oracle before the layer's attention reads them."""
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
            compare_state(rep, g, orc, range(L), kv="adopt")
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
                adopt_rebuilt(rep, g, orc, l)
                q_rows = w.q_rows(n, l, orc.x, orc.info.rebuild_tok)
                K_before, V_before = orc.Kc[l].copy(), orc.Vc[l].copy()
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
                    compare_attention(rep, cfg, q_rows[idx, :, i], k[idx], K_before[idx], V_before[idx], seen, out_g[idx, :, i],
                                      w_g[idx, :, i], out_o[idx, :, i], w_o[idx, :, i], own_row=(i == R1 - 1))
            rep.steps += 1
            lib.adore_cache_sync_status(g.handle)
            orc.check_invariants()
            compare_state(rep, g, orc, range(L))
        lib.adore_cache_sync_status(g.handle)
    finally:
        g.close()
    return rep


# --------------------------------------------------------------------------------------------------------------------
# large configurations: the library runs the whole shape, the oracle follows some sequences and layers
# --------------------------------------------------------------------------------------------------------------------
class _DeviceInputs:
    """Inputs of a full-shape run. The sequences and layers the oracle follows get the seeded numpy numbers of the
    workload; every other sequence (and the projections of every other layer) gets device-drawn numbers of the same
    distribution. During the free steps q, k_new and v_new of ALL sequences are float32 projections made on the device:
    what reaches the cache through them is checked against the oracle's definition when the oracle takes the rows over."""

    def __init__(self, cfg: wl.WorkloadConfig, w: Workload, layers: Sequence[int]):
        self.cfg, self.w, self.layers = cfg, w, list(layers)
        self.dt = torch_dtype(cfg)
        self.gen = torch.Generator(device="cuda")
        self.gen.manual_seed(cfg.seed)
        N = cfg.n_heads * cfg.head_dim
        self.w_kv, self.w_q = [], []
        for l in range(cfg.n_layers):
            if l in self.layers:
                i = self.layers.index(l)
                self.w_kv.append(to_dev(w.w_kv[i], cfg))
                self.w_q.append(to_dev(w.w_q[i], cfg))
            else:
                self.w_kv.append((torch.randn((2 * N, cfg.hidden), generator=self.gen, device="cuda") * 0.02).to(self.dt))
                self.w_q.append((torch.randn((N, cfg.hidden), generator=self.gen, device="cuda") * 0.02).to(self.dt))

    def rows(self, first: int, count: int, layer: int) -> torch.Tensor:
        """[B, count, d] layer-input rows: the first sequences from the workload (layers the oracle follows), the rest drawn here."""
        cfg, w = self.cfg, self.w
        x = torch.randn((cfg.batch, count, cfg.hidden), generator=self.gen, device="cuda")
        if cfg.per_layer_inputs:
            x = x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + 1e-5)
        x = x.to(self.dt)
        src = layer if cfg.per_layer_inputs else 0
        if src in self.layers:
            i = self.layers.index(src)
            for t0 in range(0, count, 64):
                c1 = min(64, count - t0)
                x[: w.batch, t0: t0 + c1] = to_dev(w.rows(first + t0, c1, i), cfg)
        return x

    def rope(self, y: torch.Tensor, n: int) -> torch.Tensor:
        c = self.cfg
        if c.rope_theta == 0.0:
            return y
        j = torch.arange(c.head_dim // 2, device=y.device, dtype=torch.float64)
        ang = n * torch.pow(torch.tensor(c.rope_theta, dtype=torch.float64, device=y.device), -2.0 * j / c.head_dim)
        cs, sn = torch.cos(ang).float(), torch.sin(ang).float()
        a, b = y[..., 0::2], y[..., 1::2]
        out = torch.empty_like(y)
        out[..., 0::2] = a * cs - b * sn
        out[..., 1::2] = a * sn + b * cs
        return out

    def qkv(self, n: int, layer: int, x: torch.Tensor):
        c = self.cfg
        B, H, dh = x.shape[0], c.n_heads, c.head_dim
        kv = x.float() @ self.w_kv[layer].float().t()
        k = self.rope(kv[:, : H * dh].reshape(B, H, dh), n).to(self.dt)
        v = kv[:, H * dh:].reshape(B, H, dh).to(self.dt)
        q = (c.q_scale * self.rope((x.float() @ self.w_q[layer].float().t()).reshape(B, H, dh), n)).to(self.dt)
        return q.contiguous(), k.contiguous(), v.contiguous()

    def explicit(self, step: int, n: int):
        """Device lists [B, r_in] / counts [B]: the followed sequences' flags from the workload, the others drawn here."""
        c, w = self.cfg, self.w
        if c.rebuild_mode != "explicit":
            return None, None, None
        r_in = w.r_in
        flag = torch.rand((c.batch, max(n, 1)), generator=self.gen, device="cuda")[:, :n] < c.rebuild_p
        key = torch.where(flag, torch.arange(n, device="cuda").expand(c.batch, n), torch.full((c.batch, n), 1 << 30, device="cuda"))
        srt = key.sort(dim=1).values[:, :r_in]
        lists = torch.full((c.batch, r_in), -1, dtype=torch.int32, device="cuda")
        lists[:, : srt.shape[1]] = torch.where(srt < (1 << 30), srt, torch.full_like(srt, -1)).to(torch.int32)
        counts = flag.sum(1).clamp(max=r_in).to(torch.int32)
        hl, hc = w.explicit(step, n)
        lists[: w.batch] = torch.from_numpy(hl).cuda()
        counts[: w.batch] = torch.from_numpy(hc).cuda()
        return lists.contiguous(), counts.contiguous(), explicit_as_lists(hl, hc)


def run_sampled_parity(cfg: wl.WorkloadConfig, free_steps: int, check_steps: int, seqs: int = 2,
                       layers: Optional[Sequence[int]] = None) -> Report:
    """Parity of a large configuration at full size. The library holds ALL sequences and ALL layers of `cfg` and runs
    `free_steps` decode steps with no host wait and no help from the oracle; the oracle follows the first `seqs`
    sequences, simulating scoring and selection alone (the small state does not depend on any attention result).
    Then the two small states must be equal bit for bit, the oracle adopts the library's exported state through its
    own import_state (K/V by definition for the layers in `layers`), takes over the library's cache rows after the
    one-unit row check, and `check_steps` steps run in lockstep with every output of those sequences and layers
    compared as in run_parity."""
    layers = list(range(cfg.n_layers)) if layers is None else list(layers)
    w = Workload(cfg, seqs, layers)
    assert layers[0] == 0, "scoring and selection belong to layer 0"
    sim = ao.AdoreOracle(oracle_config(w.cfg, seqs), w.ctrl)     # no projection: scores and selection only
    inp = _DeviceInputs(cfg, w, layers)
    g = GpuCache(w, cfg=cfg, batch=cfg.batch, layers=layers, w_kv_dev=inp.w_kv)
    rep = Report()
    L = cfg.n_layers
    per_layer = cfg.per_layer_inputs
    try:
        tables = None
        if per_layer:
            tables = [torch.zeros((cfg.batch, cfg.max_tokens, cfg.hidden), dtype=inp.dt, device="cuda") for _ in range(L)]
        if cfg.prompt:
            xp = inp.rows(0, cfg.prompt, 0)
            lib.adore_cache_append_tokens(g.handle, xp, cfg.prompt)
            sim.append_tokens(w.prompt(0))                       # no projection set: scores and selection only
            if per_layer:
                tables[0][:, : cfg.prompt] = xp
                for l in range(1, L):
                    tables[l][:, : cfg.prompt] = inp.rows(0, cfg.prompt, l)
                    lib.adore_cache_fill_layer(g.handle, l, tables[l])
            del xp
        out_dev = torch.empty((L, cfg.batch, cfg.n_heads, cfg.head_dim), dtype=inp.dt, device="cuda")
        w_dev = torch.empty((L, cfg.batch, cfg.n_heads, cfg.capacity + 1), dtype=torch.float32, device="cuda")
        # ---- free steps: the library alone; the oracle's small state follows on its own ----
        for s in range(free_steps):
            n = cfg.prompt + s
            dl, dc, ex = inp.explicit(s, n)
            x0 = None
            for l in range(L):
                x = inp.rows(n, 1, l)[:, 0].contiguous() if (per_layer or l == 0) else x0
                if l == 0:
                    x0 = x
                if per_layer:
                    tables[l][:, n] = x
                q, k, v = inp.qkv(n, l, x)
                lib.adore_decode_step(g.handle, l, q, k, v, x if l == 0 else None, dl if l == 0 else None,
                                      dc if l == 0 else None, w.r_in if l == 0 else 0, out_dev[l], w_dev[l])
                lib.adore_rebuild(g.handle, l, tables[l] if (per_layer and l > 0) else None)
            sim.step_begin(w.x_new(n, 0), ex)
        lib.adore_cache_sync_status(g.handle)
        sim.check_invariants()
        # ---- the two small states, bit for bit; then the oracle that goes on is made from the library's export ----
        compare_state(rep, g, sim, [])
        snap = g.snapshot()
        n_now = int(snap["n"])
        assert n_now == sim.n
        orc = make_oracle(w)
        x_tabs = []
        for i in range(len(layers)):
            t = np.zeros((seqs, cfg.max_tokens, cfg.hidden), np.float32)
            for t0 in range(0, n_now, 64):
                t[:, t0: min(n_now, t0 + 64)] = w.rows(t0, min(64, n_now - t0), i)
            x_tabs.append(t)
        cnt = snap["rebuild_count"][:seqs]
        orc.import_state(n_now, snap["slot_tok"][:seqs], snap["slot_role"][:seqs], snap["score"][:seqs], snap["sigma"][:seqs],
                         snap["z"][:seqs], x_tabs[0], [snap["rebuild_tok"][b, : cnt[b]] for b in range(seqs)],
                         [snap["rebuild_slot"][b, : cnt[b]] for b in range(seqs)], snap["admit_slot"][:seqs],
                         snap["evicted_tok"][:seqs], x_tables=x_tabs if per_layer else None)
        assert np.array_equal(orc.tok_slot, sim.tok_slot) and np.array_equal(orc.tok_slot[:, :n_now], snap["tok_slot"][:seqs, :n_now])
        assert np.allclose(orc.z, sim.z, rtol=1e-12, atol=1e-15), "GRU state of the library and of the oracle's own scan differ"
        compare_state(rep, g, orc, range(len(layers)), kv="adopt", gpu_layers=layers)
        # ---- lockstep steps ----
        for s in range(free_steps, free_steps + check_steps):
            n = orc.n
            dl, dc, ex = inp.explicit(s, n)
            x0 = None
            for l in range(L):
                x = inp.rows(n, 1, l)[:, 0].contiguous() if (per_layer or l == 0) else x0
                if l == 0:
                    x0 = x
                if per_layer:
                    tables[l][:, n] = x
                q, k, v = inp.qkv(n, l, x)
                i = layers.index(l) if l in layers else -1
                if i >= 0:                                    # the followed sequences get the harness's own q, k, v
                    xo = w.x_new(n, i)
                    assert np.array_equal(xo, x[:seqs].float().cpu().numpy())
                    qo, ko, vo = w.qkv(n, i, xo)
                    q[:seqs], k[:seqs], v[:seqs] = to_dev(qo, cfg), to_dev(ko, cfg), to_dev(vo, cfg)
                    if per_layer:
                        x_tabs[i][:, n] = xo
                    attn_map = orc.slot_tok.copy() if i == 0 else orc.attn_slot_tok.copy()
                    K_before, V_before = orc.Kc[i].copy(), orc.Vc[i].copy()
                    out_o, w_o = orc.decode_step(i, qo, ko, vo, xo if i == 0 else None, ex if i == 0 else None)
                lib.adore_decode_step(g.handle, l, q, k, v, x if l == 0 else None, dl if l == 0 else None,
                                      dc if l == 0 else None, w.r_in if l == 0 else 0, out_dev[l], w_dev[l])
                lib.adore_rebuild(g.handle, l, tables[l] if (per_layer and l > 0) else None)
                if i >= 0:
                    out_g, w_g = out_dev[l, :seqs].float().cpu().numpy(), w_dev[l, :seqs].cpu().numpy()
                    compare_attention(rep, cfg, qo, ko, K_before, V_before, attn_map, out_g, w_g, out_o, w_o)
                    orc.rebuild(i, x_tabs[i] if (per_layer and i > 0) else None)
                    adopt_rebuilt(rep, g, orc, i, l)
            rep.steps += 1
            lib.adore_cache_sync_status(g.handle)
            orc.check_invariants()
            compare_state(rep, g, orc, range(len(layers)), gpu_layers=layers)
    finally:
        g.close()
    return rep
