"""Drives the oracle over a workload (test infrastructure, like the rest of this package).

The per-step inputs come from `workloads` (random numbers only). Queries and the current
token's key/value rows are the harness's stand-in for the backbone model: they are made
here from the same hidden row with the oracle's projection, so that a token admitted with
k_new and later rebuilt from x must get the same cache row back.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import numpy as np

import workloads as wl
from oracle import adore_oracle as ao


def oracle_config(cfg: wl.WorkloadConfig, batch: Optional[int] = None) -> ao.OracleConfig:
    return ao.OracleConfig(batch=cfg.batch if batch is None else batch, n_layers=cfg.n_layers,
                           n_heads=cfg.n_heads, head_dim=cfg.head_dim, hidden=cfg.hidden,
                           capacity=cfg.capacity, rebuild_max=cfg.rebuild_max, topk=cfg.topk,
                           max_tokens=cfg.max_tokens, ctrl_hidden=cfg.ctrl_hidden, dtype=cfg.dtype,
                           rebuild_mode=cfg.rebuild_mode, rope_theta=cfg.rope_theta,
                           pos_scale=cfg.pos_scale, no_recurrence=cfg.ctrl_no_recurrence,
                           score_from_attention=cfg.score_from_attention,
                           relative_position=cfg.ctrl_relative_position)


class Workload:
    """Seeded inputs of one config, restricted to the first `batch` sequences and, with `layers`, to some of its
    layers: layer index l of this object (and of the oracle made from it) then stands for layer layers[l] of `cfg`."""

    def __init__(self, cfg: wl.WorkloadConfig, batch: Optional[int] = None, layers: Optional[List[int]] = None):
        self.batch = cfg.batch if batch is None else batch
        self.layers = list(range(cfg.n_layers)) if layers is None else list(layers)
        self.full_cfg = cfg                                   # what the random streams are keyed by
        self.cfg = cfg if layers is None else cfg.scaled(n_layers=len(self.layers))
        # every random tensor is drawn row by row from one stream, so a generator asked for fewer sequences returns the
        # same first rows: the numbers are drawn for `batch` sequences only
        self.gen_cfg = cfg.scaled(batch=self.batch)
        self.ctrl = wl.controller_weights(cfg)
        self.w_kv = [wl.projection_weights(cfg, l) for l in self.layers]
        self.w_q = [wl.query_weights(cfg, l) for l in self.layers]
        self.w_kv64 = [w.astype(np.float64) for w in self.w_kv]
        self.w_q64 = [w.astype(np.float64) for w in self.w_q]
        self.r_in = self._r_in()

    def _r_in(self) -> int:
        if self.cfg.rebuild_mode != "explicit":
            return 0
        n = max(self.cfg.max_tokens, 1)
        mean = n * self.cfg.rebuild_p
        return int(min(n, np.ceil(mean + 6 * np.sqrt(mean) + 8)))

    def rows(self, first: int, count: int, layer: int = 0) -> np.ndarray:
        """Layer-input rows [batch, count, d] of tokens first .. first+count-1 for this object's layer `layer`."""
        src = self.layers[layer] if self.cfg.per_layer_inputs else 0
        return wl.hidden_rows(self.gen_cfg, first, count, src, self.batch)

    def prompt(self, layer: int = 0) -> np.ndarray:
        return self.rows(0, self.cfg.prompt, layer)

    def x_new(self, n: int, layer: int = 0) -> np.ndarray:
        return self.rows(n, 1, layer)[:, 0, :]

    def qkv(self, n: int, layer: int, x_row: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """q, k_new, v_new [B, H, dh] of the token at position n (all sequences in one product)."""
        c = self.cfg
        B, hd = x_row.shape[0], c.n_heads * c.head_dim
        x64 = x_row.astype(np.float64)
        ykv = x64 @ self.w_kv64[layer].T
        k = ao.round_store(ao.rope_rotate(ykv[:, :hd].reshape(B, c.n_heads, c.head_dim), n, c.rope_theta), c.dtype)
        v = ao.round_store(ykv[:, hd:].reshape(B, c.n_heads, c.head_dim), c.dtype)
        if c.identity_projection:          # q, k, v i.i.d. N(0,1): q is its own draw
            q = np.stack([wl.gaussian(c.seed, "q", (c.n_heads, c.head_dim), 1.0, c.dtype, idx=(self.layers[layer], n, b))
                          for b in range(B)])
        else:
            yq = x64 @ self.w_q64[layer].T
            q = ao.round_store(c.q_scale * ao.rope_rotate(yq.reshape(B, c.n_heads, c.head_dim), n, c.rope_theta), c.dtype)
        return q, k, v

    def q_rows(self, n: int, layer: int, x_table: np.ndarray, lists) -> np.ndarray:
        """Query rows [B, H, R_max+1, dh] of the step in the order of Section 2.3: row i < R_max for the i-th token of
        sequence b's rebuild list (zeros past the list's end), the last row for the current token n; each row is
        projected from that token's layer input x_table[b, tok] and rotated to the token's own position."""
        c = self.cfg
        R1 = c.rebuild_max + 1
        out = np.zeros((self.batch, c.n_heads, R1, c.head_dim), np.float32)
        for b in range(self.batch):
            toks = [int(t) for t in lists[b]] + [-1] * (c.rebuild_max - len(lists[b])) + [n]
            for i, tok in enumerate(toks):
                if tok < 0:
                    continue
                if c.identity_projection:
                    out[b, :, i] = wl.gaussian(c.seed, "q", (c.n_heads, c.head_dim), 1.0, c.dtype, idx=(self.layers[layer], tok, b))
                else:
                    out[b, :, i] = ao.project_q(self.w_q64[layer], x_table[b, tok], tok, c.n_heads, c.head_dim,
                                                c.rope_theta, c.dtype)
        return out

    def explicit(self, step: int, n: int) -> Tuple[Optional[np.ndarray], Optional[np.ndarray]]:
        if self.cfg.rebuild_mode != "explicit":
            return None, None
        return wl.rebuild_flags(self.gen_cfg, step, n, self.r_in, self.batch)


def make_oracle(w: Workload) -> ao.AdoreOracle:
    orc = ao.AdoreOracle(oracle_config(w.cfg, w.batch), w.ctrl)
    for l in range(w.cfg.n_layers):
        orc.set_projection(l, w.w_kv64[l])
    return orc


def explicit_as_lists(lists: Optional[np.ndarray], counts: Optional[np.ndarray]) -> Optional[List[np.ndarray]]:
    if lists is None:
        return None
    return [lists[b, : counts[b]] for b in range(lists.shape[0])]
