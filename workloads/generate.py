"""Seeded random tensors for the workloads. Numbers only: no method arithmetic here.

Every tensor has its own sub-stream, keyed by (config seed, tensor name, optional
indices), so that a tensor's values do not depend on which other tensors were drawn or
in what order. All arrays come back as float32 whose values are exactly representable
in the config's element type, so both consumers start from identical inputs.
"""
from __future__ import annotations

import zlib
from typing import Dict, Tuple

import numpy as np

from .configs import WorkloadConfig


def substream(seed: int, name: str, *idx: int) -> np.random.Generator:
    key = [int(seed) & 0xFFFFFFFF, zlib.crc32(name.encode()) & 0xFFFFFFFF]
    key.extend(int(i) & 0xFFFFFFFF for i in idx)
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(key)))


def round_to_dtype(a: np.ndarray, dtype: str) -> np.ndarray:
    """Return float32 values representable in `dtype` ("f32" or "bf16", nearest-even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    bits = a.view(np.uint32).astype(np.uint64)
    bits = bits + 0x7FFF + ((bits >> 16) & 1)
    return (bits & 0xFFFF0000).astype(np.uint32).view(np.float32).reshape(a.shape)


def gaussian(seed: int, name: str, shape: Tuple[int, ...], std: float = 1.0,
             dtype: str = "f32", idx: Tuple[int, ...] = ()) -> np.ndarray:
    g = substream(seed, name, *idx)
    a = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return round_to_dtype(a, dtype)


def controller_weights(cfg: WorkloadConfig, std: float | None = None) -> Dict[str, np.ndarray]:
    """Random-init controller: GRU(d -> d'), position FC(1 -> d'), FC(d' -> d'), FC(d' -> 1).

    Gate order of the stacked GRU matrices is reset, update, candidate. All fp32. The standard deviation is the
    config's `ctrl_weight_std` (0.02) unless given.
    """
    d, h, s = cfg.hidden, cfg.ctrl_hidden, cfg.seed
    std = cfg.ctrl_weight_std if std is None else std
    return {
        "gru_w_ih": gaussian(s, "gru_w_ih", (3 * h, d), std),
        "gru_w_hh": gaussian(s, "gru_w_hh", (3 * h, h), std),
        "gru_b_ih": gaussian(s, "gru_b_ih", (3 * h,), std),
        "gru_b_hh": gaussian(s, "gru_b_hh", (3 * h,), std),
        "pos_w": gaussian(s, "pos_w", (h,), std),
        "pos_b": gaussian(s, "pos_b", (h,), std),
        "mlp_w1": gaussian(s, "mlp_w1", (h, h), std),
        "mlp_b1": gaussian(s, "mlp_b1", (h,), std),
        "mlp_w2": gaussian(s, "mlp_w2", (h,), std),
        "mlp_b2": gaussian(s, "mlp_b2", (1,), std),
    }


def hidden_rows(cfg: WorkloadConfig, first_token: int, count: int, layer: int = 0,
                batch: int | None = None) -> np.ndarray:
    """Layer-input rows x[b, t, :] for tokens first_token .. first_token+count-1.

    Drawn token by token (one sub-stream per (layer, token)) so that any window of the
    sequence can be regenerated on its own. With per_layer_inputs the rows are scaled to
    unit root-mean-square (weight 1, eps 1e-5) before rounding.
    """
    b = cfg.batch if batch is None else batch
    out = np.empty((b, count, cfg.hidden), dtype=np.float32)
    for t in range(count):
        g = substream(cfg.seed, "x", layer, first_token + t)
        rows = g.standard_normal(size=(cfg.batch, cfg.hidden), dtype=np.float32)[:b]
        if cfg.per_layer_inputs:
            ms = np.mean(rows.astype(np.float64) ** 2, axis=-1, keepdims=True)
            rows = (rows / np.sqrt(ms + 1e-5)).astype(np.float32)
        out[:, t, :] = rows
    return round_to_dtype(out, cfg.dtype)


def projection_weights(cfg: WorkloadConfig, layer: int = 0) -> np.ndarray:
    """W_kv[layer] of shape [2*H*dh, d]: key rows first, then value rows."""
    n = cfg.n_heads * cfg.head_dim
    if cfg.identity_projection:
        assert cfg.hidden == n
        eye = np.eye(n, dtype=np.float32)
        return np.concatenate([eye, eye], axis=0)
    return gaussian(cfg.seed, "w_kv", (2 * n, cfg.hidden), 0.02, cfg.dtype, idx=(layer,))


def query_weights(cfg: WorkloadConfig, layer: int = 0) -> np.ndarray:
    """W_q[layer] of shape [H*dh, d] (used by the harness to make queries)."""
    n = cfg.n_heads * cfg.head_dim
    return gaussian(cfg.seed, "w_q", (n, cfg.hidden), 0.02, cfg.dtype, idx=(layer,))


def rebuild_flags(cfg: WorkloadConfig, step: int, n_tokens: int, r_in: int,
                  batch: int | None = None) -> Tuple[np.ndarray, np.ndarray]:
    """Explicit-mode rebuild candidates for one step.

    Every token position < n_tokens is flagged independently with probability
    rebuild_p; the flagged positions are returned as a padded int32 list [B, r_in]
    (ascending, -1 padded) with their counts [B]. Tokens that are still resident are
    not filtered out here: the consumer intersects the list with its released set.
    """
    b = cfg.batch if batch is None else batch
    g = substream(cfg.seed, "rebuild_flags", step)
    u = g.random(size=(cfg.batch, max(n_tokens, 1)), dtype=np.float32)[:b, :n_tokens]
    lists = np.full((b, r_in), -1, dtype=np.int32)
    counts = np.zeros((b,), dtype=np.int32)
    for i in range(b):
        idx = np.nonzero(u[i] < cfg.rebuild_p)[0][:r_in]
        lists[i, : idx.size] = idx
        counts[i] = idx.size
    return lists, counts


def slot_weights(seed: int, n_layers: int, batch: int, n_heads: int, n_slots: int, nonzero: int,
                 empty_frac: float = 0.1) -> np.ndarray:
    """Per-slot weights with the shape of what a decode step emits: float32 [L, B, H, n_slots], at most `nonzero`
    positive entries per (layer, sequence, head) row, rows summing to one, empty slots zero everywhere, long-tailed
    values, and a per-sequence set of slots that every layer and head tends to favour."""
    out = np.zeros((n_layers, batch, n_heads, n_slots), np.float32)
    for b in range(batch):
        rng = substream(seed, "slot_weights", b)
        occupied = np.nonzero(rng.random(n_slots) >= empty_frac)[0]
        favour = rng.random(n_slots) ** 4                      # a few slots matter to every head
        for l in range(n_layers):
            for h in range(n_heads):
                k = min(nonzero, occupied.size)
                pick_score = favour[occupied] + 0.3 * rng.random(occupied.size)
                chosen = occupied[np.argsort(-pick_score, kind="stable")[:k]]
                vals = rng.exponential(1.0, k) ** 3
                out[l, b, h, chosen] = (vals / vals.sum()).astype(np.float32)
    return out
