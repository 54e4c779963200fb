"""CPU oracle for the ADORE decode path (adaptive token release with KV rebuild).

TEST INFRASTRUCTURE ONLY. This is a slow, plain restatement of what the paper defines,
kept for checking the CUDA library. It shares no code with that library and must never
sit on a product path. Floating point is float64 throughout; values are rounded to the
cache element type only where the method stores them (cache rows, scores).

Every function cites the passage of the paper it follows:

* Section 2.1, Eq. 1 and the unnumbered target equation after it: scaled dot-product
  attention over the full history / over m selected rows plus the current token.
* Section 2.2: top-K masking of attention weights, one retain/release decision per
  token for all layers, append-newest / release-lowest-sigma update, controller
  z_i = GRU(x_i, z_{i-1}), sigma_i = Sigmoid(MLP(p_i + z_i)) (Eq. 2 and the line after).
* Section 2.3: rebuild of the top-R released tokens and attention over m+R+1 rows.
* Section 2.4: row deletion written as multiplication by a slicing matrix S_j.
* Appendix B: controller layer sizes (GRU d->128, position FC 1->128, FC 128 + Tanh,
  FC -> 1 + Sigmoid).

Parity pins: every function below is pinned by tests/test_oracle_*.py (brute-force full
attention, rank counting, torch's GRU cell, closed forms, invariants). Nothing here is
"parity unpinned"; what cannot be pinned is the paper's printed quality/throughput
tables, which need its datasets and trained weights.

Readings where the paper is silent (each is listed with its reason in the design notes):
standard three-gate GRU with the reset gate applied to the hidden-side candidate term;
position feature u = i / pos_scale; the mask keeps the K largest logits with the lower
index winning ties; sqrt of the head dimension; newer token wins score ties; rebuilt
states live for one step; rotary embedding at the token's original position on adjacent
pairs (2j, 2j+1). A second reading of the position feature, u = (n - i) / pos_scale with every token
scored anew at every step (controller_rescore), is kept beside the first as an option.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Tuple

import numpy as np

EMPTY, RETAINED, REBUILT = 0, 1, 2


# --------------------------------------------------------------------------------------
# element types
# --------------------------------------------------------------------------------------
def round_bf16(a: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64/float32 values to bfloat16, returned as float32."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    # the float64 -> float32 step can double-round only when the float64 value sits within
    # 2^-29 relative of a bf16 tie, which the test data never does on purpose
    u = f.view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u & 0xFFFF0000).astype(np.uint32).view(np.float32).reshape(f.shape)


def round_store(a: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_bf16(a)
    if dtype == "f32":
        return np.asarray(a, dtype=np.float64).astype(np.float32)
    raise ValueError(dtype)


# --------------------------------------------------------------------------------------
# attention (Section 2.1; top-K mask Section 2.2 first bullet)
# --------------------------------------------------------------------------------------
def full_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Eq. 1 for one head: softmax(q K^T / sqrt(dh)) V over all n rows."""
    q = np.asarray(q, np.float64)
    K = np.asarray(K, np.float64)
    V = np.asarray(V, np.float64)
    logit = K @ q / np.sqrt(q.shape[-1])
    w = np.exp(logit - logit.max())
    w /= w.sum()
    return w @ V


def topk_keep(logits: np.ndarray, valid: np.ndarray, k: int) -> np.ndarray:
    """Mask of the k largest valid logits per row; on equal logits the lower index wins.

    logits, valid: [..., n]. If a row has at most k valid entries all of them are kept.
    """
    lg = np.where(valid, logits, -np.inf)
    order = np.argsort(-lg, axis=-1, kind="stable")         # equal keys keep index order
    rank = np.argsort(order, axis=-1, kind="stable")        # inverse permutation = rank of each entry
    return valid & (rank < k)


def sparse_attention(q: np.ndarray, Kc: np.ndarray, Vc: np.ndarray, occupied: np.ndarray,
                     k_new: np.ndarray, v_new: np.ndarray, topk: int, own_row: bool = True
                     ) -> Tuple[np.ndarray, np.ndarray]:
    """Target / rebuild attention for one sequence, all heads (Section 2.1, Section 2.3).

    q, k_new, v_new: [H, dh]; Kc, Vc: [H, C, dh]; occupied: [C] bool (same for all heads).
    Candidates are the occupied slots followed by the current token's own row (index C).
    Only the `topk` largest logits keep a weight. Returns out [H, dh] and weights
    [H, C+1] (float64; zero for empty or masked rows). own_row=False drops the row at index C from the
    candidates (a rebuilt token's query must not see the current token, which comes after it).
    """
    H, C, dh = Kc.shape
    q = np.asarray(q, np.float64)
    Kall = np.concatenate([np.asarray(Kc, np.float64), np.asarray(k_new, np.float64)[:, None, :]], 1)
    Vall = np.concatenate([np.asarray(Vc, np.float64), np.asarray(v_new, np.float64)[:, None, :]], 1)
    valid = np.concatenate([np.asarray(occupied, bool), [bool(own_row)]])[None, :].repeat(H, 0)
    logit = np.einsum("hd,hcd->hc", q, Kall) / np.sqrt(dh)
    keep = topk_keep(logit, valid, topk)
    lg = np.where(keep, logit, -np.inf)
    w = np.exp(lg - lg.max(axis=-1, keepdims=True))
    w = np.where(keep, w, 0.0)
    w /= w.sum(axis=-1, keepdims=True)
    # empty slots may hold stale (even non-finite) bytes: they must not reach the sum
    Vall = np.where(valid[:, :, None], Vall, 0.0)
    out = np.einsum("hc,hcd->hd", w, Vall)
    return out, w


# --------------------------------------------------------------------------------------
# controller (Section 2.2 Eq. 2, Appendix B)
# --------------------------------------------------------------------------------------
def _sigm(a: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-a))


def gru_step(x: np.ndarray, z_prev: np.ndarray, w: Dict[str, np.ndarray]) -> np.ndarray:
    """One step of the single-layer unidirectional GRU, z_i = GRU(x_i, z_{i-1}).

    x: [..., d], z_prev: [..., d']. Stacked gate order: reset, update, candidate.
    """
    h = z_prev.shape[-1]
    w_ih = np.asarray(w["gru_w_ih"], np.float64)
    w_hh = np.asarray(w["gru_w_hh"], np.float64)
    gi = np.asarray(x, np.float64) @ w_ih.T + np.asarray(w["gru_b_ih"], np.float64)
    gh = np.asarray(z_prev, np.float64) @ w_hh.T + np.asarray(w["gru_b_hh"], np.float64)
    r = _sigm(gi[..., 0:h] + gh[..., 0:h])
    g = _sigm(gi[..., h:2 * h] + gh[..., h:2 * h])
    c = np.tanh(gi[..., 2 * h:] + r * gh[..., 2 * h:])
    return (1.0 - g) * c + g * np.asarray(z_prev, np.float64)


def controller_score(z: np.ndarray, position: float, pos_scale: float,
                     w: Dict[str, np.ndarray]) -> np.ndarray:
    """Pre-sigmoid output of MLP(p_i + z_i) with p_i = FC(1->d') of u = position/pos_scale."""
    u = float(position) / float(pos_scale)
    p = np.asarray(w["pos_w"], np.float64) * u + np.asarray(w["pos_b"], np.float64)
    t = np.tanh((p + z) @ np.asarray(w["mlp_w1"], np.float64).T + np.asarray(w["mlp_b1"], np.float64))
    return t @ np.asarray(w["mlp_w2"], np.float64) + float(np.asarray(w["mlp_b2"]).reshape(-1)[0])


def controller_rescore(z_rows: np.ndarray, n: int, pos_scale: float, w: Dict[str, np.ndarray]) -> np.ndarray:
    """Scores of tokens 0..n as seen from the current token n. Section 1 and the caption of Figure 2 describe the
    controller's importance as one taken with respect to the token being decoded, over all earlier tokens, cached
    or released. Read that way, sigma_i = Sigmoid(MLP(p + z_i)) of Eq. 2 takes its position feature RELATIVE to
    the current token, u = (n - i) / pos_scale: a token's score moves as the sequence grows, while its GRU state
    z_i stays what it was when the token arrived.

    z_rows: [..., n+1, d'] states of tokens 0..n. Returns the pre-sigmoid scores [..., n+1] (float64).
    """
    z_rows = np.asarray(z_rows, np.float64)
    assert z_rows.shape[-2] == n + 1
    out = np.zeros(z_rows.shape[:-1], np.float64)
    for i in range(n + 1):
        out[..., i] = controller_score(z_rows[..., i, :], n - i, pos_scale, w)
    return out


def controller_param_count(d: int, h: int) -> int:
    """Number of parameters of the Appendix B controller."""
    return 3 * h * (d + h) + 2 * 3 * h + (h + h) + (h * h + h) + (h + 1)


# --------------------------------------------------------------------------------------
# value order and selection (Section 2.2 release rule, Section 2.3 top-R of released)
# --------------------------------------------------------------------------------------
def by_value_desc(tokens: np.ndarray, score32: np.ndarray) -> np.ndarray:
    """Tokens sorted most valuable first: higher score, then newer (larger position).

    Ranking on the pre-sigmoid score equals ranking on sigma (the sigmoid is monotone).
    """
    tokens = np.asarray(tokens, np.int64)
    s = np.asarray(score32, np.float32)[tokens]
    order = np.lexsort((-tokens, -s.astype(np.float64)))
    return tokens[order]


def slicing_matrix(m: int, j: int) -> np.ndarray:
    """S_j of Section 2.4: the m x m identity without its j-th row (0-based j)."""
    return np.delete(np.eye(m), j, axis=0)


# --------------------------------------------------------------------------------------
# rotary embedding and projection (Section 2.3: rebuilt K/V are recomputed states)
# --------------------------------------------------------------------------------------
def rope_rotate(v: np.ndarray, position: int, theta: float) -> np.ndarray:
    """Rotate adjacent pairs (2j, 2j+1) of the last axis by position * theta^(-2j/dh)."""
    v = np.asarray(v, np.float64)
    if theta == 0.0:
        return v.copy()
    dh = v.shape[-1]
    j = np.arange(dh // 2, dtype=np.float64)
    ang = float(position) * np.power(float(theta), -2.0 * j / dh)
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty_like(v)
    out[..., 0::2] = v[..., 0::2] * c - v[..., 1::2] * s
    out[..., 1::2] = v[..., 0::2] * s + v[..., 1::2] * c
    return out


def project_q(w_q: np.ndarray, x_row: np.ndarray, position: int, n_heads: int, head_dim: int,
              theta: float, dtype: str) -> np.ndarray:
    """Query rows [H, dh] of the current token (harness side: same rotation as the keys)."""
    y = np.asarray(w_q, np.float64) @ np.asarray(x_row, np.float64)
    return round_store(rope_rotate(y.reshape(n_heads, head_dim), position, theta), dtype)


# --------------------------------------------------------------------------------------
# labels for training the controller (Section 2.2 last paragraph, Appendix B, Appendix C)
# --------------------------------------------------------------------------------------
def attention_labels(weights: np.ndarray, topk: int):
    """Uniform token set of one decode step from its per-slot attention weights.

    weights: [L, B, H, S] (what the step emits; zero = masked or empty). For every (layer, head) the set of the
    topk // 2 slots with the largest positive weight is taken (equal weights: lower slot first; fewer if fewer are
    positive). count[b, s] is the number of these sets that contain slot s; the label is 1 for the `topk` slots of
    a sequence with the largest positive count (equal counts: lower slot first), 0 for all others.
    Also the two statistics of Appendix C (Figure 7): coverage[l, b], the share of layer l's set members that carry
    the label, and mass[l, b], the attention weight of the labelled slots at layer l averaged over heads.

    Returns sets [L, B, H, topk // 2] int32 (-1 padded, in descending weight order), count [B, S] int32,
    label [B, S] uint8, coverage [L, B] float64, mass [L, B] float64.
    """
    w = np.asarray(weights)
    L, B, H, S = w.shape
    half = topk // 2
    sets = np.full((L, B, H, half), -1, np.int32)
    count = np.zeros((B, S), np.int32)
    for l in range(L):
        for b in range(B):
            for h in range(H):
                row = w[l, b, h]
                order = sorted((s for s in range(S) if row[s] > 0), key=lambda s: (-float(row[s]), s))[:half]
                sets[l, b, h, : len(order)] = order
                for s in order:
                    count[b, s] += 1
    label = np.zeros((B, S), np.uint8)
    for b in range(B):
        order = sorted((s for s in range(S) if count[b, s] > 0), key=lambda s: (-int(count[b, s]), s))[:topk]
        label[b, order] = 1
    coverage = np.zeros((L, B), np.float64)
    mass = np.zeros((L, B), np.float64)
    for l in range(L):
        for b in range(B):
            members = sets[l, b][sets[l, b] >= 0]
            coverage[l, b] = float(label[b, members].sum()) / members.size if members.size else 0.0
            mass[l, b] = float(np.asarray(w[l, b], np.float64)[:, label[b] == 1].sum()) / H
    return sets, count, label, coverage, mass


# --------------------------------------------------------------------------------------
# the stateful path
# --------------------------------------------------------------------------------------
@dataclass
class OracleConfig:
    batch: int
    n_layers: int
    n_heads: int
    head_dim: int
    hidden: int
    capacity: int
    rebuild_max: int
    topk: int
    max_tokens: int
    ctrl_hidden: int = 128
    dtype: str = "bf16"
    rebuild_mode: str = "policy"
    rope_theta: float = 1.0e4
    pos_scale: float = 4096.0
    no_recurrence: bool = False    # Section 3.5.3 "w/o GRU": z_i = GRU(x_i, 0), no memory of earlier tokens
    score_from_attention: bool = False   # Section 3.1 baselines 6 and 7: a token's value is its cumulative attention
    relative_position: bool = False      # every token is re-scored at every step with its distance to the current token

    @property
    def retained_max(self) -> int:
        return self.capacity - self.rebuild_max


@dataclass
class StepInfo:
    admit_slot: np.ndarray            # [B]
    evicted_tok: np.ndarray           # [B], -1 if nothing was evicted
    rebuild_tok: List[np.ndarray]     # per sequence, most valuable first
    rebuild_slot: List[np.ndarray]


class AdoreOracle:
    """Fixed-capacity slot cache with controller-driven release and one-step rebuild.

    State per sequence (one map for all heads and layers, Section 2.2 second bullet):
    slot_tok[C] (token position or -1), slot_role[C], and per token: hidden row x_i,
    score_i (pre-sigmoid, stored in float32), sigma_i, tok_slot[i] (-1 = released).
    """

    def __init__(self, cfg: OracleConfig, ctrl: Dict[str, np.ndarray]):
        if not (0 <= cfg.rebuild_max < cfg.capacity):
            raise ValueError("need 0 <= rebuild_max < capacity")
        self.cfg = cfg
        self.ctrl = ctrl
        B, C, T = cfg.batch, cfg.capacity, cfg.max_tokens
        self.n = 0                                             # tokens seen per sequence
        self.x = np.zeros((B, T, cfg.hidden), np.float32)
        self.z = np.zeros((B, cfg.ctrl_hidden), np.float64)    # z_{-1} = 0
        if cfg.relative_position and cfg.score_from_attention:
            raise ValueError("relative positions belong to the controller's score")
        self.z_rows = np.zeros((B, T, cfg.ctrl_hidden), np.float64) if cfg.relative_position else None
        self.score = np.zeros((B, T), np.float32)
        self.sigma = np.zeros((B, T), np.float32)
        self.tok_slot = np.full((B, T), -1, np.int32)
        self.slot_tok = np.full((B, C), -1, np.int32)
        self.slot_role = np.zeros((B, C), np.uint8)
        self.attn_slot_tok = self.slot_tok.copy()              # map the caches currently follow
        self.Kc = np.zeros((cfg.n_layers, B, cfg.n_heads, C, cfg.head_dim), np.float32)
        self.Vc = np.zeros_like(self.Kc)
        self.w_kv: List[Optional[np.ndarray]] = [None] * cfg.n_layers
        self.info: Optional[StepInfo] = None
        self.kept: Optional[np.ndarray] = None                 # last attention's kept mask

    # -- set-up ------------------------------------------------------------------------
    def set_projection(self, layer: int, w_kv: np.ndarray) -> None:
        assert w_kv.shape == (2 * self.cfg.n_heads * self.cfg.head_dim, self.cfg.hidden)
        self.w_kv[layer] = np.asarray(w_kv, np.float64)

    # -- controller --------------------------------------------------------------------
    def _score_new_token(self, x_new: np.ndarray, rescore: bool = True) -> None:
        """z_n, score_n, sigma_n for the token at position self.n of every sequence. With relative positions
        the states of all tokens are kept and (unless `rescore` is off) tokens 0..n are all scored anew."""
        c, n = self.cfg, self.n
        self.x[:, n, :] = x_new
        if c.score_from_attention:          # no controller: the token starts at zero and earns weight when attended
            self.score[:, n] = 0.0
            self.sigma[:, n] = 0.0
            return
        z_prev = np.zeros_like(self.z) if c.no_recurrence else self.z
        self.z = gru_step(x_new, z_prev, self.ctrl)
        if c.relative_position:
            self.z_rows[:, n, :] = self.z
            if rescore:
                s = controller_rescore(self.z_rows[:, : n + 1, :], n, c.pos_scale, self.ctrl)
                self.score[:, : n + 1] = s.astype(np.float32)
                self.sigma[:, : n + 1] = _sigm(s).astype(np.float32)
            return
        s = controller_score(self.z, n, c.pos_scale, self.ctrl)
        self.score[:, n] = s.astype(np.float32)
        self.sigma[:, n] = _sigm(s).astype(np.float32)

    # -- selection ---------------------------------------------------------------------
    def _free(self, b: int, slot: int) -> None:
        self.tok_slot[b, self.slot_tok[b, slot]] = -1
        self.slot_tok[b, slot] = -1
        self.slot_role[b, slot] = EMPTY

    def _place(self, b: int, tok: int, slot: int, role: int) -> None:
        assert self.slot_role[b, slot] == EMPTY
        self.slot_tok[b, slot] = tok
        self.slot_role[b, slot] = role
        self.tok_slot[b, tok] = slot

    def _rebuild_list(self, b: int, n_seen: int, explicit: Optional[np.ndarray]) -> np.ndarray:
        """Tokens to rebuild, most valuable first (Section 2.3, first sentence)."""
        c = self.cfg
        released = np.nonzero(self.tok_slot[b, :n_seen] < 0)[0]
        if c.rebuild_mode == "policy":
            cand = released
        else:
            e = np.asarray([] if explicit is None else explicit, np.int64)
            e = e[(e >= 0) & (e < n_seen)]
            cand = np.intersect1d(e, released)                 # drops residents and duplicates
        return by_value_desc(cand, self.score[b])[: c.rebuild_max]

    def _select_one(self, b: int, explicit: Optional[np.ndarray]) -> Tuple[int, int, np.ndarray, np.ndarray]:
        """Release / admit / choose the rebuild list for sequence b; the new token is self.n."""
        c, n = self.cfg, self.n
        # 1. rebuilt states live for one step only: top-R is re-derived every step
        for s in np.nonzero(self.slot_role[b] == REBUILT)[0]:
            self._free(b, int(s))
        # 2. constant cache size: full => release the least valuable retained token
        evicted = -1
        ret = np.nonzero(self.slot_role[b] == RETAINED)[0]
        if ret.size == c.retained_max:
            evicted = int(by_value_desc(self.slot_tok[b, ret], self.score[b])[-1])
            self._free(b, int(self.tok_slot[b, evicted]))
        # 3. append the most recent token: lowest-index empty slot
        admit = int(np.nonzero(self.slot_role[b] == EMPTY)[0][0])
        self._place(b, n, admit, RETAINED)
        # 4./5. rebuild list among released tokens, most valuable first, into empty slots
        lst = self._rebuild_list(b, n, explicit)
        empty = np.nonzero(self.slot_role[b] == EMPTY)[0][: lst.size]
        for tok, s in zip(lst, empty):
            self._place(b, int(tok), int(s), REBUILT)
        return admit, evicted, lst.astype(np.int32), empty.astype(np.int32)

    def check_invariants(self) -> None:
        c = self.cfg
        for b in range(c.batch):
            role = self.slot_role[b]
            assert (role == RETAINED).sum() <= c.retained_max
            assert (role == REBUILT).sum() <= c.rebuild_max
            assert (role != EMPTY).sum() <= c.capacity
            occ = np.nonzero(self.slot_tok[b] >= 0)[0]
            assert np.array_equal(occ, np.nonzero(role != EMPTY)[0])
            assert np.array_equal(self.tok_slot[b, self.slot_tok[b, occ]], occ)
            res = np.nonzero(self.tok_slot[b, : self.n] >= 0)[0]
            assert res.size == occ.size
            assert np.array_equal(self.slot_tok[b, self.tok_slot[b, res]], res)

    # -- adopting a state from outside ---------------------------------------------------
    def import_state(self, n: int, slot_tok: np.ndarray, slot_role: np.ndarray, score: np.ndarray, sigma: np.ndarray,
                     z: np.ndarray, x_rows: np.ndarray, rebuild_tok: List[np.ndarray], rebuild_slot: List[np.ndarray],
                     admit_slot: Optional[np.ndarray] = None, evicted_tok: Optional[np.ndarray] = None,
                     z_rows: Optional[np.ndarray] = None, x_tables: Optional[List[np.ndarray]] = None) -> None:
        """Continue from the small state of Sections 2.2-2.3 as somebody else left it after `n` tokens: which token
        holds which slot in which role, every token's score and sigma, the GRU state z_{n-1}, the tokens' stored
        embeddings and the last step's rebuild list. The token-to-slot table is the inverse of the slot map. The cache
        rows are not taken over: by Section 2.3 a resident token's K/V state IS its recomputed state, so every layer
        with a projection is filled by definition, from x_rows or, for stacks whose layers have their own input rows,
        from x_tables[layer].

        slot_tok, slot_role: [B, C]; score, sigma: [B, >= n] float32; z: [B, d']; x_rows: [B, >= n, d];
        rebuild_tok / rebuild_slot: per sequence, most valuable first. z_rows [B, >= n, d'] only with relative positions.
        """
        c = self.cfg
        B, C = c.batch, c.capacity
        slot_tok = np.asarray(slot_tok, np.int32)
        slot_role = np.asarray(slot_role, np.uint8)
        if slot_tok.shape != (B, C) or slot_role.shape != (B, C) or not (0 <= n <= c.max_tokens):
            raise ValueError("state of another shape")
        self.n = int(n)
        self.slot_tok = slot_tok.copy()
        self.slot_role = slot_role.copy()
        self.tok_slot = np.full((B, c.max_tokens), -1, np.int32)
        for b in range(B):
            for s in range(C):
                t = int(slot_tok[b, s])
                if t >= 0:
                    if not (t < n) or self.tok_slot[b, t] != -1 or slot_role[b, s] == EMPTY:
                        raise ValueError("slot map is not a one-to-one map of tokens < n")
                    self.tok_slot[b, t] = s
                elif slot_role[b, s] != EMPTY:
                    raise ValueError("an unoccupied slot carries a role")
        self.score = np.zeros((B, c.max_tokens), np.float32)
        self.sigma = np.zeros((B, c.max_tokens), np.float32)
        self.score[:, :n] = np.asarray(score, np.float32)[:, :n]
        self.sigma[:, :n] = np.asarray(sigma, np.float32)[:, :n]
        self.z = np.asarray(z, np.float64).reshape(B, c.ctrl_hidden).copy()
        self.x = np.zeros((B, c.max_tokens, c.hidden), np.float32)
        self.x[:, :n] = np.asarray(x_rows, np.float32)[:, :n]
        if c.relative_position:
            self.z_rows = np.zeros((B, c.max_tokens, c.ctrl_hidden), np.float64)
            self.z_rows[:, :n] = np.asarray(z_rows, np.float64)[:, :n]
        lists = [np.asarray(t, np.int32).copy() for t in rebuild_tok]
        slots = [np.asarray(s, np.int32).copy() for s in rebuild_slot]
        for b in range(B):                                    # the list must be what the map shows as rebuilt
            where = np.nonzero(self.slot_role[b] == REBUILT)[0]
            if not (np.array_equal(np.sort(slots[b]), where) and np.array_equal(self.slot_tok[b, slots[b]], lists[b])):
                raise ValueError("rebuild list and slot map disagree")
        self.info = StepInfo(np.full(B, -1, np.int32) if admit_slot is None else np.asarray(admit_slot, np.int32).copy(),
                             np.full(B, -1, np.int32) if evicted_tok is None else np.asarray(evicted_tok, np.int32).copy(),
                             lists, slots)
        self.attn_slot_tok = self.slot_tok.copy()
        self.kept = None
        self.check_invariants()
        for layer in range(c.n_layers):
            if self.w_kv[layer] is not None:
                self.fill_layer(layer, None if (x_tables is None or layer == 0) else x_tables[layer])

    # -- cache rows --------------------------------------------------------------------
    def _store_projections(self, layer: int, rows: List[Tuple[int, int, int]], src: np.ndarray) -> None:
        """Y = X_L W_kv^T for the listed (b, tok, slot) rows, rotated, rounded and stored."""
        if not rows:
            return
        c = self.cfg
        n = c.n_heads * c.head_dim
        X = np.stack([np.asarray(src[b, tok], np.float64) for b, tok, _ in rows])
        Y = X @ self.w_kv[layer].T
        for (b, tok, slot), y in zip(rows, Y):
            k = rope_rotate(y[:n].reshape(c.n_heads, c.head_dim), tok, c.rope_theta)
            self.Kc[layer, b, :, slot, :] = round_store(k, c.dtype)
            self.Vc[layer, b, :, slot, :] = round_store(y[n:].reshape(c.n_heads, c.head_dim), c.dtype)

    # -- prompt ------------------------------------------------------------------------
    def append_tokens(self, x: np.ndarray, explicit: Optional[List[np.ndarray]] = None) -> None:
        """Bulk load of T prompt tokens into an empty cache.

        Scores all tokens, then retains the newest token plus the min(m-1, T-1) most
        valuable earlier ones, laid out in ascending position from slot 0; this is the
        set that token-by-token release would reach, because a token's score does not
        change after it arrives. The rebuild list follows as in a decode step (empty in
        explicit mode). Every layer with a projection is filled from these rows.

        With relative positions the prompt is given at once, so its tokens are scored
        once, as seen from the last prompt token, and the same selection is made on those
        scores (token-by-token release would differ here: scores move with the position).
        """
        c = self.cfg
        assert self.n == 0, "bulk load needs an empty cache"
        B, T, _ = x.shape
        for t in range(T):
            self._score_new_token(x[:, t, :], rescore=(t == T - 1))
            self.n += 1
        last = T - 1
        lists, slots = [], []
        for b in range(B):
            keep = by_value_desc(np.arange(last), self.score[b])[: min(c.retained_max - 1, last)]
            for s, tok in enumerate(np.sort(np.concatenate([keep, [last]]))):
                self._place(b, int(tok), s, RETAINED)
            lst = self._rebuild_list(b, T, None) if c.rebuild_mode == "policy" else np.zeros(0, np.int64)
            empty = np.nonzero(self.slot_role[b] == EMPTY)[0][: lst.size]
            for tok, s in zip(lst, empty):
                self._place(b, int(tok), int(s), REBUILT)
            lists.append(lst.astype(np.int32))
            slots.append(empty.astype(np.int32))
        self.info = StepInfo(np.full(B, -1, np.int32), np.full(B, -1, np.int32), lists, slots)
        for layer in range(c.n_layers):
            if self.w_kv[layer] is not None:
                self.fill_layer(layer, None)
        self.attn_slot_tok = self.slot_tok.copy()

    def fill_layer(self, layer: int, x_table: Optional[np.ndarray]) -> None:
        """Project every resident token of `layer` from x_table[b, tok] (default: stored rows)."""
        src = self.x if x_table is None else x_table
        rows = [(b, int(self.slot_tok[b, s]), int(s)) for b in range(self.cfg.batch)
                for s in np.nonzero(self.slot_tok[b] >= 0)[0]]
        self._store_projections(layer, rows, src)

    # -- one decode step for one layer ---------------------------------------------------
    def decode_step(self, layer: int, q: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
                    x_new: Optional[np.ndarray] = None,
                    explicit: Optional[List[np.ndarray]] = None) -> Tuple[np.ndarray, np.ndarray]:
        """Attention for `layer`, then (layer 0) controller + selection, then admission.

        q, k_new, v_new: [B, H, dh] (k_new already rotated to position n by the caller).
        Returns out [B, H, dh] float64 and weights [B, H, C+1] float64.
        """
        c = self.cfg
        B, H, C, dh = c.batch, c.n_heads, c.capacity, c.head_dim
        if layer == 0:
            if self.n >= c.max_tokens:
                raise IndexError("token table full")
            self.attn_slot_tok = self.slot_tok.copy()
        out = np.zeros((B, H, dh), np.float64)
        wts = np.zeros((B, H, C + 1), np.float64)
        for b in range(B):
            out[b], wts[b] = sparse_attention(q[b], self.Kc[layer, b], self.Vc[layer, b],
                                              self.attn_slot_tok[b] >= 0, k_new[b], v_new[b], c.topk)
        if layer == 0:
            self._score_new_token(x_new)
            admit = np.zeros(B, np.int32)
            evict = np.zeros(B, np.int32)
            lists, slots = [], []
            for b in range(B):
                a, e, lst, sl = self._select_one(b, None if explicit is None else explicit[b])
                admit[b], evict[b] = a, e
                lists.append(lst)
                slots.append(sl)
            self.info = StepInfo(admit, evict, lists, slots)
            self.n += 1
        for b in range(B):
            s = int(self.info.admit_slot[b])
            self.Kc[layer, b, :, s, :] = round_store(k_new[b], c.dtype)
            self.Vc[layer, b, :, s, :] = round_store(v_new[b], c.dtype)
        if c.score_from_attention:
            self._add_attention(wts, self.attn_slot_tok, self.n - 1)
        return out, wts

    def _add_attention(self, wts: np.ndarray, slot_tok: np.ndarray, n_cur: int) -> None:
        """Cumulative attention as the tokens' value: every attended token gains the weight its row received, summed
        over the heads (float32, heads in ascending order, as the ranking is done on float32); the selection of the
        NEXT step is the first to see it."""
        B, H, C1 = wts.shape
        w32 = wts.astype(np.float32)
        for b in range(B):
            for s in range(C1):
                tok = n_cur if s == C1 - 1 else int(slot_tok[b, s])
                if tok < 0:
                    continue
                acc = np.float32(0.0)
                for h in range(H):
                    acc = np.float32(acc + w32[b, h, s])
                self.score[b, tok] = np.float32(self.score[b, tok] + acc)

    # -- the step in the order Section 2.3 prints it: select, rebuild, then attend with R+1 query rows ----
    def step_begin(self, x_new: np.ndarray, explicit: Optional[List[np.ndarray]] = None) -> None:
        """Controller and selection for token n before any attention of the step: afterwards the map holds the
        retained tokens, the slots of this step's rebuild list and the slot token n will be written to."""
        c = self.cfg
        if self.n >= c.max_tokens:
            raise IndexError("token table full")
        self._score_new_token(x_new)
        admit = np.zeros(c.batch, np.int32)
        evict = np.zeros(c.batch, np.int32)
        lists, slots = [], []
        for b in range(c.batch):
            a, e, lst, sl = self._select_one(b, None if explicit is None else explicit[b])
            admit[b], evict[b] = a, e
            lists.append(lst)
            slots.append(sl)
        self.info = StepInfo(admit, evict, lists, slots)
        self.n += 1

    def attend_rows(self, layer: int, q_rows: np.ndarray, k_new: np.ndarray, v_new: np.ndarray
                    ) -> Tuple[np.ndarray, np.ndarray]:
        """The attention of Section 2.3 for `layer`, after step_begin() and rebuild(layer): R_max + 1 query rows per
        sequence, row i < R_max for the i-th token of the rebuild list (rows past the list's end are padding and
        return zeros), the last row for the current token. Keys and values are the cached rows, the rebuilt rows
        (already in their slots) and the current token's own row; a query sees only tokens at positions up to its
        own, and keeps the `topk` largest logits. Then the current token's row is stored in its slot.

        q_rows: [B, H, R_max+1, dh]; returns out [B, H, R_max+1, dh] and weights [B, H, R_max+1, C+1].
        """
        c = self.cfg
        assert not c.score_from_attention, "the cumulative-attention score source is defined for the attend-first step"
        B, H, C, dh, R1 = c.batch, c.n_heads, c.capacity, c.head_dim, c.rebuild_max + 1
        n = self.n - 1                                        # position of the current token
        out = np.zeros((B, H, R1, dh), np.float64)
        wts = np.zeros((B, H, R1, C + 1), np.float64)
        for b in range(B):
            lst = self.info.rebuild_tok[b]
            for i in range(R1):
                tok = n if i == R1 - 1 else (int(lst[i]) if i < len(lst) else -1)
                if tok < 0:
                    continue
                st = self.slot_tok[b]
                seen = (st >= 0) & (st <= tok) & (st != n)     # token n's slot is reserved, its row not written yet
                out[b, :, i], wts[b, :, i] = sparse_attention(q_rows[b, :, i], self.Kc[layer, b], self.Vc[layer, b], seen,
                                                              k_new[b], v_new[b], c.topk, own_row=(tok == n))
        for b in range(B):
            s_ = int(self.info.admit_slot[b])
            self.Kc[layer, b, :, s_, :] = round_store(k_new[b], c.dtype)
            self.Vc[layer, b, :, s_, :] = round_store(v_new[b], c.dtype)
        return out, wts

    def rebuild(self, layer: int, x_table: Optional[np.ndarray] = None) -> int:
        """Recompute K/V of this step's rebuild list for `layer` and store them in their slots."""
        src = self.x if x_table is None else x_table
        rows = [(b, int(tok), int(slot)) for b in range(self.cfg.batch)
                for tok, slot in zip(self.info.rebuild_tok[b], self.info.rebuild_slot[b])]
        self._store_projections(layer, rows, src)
        return len(rows)
