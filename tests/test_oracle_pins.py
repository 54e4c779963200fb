"""Pins of the CPU oracle against things other than itself.

Each test names the passage it checks. The checks are brute force on tiny inputs, library
routines the definition reduces to, closed forms and invariants; the last test plants
plausible mistakes in the oracle and verifies that a pin notices each of them.
"""
import math

import numpy as np
import pytest
import torch

import workloads as wl
from oracle import adore_oracle as ao
from oracle.harness import Workload, make_oracle, explicit_as_lists

TINY = wl.WorkloadConfig(name="tiny", dtype="f32", n_layers=1, batch=2, n_heads=2, head_dim=8,
                         hidden=16, capacity=8, topk=4, rebuild_max=2, prompt=0, steps=24,
                         rope_theta=1.0e4, rebuild_mode="policy", rebuild_p=0.0, seed=11,
                         ctrl_hidden=8, pos_scale=64.0)


# ----------------------------------------------------------------------------- attention
def brute_attention(q, K, V):
    """Eq. 1 with explicit loops (Section 2.1)."""
    n, dh = len(K), len(q)
    logit = [sum(float(q[e]) * float(K[i][e]) for e in range(dh)) / math.sqrt(dh) for i in range(n)]
    mx = max(logit)
    ex = [math.exp(l - mx) for l in logit]
    tot = sum(ex)
    return np.array([sum(ex[i] / tot * float(V[i][e]) for i in range(n)) for e in range(dh)])


def test_full_attention_matches_loops_and_torch_sdpa():
    g = np.random.default_rng(0)
    q, K, V = g.standard_normal(16), g.standard_normal((9, 16)), g.standard_normal((9, 16))
    a = ao.full_attention(q, K, V)
    assert np.allclose(a, brute_attention(q, K, V), rtol=0, atol=1e-13)
    t = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q)[None, None], torch.tensor(K)[None], torch.tensor(V)[None])
    assert np.allclose(a, t[0, 0].numpy(), rtol=0, atol=1e-13)


def test_topk_keep_equals_rank_counting():
    """Ideal selection keeps the largest products (Section 2.1, last paragraph)."""
    g = np.random.default_rng(1)
    for trial in range(200):
        n = int(g.integers(1, 14))
        k = int(g.integers(1, 16))
        lg = g.integers(-3, 4, size=n).astype(np.float64)      # many exact ties
        valid = g.random(n) < 0.8
        keep = ao.topk_keep(lg[None], valid[None], k)[0]
        for i in range(n):
            beats = sum(1 for j in range(n) if valid[j] and (lg[j] > lg[i] or (lg[j] == lg[i] and j < i)))
            assert keep[i] == (bool(valid[i]) and beats < k)


def test_zero_query_gives_mean_of_lowest_index_rows():
    """Closed form: q = 0 makes all logits tie, so the K lowest-index candidates share weight 1/K."""
    g = np.random.default_rng(2)
    H, C, dh, K = 2, 6, 4, 3
    Kc, Vc = g.standard_normal((H, C, dh)), g.standard_normal((H, C, dh))
    occ = np.array([0, 1, 1, 0, 1, 1], bool)
    out, w = ao.sparse_attention(np.zeros((H, dh)), Kc, Vc, occ, g.standard_normal((H, dh)),
                                 g.standard_normal((H, dh)), K)
    kept = [1, 2, 4]
    assert np.allclose(out, Vc[:, kept].mean(axis=1), atol=1e-15)
    assert np.allclose(w[:, kept], 1 / 3) and np.count_nonzero(w) == H * K


def test_weights_are_a_distribution_with_min_k_candidates_nonzero():
    g = np.random.default_rng(3)
    H, C, dh = 3, 10, 8
    for K in (1, 4, 11, 50):
        occ = g.random(C) < 0.7
        out, w = ao.sparse_attention(g.standard_normal((H, dh)), g.standard_normal((H, C, dh)),
                                     g.standard_normal((H, C, dh)), occ, g.standard_normal((H, dh)),
                                     g.standard_normal((H, dh)), K)
        assert (w >= 0).all() and np.allclose(w.sum(-1), 1.0, atol=1e-14)
        assert ((w > 0).sum(-1) == min(K, occ.sum() + 1)).all()
        assert (w[:, :-1][:, ~occ] == 0).all()


def test_empty_cache_returns_the_new_value_row():
    H, C, dh = 2, 4, 4
    v = np.arange(8.0).reshape(H, dh)
    out, w = ao.sparse_attention(np.ones((H, dh)), np.full((H, C, dh), np.nan), np.full((H, C, dh), np.nan),
                                 np.zeros(C, bool), np.ones((H, dh)), v, 2)
    assert np.array_equal(out, v) and np.array_equal(w[:, -1], np.ones(H)) and w[:, :-1].sum() == 0


def test_topk_over_cache_equals_topk_over_history_when_topk_rows_are_cached():
    """Section 2.2, first bullet: masking to top-K is unaffected by what else is dropped."""
    g = np.random.default_rng(4)
    H, n, dh, K = 2, 40, 8, 5
    q = g.standard_normal((H, dh))
    Kh = 0.05 * g.standard_normal((H, n, dh))
    Vh = g.standard_normal((H, n, dh))
    planted = np.sort(g.choice(n, K - 1, replace=False))       # K-1 large rows + the token itself
    Kh[:, planted] = 3.0 * q[:, None, :] + 0.05 * g.standard_normal((H, K - 1, dh))
    k_new = 3.0 * q
    v_new = g.standard_normal((H, dh))
    full, _ = ao.sparse_attention(q, Kh, Vh, np.ones(n, bool), k_new, v_new, K)
    others = np.setdiff1d(np.arange(n), planted)[:6]
    cached = np.sort(np.concatenate([planted, others]))
    part, _ = ao.sparse_attention(q, Kh[:, cached], Vh[:, cached], np.ones(cached.size, bool), k_new, v_new, K)
    assert np.allclose(full, part, atol=1e-14)


# ---------------------------------------------------------------------------- controller
def _ctrl(d, h, seed=5, std=0.3):
    g = np.random.default_rng(seed)
    shapes = dict(gru_w_ih=(3 * h, d), gru_w_hh=(3 * h, h), gru_b_ih=(3 * h,), gru_b_hh=(3 * h,),
                  pos_w=(h,), pos_b=(h,), mlp_w1=(h, h), mlp_b1=(h,), mlp_w2=(h,), mlp_b2=(1,))
    return {k: (std * g.standard_normal(s)).astype(np.float32) for k, s in shapes.items()}


def test_gru_step_equals_torch_gru_cell():
    """Section 2.2 Eq. 2: single-layer GRU; torch's cell uses the same three-gate form."""
    d, h = 12, 5
    w = _ctrl(d, h)
    cell = torch.nn.GRUCell(d, h, dtype=torch.float64)
    with torch.no_grad():
        cell.weight_ih.copy_(torch.tensor(w["gru_w_ih"], dtype=torch.float64))
        cell.weight_hh.copy_(torch.tensor(w["gru_w_hh"], dtype=torch.float64))
        cell.bias_ih.copy_(torch.tensor(w["gru_b_ih"], dtype=torch.float64))
        cell.bias_hh.copy_(torch.tensor(w["gru_b_hh"], dtype=torch.float64))
    g = np.random.default_rng(6)
    z = np.zeros((3, h))
    zt = torch.zeros(3, h, dtype=torch.float64)
    for _ in range(7):
        x = g.standard_normal((3, d))
        z = ao.gru_step(x, z, w)
        with torch.no_grad():
            zt = cell(torch.tensor(x), zt)
        assert np.allclose(z, zt.numpy(), rtol=0, atol=1e-14)


def test_gru_closed_form_without_recurrence_and_fixed_point():
    d, h = 6, 4
    w = _ctrl(d, h)
    w0 = dict(w, gru_w_hh=np.zeros((3 * h, h), np.float32), gru_b_hh=np.zeros(3 * h, np.float32),
              gru_b_ih=np.zeros(3 * h, np.float32))
    x = np.random.default_rng(7).standard_normal(d)
    W = w0["gru_w_ih"].astype(np.float64)
    upd = 1 / (1 + np.exp(-(W[h:2 * h] @ x)))
    assert np.allclose(ao.gru_step(x, np.zeros(h), w0), (1 - upd) * np.tanh(W[2 * h:] @ x), atol=1e-15)
    z = np.zeros(h)
    for _ in range(400):                       # constant input: the state settles on a fixed point
        z = ao.gru_step(x, z, w)
    assert np.allclose(ao.gru_step(x, z, w), z, atol=1e-12)


def test_controller_score_equals_torch_modules_and_parameter_count():
    """Appendix B: position FC(1->d'), interaction FC(d'->d') + Tanh, output FC(d'->1)."""
    d, h = 10, 6
    w = _ctrl(d, h)
    pos, fc1, fc2 = torch.nn.Linear(1, h), torch.nn.Linear(h, h), torch.nn.Linear(h, 1)
    for m in (pos, fc1, fc2):
        m.double()
    with torch.no_grad():
        pos.weight.copy_(torch.tensor(w["pos_w"], dtype=torch.float64)[:, None])
        pos.bias.copy_(torch.tensor(w["pos_b"], dtype=torch.float64))
        fc1.weight.copy_(torch.tensor(w["mlp_w1"], dtype=torch.float64))
        fc1.bias.copy_(torch.tensor(w["mlp_b1"], dtype=torch.float64))
        fc2.weight.copy_(torch.tensor(w["mlp_w2"], dtype=torch.float64)[None, :])
        fc2.bias.copy_(torch.tensor(w["mlp_b2"], dtype=torch.float64))
        z = torch.tensor(np.random.default_rng(8).standard_normal((4, h)))
        ref = fc2(torch.tanh(fc1(pos(torch.tensor([[37 / 64.0]], dtype=torch.float64)) + z)))[:, 0]
    assert np.allclose(ao.controller_score(z.numpy(), 37, 64.0, w), ref.numpy(), atol=1e-14)
    gru = torch.nn.GRU(4096, 128)
    n = sum(p.numel() for m in (gru, torch.nn.Linear(1, 128), torch.nn.Linear(128, 128), torch.nn.Linear(128, 1))
            for p in m.parameters())
    assert ao.controller_param_count(4096, 128) == n


# ------------------------------------------------------------------- rounding, RoPE, Eq.S
def test_round_bf16_equals_torch():
    a = np.random.default_rng(9).standard_normal(4096).astype(np.float32) * 37.0
    a[:4] = [0.0, -0.0, 1.00390625, 1.01171875]               # exact ties: round to even
    t = torch.tensor(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ao.round_bf16(a), t)


def test_rope_is_complex_rotation_and_depends_on_relative_position_only():
    g = np.random.default_rng(10)
    dh, theta = 16, 1.0e4
    v = g.standard_normal(dh)
    z = (v[0::2] + 1j * v[1::2]) * np.exp(1j * 13 * theta ** (-2.0 * np.arange(dh // 2) / dh))
    r = ao.rope_rotate(v, 13, theta)
    assert np.allclose(r[0::2], z.real, atol=1e-14) and np.allclose(r[1::2], z.imag, atol=1e-14)
    q, k = g.standard_normal(dh), g.standard_normal(dh)
    a = ao.rope_rotate(q, 100, theta) @ ao.rope_rotate(k, 93, theta)
    b = ao.rope_rotate(q, 20, theta) @ ao.rope_rotate(k, 13, theta)
    assert abs(a - b) < 1e-12
    assert np.array_equal(ao.rope_rotate(v, 5, 0.0), v)


def test_slicing_matrix_deletes_a_row():
    """Section 2.4: S_j K equals K without row j, which is what freeing a slot does."""
    K = np.random.default_rng(11).standard_normal((7, 5))
    for j in range(7):
        assert np.array_equal(ao.slicing_matrix(7, j) @ K, np.delete(K, j, axis=0))


# ---------------------------------------------------------------------------- whole path
def run_free(cfg, steps=None, batch=None, check=True):
    w = Workload(cfg, batch)
    orc = make_oracle(w)
    if cfg.prompt:
        orc.append_tokens(w.prompt())
        if check:
            orc.check_invariants()
    hist = []
    for s in range(cfg.steps if steps is None else steps):
        n = orc.n
        x = w.x_new(n)
        q, k, v = w.qkv(n, 0, x)
        lists, counts = w.explicit(s, n)
        out, wts = orc.decode_step(0, q, k, v, x, explicit_as_lists(lists, counts))
        orc.rebuild(0)
        if check:
            orc.check_invariants()
        hist.append((q, out, wts))
    return w, orc, hist


def history_kv(w, orc, upto):
    """From-scratch K/V of tokens 0..upto-1, explicit loops over the projection and rotation."""
    c = w.cfg
    n_out = c.n_heads * c.head_dim
    K = np.zeros((w.batch, c.n_heads, upto, c.head_dim))
    V = np.zeros_like(K)
    W = w.w_kv[0].astype(np.float64)
    for b in range(w.batch):
        for t in range(upto):
            y = W @ orc.x[b, t].astype(np.float64)
            for h in range(c.n_heads):
                for j in range(c.head_dim // 2):
                    ang = t * c.rope_theta ** (-2.0 * j / c.head_dim) if c.rope_theta else 0.0
                    a, bb = y[h * c.head_dim + 2 * j], y[h * c.head_dim + 2 * j + 1]
                    K[b, h, t, 2 * j] = a * math.cos(ang) - bb * math.sin(ang)
                    K[b, h, t, 2 * j + 1] = a * math.sin(ang) + bb * math.cos(ang)
                V[b, h, t] = y[n_out + h * c.head_dim: n_out + (h + 1) * c.head_dim]
    return K.astype(np.float32).astype(np.float64), V.astype(np.float32).astype(np.float64)


@pytest.mark.parametrize("rebuild_max,prompt", [(0, 0), (0, 5), (20, 0), (27, 6)])
def test_path_equals_full_attention_when_every_token_is_resident(rebuild_max, prompt):
    """Sections 2.1 and 2.3: with room for the whole history (directly, or through the rebuild
    path with a small retained budget) the step must reproduce Eq. 1 over all tokens."""
    cfg = TINY.scaled(capacity=32, topk=64, rebuild_max=rebuild_max, prompt=prompt, steps=30 - prompt)
    w, orc, hist = run_free(cfg)
    K, V = history_kv(w, orc, orc.n)
    for s, (q, out, _) in enumerate(hist):
        n = prompt + s
        for b in range(w.batch):
            for h in range(cfg.n_heads):
                ref = brute_attention(q[b, h], K[b, h, : n + 1], V[b, h, : n + 1])
                assert np.allclose(out[b, h], ref, rtol=0, atol=1e-12)


def run_rebuild_first(cfg, steps=None):
    """The step in the order Section 2.3 prints it: select, rebuild, attend with R_max + 1 query rows."""
    w = Workload(cfg)
    orc = make_oracle(w)
    if cfg.prompt:
        orc.append_tokens(w.prompt())
    hist = []
    for s in range(cfg.steps if steps is None else steps):
        n = orc.n
        x = w.x_new(n)
        _, k, v = w.qkv(n, 0, x)
        lists, counts = w.explicit(s, n)
        orc.step_begin(x, explicit_as_lists(lists, counts))
        orc.rebuild(0)
        q_rows = w.q_rows(n, 0, orc.x, orc.info.rebuild_tok)
        out, wts = orc.attend_rows(0, q_rows, k, v)
        orc.check_invariants()
        hist.append((n, [list(map(int, l)) for l in orc.info.rebuild_tok], q_rows, out, wts))
    return w, orc, hist


@pytest.mark.parametrize("rebuild_max,prompt", [(20, 0), (27, 6)])
def test_rebuilt_query_rows_equal_causal_full_attention_when_every_token_is_resident(rebuild_max, prompt):
    """Section 2.3: with every token either retained or rebuilt, query row i must be Eq. 1 for its own token over the
    tokens up to its own position, and the last row Eq. 1 for the current token; rows past the list are zero."""
    cfg = TINY.scaled(capacity=32, topk=64, rebuild_max=rebuild_max, prompt=prompt, steps=30 - prompt)
    w, orc, hist = run_rebuild_first(cfg)
    K, V = history_kv(w, orc, orc.n)
    rows_checked = 0
    for n, lists, q_rows, out, _ in hist:
        for b in range(w.batch):
            toks = lists[b] + [-1] * (rebuild_max - len(lists[b])) + [n]
            for i, tok in enumerate(toks):
                for h in range(cfg.n_heads):
                    if tok < 0:
                        assert not out[b, h, i].any()
                        continue
                    ref = brute_attention(q_rows[b, h, i].astype(np.float64), K[b, h, : tok + 1], V[b, h, : tok + 1])
                    assert np.allclose(out[b, h, i], ref, rtol=0, atol=1e-12)
                    rows_checked += 1
    assert rows_checked > 200


def test_rebuilt_query_rows_do_not_see_later_tokens():
    """A row's output must not move when the cache row of a LATER token changes, and must move when an earlier one does."""
    cfg = TINY.scaled(capacity=32, topk=64, rebuild_max=20, prompt=0, steps=20)
    w, orc, hist = run_rebuild_first(cfg, steps=19)
    n = orc.n
    x = w.x_new(n)
    _, k, v = w.qkv(n, 0, x)
    orc.step_begin(x, None)
    orc.rebuild(0)
    lst = [int(t) for t in orc.info.rebuild_tok[0]]
    assert len(lst) >= 3
    q_rows = w.q_rows(n, 0, orc.x, orc.info.rebuild_tok)
    import copy
    base, _ = copy.deepcopy(orc).attend_rows(0, q_rows, k, v)
    i = int(np.argmin(lst))                                  # the oldest rebuilt token's row
    later = [s for s in range(cfg.capacity) if orc.slot_tok[0, s] > lst[i] and orc.slot_tok[0, s] != n]
    earlier = [s for s in range(cfg.capacity) if 0 <= orc.slot_tok[0, s] <= lst[i]]
    assert later and earlier
    o2 = copy.deepcopy(orc)
    o2.Vc[0, 0, :, later[0], :] += 1.0
    moved, _ = o2.attend_rows(0, q_rows, k, v)
    assert np.array_equal(moved[0, :, i], base[0, :, i])
    o3 = copy.deepcopy(orc)
    o3.Vc[0, 0, :, earlier[0], :] += 1.0
    moved, _ = o3.attend_rows(0, q_rows, k, v)
    assert not np.allclose(moved[0, :, i], base[0, :, i])
    # the current token's own row reaches the last query only
    o4 = copy.deepcopy(orc)
    moved, _ = o4.attend_rows(0, q_rows, k, v + 1.0)
    assert np.array_equal(moved[0, :, :-1], base[0, :, :-1]) and not np.allclose(moved[0, :, -1], base[0, :, -1])


def brute_select(score, slot_tok, slot_role, n, m, r_max, explicit):
    """Section 2.2 release rule and Section 2.3 list choice with Python sorts on (score, tok)."""
    slot_tok, slot_role = list(slot_tok), list(slot_role)
    for s in range(len(slot_tok)):
        if slot_role[s] == ao.REBUILT:
            slot_tok[s], slot_role[s] = -1, ao.EMPTY
    ret = [s for s in range(len(slot_tok)) if slot_role[s] == ao.RETAINED]
    evicted = -1
    if len(ret) == m:
        victim = min(ret, key=lambda s: (float(score[slot_tok[s]]), slot_tok[s]))
        evicted = slot_tok[victim]
        slot_tok[victim], slot_role[victim] = -1, ao.EMPTY
    admit = slot_role.index(ao.EMPTY)
    slot_tok[admit], slot_role[admit] = n, ao.RETAINED
    resident = set(t for t in slot_tok if t >= 0)
    cand = [t for t in range(n) if t not in resident]
    if explicit is not None:
        cand = [t for t in cand if t in set(int(e) for e in explicit)]
    cand.sort(key=lambda t: (float(score[t]), t), reverse=True)
    lst = cand[:r_max]
    empties = [s for s in range(len(slot_tok)) if slot_role[s] == ao.EMPTY]
    for t, s in zip(lst, empties):
        slot_tok[s], slot_role[s] = t, ao.REBUILT
    return slot_tok, slot_role, admit, evicted, lst


@pytest.mark.parametrize("mode", ["policy", "explicit"])
def test_selection_equals_full_sort_and_invariants_hold(mode):
    cfg = TINY.scaled(rebuild_mode=mode, rebuild_p=0.3, steps=40, capacity=8, rebuild_max=3)
    w = Workload(cfg)
    orc = make_oracle(w)
    g = np.random.default_rng(12)
    for s in range(cfg.steps):
        n = orc.n
        x = w.x_new(n)
        q, k, v = w.qkv(n, 0, x)
        lists, counts = w.explicit(s, n)
        ex = explicit_as_lists(lists, counts)
        if ex is not None and n > 2:      # hostile entries: duplicates, residents, out of range
            ex = [np.concatenate([e, e[:2], [n, n + 5, -1], g.integers(0, n, 3)]) for e in ex]
        before = (orc.slot_tok.copy(), orc.slot_role.copy())
        orc.decode_step(0, q, k, v, x, ex)
        orc.check_invariants()
        # ties: quantise scores after the fact is not possible, so ties are planted below instead
        for b in range(w.batch):
            st, sr, admit, ev, lst = brute_select(orc.score[b], before[0][b], before[1][b], n,
                                                  cfg.retained_max, cfg.rebuild_max,
                                                  None if ex is None else ex[b])
            assert st == orc.slot_tok[b].tolist() and sr == orc.slot_role[b].tolist()
            assert admit == orc.info.admit_slot[b] and ev == orc.info.evicted_tok[b]
            assert lst == orc.info.rebuild_tok[b].tolist()
        orc.rebuild(0)


def test_value_order_breaks_ties_towards_the_newer_token():
    score = np.array([0.5, 0.25, 0.5, 0.25, 0.75], np.float32)
    assert ao.by_value_desc(np.array([0, 1, 2, 3, 4]), score).tolist() == [4, 2, 0, 3, 1]
    assert ao.by_value_desc(np.array([3, 1]), score).tolist() == [3, 1]


@pytest.mark.parametrize("prompt", [1, 2, 7, 19, 64])
def test_bulk_load_retains_what_token_by_token_release_reaches(prompt):
    """The prompt's retained set equals the one reached by releasing one token at a time."""
    cfg = TINY.scaled(prompt=prompt, steps=2, capacity=8, rebuild_max=3, batch=2)
    w = Workload(cfg)
    bulk = make_oracle(w)
    bulk.append_tokens(w.prompt())
    bulk.check_invariants()
    seq = make_oracle(w)
    xs = w.prompt()
    for t in range(prompt):
        q, k, v = w.qkv(t, 0, xs[:, t])
        seq.decode_step(0, q, k, v, xs[:, t])
        seq.rebuild(0)
    for b in range(w.batch):
        r_bulk = np.sort(bulk.slot_tok[b][bulk.slot_role[b] == ao.RETAINED])
        r_seq = np.sort(seq.slot_tok[b][seq.slot_role[b] == ao.RETAINED])
        assert np.array_equal(r_bulk, r_seq)
        rb_bulk = bulk.slot_tok[b][bulk.slot_role[b] == ao.REBUILT]
        rb_seq = seq.slot_tok[b][seq.slot_role[b] == ao.REBUILT]
        assert np.array_equal(np.sort(rb_bulk), np.sort(rb_seq))
        assert np.array_equal(bulk.slot_tok[b][: r_bulk.size], r_bulk)          # canonical layout
    assert np.array_equal(bulk.score[:, :prompt], seq.score[:, :prompt])


@pytest.mark.parametrize("cfgname", ["tiny_policy", "tiny_explicit", "tiny_bf16"])
def test_resident_rows_equal_from_scratch_projection(cfgname):
    """Section 2.3: a rebuilt state is the recomputed state, whichever way the row got there."""
    cfg = {"tiny_policy": TINY.scaled(prompt=9),
           "tiny_explicit": TINY.scaled(rebuild_mode="explicit", rebuild_p=0.4),
           "tiny_bf16": TINY.scaled(dtype="bf16", prompt=5)}[cfgname]
    w, orc, _ = run_free(cfg)
    K, V = history_kv(w, orc, orc.n)
    seen_rebuilt = 0
    for b in range(w.batch):
        for s in range(cfg.capacity):
            t = orc.slot_tok[b, s]
            if t < 0:
                continue
            seen_rebuilt += orc.slot_role[b, s] == ao.REBUILT
            kk, vv = K[b, :, t], V[b, :, t]
            if cfg.dtype == "bf16":
                kk, vv = ao.round_bf16(kk), ao.round_bf16(vv)
            assert np.allclose(orc.Kc[0, b, :, s], kk, rtol=0, atol=1e-6 if cfg.dtype == "f32" else 0)
            assert np.allclose(orc.Vc[0, b, :, s], vv, rtol=0, atol=1e-6 if cfg.dtype == "f32" else 0)
    assert seen_rebuilt > 0


def test_occupancy_never_exceeds_capacity_on_config_one():
    cfg = wl.get_config(1).scaled(steps=96)
    w, orc, hist = run_free(cfg)            # invariants are asserted after every step
    occ = (orc.slot_tok >= 0).sum(-1)
    assert (occ <= cfg.capacity).all() and (orc.slot_role == ao.RETAINED).sum() == cfg.retained_max
    assert sum(len(l) for l in orc.info.rebuild_tok) >= 0


def test_controller_without_recurrence_forgets_earlier_tokens():
    """Section 3.5.3 "w/o GRU": the score of a token depends on its own embedding and position only, so shuffling the
    tokens before it changes nothing; with the recurrence the same shuffle moves the score."""
    cfg = wl.WorkloadConfig(name="norec", dtype="f32", n_layers=1, batch=2, n_heads=2, head_dim=64, hidden=128,
                            capacity=16, topk=8, rebuild_max=2, prompt=0, steps=12, rope_theta=0.0,
                            rebuild_mode="policy", rebuild_p=0.0, seed=77, ctrl_hidden=32)
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 9, 128)).astype(np.float32)
    perm = np.array([3, 0, 6, 1, 7, 5, 2, 4, 8])                 # the last token stays last
    last = {}
    for norec in (True, False):
        for name, xs in (("plain", x), ("shuffled", x[:, perm])):
            w = Workload(cfg.scaled(ctrl_no_recurrence=norec))
            orc = make_oracle(w)
            orc.append_tokens(xs)
            last[norec, name] = orc.score[:, 8].copy()
    assert np.array_equal(last[True, "plain"], last[True, "shuffled"])
    assert not np.allclose(last[False, "plain"], last[False, "shuffled"], rtol=0, atol=1e-7)
    # and it is the cell applied to a zero state: one token alone in an empty cache scores the same
    w = Workload(cfg.scaled(ctrl_no_recurrence=True))
    alone = make_oracle(w)
    alone.n = 8                                                   # same position, nothing before it
    alone._score_new_token(x[:, 8])
    assert np.array_equal(alone.score[:, 8], last[True, "plain"])


def test_labels_equal_counter_brute_force_and_invariants():
    """Section 2.2 / Appendix C: the label set is the top-K of the membership counts of the per-(layer, head) top-K/2
    sets; checked with collections.Counter and Python sets on seeded weights, plus what must always hold."""
    from collections import Counter
    L, B, H, S, K = 3, 2, 4, 41, 12
    w = wl.slot_weights(9, L, B, H, S, nonzero=K, empty_frac=0.2)
    sets, count, label, coverage, mass = ao.attention_labels(w, K)
    for b in range(B):
        c = Counter()
        per_layer = []
        for l in range(L):
            members = []
            for h in range(H):
                pos = [(float(w[l, b, h, s]), -s) for s in range(S) if w[l, b, h, s] > 0]
                top = [-i for _, i in sorted(pos, reverse=True)[: K // 2]]
                assert list(sets[l, b, h][sets[l, b, h] >= 0]) == top
                members += top
            c.update(members)
            per_layer.append(members)
        assert all(count[b, s] == c.get(s, 0) for s in range(S))
        ranked = sorted(c, key=lambda s: (-c[s], s))[:K]
        assert set(np.nonzero(label[b])[0]) == set(ranked)
        for l in range(L):
            assert coverage[l, b] == pytest.approx(sum(s in ranked for s in per_layer[l]) / len(per_layer[l]))
            assert mass[l, b] == pytest.approx(sum(float(w[l, b, h, s]) for h in range(H) for s in ranked) / H)
    assert count.sum() == sum(min(K // 2, int((w[l, b, h] > 0).sum())) for l in range(L) for b in range(B) for h in range(H))
    assert (label.sum(-1) <= K).all() and ((mass >= 0) & (mass <= 1 + 1e-6)).all()
    # the same row in every layer and head: the labelled set contains every set, so coverage is one
    same = np.broadcast_to(w[0, :, 0][None, :, None, :], w.shape).copy()
    _, _, lab, cov, _ = ao.attention_labels(same, K)
    assert (cov == 1.0).all() and (lab.sum(-1) == K // 2).all()
    # the order of the layers does not matter to the labels
    _, cnt2, lab2, _, _ = ao.attention_labels(w[::-1].copy(), K)
    assert np.array_equal(cnt2, count) and np.array_equal(lab2, label)


def test_cumulative_attention_scores_equal_column_sums_of_the_causal_attention_matrix():
    """Section 3.1 baseline 6 as a score source: with every token resident and no top-K mask, a token's value after S
    steps is the sum, over the steps that saw it and over the heads, of its softmax weight, i.e. a column sum of the
    dense causal attention matrix built from scratch; and every step hands out exactly one unit per head."""
    cfg = TINY.scaled(capacity=40, topk=100, rebuild_max=0, prompt=0, steps=30, score_from_attention=True)
    w, orc, hist = run_free(cfg)
    K, _ = history_kv(w, orc, orc.n)
    expect = np.zeros((w.batch, orc.n))
    for i, (q, _, _) in enumerate(hist):
        for b in range(w.batch):
            for h in range(cfg.n_heads):
                logit = np.array([float(np.dot(q[b, h].astype(np.float64), K[b, h, j])) / math.sqrt(cfg.head_dim) for j in range(i + 1)])
                e = np.exp(logit - logit.max())
                expect[b, : i + 1] += e / e.sum()
    assert np.allclose(orc.score[:, : orc.n], expect, rtol=1e-5, atol=1e-6)
    assert np.allclose(orc.score[:, : orc.n].sum(-1), len(hist) * cfg.n_heads, rtol=1e-5)
    # with a small cache the least attended retained token is the one that leaves
    small = TINY.scaled(capacity=8, topk=100, rebuild_max=2, prompt=0, steps=20, score_from_attention=True)
    w2 = Workload(small)
    o2 = make_oracle(w2)
    for s_ in range(small.steps):
        n = o2.n
        x = w2.x_new(n)
        q, k, v = w2.qkv(n, 0, x)
        before_tok, before_role, before_score = o2.slot_tok.copy(), o2.slot_role.copy(), o2.score.copy()
        o2.decode_step(0, q, k, v, x, None)
        o2.rebuild(0)
        for b in range(w2.batch):
            ev = int(o2.info.evicted_tok[b])
            if ev >= 0:
                ret = [int(t) for t, r in zip(before_tok[b], before_role[b]) if r == ao.RETAINED]
                assert ev == min(ret, key=lambda t: (float(before_score[b, t]), t))


# ------------------------------------------------------ relative positions (re-scoring every step)
def test_relative_rescoring_equals_torch_modules_on_the_distance_to_the_current_token():
    """Scores as seen from token n: the Appendix B modules fed with (n - i) / pos_scale and the state of token i."""
    d, h, n = 10, 6, 9
    w = _ctrl(d, h)
    pos, fc1, fc2 = torch.nn.Linear(1, h).double(), torch.nn.Linear(h, h).double(), torch.nn.Linear(h, 1).double()
    z = np.random.default_rng(21).standard_normal((3, n + 1, h))
    with torch.no_grad():
        pos.weight.copy_(torch.tensor(w["pos_w"], dtype=torch.float64)[:, None])
        pos.bias.copy_(torch.tensor(w["pos_b"], dtype=torch.float64))
        fc1.weight.copy_(torch.tensor(w["mlp_w1"], dtype=torch.float64))
        fc1.bias.copy_(torch.tensor(w["mlp_b1"], dtype=torch.float64))
        fc2.weight.copy_(torch.tensor(w["mlp_w2"], dtype=torch.float64)[None, :])
        fc2.bias.copy_(torch.tensor(w["mlp_b2"], dtype=torch.float64))
        dist = torch.tensor([[float(n - i)] for i in range(n + 1)], dtype=torch.float64) / 64.0     # [n+1, 1]
        ref = fc2(torch.tanh(fc1(pos(dist)[None] + torch.tensor(z))))[..., 0]
    got = ao.controller_rescore(z, n, 64.0, w)
    assert got.shape == (3, n + 1) and np.allclose(got, ref.numpy(), atol=1e-14)
    assert not np.allclose(got[:, :-1], got[:, 1:], atol=1e-6)          # the position feature does move the scores


REL = wl.WorkloadConfig(name="rel", dtype="f32", n_layers=1, batch=2, n_heads=2, head_dim=8, hidden=16, capacity=8,
                        topk=4, rebuild_max=2, prompt=0, steps=24, rope_theta=1.0e4, rebuild_mode="policy",
                        rebuild_p=0.0, seed=31, ctrl_hidden=8, pos_scale=16.0, ctrl_relative_position=True)


def test_relative_scores_shift_with_the_sequence_and_meet_the_absolute_score_at_the_same_distance():
    """Without the GRU's memory and with one and the same embedding for every token all states are equal, so the
    score as seen from token n depends on the distance n - i alone: the scores of step n + 1 are those of step n
    moved by one position, and a token at distance k scores what a token at ABSOLUTE position k scores under the
    absolute reading (which is pinned above)."""
    cfg = REL.scaled(ctrl_no_recurrence=True)
    w = Workload(cfg)
    x = np.tile(w.x_new(0)[:1, None, :], (cfg.batch, 1, 1))[:, 0]       # the same row for every sequence and token
    rel, ab = make_oracle(w), make_oracle(Workload(cfg.scaled(ctrl_relative_position=False)))
    prev = None
    for n in range(12):
        rel._score_new_token(x)
        ab._score_new_token(x)
        rel.n += 1
        ab.n += 1
        cur = rel.score[:, : n + 1].copy()
        assert np.array_equal(cur[:, ::-1], ab.score[:, : n + 1])      # distance k  <->  absolute position k
        if prev is not None:
            assert np.array_equal(cur[:, 1:], prev)
        prev = cur
    assert len(np.unique(prev[0])) == prev.shape[1]                    # the scores are not all alike


def test_relative_rescoring_with_a_zero_position_weight_is_the_absolute_path():
    """If the position layer ignores its input, the reading of the position cannot matter: same maps, same lists."""
    runs = []
    for relative in (True, False):
        w = Workload(REL.scaled(ctrl_relative_position=relative))
        w.ctrl = dict(w.ctrl, pos_w=np.zeros_like(w.ctrl["pos_w"]))
        orc = make_oracle(w)
        trace = []
        for s in range(REL.steps):
            x = w.x_new(orc.n)
            q, k, v = w.qkv(orc.n, 0, x)
            orc.decode_step(0, q, k, v, x, None)
            orc.rebuild(0)
            orc.check_invariants()
            trace.append((orc.slot_tok.copy(), orc.info.evicted_tok.copy(), [l.copy() for l in orc.info.rebuild_tok]))
        runs.append(trace)
    for (st_a, ev_a, l_a), (st_b, ev_b, l_b) in zip(*runs):
        assert np.array_equal(st_a, st_b) and np.array_equal(ev_a, ev_b)
        assert all(np.array_equal(a, b) for a, b in zip(l_a, l_b))
    assert any((ev >= 0).any() for _, ev, _ in runs[0])


@pytest.mark.parametrize("mode", ["policy", "explicit"])
def test_relative_selection_ranks_by_the_scores_of_the_current_step(mode):
    """Release rule and list choice with Python sorts, on the scores as seen from the token that was just added;
    over the run the order of two tokens must actually change (else the re-scoring would not be exercised)."""
    cfg = REL.scaled(rebuild_mode=mode, rebuild_p=0.3, steps=40, rebuild_max=3)
    w = Workload(cfg)
    # weights of order one instead of 0.02: the Tanh layer leaves its linear range, where a change of position would
    # move every token's score by the same amount and never change an order
    w.ctrl = {k: (v * 50.0 if k in ("pos_w", "pos_b", "mlp_w1", "mlp_b1", "gru_w_hh") else v) for k, v in w.ctrl.items()}
    orc = make_oracle(w)
    flips, before_scores = 0, None
    for s in range(cfg.steps):
        n = orc.n
        x = w.x_new(n)
        q, k, v = w.qkv(n, 0, x)
        ex = explicit_as_lists(*w.explicit(s, n))
        before = (orc.slot_tok.copy(), orc.slot_role.copy())
        orc.decode_step(0, q, k, v, x, ex)
        orc.check_invariants()
        assert np.allclose(orc.score[:, : n + 1], ao.controller_rescore(orc.z_rows[:, : n + 1], n, cfg.pos_scale, w.ctrl),
                           rtol=1e-6, atol=1e-9)
        for b in range(w.batch):
            st, sr, admit, ev, lst = brute_select(orc.score[b], before[0][b], before[1][b], n, cfg.retained_max,
                                                  cfg.rebuild_max, None if ex is None else ex[b])
            assert st == orc.slot_tok[b].tolist() and sr == orc.slot_role[b].tolist()
            assert admit == orc.info.admit_slot[b] and ev == orc.info.evicted_tok[b]
            assert lst == orc.info.rebuild_tok[b].tolist()
        if before_scores is not None:
            a, c = before_scores[0, :n], orc.score[0, :n]
            flips += int((np.sign(a[:, None] - a[None, :]) * np.sign(c[:, None] - c[None, :]) < 0).sum())
        before_scores = orc.score.copy()
        orc.rebuild(0)
    assert flips > 0


@pytest.mark.parametrize("prompt", [1, 5, 19])
def test_relative_bulk_load_selects_on_the_scores_seen_from_the_last_prompt_token(prompt):
    cfg = REL.scaled(prompt=prompt, steps=2)
    w = Workload(cfg)
    orc = make_oracle(w)
    orc.append_tokens(w.prompt())
    orc.check_invariants()
    want = ao.controller_rescore(orc.z_rows[:, :prompt], prompt - 1, cfg.pos_scale, w.ctrl).astype(np.float32)
    assert np.array_equal(orc.score[:, :prompt], want)
    for b in range(w.batch):
        ranked = sorted(range(prompt - 1), key=lambda t: (float(want[b, t]), t), reverse=True)
        keep = sorted(ranked[: cfg.retained_max - 1] + [prompt - 1])
        ret = orc.slot_tok[b][orc.slot_role[b] == ao.RETAINED].tolist()
        assert ret == keep
        assert orc.info.rebuild_tok[b].tolist() == ranked[cfg.retained_max - 1:][: cfg.rebuild_max]


# ------------------------------------------------- query projection, adopting a state
def test_query_projection_equals_explicit_loops():
    """The harness's query rows: y = W_q x with explicit loops, adjacent pairs (2j, 2j+1) of every head turned by
    position * theta^(-2j/dh) (the same rotation as the keys, so that q.k depends on the distance only), rounded to the
    element type by torch."""
    g = np.random.default_rng(21)
    H, dh, d, pos, theta = 3, 8, 10, 37, 1.0e4
    W = g.standard_normal((H * dh, d))
    x = g.standard_normal(d)
    y = [sum(float(W[i, j]) * float(x[j]) for j in range(d)) for i in range(H * dh)]
    ref = np.zeros((H, dh))
    for h in range(H):
        for j in range(dh // 2):
            ang = pos * theta ** (-2.0 * j / dh)
            a, b = y[h * dh + 2 * j], y[h * dh + 2 * j + 1]
            ref[h, 2 * j] = a * math.cos(ang) - b * math.sin(ang)
            ref[h, 2 * j + 1] = a * math.sin(ang) + b * math.cos(ang)
    got32 = ao.project_q(W, x, pos, H, dh, theta, "f32")
    assert got32.shape == (H, dh) and np.allclose(got32, ref, rtol=1e-6, atol=1e-6)
    got16 = ao.project_q(W, x, pos, H, dh, theta, "bf16")
    assert np.array_equal(got16, torch.from_numpy(ref).to(torch.bfloat16).float().numpy())
    # q.k of two rotated rows depends on the distance of their positions only
    k = g.standard_normal(d)
    dots = []
    for p0 in (5, 100):
        qq = ao.project_q(W, x, p0 + 9, H, dh, theta, "f32").astype(np.float64)
        kk = ao.project_q(W, k, p0, H, dh, theta, "f32").astype(np.float64)
        dots.append((qq * kk).sum(-1))
    assert np.allclose(dots[0], dots[1], atol=1e-4)


@pytest.mark.parametrize("mode", ["policy", "explicit"])
def test_a_run_continued_from_an_imported_state_equals_the_uninterrupted_run(mode):
    """Sections 2.2-2.3: the small state (slot map, roles, scores, z, stored embeddings, the last rebuild list) plus
    "a resident token's K/V is its recomputed state" determine everything that follows. A fresh oracle that adopts
    that state after 17 steps must produce, for the next 12 steps, the outputs and the state of the run that never
    stopped; a state whose list contradicts its map, or whose map names a token twice, is refused."""
    cfg = TINY.scaled(rebuild_mode=mode, rebuild_p=0.4, prompt=6, steps=40, capacity=8, rebuild_max=3, dtype="bf16")
    w, orc, _ = run_free(cfg, steps=17)
    other = make_oracle(w)
    other.import_state(orc.n, orc.slot_tok, orc.slot_role, orc.score, orc.sigma, orc.z, orc.x, orc.info.rebuild_tok,
                       orc.info.rebuild_slot, orc.info.admit_slot, orc.info.evicted_tok)
    occ = orc.slot_tok >= 0
    m = np.broadcast_to(occ[:, None, :, None], orc.Kc[0].shape)
    assert np.array_equal(other.Kc[0][m], orc.Kc[0][m]) and np.array_equal(other.Vc[0][m], orc.Vc[0][m])
    assert np.array_equal(other.tok_slot, orc.tok_slot)
    for s in range(17, 29):
        n = orc.n
        x = w.x_new(n)
        q, k, v = w.qkv(n, 0, x)
        lists, counts = w.explicit(s, n)
        ex = explicit_as_lists(lists, counts)
        o1, w1 = orc.decode_step(0, q, k, v, x, ex)
        o2, w2 = other.decode_step(0, q, k, v, x, ex)
        orc.rebuild(0)
        other.rebuild(0)
        other.check_invariants()
        assert np.array_equal(o1, o2) and np.array_equal(w1, w2)
        assert np.array_equal(orc.slot_tok, other.slot_tok) and np.array_equal(orc.slot_role, other.slot_role)
        assert np.array_equal(orc.score[:, : orc.n], other.score[:, : orc.n])
    bad = make_oracle(w)
    st = orc.slot_tok.copy()
    st[0, 0] = st[0, 1]                                        # one token in two slots
    with pytest.raises(ValueError):
        bad.import_state(orc.n, st, orc.slot_role, orc.score, orc.sigma, orc.z, orc.x, orc.info.rebuild_tok, orc.info.rebuild_slot)
    with pytest.raises(ValueError):                            # a list that the map does not show
        bad.import_state(orc.n, orc.slot_tok, orc.slot_role, orc.score, orc.sigma, orc.z, orc.x,
                         [l[:-1] for l in orc.info.rebuild_tok], [l[:-1] for l in orc.info.rebuild_slot])


# ------------------------------------------------------------------ planted mistakes
def test_pins_notice_planted_mistakes(monkeypatch):
    """Each plausible slip, planted in the oracle, must make one of the pins above fail."""
    def fails(test, *a):
        try:
            test(*a)
        except AssertionError:
            return True
        return False

    real_gru = ao.gru_step

    def gru_swapped_gates(x, z, w):          # update and reset gates exchanged
        h = z.shape[-1]
        perm = np.r_[h:2 * h, 0:h, 2 * h:3 * h]
        w2 = dict(w, gru_w_ih=w["gru_w_ih"][perm], gru_w_hh=w["gru_w_hh"][perm],
                  gru_b_ih=w["gru_b_ih"][perm], gru_b_hh=w["gru_b_hh"][perm])
        return real_gru(x, z, w2)

    monkeypatch.setattr(ao, "gru_step", gru_swapped_gates)
    assert fails(test_gru_step_equals_torch_gru_cell)
    monkeypatch.setattr(ao, "gru_step", real_gru)

    real_keep = ao.topk_keep
    monkeypatch.setattr(ao, "topk_keep", lambda lg, valid, k: real_keep(lg[..., ::-1], valid[..., ::-1], k)[..., ::-1])
    assert fails(test_topk_keep_equals_rank_counting)         # ties now go to the higher index
    assert fails(test_zero_query_gives_mean_of_lowest_index_rows)
    monkeypatch.setattr(ao, "topk_keep", real_keep)

    real_rope = ao.rope_rotate
    monkeypatch.setattr(ao, "rope_rotate", lambda v, p, t: real_rope(v, -p, t))   # wrong sign
    assert fails(test_rope_is_complex_rotation_and_depends_on_relative_position_only)
    assert fails(test_resident_rows_equal_from_scratch_projection, "tiny_policy")
    monkeypatch.setattr(ao, "rope_rotate", real_rope)

    real_order = ao.by_value_desc
    monkeypatch.setattr(ao, "by_value_desc", lambda t, s: real_order(t, -np.asarray(s)))  # keeps the worst
    assert fails(test_selection_equals_full_sort_and_invariants_hold, "policy")
    monkeypatch.setattr(ao, "by_value_desc", real_order)

    real_attn = ao.sparse_attention

    def attn_no_scale(q, *a):                # forgot 1/sqrt(dh)
        return real_attn(np.asarray(q, np.float64) * math.sqrt(q.shape[-1]), *a)

    monkeypatch.setattr(ao, "sparse_attention", attn_no_scale)
    assert fails(test_path_equals_full_attention_when_every_token_is_resident, 0, 0)
    monkeypatch.setattr(ao, "sparse_attention", real_attn)

    real_rescore = ao.controller_rescore
    monkeypatch.setattr(ao, "controller_rescore",                      # distance counted from the wrong end
                        lambda z, n, ps, w: real_rescore(np.asarray(z)[..., ::-1, :], n, ps, w)[..., ::-1])
    assert fails(test_relative_rescoring_equals_torch_modules_on_the_distance_to_the_current_token)
    assert fails(test_relative_scores_shift_with_the_sequence_and_meet_the_absolute_score_at_the_same_distance)
    monkeypatch.setattr(ao, "controller_rescore", lambda z, n, ps, w: real_rescore(z, n, ps / 2, w))   # wrong scale
    assert fails(test_relative_scores_shift_with_the_sequence_and_meet_the_absolute_score_at_the_same_distance)
    monkeypatch.setattr(ao, "controller_rescore", real_rescore)

    real_pq = ao.project_q
    monkeypatch.setattr(ao, "project_q", lambda w, x, p, H, dh, t, dt: real_pq(w, x, p + 1, H, dh, t, dt))
    assert fails(test_query_projection_equals_explicit_loops)          # rotated to the neighbouring position
    monkeypatch.setattr(ao, "project_q", real_pq)

    real_import = ao.AdoreOracle.import_state

    def import_without_z(self, n, st, sr, sc, sg, z, *a, **k):          # forgets the GRU state
        return real_import(self, n, st, sr, sc, sg, np.zeros_like(z), *a, **k)

    monkeypatch.setattr(ao.AdoreOracle, "import_state", import_without_z)
    assert fails(test_a_run_continued_from_an_imported_state_equals_the_uninterrupted_run, "policy")
    monkeypatch.setattr(ao.AdoreOracle, "import_state", real_import)
