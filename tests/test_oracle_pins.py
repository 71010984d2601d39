"""Pins of the CPU oracle against things other than itself (CPU only).

Full attention is pinned to the library SDPA, the top-k to a brute-force ranking, the sparse
attention to its two limiting cases (k >= context -> full causal attention, k = 0 ->
sliding-window attention) and to closed forms; two hand-worked vectors pin the tie-break, the
window and the reading of the GQA aggregation (Sections 3.3 and 3.4 of the paper).
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from gen import make_inputs, scaled

from conftest import read_golden


def _rand(shape, seed, dtype=torch.float32):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(*shape, generator=g).to(dtype)


def _sdpa(q, k, v, mask, scale=None):
    """Library attention in fp64 with an explicit boolean mask [Lq, Lk]; K/V repeated per group."""
    B, Lq, Hq, D = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    qq = q.double().permute(0, 2, 1, 3)
    kk = k.double().repeat_interleave(G, dim=2).permute(0, 2, 1, 3)
    vv = v.double().repeat_interleave(G, dim=2).permute(0, 2, 1, 3)
    o = F.scaled_dot_product_attention(qq, kk, vv, attn_mask=mask, scale=scale)
    return o.permute(0, 2, 1, 3).numpy()          # [B, Lq, Hq, D]


def _causal_mask(Lq, Lk):
    pos = torch.arange(Lq)[:, None] + (Lk - Lq)
    return torch.arange(Lk)[None, :] <= pos


# ---------------------------------------------------------------- full attention (Section 3.4)

@pytest.mark.parametrize("B,Lq,Lk,Hq,Hkv,D,dtype", [
    (2, 37, 37, 4, 2, 16, torch.float32),
    (1, 9, 50, 8, 1, 32, torch.bfloat16),      # chunked prefill: queries are the last 9 tokens
    (1, 64, 64, 6, 3, 8, torch.bfloat16),
])
def test_full_attention_matches_library_sdpa(B, Lq, Lk, Hq, Hkv, D, dtype):
    q, k, v = _rand((B, Lq, Hq, D), 1, dtype), _rand((B, Lk, Hkv, D), 2, dtype), _rand((B, Lk, Hkv, D), 3, dtype)
    O, LSE, _, _ = oracle.full_attn_select(q, k, v, 4, 2, want_idx=False)
    ref = _sdpa(q, k, v, _causal_mask(Lq, Lk))
    np.testing.assert_allclose(O.reshape(B, Lq, Hq, D), ref, rtol=0, atol=1e-12)
    # LSE against torch.logsumexp of the masked logits
    G = Hq // Hkv
    logits = torch.einsum("bihd,bjhd->bhij", q.double(), k.double().repeat_interleave(G, dim=2)) / math.sqrt(D)
    logits = logits.masked_fill(~_causal_mask(Lq, Lk), float("-inf"))
    lse = torch.logsumexp(logits, dim=-1).permute(0, 2, 1).numpy()
    np.testing.assert_allclose(LSE.reshape(B, Lq, Hq), lse, rtol=0, atol=1e-12)


def test_full_attention_explicit_scale_and_ragged_lengths():
    B, Lq, Lk, Hq, Hkv, D = 2, 5, 40, 4, 2, 16
    q, k, v = _rand((B, Lq, Hq, D), 4), _rand((B, Lk, Hkv, D), 5), _rand((B, Lk, Hkv, D), 6)
    kv_lens, q_start = [40, 23], [35, 10]
    O, _, _, _ = oracle.full_attn_select(q, k, v, 4, 2, scale=0.3, q_start=q_start, kv_lens=kv_lens,
                                         want_idx=False)
    O = O.reshape(B, Lq, Hq, D)
    for b in range(B):
        pos = torch.arange(Lq)[:, None] + q_start[b]
        j = torch.arange(Lk)[None, :]
        mask = (j <= pos) & (j < kv_lens[b])
        ref = _sdpa(q[b:b + 1], k[b:b + 1], v[b:b + 1], mask, scale=0.3)
        np.testing.assert_allclose(O[b], ref[0], rtol=0, atol=1e-12)


def test_scores_are_probabilities_rows_sum_to_one_when_group_is_one():
    B, L, H, D = 1, 33, 3, 8
    q, k, v = _rand((B, L, H, D), 7), _rand((B, L, H, D), 8), _rand((B, L, H, D), 9)
    _, LSE, _, sc = oracle.full_attn_select(q, k, v, 4, 2, want_idx=False, want_scores=True)
    sc = sc.reshape(L, H, L)
    for i in range(L):
        assert np.allclose(sc[i, :, :i + 1].sum(-1), 1.0, atol=1e-13)
        assert np.all(np.isneginf(sc[i, :, i + 1:]))


def test_uniform_logits_closed_form():
    """q = 0: every visible key has probability 1/(p+1); O = running mean of V; LSE = log(p+1)."""
    B, L, Hq, Hkv, D = 1, 20, 4, 2, 8
    q = torch.zeros(B, L, Hq, D)
    k, v = _rand((B, L, Hkv, D), 10), _rand((B, L, Hkv, D), 11)
    O, LSE, idx, _ = oracle.full_attn_select(q, k, v, k_sel=5, window=3)
    O = O.reshape(L, Hq, D)
    vd = v[0].double().numpy()
    for i in range(L):
        for h in range(Hq):
            np.testing.assert_allclose(O[i, h], vd[:i + 1, h // 2].mean(0), atol=1e-13)
        np.testing.assert_allclose(LSE[i], math.log(i + 1), atol=1e-13)
        # all-equal scores: the lower key index wins -> {0..k-1} among the candidates 0..i-3
        nc = max(0, i - 3 + 1)
        want = list(range(min(5, nc))) + [-1] * (5 - min(5, nc))
        assert idx[i, 0].tolist() == want and idx[i, 1].tolist() == want


# ---------------------------------------------------------------- top-k (Section 3.3)

def _brute_force_topk(score, pos, kvlen, w, k):
    """A candidate is kept iff fewer than k candidates beat it (higher score, or equal and lower index)."""
    last = min(pos - w, kvlen - 1)
    cand = list(range(0, last + 1))
    keep = []
    for j in cand:
        beaten_by = sum(1 for t in cand if score[t] > score[j] or (score[t] == score[j] and t < j))
        if beaten_by < k:
            keep.append(j)
    return keep + [-1] * (k - len(keep))


@pytest.mark.parametrize("seed", range(6))
def test_topk_matches_brute_force_ranking(seed):
    rng = np.random.default_rng(seed)
    Lk = 23
    for trial in range(40):
        levels = rng.integers(2, 9)
        score = rng.integers(0, levels, size=Lk).astype(np.float64) / 4.0 - 0.5     # many duplicates
        if trial % 5 == 0:
            score[rng.integers(0, Lk)] = -0.0
        pos = int(rng.integers(0, Lk + 3))
        kvlen = int(rng.integers(1, Lk + 1))
        w = int(rng.integers(0, 6))
        k = int(rng.integers(0, 12))
        got = oracle.select(score[None, :], pos, kvlen, w, k)[0].tolist()
        assert got == _brute_force_topk(score, pos, kvlen, w, k), (score, pos, kvlen, w, k)


def test_topk_invariants_on_random_scores():
    rng = np.random.default_rng(11)
    n, Lk, w, k = 64, 300, 7, 40
    score = rng.standard_normal((n, Lk))
    pos = rng.integers(0, Lk, size=n).astype(np.int32)
    idx = oracle.select(score, pos, Lk, w, k)
    idx_k1 = oracle.select(score, pos, Lk, w, k + 1)
    for r in range(n):
        sel = idx[r][idx[r] >= 0]
        nc = max(0, pos[r] - w + 1)
        assert len(sel) == min(k, nc)                              # count
        assert np.all(np.diff(sel) > 0)                            # strictly ascending, unique
        assert np.all(idx[r][len(sel):] == -1)                     # -1 padding at the end
        assert np.all(sel <= pos[r] - w)                           # never inside the window
        rest = np.setdiff1d(np.arange(nc), sel)
        if len(sel) and len(rest):
            assert score[r, sel].min() >= score[r, rest].max()     # nothing left out beats a kept one
        sel1 = idx_k1[r][idx_k1[r] >= 0]
        assert set(sel.tolist()) <= set(sel1.tolist())             # nested in k
    # argsort cross-check (stable sort of -score keeps the lower index first)
    for r in range(8):
        nc = max(0, pos[r] - w + 1)
        order = np.argsort(-score[r, :nc], kind="stable")[:k]
        assert sorted(order.tolist()) == idx[r][idx[r] >= 0].tolist()


def test_signed_zero_scores_tie():
    score = np.array([[0.0, -0.0, 0.0, -0.0, -1.0]])
    assert oracle.select(score, 4, 5, 0, 2)[0].tolist() == [0, 1]


# ---------------------------------------------------------------- hand-worked vectors

def test_E1_tiebreak_window_and_budget_sweep():
    g = read_golden("e1_tiebreak_window.txt")
    K = np.array(g["K"], dtype=np.float32).reshape(1, 6, 1, 1)
    q = np.ones((1, 6, 1, 1), dtype=np.float32)
    v = np.arange(6, dtype=np.float32).reshape(1, 6, 1, 1)
    w, i = int(g["window"][0]), int(g["query"][0])
    O, _, _, sc = oracle.full_attn_select(q, K, v, 1, w, rows=[(0, i)], scale=1.0, want_scores=True)
    np.testing.assert_allclose(sc[0, 0], g["P_full"], atol=2e-10)
    np.testing.assert_allclose(O[0, 0, 0], g["O_full"][0], atol=2e-10)
    for kk in (0, 1, 2, 4, 6):
        _, _, idx, _ = oracle.full_attn_select(q, K, v, kk, w, rows=[(0, i)], scale=1.0)
        assert idx[0, 0].tolist() == [int(t) for t in g["k%d_idx" % kk]]
        Os, _, mem = oracle.sparse_attn(q, K, v, idx, w, rows=[(0, i)], scale=1.0, want_member=True)
        np.testing.assert_allclose(Os[0, 0, 0], g["k%d_O" % kk][0], atol=2e-10)
        assert mem[0, 0, 4] == 1 and mem[0, 0, 5] == 1            # the window is always there
    P = np.array(g["P_full"])
    assert abs(P[[1, 3, 4, 5]].sum() - g["k2_mass"][0]) < 2e-10


def test_E2_group_aggregation_reading():
    g = read_golden("e2_group_aggregation.txt")
    K = np.array(g["K"], dtype=np.float32).reshape(1, 5, 1, 2)
    q = np.zeros((1, 5, 2, 2), dtype=np.float32)
    q[0, 4, 0], q[0, 4, 1] = g["q_h0"], g["q_h1"]
    v = np.zeros((1, 5, 1, 2), dtype=np.float32)
    for agg, key in ((oracle.AGG_MAX_PROB, "idx_max_prob"), (oracle.AGG_MAX_LOGIT, "idx_max_logit"),
                     (oracle.AGG_SUM_PROB, "idx_sum_prob")):
        _, _, idx, sc = oracle.full_attn_select(q, K, v, 1, 1, rows=[(0, 4)], scale=1.0, agg=agg,
                                                want_scores=True)
        assert idx[0, 0].tolist() == [int(g[key][0])], key
    _, _, _, sc = oracle.full_attn_select(q, K, v, 1, 1, rows=[(0, 4)], scale=1.0, want_scores=True)
    want = np.maximum(np.array(g["P_h0"]), np.array(g["P_h1"]))
    np.testing.assert_allclose(sc[0, 0], want, atol=6e-9)


def test_selection_is_invariant_under_head_permutation_inside_a_group():
    wl = scaled("cfg2", q_len=96, kv_len=96, n_q_heads=8, n_kv_heads=2, head_dim=16, k_sel=12, window=5,
                n_needles=4)
    inp = make_inputs(wl)
    _, _, idx, _ = oracle.full_attn_select(inp.q_full, inp.k, inp.v, wl.k_sel, wl.window)
    perm = [2, 0, 3, 1, 5, 7, 4, 6]                                # permutes inside each group of 4
    _, _, idx_p, _ = oracle.full_attn_select(inp.q_full[:, :, perm], inp.k, inp.v, wl.k_sel, wl.window)
    assert np.array_equal(idx, idx_p)


def test_group_of_one_selects_by_raw_logits():
    """With one query head per KV head the softmax is monotone per row: both readings agree with argsort."""
    B, L, H, D, k, w = 1, 48, 2, 8, 6, 4
    q, kk, v = _rand((B, L, H, D), 21), _rand((B, L, H, D), 22), _rand((B, L, H, D), 23)
    _, _, idx_p, _ = oracle.full_attn_select(q, kk, v, k, w, agg=oracle.AGG_MAX_PROB)
    logits = torch.einsum("ihd,jhd->hij", q[0].double(), kk[0].double()).numpy()
    for i in range(L):
        nc = max(0, i - w + 1)
        for h in range(H):
            order = np.argsort(-logits[h, i, :nc], kind="stable")[:k]
            assert sorted(order.tolist()) == idx_p[i, h][idx_p[i, h] >= 0].tolist()


# ---------------------------------------------------------------- sparse attention (Section 3.3)

def _inputs_small(dtype="bf16"):
    wl = scaled("cfg2", q_len=80, kv_len=80, n_q_heads=8, n_kv_heads=2, head_dim=16, k_sel=10, window=6,
                n_needles=4, dtype=dtype)
    return wl, make_inputs(wl)


def test_budget_covering_the_context_gives_full_causal_attention():
    wl, inp = _inputs_small()
    L = wl.kv_len
    _, _, idx, _ = oracle.full_attn_select(inp.q_full, inp.k, inp.v, L, wl.window)     # k >= context
    qs = inp.q_sparse[0]
    Os, LSEs, _ = oracle.sparse_attn(qs, inp.k, inp.v, idx, wl.window)
    Of, LSEf, _, _ = oracle.full_attn_select(qs, inp.k, inp.v, 1, 1, want_idx=False)
    np.testing.assert_allclose(Os, Of, atol=1e-12)
    np.testing.assert_allclose(LSEs, LSEf, atol=1e-12)
    ref = _sdpa(qs, inp.k, inp.v, _causal_mask(L, L))
    np.testing.assert_allclose(Os.reshape(1, L, wl.n_q_heads, wl.head_dim), ref, atol=1e-12)


def test_zero_budget_gives_sliding_window_attention():
    wl, inp = _inputs_small()
    L, w = wl.kv_len, wl.window
    idx = np.zeros((L, wl.n_kv_heads, 0), dtype=np.int32)
    qs = inp.q_sparse[0]
    Os, _, _ = oracle.sparse_attn(qs, inp.k, inp.v, idx, w)
    i, j = torch.arange(L)[:, None], torch.arange(L)[None, :]
    band = (j <= i) & (j > i - w)
    ref = _sdpa(qs, inp.k, inp.v, band)
    np.testing.assert_allclose(Os.reshape(1, L, wl.n_q_heads, wl.head_dim), ref, atol=1e-12)


def test_window_always_selected_topk_outside_it_and_set_size():
    wl, inp = _inputs_small()
    L, w, k = wl.kv_len, wl.window, wl.k_sel
    _, _, idx, _ = oracle.full_attn_select(inp.q_full, inp.k, inp.v, k, w)
    _, _, mem = oracle.sparse_attn(inp.q_sparse[0], inp.k, inp.v, idx, w, want_member=True)
    for i in range(L):
        for g in range(wl.n_kv_heads):
            m = mem[i, g]
            assert m[max(0, i - w + 1):i + 1].all()                       # forced window
            assert not m[i + 1:].any()                                    # causal
            sel = idx[i, g][idx[i, g] >= 0]
            assert np.all(sel <= i - w)                                   # top-k taken outside the window
            assert m.sum() == min(i + 1, w) + min(k, max(0, i + 1 - w))    # |S|


def test_malformed_indices_are_ignored():
    """Entries that are negative, inside the window, in the future, past the cache or repeated add nothing."""
    wl, inp = _inputs_small()
    w = wl.window
    i = 50
    good = np.array([3, 9, 17, 30], dtype=np.int32)
    bad = np.array([3, -1, 9, 48, 17, 60, 30, 200, -7, 9], dtype=np.int32)     # 48 in window, 60 future
    def run(row):
        idx = np.tile(row, (1, wl.n_kv_heads, 1))
        return oracle.sparse_attn(inp.q_sparse[0], inp.k, inp.v, idx, w, rows=[(0, i)])[0]
    np.testing.assert_allclose(run(bad), run(good), atol=1e-14)


def test_same_queries_give_the_renormalised_restriction_of_the_full_softmax():
    """With the full layer's own Q the sparse output is sum_{j in S} P_j V_j / sum_{j in S} P_j."""
    wl, inp = _inputs_small()
    L, w, k, G = wl.kv_len, wl.window, wl.k_sel, wl.group
    rows = [(0, i) for i in (0, 5, 6, 17, 40, 79)]
    Of, LSEf, idx, _ = oracle.full_attn_select(inp.q_full, inp.k, inp.v, k, w, rows=rows)
    Os, LSEs, mem = oracle.sparse_attn(inp.q_full, inp.k, inp.v, idx, w, rows=rows, want_member=True)
    qd, kd, vd = inp.q_full[0].double().numpy(), inp.k[0].double().numpy(), inp.v[0].double().numpy()
    for r, (_, i) in enumerate(rows):
        for h in range(wl.n_q_heads):
            g = h // G
            s = kd[:i + 1, g] @ qd[i, h] / math.sqrt(wl.head_dim)
            P = np.exp(s - LSEf[r, h])
            S = np.nonzero(mem[r, g][:i + 1])[0]
            mass = P[S].sum()
            np.testing.assert_allclose(Os[r, h], (P[S, None] * vd[S, g]).sum(0) / mass, atol=1e-12)
            np.testing.assert_allclose(LSEs[r, h], LSEf[r, h] + math.log(mass), atol=1e-12)
            bound = 2.0 * (1.0 - mass) * np.abs(vd[:i + 1, g]).max()
            assert np.abs(Os[r, h] - Of[r, h]).max() <= bound + 1e-12


def test_sink_bias_closed_form():
    wl, inp = _inputs_small()
    w, k = wl.window, wl.k_sel
    rows = [(0, 3), (0, 33), (0, 79)]
    _, _, idx, _ = oracle.full_attn_select(inp.q_full, inp.k, inp.v, k, w, rows=rows)
    qs = inp.q_sparse[0]
    O0, LSE0, _ = oracle.sparse_attn(qs, inp.k, inp.v, idx, w, rows=rows)
    Oinf, LSEinf, _ = oracle.sparse_attn(qs, inp.k, inp.v, idx, w, rows=rows,
                                         sink=np.full(wl.n_q_heads, -np.inf))
    np.testing.assert_allclose(Oinf, O0, atol=0)
    np.testing.assert_allclose(LSEinf, LSE0, atol=0)
    sink = np.linspace(-2.0, 3.0, wl.n_q_heads)
    Os, LSEs, _ = oracle.sparse_attn(qs, inp.k, inp.v, idx, w, rows=rows, sink=sink)
    shrink = np.exp(LSE0) / (np.exp(LSE0) + np.exp(sink)[None, :])        # the sink only enlarges the denominator
    np.testing.assert_allclose(Os, O0 * shrink[:, :, None], atol=1e-12)
    np.testing.assert_allclose(LSEs, np.logaddexp(LSE0, sink[None, :]), atol=1e-12)


def test_decode_equals_last_row_of_prefill():
    wl, inp = _inputs_small()
    L, w, k = wl.kv_len, wl.window, wl.k_sel
    Of, LSEf, idxf, _ = oracle.full_attn_select(inp.q_full, inp.k, inp.v, k, w, rows=[(0, L - 1)])
    q1 = inp.q_full[:, L - 1:L].contiguous()
    Od, LSEd, idxd, _ = oracle.full_attn_select(q1, inp.k, inp.v, k, w)               # Lq = 1
    np.testing.assert_allclose(Od, Of, atol=0)
    assert np.array_equal(idxd, idxf)
    qs1 = inp.q_sparse[0][:, L - 1:L].contiguous()
    Osd, _, _ = oracle.sparse_attn(qs1, inp.k, inp.v, idxd, w)
    Osp, _, _ = oracle.sparse_attn(inp.q_sparse[0], inp.k, inp.v, idxf, w, rows=[(0, L - 1)])
    np.testing.assert_allclose(Osd, Osp, atol=0)


def test_sparse_attention_with_causal_offsets_and_ragged_cache_lengths():
    """`q_start` / `kv_lens`: the sparse row is the library attention under an explicit mask built from
    the definition - key j is attended iff j < kv_lens[b] and (j in the forced window [pos-w+1, pos] or j a listed
    index <= pos - w), pos = q_start[b] + i.  The second sequence's cache length cuts its windows (and, for its last
    queries, removes the query's own token), the third has queries whose window is cut to nothing but one key."""
    B, Lq, Lk, Hq, Hkv, D, w, k = 3, 7, 48, 4, 2, 16, 6, 5
    q, kk, v = _rand((B, Lq, Hq, D), 31), _rand((B, Lk, Hkv, D), 32), _rand((B, Lk, Hkv, D), 33)
    q_start, kv_lens = [41, 20, 9], [48, 23, 11]      # seq 1: pos 20..26 vs 23 keys; seq 2: pos 9..15 vs 11 keys
    rng = np.random.default_rng(5)
    rows = [(b, i) for b in range(B) for i in range(Lq)]
    # listed indices: random keys of the whole tensor extent, so some are in the window, in the future or past the
    # ragged end (all of which the definition drops); no duplicates inside a row
    idx = np.stack([np.stack([np.sort(rng.choice(Lk, size=k, replace=False)) for _ in range(Hkv)]) for _ in rows])
    idx = idx.astype(np.int32)
    idx[3, 0, 1] = -1
    O, LSE, mem = oracle.sparse_attn(q, kk, v, idx, w, rows=rows, scale=0.37, q_start=q_start, kv_lens=kv_lens,
                                     want_member=True)
    G = Hq // Hkv
    cut_window = cut_self = 0
    for r, (b, i) in enumerate(rows):
        pos = q_start[b] + i
        for g in range(Hkv):
            mask = torch.zeros(Lk, dtype=torch.bool)
            for j in range(Lk):
                listed = j in idx[r, g].tolist() and j <= pos - w
                in_window = pos - w + 1 <= j <= pos
                mask[j] = (listed or in_window) and j < kv_lens[b]
            assert np.array_equal(mem[r, g].astype(bool), mask.numpy())
            assert mask.any()
            cut_window += int(pos - w + 1 < kv_lens[b] <= pos)
            cut_self += int(kv_lens[b] <= pos)
            hs = slice(g * G, (g + 1) * G)
            ref = _sdpa(q[b:b + 1, i:i + 1, hs], kk[b:b + 1, :, g:g + 1], v[b:b + 1, :, g:g + 1], mask[None, :],
                        scale=0.37)
            np.testing.assert_allclose(O[r, hs], ref[0, 0], rtol=0, atol=1e-12)
            logits = 0.37 * torch.einsum("hd,jd->hj", q[b, i, hs].double(), kk[b, :, g].double())
            lse = torch.logsumexp(logits.masked_fill(~mask[None, :], float("-inf")), dim=-1).numpy()
            np.testing.assert_allclose(LSE[r, hs], lse, rtol=0, atol=1e-12)
    assert cut_window >= 8 and cut_self >= 8          # the ragged end really cuts windows in this case


def test_fp32_and_bf16_inputs_are_read_exactly():
    """bf16 bit patterns are widened exactly: the same values given as fp32 produce the same result."""
    wl, inp = _inputs_small()
    rows = [(0, 20), (0, 79)]
    a = oracle.full_attn_select(inp.q_full, inp.k, inp.v, wl.k_sel, wl.window, rows=rows)
    b = oracle.full_attn_select(inp.q_full.float(), inp.k.float(), inp.v.float(), wl.k_sel, wl.window, rows=rows)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[2], b[2])


def test_output_gate_special_values_and_library_sigmoid():
    """Sigmoid output gate of the sparse layers (Section 4.1): logit 0 halves the output exactly, a large logit
    leaves it unchanged, a very negative one removes it, LSE is untouched, and a random gate agrees with torch's
    own fp64 sigmoid applied to the ungated result."""
    wl = scaled("cfg1", q_len=24, kv_len=24, k_sel=6, window=3)
    inp = make_inputs(wl)
    _, _, idx, _ = oracle.full_attn_select(inp.q_full, inp.k, inp.v, wl.k_sel, wl.window)
    q = inp.q_sparse[0]
    O0, L0, _ = oracle.sparse_attn(q, inp.k, inp.v, idx, wl.window)
    for val, fac in ((0.0, 0.5), (40.0, 1.0), (-700.0, 0.0)):
        g = torch.full(q.shape, val, dtype=torch.float32)
        O1, L1, _ = oracle.sparse_attn(q, inp.k, inp.v, idx, wl.window, gate=g)
        assert np.allclose(O1, O0 * fac, rtol=0, atol=1e-15)
        assert np.array_equal(L1, L0)
    g = torch.randn(q.shape, generator=torch.Generator().manual_seed(5), dtype=torch.float32) * 3
    O2, _, _ = oracle.sparse_attn(q, inp.k, inp.v, idx, wl.window, gate=g)
    B, Lq, Hq, D = q.shape
    want = O0 * torch.sigmoid(g.double()).reshape(B * Lq, Hq, D).numpy()
    assert np.abs(O2 - want).max() < 1e-14
    gb = g.to(torch.bfloat16)                       # bf16 logits are read exactly
    O3, _, _ = oracle.sparse_attn(q, inp.k, inp.v, idx, wl.window, gate=gb)
    want = O0 * torch.sigmoid(gb.double()).reshape(B * Lq, Hq, D).numpy()
    assert np.abs(O3 - want).max() < 1e-14


def test_e4m3_decoder_against_the_format_and_torch():
    """The oracle's e4m3 decoder: landmark codes from the format definition, and all 256 codes against torch's
    float8_e4m3fn -> float32 conversion."""
    codes = np.arange(256, dtype=np.uint8)
    val = oracle.decode_e4m3(codes)
    assert val[0x00] == 0.0 and val[0x38] == 1.0 and val[0x7E] == 448.0 and val[0x01] == 2.0 ** -9 and val[0x08] == 2.0 ** -6
    assert val[0xB8] == -1.0 and np.isnan(val[0x7F]) and np.isnan(val[0xFF])
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    ok = ~np.isnan(ref)
    assert np.array_equal(np.isnan(val), ~ok) and np.array_equal(val[ok], ref[ok])
    x = torch.randn(2, 5, 3, 16, generator=torch.Generator().manual_seed(3))
    from gen.workloads import quantize_kv_e4m3
    c8, sc = quantize_kv_e4m3(x)
    deq = oracle.dequant_e4m3(c8, sc)
    assert deq.dtype == np.float32 and np.abs(deq - x.numpy()).max() <= np.abs(x.numpy()).max() / 16 + 1e-6   # 3 mantissa bits
    assert np.abs(deq).reshape(-1, 16).max(axis=1).max() <= np.abs(x.numpy()).max() * (1 + 1e-6)


def test_block_level_selection_reduces_to_token_level_and_matches_brute_force():
    """Block-level selection (Section 5, Ablation 1): block size 1 is the token-level selection; for larger blocks
    a block is kept iff fewer than k/B candidate blocks beat it (score, then lower index), and exactly the candidate
    keys of the kept blocks are listed, ascending."""
    rng = np.random.default_rng(7)
    n, Lk, w = 40, 97, 5
    sc = np.round(rng.normal(size=(n, Lk)) * 2) / 2          # many ties
    pos = rng.integers(0, Lk + 10, size=n)
    kvl = rng.integers(1, Lk + 1, size=n)
    assert np.array_equal(oracle.select_blocks(sc, pos, kvl, w, 12, 1), oracle.select(sc, pos, kvl, w, 12))
    for B, k in ((4, 12), (8, 16), (16, 64)):
        idx = oracle.select_blocks(sc, pos, kvl, w, k, B)
        for r in range(n):
            nk = max(0, min(pos[r] - w + 1, kvl[r]))
            nb = -(-nk // B)
            bmax = [sc[r, m * B:min(nk, (m + 1) * B)].max() for m in range(nb)]
            kept = {m for m in range(nb)
                    if sum(1 for o in range(nb) if bmax[o] > bmax[m] or (bmax[o] == bmax[m] and o < m)) < k // B}
            want = [j for m in sorted(kept) for j in range(m * B, min(nk, (m + 1) * B))]
            got = [j for j in idx[r] if j >= 0]
            assert got == want and all(j == -1 for j in idx[r, len(got):])


def test_kv_projection_is_the_plain_sum_of_products():
    g = torch.Generator().manual_seed(2)
    h = torch.randn(5, 7, generator=g).to(torch.bfloat16)
    w = torch.randn(3, 7, generator=g).to(torch.bfloat16)
    c = oracle.kv_project(h, w)
    for t in range(5):
        for n in range(3):
            want = sum(float(h[t, d]) * float(w[n, d]) for d in range(7))
            assert abs(c[t, n] - want) < 1e-12
