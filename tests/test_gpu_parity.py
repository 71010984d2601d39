"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle on the same seeded bytes."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_26368_b200 as hs2
from gen import CONFIGS, make_inputs, scaled
from parity import BlockRun, TOL, assert_output_close, check_idx_against_oracle, gather_rows, rows_all, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    hs2.load_library()


# ---------------------------------------------------------------- configuration 1 (fp32), everything, every row

def test_cfg1_block_every_row():
    run = BlockRun(make_inputs(CONFIGS["cfg1"])).run_full(want_scores=True)
    run.check_full(check_scores=True)
    run.check_idx_bitexact_on_gpu_scores()
    out, lse = run.run_sparse(0)
    run.check_sparse(out, lse, 0)


def test_cfg1_strip_path_equals_debug_path():
    """Without scores_dbg the scores go through bounded workspace strips, a few rows at a time."""
    inp = make_inputs(CONFIGS["cfg1"])
    a = BlockRun(inp).run_full(want_scores=True)
    ws = torch.empty(7 * 512 * 4 + 256, dtype=torch.uint8, device="cuda")      # 7 rows per launch
    b = BlockRun(inp).run_full(want_scores=False, ws=ws)
    assert torch.equal(a.idx, b.idx)
    c = BlockRun(inp).run_full(want_scores=False)                               # recommended workspace
    assert torch.equal(a.idx, c.idx)
    assert torch.equal(a.O, c.O)


# ---------------------------------------------------------------- top-k on given scores: bit exact

def _topk_case(scores: torch.Tensor, k, w, q_start=None, kv_lens=None):
    B, Hkv, Lq, Lk = scores.shape
    qs = None if q_start is None else torch.tensor(q_start, dtype=torch.int32, device="cuda")
    kl = None if kv_lens is None else torch.tensor(kv_lens, dtype=torch.int32, device="cuda")
    prob = hs2.Problem(B, Lq, Lk, Hkv, Hkv, 1, k, w, dtype=torch.float32, q_start=qs, kv_lens=kl)
    got = hs2.hs2_topk_select(prob, scores.cuda().contiguous()).cpu().numpy()
    pos, kvl = [], []
    for b in range(B):
        n = Lk if kv_lens is None else kv_lens[b]
        q0 = n - Lq if q_start is None else q_start[b]
        for g in range(Hkv):
            for i in range(Lq):
                pos.append(q0 + i)
                kvl.append(n)
    want = oracle.select(scores.numpy().reshape(-1, Lk), np.array(pos), np.array(kvl), w, k)
    assert np.array_equal(got.reshape(-1, k), want)


@pytest.mark.parametrize("Lk,k,w", [(512, 64, 16), (1000, 100, 0), (3000, 700, 5), (4099, 257, 33), (9001, 1024, 128),
                                     (14000, 3000, 64), (30000, 2048, 128)])   # every row class of the register kernels
def test_topk_random_scores(Lk, k, w):
    g = torch.Generator().manual_seed(Lk)
    _topk_case(torch.randn(2, 2, 37, Lk, generator=g), k, w, q_start=[Lk - 37, Lk // 2], kv_lens=[Lk, Lk - 5])
    # positions known on the host: every class launch covers only its own queries
    _topk_case(torch.randn(1, 2, 61, Lk, generator=g) * 3.0 - 9.0, k, w)


@pytest.mark.parametrize("Lk", [2500, 12000, 20000])   # 128, 512 and 512 x 64 thread classes
def test_topk_adversarial_rows(Lk):
    g = torch.Generator().manual_seed(5)
    rows = [
        torch.zeros(Lk),                                                   # all equal: lowest indices win
        torch.full((Lk,), -3.25),
        torch.randint(0, 4, (Lk,), generator=g).float(),                   # four distinct values
        torch.where(torch.arange(Lk) % 2 == 0, torch.tensor(0.0), torch.tensor(-0.0)),     # +0 / -0 tie
        torch.randn(Lk, generator=g) * 1e-41,                              # denormals
        torch.cat([torch.full((Lk // 2,), float("-inf")), torch.randn(Lk - Lk // 2, generator=g)]),
        torch.cat([torch.full((5,), float("inf")), torch.randn(Lk - 5, generator=g)]),
        -torch.rand(Lk, generator=g) * 30.0,                               # log-probability like
        torch.arange(Lk).float(),                                          # ascending: the last k candidates
        -torch.arange(Lk).float(),                                         # descending: the first k
        torch.randn(Lk, generator=g).abs().log(),
        (torch.randn(Lk, generator=g) * 4).round() / 4 - 12.0,             # dense near-ties
    ]
    scores = torch.stack(rows).view(1, 1, len(rows), Lk)
    for k, w in [(1, 0), (300, 7), (1024, 128), (2400, 50), (4000, 0)]:     # k >= candidates included
        _topk_case(scores, k, w, q_start=[Lk - 1 - len(rows) + 1])


def test_topk_host_known_positions_adversarial_rows_in_the_longest_register_class():
    """Positions known on the host (every class launch covers only its own queries) and rows of 16385..32768 candidates
    that are staged through the shared list's memory: rows whose threshold bin holds (nearly) the whole row then fill
    that list completely; ties, flat rows, denormals; staged and unstaged output rows."""
    Lk, Lq = 24000, 40
    g = torch.Generator().manual_seed(77)
    s = torch.randn(1, 2, Lq, Lk, generator=g) * 2.0 - 10.0
    s[0, 0, 3] = -4.0                                              # all equal: the list holds the whole row
    s[0, 0, 4] = (s[0, 0, 4] * 2).round() / 2                      # heavy ties
    s[0, 0, 17, : Lk // 2] = -7.5                                  # half of the row in one bin
    s[0, 1, 20:23] = 0.0
    s[0, 1, 30] = torch.where(torch.arange(Lk) % 3 == 0, torch.tensor(-1.0), torch.tensor(-1.0e-41))   # denormals against a flat rest
    for k, w in [(2048, 128), (1000, 0), (4096, 333), (5000, 64)]:    # staged and unstaged output rows
        _topk_case(s, k, w)


@pytest.mark.parametrize("Lk,k,w", [(40000, 2048, 128), (70001, 4096, 256), (131072, 4096, 256), (200003, 1000, 17),
                                     (262144, 4096, 0), (300000, 512, 64)])
def test_topk_long_rows_cluster_and_streaming_variants(Lk, k, w):
    """Rows beyond 32768 candidates: cluster kernels of 2, 4 and 8 CTAs, and the streaming kernel above that."""
    g = torch.Generator().manual_seed(Lk)
    s = torch.randn(1, 2, 6, Lk, generator=g) - 9.0
    s[0, 0, 1] = (s[0, 0, 1] * 2).round() / 2                      # heavy ties
    s[0, 1, 2] = -5.0                                              # all equal
    _topk_case(s, k, w, q_start=[Lk - 6])
    _topk_case(s, k, w, q_start=[Lk // 2])                         # rows that fall into a smaller variant


@pytest.mark.parametrize("Lk", [8192, 20000, 40000, 100000])
def test_topk_threshold_bin_larger_than_the_shared_list(Lk):
    """Few distinct values over long rows: the bin that holds the k-th value has thousands of members,
    so the register kernels must fall back from their shared-memory candidate list (both variants),
    and the streaming kernel sees heavy ties."""
    g = torch.Generator().manual_seed(Lk)
    rows = [
        torch.randint(0, 3, (Lk,), generator=g).float() - 9.0,                  # three values
        (torch.randn(Lk, generator=g) * 0.01).round() - 11.0,                    # almost everything equal
        torch.where(torch.rand(Lk, generator=g) < 0.5, torch.tensor(-7.5), torch.tensor(-7.25)),
        -8.0 - torch.rand(Lk, generator=g) * 2.0 ** -12,                         # differ only in the low mantissa bits
        torch.randn(Lk, generator=g) - 10.0,
    ]
    scores = torch.stack(rows).view(1, 1, len(rows), Lk)
    for k, w in [(1024, 128), (5, 0), (Lk // 2, 64)]:
        _topk_case(scores, k, w, q_start=[Lk - len(rows)])


def test_topk_edges_window_and_lengths():
    g = torch.Generator().manual_seed(9)
    s = torch.randn(1, 3, 1, 777, generator=g)
    _topk_case(s, 50, 10)                                                  # Lq = 1 (decode)
    _topk_case(s, 50, 777)                                                 # window covers everything: all -1
    _topk_case(s, 50, 5000)
    _topk_case(s, 900, 3)                                                  # k above the context
    s2 = torch.randn(2, 1, 40, 129, generator=g)
    _topk_case(s2, 16, 4, q_start=[0, 60], kv_lens=[129, 77])              # early rows; query past a short cache
    _topk_case(s2, 16, 4, q_start=[-3, 200], kv_lens=[129, 0])             # negative positions; empty cache


# ---------------------------------------------------------------- small shapes, both dtypes, ragged tails, strides

SMALL = [
    # name, overrides
    ("cfg1", dict(q_len=131, kv_len=131, k_sel=17, window=5)),
    ("cfg1", dict(q_len=40, kv_len=300, k_sel=33, window=9, n_q_heads=6, n_kv_heads=2, head_dim=32)),
    ("cfg2", dict(q_len=333, kv_len=333, k_sel=48, window=13, n_needles=8)),
    ("cfg2", dict(q_len=257, kv_len=257, k_sel=64, window=16, n_q_heads=8, n_kv_heads=2, head_dim=64, n_needles=8)),
    ("cfg2", dict(q_len=96, kv_len=1029, k_sel=128, window=32, n_needles=8, batch=2)),
    ("cfg4", dict(q_len=600, kv_len=600, k_sel=100, window=20, n_clusters=8)),
    ("cfg2", dict(q_len=200, kv_len=200, k_sel=300, window=8, n_needles=4)),            # k above the context
    ("cfg2", dict(q_len=200, kv_len=200, k_sel=0, window=24, n_needles=4)),              # pure sliding window
    ("cfg2", dict(q_len=200, kv_len=200, k_sel=40, window=0, n_needles=4)),              # no window
    ("cfg2", dict(q_len=150, kv_len=150, k_sel=16, window=4, n_q_heads=4, n_kv_heads=4, n_needles=4)),   # group of 1
    ("cfg2", dict(q_len=150, kv_len=150, k_sel=16, window=4, n_q_heads=16, n_kv_heads=1, n_needles=4)),  # MQA 16
    ("cfg2", dict(q_len=130, kv_len=420, k_sel=48, window=10, n_q_heads=48, n_kv_heads=3, n_needles=4, batch=2)),  # groups of 16
    ("cfg2", dict(q_len=90, kv_len=300, k_sel=32, window=8, n_q_heads=64, n_kv_heads=2, n_needles=4)),   # groups of 32
    ("cfg2", dict(q_len=140, kv_len=380, k_sel=40, window=12, n_q_heads=24, n_kv_heads=2, n_needles=4)),  # groups of 12 (padded to 16)
    ("cfg2", dict(q_len=100, kv_len=330, k_sel=40, window=12, n_q_heads=6, n_kv_heads=2, head_dim=256, n_needles=4)),  # groups of 3, dim 256
    ("cfg2", dict(q_len=100, kv_len=330, k_sel=40, window=12, n_q_heads=3, n_kv_heads=3, head_dim=256, n_needles=4)),  # groups of 1, dim 256
    ("cfg2", dict(q_len=70, kv_len=280, k_sel=40, window=12, n_q_heads=48, n_kv_heads=1, head_dim=256, n_needles=4)),  # group of 48, dim 256
    ("cfg2", dict(q_len=300, kv_len=300, k_sel=64, window=16, n_q_heads=16, n_kv_heads=2, head_dim=256, n_needles=8)),
    ("cfg2", dict(q_len=260, kv_len=700, k_sel=64, window=16, n_q_heads=64, n_kv_heads=1, head_dim=256, n_needles=8)),  # paper's shape
]


@pytest.mark.parametrize("name,over", SMALL)
def test_small_block_every_row(name, over):
    wl = scaled(name, **over)
    run = BlockRun(make_inputs(wl)).run_full(want_scores=True)
    run.check_full(check_scores=True)
    if wl.k_sel > 0:
        run.check_idx_bitexact_on_gpu_scores()
    for layer in range(len(run.qs)):
        out, lse = run.run_sparse(layer)
        run.check_sparse(out, lse, layer)


def test_filtered_selection_equals_selection_on_the_full_score_rows():
    """bf16 tensor-core path: without scores_dbg the layer thresholds a 1/8 sample, keeps ordered candidate lists
    and selects from them; with scores_dbg it selects from complete score rows.  Same scores, same indices."""
    old = hs2.hs2_set_filter_min_keys(1)          # force the filtered path on these small shapes
    try:
        _filtered_equals_full_rows()
    finally:
        hs2.hs2_set_filter_min_keys(old)


def _filtered_equals_full_rows():
    for over in (dict(q_len=4096, kv_len=4096, k_sel=256, window=64, n_needles=16),
                 dict(q_len=700, kv_len=6000, k_sel=512, window=128, n_needles=16, batch=2),
                 dict(q_len=1500, kv_len=3000, k_sel=300, window=0, n_q_heads=16, n_kv_heads=4, n_needles=8)):
        inp = make_inputs(scaled("cfg2", **over))
        a = BlockRun(inp).run_full(want_scores=True)
        b = BlockRun(inp).run_full(want_scores=False)
        assert torch.equal(a.idx, b.idx)
        assert hs2.hs2_device_error_flags() == 0


def test_filtered_selection_with_ragged_lengths_offsets_and_an_explicit_scale():
    """The filtered path under per-sequence causal offsets, cache lengths that cut the key range, and a softmax scale
    that is not 1/sqrt(D) (the sweep compares in the accumulator's units, i.e. divides the threshold by it): same
    indices as the selection from complete score rows, which the oracle checks."""
    old = hs2.hs2_set_filter_min_keys(1)
    try:
        wl = scaled("cfg2", batch=3, q_len=600, kv_len=3000, k_sel=128, window=16, n_needles=8)
        inp = make_inputs(wl)
        q_start, kv_lens = [2400, 700, 0], [3000, 1500, 640]
        qs_t = torch.tensor(q_start, dtype=torch.int32, device="cuda")
        kl_t = torch.tensor(kv_lens, dtype=torch.int32, device="cuda")
        q, k, v = inp.q_full.cuda(), inp.k.cuda(), inp.v.cuda()
        for scale in (0.11, 0.023):
            prob = hs2.Problem.from_tensors(q, k, wl.k_sel, wl.window, softmax_scale=scale, q_start=qs_t, kv_lens=kl_t)
            Oa, LSEa, idx_a, sc = hs2.hs2_full_attn_select(prob, q, k, v, want_scores=True)    # complete rows
            Ob, LSEb, idx_b, _ = hs2.hs2_full_attn_select(prob, q, k, v, want_scores=False)    # filtered
            torch.cuda.synchronize()
            assert torch.equal(idx_a, idx_b)
            assert hs2.hs2_device_error_flags() == 0
            rows = [(b, i) for b in range(wl.batch) for i in (0, 1, 17, 300, 598, 599)]
            _, _, idxo, sco = oracle.full_attn_select(inp.q_full, inp.k, inp.v, wl.k_sel, wl.window, scale=scale,
                                                      q_start=q_start, kv_lens=kv_lens, want_scores=True, rows=rows)
            check_idx_against_oracle(gather_rows(idx_b, rows, "bgik").cpu().numpy(), idxo, sco)
    finally:
        hs2.hs2_set_filter_min_keys(old)


def test_filtered_selection_breaks_ties_at_the_threshold_by_key_index():
    """Every key row appears twice (keys 2j and 2j+1 are equal), so every score appears twice and about half of the rows
    have a tied pair straddling the k-th place: the candidate select must keep the lower key of the pair, as the
    selection from complete score rows and the oracle's ordering do."""
    old = hs2.hs2_set_filter_min_keys(1)
    try:
        wl = scaled("cfg2", q_len=1024, kv_len=4096, k_sel=255, window=32, n_needles=4)
        inp = make_inputs(wl)
        inp.k[:, 1::2] = inp.k[:, 0::2]
        a = BlockRun(inp).run_full(want_scores=True)           # complete rows, the same tensor-core scores
        b = BlockRun(inp).run_full(want_scores=False)          # sampled threshold, candidate lists, candidate select
        assert torch.equal(a.idx, b.idx)
        a.check_idx_bitexact_on_gpu_scores(rows=[(0, i) for i in range(0, wl.q_len, 37)])
        # the case really has straddling pairs: rows whose last kept key (by score) has an unkept twin
        sc = a.scores[0, 0]                                    # [Lq, Lk]
        kept = torch.zeros_like(sc, dtype=torch.bool)
        rows = torch.arange(wl.q_len, device="cuda").unsqueeze(1).expand(-1, wl.k_sel)
        kept[rows, a.idx[0, 0].long()] = True
        twins = kept[:, 0::2] != kept[:, 1::2]
        assert int(twins.any(dim=1).sum()) > wl.q_len // 8
        assert bool((kept[:, 0::2] | ~kept[:, 1::2]).all())    # never the higher key of a pair without the lower one
        assert hs2.hs2_device_error_flags() == 0
    finally:
        hs2.hs2_set_filter_min_keys(old)


def test_filtered_selection_redoes_rows_whose_sample_misleads():
    """Scores that depend on the key tile's phase defeat a tile-strided sample: the threshold comes out too
    high (lists shorter than k) or too low (lists overflow).  Those rows must be redone exactly."""
    old = hs2.hs2_set_filter_min_keys(1)
    try:
        _filtered_redo()
    finally:
        hs2.hs2_set_filter_min_keys(old)


def _filtered_redo():
    wl = scaled("cfg2", q_len=2048, kv_len=8192, k_sel=512, window=32, n_needles=4)
    for sampled_high in (True, False):
        inp = make_inputs(wl)
        tile = (torch.arange(wl.kv_len) // 128) % 16 == 0                 # the key tiles the sample looks at
        scale_rows = torch.where(tile == sampled_high, 3.0, 0.05).to(inp.k.dtype)
        # keys of the favoured tiles line up with every query (large logits), the others are near zero
        inp.k.mul_(scale_rows.view(1, -1, 1, 1))
        run = BlockRun(inp)
        n_rows = wl.batch * wl.n_kv_heads * wl.q_len
        from paper_2609_26368_b200 import binding
        ws = torch.zeros(hs2.hs2_workspace_bytes(run.prob, binding.HS2_OP_FULL_ATTN_SELECT), dtype=torch.uint8, device="cuda")
        run.run_full(want_scores=False, ws=ws)
        # white box: the workspace starts with one threshold word and one flag word per row (one block here)
        flags = ws[: 8 * n_rows].view(torch.int32)[n_rows: 2 * n_rows]
        assert int(flags.sum()) > n_rows // 4, "the adversarial rows were not sent to the exact redo"
        rows = [(0, i) for i in (0, 600, 1500, 2047)]
        run.check_full(rows=rows)
        ref = BlockRun(inp).run_full(want_scores=True)
        # Rows that were not redone select from the same tensor-core scores as the strip path: bit-equal.  A redone row
        # is selected from scores recomputed with fp32 FMAs, so it may swap keys whose scores agree to within rounding:
        # every key in the symmetric difference must lie in the near-tie band around the row's k-th score.
        differ = (run.idx != ref.idx).any(-1).reshape(-1)
        assert not bool((differ & (flags == 0)).any()), "a row that was not redone differs from the strip path"
        sc = ref.scores.reshape(n_rows, wl.kv_len)
        for r in torch.nonzero(differ).flatten().tolist()[:256]:
            a, b = run.idx.reshape(n_rows, -1)[r], ref.idx.reshape(n_rows, -1)[r]
            a, b = a[a >= 0], b[b >= 0]
            assert a.numel() == b.numel() and bool((a[1:] > a[:-1]).all())
            tau = sc[r, b.long()].min()
            sym = torch.tensor(sorted(set(a.tolist()) ^ set(b.tolist())), device="cuda")
            assert bool(((sc[r, sym] - tau).abs() <= 1e-3).all()), "row %d: swap outside the near-tie band" % r
    # and ordinary data does not need the redo at all
    inp = make_inputs(wl)
    run = BlockRun(inp)
    ws = torch.zeros(hs2.hs2_workspace_bytes(run.prob, binding.HS2_OP_FULL_ATTN_SELECT), dtype=torch.uint8, device="cuda")
    run.run_full(want_scores=False, ws=ws)
    assert int(ws[: 8 * n_rows].view(torch.int32)[n_rows: 2 * n_rows].sum()) == 0


def test_mma_sync_fallback_kernels_of_the_full_layer():
    """The mma.sync attention and score kernels are what runs when TMA tensor maps cannot be built."""
    old = hs2.hs2_set_tcgen05_enabled(0)
    try:
        for over in (dict(q_len=333, kv_len=333, k_sel=48, window=13, n_needles=8),
                     dict(q_len=200, kv_len=900, k_sel=64, window=16, n_q_heads=8, n_kv_heads=2, n_needles=8, batch=2)):
            wl = scaled("cfg2", **over)
            run = BlockRun(make_inputs(wl)).run_full(want_scores=True)
            run.check_full(check_scores=True)
            run.check_idx_bitexact_on_gpu_scores()
            b = BlockRun(make_inputs(wl)).run_full(want_scores=False)
            assert torch.equal(run.idx, b.idx)
    finally:
        hs2.hs2_set_tcgen05_enabled(old)


def test_full_layer_on_a_cache_larger_than_l2():
    """A cache above 96 MB switches the attention kernel to its head-major CTA order (and chunks the score strips);
    queries at the end of a 50K context, sampled rows against the oracle."""
    wl = scaled("cfg2", q_len=384, kv_len=50176, k_sel=96, window=32, n_needles=8)
    run = BlockRun(make_inputs(wl)).run_full()
    rows = [(0, i) for i in (0, 1, 127, 128, 129, 255, 300, 383)]
    run.check_full(rows=rows)
    out, lse = run.run_sparse(0)
    run.check_sparse(out, lse, 0, rows=rows)


def test_filtered_selection_on_a_context_of_70k_keys():
    """Contexts from 65537 keys on take the filtered selection by default; between 65537 and about 90000 keys its
    candidate select needs the opt-in to more than 48 KB of shared memory for static plus dynamic together."""
    wl = scaled("cfg2", q_len=512, kv_len=70016, k_sel=1024, window=64, n_needles=8)
    run = BlockRun(make_inputs(wl)).run_full()
    rows = [(0, i) for i in (0, 1, 255, 256, 511)]
    run.check_full(rows=rows)
    ref = BlockRun(run.inp).run_full(want_scores=True)
    assert torch.equal(run.idx, ref.idx)
    assert hs2.hs2_device_error_flags() == 0


def test_paper_native_shape_mqa64_dim256_with_sink():
    """The attention shape of the paper's own model (Table 1: 64 query heads / 1 KV head, head dim 256,
    128 forced local + 1024 global tokens, per-head sink bias in the sparse layers), scaled in length."""
    wl = scaled("cfg2", q_len=1536, kv_len=1536, n_q_heads=64, n_kv_heads=1, head_dim=256, k_sel=1024, window=128,
                n_needles=8)
    run = BlockRun(make_inputs(wl)).run_full()
    rows = [(0, i) for i in (0, 127, 128, 1151, 1152, 1300, 1535)]
    run.check_full(rows=rows)
    sink = torch.linspace(-2.0, 2.0, 64, device="cuda")
    out, lse = run.run_sparse(0, sink=sink)
    run.check_sparse(out, lse, 0, rows=rows, sink=sink)
    q1 = run.qs[0][:, -1:].contiguous()
    prob1 = hs2.Problem.from_tensors(q1, run.k, wl.k_sel, wl.window)
    od, ld = hs2.hs2_sparse_attn_decode(prob1, q1, run.k, run.v, run.idx[:, :, -1:].contiguous(), sink=sink, want_lse=True)
    torch.cuda.synchronize()
    run.check_decode(od, ld, 0, sink=sink)


def test_tcgen05_sparse_kernel_large_head_groups():
    """Groups of more than 8 heads take the tensor-core gather kernel: odd group sizes, both head dims, ragged
    lengths, sink, several KV heads; every row against the oracle and against the SIMT kernel."""
    cases = [
        dict(q_len=90, kv_len=500, k_sel=100, window=20, n_q_heads=96, n_kv_heads=2, head_dim=256, batch=2),   # G = 48
        dict(q_len=70, kv_len=330, k_sel=64, window=64, n_q_heads=128, n_kv_heads=1, head_dim=128),            # G = 128
        dict(q_len=150, kv_len=150, k_sel=7, window=3, n_q_heads=24, n_kv_heads=2, head_dim=128),              # one ragged tile
        dict(q_len=64, kv_len=400, k_sel=0, window=130, n_q_heads=64, n_kv_heads=1, head_dim=256),             # window only
    ]
    for over in cases:
        wl = scaled("cfg2", n_needles=4, **over)
        run = BlockRun(make_inputs(wl)).run_full()
        sink = torch.linspace(-1.5, 2.5, wl.n_q_heads, device="cuda")
        for sk in (None, sink):
            out, lse = run.run_sparse(0, sink=sk)
            run.check_sparse(out, lse, 0, sink=sk)
            old = hs2.hs2_set_tcgen05_enabled(0)
            try:
                out_g, lse_g = run.run_sparse(0, sink=sk)
            finally:
                hs2.hs2_set_tcgen05_enabled(old)
            assert (out.float() - out_g.float()).abs().max().item() <= 2e-2
            fin = torch.isfinite(lse_g)
            assert torch.equal(torch.isfinite(lse), fin)
            assert (lse[fin] - lse_g[fin]).abs().max().item() <= 2e-3
            # decode of the last position: few queries, so the keys of a query are split over CTAs and combined
            q1 = run.qs[0][:, -1:].contiguous()
            prob1 = hs2.Problem.from_tensors(q1, run.k, wl.k_sel, wl.window)
            assert hs2.hs2_workspace_bytes(prob1, hs2.binding.HS2_OP_SPARSE_ATTN_DECODE) > 0 or wl.k_sel + wl.window <= 64
            od, ld = hs2.hs2_sparse_attn_decode(prob1, q1, run.k, run.v, run.idx[:, :, -1:].contiguous(), sink=sk,
                                                want_lse=True)
            torch.cuda.synchronize()
            run.check_decode(od, ld, 0, sink=sk)
    assert hs2.hs2_device_error_flags() == 0


def test_sigmoid_output_gate_in_every_sparse_kernel_family():
    """The gated entry points (Section 4.1: sigmoid output gates in the sparse layers) against the oracle: SIMT fp32,
    mma.sync (group of 8), tcgen05 (group of 64, head_dim 256), prefill and decode (split and unsplit)."""
    cases = [
        ("cfg1", dict(q_len=80, kv_len=200, k_sel=20, window=6)),
        ("cfg2", dict(q_len=120, kv_len=500, k_sel=64, window=16, n_needles=4, batch=2)),
        ("cfg2", dict(q_len=70, kv_len=400, k_sel=100, window=28, n_q_heads=64, n_kv_heads=1, head_dim=256, n_needles=4)),
    ]
    for name, over in cases:
        wl = scaled(name, **over)
        run = BlockRun(make_inputs(wl)).run_full()
        g = torch.Generator(device="cuda").manual_seed(11)
        gate = (torch.randn(run.qs[0].shape, device="cuda", generator=g) * 2.5).to(run.qs[0].dtype)
        sink = torch.linspace(-1.0, 1.0, wl.n_q_heads, device="cuda")
        out0, lse0 = run.run_sparse(0, sink=sink)
        out, lse = run.run_sparse(0, sink=sink, gate=gate)
        run.check_sparse(out, lse, 0, sink=sink, gate=gate)
        assert torch.equal(lse, lse0)                     # the gate leaves LSE alone
        # decode of the last position, gated
        q1 = run.qs[0][:, -1:].contiguous()
        g1 = gate[:, -1:].contiguous()
        prob1 = hs2.Problem.from_tensors(q1, run.k, wl.k_sel, wl.window)
        od, ld = hs2.hs2_sparse_attn_decode(prob1, q1, run.k, run.v, run.idx[:, :, -1:].contiguous(), sink=sink, gate=g1,
                                            want_lse=True)
        torch.cuda.synchronize()
        run.check_decode(od, ld, 0, sink=sink, gate=gate)
    with pytest.raises(hs2.HS2Error):                     # the gated call needs a gate
        lib = hs2.load_library()
        c = run.prob.c_struct(run.qs[0], run.k, out)
        import ctypes as C
        st = lib.hs2_sparse_attn_prefill_gated(C.byref(c), run.qs[0].data_ptr(), run.k.data_ptr(), run.v.data_ptr(),
                                               run.idx.data_ptr(), None, None, out.data_ptr(), None, None, 0, None)
        if st != 0:
            raise hs2.HS2Error(st, "hs2_sparse_attn_prefill_gated")
    assert hs2.hs2_device_error_flags() == 0


def test_fp8_kv_cache_sparse_prefill_and_decode():
    """Sparse attention on an e4m3 KV cache (codes + per-(token, KV head) scales) against the oracle run on the
    dequantised cache: groups of 8, 4 and 1, ragged lengths, sink, a strided (fused K|V) cache, prefill and decode."""
    from gen.workloads import quantize_kv_e4m3
    cases = [
        dict(q_len=150, kv_len=600, k_sel=100, window=24, batch=2),
        dict(q_len=64, kv_len=300, k_sel=37, window=5, n_q_heads=8, n_kv_heads=2),
        dict(q_len=40, kv_len=200, k_sel=0, window=50, n_q_heads=4, n_kv_heads=4),
        dict(q_len=48, kv_len=260, k_sel=40, window=12, n_q_heads=32, n_kv_heads=2),     # groups of 16: two sub-groups of 8
    ]
    for ci, over in enumerate(cases):
        wl = scaled("cfg2", n_needles=4, **over)
        inp = make_inputs(wl)
        run = BlockRun(inp).run_full()               # indices from the bf16 full layer
        B, Lk, Hkv, D = inp.k.shape
        k8, ksc = quantize_kv_e4m3(run.k)
        v8, vsc = quantize_kv_e4m3(run.v)
        if ci == 0:                                  # K and V as slices of one fused cache
            fused = torch.empty(B, Lk, 2, Hkv, D, dtype=torch.uint8, device="cuda")
            fused[:, :, 0].copy_(k8)
            fused[:, :, 1].copy_(v8)
            k8, v8 = fused[:, :, 0], fused[:, :, 1]
        kv_lens = [Lk - 7 * b for b in range(wl.batch)]
        kl_t = torch.tensor(kv_lens, dtype=torch.int32, device="cuda")
        q = run.qs[0]
        prob = hs2.Problem.from_tensors(q, k8, wl.k_sel, wl.window, kv_lens=kl_t)
        sink = torch.linspace(-1.0, 1.5, wl.n_q_heads, device="cuda")
        kd = oracle.dequant_e4m3(k8.contiguous(), ksc)
        vd = oracle.dequant_e4m3(v8.contiguous(), vsc)
        idx_rows = run.idx.permute(0, 2, 1, 3).reshape(B * wl.q_len, Hkv, wl.k_sel).cpu().numpy()
        for sk in (None, sink):
            out, lse = hs2.hs2_sparse_attn_prefill_fp8kv(prob, q, k8, v8, ksc, vsc, run.idx, sink=sk, want_lse=True)
            torch.cuda.synchronize()
            Oo, LSEo, _ = oracle.sparse_attn(q.float().cpu().numpy(), kd, vd, idx_rows, wl.window, kv_lens=kv_lens,
                                             sink=None if sk is None else sk.cpu().numpy().astype(np.float64))
            assert_output_close(out.reshape(-1, wl.n_q_heads, D), Oo, wl.torch_dtype, "fp8 sparse O")
            l = lse.permute(0, 2, 1).reshape(B * wl.q_len, wl.n_q_heads).cpu().numpy()
            fin = np.isfinite(LSEo)
            assert np.array_equal(np.isfinite(l), fin) and np.abs(l[fin] - LSEo[fin]).max() <= TOL[wl.torch_dtype]["lse"]
            q1 = q[:, -1:].contiguous()
            prob1 = hs2.Problem.from_tensors(q1, k8, wl.k_sel, wl.window, kv_lens=kl_t)
            od, ld = hs2.hs2_sparse_attn_decode_fp8kv(prob1, q1, k8, v8, ksc, vsc, run.idx[:, :, -1:].contiguous(), sink=sk,
                                                      want_lse=True)
            torch.cuda.synchronize()
            last = [b * wl.q_len + wl.q_len - 1 for b in range(B)]          # the oracle's rows of the decode position
            assert_output_close(od[:, 0], Oo[last], wl.torch_dtype, "fp8 sparse decode O")
            ldh = ld[:, :, 0].cpu().numpy()
            assert np.abs(ldh - LSEo[last]).max() <= TOL[wl.torch_dtype]["lse"]
    # shapes the FP8 kernels do not cover are refused, not mis-computed
    wl = scaled("cfg2", q_len=16, kv_len=64, k_sel=8, window=4, n_q_heads=4, n_kv_heads=1, head_dim=64, n_needles=4)
    inp = make_inputs(wl, "cuda")
    k8, ksc = quantize_kv_e4m3(inp.k)
    prob = hs2.Problem.from_tensors(inp.q_full, k8, wl.k_sel, wl.window)
    idx = torch.zeros(1, 1, 16, 8, dtype=torch.int32, device="cuda")
    with pytest.raises(hs2.HS2Error):
        hs2.hs2_sparse_attn_prefill_fp8kv(prob, inp.q_full, k8, k8, ksc, ksc, idx)


def _fp8_records(k8, v8, ksc, vsc):
    """One record per (token, KV head): [K codes | V codes | K scale | V scale | pad to 32 bytes]; returns views."""
    B, Lk, Hkv, D = k8.shape
    rec_bytes = (2 * D + 8 + 31) // 32 * 32
    rec = torch.zeros(B, Lk, Hkv, rec_bytes, dtype=torch.uint8, device=k8.device)
    rec[..., :D].copy_(k8)
    rec[..., D:2 * D].copy_(v8)
    recf = rec.view(torch.float32)                       # [B, Lk, Hkv, rec_bytes / 4]
    recf[..., 2 * D // 4].copy_(ksc)
    recf[..., 2 * D // 4 + 1].copy_(vsc)
    return rec[..., :D], rec[..., D:2 * D], recf[..., 2 * D // 4], recf[..., 2 * D // 4 + 1]


def test_fp8_cache_as_one_record_per_token_and_head():
    """K codes, V codes and both scales of a (token, KV head) in one record (kv_stride and kv_scale_stride describe it):
    every FP8 entry point gives bit for bit what it gives on four separate packed arrays, which the tests above hold
    against the oracle."""
    from gen.workloads import quantize_kv_e4m3
    cases = [
        dict(q_len=130, kv_len=700, k_sel=96, window=24, batch=2),                                        # mma.sync kernels, group of 8
        dict(q_len=100, kv_len=520, k_sel=64, window=16, n_q_heads=64, n_kv_heads=4),                     # group of 16: two sub-groups
        dict(q_len=96, kv_len=448, k_sel=80, window=32, n_q_heads=64, n_kv_heads=1, head_dim=256),       # tcgen05 gather kernel
        dict(q_len=80, kv_len=400, k_sel=50, window=10, n_q_heads=48, n_kv_heads=2, head_dim=128, batch=2),
    ]
    for over in cases:
        wl = scaled("cfg2", n_needles=4, **over)
        inp = make_inputs(wl)
        run = BlockRun(inp).run_full()
        k8, ksc = quantize_kv_e4m3(run.k)
        v8, vsc = quantize_kv_e4m3(run.v)
        rk, rv, rks, rvs = _fp8_records(k8, v8, ksc, vsc)
        assert not rks.is_contiguous() and rk.stride() == rv.stride()
        q = run.qs[0]
        prob = hs2.Problem.from_tensors(q, k8, wl.k_sel, wl.window)
        a, la = hs2.hs2_sparse_attn_prefill_fp8kv(prob, q, k8, v8, ksc, vsc, run.idx, want_lse=True)
        b, lb = hs2.hs2_sparse_attn_prefill_fp8kv(prob, q, rk, rv, rks, rvs, run.idx, want_lse=True)
        torch.cuda.synchronize()
        assert torch.equal(a, b) and torch.equal(la, lb)
        q1 = q[:, -1:].contiguous()
        idx1 = run.idx[:, :, -1:].contiguous()
        prob1 = hs2.Problem.from_tensors(q1, k8, wl.k_sel, wl.window)
        a, la = hs2.hs2_sparse_attn_decode_fp8kv(prob1, q1, k8, v8, ksc, vsc, idx1, want_lse=True)
        b, lb = hs2.hs2_sparse_attn_decode_fp8kv(prob1, q1, rk, rv, rks, rvs, idx1, want_lse=True)
        torch.cuda.synchronize()
        assert_output_close(b[:, 0].float(), a[:, 0].double().cpu().numpy(), wl.torch_dtype, "record layout, decode O")
        assert float((la - lb).abs().max()) <= 1e-5      # (the splits of a decode step may merge in another order)
        qf = run.q[:, -1:].contiguous()
        Oa, La, ia = hs2.hs2_full_attn_select_fp8kv(prob1, qf, k8, v8, ksc, vsc)
        Ob, Lb, ib = hs2.hs2_full_attn_select_fp8kv(prob1, qf, rk, rv, rks, rvs)
        torch.cuda.synchronize()
        assert torch.equal(ia, ib)
        assert_output_close(Ob[:, 0].float(), Oa[:, 0].double().cpu().numpy(), wl.torch_dtype, "record layout, full-layer decode O")
        assert hs2.hs2_device_error_flags() == 0


def test_fp8_kv_cache_on_large_head_groups_and_head_dim_256():
    """The e4m3 cache at the paper's own attention shape (Table 1: 64 query heads on one KV head, head_dim 256; the cost
    analysis of Section 4 assumes FP8 storage) and on other shapes of the tensor-core gather kernel, which dequantises
    while it gathers: prefill every row and the decode step against the oracle on the dequantised cache."""
    from gen.workloads import quantize_kv_e4m3
    cases = [
        dict(q_len=192, kv_len=640, k_sel=128, window=32, n_q_heads=64, n_kv_heads=1, head_dim=256),            # the paper's shape
        dict(q_len=90, kv_len=500, k_sel=100, window=20, n_q_heads=96, n_kv_heads=2, head_dim=256, batch=2),    # G = 48, two KV heads
        dict(q_len=150, kv_len=330, k_sel=64, window=64, n_q_heads=24, n_kv_heads=2, head_dim=128),             # G = 12, head_dim 128
        dict(q_len=64, kv_len=400, k_sel=0, window=130, n_q_heads=128, n_kv_heads=1, head_dim=128),             # window only, two sub-groups
        dict(q_len=70, kv_len=300, k_sel=37, window=9, n_q_heads=8, n_kv_heads=2, head_dim=256),                # small group at head_dim 256
    ]
    for over in cases:
        wl = scaled("cfg2", n_needles=4, **over)
        inp = make_inputs(wl)
        run = BlockRun(inp).run_full()               # indices from the bf16 full layer
        B, Lk, Hkv, D = inp.k.shape
        k8, ksc = quantize_kv_e4m3(run.k)
        v8, vsc = quantize_kv_e4m3(run.v)
        kv_lens = [Lk - 11 * b for b in range(wl.batch)]
        kl_t = torch.tensor(kv_lens, dtype=torch.int32, device="cuda")
        q = run.qs[0]
        prob = hs2.Problem.from_tensors(q, k8, wl.k_sel, wl.window, kv_lens=kl_t)
        sink = torch.linspace(-1.0, 1.5, wl.n_q_heads, device="cuda")
        kd = oracle.dequant_e4m3(k8, ksc)
        vd = oracle.dequant_e4m3(v8, vsc)
        idx_rows = run.idx.permute(0, 2, 1, 3).reshape(B * wl.q_len, Hkv, wl.k_sel).cpu().numpy()
        for sk in (None, sink):
            out, lse = hs2.hs2_sparse_attn_prefill_fp8kv(prob, q, k8, v8, ksc, vsc, run.idx, sink=sk, want_lse=True)
            torch.cuda.synchronize()
            Oo, LSEo, _ = oracle.sparse_attn(q.float().cpu().numpy(), kd, vd, idx_rows, wl.window, kv_lens=kv_lens,
                                             sink=None if sk is None else sk.cpu().numpy().astype(np.float64))
            assert_output_close(out.reshape(-1, wl.n_q_heads, D), Oo, wl.torch_dtype, "fp8 sparse O (tensor-core gather)")
            l = lse.permute(0, 2, 1).reshape(B * wl.q_len, wl.n_q_heads).cpu().numpy()
            fin = np.isfinite(LSEo)
            assert np.array_equal(np.isfinite(l), fin) and np.abs(l[fin] - LSEo[fin]).max() <= TOL[wl.torch_dtype]["lse"]
            q1 = q[:, -1:].contiguous()
            prob1 = hs2.Problem.from_tensors(q1, k8, wl.k_sel, wl.window, kv_lens=kl_t)
            od, ld = hs2.hs2_sparse_attn_decode_fp8kv(prob1, q1, k8, v8, ksc, vsc, run.idx[:, :, -1:].contiguous(), sink=sk,
                                                      want_lse=True)
            torch.cuda.synchronize()
            last = [b * wl.q_len + wl.q_len - 1 for b in range(B)]
            assert_output_close(od[:, 0], Oo[last], wl.torch_dtype, "fp8 sparse decode O (tensor-core gather)")
            assert np.abs(ld[:, :, 0].cpu().numpy() - LSEo[last]).max() <= TOL[wl.torch_dtype]["lse"]
    assert hs2.hs2_device_error_flags() == 0


def test_fp8_kv_cache_full_layer_decode_step():
    """The full-attention layer's decode step on the e4m3 cache: O, LSE and the selected indices against the oracle
    run on the dequantised cache (groups of 8, 4 and 1, ragged lengths, a strided cache, several key tiles per warp;
    then the paper's own shape - 64 heads on one KV head, head_dim 256 - and other large groups, which take the
    tensor-core gather kernel for the attention and a second pass over the K codes for the scores)."""
    from gen.workloads import quantize_kv_e4m3
    cases = [
        dict(kv_len=3000, k_sel=200, window=32, batch=3),
        dict(kv_len=700, k_sel=64, window=16, n_q_heads=8, n_kv_heads=2, batch=2),
        dict(kv_len=450, k_sel=100, window=0, n_q_heads=4, n_kv_heads=4, batch=1),
        dict(kv_len=2100, k_sel=256, window=32, n_q_heads=64, n_kv_heads=1, head_dim=256, batch=3),
        dict(kv_len=900, k_sel=100, window=16, n_q_heads=24, n_kv_heads=2, head_dim=128, batch=2),      # G = 12: padded n-tile
        dict(kv_len=640, k_sel=64, window=0, n_q_heads=128, n_kv_heads=1, head_dim=128, batch=1),
    ]
    for ci, over in enumerate(cases):
        wl = scaled("cfg5", q_len=1, n_needles=6, **over)
        inp = make_inputs(wl, "cuda")
        B, Lk, Hkv, D = inp.k.shape
        k8, ksc = quantize_kv_e4m3(inp.k)
        v8, vsc = quantize_kv_e4m3(inp.v)
        if ci == 0:                                  # K and V as slices of one fused cache
            fused = torch.empty(B, Lk, 2, Hkv, D, dtype=torch.uint8, device="cuda")
            fused[:, :, 0].copy_(k8)
            fused[:, :, 1].copy_(v8)
            k8, v8 = fused[:, :, 0], fused[:, :, 1]
        kv_lens = [Lk - 11 * b for b in range(wl.batch)]
        kl_t = torch.tensor(kv_lens, dtype=torch.int32, device="cuda")
        q = inp.q_full
        prob = hs2.Problem.from_tensors(q, k8, wl.k_sel, wl.window, kv_lens=kl_t)
        O, LSE, idx = hs2.hs2_full_attn_select_fp8kv(prob, q, k8, v8, ksc, vsc)
        torch.cuda.synchronize()
        kd = torch.from_numpy(oracle.dequant_e4m3(k8.contiguous(), ksc))
        vd = torch.from_numpy(oracle.dequant_e4m3(v8.contiguous(), vsc))
        rows = rows_all(B, 1)
        Oo, LSEo, idxo, sco = oracle.full_attn_select(q.float().cpu(), kd, vd, wl.k_sel, wl.window, rows=rows,
                                                      want_scores=True, kv_lens=kv_lens)
        assert_output_close(O.reshape(-1, wl.n_q_heads, D), Oo, wl.torch_dtype, "fp8 full attention O")
        l = LSE.permute(0, 2, 1).reshape(B, wl.n_q_heads).cpu().numpy().astype(np.float64)
        assert np.abs(l - LSEo).max() <= TOL[wl.torch_dtype]["lse"]
        check_idx_against_oracle(idx.permute(0, 2, 1, 3).reshape(B, Hkv, wl.k_sel).cpu().numpy(), idxo, sco)
        # attention only: no scratch, same O
        O2, _, none = hs2.hs2_full_attn_select_fp8kv(prob, q, k8, v8, ksc, vsc, want_idx=False)
        assert none is None and torch.equal(O, O2)
    # more than one query per sequence is refused
    wl = scaled("cfg2", q_len=4, kv_len=64, k_sel=8, window=4, n_needles=4)
    inp = make_inputs(wl, "cuda")
    k8, ksc = quantize_kv_e4m3(inp.k)
    prob = hs2.Problem.from_tensors(inp.q_full, k8, wl.k_sel, wl.window)
    with pytest.raises(hs2.HS2Error):
        hs2.hs2_full_attn_select_fp8kv(prob, inp.q_full, k8, k8, ksc, ksc)


def test_block_level_selection_variant():
    """select_block = B (Section 5, Ablation 1: blocks of 64, 16 blocks) against the oracle: bit-exact on the GPU's
    own fp32 scores, through hs2_topk_select on given scores (ties, partial last blocks, ragged lengths), and the
    sparse layer consuming the block-structured index rows."""
    rng = np.random.default_rng(3)
    B_, Hkv, Lq, Lk, w = 2, 2, 50, 700, 9
    sc = torch.tensor(np.round(rng.normal(size=(B_, Hkv, Lq, Lk)) * 4) / 4, dtype=torch.float32, device="cuda")
    qs = torch.tensor([600, 37], dtype=torch.int32, device="cuda")
    kl = torch.tensor([700, 90], dtype=torch.int32, device="cuda")
    for blk, k in ((64, 256), (16, 48), (4, 64), (4, 512), (1, 30)):     # (4, 512): more than 64 blocks per row
        prob = hs2.Problem(B_, Lq, Lk, 4, Hkv, 64, k, w, q_start=qs, kv_lens=kl, select_block=blk)
        idx = hs2.hs2_topk_select(prob, sc)
        torch.cuda.synchronize()
        for b in range(B_):
            pos = qs[b].item() + np.arange(Lq)
            for g in range(Hkv):
                want = oracle.select_blocks(sc[b, g].cpu().numpy(), pos, kl[b].item(), w, k, blk)
                assert np.array_equal(idx[b, g].cpu().numpy(), want), (blk, b, g)
    with pytest.raises(hs2.HS2Error):      # k must be a whole number of blocks
        hs2.hs2_topk_select(hs2.Problem(B_, Lq, Lk, 4, Hkv, 64, 100, w, select_block=64), sc)
    # the full layer in block mode, then a sparse layer on its indices
    wl = scaled("cfg2", q_len=300, kv_len=900, k_sel=256, window=32, n_needles=8)
    inp = make_inputs(wl, "cuda")
    prob = hs2.Problem.from_tensors(inp.q_full, inp.k, wl.k_sel, wl.window, select_block=64)
    O, LSE, idx, scores = hs2.hs2_full_attn_select(prob, inp.q_full, inp.k, inp.v, want_scores=True)
    idx2 = hs2.hs2_full_attn_select(prob, inp.q_full, inp.k, inp.v)[2]      # strip path
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2)
    pos = wl.kv_len - wl.q_len + np.arange(wl.q_len)
    for g in range(wl.n_kv_heads):
        want = oracle.select_blocks(scores[0, g].cpu().numpy(), pos, wl.kv_len, wl.window, wl.k_sel, 64)
        assert np.array_equal(idx[0, g].cpu().numpy(), want)
    out, _ = hs2.hs2_sparse_attn_prefill(prob, inp.q_sparse[0], inp.k, inp.v, idx)
    torch.cuda.synchronize()
    idx_rows = idx.permute(0, 2, 1, 3).reshape(wl.q_len, wl.n_kv_heads, wl.k_sel).cpu().numpy()
    Oo, _, _ = oracle.sparse_attn(to_host(inp.q_sparse[0]), to_host(inp.k), to_host(inp.v), idx_rows, wl.window)
    assert_output_close(out.reshape(-1, wl.n_q_heads, wl.head_dim), Oo, wl.torch_dtype, "sparse O on block indices")


def test_kv_projection_bf16_and_fp8_outputs():
    """The cache producer C = H W^T (Section 3.2, KV Bridging) against the fp64 product: bf16 output into a slice of a
    fused cache, and e4m3 codes + scales within the format's rounding bound; the FP8 caches it writes are then read
    by the FP8 sparse kernel."""
    g = torch.Generator(device="cuda").manual_seed(4)
    T, dm, Hkv, D = 300, 320, 2, 128
    N = 2 * Hkv * D                                         # K and V of one layer side by side
    h = (torch.randn(T, dm, device="cuda", generator=g)).to(torch.bfloat16)
    w = (torch.randn(N, dm, device="cuda", generator=g) / dm ** 0.5).to(torch.bfloat16)
    want = oracle.kv_project(h.cpu(), w.cpu())
    fused = torch.zeros(T, N + 64, dtype=torch.bfloat16, device="cuda")      # a wider row: strided output
    out = hs2.hs2_kv_project(h, w, out=fused[:, :N])
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-5)
    assert torch.count_nonzero(fused[:, N:]) == 0
    c8, sc = hs2.hs2_kv_project(h, w, fp8=True)
    torch.cuda.synchronize()
    amax = np.abs(want).reshape(T, N // 128, 128).max(axis=2)
    s_np = sc.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(s_np - amax / 448.0) <= 1e-4 * amax / 448.0 + 1e-12)
    deq = oracle.dequant_e4m3(c8.cpu().numpy().reshape(T, N // 128, 128), s_np).astype(np.float64).reshape(T, N)
    assert not np.isnan(deq).any()
    s_full = np.repeat(s_np, 128, axis=1)
    bound = np.maximum(np.abs(want) * 2.0 ** -4, s_full * 2.0 ** -10) * 1.01 + 1e-5
    assert np.all(np.abs(deq - want) <= bound)
    # the produced FP8 caches through the FP8 sparse kernel: [1, T, Hkv, D] K and V are column halves of the output
    k8, v8 = c8[:, :Hkv * D].reshape(1, T, Hkv, D), c8[:, Hkv * D:].reshape(1, T, Hkv, D)
    ksc, vsc = sc[:, :Hkv].reshape(1, T, Hkv).contiguous(), sc[:, Hkv:].reshape(1, T, Hkv).contiguous()
    Lq, k_sel, win = 40, 32, 8
    q = torch.randn(1, Lq, 8 * Hkv, D, device="cuda", generator=g).to(torch.bfloat16)
    idx = torch.stack([torch.sort(torch.randperm(T - Lq - win, device="cuda", generator=g)[:k_sel]).values
                       for _ in range(Hkv * Lq)]).to(torch.int32).reshape(1, Hkv, Lq, k_sel).contiguous()
    prob = hs2.Problem.from_tensors(q, k8, k_sel, win)
    o8, _ = hs2.hs2_sparse_attn_prefill_fp8kv(prob, q, k8, v8, ksc, vsc, idx)
    torch.cuda.synchronize()
    kd = oracle.dequant_e4m3(k8.contiguous(), ksc)
    vd = oracle.dequant_e4m3(v8.contiguous(), vsc)
    Oo, _, _ = oracle.sparse_attn(q.float().cpu().numpy(), kd, vd, idx.permute(0, 2, 1, 3).reshape(Lq, Hkv, k_sel).cpu().numpy(), win)
    assert_output_close(o8.reshape(-1, 8 * Hkv, D), Oo, torch.bfloat16, "sparse O on the projected FP8 cache")
    # the same projections written straight into a cache of records [K codes | V codes | K scale | V scale | spare] per
    # (token, KV head): same codes, same scales, and the sparse kernel reads the records through strides
    rec = torch.zeros(1, T, Hkv, 272, dtype=torch.uint8, device="cuda")
    recf = rec.view(torch.float32)
    wk, wv = w[:Hkv * D], w[Hkv * D:]
    hs2.hs2_kv_project_fp8_records(h, wk, rec[0, :, :, :D], recf[0, :, :, 64])
    hs2.hs2_kv_project_fp8_records(h, wv, rec[0, :, :, D:2 * D], recf[0, :, :, 65])
    torch.cuda.synchronize()
    assert torch.equal(rec[..., :D], k8) and torch.equal(rec[..., D:2 * D], v8)
    assert torch.equal(recf[..., 64], ksc) and torch.equal(recf[..., 65], vsc)
    assert torch.count_nonzero(rec[..., 264:]) == 0
    o8r, _ = hs2.hs2_sparse_attn_prefill_fp8kv(prob, q, rec[..., :D], rec[..., D:2 * D], recf[..., 64], recf[..., 65], idx)
    torch.cuda.synchronize()
    assert torch.equal(o8r, o8)
    with pytest.raises(hs2.HS2Error):                       # a group stride below the 128 bytes of a group
        bad = torch.zeros(T, Hkv, 128, dtype=torch.uint8, device="cuda")
        hs2.hs2_kv_project_fp8_records(h, wk, bad.as_strided((T, Hkv, 128), (Hkv * 128, 64, 1)), recf[0, :, :, 64])
    with pytest.raises(hs2.HS2Error):                       # n_out must be a multiple of 256
        hs2.hs2_kv_project(h, w[:128])
    # more shapes of the CTA-pair kernel: a single tile with one row, ragged token counts across several 256-row tiles,
    # one and many k-blocks, more tiles than CTA pairs
    for T2, dm2, N2 in [(1, 64, 256), (257, 64, 256), (777, 128, 768), (1300, 2048, 512), (40000, 64, 512)]:
        h2 = (torch.randn(T2, dm2, device="cuda", generator=g)).to(torch.bfloat16)
        w2 = (torch.randn(N2, dm2, device="cuda", generator=g) / dm2 ** 0.5).to(torch.bfloat16)
        got2 = hs2.hs2_kv_project(h2, w2).float()
        torch.cuda.synchronize()
        want2 = h2.double() @ w2.double().T                 # (the oracle's product, on the device for the large case)
        assert bool(((got2.double() - want2).abs() <= want2.abs() * 2.0 ** -8 + 1e-5).all()), (T2, dm2, N2)
    assert hs2.hs2_device_error_flags() == 0


def test_union_mode_selection_is_the_full_layer_with_window_zero():
    """The alternative reading of the budget (k counted over all visible tokens, window included): select with
    window 0, attend with window w.  Selected tokens that fall inside the window are ignored by the sparse kernels
    (they are covered by the window slots), exactly as the oracle's set semantics say."""
    wl = scaled("cfg2", q_len=200, kv_len=500, k_sel=64, window=24, n_needles=8)
    inp = make_inputs(wl, "cuda")
    prob_sel = hs2.Problem.from_tensors(inp.q_full, inp.k, wl.k_sel, 0)
    prob_att = hs2.Problem.from_tensors(inp.q_full, inp.k, wl.k_sel, wl.window)
    _, _, idx, scores = hs2.hs2_full_attn_select(prob_sel, inp.q_full, inp.k, inp.v, want_scores=True)
    out, _ = hs2.hs2_sparse_attn_prefill(prob_att, inp.q_sparse[0], inp.k, inp.v, idx)
    torch.cuda.synchronize()
    pos = wl.kv_len - wl.q_len + np.arange(wl.q_len)
    for g in range(wl.n_kv_heads):       # bit-exact on the GPU's own scores, window 0: every visible key is a candidate
        assert np.array_equal(idx[0, g].cpu().numpy(), oracle.select(scores[0, g].cpu().numpy(), pos, wl.kv_len, 0, wl.k_sel))
    assert (idx[0, :, -1] > wl.kv_len - 1 - wl.window).any()      # some selected tokens do sit inside the window
    idx_rows = idx.permute(0, 2, 1, 3).reshape(wl.q_len, wl.n_kv_heads, wl.k_sel).cpu().numpy()
    Oo, _, member = oracle.sparse_attn(to_host(inp.q_sparse[0]), to_host(inp.k), to_host(inp.v), idx_rows, wl.window,
                                       want_member=True)
    assert_output_close(out.reshape(-1, wl.n_q_heads, wl.head_dim), Oo, wl.torch_dtype, "union-mode sparse O")
    assert member.sum(axis=2).max() <= wl.k_sel + wl.window


def test_ragged_lengths_offsets_strides_and_sink():
    wl = scaled("cfg2", batch=3, q_len=70, kv_len=400, k_sel=40, window=12, n_needles=4)
    inp = make_inputs(wl)
    dev = "cuda"
    q_start, kv_lens = [330, 100, 0], [400, 250, 64]
    qs_t = torch.tensor(q_start, dtype=torch.int32, device=dev)
    kl_t = torch.tensor(kv_lens, dtype=torch.int32, device=dev)
    # non-packed views: Q inside a wider buffer, K/V as slices of a fused [.., 2, Hkv, D] cache
    B, Lq, Hq, D = inp.q_full.shape
    qbuf = torch.zeros(B, Lq, Hq + 3, D + 8, dtype=inp.q_full.dtype, device=dev)
    q = qbuf[:, :, 1:1 + Hq, :D]
    q.copy_(inp.q_full)
    kvbuf = torch.zeros(B, wl.kv_len, 2, wl.n_kv_heads, D, dtype=inp.k.dtype, device=dev)
    kvbuf[:, :, 0].copy_(inp.k)
    kvbuf[:, :, 1].copy_(inp.v)
    k, v = kvbuf[:, :, 0], kvbuf[:, :, 1]
    prob = hs2.Problem.from_tensors(q, k, wl.k_sel, wl.window, softmax_scale=0.11, q_start=qs_t, kv_lens=kl_t)
    O, LSE, idx, sc = hs2.hs2_full_attn_select(prob, q, k, v, want_scores=True)
    torch.cuda.synchronize()
    Oo, LSEo, idxo, sco = oracle.full_attn_select(inp.q_full, inp.k, inp.v, wl.k_sel, wl.window, scale=0.11,
                                                  q_start=q_start, kv_lens=kv_lens, want_scores=True)
    dt = wl.torch_dtype
    assert_output_close(O.reshape(-1, Hq, D), Oo, dt, "full O")
    from parity import check_idx_against_oracle
    idx_rows = idx.permute(0, 2, 1, 3).reshape(B * Lq, wl.n_kv_heads, wl.k_sel).cpu().numpy()
    check_idx_against_oracle(idx_rows, idxo, sco)
    sink = torch.linspace(-1.0, 2.0, Hq, device=dev)
    qsp = inp.q_sparse[0].to(dev)
    for fn_sink in (None, sink):
        out, lse = hs2.hs2_sparse_attn_prefill(prob, qsp, k, v, idx, sink=fn_sink, want_lse=True)
        torch.cuda.synchronize()
        Os, LSEs, _ = oracle.sparse_attn(inp.q_sparse[0], inp.k, inp.v, idx_rows, wl.window, scale=0.11,
                                         q_start=q_start, kv_lens=kv_lens,
                                         sink=None if fn_sink is None else fn_sink.cpu().numpy())
        assert_output_close(out.reshape(-1, Hq, D), Os, dt, "sparse O")
        l = lse.permute(0, 2, 1).reshape(B * Lq, Hq).cpu().numpy()
        fin = np.isfinite(LSEs)
        assert np.array_equal(np.isfinite(l), fin)
        assert np.abs(l[fin] - LSEs[fin]).max() <= TOL[dt]["lse"]


def _close_for_its_size(got, want, dtype, what):
    """The tolerance of the parity contract plus the rounding of the output itself: a draw with a handful of attended keys
    has outputs as large as single V rows (|O| up to 4 and more), where one bf16 unit in the last place is already
    1.6e-2; elementwise |error| <= contract tolerance + |expected| * 2^-7 (bf16) or * 2^-20 (fp32)."""
    g = got.detach().float().cpu().numpy().astype(np.float64)
    err = np.abs(g - want)
    tol = TOL[dtype]
    assert np.isfinite(g).all(), what + ": non-finite output"
    slack = np.abs(want) * (2.0 ** -7 if dtype == torch.bfloat16 else 2.0 ** -20)
    worst = float((err - slack).max())
    assert worst <= tol["max_abs"], "%s: max-abs beyond the output's own rounding %.3e > %.1e" % (what, worst, tol["max_abs"])
    assert err.mean() <= tol["mean_abs"] + slack.mean(), "%s: mean-abs %.3e" % (what, err.mean())


def test_seeded_random_problems_against_the_oracle():
    """Forty problems drawn from a fixed seed: head dims, group sizes, lengths, budgets, causal offsets and cache
    lengths at random, so that shapes nobody thought of reach every kernel family (SIMT, mma.sync, tcgen05; strips and
    the filtered selection, which is forced on every other case).  Every row of the full layer, the sparse layer and
    the decode step is held against the oracle."""
    import random
    rnd = random.Random(260926368)
    old = hs2.hs2_set_filter_min_keys(0)
    try:
        for case in range(40):
            D = rnd.choice([64, 128, 128, 128, 256])
            Hkv = rnd.choice([1, 2, 4])
            G = rnd.choice([1, 2, 4, 8, 8, 16]) if D != 256 else rnd.choice([2, 8, 32])
            B = rnd.choice([1, 2, 3])
            Lq = rnd.randint(1, 160)
            Lk = Lq + rnd.randint(0, 500)
            k = rnd.choice([0, 1, 7, 32, 100, 128])
            w = rnd.choice([0, 1, 5, 16, 64]) if k > 0 else rnd.choice([1, 5, 16, 64])
            dtype = "f32" if (D == 64 or rnd.random() < 0.15) else "bf16"
            wl = scaled("cfg2", batch=B, q_len=Lq, kv_len=Lk, n_q_heads=G * Hkv, n_kv_heads=Hkv, head_dim=D, dtype=dtype,
                        k_sel=k, window=w, n_needles=min(4, max(1, Lk // 8)), seed=1000 + case)
            inp = make_inputs(wl)
            kv_lens = [rnd.randint(max(1, Lk // 3), Lk) for _ in range(B)]
            q_start = [rnd.randint(-2, max(0, kv_lens[b] - Lq)) for b in range(B)]
            if rnd.random() < 0.3:
                q_start = [kv_lens[b] - Lq for b in range(B)]            # the default alignment, some of it negative
            qs_t = torch.tensor(q_start, dtype=torch.int32, device="cuda")
            kl_t = torch.tensor(kv_lens, dtype=torch.int32, device="cuda")
            scale = rnd.choice([0.0, 0.0, 0.07, 0.2])
            q, kk, v = inp.q_full.cuda(), inp.k.cuda(), inp.v.cuda()
            hs2.hs2_set_filter_min_keys(1 if case % 2 else 1 << 30)
            prob = hs2.Problem.from_tensors(q, kk, k, w, softmax_scale=scale, q_start=qs_t, kv_lens=kl_t)
            what = "case %d: D=%d G=%d Hkv=%d B=%d Lq=%d Lk=%d k=%d w=%d %s q_start=%s kv_lens=%s" % (
                case, D, G, Hkv, B, Lq, Lk, k, w, dtype, q_start, kv_lens)
            O, LSE, idx, _ = hs2.hs2_full_attn_select(prob, q, kk, v, want_idx=k > 0)
            torch.cuda.synchronize()
            okw = dict(scale=scale if scale > 0 else None, q_start=q_start, kv_lens=kv_lens)
            Oo, LSEo, idxo, sco = oracle.full_attn_select(inp.q_full, inp.k, inp.v, k, w, want_idx=k > 0, want_scores=k > 0, **okw)
            dt = wl.torch_dtype
            Hq = G * Hkv
            _close_for_its_size(O.reshape(-1, Hq, D), Oo, dt, what + ": full O")
            l = LSE.permute(0, 2, 1).reshape(B * Lq, Hq).cpu().numpy()
            fin = np.isfinite(LSEo)
            assert np.array_equal(np.isfinite(l), fin), what
            assert not fin.any() or np.abs(l[fin] - LSEo[fin]).max() <= TOL[dt]["lse"], what
            if k > 0:
                idx_rows = idx.permute(0, 2, 1, 3).reshape(B * Lq, Hkv, k).cpu().numpy()
                check_idx_against_oracle(idx_rows, idxo, sco)
            else:
                idx_rows = np.zeros((B * Lq, Hkv, 0), dtype=np.int32)
            qsp = inp.q_sparse[0].cuda()
            out, lse = hs2.hs2_sparse_attn_prefill(prob, qsp, kk, v, idx if k > 0 else None, want_lse=True)
            torch.cuda.synchronize()
            Os, LSEs, _ = oracle.sparse_attn(inp.q_sparse[0], inp.k, inp.v, idx_rows, w, **okw)
            _close_for_its_size(out.reshape(-1, Hq, D), Os, dt, what + ": sparse O")
            q1 = qsp[:, -1:].contiguous()
            qs1 = torch.tensor([q_start[b] + Lq - 1 for b in range(B)], dtype=torch.int32, device="cuda")
            prob1 = hs2.Problem.from_tensors(q1, kk, k, w, softmax_scale=scale, q_start=qs1, kv_lens=kl_t)
            od, _ = hs2.hs2_sparse_attn_decode(prob1, q1, kk, v, idx[:, :, -1:].contiguous() if k > 0 else None)
            torch.cuda.synchronize()
            last = [b * Lq + Lq - 1 for b in range(B)]
            _close_for_its_size(od[:, 0], Os[last], dt, what + ": decode O")
            if dtype == "bf16" and D in (128, 256):
                # the same sparse layer on an e4m3 cache, with a sink bias and the output gate (Section 4.1)
                from gen.workloads import quantize_kv_e4m3
                k8, ksc = quantize_kv_e4m3(kk)
                v8, vsc = quantize_kv_e4m3(v)
                sink = torch.linspace(-1.0, 1.0, Hq, device="cuda")
                o8, _ = hs2.hs2_sparse_attn_prefill_fp8kv(prob, qsp, k8, v8, ksc, vsc, idx if k > 0 else None, sink=sink)
                gate = torch.randn_like(qsp)
                og, _ = hs2.hs2_sparse_attn_prefill(prob, qsp, kk, v, idx if k > 0 else None, sink=sink, gate=gate)
                torch.cuda.synchronize()
                kd, vd = oracle.dequant_e4m3(k8, ksc), oracle.dequant_e4m3(v8, vsc)
                O8, _, _ = oracle.sparse_attn(qsp.float().cpu().numpy(), kd, vd, idx_rows, w, sink=sink.cpu().numpy().astype(np.float64), **okw)
                _close_for_its_size(o8.reshape(-1, Hq, D), O8, dt, what + ": FP8 sparse O")
                Og, _, _ = oracle.sparse_attn(inp.q_sparse[0], inp.k, inp.v, idx_rows, w, sink=sink.cpu().numpy().astype(np.float64),
                                              gate=gate.cpu(), **okw)
                _close_for_its_size(og.reshape(-1, Hq, D), Og, dt, what + ": gated sparse O")
            assert hs2.hs2_device_error_flags() == 0, what
    finally:
        hs2.hs2_set_filter_min_keys(old)


def test_seeded_random_medium_problems_on_the_tensor_core_kernels():
    """Eight larger draws at head_dim 128 and 256 in bf16 (several query and key tiles, ragged tails, offsets, cache
    lengths), the filtered selection forced on every other one; every seventh row against the oracle."""
    import random
    rnd = random.Random(26368)
    old = hs2.hs2_set_filter_min_keys(0)
    try:
        for case in range(8):
            D = rnd.choice([128, 128, 128, 256])
            Hkv = rnd.choice([1, 2])
            G = rnd.choice([4, 8, 16]) if D == 128 else rnd.choice([8, 64])
            B = rnd.choice([1, 2])
            Lq = rnd.randint(300, 900)
            Lk = Lq + rnd.randint(0, 4000)
            k = rnd.choice([64, 200, 512])
            w = rnd.choice([0, 8, 100])
            wl = scaled("cfg2", batch=B, q_len=Lq, kv_len=Lk, n_q_heads=G * Hkv, n_kv_heads=Hkv, head_dim=D, k_sel=k,
                        window=w, n_needles=8, seed=2000 + case)
            inp = make_inputs(wl)
            kv_lens = [rnd.randint(Lk // 2, Lk) for _ in range(B)]
            q_start = [rnd.randint(0, max(0, kv_lens[b] - Lq)) for b in range(B)]
            qs_t = torch.tensor(q_start, dtype=torch.int32, device="cuda")
            kl_t = torch.tensor(kv_lens, dtype=torch.int32, device="cuda")
            q, kk, v = inp.q_full.cuda(), inp.k.cuda(), inp.v.cuda()
            hs2.hs2_set_filter_min_keys(1 if case % 2 else 1 << 30)
            prob = hs2.Problem.from_tensors(q, kk, k, w, q_start=qs_t, kv_lens=kl_t)
            what = "case %d: D=%d G=%d Hkv=%d B=%d Lq=%d Lk=%d k=%d w=%d q_start=%s kv_lens=%s" % (
                case, D, G, Hkv, B, Lq, Lk, k, w, q_start, kv_lens)
            O, LSE, idx, _ = hs2.hs2_full_attn_select(prob, q, kk, v)
            torch.cuda.synchronize()
            rows = [(b, i) for b in range(B) for i in sorted(set(range(0, Lq, 7)) | {Lq - 1})]
            okw = dict(q_start=q_start, kv_lens=kv_lens, rows=rows)
            Oo, LSEo, idxo, sco = oracle.full_attn_select(inp.q_full, inp.k, inp.v, k, w, want_scores=True, **okw)
            dt = wl.torch_dtype
            assert_output_close(gather_rows(O, rows, "bihd"), Oo, dt, what + ": full O")
            l = gather_rows(LSE, rows, "bhi").cpu().numpy()
            fin = np.isfinite(LSEo)
            assert np.array_equal(np.isfinite(l), fin), what
            assert np.abs(l[fin] - LSEo[fin]).max() <= TOL[dt]["lse"], what
            idx_rows = gather_rows(idx, rows, "bgik").cpu().numpy()
            check_idx_against_oracle(idx_rows, idxo, sco)
            qsp = inp.q_sparse[0].cuda()
            out, _ = hs2.hs2_sparse_attn_prefill(prob, qsp, kk, v, idx)
            torch.cuda.synchronize()
            Os, _, _ = oracle.sparse_attn(inp.q_sparse[0], inp.k, inp.v, idx_rows, w, **okw)
            assert_output_close(gather_rows(out, rows, "bihd"), Os, dt, what + ": sparse O")
            assert hs2.hs2_device_error_flags() == 0, what
    finally:
        hs2.hs2_set_filter_min_keys(old)


def test_malformed_indices_cannot_read_out_of_bounds():
    wl = scaled("cfg2", q_len=64, kv_len=64, k_sel=32, window=8, n_needles=4)
    inp = make_inputs(wl)
    run = BlockRun(inp)
    g = torch.Generator().manual_seed(3)
    idx = torch.randint(-50, 1 << 30, (1, wl.n_kv_heads, 64, 32), generator=g, dtype=torch.int32)
    idx[..., ::3] = torch.randint(0, 64, idx[..., ::3].shape, generator=g, dtype=torch.int32)
    # keep the rows free of repeated valid entries (repeats are a documented caller error)
    for gh in range(wl.n_kv_heads):
        for i in range(64):
            row = idx[0, gh, i]
            seen = set()
            for t in range(32):
                j = int(row[t])
                if 0 <= j <= i - 8:
                    if j in seen:
                        row[t] = -1
                    seen.add(j)
    run.idx = idx.cuda()
    out, lse = run.run_sparse(0)
    run.check_sparse(out, lse, 0)


def test_gather_probe_runs_on_the_attention_calls_arguments():
    """hs2_probe_gather (the bare row fetches of the sparse prefill, a measurement aid) accepts what the attention call
    accepts - ragged lengths, malformed indices - touches neither indices nor cache, and sets no error."""
    wl = scaled("cfg2", q_len=300, kv_len=700, k_sel=96, window=24, n_needles=4, batch=2)
    run = BlockRun(make_inputs(wl)).run_full()
    idx = run.idx.clone()
    idx[0, 0, 5, :4] = torch.tensor([-1, 10 ** 6, 699, 3], dtype=torch.int32, device="cuda")   # void, past the cache, in the window, fine
    kv_lens = torch.tensor([700, 333], dtype=torch.int32, device="cuda")
    prob = hs2.Problem.from_tensors(run.q, run.k, wl.k_sel, wl.window, kv_lens=kv_lens)
    k0, v0, i0 = run.k.clone(), run.v.clone(), idx.clone()
    for mode in (0, 1):
        word = hs2.hs2_probe_gather(prob, run.k, run.v, idx, mode=mode)
        torch.cuda.synchronize()
        assert int(word.item()) in (0, 1, 2)
    assert torch.equal(run.k, k0) and torch.equal(run.v, v0) and torch.equal(idx, i0)
    assert hs2.hs2_device_error_flags() == 0


# ---------------------------------------------------------------- decode

@pytest.mark.parametrize("heads", [(32, 4), (64, 4)])      # groups of 8, and of 16 (two sub-groups of 8)
def test_decode_small_matches_oracle_and_prefill_last_row(heads):
    wl = scaled("cfg5", batch=5, kv_len=3000, k_sel=256, window=32, n_needles=8, n_q_heads=heads[0], n_kv_heads=heads[1])
    run = BlockRun(make_inputs(wl)).run_full(want_scores=True)
    run.check_full(check_scores=True)
    run.check_idx_bitexact_on_gpu_scores()
    out_d, lse_d = run.run_sparse(0, decode=True)
    run.check_sparse(out_d, lse_d, 0)
    out_p, lse_p = run.run_sparse(0, decode=False)
    assert (out_d.float() - out_p.float()).abs().max() <= 2e-2
    kv_lens = torch.tensor([3000, 1, 17, 2999, 300], dtype=torch.int32, device="cuda")
    prob = hs2.Problem.from_tensors(run.q, run.k, wl.k_sel, wl.window, kv_lens=kv_lens)
    O, LSE, idx, _ = hs2.hs2_full_attn_select(prob, run.q, run.k, run.v)
    out, _ = hs2.hs2_sparse_attn_decode(prob, run.qs[0], run.k, run.v, idx)
    torch.cuda.synchronize()
    Oo, _, idxo, sco = oracle.full_attn_select(to_host(run.q), to_host(run.k), to_host(run.v), wl.k_sel, wl.window,
                                               kv_lens=kv_lens.cpu().numpy(), want_scores=True)
    assert_output_close(O[:, 0], Oo, wl.torch_dtype, "ragged decode full O")
    idx_rows = idx[:, :, 0].cpu().numpy()
    from parity import check_idx_against_oracle
    check_idx_against_oracle(idx_rows, idxo, sco)
    Os, _, _ = oracle.sparse_attn(to_host(run.qs[0]), to_host(run.k), to_host(run.v), idx_rows, wl.window,
                                  kv_lens=kv_lens.cpu().numpy())
    assert_output_close(out[:, 0], Os, wl.torch_dtype, "ragged decode sparse O")
