"""Pins for the CPU oracle: each checks it against something other than itself - values the
paper prints, closed forms, brute force written with different loops, invariants and special
cases.  No GPU, no CUDA package."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import scalekv_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SIDES_13 = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)
SIDES_16 = SIDES_13 + (80, 96, 128)


def read_table(name):
    rows = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append(line.split())
    return rows


# ---------------------------------------------------------------- closed forms / paper values
def test_token_count_closed_forms():
    # sum over scales of h_k*w_k (Sec. 3.1); Sec. 1: a 1024x1024 image needs "over 10K" tokens
    assert sum(orc.scale_token_counts((1, 2, 4, 8))) == 85
    n13 = orc.scale_token_counts(SIDES_13)
    assert sum(n13) == 10521
    assert sum(orc.scale_token_counts(SIDES_16)) == 42521
    assert orc.cumulative_token_counts(n13)[-2] == 6425 == orc.cached_positions(n13)
    assert orc.cached_positions(orc.scale_token_counts((1, 2, 4, 8))) == 21
    assert orc.cached_positions(orc.scale_token_counts(SIDES_16)) == 26137
    consts = dict((k, float(v)) for k, v in read_table("sec43_budget_constants.txt"))
    assert sum(n13) > consts["min_total_tokens_1024"]
    # sums of squares of the sides: n_k = a_k^2 (independent formula)
    assert sum(n13) == sum(a * a for a in SIDES_13)
    N = orc.cumulative_token_counts(n13)
    assert sum(n * Nk for n, Nk in zip(n13, N[1:])) == 68484681
    assert sum(n * n for n in n13) == 26277921
    # rectangular maps: h_k * w_k tokens per scale (Sec. 3.1 writes r_k as an h_k x w_k map)
    assert orc.scale_token_counts((1, 2, 3, 5), (2, 3, 5, 4)) == [2, 6, 15, 20]
    assert orc.cumulative_token_counts([2, 6, 15, 20]) == [0, 2, 8, 23, 43]


def test_table1_accounting():
    """Table 1's KV-cache column is linear in retained tokens and counts exactly T_c = 6425
    positions for the full cache: full_MB / T_c * tokens reproduces every printed entry."""
    rows = {int(r[0]): (int(r[1]), int(r[2])) for r in read_table("table1_kv_cache_mb.txt")}
    n13 = orc.scale_token_counts(SIDES_13)
    t_c = orc.cached_positions(n13)
    consts = dict((k, float(v)) for k, v in read_table("sec43_budget_constants.txt"))
    tokens = {100: t_c, 10: int(consts["tokens_per_head_layer_at_10pct"]), 20: 1300, 4: 265}
    for col in (0, 1):
        per_pos = rows[100][col] / t_c
        # same geometry constant in both columns' rows: bytes scale with tokens only
        for pct, tok in tokens.items():
            unit = orc.kv_cache_bytes(1, 1, 1, 1, 1, tok) / orc.kv_cache_bytes(1, 1, 1, 1, 1, t_c)
            assert abs(unit * rows[100][col] - rows[pct][col]) < 1.0, (pct, col)
        assert abs(per_pos * 650 - rows[10][col]) < 1.0
    # 10 % of T_c is 642.5, rounded half up to 643 (the paper quotes 650)
    assert orc.budget_tokens(0.10, n13) == 643
    assert orc.budget_tokens(0.30, n13) == 1928 and orc.budget_tokens(0.03, n13) == 193
    # accounting is linear in every geometric factor
    assert orc.kv_cache_bytes(32, 8, 16, 128, 2, 10521) * 40 * 32 == orc.kv_cache_bytes(40, 8, 32, 128, 2, 10521) * 32 * 16
    assert orc.kv_cache_bytes(40, 8, 32, 128, 2, 10521) == 55160340480  # "about 55 GB"


def test_table3_linear_in_batch():
    rows = [(int(r[0]), float(r[1]), float(r[2])) for r in read_table("table3_memory_gb.txt")]
    b1 = rows[0]
    for b, full, comp in rows:
        ratio = orc.kv_cache_bytes(1, b, 1, 1, 1, 1) / orc.kv_cache_bytes(1, 1, 1, 1, 1, 1)
        assert abs(ratio * b1[1] - full) / full < 0.02
        assert abs(ratio * b1[2] - comp) / comp < 0.04
        assert abs(comp / full - 0.10) < 0.006


# ---------------------------------------------------------------- brute force attention
def brute_attention(Q, K, V, scale):
    """Definition written with scalar loops and math.fsum (two passes, no numpy matmul)."""
    n, d = len(Q), len(Q[0])
    L = len(K)
    out, lse = [], []
    for i in range(n):
        z = [scale * math.fsum(Q[i][c] * K[j][c] for c in range(d)) for j in range(L)]
        m = max(z)
        p = [math.exp(x - m) for x in z]
        Z = math.fsum(p)
        out.append([math.fsum(p[j] * V[j][c] for j in range(L)) / Z for c in range(d)])
        lse.append(m + math.log(Z))
    return np.array(out), np.array(lse)


@pytest.mark.parametrize("n,L,d", [(1, 1, 4), (3, 7, 8), (5, 21, 16), (4, 33, 64)])
def test_attend_vs_brute_force(n, L, d):
    rng = np.random.default_rng(10 + n + L)
    Q, K, V = rng.normal(size=(n, d)), rng.normal(size=(L, d)) * 2.0, rng.normal(size=(L, d))
    O, lse = orc.attend(Q, K, V)
    Ob, lb = brute_attention(Q.tolist(), K.tolist(), V.tolist(), 1.0 / math.sqrt(d))
    assert np.max(np.abs(O - Ob)) < 1e-12
    assert np.max(np.abs(lse - lb)) < 1e-12
    # explicit scale argument
    O2, _ = orc.attend(Q, K, V, 0.37)
    Ob2, _ = brute_attention(Q.tolist(), K.tolist(), V.tolist(), 0.37)
    assert np.max(np.abs(O2 - Ob2)) < 1e-12


def test_attend_special_cases():
    rng = np.random.default_rng(3)
    d, L = 16, 40
    K, V = rng.normal(size=(L, d)), rng.normal(size=(L, d))
    # zero queries: uniform attention, O = mean of V, lse = log L
    O, lse = orc.attend(np.zeros((3, d)), K, V)
    assert np.max(np.abs(O - V.mean(axis=0))) < 1e-13
    assert np.max(np.abs(lse - math.log(L))) < 1e-13
    # one key aligned with the query and very long: output tends to its value row
    q = rng.normal(size=(1, d))
    K2 = K.copy()
    K2[17] = 200.0 * q[0]
    O, _ = orc.attend(q, K2, V)
    assert np.max(np.abs(O[0] - V[17])) < 1e-9
    # permuting cache entries does not change the output
    perm = rng.permutation(L)
    Q = rng.normal(size=(4, d))
    assert np.max(np.abs(orc.attend(Q, K, V)[0] - orc.attend(Q, K[perm], V[perm])[0])) < 1e-13
    # transposition check: O is linear in V, not in K
    assert np.max(np.abs(orc.attend(Q, K, 2.0 * V)[0] - 2.0 * orc.attend(Q, K, V)[0])) < 1e-13


# ---------------------------------------------------------------- scores (Eq. 5)
def brute_scores(Qw, K, scale):
    w, L, d = len(Qw), len(K), len(K[0])
    s = [0.0] * L
    for j in range(w):
        z = [scale * sum(Qw[j][c] * K[i][c] for c in range(d)) for i in range(L)]
        m = max(z)
        e = [math.exp(x - m) for x in z]
        Z = math.fsum(e)
        for i in range(L):
            s[i] += e[i] / Z
    return np.array(s) / w


def test_window_scores_vs_brute_and_invariants():
    rng = np.random.default_rng(5)
    for (w, L, d) in [(1, 5, 4), (4, 21, 8), (16, 57, 16)]:
        Qw, K = rng.normal(size=(w, d)), rng.normal(size=(L, d)) * 1.5
        s = orc.window_scores(Qw, K)
        assert np.max(np.abs(s - brute_scores(Qw.tolist(), K.tolist(), 1 / math.sqrt(d)))) < 1e-13
        assert np.all(s >= 0) and abs(s.sum() - 1.0) < 1e-12
    # zero window queries: every key gets 1/L
    s = orc.window_scores(np.zeros((4, 8)), rng.normal(size=(11, 8)))
    assert np.max(np.abs(s - 1.0 / 11)) < 1e-15
    # a key that all window rows point at collects (almost) all of the mass
    Qw = np.tile(rng.normal(size=(1, 8)), (3, 1))
    K = rng.normal(size=(9, 8))
    K[4] = 100.0 * Qw[0]
    assert orc.window_scores(Qw, K)[4] > 1 - 1e-9


# ---------------------------------------------------------------- selection
def test_select_is_the_best_subset_by_exhaustive_search():
    """Keeping the k' highest-scored candidates maximises the kept score mass; check by
    enumerating every subset (distinct scores => unique optimum)."""
    rng = np.random.default_rng(7)
    for trial in range(20):
        n_prev = 6
        pos = np.arange(n_prev + 4)            # 6 history + a 2x2 current map
        s = rng.permutation(len(pos)).astype(float) + rng.random(len(pos)) * 0.5
        window = [1, 2]
        budget = int(rng.integers(0, 9))
        keep = orc.select(s, pos, n_prev, window, budget)
        cand = [i for i in range(len(pos)) if i not in (n_prev + 1, n_prev + 2)]
        kk = min(budget, len(cand))
        best = max(itertools.combinations(cand, kk), key=lambda c: sum(s[list(c)]))
        assert sorted(keep.tolist()) == sorted(list(best) + [n_prev + 1, n_prev + 2])
        assert len(keep) == kk + 2


def test_select_ties_and_limits():
    pos = np.array([0, 3, 4, 9, 10, 11, 12, 13])   # a pruned history, then a 2x2 map at 10..13
    s = np.full(8, 0.125)
    keep = orc.select(s, pos, 10, [3], 2)
    # all tied: lowest positions win among candidates; window entry (pos 13) always kept
    assert pos[keep].tolist() == [0, 3, 13]
    assert orc.select(s, pos, 10, [3], orc.KEEP_ALL).tolist() == list(range(8))
    assert orc.select(s, pos, 10, [3], 100).tolist() == list(range(8))
    assert pos[orc.select(s, pos, 10, [0, 1, 2, 3], 0)].tolist() == [10, 11, 12, 13]
    # a strictly larger score beats a lower position
    s2 = s.copy()
    s2[5] = 0.2
    assert pos[orc.select(s2, pos, 10, [3], 2)].tolist() == [0, 11, 13]


# ---------------------------------------------------------------- stepping invariants
def run_pass(sides, d, H_budget, window_fn, seed, compress_last=False):
    n = orc.scale_token_counts(sides)
    rng = np.random.default_rng(seed)
    cache = orc.SliceCache(n, d)
    outs, kept, data = [], [], []
    for k, nk in enumerate(n):
        Q, K, V = rng.normal(size=(nk, d)), rng.normal(size=(nk, d)), rng.normal(size=(nk, d))
        data.append((Q, K, V))
        cache.append(K, V)
        O, _ = cache.attend(Q)
        outs.append(O)
        if k + 1 < len(n) or compress_last:
            wpos = window_fn(sides[k])
            before = set(cache.pos.tolist())
            L = len(cache)
            kp, s = cache.compress(Q[wpos], wpos, H_budget)
            # count rule and validity
            cand = L - len(wpos)
            expect = cand if H_budget == orc.KEEP_ALL else min(H_budget, cand)
            assert len(kp) == expect + len(wpos)
            assert np.all(np.diff(kp) > 0)
            assert set(kp.tolist()) <= before
            base = cache.N[k]
            assert all(base + p in set(kp.tolist()) for p in wpos)
            assert abs(s.sum() - 1) < 1e-12
            kept.append(kp)
    return outs, kept, data


def test_full_budget_equals_block_causal_attention():
    """With nothing evicted, the step-wise outputs equal masked attention over the whole
    sequence, a query of scale k seeing every key of scales <= k (Sec. 3.1 conditioning)."""
    sides, d = (1, 2, 3, 4), 8
    outs, _, data = run_pass(sides, d, orc.KEEP_ALL, lambda a: orc.window_centroids(a, a, 4), seed=11)
    Q = np.concatenate([x[0] for x in data])
    K = np.concatenate([x[1] for x in data])
    V = np.concatenate([x[2] for x in data])
    sc = np.concatenate([[k] * (a * a) for k, a in enumerate(sides)])
    Z = (Q @ K.T) / math.sqrt(d)
    Z[sc[:, None] < sc[None, :]] = -np.inf
    P = np.exp(Z - Z.max(axis=1, keepdims=True))
    P /= P.sum(axis=1, keepdims=True)
    ref = P @ V
    assert np.max(np.abs(np.concatenate(outs) - ref)) < 1e-12
    # budget larger than the cache behaves like KEEP_ALL
    outs2, _, _ = run_pass(sides, d, 10_000, lambda a: orc.window_centroids(a, a, 4), seed=11)
    assert all(np.array_equal(a, b) for a, b in zip(outs, outs2))


def test_count_rule_and_eviction_changes_outputs():
    sides, d = (1, 2, 4, 8), 16
    full, _, _ = run_pass(sides, d, orc.KEEP_ALL, lambda a: list(range(a * a)), seed=2)
    for budget in (2, 4, 8, 16):
        outs, kept, _ = run_pass(sides, d, budget, lambda a: list(range(a * a)), seed=2, compress_last=True)
        # window = whole current map: after compress the cache is min(budget, history) + n_k
        hist = [0, 1, min(budget, 1) + 4, None]
        assert len(kept[0]) == 1 and len(kept[1]) == min(budget, 1) + 4
        assert len(kept[3]) == min(budget, len(kept[2])) + 64
        if budget <= 4:
            assert np.max(np.abs(outs[3] - full[3])) > 1e-6   # eviction at scales 2-3 shows later


def test_permutation_invariance_of_kept_positions():
    rng = np.random.default_rng(9)
    d, L, n_prev = 8, 30, 26
    pos = np.arange(L)
    K = rng.normal(size=(L, d))
    Qw = rng.normal(size=(2, d))
    s = orc.window_scores(Qw, K)
    keep = orc.select(s, pos, n_prev, [0, 3], 7)
    # same cache with history rows listed in another (still ascending-pos relabelled) order:
    # scores follow the rows, so the kept *positions* are the same set
    perm = np.concatenate([rng.permutation(n_prev), np.arange(n_prev, L)])
    s2 = orc.window_scores(Qw, K[perm])
    order = np.argsort(pos[perm], kind="stable")
    keep2 = orc.select(s2[order], pos[perm][order], n_prev, [0, 3], 7)
    assert pos[keep].tolist() == pos[perm][order][keep2].tolist()


# ---------------------------------------------------------------- window geometry (reading)
@pytest.mark.parametrize("a", SIDES_16)
def test_window_centroids_shape(a):
    w = orc.window_centroids(a, a, 16)
    assert len(w) == min(16, a * a) and len(set(w)) == len(w)
    assert w == sorted(w) and 0 <= w[0] and w[-1] < a * a
    if a >= 8 and a % 4 == 0:
        # one centroid per patch of a 4x4 partition
        cells = {(p // a) // (a // 4) * 4 + (p % a) // (a // 4) for p in w}
        assert cells == set(range(16))


# ---------------------------------------------------------------- ASI (Eq. 2), roles (Eq. 3), budgets (Eq. 4)
def test_layer_stats_invariants_and_uniform_closed_form():
    rng = np.random.default_rng(4)
    d, n_prev, nk = 8, 21, 16
    pos = np.arange(n_prev + nk)
    K = rng.normal(size=(n_prev + nk, d))
    Q = rng.normal(size=(nk, d))
    for kp in (1, 4, 16, 1000):
        sc, st, cnt = orc.layer_stats_slice(Q, K, pos, n_prev, kp)
        asi, car, htk = orc.asi_from_sums(sc, st, cnt)
        assert cnt == nk and 0 <= car <= 1 and 0 <= htk <= 1 - car + 1e-12
        assert 0 <= asi <= 0.25 + 1e-12
        if kp >= n_prev:
            assert abs(htk - (1 - car)) < 1e-12        # top-K' covers the whole history
    # monotone in K'
    h = [orc.layer_stats_slice(Q, K, pos, n_prev, kp)[1] for kp in (1, 2, 4, 8, 16, 32)]
    assert all(b >= a - 1e-15 for a, b in zip(h, h[1:]))
    # uniform attention (Q = 0): CAR = n_k/N_k, HTK = min(K', N_{k-1})/N_k
    for kp in (5, 50):
        sc, st, cnt = orc.layer_stats_slice(np.zeros((nk, d)), K, pos, n_prev, kp)
        _, car, htk = orc.asi_from_sums(sc, st, cnt)
        assert abs(car - nk / (n_prev + nk)) < 1e-13
        assert abs(htk - min(kp, n_prev) / (n_prev + nk)) < 1e-13
    # first scale: no history => ASI = 0
    sc, st, cnt = orc.layer_stats_slice(Q[:1], K[:1], pos[:1], 0, 16)
    assert orc.asi_from_sums(sc, st, cnt)[0] == 0.0
    # query stride samples rows 0, s, 2s, ...
    a = orc.layer_stats_slice(Q, K, pos, n_prev, 4, query_stride=4)
    b = orc.layer_stats_slice(Q[::4], K, pos, n_prev, 4)
    assert a == b and a[2] == 4


def test_layer_stats_topk_vs_loops():
    rng = np.random.default_rng(14)
    d, n_prev, nk, kp = 4, 9, 4, 3
    pos = np.arange(n_prev + nk)
    K, Q = rng.normal(size=(n_prev + nk, d)), rng.normal(size=(nk, d))
    sc = st = 0.0
    for i in range(nk):
        z = [sum(Q[i][c] * K[j][c] for c in range(d)) / math.sqrt(d) for j in range(n_prev + nk)]
        e = [math.exp(x - max(z)) for x in z]
        a = [x / math.fsum(e) for x in e]
        sc += math.fsum(a[n_prev:])
        st += math.fsum(sorted(a[:n_prev], reverse=True)[:kp])
    got = orc.layer_stats_slice(Q, K, pos, n_prev, kp)
    assert abs(got[0] - sc) < 1e-13 and abs(got[1] - st) < 1e-13


def test_assign_roles():
    rng = np.random.default_rng(6)
    L, K = 8, 6
    asi = rng.random((L, K)) * np.linspace(0.01, 0.2, K)[None, :]     # scale-dependent magnitude
    low = [1, 5]
    asi[low, :] *= 0.05                                              # planted drafters
    r1 = orc.assign_roles(asi, 2, mode=1)
    assert r1[:, 0].sum() == 0 and r1[:, K - 1].sum() == 0            # unranked scales
    for k in range(1, K - 1):
        assert np.nonzero(r1[:, k])[0].tolist() == low
    r0 = orc.assign_roles(asi, 2 * (K - 2), mode=0)
    assert r0.sum() == 2 * (K - 2)
    # Z-scores are invariant to a per-scale affine change of ASI
    r0b = orc.assign_roles(asi * np.linspace(1, 9, K)[None, :] + 3.0, 2 * (K - 2), mode=0, eps=0.0)
    r0a = orc.assign_roles(asi, 2 * (K - 2), mode=0, eps=0.0)
    assert np.array_equal(r0a, r0b)
    # brute Z for one cell
    k = 2
    z = (asi[3, k] - sum(asi[:, k]) / L) / (math.sqrt(sum((x - sum(asi[:, k]) / L) ** 2 for x in asi[:, k]) / L) + 1e-6)
    mu, sd = asi[:, k].mean(), asi[:, k].std()
    assert abs(z - (asi[3, k] - mu) / (sd + 1e-6)) < 1e-12


def test_make_budgets_satisfies_eq4():
    consts = dict((k, float(v)) for k, v in read_table("sec43_budget_constants.txt"))
    L, K = 32, 13
    rng = np.random.default_rng(8)
    roles = np.zeros((L, K), dtype=bool)
    for k in range(1, K - 1):
        roles[rng.permutation(L)[: 8], k] = True
    bu, br0 = consts["tokens_per_head_layer_at_10pct"], consts["refiner_initial_budget"]
    for delta in (consts["decay_min"], 10, 35, consts["decay_max"]):
        B = orc.make_budgets(roles, bu, br0, delta)
        total = 0
        for k in range(K):
            nd = roles[:, k].sum()
            bd = B[roles[:, k], k]
            brk = B[~roles[:, k], k]
            assert len(set(bd.tolist())) <= 1 and len(set(brk.tolist())) == 1
            total += B[:, k].sum()
            if nd:
                expect_r = max(br0 - delta * (k + 1), 0)
                assert brk[0] == int(math.floor(expect_r + 0.5))
                assert abs(B[:, k].sum() - bu * L) <= nd          # per-scale balance up to rounding
                assert bd[0] > brk[0]                             # B_d >> B_r
            else:
                assert brk[0] == bu
        assert abs(total - bu * L * K) <= L * K                    # Eq. 4 up to rounding
    # larger decay moves budget from refiners to drafters
    B0 = orc.make_budgets(roles, bu, br0, 0)
    B70 = orc.make_budgets(roles, bu, br0, 70)
    assert B70[roles].sum() > B0[roles].sum() and B70[~roles].sum() < B0[~roles].sum()


# ---- alternative selection rules (pooling along the key axis, positional policies) -------------------
def test_pool_scores_against_brute_force_and_closed_forms():
    rng = np.random.default_rng(11)
    s = rng.random(37)
    for k in (1, 3, 7, 9):
        got = orc.pool_scores(s, k)
        want = np.zeros_like(s)
        for i in range(len(s)):
            for d in range(-(k // 2), k // 2 + 1):
                if 0 <= i + d < len(s):
                    want[i] += s[i + d]
            want[i] /= k
        assert np.allclose(got, want, atol=1e-15)
    assert np.array_equal(orc.pool_scores(s, 1), s)
    ones = np.ones(10)
    p = orc.pool_scores(ones, 5)
    assert np.allclose(p[2:8], 1.0) and np.allclose(p[[0, 9]], 3 / 5) and np.allclose(p[[1, 8]], 4 / 5)
    # a single spike spreads evenly over its neighbourhood and keeps its mass
    e = np.zeros(21); e[10] = 1.0
    q = orc.pool_scores(e, 7)
    assert np.allclose(q[7:14], 1 / 7) and np.isclose(q.sum(), 1.0) and q[6] == 0


def test_select_recent_brute_force_and_count_rule():
    rng = np.random.default_rng(12)
    for trial in range(30):
        L = int(rng.integers(1, 40))
        pos = np.sort(rng.choice(200, size=L, replace=False))
        budget = int(rng.integers(0, L + 3))
        n_sink = int(rng.integers(0, 6))
        keep = orc.select_recent(pos, budget, n_sink)
        if budget >= L:
            assert np.array_equal(keep, np.arange(L))
            continue
        sinks = [i for i in range(L) if pos[i] < n_sink]
        rest = sorted((i for i in range(L) if pos[i] >= n_sink), key=lambda i: -pos[i])
        want = sorted(sinks + rest[: max(budget - len(sinks), 0)])
        assert keep.tolist() == want
        assert len(keep) == max(budget, len(sinks))
    assert np.array_equal(orc.select_recent(np.arange(5), orc.KEEP_ALL, 2), np.arange(5))
    # sliding window: the last entries; sinks + recent: the first n_sink and the last ones
    assert orc.select_recent(np.arange(10), 3).tolist() == [7, 8, 9]
    assert orc.select_recent(np.arange(10), 5, 2).tolist() == [0, 1, 7, 8, 9]


def test_head_shared_compress_brute_force_and_special_cases():
    """compress_head_shared against loops written here: attention of every window row to every entry
    with math.exp, summed over rows and heads; the budget's largest non-window entries stay, ties
    to the lowest position.  Special cases: one head, and identical heads, reduce to the per-head rule."""
    rng = np.random.default_rng(21)
    sides = (2, 3, 5)
    n = orc.scale_token_counts(sides)
    N = orc.cumulative_token_counts(n)
    d, H, budget = 8, 3, 9
    caches = [orc.SliceCache(n, d) for _ in range(H)]
    solo = orc.SliceCache(n, d)          # head 0 alone, per-head rule
    twins = [orc.SliceCache(n, d) for _ in range(2)]   # two copies of head 0, shared rule
    diverged = False
    for k in range(len(sides)):
        Q = rng.normal(size=(H, n[k], d)); K = rng.normal(size=(H, n[k], d)); V = rng.normal(size=(H, n[k], d))
        for h in range(H):
            caches[h].append(K[h], V[h])
        solo.append(K[0], V[0])
        for c in twins:
            c.append(K[0], V[0])
        wpos = orc.window_centroids(sides[k], sides[k], 4)
        pos = caches[0].pos.copy()
        L = len(pos)
        total = [0.0] * L
        for h in range(H):
            for i in wpos:
                z = [sum(Q[h, i, e] * caches[h].K[j, e] for e in range(d)) / math.sqrt(d) for j in range(L)]
                zmax = max(z)
                ez = [math.exp(v - zmax) for v in z]
                den = sum(ez)
                for j in range(L):
                    total[j] += ez[j] / den
        win_abs = {N[k] + i for i in wpos}
        cand = [j for j in range(L) if int(pos[j]) not in win_abs]
        cand.sort(key=lambda j: (-total[j], pos[j]))
        want = sorted(cand[:budget] + [j for j in range(L) if int(pos[j]) in win_abs])
        got, s = orc.compress_head_shared(caches, [Q[h][wpos] for h in range(H)], wpos, budget)
        assert got.tolist() == pos[want].tolist()
        assert np.allclose(s, np.array(total) / (H * len(wpos)), rtol=1e-12, atol=1e-15)
        for c in caches:
            assert np.array_equal(c.pos, got)
        # identical heads and a single head: the per-head rule
        p_solo, _ = solo.compress(Q[0][wpos], wpos, budget)
        p_twin, _ = orc.compress_head_shared(twins, [Q[0][wpos]] * 2, wpos, budget)
        assert np.array_equal(p_solo, p_twin)
        diverged = diverged or not np.array_equal(p_solo, got)
    assert diverged          # the shared rule is not the per-head rule in disguise
    # heads that hold different entries are refused
    a, b = orc.SliceCache(n, d), orc.SliceCache(n, d)
    for c in (a, b):
        c.append(rng.normal(size=(n[0], d)), rng.normal(size=(n[0], d)))
        c.append(rng.normal(size=(n[1], d)), rng.normal(size=(n[1], d)))
    a.adopt(np.arange(1, len(a)))
    b.adopt(np.arange(0, len(b) - 1))
    with pytest.raises(ValueError):
        orc.compress_head_shared([a, b], [rng.normal(size=(1, d))] * 2, [0], 2)


def test_normalized_current_attention_closed_forms():
    """Uniform attention gives 1; all mass on the current map gives L / n_k; none gives 0; and the
    value is CAR * L / n_k computed with plain loops."""
    rng = np.random.default_rng(8)
    d, n_prev, nk = 8, 30, 12
    L = n_prev + nk
    pos = np.arange(L)
    K = rng.normal(size=(L, d))
    assert abs(orc.normalized_current_attention(np.zeros((nk, d)), K, pos, n_prev) - 1.0) < 1e-13
    # keys of the current map aligned with the queries, scaled up: the mass moves onto the current map
    big = np.zeros((L, d)); big[n_prev:, 0] = 50.0; big[:n_prev, 0] = -50.0
    q = np.zeros((nk, d)); q[:, 0] = 10.0
    assert abs(orc.normalized_current_attention(q, big, pos, n_prev) - L / nk) < 1e-9
    assert orc.normalized_current_attention(-q, big, pos, n_prev) < 1e-9
    Q = rng.normal(size=(nk, d))
    total = 0.0
    for i in range(0, nk, 3):
        z = [sum(Q[i, e] * K[j, e] for e in range(d)) / math.sqrt(d) for j in range(L)]
        zmax = max(z)
        ez = [math.exp(v - zmax) for v in z]
        total += sum(ez[n_prev:]) / sum(ez) * L / nk
    assert abs(orc.normalized_current_attention(Q, K, pos, n_prev, query_stride=3) - total / 4) < 1e-12
    sc, _, cnt = orc.layer_stats_slice(Q, K, pos, n_prev, 4, query_stride=3)
    assert abs(orc.normalized_current_attention(Q, K, pos, n_prev, query_stride=3) - sc / cnt * L / nk) < 1e-12


def test_comparison_policy_helpers_closed_forms():
    """window_last: the tail of the raster order.  policy_budgets: "pyramid" is an arithmetic series over the
    layers whose mean is b_mean (so the total equals the uniform table's up to rounding), strictly falling, from
    2 b_mean - b_mean / beta down to b_mean / beta; beta = 1, one layer and "uniform" all give b_mean."""
    assert orc.window_last(3, 5, 16) == list(range(15)) and orc.window_last(8, 8, 16) == list(range(48, 64))
    assert orc.window_last(6, 10, 4) == [56, 57, 58, 59] and orc.window_last(1, 1, 16) == [0]
    for L, b, beta in ((32, 627, 20.0), (40, 1300, 20.0), (5, 100, 4.0), (2, 11, 3.0)):
        t = orc.policy_budgets("pyramid", L, 3, b, beta)
        assert t.shape == (L, 3) and np.all(t[:, 0] == t[:, 1]) and np.all(t[:, 0] == t[:, 2])
        col = t[:, 0]
        assert abs(int(col.sum()) - L * b) <= L // 2 + 1          # rounding residue of an exact series sum L * b
        assert np.all(np.diff(col) < 0)
        assert col[0] == math.floor(2 * b - b / beta + 0.5) and col[-1] == math.floor(b / beta + 0.5)
        assert abs((col[0] + col[-1]) / 2 - b) <= 1
    assert np.all(orc.policy_budgets("pyramid", 6, 2, 50, 1.0) == 50)
    assert np.all(orc.policy_budgets("pyramid", 1, 4, 77, 20.0) == 77)
    assert np.all(orc.policy_budgets("uniform", 7, 3, 642.5) == 643)

