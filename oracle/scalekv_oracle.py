"""CPU oracle for the ScaleKV per-scale step (arXiv 2505.19602).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, fp64 statement of what the hot
path computes.  Only the test-suite, the smoke check and the benchmark's CPU-baseline /
reference legs may import it; the product path never does, and this file imports nothing
from the CUDA package (numpy is its only dependency).

Every function cites the passage of the paper it restates.  Arithmetic is float64
throughout; callers round inputs to the storage dtype (bf16 or fp32) before handing them
in, so both sides see the same numbers.  There is no blocking, fusion or reordering: one
slice (layer, batch, head) at a time, whole matrices, one library matmul per contraction.

Notation (paper, Sec. 3.1 / 3.3): scale k has an h_k x w_k token map with n_k = h_k*w_k
tokens; N_k = n_1 + ... + n_k; P_{k-1} = history indices (positions < N_{k-1}); C_k = current
map indices (positions N_{k-1} .. N_k - 1); W = observation window (query rows of r_k);
k^l = layer budget (number of non-window entries kept).

Readings of passages where the paper is silent or ambiguous are marked "Reading:" below.

Pins: attend/window_scores are pinned by brute-force loops, closed forms and special
cases; select/compress by exhaustive subset search on tiny inputs and the count rule;
SliceCache stepping by the full-budget == block-causal attention invariant; schedule and
accounting helpers by the values printed in Table 1, Table 3 and Sec. 4.3; layer_stats by
its invariants and the uniform-attention closed form; make_budgets by Eq. 4 itself.
window_centroids (patch geometry) and assign_roles tie order are readings with no printed
value to check against: parity unpinned for those two choices (their invariants are
tested).  window_last and policy_budgets (the comparison policies as configurations of this
store) are pinned by their closed forms: the arithmetic series' sum, monotonicity, endpoints.
"""
from __future__ import annotations

import math

import numpy as np

KEEP_ALL = -1


# --------------------------------------------------------------------------------------
# Schedule arithmetic (Sec. 3.1: each step k emits h_k x w_k tokens; Sec. 1: the cache must
# hold the K/V of all previous token maps).
# --------------------------------------------------------------------------------------
def scale_token_counts(sides_h, sides_w=None):
    """n_k = h_k * w_k for every scale (Sec. 3.1, text under Eq. 1)."""
    sides_h = [int(x) for x in sides_h]
    sides_w = sides_h if sides_w is None else [int(x) for x in sides_w]
    return [h * w for h, w in zip(sides_h, sides_w)]


def cumulative_token_counts(n):
    """N_k = sum_{i<=k} n_i ; returned with N_0 = 0 in front (length K+1)."""
    out = [0]
    for x in n:
        out.append(out[-1] + int(x))
    return out


def cached_positions(n):
    """T_c: positions that a later step ever reads = all scales but the last.

    Reading (Table 1 arithmetic): the printed full-cache sizes divide exactly by
    N_{K-1}, i.e. the last map is never counted as cached.
    """
    return sum(int(x) for x in n[:-1])


def kv_cache_bytes(n_layers, batch, n_heads, head_dim, elem_bytes, tokens_per_head_layer):
    """Memory of a K and a V row per kept token per head per layer (Sec. 4, Tables 1 and 3)."""
    return int(n_layers) * int(batch) * int(n_heads) * int(tokens_per_head_layer) * 2 * int(head_dim) * int(elem_bytes)


def budget_tokens(fraction, n):
    """Reading (Sec. 4.1 "of the original KV cache size", Sec. 4.3 "10% ... 650 tokens"):
    a percentage budget is that fraction of T_c, rounded half up, fixed per layer."""
    from fractions import Fraction

    x = Fraction(str(fraction)) * cached_positions(n)      # exact, so that .5 cases round up
    return int(math.floor(x + Fraction(1, 2)))


# --------------------------------------------------------------------------------------
# Attention (Sec. 3.3, Eq. 5: A = softmax(Q K^T / sqrt(d_k)); Sec. 3.3 ASI paragraph:
# queries of r_k see history P_{k-1} and current map C_k, which is everything in the cache
# once r_k has been appended, so no mask is needed).
# --------------------------------------------------------------------------------------
def softmax_rows(Z):
    """Row-wise softmax and log-sum-exp of a logit matrix."""
    m = Z.max(axis=1, keepdims=True)
    P = np.exp(Z - m)
    S = P.sum(axis=1, keepdims=True)
    return P / S, (m + np.log(S))[:, 0]


def attend(Q, K, V, softmax_scale=None):
    """O = softmax(Q K^T * scale) V over all L cache entries; also returns lse per row.

    Q [n, d], K [L, d], V [L, d] float64.  scale defaults to 1/sqrt(d) (Eq. 5).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    scale = 1.0 / math.sqrt(Q.shape[1]) if not softmax_scale else float(softmax_scale)
    A, lse = softmax_rows(scale * (Q @ K.T))
    return A @ V, lse


def window_scores(Qw, K, softmax_scale=None):
    """Importance of every cache entry (Eq. 5, the importance score, and the paragraph after it).

    A = softmax(Q_W K^T * scale) row-wise over all L entries; s_i = sum_{j in W} A_ji.
    Reading ("average pooling ... unified importance metric"): the aggregate is the mean
    over the window rows, per head, so sum_i s_i = 1.  Mean and sum rank identically.
    """
    Qw = np.asarray(Qw, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    scale = 1.0 / math.sqrt(Qw.shape[1]) if not softmax_scale else float(softmax_scale)
    A, _ = softmax_rows(scale * (Qw @ K.T))
    return A.sum(axis=0) / Qw.shape[0]


def select(scores, pos, n_prev, window_pos, budget):
    """Which cache entries survive a compress (Sec. 3.3, "KV Cache Selection").

    scores [L], pos [L] ascending original positions, n_prev = N_{k-1}, window_pos = raster
    indices of W inside r_k, budget = k^l (KEEP_ALL keeps everything).
    Window entries (pos - n_prev in W) are always kept and are not candidates; the
    candidates are all remaining entries, history and current alike ("the remaining
    tokens").  The k' = min(k^l, #candidates) candidates with the largest score are kept.
    Reading: equal scores are ordered by lowest position.
    Returns the ascending slot indices that are kept.
    """
    scores = np.asarray(scores, dtype=np.float64)
    pos = np.asarray(pos, dtype=np.int64)
    L = pos.shape[0]
    wabs = set(int(n_prev) + int(p) for p in window_pos)
    is_window = np.array([int(p) in wabs for p in pos], dtype=bool)
    cand = np.nonzero(~is_window)[0]
    kprime = len(cand) if budget == KEEP_ALL else min(int(budget), len(cand))
    order = np.lexsort((pos[cand], -scores[cand]))  # primary: score descending; then pos ascending
    chosen = cand[order[:kprime]]
    keep = np.zeros(L, dtype=bool)
    keep[chosen] = True
    keep |= is_window
    return np.nonzero(keep)[0]


def pool_scores(scores, kernel):
    """1-D average pooling of the importance along the slot axis (Sec. 3.3 speaks of "average pooling",
    and of the selection being "similar to" SnapKV, which smooths its votes this way).

    Reading: window of odd width `kernel` centred on the entry, zeros beyond both ends, always divided
    by `kernel` (the usual avg_pool1d with padding kernel // 2); the neighbours are the entries next to
    it in the cache as it stands (ascending original position), window entries included.  kernel = 1
    leaves the scores as they are.  This is the alternative to the default reading (no pooling along
    keys); parity between the two readings is unpinned.
    """
    s = np.asarray(scores, dtype=np.float64)
    k = int(kernel)
    if k <= 1:
        return s.copy()
    assert k % 2 == 1
    r = k // 2
    padded = np.concatenate([np.zeros(r), s, np.zeros(r)])
    out = np.zeros_like(s)
    for d in range(k):
        out += padded[d:d + s.shape[0]]
    return out / k


def select_recent(pos, budget, n_sink=0):
    """Positional keep rule used by the paper's comparison policies (Sec. 4.1: sliding window;
    sinks + recent tokens): of the L entries keep those whose original position is below n_sink,
    and of the others the most recent ones, `budget` entries in all (KEEP_ALL keeps everything).
    Returns the ascending slot indices that are kept."""
    pos = np.asarray(pos, dtype=np.int64)
    L = pos.shape[0]
    if budget == KEEP_ALL or budget >= L:
        return np.arange(L)
    sink = pos < int(n_sink)
    n_recent = max(int(budget) - int(sink.sum()), 0)
    others = np.nonzero(~sink)[0]
    order = np.argsort(-pos[others], kind="stable")
    keep = np.zeros(L, dtype=bool)
    keep[others[order[:n_recent]]] = True
    keep |= sink
    return np.nonzero(keep)[0]


# --------------------------------------------------------------------------------------
# One slice's cache and the per-scale step (call order append -> attend -> compress).
# --------------------------------------------------------------------------------------
class SliceCache:
    """The cache of one (layer, batch, head) slice: entries (pos, k, v) in ascending pos."""

    def __init__(self, n_per_scale, head_dim, softmax_scale=None):
        self.n = [int(x) for x in n_per_scale]
        self.N = cumulative_token_counts(self.n)
        self.d = int(head_dim)
        self.scale = softmax_scale
        self.reset()

    def reset(self):
        self.pos = np.zeros(0, dtype=np.int64)
        self.K = np.zeros((0, self.d), dtype=np.float64)
        self.V = np.zeros((0, self.d), dtype=np.float64)
        self.k = 0  # number of scales appended so far

    def __len__(self):
        return self.pos.shape[0]

    def append(self, Kk, Vk):
        """The current map joins the cache: keys = P_{k-1} U C_k (Sec. 1; Sec. 3.3)."""
        Kk = np.asarray(Kk, dtype=np.float64)
        Vk = np.asarray(Vk, dtype=np.float64)
        nk = self.n[self.k]
        assert Kk.shape == (nk, self.d) and Vk.shape == (nk, self.d)
        self.pos = np.concatenate([self.pos, self.N[self.k] + np.arange(nk, dtype=np.int64)])
        self.K = np.concatenate([self.K, Kk])
        self.V = np.concatenate([self.V, Vk])
        self.k += 1

    def attend(self, Qk):
        return attend(Qk, self.K, self.V, self.scale)

    def scores(self, Qw):
        return window_scores(Qw, self.K, self.scale)

    def compress(self, Qw, window_pos, budget, pool_kernel=1):
        """Score, (pool,) select, prune (Sec. 3.3).  Returns (kept original positions, scores)."""
        s = pool_scores(self.scores(Qw), pool_kernel)
        keep = select(s, self.pos, self.N[self.k - 1], window_pos, budget)
        self.adopt(keep)
        return self.pos.copy(), s

    def compress_recent(self, budget, n_sink=0):
        """Positional pruning (sliding window, sinks + recent).  Returns the kept original positions."""
        self.adopt(select_recent(self.pos, budget, n_sink))
        return self.pos.copy()

    def adopt(self, keep_slots):
        """Prune to the given ascending slot list."""
        keep_slots = np.asarray(keep_slots, dtype=np.int64)
        self.pos = self.pos[keep_slots]
        self.K = self.K[keep_slots]
        self.V = self.V[keep_slots]

    def adopt_positions(self, kept_pos):
        """Prune to the entries whose original positions are listed (must be a subset)."""
        kept_pos = np.asarray(kept_pos, dtype=np.int64)
        idx = np.searchsorted(self.pos, kept_pos)
        assert np.array_equal(self.pos[idx], kept_pos)
        self.adopt(idx)


def compress_head_shared(caches, Qws, window_pos, budget, pool_kernel=1):
    """Sec. 3.3 with the "unified importance metric" read as shared between heads: the per-head
    importances of the heads of one batch element are averaged entry by entry, (pooled,) and one
    selection prunes every head's cache alike.  caches / Qws: one SliceCache / window query block per
    head; the heads must hold the same original positions.  Returns (kept positions, importance)."""
    first = caches[0]
    for c in caches[1:]:
        if not np.array_equal(c.pos, first.pos):
            raise ValueError("head-shared selection needs the same entries in every head")
    per_head = np.stack([c.scores(Qw) for c, Qw in zip(caches, Qws)], axis=0)
    s = pool_scores(per_head.mean(axis=0), pool_kernel)
    keep = select(s, first.pos, first.N[first.k - 1], window_pos, budget)
    for c in caches:
        c.adopt(keep)
    return first.pos.copy(), s


# --------------------------------------------------------------------------------------
# Observation window geometry (Sec. 3.3: partition r_k into N patches, take each patch's
# centroid token; "typically 16 tokens").
# --------------------------------------------------------------------------------------
def window_centroids(h, w, n_patches=16):
    """Raster indices (r*w + c) of the window tokens of an h x w map, ascending.

    Reading (the paper gives no patch shape): g = floor(sqrt(N)) patches per side; if the
    map has at most N tokens the window is the whole map; otherwise patch (a, b) spans rows
    [floor(a*h/g), floor((a+1)*h/g)) and columns alike, and its centroid is the lower-middle
    cell (floor((r0 + r1 - 1)/2), floor((c0 + c1 - 1)/2)).  Parity unpinned.
    """
    h, w, n_patches = int(h), int(w), int(n_patches)
    if h * w <= n_patches:
        return list(range(h * w))
    g = int(math.isqrt(n_patches))
    out = set()
    for a in range(g):
        r0, r1 = (a * h) // g, ((a + 1) * h) // g
        if r1 <= r0:
            continue
        for b in range(g):
            c0, c1 = (b * w) // g, ((b + 1) * w) // g
            if c1 <= c0:
                continue
            out.add(((r0 + r1 - 1) // 2) * w + (c0 + c1 - 1) // 2)
    return sorted(out)


# --------------------------------------------------------------------------------------
# Attention Selectivity Index (Sec. 3.3, Eq. 2) and role assignment (Eq. 3, the Z-score /
# drafter-selection equation).
# --------------------------------------------------------------------------------------
def layer_stats_slice(Q, K, pos, n_prev, topk_prime, query_stride=1, softmax_scale=None):
    """Per-slice sums for Eq. 2 with a full cache.

    For every sampled query i of r_k (rows 0, stride, 2*stride, ...): alpha_i = softmax row
    over all entries; c_i = sum of alpha over the current map (pos >= N_{k-1}); t_i = sum of
    the min(K', |history|) largest alpha over the history (TopKSum'; empty history gives 0).
    Returns (sum_i c_i, sum_i t_i, number of sampled queries).
    """
    Q = np.asarray(Q, dtype=np.float64)[:: int(query_stride)]
    K = np.asarray(K, dtype=np.float64)
    pos = np.asarray(pos, dtype=np.int64)
    scale = 1.0 / math.sqrt(Q.shape[1]) if not softmax_scale else float(softmax_scale)
    A, _ = softmax_rows(scale * (Q @ K.T))
    cur = pos >= int(n_prev)
    c = A[:, cur].sum(axis=1)
    H = A[:, ~cur]
    kk = min(int(topk_prime), H.shape[1])
    if kk > 0:
        t = np.sort(H, axis=1)[:, H.shape[1] - kk:].sum(axis=1)
    else:
        t = np.zeros(Q.shape[0])
    return float(c.sum()), float(t.sum()), int(Q.shape[0])


def normalized_current_attention(Q, K, pos, n_prev, query_stride=1, softmax_scale=None):
    """Sec. 4.3, "normalized current scale attention" of one slice: for each sampled query the average
    attention per token of the current map over the average attention per entry of the whole sequence,
    (sum_{j in r_k} alpha_ij / n_k) / (sum_j alpha_ij / L), then the mean over the sampled queries."""
    Q = np.asarray(Q, dtype=np.float64)[:: int(query_stride)]
    K = np.asarray(K, dtype=np.float64)
    pos = np.asarray(pos, dtype=np.int64)
    scale = 1.0 / math.sqrt(Q.shape[1]) if not softmax_scale else float(softmax_scale)
    A, _ = softmax_rows(scale * (Q @ K.T))
    cur = pos >= int(n_prev)
    per_query = (A[:, cur].sum(axis=1) / cur.sum()) / (A.sum(axis=1) / A.shape[1])
    return float(per_query.mean())


def asi_from_sums(sum_c, sum_t, count):
    """ASI = (mean current-attention ratio) * (mean history top-K' ratio)  (Eq. 2)."""
    car = sum_c / count
    htk = sum_t / count
    return car * htk, car, htk


def assign_roles(asi, n_drafters, mode=0, eps=1e-6, first_scale=1, last_scale=None):
    """Drafter table from ASI values (Eq. 3, drafter selection).

    asi [L][K].  Z^{(l,k)} = (ASI - mu_k) / (sigma_k + eps) with mu_k, sigma_k the mean and
    (population) standard deviation over layers at scale k.  Scales outside
    [first_scale, last_scale) (0-based) are not ranked (scale 1 has no history, nothing
    follows the last scale) and stay refiners.
    mode 0: the n_drafters (layer, scale) pairs with the lowest Z over all ranked pairs
            (the equation as printed).
    mode 1: at every ranked scale, the n_drafters layers with the lowest Z.
    Reading: Z ties go to the lower scale, then the lower layer.  Returns a bool [L][K].
    """
    asi = np.asarray(asi, dtype=np.float64)
    L, K = asi.shape
    last_scale = K - 1 if last_scale is None else int(last_scale)
    mu = asi.mean(axis=0, keepdims=True)
    sd = asi.std(axis=0, keepdims=True)
    Z = (asi - mu) / (sd + eps)
    roles = np.zeros((L, K), dtype=bool)
    ranked = list(range(int(first_scale), last_scale))
    if mode == 0:
        pairs = sorted(((Z[l, k], k, l) for k in ranked for l in range(L)))
        for _, k, l in pairs[: int(n_drafters)]:
            roles[l, k] = True
    else:
        for k in ranked:
            order = sorted(((Z[l, k], l) for l in range(L)))
            for _, l in order[: int(n_drafters)]:
                roles[l, k] = True
    return roles


def make_budgets(is_drafter, b_uniform, b_r0, delta):
    """Budget table B(l, k) from roles (Sec. 3.3, Eq. 4, the budget constraint).

    B_r(k) = B_r(0) - delta*k with k = 1..K as printed.  Reading: one equation cannot fix K
    drafter budgets, so the balance is imposed per scale,
        N_d^k B_d(k) + N_r^k B_r(k) = B_uniform * L,
    which implies Eq. 4 when summed over k; B_r(k) is clamped at 0; values are rounded half
    up; a scale without drafters gives every layer B_uniform.
    Returns int64 [L][K].
    """
    is_drafter = np.asarray(is_drafter, dtype=bool)
    L, K = is_drafter.shape
    out = np.zeros((L, K), dtype=np.int64)
    for k in range(K):
        nd = int(is_drafter[:, k].sum())
        nr = L - nd
        br = max(float(b_r0) - float(delta) * (k + 1), 0.0)
        if nd == 0:
            out[:, k] = int(math.floor(b_uniform + 0.5))
            continue
        bd = (float(b_uniform) * L - nr * br) / nd
        out[is_drafter[:, k], k] = int(math.floor(bd + 0.5))
        out[~is_drafter[:, k], k] = int(math.floor(br + 0.5))
    return out


# --------------------------------------------------------------------------------------
# The comparison policies of Sec. 4.1 ("Compression Baselines") stated as configurations of the same
# store: which rows observe, how the importance is smoothed, how the budget is spread over layers.
# Their image quality is not in scope; these are keep-rules that run on the same cache for timing.
# --------------------------------------------------------------------------------------
def window_last(h, w, n_obs=16):
    """Observation window of the SnapKV-like rule: the last n_obs tokens of the h x w map in raster
    order (that method observes with the end of its input); a map with at most n_obs tokens is its
    own window.  Ascending raster indices."""
    n = int(h) * int(w)
    m = min(int(n_obs), n)
    return list(range(n - m, n))


def policy_budgets(policy, n_layers, n_scales, b_mean, beta=20.0):
    """Budget table [L][K] of a comparison policy with the same mean per layer as `b_mean`.

    "uniform": every layer and scale gets b_mean (sliding window, sinks + recent, SnapKV-like).
    "pyramid": budgets fall linearly with the layer index from b_max at the first layer to
    b_min = b_mean / beta at the last one, b_max = 2 b_mean - b_min, so that the mean over layers is
    b_mean (the pyramid-shaped allocation of PyramidKV); the same row for every scale; one layer
    gets b_mean.  Values are rounded half up.
    Returns int64 [L][K]."""
    L, K = int(n_layers), int(n_scales)
    out = np.zeros((L, K), dtype=np.int64)
    if policy == "uniform" or L == 1:
        out[:, :] = int(math.floor(float(b_mean) + 0.5))
        return out
    if policy != "pyramid":
        raise ValueError(policy)
    b_min = float(b_mean) / float(beta)
    b_max = 2.0 * float(b_mean) - b_min
    for l in range(L):
        b = b_max - (b_max - b_min) * l / (L - 1)
        out[l, :] = int(math.floor(b + 0.5))
    return out

