"""The pins must bite: every plausible mistake planted in the oracle here (on the CPU, in a patched copy of
one function at a time) has to make at least one of the pin tests fail.  A mistake that slips through all
of them would mean that the GPU path is checked against an oracle nothing vouches for."""
import math

import numpy as np
import pytest

import test_oracle_pins as pins
from oracle import scalekv_oracle as orc


# ---- the planted mistakes: each returns the wrong function to put in place of orc.<name> ----------
def attend_without_scale(Q, K, V, softmax_scale=None):
    A, lse = orc.softmax_rows(np.asarray(Q, float) @ np.asarray(K, float).T)         # dropped 1/sqrt(d)
    return A @ np.asarray(V, float), lse


def attend_values_from_keys(Q, K, V, softmax_scale=None):
    Q, K = np.asarray(Q, float), np.asarray(K, float)
    scale = 1.0 / math.sqrt(Q.shape[1]) if not softmax_scale else float(softmax_scale)
    A, lse = orc.softmax_rows(scale * (Q @ K.T))
    return A @ K, lse                                                                  # wrong operand


def attend_lse_without_max(Q, K, V, softmax_scale=None):
    Q, K = np.asarray(Q, float), np.asarray(K, float)
    scale = 1.0 / math.sqrt(Q.shape[1]) if not softmax_scale else float(softmax_scale)
    Z = scale * (Q @ K.T)
    A, _ = orc.softmax_rows(Z)
    return A @ np.asarray(V, float), np.log(np.exp(Z - Z.max(axis=1, keepdims=True)).sum(axis=1))   # dropped + max


def scores_softmax_over_window_axis(Qw, K, softmax_scale=None):
    Qw, K = np.asarray(Qw, float), np.asarray(K, float)
    scale = 1.0 / math.sqrt(Qw.shape[1]) if not softmax_scale else float(softmax_scale)
    Z = scale * (Qw @ K.T)
    A = np.exp(Z - Z.max(axis=0, keepdims=True))
    A /= A.sum(axis=0, keepdims=True)                                                  # normalised over the wrong axis
    return A.sum(axis=0) / Qw.shape[0]


def scores_sum_not_mean(Qw, K, softmax_scale=None):
    Qw, K = np.asarray(Qw, float), np.asarray(K, float)
    scale = 1.0 / math.sqrt(Qw.shape[1]) if not softmax_scale else float(softmax_scale)
    A, _ = orc.softmax_rows(scale * (Qw @ K.T))
    return A.sum(axis=0)


def select_variant(tie_high=False, window_competes=False, smallest=False):
    def select(scores, pos, n_prev, window_pos, budget):
        scores, pos = np.asarray(scores, float), np.asarray(pos, np.int64)
        L = pos.shape[0]
        wabs = set(int(n_prev) + int(p) for p in window_pos)
        is_window = np.array([int(p) in wabs for p in pos], dtype=bool)
        cand = np.arange(L) if window_competes else np.nonzero(~is_window)[0]
        kprime = len(cand) if budget == orc.KEEP_ALL else min(int(budget), len(cand))
        key = scores[cand] if smallest else -scores[cand]
        order = np.lexsort((-pos[cand] if tie_high else pos[cand], key))
        keep = np.zeros(L, dtype=bool)
        keep[cand[order[:kprime]]] = True
        keep |= is_window
        return np.nonzero(keep)[0]
    return select


def pool_divides_by_neighbours_present(scores, kernel):
    s = np.asarray(scores, float)
    k = int(kernel)
    if k <= 1:
        return s.copy()
    r = k // 2
    return np.array([s[max(i - r, 0):i + r + 1].mean() for i in range(len(s))])


def pool_one_sided(scores, kernel):
    s = np.asarray(scores, float)
    k = int(kernel)
    if k <= 1:
        return s.copy()
    padded = np.concatenate([s, np.zeros(k - 1)])
    return np.array([padded[i:i + k].sum() / k for i in range(len(s))])               # window not centred


def recent_sinks_on_top(pos, budget, n_sink=0):
    pos = np.asarray(pos, np.int64)
    L = pos.shape[0]
    if budget == orc.KEEP_ALL or budget >= L:
        return np.arange(L)
    sink = pos < int(n_sink)
    others = np.nonzero(~sink)[0]
    order = np.argsort(-pos[others], kind="stable")
    keep = np.zeros(L, dtype=bool)
    keep[others[order[:int(budget)]]] = True                                           # sinks not counted in the budget
    keep |= sink
    return np.nonzero(keep)[0]


def recent_keeps_oldest(pos, budget, n_sink=0):
    pos = np.asarray(pos, np.int64)
    L = pos.shape[0]
    if budget == orc.KEEP_ALL or budget >= L:
        return np.arange(L)
    sink = pos < int(n_sink)
    others = np.nonzero(~sink)[0]
    keep = np.zeros(L, dtype=bool)
    keep[others[:max(int(budget) - int(sink.sum()), 0)]] = True
    keep |= sink
    return np.nonzero(keep)[0]


def stats_topk_over_everything(Q, K, pos, n_prev, topk_prime, query_stride=1, softmax_scale=None):
    Q = np.asarray(Q, float)[:: int(query_stride)]
    K, pos = np.asarray(K, float), np.asarray(pos, np.int64)
    scale = 1.0 / math.sqrt(Q.shape[1]) if not softmax_scale else float(softmax_scale)
    A, _ = orc.softmax_rows(scale * (Q @ K.T))
    cur = pos >= int(n_prev)
    kk = min(int(topk_prime), A.shape[1])
    t = np.sort(A, axis=1)[:, A.shape[1] - kk:].sum(axis=1) if kk > 0 else np.zeros(Q.shape[0])   # not history only
    return float(A[:, cur].sum(axis=1).sum()), float(t.sum()), int(Q.shape[0])


def stats_current_map_off_by_one(Q, K, pos, n_prev, topk_prime, query_stride=1, softmax_scale=None):
    return ORIGINAL["layer_stats_slice"](Q, K, pos, int(n_prev) + 1, topk_prime, query_stride, softmax_scale)


def token_counts_without_width(sides_h, sides_w=None):
    return [int(h) * int(h) for h in sides_h] if sides_w is not None else ORIGINAL["scale_token_counts"](sides_h)


def cumulative_inclusive(n):
    out, acc = [], 0
    for x in n:
        acc += int(x)
        out.append(acc)                                                                # N_k instead of N_{k-1}
    return out + [acc]


def nca_over_window_not_sequence(Q, K, pos, n_prev, query_stride=1, softmax_scale=None):
    Q = np.asarray(Q, float)[:: int(query_stride)]
    K, pos = np.asarray(K, float), np.asarray(pos, np.int64)
    scale = 1.0 / math.sqrt(Q.shape[1]) if not softmax_scale else float(softmax_scale)
    A, _ = orc.softmax_rows(scale * (Q @ K.T))
    cur = pos >= int(n_prev)
    return float((A[:, cur].sum(axis=1) / cur.sum()).mean())                           # not divided by the sequence average


def head_shared_by_max(caches, Qws, window_pos, budget, pool_kernel=1):
    first = caches[0]
    per_head = np.stack([c.scores(Qw) for c, Qw in zip(caches, Qws)], axis=0)
    s = orc.pool_scores(per_head.max(axis=0), pool_kernel)                             # max over heads, not the mean
    keep = orc.select(s, first.pos, first.N[first.k - 1], window_pos, budget)
    for c in caches:
        c.adopt(keep)
    return first.pos.copy(), s


def budgets_growing_refiners(is_drafter, b_uniform, b_r0, delta):
    return ORIGINAL["make_budgets"](is_drafter, b_uniform, b_r0, -float(delta))          # decay with the wrong sign


def budgets_decay_from_zero(is_drafter, b_uniform, b_r0, delta):
    is_drafter = np.asarray(is_drafter, dtype=bool)
    shifted = ORIGINAL["make_budgets"](is_drafter, b_uniform, float(b_r0) + float(delta), delta)   # k counted from 0
    return shifted


def roles_highest_z(asi, n_drafters, mode=0, eps=1e-6, first_scale=1, last_scale=None):
    return ORIGINAL["assign_roles"](-np.asarray(asi, float), n_drafters, mode, eps, first_scale, last_scale)


def roles_rank_every_scale(asi, n_drafters, mode=0, eps=1e-6, first_scale=1, last_scale=None):
    asi = np.asarray(asi, float)
    return ORIGINAL["assign_roles"](asi, n_drafters, mode, eps, 0, asi.shape[1])


def budget_rounds_down(fraction, n):
    return int(math.floor(float(fraction) * orc.cached_positions(n)))


def cache_bytes_keys_only(n_layers, batch, n_heads, head_dim, elem_bytes, tokens_per_head_layer):
    return ORIGINAL["kv_cache_bytes"](n_layers, batch, n_heads, head_dim, elem_bytes, tokens_per_head_layer) // 2


def cached_positions_with_last_map(n):
    return sum(int(x) for x in n)


ORIGINAL = {name: getattr(orc, name) for name in (
    "make_budgets", "assign_roles", "budget_tokens", "kv_cache_bytes", "cached_positions",
    "attend", "window_scores", "select", "pool_scores", "select_recent", "layer_stats_slice", "scale_token_counts",
    "cumulative_token_counts", "normalized_current_attention")}

# (function replaced, the wrong version, pins that ought to notice: (test function, arguments) ...)
MUTANTS = [
    ("attend", attend_without_scale, [(pins.test_attend_vs_brute_force, (3, 7, 8))]),
    ("attend", attend_values_from_keys, [(pins.test_attend_vs_brute_force, (3, 7, 8)), (pins.test_attend_special_cases, ())]),
    ("attend", attend_lse_without_max, [(pins.test_attend_vs_brute_force, (5, 21, 16))]),
    ("window_scores", scores_softmax_over_window_axis, [(pins.test_window_scores_vs_brute_and_invariants, ())]),
    ("window_scores", scores_sum_not_mean, [(pins.test_window_scores_vs_brute_and_invariants, ())]),
    ("select", select_variant(tie_high=True), [(pins.test_select_ties_and_limits, ())]),
    ("select", select_variant(window_competes=True), [(pins.test_select_is_the_best_subset_by_exhaustive_search, ())]),
    ("select", select_variant(smallest=True), [(pins.test_select_is_the_best_subset_by_exhaustive_search, ())]),
    ("pool_scores", pool_divides_by_neighbours_present, [(pins.test_pool_scores_against_brute_force_and_closed_forms, ())]),
    ("pool_scores", pool_one_sided, [(pins.test_pool_scores_against_brute_force_and_closed_forms, ())]),
    ("select_recent", recent_sinks_on_top, [(pins.test_select_recent_brute_force_and_count_rule, ())]),
    ("select_recent", recent_keeps_oldest, [(pins.test_select_recent_brute_force_and_count_rule, ())]),
    ("layer_stats_slice", stats_topk_over_everything, [(pins.test_layer_stats_invariants_and_uniform_closed_form, ()),
                                                       (pins.test_layer_stats_topk_vs_loops, ())]),
    ("layer_stats_slice", stats_current_map_off_by_one, [(pins.test_layer_stats_invariants_and_uniform_closed_form, ())]),
    ("scale_token_counts", token_counts_without_width, [(pins.test_token_count_closed_forms, ())]),
    ("cumulative_token_counts", cumulative_inclusive, [(pins.test_token_count_closed_forms, ()),
                                                       (pins.test_full_budget_equals_block_causal_attention, ())]),
    ("normalized_current_attention", nca_over_window_not_sequence, [(pins.test_normalized_current_attention_closed_forms, ())]),
    ("compress_head_shared", head_shared_by_max, [(pins.test_head_shared_compress_brute_force_and_special_cases, ())]),
    ("make_budgets", budgets_growing_refiners, [(pins.test_make_budgets_satisfies_eq4, ())]),
    ("make_budgets", budgets_decay_from_zero, [(pins.test_make_budgets_satisfies_eq4, ())]),
    ("assign_roles", roles_highest_z, [(pins.test_assign_roles, ())]),
    ("assign_roles", roles_rank_every_scale, [(pins.test_assign_roles, ())]),
    ("budget_tokens", budget_rounds_down, [(pins.test_table1_accounting, ()), (pins.test_make_budgets_satisfies_eq4, ())]),
    ("kv_cache_bytes", cache_bytes_keys_only, [(pins.test_table1_accounting, ()), (pins.test_table3_linear_in_batch, ())]),
    ("cached_positions", cached_positions_with_last_map, [(pins.test_token_count_closed_forms, ()), (pins.test_table1_accounting, ())]),
]


@pytest.mark.parametrize("name,wrong,detectors", MUTANTS, ids=[f"{m[0]}:{m[1].__name__}" for m in MUTANTS])
def test_a_planted_mistake_fails_a_pin(monkeypatch, name, wrong, detectors):
    for fn, args in detectors:            # sanity: the pins pass on the oracle as it stands
        fn(*args)
    monkeypatch.setattr(orc, name, wrong)
    caught = 0
    for fn, args in detectors:
        try:
            fn(*args)
        except AssertionError:
            caught += 1
        except Exception:
            caught += 1
    assert caught > 0, f"no pin noticed the mistake planted in {name} ({wrong.__name__})"
