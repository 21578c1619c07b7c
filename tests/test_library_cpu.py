"""CPU-only checks of the C-ABI library: it builds for sm_100a, loads, exports every symbol the
header declares, and its host-only helpers agree with the oracle.  No kernel is launched."""
import ctypes as C
import math

import numpy as np
import pytest

from oracle import scalekv_oracle as orc
from paper_2505_19602_b200 import binding

SIDES_13 = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)
SIDES_16 = SIDES_13 + (80, 96, 128)


@pytest.fixture(scope="module")
def lib():
    binding.build_library()
    return binding.load_library()


def test_exports_every_declared_symbol(lib):
    names = binding.exported_symbols()
    assert len(names) >= 20 and "scalekv_attend" in names and "scalekv_compress" in names
    for name in names:
        assert hasattr(lib, name), name


def test_window_centroids_match_oracle(lib):
    for a in SIDES_16:
        for n in (16, 4, 9, 1):
            assert binding.scalekv_window_centroids(a, a, n) == orc.window_centroids(a, a, n)
    assert binding.scalekv_window_centroids(6, 10, 16) == orc.window_centroids(6, 10, 16)


def test_assign_roles_and_budgets_match_oracle(lib):
    rng = np.random.default_rng(0)
    asi = rng.random((12, 7)) * 0.2
    for mode, nd in ((0, 9), (1, 3)):
        assert np.array_equal(binding.scalekv_assign_roles(asi, nd, mode), orc.assign_roles(asi, nd, mode))
    roles = orc.assign_roles(asi, 3, 1)
    for delta in (0, 20, 70):
        assert np.array_equal(binding.scalekv_make_budgets(roles, 650, 600, delta), orc.make_budgets(roles, 650, 600, delta))


def make_cfg(n_layers, B, H, d, dtype, sides, budgets, max_window=16, page_tokens=0):
    cfg = binding.scalekv_config()
    cfg.n_layers, cfg.batch, cfg.n_heads, cfg.head_dim, cfg.dtype = n_layers, B, H, d, dtype
    cfg.n_scales = len(sides)
    keep = (binding._i32_array(sides), binding._i32_array([x for r in budgets for x in r]))
    cfg.scale_h, cfg.scale_w, cfg.budgets = keep[0], keep[0], keep[1]
    cfg.max_window, cfg.page_tokens = max_window, page_tokens
    return cfg, keep


def test_query_sizes_accounting(lib):
    n13 = orc.scale_token_counts(SIDES_13)
    # full cache, one layer, B 8, H 16: K and V pages cover 10521 tokens per slice
    cfg, keep = make_cfg(1, 8, 16, 128, binding.BF16, SIDES_13, [[-1] * 13])
    pb, wb = C.c_size_t(), C.c_size_t()
    assert lib.scalekv_query_sizes(C.byref(cfg), C.byref(pb), C.byref(wb)) == 0
    pages = math.ceil(10521 / 128)
    kv_bytes = 128 * pages * 128 * 2 * 2 * 128
    assert kv_bytes <= pb.value <= kv_bytes * 1.05
    # 10 % drafter/refiner budgets need far less than the full cache
    bd, br = orc.budget_tokens(0.30, n13), orc.budget_tokens(0.03, n13)
    budgets = [[bd] * 13 if l < 8 else [br] * 13 for l in range(32)]
    cfg2, keep2 = make_cfg(32, 8, 16, 128, binding.BF16, SIDES_13, budgets)
    pb2 = C.c_size_t()
    assert lib.scalekv_query_sizes(C.byref(cfg2), C.byref(pb2), C.byref(wb)) == 0
    full32 = 32 * kv_bytes
    assert pb2.value < 0.2 * full32


def test_query_sizes_rejects_bad_configs(lib):
    pb, wb = C.c_size_t(), C.c_size_t()
    cfg, keep = make_cfg(1, 1, 4, 64, binding.BF16, (1, 2), [[-1, -1]])
    assert lib.scalekv_query_sizes(C.byref(cfg), C.byref(pb), C.byref(wb)) == 4      # UNSUPPORTED
    cfg, keep = make_cfg(1, 1, 4, 64, binding.F32, (1, 2), [[-1, -1]], max_window=65)
    assert lib.scalekv_query_sizes(C.byref(cfg), C.byref(pb), C.byref(wb)) == 1      # INVALID_ARG
    cfg, keep = make_cfg(1, 1, 4, 64, binding.F32, (1, 2), [[-1, -1]], page_tokens=48)
    assert lib.scalekv_query_sizes(C.byref(cfg), C.byref(pb), C.byref(wb)) == 1
    cfg, keep = make_cfg(1, 1, 4, 64, binding.F32, (1, 2), [[-1, -5]])
    assert lib.scalekv_query_sizes(C.byref(cfg), C.byref(pb), C.byref(wb)) == 1
    assert lib.scalekv_query_sizes(None, C.byref(pb), C.byref(wb)) == 1


def test_product_path_refuses_to_run_without_gpu():
    import torch

    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        binding.ScaleKV(1, 1, 4, 64, "f32", (1, 2), (1, 2), [[-1, -1]])


def test_budget_tokens_matches_oracle(lib):
    """The fraction -> tokens rule behind the ABI against the oracle's exact-rational version, on the fractions the
    workloads use (30 %, 3 %, 10 %, the 4 / 10 / 20 % sweep's drafter and refiner shares) and on .5 cases."""
    for sides in (SIDES_13, SIDES_16, (1, 2, 4, 8)):
        n = orc.scale_token_counts(sides)
        for f in (0.30, 0.03, 0.10, 0.04, 0.20, 0.0123, 0.123, 0.01231, 0.03077, 0.3077, 0.06154, 0.6154, 1.0, 0.0, 0.5):
            assert binding.scalekv_budget_tokens(f, sides) == orc.budget_tokens(f, n), (sides, f)
    assert binding.scalekv_budget_tokens(0.30, SIDES_13) == 1928        # 1927.5 rounds up
    assert binding.scalekv_budget_tokens(0.5, (1, 1, 1)) == 1 and binding.scalekv_budget_tokens(0.25, (1, 1, 1)) == 1


def test_comparison_policy_helpers_match_oracle(lib):
    for h, w, n in ((3, 5, 16), (8, 8, 16), (6, 10, 4), (1, 1, 16), (64, 64, 16)):
        assert binding.scalekv_window_last(h, w, n) == orc.window_last(h, w, n)
    for shape in ("uniform", "pyramid"):
        for L, b, beta in ((32, 627, 20.0), (40, 1300.5, 20.0), (5, 100, 4.0), (1, 77, 20.0), (6, 50, 1.0)):
            assert np.array_equal(binding.scalekv_policy_budgets(shape, L, 4, b, beta), orc.policy_budgets(shape, L, 4, b, beta))



def test_pass_work_counts_what_a_one_call_step_leaves_out():
    """The algorithmic byte count of attend (the bench's roofline traffic comes from it): same flop either way; with
    one-call steps the appended rows of evicting steps and of the last scale are not counted, and nobody records window
    logits after the last scale.  Checked against a count written out here for a two-scale, one-layer schedule."""
    from paper_2505_19602_b200 import pipeline, synth
    sides = (4, 12)                      # 16 and 144 tokens
    wl = synth.Workload("pw", 1, 1, 2, 128, "bf16", sides, seed=1)
    windows = [[0, 5], [3, 77]]          # two window rows per scale
    budgets = [[6, 6]]                   # scale 0: 16 - 2 candidates > 6: evicts; scale 1 is the last
    full = pipeline.pass_work(wl, budgets, windows, one_call_steps=False)
    step = pipeline.pass_work(wl, budgets, windows, one_call_steps=True)
    assert full["attend_flop"] == step["attend_flop"] == 4 * 128 * 2 * (16 * 16 + 144 * (8 + 144))
    row = 128 * 2
    kv_q_o = 2 * ((2 * 16 + 2 * 16) + (2 * (8 + 144) + 2 * 144)) * row          # K, V of L entries, Q and O, both slices
    logits = 2 * 4 * 2 * 16                                                   # w x L floats at scale 0 only
    appended = 2 * ((2 * 16 * row + 4 * 16) + (2 * 144 * row + 4 * 144))
    assert full["attend_min_bytes"] == kv_q_o + logits + appended
    assert step["attend_min_bytes"] == kv_q_o + logits                        # scale 0 evicts, scale 1 is the last
    assert full["compress_bytes"] == step["compress_bytes"] and step["compress_launches"] == 1
