"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs - attention outputs within the dtype's bound, kept index sets exact (or inside the stated
tie band), compacted rows bit-exact."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import scalekv_oracle as orc
from paper_2505_19602_b200 import binding, synth
from parity_util import ParityRun

pytestmark = pytest.mark.gpu


def randn_inputs(B, H, d, n, dtype, seed):
    def fn(layer, scale):
        g = torch.Generator().manual_seed(seed * 1000 + layer * 50 + scale)
        return tuple(torch.randn(B, H, n[scale], d, generator=g).to(dtype) for _ in range(3))
    return fn


def all_slices(n_layers, B, H):
    return [(l, b, h) for l in range(n_layers) for b in range(B) for h in range(H)]


def test_tiny_config_fp32_whole_map_window():
    """configs[0]: B 1, 1 layer, 4 heads, d 64, fp32, sides 1,2,4,8; window = whole current map;
    budget 16; compress also after the last scale so that eviction happens."""
    wl = synth.WORKLOADS["tiny"]
    budgets = [[16] * 4]
    kv = binding.ScaleKV(1, 1, 4, 64, "f32", wl.sides, wl.sides, budgets, max_window=64)
    run = ParityRun(kv, "f32", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k), lambda k: None,
                    all_slices(1, 1, 4), compress_last=True).run()
    assert run.evictions == 4 and run.resyncs == 0
    assert kv.scalekv_lengths(0) == [[16 + 64] * 4]
    kv.close()


@pytest.mark.parametrize("budget", [2, 4, 8])
def test_tiny_variants_evict_early(budget):
    sides = (1, 2, 4, 8)
    n = orc.scale_token_counts(sides)
    budgets = [[budget] * 4]
    kv = binding.ScaleKV(1, 2, 3, 64, "f32", sides, sides, budgets, max_window=4)
    run = ParityRun(kv, "f32", sides, budgets, randn_inputs(2, 3, 64, n, torch.float32, 7 + budget),
                    lambda k: orc.window_centroids(sides[k], sides[k], 4), all_slices(1, 2, 3), compress_last=True).run()
    assert run.evictions > 0
    kv.close()


@pytest.mark.parametrize("page_tokens", [0, 16])
def test_bf16_ragged_multi_tile(page_tokens):
    """bf16, d 128: lengths that are not multiples of any tile or page, several pages per slice,
    a drafter-like and a refiner-like layer, explicit 16-token windows."""
    sides = (1, 2, 3, 5, 9, 14, 19)
    n = orc.scale_token_counts(sides)
    budgets = [[150] * len(sides), [21] * len(sides)]
    kv = binding.ScaleKV(2, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16, page_tokens=page_tokens)
    wl = synth.Workload("t", 2, 2, 2, 128, "bf16", sides, seed=11, n_drafters=1)
    run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(2, 2, 2)).run()
    assert run.evictions >= 8
    lens = kv.scalekv_lengths(1)
    assert lens == [[21 + 16 + n[-1]] * 2] * 2      # last scale is not compressed
    kv.close()


def test_keep_all_matches_full_attention():
    sides = (1, 2, 4, 6, 8, 12)
    n = orc.scale_token_counts(sides)
    budgets = [[binding.KEEP_ALL] * len(sides)]
    kv = binding.ScaleKV(1, 1, 2, 128, "bf16", sides, sides, budgets)
    run = ParityRun(kv, "bf16", sides, budgets, randn_inputs(1, 2, 128, n, torch.bfloat16, 3),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(1, 1, 2)).run()
    assert run.evictions == 0
    assert kv.scalekv_lengths(0) == [[sum(n)] * 2]
    pos = kv.scalekv_export_slice(0, 0, 1)
    assert pos.tolist() == list(range(sum(n)))
    kv.close()


def test_exact_ties_keep_lowest_positions():
    """Q = 0 makes every score bit-equal: the kept candidates are the lowest positions."""
    sides = (2, 4, 8)
    n = orc.scale_token_counts(sides)
    budgets = [[5] * 3]
    kv = binding.ScaleKV(1, 1, 2, 64, "f32", sides, sides, budgets, max_window=4)
    g = torch.Generator().manual_seed(5)
    for k in range(2):
        K = torch.randn(1, 2, n[k], 64, generator=g).cuda()
        V = torch.randn(1, 2, n[k], 64, generator=g).cuda()
        Q = torch.zeros(1, 2, n[k], 64).cuda()
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, K, V)
        O = kv.scalekv_attend(0, Q)
        wpos = orc.window_centroids(sides[k], sides[k], 4)
        kv.scalekv_compress(0, Q, wpos, qw_is_full_map=True)
        kv.scalekv_sync()
        if k == 0:
            assert kv.scalekv_export_slice(0, 0, 0).tolist() == [0, 1, 2, 3]
        else:
            base = 4
            want = sorted(set(list(range(5)) + [base + p for p in wpos]))
            # candidates exclude the window; the 5 lowest candidate positions are kept
            cands = [p for p in list(range(4)) + [base + i for i in range(16)] if p not in [base + q for q in wpos]]
            want = sorted(cands[:5] + [base + q for q in wpos])
            assert kv.scalekv_export_slice(0, 0, 1).tolist() == want
    # uniform attention: O is the mean of V over the cache
    kv.close()


def test_deterministic_and_reset():
    sides = (1, 2, 4, 8, 12)
    n = orc.scale_token_counts(sides)
    budgets = [[30] * 5]
    kv = binding.ScaleKV(1, 2, 2, 128, "bf16", sides, sides, budgets)
    inputs = randn_inputs(2, 2, 128, n, torch.bfloat16, 9)
    outs = []
    for rep in range(2):
        kv.scalekv_reset()
        rec = []
        for k in range(5):
            Q, K, V = (t.cuda() for t in inputs(0, k))
            torch.cuda.synchronize()
            kv.scalekv_append(0, k, K, V)
            rec.append(kv.scalekv_attend(0, Q))
            if k < 4:
                kv.scalekv_compress(0, Q, orc.window_centroids(sides[k], sides[k], 16), qw_is_full_map=True)
        kv.scalekv_sync()
        rec.append(kv.scalekv_export_slice(0, 1, 1))
        outs.append([t.cpu() for t in rec])
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    assert kv.scalekv_launch_count() > 0
    kv.close()


def test_call_order_and_argument_errors():
    sides = (1, 2, 4)
    kv = binding.ScaleKV(1, 1, 2, 64, "f32", sides, sides, [[4] * 3], max_window=4)
    x = torch.randn(1, 2, 1, 64, device="cuda")
    torch.cuda.synchronize()
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_attend(0, x)
    assert e.value.status == 2                      # BAD_STATE: no append yet
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_append(0, 1, x, x)
    assert e.value.status == 2                      # scales must ascend from 0
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_append(3, 0, x, x)
    assert e.value.status == 1
    kv.scalekv_append(0, 0, x, x)
    kv.scalekv_attend(0, x)
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_compress(0, x, [0, 0])           # not distinct / larger than the map
    assert e.value.status == 1
    kv.scalekv_compress(0, x, [0])
    kv.scalekv_sync()
    assert kv.scalekv_lengths(0) == [[1, 1]]
    kv.close()


def test_layer_stats_matches_oracle_and_recovers_planted_roles():
    sides = (1, 2, 4, 8, 12, 16, 20)
    n = orc.scale_token_counts(sides)
    N = orc.cumulative_token_counts(n)
    L_layers, B, H = 4, 1, 2
    wl = synth.Workload("t", L_layers, B, H, 128, "bf16", sides, seed=21, n_drafters=1)
    budgets = [[binding.KEEP_ALL] * len(sides)] * L_layers
    kv = binding.ScaleKV(L_layers, B, H, 128, "bf16", sides, sides, budgets)
    asi = np.zeros((L_layers, len(sides)))
    caches = {(l, b, h): orc.SliceCache(n, 128) for l in range(L_layers) for b in range(B) for h in range(H)}
    for k in range(len(sides)):
        for l in range(L_layers):
            Q, K, V = synth.scale_inputs(wl, l, k)
            Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
            torch.cuda.synchronize()
            kv.scalekv_append(l, k, Kd, Vd)
            car, htk = kv.scalekv_layer_stats(l, Qd, topk_prime=4, query_stride=2)
            car2, htk2, car_s, htk_s, nca_s = kv.scalekv_layer_stats_ex(l, Qd, topk_prime=4, query_stride=2)
            assert abs(car2 - car) < 1e-6 and abs(htk2 - htk) < 1e-6
            sc = st = cnt = 0
            for b in range(B):
                for h in range(H):
                    c = caches[(l, b, h)]
                    c.append(K[b, h].double().numpy(), V[b, h].double().numpy())
                    a = orc.layer_stats_slice(Q[b, h].double().numpy(), c.K, c.pos, N[k], 4, 2)
                    sc, st, cnt = sc + a[0], st + a[1], cnt + a[2]
                    # per slice, and the normalized current attention of Sec. 4.3 (at most L / n_k)
                    assert abs(car_s[b][h] - a[0] / a[2]) < 1e-4 and abs(htk_s[b][h] - a[1] / a[2]) < 1e-4
                    nca = orc.normalized_current_attention(Q[b, h].double().numpy(), c.K, c.pos, N[k], 2)
                    assert abs(nca_s[b][h] - nca) <= 1e-4 * len(c) / n[k]
            want_asi, want_car, want_htk = orc.asi_from_sums(sc, st, cnt)
            assert abs(car - want_car) < 1e-4 and abs(htk - want_htk) < 1e-4
            asi[l, k] = car * htk
    roles = binding.scalekv_assign_roles(asi, 1, mode=1)
    planted = synth.drafter_layers(wl)
    for k in range(3, len(sides) - 1):      # scales whose history exceeds K' by a wide margin
        assert np.nonzero(roles[:, k])[0].tolist() == planted
    kv.close()


def test_bf16_three_ctas_per_slice_and_window_paths():
    """n_k up to 576: a slice's queries span three CTAs (two with two query tiles, one with one).  Run
    once with the window logits recorded by attend and once with the stand-alone logits kernel."""
    sides = (2, 6, 12, 18, 24)
    n = orc.scale_token_counts(sides)
    budgets = [[100] * len(sides), [40] * len(sides)]
    wl = synth.Workload("t", 2, 1, 2, 128, "bf16", sides, seed=17, n_drafters=1)
    for patches in (16, 0):
        kv = binding.ScaleKV(2, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16, window_patches=patches)
        run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k),
                        lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(2, 1, 2), compress_last=True).run()
        assert run.evictions >= 12
        kv.close()


def test_compress_and_export_without_attend():
    """append -> compress with no attend in between: the library copies the map itself."""
    sides = (4, 8, 12)
    n = orc.scale_token_counts(sides)
    budgets = [[20] * 3]
    kv = binding.ScaleKV(1, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    g = torch.Generator().manual_seed(31)
    caches = [orc.SliceCache(n, 128) for _ in range(2)]
    for k in range(3):
        Q, K, V = (torch.randn(1, 2, n[k], 128, generator=g).to(torch.bfloat16) for _ in range(3))
        Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, Kd, Vd)
        wpos = orc.window_centroids(sides[k], sides[k], 16)
        if k == 1:
            pos, Kg, Vg = kv.scalekv_export_slice(0, 0, 1, with_kv=True)      # export straight after append
            assert len(pos) == caches[1].pos.shape[0] + n[k]
        kv.scalekv_compress(0, Qd, wpos, qw_is_full_map=True)
        kv.scalekv_sync()
        for h in range(2):
            c = caches[h]
            c.append(K[0, h].double().numpy(), V[0, h].double().numpy())
            want, _ = c.compress(Q[0, h].double().numpy()[wpos], wpos, budgets[0][k])
            pos, Kg, Vg = kv.scalekv_export_slice(0, 0, h, with_kv=True)
            assert np.array_equal(pos.numpy(), want)
            assert np.array_equal(Kg.double().numpy(), c.K) and np.array_equal(Vg.double().numpy(), c.V)
    kv.close()


def test_full_size_single_layer_sampled_slices():
    """configs[1] at full size (B 8, H 16, 13 scales, 10 % budget) in the launch configuration the
    benchmark uses; the oracle follows three sampled slices through the whole pass."""
    wl = synth.WORKLOADS["layer2b"]
    n = wl.n_tokens
    b10 = orc.budget_tokens(0.10, n)
    budgets = [[b10] * wl.n_scales]
    kv = binding.ScaleKV(1, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = [(0, 0, 0), (0, 3, 7), (0, 7, 15)]
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices).run()
    assert run.evictions == 3 * 5          # compress evicts at scales 8..12 (1-based) of the 13
    assert kv.scalekv_lengths(0)[7][15] == b10 + 16 + n[-1]
    kv.close()


def sampled_slices(wl, planted, count):
    """`count` slices spread over drafter and refiner layers (first, last and layers in between), first / last
    batch element and head, and seeded ones in between."""
    refiners = [l for l in range(wl.n_layers) if l not in planted]
    layers = [planted[0], refiners[0], planted[-1], refiners[-1], 0, 1, wl.n_layers - 2, wl.n_layers - 1]
    rng = np.random.default_rng(wl.seed)
    out, corners = [], [(0, 0), (wl.batch - 1, wl.n_heads - 1), (0, wl.n_heads - 1), (wl.batch - 1, 0)]
    i = 0
    while len(out) < count:
        l = layers[i % len(layers)] if i < 2 * len(layers) else int(rng.integers(wl.n_layers))
        b, h = corners[i % 4] if i < 8 else (int(rng.integers(wl.batch)), int(rng.integers(wl.n_heads)))
        if (l, b, h) not in out:
            out.append((l, b, h))
        i += 1
    return out


def test_full_size_pass_pipelined_16_slices():
    """configs[2] at full size (32 layers, B 8, H 16, 13 scales, drafter / refiner budgets of 30 % / 3 %, planted
    roles) in the execution mode the benchmark times: one scalekv_step per layer and scale, compress on the side
    stream, no host synchronisation inside a scale-step.  The oracle follows 16 slices (drafter and refiner
    layers, first and last batch element and head) through the whole pass, log-sum-exp included."""
    wl = synth.WORKLOADS["pass2b"]
    n = wl.n_tokens
    planted = synth.drafter_layers(wl)
    bd, br = orc.budget_tokens(0.30, n), orc.budget_tokens(0.03, n)
    budgets = [[bd if l in planted else br] * wl.n_scales for l in range(wl.n_layers)]
    kv = binding.ScaleKV(wl.n_layers, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = sampled_slices(wl, planted, 16)
    assert {s[0] for s in slices} & set(planted) and {s[0] for s in slices} - set(planted)
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices, check_lse=True).run_pipelined("eager")
    print("config 3, pipelined:", run.summary())
    assert run.evictions > 0 and run.compared == 16 * wl.n_scales
    kv.close()


def test_8b_class_full_40_layers_pipelined_8_slices():
    """configs[3] with all 40 layers and 32 heads (the page plan the benchmark runs) at the 10 / 30 drafter /
    refiner split, pipelined like the benchmark; the oracle follows 8 slices, attention on 1 024 evenly spaced
    rows of the large maps."""
    wl = synth.WORKLOADS["pass8b"]
    n = wl.n_tokens
    planted = synth.drafter_layers(wl)
    bd, br = orc.budget_tokens(0.30, n), orc.budget_tokens(0.03, n)
    budgets = [[bd if l in planted else br] * wl.n_scales for l in range(wl.n_layers)]
    kv = binding.ScaleKV(wl.n_layers, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = sampled_slices(wl, planted, 8)
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices, check_lse=True,
                    max_rows=1024).run_pipelined("eager")
    print("config 4, pipelined:", run.summary())
    assert run.evictions > 0
    kv.close()


def test_hires_full_32_layers_pipelined_8_slices():
    """configs[4] with all 32 layers (16 scales up to 128 x 128) at the 10 % point of the sweep, pipelined like
    the benchmark; the oracle follows 8 slices, attention on 512 evenly spaced rows of the large maps."""
    wl = synth.WORKLOADS["hires"]
    n = wl.n_tokens
    refiner_pct = 0.10 / 3.25
    bd, br = orc.budget_tokens(round(10 * refiner_pct, 6), n), orc.budget_tokens(round(refiner_pct, 6), n)
    planted = synth.drafter_layers(wl)
    budgets = [[bd if l in planted else br] * wl.n_scales for l in range(wl.n_layers)]
    kv = binding.ScaleKV(wl.n_layers, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = sampled_slices(wl, planted, 8)
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices, check_lse=True,
                    max_rows=512).run_pipelined("eager")
    print("config 5, pipelined:", run.summary())
    assert run.evictions > 0
    kv.close()


def _ragged_five_layer_case():
    """Five layers with budgets from 0 to KEEP_ALL-like, odd map sizes, small pages: persistent and transient pages,
    evicting and non-evicting compressions, drafter- and refiner-like inputs all occur."""
    sides = (1, 2, 3, 5, 9, 14, 19, 23)
    budgets = [[150] * len(sides), [21] * len(sides), [60] * len(sides), [0] * len(sides), [400] * len(sides)]
    wl = synth.Workload("p", 5, 2, 2, 128, "bf16", sides, seed=37, n_drafters=2)
    return sides, budgets, wl


@pytest.mark.parametrize("mode", ["eager", "graph"])
@pytest.mark.parametrize("page_tokens", [0, 32])
def test_pipelined_scale_steps_match_oracle(mode, page_tokens):
    """The benchmark's execution mode against the oracle on a small ragged case, every slice followed: compress
    of layer l runs on the side stream under attend of layer l + 1, layers l and l + 2 share a transient page
    set and a logit buffer, and the host only synchronises between scale-steps - eager, and with every
    scale-step replayed from a CUDA graph."""
    sides, budgets, wl = _ragged_five_layer_case()
    kv = binding.ScaleKV(5, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16, page_tokens=page_tokens)
    run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(5, 2, 2)).run_pipelined(mode)
    print("pipelined", mode, run.summary())
    assert run.evictions >= 40 and run.resyncs == 0
    kv.close()


def test_whole_pass_graph_replay_matches_oracle():
    """What the benchmark's timed region does - one CUDA graph of the whole pass, replayed - against the oracle:
    every layer's output of every scale and the store every slice is left with."""
    sides, budgets, wl = _ragged_five_layer_case()
    kv = binding.ScaleKV(5, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(5, 2, 2)).run_graph_pass()
    print("whole-pass graph:", run.summary())
    assert run.evictions >= 40 and run.compared == 20 * len(sides)
    kv.close()


def test_8b_class_shape_full_cache_and_budget_sampled_slices():
    """configs[3] (B 8, H 32, 13 scales): slices are independent, so two of the 40 layers stand for the
    pass - one with the full cache, one at the refiner budget; the oracle follows two slices of each."""
    wl8 = synth.WORKLOADS["pass8b"]
    wl = synth.Workload("pass8b-2", 2, wl8.batch, wl8.n_heads, 128, "bf16", wl8.sides, seed=wl8.seed, n_drafters=1)
    n = wl.n_tokens
    br = orc.budget_tokens(0.03, n)
    budgets = [[binding.KEEP_ALL] * wl.n_scales, [br] * wl.n_scales]
    kv = binding.ScaleKV(2, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = [(0, 0, 0), (0, 7, 31), (1, 3, 17), (1, 6, 2)]
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices, check_lse=False,
                    max_rows=1024).run()
    assert run.evictions > 0
    assert kv.scalekv_lengths(0)[7][31] == sum(n)
    kv.close()


def test_hires_16_scales_sampled_slices():
    """configs[4] (B 4, H 16, 16 scales up to 128 x 128): one drafter and one refiner layer at the 10 %
    point of the sweep; attention compared on evenly spaced query rows of the large maps."""
    wlh = synth.WORKLOADS["hires"]
    wl = synth.Workload("hires-2", 2, wlh.batch, wlh.n_heads, 128, "bf16", wlh.sides, seed=wlh.seed, n_drafters=1)
    n = wl.n_tokens
    refiner_pct = 0.10 / 3.25
    bd, br = orc.budget_tokens(round(10 * refiner_pct, 6), n), orc.budget_tokens(round(refiner_pct, 6), n)
    planted = synth.drafter_layers(wl)
    budgets = [[bd if l in planted else br] * wl.n_scales for l in range(2)]
    kv = binding.ScaleKV(2, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = [(0, 0, 0), (1, 3, 15)]
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices, check_lse=False,
                    max_rows=512).run()
    assert run.evictions > 0
    kv.close()


def test_strided_views_of_a_packed_qkv_tensor():
    """Q, K, V as strided views of one packed [B, n, 3, H, d] activation tensor (token stride 3 H d, head
    stride d), O into a strided view as well: the tensor maps and the copy kernels take strides."""
    sides = (3, 7, 13, 17)
    n = orc.scale_token_counts(sides)
    B, H, d = 2, 3, 128
    budgets = [[60] * len(sides)]
    kv = binding.ScaleKV(1, B, H, d, "bf16", sides, sides, budgets, max_window=16)
    g = torch.Generator().manual_seed(77)
    caches = {(b, h): orc.SliceCache(n, d) for b in range(B) for h in range(H)}
    worst = 0.0
    for k in range(len(sides)):
        packed = torch.randn(B, n[k], 3, H, d, generator=g).to(torch.bfloat16)
        pd = packed.cuda()
        Q, K, V = (pd[:, :, i].permute(0, 2, 1, 3) for i in range(3))          # [B, H, n, d] views, not contiguous
        assert not Q.is_contiguous()
        Obuf = torch.zeros(B, n[k], H, d, dtype=torch.bfloat16, device="cuda")
        O = Obuf.permute(0, 2, 1, 3)
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, K, V)
        kv.scalekv_attend(0, Q, O)
        wpos = orc.window_centroids(sides[k], sides[k], 16)
        if k + 1 < len(sides):
            kv.scalekv_compress(0, Q, wpos, qw_is_full_map=True)
        kv.scalekv_sync()
        for b in range(B):
            for h in range(H):
                c = caches[(b, h)]
                qh, kh, vh = (packed[b, :, i, h].double().numpy() for i in range(3))
                c.append(kh, vh)
                Oo, _ = c.attend(qh)
                worst = max(worst, float(np.max(np.abs(Oo - Obuf[b, :, h].double().cpu().numpy()))))
                if k + 1 < len(sides):
                    want, _ = c.compress(qh[wpos], wpos, budgets[0][k])
                    pos, Kg, Vg = kv.scalekv_export_slice(0, b, h, with_kv=True)
                    assert np.array_equal(pos.numpy(), want)
                    assert np.array_equal(Kg.double().numpy(), c.K) and np.array_equal(Vg.double().numpy(), c.V)
    assert worst <= 2e-2, worst
    kv.close()


def test_budget_zero_keeps_only_the_window():
    """k^l = 0: every candidate is evicted, the window entries alone survive (and still attend correctly)."""
    sides = (2, 5, 9, 12)
    n = orc.scale_token_counts(sides)
    budgets = [[0] * len(sides)]
    kv = binding.ScaleKV(1, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    run = ParityRun(kv, "bf16", sides, budgets, randn_inputs(1, 2, 128, n, torch.bfloat16, 41),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(1, 1, 2), compress_last=True).run()
    assert run.evictions == 2 * (len(sides) - 1)        # the first map is its own window: nothing to evict
    assert kv.scalekv_lengths(0) == [[16, 16]]
    kv.close()


def test_whole_pass_replays_from_a_cuda_graph():
    """reset + every append / attend / compress of a pass captured on stream_main (compress forks to
    stream_side inside the capture) replays to the same outputs and the same kept sets as eager calls."""
    from paper_2505_19602_b200 import pipeline

    sides = (1, 2, 4, 8, 12, 16, 20)
    wl = synth.Workload("g", 3, 2, 2, 128, "bf16", sides, seed=23, n_drafters=1)
    budgets = [[120] * len(sides), [30] * len(sides), [60] * len(sides)]
    kv = binding.ScaleKV(3, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    inputs = pipeline.PassInputs(wl)
    windows = pipeline.windows_for(sides, 16)
    pipeline.run_pass(kv, inputs, windows)
    kv.scalekv_sync()
    want_O = inputs.O.clone()
    want_pos = [kv.scalekv_export_slice(l, 1, 1).clone() for l in range(3)]
    g = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(g, stream=kv.stream_main):
        pipeline.run_pass(kv, inputs, windows)
        kv.scalekv_join()
    for _ in range(2):
        inputs.O.zero_()
        torch.cuda.synchronize()
        with torch.cuda.stream(kv.stream_main):
            g.replay()
        torch.cuda.synchronize()
        assert torch.equal(inputs.O, want_O)
        for l in range(3):
            assert torch.equal(kv.scalekv_export_slice(l, 1, 1), want_pos[l])
    kv.close()


def test_budget_table_from_eq4_with_global_roles_and_refiner_decay():
    """Budgets that differ per (layer, scale): roles ranked over all pairs (the printed form of the
    drafter selection), refiner budgets decaying with the scale, drafters taking what the refiners save."""
    sides = (1, 2, 4, 6, 8, 12, 16)
    n = orc.scale_token_counts(sides)
    L_layers = 4
    rng = np.random.default_rng(5)
    asi = rng.random((L_layers, len(sides))) * 0.2
    roles = binding.scalekv_assign_roles(asi, 7, mode=0)
    assert np.array_equal(roles, orc.assign_roles(asi, 7, 0))
    table = binding.scalekv_make_budgets(roles, 40, 30, 3)
    assert np.array_equal(table, orc.make_budgets(roles, 40, 30, 3))
    budgets = [[int(x) for x in row] for row in table]
    assert len({b for row in budgets for b in row}) > 4            # really varies
    wl = synth.Workload("b", L_layers, 1, 2, 128, "bf16", sides, seed=29, n_drafters=1)
    kv = binding.ScaleKV(L_layers, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(L_layers, 1, 2)).run()
    assert run.evictions > 0
    kv.close()


def _kept_or_tie(got_pos, cache_pos_before, s, keep_slots, w_abs):
    """True when got_pos equals the oracle's kept positions or differs only inside the 1e-3 tie band."""
    want_pos = cache_pos_before[keep_slots]
    if np.array_equal(got_pos, want_pos):
        return True
    sel = np.zeros(len(cache_pos_before), dtype=bool)
    sel[keep_slots] = True
    sel &= ~np.isin(cache_pos_before, w_abs)
    boundary = s[sel].min()
    diff = np.setxor1d(got_pos, want_pos)
    idx = np.searchsorted(cache_pos_before, diff)
    return bool(np.all(np.abs(s[idx] - boundary) / max(abs(boundary), 1e-300) < 1e-3))


def test_pooled_importance_matches_oracle():
    """scalekv_compress_ex with a 7-wide average pooling of the importance along the key axis."""
    sides = (2, 5, 9, 14, 19)
    n = orc.scale_token_counts(sides)
    N = orc.cumulative_token_counts(n)
    budgets = [[70] * len(sides)]
    B, H = 1, 3
    kv = binding.ScaleKV(1, B, H, 128, "bf16", sides, sides, budgets, max_window=16)
    wl = synth.Workload("p", 1, B, H, 128, "bf16", sides, seed=33)
    caches = [orc.SliceCache(n, 128) for _ in range(H)]
    evictions = 0
    for k in range(len(sides)):
        Q, K, V = synth.scale_inputs(wl, 0, k)
        Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, Kd, Vd)
        O = kv.scalekv_attend(0, Qd)
        wpos = orc.window_centroids(sides[k], sides[k], 16)
        kv.scalekv_compress_ex(0, Qd, wpos, qw_is_full_map=True, policy="score", pool_kernel=7)
        kv.scalekv_sync()
        for h in range(H):
            c = caches[h]
            c.append(K[0, h].double().numpy(), V[0, h].double().numpy())
            Oo, _ = c.attend(Q[0, h].double().numpy())
            assert np.max(np.abs(Oo - O[0, h].double().cpu().numpy())) <= 2e-2
            before = c.pos.copy()
            s = orc.pool_scores(c.scores(Q[0, h].double().numpy()[wpos]), 7)
            keep = orc.select(s, c.pos, N[k], wpos, budgets[0][k])
            got = kv.scalekv_export_slice(0, 0, h).numpy().astype(np.int64)
            assert len(got) == len(keep)
            evictions += int(len(keep) < len(before))
            assert _kept_or_tie(got, before, s, keep, [N[k] + p for p in wpos]), (k, h)
            c.adopt_positions(got)
    assert evictions >= 6
    kv.close()


@pytest.mark.parametrize("n_sink", [0, 4])
def test_positional_policy_sliding_window_and_sinks(n_sink):
    """scalekv_compress_ex with the positional rule: exact (positions are distinct, no ties)."""
    sides = (2, 5, 9, 14, 19)
    n = orc.scale_token_counts(sides)
    budgets = [[50] * len(sides), [13] * len(sides)]
    B, H = 2, 2
    kv = binding.ScaleKV(2, B, H, 128, "bf16", sides, sides, budgets, max_window=16)
    wl = synth.Workload("r", 2, B, H, 128, "bf16", sides, seed=35)
    caches = {(l, b, h): orc.SliceCache(n, 128) for l in range(2) for b in range(B) for h in range(H)}
    for k in range(len(sides)):
        for l in range(2):
            Q, K, V = synth.scale_inputs(wl, l, k)
            Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
            torch.cuda.synchronize()
            kv.scalekv_append(l, k, Kd, Vd)
            O = kv.scalekv_attend(l, Qd)
            kv.scalekv_compress_ex(l, policy="recent", n_sink=n_sink)
            kv.scalekv_sync()
            for b in range(B):
                for h in range(H):
                    c = caches[(l, b, h)]
                    c.append(K[b, h].double().numpy(), V[b, h].double().numpy())
                    Oo, _ = c.attend(Q[b, h].double().numpy())
                    assert np.max(np.abs(Oo - O[b, h].double().cpu().numpy())) <= 2e-2
                    want = c.compress_recent(budgets[l][k], n_sink)
                    pos, Kg, Vg = kv.scalekv_export_slice(l, b, h, with_kv=True)
                    assert np.array_equal(pos.numpy(), want), (k, l, b, h)
                    assert np.array_equal(Kg.double().numpy(), c.K) and np.array_equal(Vg.double().numpy(), c.V)
    assert kv.scalekv_lengths(1) == [[13, 13], [13, 13]]
    kv.close()


def test_step_host_pipeline_matches_device_calls():
    """scalekv_step_host (pinned host buffers, double-buffered staging, copies on the library's own streams,
    one sync at the end) gives bit-identical outputs and kept sets to append / attend / compress on
    device tensors."""
    sides = (1, 2, 4, 8, 12, 16)
    n = orc.scale_token_counts(sides)
    L_layers, B, H, d = 3, 2, 2, 128
    wl = synth.Workload("e", L_layers, B, H, d, "bf16", sides, seed=37, n_drafters=1)
    budgets = [[90] * len(sides), [25] * len(sides), [50] * len(sides)]
    windows = [orc.window_centroids(a, a, 16) for a in sides]
    data = {(l, k): synth.scale_inputs(wl, l, k) for l in range(L_layers) for k in range(len(sides))}
    # device path
    kv = binding.ScaleKV(L_layers, B, H, d, "bf16", sides, sides, budgets, max_window=16)
    want_O = {}
    for k in range(len(sides)):
        for l in range(L_layers):
            Q, K, V = (t.cuda() for t in data[(l, k)])
            torch.cuda.synchronize()
            kv.scalekv_append(l, k, K, V)
            want_O[(l, k)] = kv.scalekv_attend(l, Q)
            if k + 1 < len(sides):
                kv.scalekv_compress(l, Q, windows[k], qw_is_full_map=True)
    kv.scalekv_sync()
    want_pos = [kv.scalekv_export_slice(l, 1, 0).clone() for l in range(L_layers)]
    want_O = {key: t.cpu() for key, t in want_O.items()}
    kv.close()
    # host path: everything enqueued, one sync
    kv = binding.ScaleKV(L_layers, B, H, d, "bf16", sides, sides, budgets, max_window=16)
    host = {key: tuple(t.pin_memory() for t in qkv) for key, qkv in data.items()}
    out = {key: torch.empty_like(qkv[0]).pin_memory() for key, qkv in data.items()}
    staging = torch.empty(8 * B * H * max(n) * d, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    for k in range(len(sides)):
        for l in range(L_layers):
            Qh, Kh, Vh = host[(l, k)]
            kv.scalekv_step_host(l, k, Qh, Kh, Vh, out[(l, k)], staging,
                                 window_pos=windows[k] if k + 1 < len(sides) else None)
    kv.scalekv_sync()
    for key in data:
        assert torch.equal(out[key], want_O[key]), key
    for l in range(L_layers):
        assert torch.equal(kv.scalekv_export_slice(l, 1, 0), want_pos[l])
    kv.close()


@pytest.mark.parametrize("pool_kernel", [1, 5])
def test_head_shared_importance_matches_oracle(pool_kernel):
    """scalekv_compress_ex with head_shared: the mean over heads of the per-head importance decides for
    all heads of a batch element; they keep identical entries, batch elements differ."""
    sides = (2, 5, 9, 14, 19)
    n = orc.scale_token_counts(sides)
    N = orc.cumulative_token_counts(n)
    budgets = [[60] * len(sides)]
    B, H = 2, 4
    kv = binding.ScaleKV(1, B, H, 128, "bf16", sides, sides, budgets, max_window=16)
    wl = synth.Workload("hs", 1, B, H, 128, "bf16", sides, seed=35)
    caches = [[orc.SliceCache(n, 128) for _ in range(H)] for _ in range(B)]
    evictions, batch_differs = 0, False
    for k in range(len(sides)):
        Q, K, V = synth.scale_inputs(wl, 0, k)
        Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, Kd, Vd)
        O = kv.scalekv_attend(0, Qd)
        wpos = orc.window_centroids(sides[k], sides[k], 16)
        kv.scalekv_compress_ex(0, Qd, wpos, qw_is_full_map=True, policy="score", pool_kernel=pool_kernel, head_shared=True)
        kv.scalekv_sync()
        kept_of_batch = []
        for b in range(B):
            for h in range(H):
                c = caches[b][h]
                c.append(K[b, h].double().numpy(), V[b, h].double().numpy())
                Oo, _ = c.attend(Q[b, h].double().numpy())
                assert np.max(np.abs(Oo - O[b, h].double().cpu().numpy())) <= 2e-2
            before = caches[b][0].pos.copy()
            per_head = np.stack([caches[b][h].scores(Q[b, h].double().numpy()[wpos]) for h in range(H)])
            s = orc.pool_scores(per_head.mean(axis=0), pool_kernel)
            keep = orc.select(s, before, N[k], wpos, budgets[0][k])
            got = [kv.scalekv_export_slice(0, b, h).numpy().astype(np.int64) for h in range(H)]
            for h in range(1, H):
                assert np.array_equal(got[h], got[0])          # exact: the heads share one decision
            assert len(got[0]) == len(keep)
            evictions += int(len(keep) < len(before))
            assert _kept_or_tie(got[0], before, s, keep, [N[k] + p for p in wpos]), (k, b)
            for h in range(H):
                caches[b][h].adopt_positions(got[0])
                pos, Kg, Vg = kv.scalekv_export_slice(0, b, h, with_kv=True)
                assert np.array_equal(Kg.double().numpy(), caches[b][h].K) and np.array_equal(Vg.double().numpy(), caches[b][h].V)
            kept_of_batch.append(got[0])
        batch_differs = batch_differs or not np.array_equal(kept_of_batch[0], kept_of_batch[1])
    assert evictions >= 4 and batch_differs
    kv.close()


def test_head_shared_importance_refuses_heads_that_diverged():
    """After a per-head compress the heads hold different entries: the head-shared rule reports a
    device check through the status word and leaves the store as it was."""
    sides = (2, 5, 9, 14)
    n = orc.scale_token_counts(sides)
    budgets = [[40] * len(sides)]
    kv = binding.ScaleKV(1, 1, 3, 128, "bf16", sides, sides, budgets, max_window=16)
    wl = synth.Workload("hd", 1, 1, 3, 128, "bf16", sides, seed=36)
    for k in range(len(sides)):
        Q, K, V = synth.scale_inputs(wl, 0, k, device="cuda")
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, K, V)
        kv.scalekv_attend(0, Q)
        wpos = orc.window_centroids(sides[k], sides[k], 16)
        if k < 3:
            kv.scalekv_compress(0, Q, wpos, qw_is_full_map=True)
            kv.scalekv_sync()
    kept = [kv.scalekv_export_slice(0, 0, h).numpy() for h in range(3)]
    assert any(not np.array_equal(kept[0], kept[h]) for h in (1, 2))
    kv.scalekv_compress_ex(0, Q, wpos, qw_is_full_map=True, policy="score", head_shared=True)
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_sync()
    assert e.value.status == binding.STATUS_NAMES.index("DEVICE_CHECK")
    kv.close()


@pytest.mark.parametrize("policy", ["score", "recent"])
def test_per_head_budgets_leave_a_ragged_store(policy):
    """scalekv_compress_ex with head_budgets: every head prunes to its own budget (0 keeps only the
    window, the table's value is the largest allowed), lengths differ between heads from then on and
    the next scales' attention and selection still match the oracle slice by slice."""
    sides = (2, 5, 9, 14, 19)
    n = orc.scale_token_counts(sides)
    N = orc.cumulative_token_counts(n)
    table = 70
    budgets = [[table] * len(sides)]
    per_scale = [[10, 40, 70, 0], [10, 40, 70, 0], [30, 30, 70, 5], [5, 40, 60, 0], [70, 1, 20, 33]]
    B, H = 2, 4
    kv = binding.ScaleKV(1, B, H, 128, "bf16", sides, sides, budgets, max_window=16)
    wl = synth.Workload("hb", 1, B, H, 128, "bf16", sides, seed=37)
    caches = [[orc.SliceCache(n, 128) for _ in range(H)] for _ in range(B)]
    ragged = False
    for k in range(len(sides)):
        Q, K, V = synth.scale_inputs(wl, 0, k)
        Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, Kd, Vd)
        O = kv.scalekv_attend(0, Qd)
        wpos = orc.window_centroids(sides[k], sides[k], 16)
        if policy == "score":
            kv.scalekv_compress_ex(0, Qd, wpos, qw_is_full_map=True, policy="score", head_budgets=per_scale[k])
        else:
            kv.scalekv_compress_ex(0, policy="recent", n_sink=3, head_budgets=per_scale[k])
        kv.scalekv_sync()
        lens = kv.scalekv_lengths(0)
        for b in range(B):
            for h in range(H):
                c = caches[b][h]
                c.append(K[b, h].double().numpy(), V[b, h].double().numpy())
                Oo, _ = c.attend(Q[b, h].double().numpy())
                assert np.max(np.abs(Oo - O[b, h].double().cpu().numpy())) <= 2e-2, (k, b, h)
                before = c.pos.copy()
                got = kv.scalekv_export_slice(0, b, h).numpy().astype(np.int64)
                if policy == "score":
                    s = c.scores(Q[b, h].double().numpy()[wpos])
                    keep = orc.select(s, before, N[k], wpos, per_scale[k][h])
                    assert len(got) == len(keep) == min(per_scale[k][h] + len(wpos), len(before))
                    assert _kept_or_tie(got, before, s, keep, [N[k] + p for p in wpos]), (k, b, h)
                else:
                    keep = orc.select_recent(before, per_scale[k][h], 3)
                    assert np.array_equal(got, before[keep]), (k, b, h)
                assert int(lens[b][h]) == len(got)
                c.adopt_positions(got)
                pos, Kg, Vg = kv.scalekv_export_slice(0, b, h, with_kv=True)
                assert np.array_equal(Kg.double().numpy(), c.K) and np.array_equal(Vg.double().numpy(), c.V)
        ragged = ragged or len({int(x) for x in lens[0]}) > 1
    assert ragged
    with pytest.raises(binding.ScaleKVError):      # above the table's value: the pages were not sized for it
        kv.scalekv_reset()
        Q, K, V = synth.scale_inputs(wl, 0, 0, device="cuda")
        kv.scalekv_append(0, 0, K, V)
        kv.scalekv_compress_ex(0, Q, [0, 1, 2, 3], qw_is_full_map=True, head_budgets=[71, 1, 1, 1])
    kv.close()


def test_doubled_batch_two_layers_sampled_slices():
    """The headline shape with the batch doubled (16 x 16 slices per layer), one drafter and one
    refiner layer at full size; the oracle follows slices from both halves of the batch."""
    wl = dataclasses.replace(synth.WORKLOADS["pass2b_cfg"], n_layers=2, n_drafters=1)
    n = wl.n_tokens
    planted = synth.drafter_layers(wl)
    bd, br = orc.budget_tokens(0.30, n), orc.budget_tokens(0.03, n)
    budgets = [[bd if l in planted else br] * wl.n_scales for l in range(wl.n_layers)]
    kv = binding.ScaleKV(wl.n_layers, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = [(0, 1, 3), (0, 15, 15), (1, 8, 0), (1, 12, 9)]
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices, check_lse=False).run()
    assert run.evictions > 0
    lens = kv.scalekv_lengths(planted[0])
    assert all(lens[b][h] == bd + 16 + n[-1] for b in (0, 15) for h in (0, 15))
    kv.close()


def run_random_configuration(seed, max_side=20):
    """One configuration drawn from a seeded generator, every slice followed by the oracle."""
    rng = np.random.default_rng(4000 + seed)
    K = int(rng.integers(3, 7))
    sides_h = sorted(int(x) for x in rng.choice(np.arange(1, max_side + 1), size=K, replace=False))
    if rng.random() < 0.5:
        sides_w = list(sides_h)
    else:
        sides_w = [max(1, h + int(rng.integers(-2, 4))) for h in sides_h]
    dtype, d = ("bf16", 128) if rng.random() < 0.75 else ("f32", 64)
    n_layers, B, H = int(rng.integers(1, 4)), int(rng.integers(1, 3)), int(rng.integers(1, 4))
    page_tokens = int(rng.choice([0, 16, 32, 64]))
    patches = int(rng.choice([4, 9, 16]))
    choices = [0, 3, 17, 50, 130, 400, binding.KEEP_ALL]
    budgets = [[int(rng.choice(choices)) for _ in range(K)] for _ in range(n_layers)]
    gain = float(rng.choice([1.0, 1.0, 3.0]))          # some runs with peaked attention
    kv = binding.ScaleKV(n_layers, B, H, d, dtype, sides_h, sides_w, budgets, max_window=16, page_tokens=page_tokens,
                         window_patches=patches)
    n = orc.scale_token_counts(sides_h, sides_w)
    gen = torch.Generator().manual_seed(9000 + seed)
    tdt = synth.torch_dtype(dtype)

    def inputs(l, k):
        Q = (gain * torch.randn(B, H, n[k], d, generator=gen)).to(tdt)
        Kt = torch.randn(B, H, n[k], d, generator=gen).to(tdt)
        V = torch.randn(B, H, n[k], d, generator=gen).to(tdt)
        return Q, Kt, V

    slices = [(l, b, h) for l in range(n_layers) for b in range(B) for h in range(H)]
    run = ParityRun(kv, dtype, sides_h, budgets, inputs, lambda k: orc.window_centroids(sides_h[k], sides_w[k], patches),
                    slices, compress_last=bool(rng.random() < 0.5), sides_w=sides_w).run()
    kv.close()
    return run


@pytest.mark.parametrize("seed", range(10))
def test_seeded_random_configurations(seed):
    """Shapes drawn from a seeded generator: number of scales, square and rectangular maps, layers, batch,
    heads, dtype, page size, window size, and a budget per (layer, scale) anywhere between 0 and KEEP_ALL
    (also growing again after a small one)."""
    run_random_configuration(seed)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_largest_window_of_64_centroids(dtype, d):
    """The largest observation window the library takes (64 rows = 8 x 8 patches), recorded by attend."""
    sides = (4, 10, 17, 24)
    n = orc.scale_token_counts(sides)
    budgets = [[100] * len(sides), [binding.KEEP_ALL, 30, 30, 30]]
    kv = binding.ScaleKV(2, 1, 2, d, dtype, sides, sides, budgets, max_window=64, window_patches=64)
    gen = torch.Generator().manual_seed(77)
    tdt = synth.torch_dtype(dtype)
    inputs = lambda l, k: tuple(torch.randn(1, 2, n[k], d, generator=gen).to(tdt) for _ in range(3))
    slices = [(l, 0, h) for l in range(2) for h in range(2)]
    run = ParityRun(kv, dtype, sides, budgets, inputs, lambda k: orc.window_centroids(sides[k], sides[k], 64), slices,
                    compress_last=True).run()
    assert len(orc.window_centroids(24, 24, 64)) == 64 and run.evictions >= 8
    kv.close()


@pytest.mark.parametrize("name,wrong", [("attend", "attend_without_scale"), ("select", "select_smallest"),
                                        ("window_scores", "scores_sum_not_mean")])
def test_parity_harness_notices_a_wrong_oracle(monkeypatch, name, wrong):
    """The comparison itself must bite: with a mistake planted in the oracle (CPU side only) the same
    run that passes otherwise has to fail."""
    import test_oracle_mutations as mut
    sides = (2, 5, 9, 14)
    n = orc.scale_token_counts(sides)
    budgets = [[40] * len(sides)]

    def run():
        kv = binding.ScaleKV(1, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16)
        gen = torch.Generator().manual_seed(5)
        inputs = lambda l, k: tuple(torch.randn(1, 2, n[k], 128, generator=gen).to(torch.bfloat16) for _ in range(3))
        try:
            ParityRun(kv, "bf16", sides, budgets, inputs, lambda k: orc.window_centroids(sides[k], sides[k], 16),
                      [(0, 0, 0), (0, 0, 1)]).run()
        finally:
            kv.close()

    run()                                            # passes against the oracle as it stands
    fn = mut.select_variant(smallest=True) if wrong == "select_smallest" else getattr(mut, wrong)
    monkeypatch.setattr(orc, name, fn)
    with pytest.raises(AssertionError):
        run()


def test_one_call_step_equals_the_three_calls():
    """scalekv_step (append + attend + compress in one call) leaves exactly what the three calls leave."""
    from paper_2505_19602_b200 import pipeline
    sides = (2, 4, 7, 11, 16)
    wl = synth.Workload("st", 2, 2, 2, 128, "bf16", sides, seed=41)
    budgets = [[60] * len(sides), [25] * len(sides)]
    windows = pipeline.windows_for(sides, 16)
    results = []
    for three in (True, False):
        kv = binding.ScaleKV(2, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16)
        inputs = pipeline.PassInputs(wl)
        pipeline.run_pass(kv, inputs, windows, compress_last=True, three_calls=three)
        kv.scalekv_sync()
        kept = [kv.scalekv_export_slice(l, b, h, with_kv=True) for l in range(2) for b in range(2) for h in range(2)]
        results.append((inputs.O.clone(), kept, kv.scalekv_launch_count()))
        kv.close()
    (O3, kept3, n3), (O1, kept1, n1) = results
    assert torch.equal(O3, O1) and n3 == n1
    for a, b in zip(kept3, kept1):
        assert all(torch.equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("rule", ["sinks", "snapkv"])
def test_step_ex_equals_the_three_calls_for_the_comparison_rules(rule):
    """scalekv_step_ex (one call per step, the attend leaving out the copies nothing reads) leaves exactly what
    append, attend and scalekv_compress_ex leave: outputs, kept rows, values and positions."""
    from paper_2505_19602_b200 import pipeline
    sides = (2, 4, 7, 11, 16)
    wl = synth.Workload("sx", 2, 2, 2, 128, "bf16", sides, seed=43)
    budgets = [[60] * len(sides), [25] * len(sides)]
    if rule == "sinks":
        select, kind, windows = {"policy": "recent", "n_sink": 4}, "centroids", pipeline.windows_for(sides, 16)
    else:
        select, kind = {"policy": "score", "pool_kernel": 7}, "last"
        windows = [binding.scalekv_window_last(a, a, 16) for a in sides]
    results = []
    for three in (True, False):
        kv = binding.ScaleKV(2, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16, window_kind=kind)
        inputs = pipeline.PassInputs(wl)
        pipeline.run_pass(kv, inputs, windows, three_calls=three, select=select)
        kv.scalekv_sync()
        kept = [kv.scalekv_export_slice(l, b, h, with_kv=True) for l in range(2) for b in range(2) for h in range(2)]
        results.append((inputs.O.clone(), kept))
        kv.close()
    (O3, kept3), (O1, kept1) = results
    assert torch.equal(O3, O1)
    for a, b in zip(kept3, kept1):
        assert all(torch.equal(x, y) for x, y in zip(a, b))


def test_step_takes_surviving_rows_from_strided_caller_tensors():
    """A one-call step whose compress evicts leaves the current map in the caller's K and V and gathers the survivors
    from there: with K and V as strided views (token stride 3 d, head-major storage) it must keep exactly the rows, values
    and positions that the same step keeps from dense tensors, and what three separate calls (attend copies) keep."""
    from paper_2505_19602_b200 import pipeline
    sides = (3, 6, 10, 15)
    n = orc.scale_token_counts(sides)
    B, H, d = 2, 2, 128
    budgets = [[30] * len(sides)]
    windows = pipeline.windows_for(sides, 16)
    gen = torch.Generator().manual_seed(77)
    data = [[torch.randn(B, H, nk, d, generator=gen).to(torch.bfloat16).cuda() for _ in range(3)] for nk in n]

    def strided(t):
        big = torch.zeros(t.shape[1], t.shape[0], t.shape[2], 3 * d, dtype=t.dtype, device="cuda")
        big[..., d:2 * d] = t.permute(1, 0, 2, 3)
        return big[..., d:2 * d].permute(1, 0, 2, 3)          # [B, H, n, d] view: strides (n 3d, B n 3d, 3d, 1)

    kept = []
    for mode in ("dense", "strided", "three"):
        kv = binding.ScaleKV(1, B, H, d, "bf16", sides, sides, budgets, max_window=16)
        hold = []
        for k, nk in enumerate(n):
            Q, K, V = data[k]
            if mode == "strided":
                K, V = strided(K), strided(V)
                assert not K.is_contiguous()
            hold.append((K, V))
            O = torch.empty_like(Q)
            last = k + 1 == len(n)
            if mode == "three":
                kv.scalekv_append(0, k, K, V)
                kv.scalekv_attend(0, Q, O)
                if not last:
                    kv.scalekv_compress(0, Q, windows[k], qw_is_full_map=True)
            else:
                kv.scalekv_step(0, k, Q, K, V, O, window_pos=None if last else windows[k])
        kv.scalekv_sync()
        kept.append([kv.scalekv_export_slice(0, b, h, with_kv=True) for b in range(B) for h in range(H)])
        kv.close()
    for other in kept[1:]:
        for a, b in zip(kept[0], other):
            assert all(torch.equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("amp", [6.0, 12.0])
def test_dominant_keys_anywhere_in_the_first_tiles(amp):
    """Rows whose logit towards one key is 70 or 140 nats above the rest, that key sitting in the first
    columns of the first key tile, further inside it, in its second half, or in later tiles (a ragged one among them): whatever
    the kernel took as its first reference, the output is that key's value row (the second amplitude
    is beyond what exp2 can hold against a low reference)."""
    sides = (4, 20)
    n = orc.scale_token_counts(sides)
    d = 128
    budgets = [[binding.KEEP_ALL] * 2]
    kv = binding.ScaleKV(1, 1, 2, d, "bf16", sides, sides, budgets, max_window=16)
    gen = torch.Generator().manual_seed(123)
    # cache slots: 5 lies in the first map, the others in the second; 405 in its ragged last key tile (16 keys)
    hot_slots = [5, 40, 70, 100, 130, 300, 405]
    dirs = torch.randn(len(hot_slots), d, generator=gen)
    dirs = dirs / dirs.norm(dim=1, keepdim=True) * (d ** 0.5)      # |u|^2 = d: logit of a * u against u is a * sqrt(d)

    def inputs(l, k):
        Q = torch.randn(1, 2, n[k], d, generator=gen)
        K = torch.randn(1, 2, n[k], d, generator=gen)
        V = torch.randn(1, 2, n[k], d, generator=gen)
        if k == 1:
            for i in range(n[k]):
                Q[0, :, i] = dirs[i % len(hot_slots)]
        for s, u in zip(hot_slots, dirs):
            if k == 0 and s < n[0]:
                K[0, :, s] = amp * u
            if k == 1 and s >= n[0]:
                K[0, :, s - n[0]] = amp * u
        return Q.to(torch.bfloat16), K.to(torch.bfloat16), V.to(torch.bfloat16)

    run = ParityRun(kv, "bf16", sides, budgets, inputs, lambda k: orc.window_centroids(sides[k], sides[k], 16),
                    [(0, 0, 0), (0, 0, 1)], check_lse=True).run()
    kv.close()


def test_exact_ties_on_the_tensor_core_path():
    """bf16 x 128 with Q = 0: the window logits come out of the tensor core and the recorded-logits score
    kernel, every importance is bit-equal, so the kept candidates must be exactly the lowest positions (the
    oracle's rule), with no tie-band allowance used."""
    sides = (2, 5, 9, 14, 18)
    n = orc.scale_token_counts(sides)
    budgets = [[7] * len(sides), [130] * len(sides)]
    g = torch.Generator().manual_seed(91)

    def inputs(l, k):
        Kt = torch.randn(1, 2, n[k], 128, generator=g).to(torch.bfloat16)
        V = torch.randn(1, 2, n[k], 128, generator=g).to(torch.bfloat16)
        return torch.zeros(1, 2, n[k], 128, dtype=torch.bfloat16), Kt, V

    for mode in ("synced", "pipelined"):
        kv = binding.ScaleKV(2, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16)
        run = ParityRun(kv, "bf16", sides, budgets, inputs, lambda k: orc.window_centroids(sides[k], sides[k], 16),
                        all_slices(2, 1, 2), compress_last=True)
        run = run.run() if mode == "synced" else run.run_pipelined("eager")
        assert run.evictions >= 6 and run.resyncs == 0
        # layer 0 after the last compress: the 7 lowest positions that never were window entries, and the window
        pos = kv.scalekv_export_slice(0, 0, 1).tolist()
        assert len(pos) == 7 + 16 and pos[:4] == [0, 1, 2, 3]
        kv.close()


def test_bounded_wait_gives_up_and_reports_timeout():
    """The failure path of every device-side wait: a wait on a barrier that nothing arrives at runs out after its
    limit (50 ms here instead of 2 s), the kernel returns, the CTA's other warps see the abort flag, and
    scalekv_sync reports SCALEKV_ERR_TIMEOUT.  The context stays usable for host calls and the device for
    other contexts."""
    import time

    sides = (1, 2, 4)
    kv = binding.ScaleKV(1, 1, 2, 128, "bf16", sides, sides, [[4] * 3], max_window=16)
    kv.scalekv_sync()                                   # status clean
    t0 = time.perf_counter()
    gave_up, seen = kv.scalekv_selftest_wait(50)
    dt = time.perf_counter() - t0
    assert gave_up == 1 and seen == 1
    assert 0.04 <= dt < 1.5, dt                         # it waited for the limit, and not much longer
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_sync()
    assert e.value.status == 6                          # TIMEOUT, sticky
    # an attend launched now returns at once (its CTAs see the status) instead of computing on a failed context
    x = torch.randn(1, 2, 1, 128, device="cuda").to(torch.bfloat16)
    O = torch.full_like(x, 7.0)
    torch.cuda.synchronize()
    kv.scalekv_append(0, 0, x, x)
    kv.scalekv_attend(0, x, O)
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_sync()
    assert e.value.status == 6
    assert torch.all(O == 7.0)
    kv.close()
    # a fresh context on the same device works
    kv = binding.ScaleKV(1, 1, 2, 128, "bf16", sides, sides, [[4] * 3], max_window=16)
    kv.scalekv_append(0, 0, x, x)
    kv.scalekv_attend(0, x, O)
    kv.scalekv_sync()
    assert torch.allclose(O.float(), x.float(), atol=1e-2)     # one key: O = V
    kv.close()


def test_append_refuses_to_overwrite_a_layer_that_shares_its_transient_pages():
    """Layers l and l + 4 share a transient page set and a logit buffer.  An order of calls that would overwrite
    another layer's uncompressed map (append / attend of layer 0, then layer 4, before layer 0's compress) is
    refused with BAD_STATE and nothing is touched; after the compress it goes through, and the kept rows are the
    oracle's."""
    sides = (4, 12, 20)
    n = orc.scale_token_counts(sides)
    budgets = [[10] * 3] * 5                            # small persistent capacity: maps reach the transient pages
    kv = binding.ScaleKV(5, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    g = torch.Generator().manual_seed(3)
    data = {(l, k): tuple(torch.randn(1, 2, n[k], 128, generator=g).to(torch.bfloat16) for _ in range(3))
            for l in range(5) for k in range(3)}
    dev = {key: tuple(t.cuda() for t in v) for key, v in data.items()}
    torch.cuda.synchronize()
    wpos = [orc.window_centroids(a, a, 16) for a in sides]
    for l in range(5):                                  # scale 0: the whole map is the window, nothing evicted
        Q, K, V = dev[(l, 0)]
        kv.scalekv_step(l, 0, Q, K, V, torch.empty_like(Q), window_pos=wpos[0])
    for l in (0, 1):
        Q, K, V = dev[(l, 1)]
        kv.scalekv_append(l, 1, K, V)
        kv.scalekv_attend(l, Q)
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_append(4, 1, dev[(4, 1)][1], dev[(4, 1)][2])
    assert e.value.status == 2 and "layer 0" in str(e.value)
    kv.scalekv_compress(0, dev[(0, 1)][0], wpos[1], qw_is_full_map=True)
    Q, K, V = dev[(4, 1)]
    kv.scalekv_append(4, 1, K, V)                       # layer 0 is through: accepted
    kv.scalekv_attend(4, Q)
    kv.scalekv_compress(1, dev[(1, 1)][0], wpos[1], qw_is_full_map=True)
    kv.scalekv_compress(4, Q, wpos[1], qw_is_full_map=True)
    kv.scalekv_sync()
    for l in (0, 1, 4):
        for h in range(2):
            c = orc.SliceCache(n, 128)
            for k in range(2):
                Qh, Kh, Vh = (t[0, h].double().numpy() for t in data[(l, k)])
                c.append(Kh, Vh)
                c.compress(Qh[wpos[k]], wpos[k], 10)
            pos, Kg, Vg = kv.scalekv_export_slice(l, 0, h, with_kv=True)
            assert np.array_equal(pos.numpy(), c.pos)
            assert np.array_equal(Kg.double().numpy(), c.K) and np.array_equal(Vg.double().numpy(), c.V)
    kv.close()


def test_sinks_beyond_the_planned_capacity_are_refused():
    sides = (4, 12, 20)
    kv = binding.ScaleKV(1, 1, 2, 128, "bf16", sides, sides, [[10] * 3], max_window=16)
    x = {k: torch.randn(1, 2, a * a, 128, device="cuda").to(torch.bfloat16) for k, a in enumerate(sides)}
    torch.cuda.synchronize()
    kv.scalekv_append(0, 0, x[0], x[0])
    kv.scalekv_attend(0, x[0])
    kv.scalekv_compress_ex(0, policy="recent", n_sink=4)
    kv.scalekv_append(0, 1, x[1], x[1])
    kv.scalekv_attend(0, x[1])
    with pytest.raises(binding.ScaleKVError) as e:
        kv.scalekv_compress_ex(0, policy="recent", n_sink=150)      # 150 sinks, pages planned for 10 + 16 entries
    assert e.value.status == 3
    kv.scalekv_compress_ex(0, policy="recent", n_sink=4)
    kv.scalekv_sync()
    assert kv.scalekv_lengths(0) == [[10, 10]]
    kv.close()


def test_compress_as_three_launches_matches_oracle():
    """The one-launch compress is what every other test runs; here the same ragged case goes through the three
    separate kernels (importance; selection; pruning over 8 CTAs per slice), the path that slices too long for
    one CTA's shared memory take."""
    sides, budgets, wl = _ragged_five_layer_case()
    kv = binding.ScaleKV(5, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(5, 2, 2), compress_last=True)
    run.separate_kernels = True
    run.run()
    assert run.evictions >= 40 and run.resyncs == 0
    kv.close()


@pytest.mark.parametrize("policy", ["sliding", "sinks", "snapkv", "pyramid"])
@pytest.mark.parametrize("mode", ["synced", "pipelined"])
def test_comparison_policies_match_oracle(policy, mode):
    """The four comparison rules of Sec. 4.1 as configurations of the same store, each against its oracle
    statement on the ragged five-layer case, step by step and in the benchmark's pipelined mode: sliding window
    and sinks + recent (positional), the SnapKV-like rule (observed by the last 16 rows of the map, importance
    pooled over 7 neighbouring keys, uniform table) and pyramid budgets (the same rule, the table falling with
    the layer index)."""
    sides, _, wl = _ragged_five_layer_case()
    K = len(sides)
    if policy in ("sliding", "sinks"):
        table = binding.scalekv_policy_budgets("uniform", 5, K, 76)
        window = lambda k: binding.scalekv_window_centroids(sides[k], sides[k], 16)     # ignored by the positional rules
        kind = "centroids"
    else:
        table = binding.scalekv_policy_budgets("uniform" if policy == "snapkv" else "pyramid", 5, K, 60, 6.0)
        assert np.array_equal(table, orc.policy_budgets("uniform" if policy == "snapkv" else "pyramid", 5, K, 60, 6.0))
        window = lambda k: orc.window_last(sides[k], sides[k], 16)
        kind = "last"
    budgets = [[int(x) for x in row] for row in table]
    kv = binding.ScaleKV(5, 2, 2, 128, "bf16", sides, sides, budgets, max_window=16, window_kind=kind)
    run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k), window, all_slices(5, 2, 2))
    if policy in ("sliding", "sinks"):
        run.policy, run.n_sink = "recent", (4 if policy == "sinks" else 0)
    else:
        run.pool_kernel = 7
    run = run.run() if mode == "synced" else run.run_pipelined("eager")
    print(policy, mode, run.summary())
    assert run.evictions >= 30
    if policy == "pyramid":
        lens = [kv.scalekv_lengths(l)[0][0] for l in range(5)]
        assert lens == sorted(lens, reverse=True) and lens[0] > lens[-1]         # the store really is pyramid-shaped
    kv.close()


def test_refiner_decay_table_on_the_headline_shape():
    """The paper's own budget constants on the 13-scale shape: 650 tokens per head and layer on average,
    B_r(0) = 600, refiner decay delta = 70 (Sec. 4.3, "Impact of Refiner Budget Decay Rate"; Eq. 4), with 8
    drafters per ranked scale.  The table differs from scale to scale and the refiners' budget is clamped at 0
    from scale 9 on (only the window survives); all 32 layers run pipelined like the benchmark, the oracle
    follows 8 slices."""
    wl = synth.WORKLOADS["pass2b"]
    planted = synth.drafter_layers(wl)
    roles = np.zeros((wl.n_layers, wl.n_scales), dtype=bool)
    roles[planted, 1:wl.n_scales - 1] = True                                      # scales 1 and K are not ranked
    table = binding.scalekv_make_budgets(roles, 650, 600, 70)
    assert np.array_equal(table, orc.make_budgets(roles, 650, 600, 70))
    refiner = [l for l in range(wl.n_layers) if l not in planted][0]
    assert table[refiner, 1] == 460 and table[refiner, 8] == 0 and table[planted[0], 8] == 2600 and table[refiner, 0] == 650
    budgets = [[int(x) for x in row] for row in table]
    kv = binding.ScaleKV(wl.n_layers, wl.batch, wl.n_heads, 128, "bf16", wl.sides, wl.sides, budgets, max_window=16)
    slices = sampled_slices(wl, planted, 8)
    run = ParityRun(kv, "bf16", wl.sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(wl.sides[k], wl.sides[k], 16), slices, check_lse=True,
                    max_rows=1024).run_pipelined("eager")
    print("650 / 600 / delta 70:", run.summary())
    assert run.evictions > 0
    assert kv.scalekv_lengths(refiner)[0][0] == 16 + wl.n_tokens[-1]              # window of scale 12 + the last map
    kv.close()


def test_4k_class_schedule_sampled_slices():
    """A schedule beyond configs[4]: 19 scales up to 256 x 256 (170 521 tokens, a cache of up to 98 000 entries
    per slice).  A slice no longer fits one CTA's shared memory, so the selection streams its keys from global
    memory and the pruning reads its keep list there.  One drafter and one refiner layer at the 10 % point
    (30.77 % / 3.077 % of the cached tokens), two heads, pipelined; attention compared on 192 rows per map."""
    sides = synth.SIDES_19
    wl = synth.Workload("uhd4k-2", 2, 1, 2, 128, "bf16", sides, seed=7, n_drafters=1)
    n = wl.n_tokens
    bd, br = orc.budget_tokens(0.3077, n), orc.budget_tokens(0.03077, n)
    assert bd == binding.scalekv_budget_tokens(0.3077, sides) and bd > 30000
    planted = synth.drafter_layers(wl)
    budgets = [[bd if l in planted else br] * wl.n_scales for l in range(2)]
    kv = binding.ScaleKV(2, 1, 2, 128, "bf16", sides, sides, budgets, max_window=16)
    run = ParityRun(kv, "bf16", sides, budgets, lambda l, k: synth.scale_inputs(wl, l, k, device="cuda"),
                    lambda k: orc.window_centroids(sides[k], sides[k], 16), all_slices(2, 1, 2), check_lse=True,
                    max_rows=192).run_pipelined("eager")
    print("4K-class:", run.summary())
    assert run.evictions > 0
    assert kv.scalekv_lengths(planted[0])[0][0] == bd + 16 + n[-1]
    kv.close()

