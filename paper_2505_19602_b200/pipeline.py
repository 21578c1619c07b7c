"""Drivers around the C-ABI context: the per-scale loop of one pass, offline role calibration and
the budget tables of the named workloads.  Only call sequencing lives here; all arithmetic runs
in the library."""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from . import binding, synth


def windows_for(sides, n_patches=16):
    """Observation-window raster indices for every scale (Sec. 3.3), from the library's helper."""
    return [binding.scalekv_window_centroids(a, a, n_patches) for a in sides]


def budget_table(wl: synth.Workload, roles, drafter_frac=0.30, refiner_frac=0.03):
    """budgets[l][k]: drafter or refiner budget by role (fractions of T_c = N_{K-1}, scalekv_budget_tokens)."""
    bd = binding.scalekv_budget_tokens(drafter_frac, wl.sides)
    br = binding.scalekv_budget_tokens(refiner_frac, wl.sides)
    return [[bd if roles[l][k] else br for k in range(wl.n_scales)] for l in range(wl.n_layers)]


def calibrate_roles(wl: synth.Workload, n_drafters, topk_prime=16, query_stride=16, batch=1, device=0):
    """Runs the workload's seeded inputs with a full cache (reduced batch) and collects the
    Attention Selectivity Index per (layer, scale) with scalekv_layer_stats (Eq. 2); returns
    (asi [L][K], is_drafter [L][K]) with the n_drafters lowest-Z layers per ranked scale (Eq. 3)."""
    cal = dataclasses.replace(wl, batch=batch)
    keep_all = [[binding.KEEP_ALL] * wl.n_scales for _ in range(wl.n_layers)]
    kv = binding.ScaleKV(wl.n_layers, batch, wl.n_heads, wl.head_dim, wl.dtype, wl.sides, wl.sides, keep_all,
                         max_window=min(wl.window, binding.MAX_WINDOW), device=device, side_stream=False)
    asi = np.zeros((wl.n_layers, wl.n_scales))
    dev = f"cuda:{device}"
    for k in range(wl.n_scales):
        stride = max(1, min(query_stride, wl.n_tokens[k] // 16))
        for l in range(wl.n_layers):
            Q, K, V = synth.scale_inputs(cal, l, k, device=dev)
            torch.cuda.synchronize()
            kv.scalekv_append(l, k, K, V)
            car, htk = kv.scalekv_layer_stats(l, Q, topk_prime, stride)
            asi[l, k] = car * htk
    kv.close()
    roles = binding.scalekv_assign_roles(asi, n_drafters, mode=1)
    return asi, roles


class PassInputs:
    """Device-resident Q/K/V of every (layer, scale) of a workload, generated once."""

    def __init__(self, wl: synth.Workload, device=0, share_layers=False):
        dev = f"cuda:{device}"
        self.wl = wl
        self.data = {}
        for l in range(wl.n_layers):
            for k in range(wl.n_scales):
                if share_layers and l > 0:
                    self.data[(l, k)] = self.data[(0, k)]
                else:
                    self.data[(l, k)] = synth.scale_inputs(wl, l, k, device=dev)
        n_max = max(wl.n_tokens)
        self.O = torch.empty(wl.batch, wl.n_heads, n_max, wl.head_dim, dtype=synth.torch_dtype(wl.dtype), device=dev)
        torch.cuda.synchronize()

    def bytes(self):
        seen, total = set(), 0
        for q, k, v in self.data.values():
            if q.data_ptr() in seen:
                continue
            seen.add(q.data_ptr())
            total += 3 * q.numel() * q.element_size()
        return total


def scale_step(kv: binding.ScaleKV, inputs: PassInputs, windows, k, compress_last=False, three_calls=False, select=None):
    """One scale-step: append -> attend -> compress of every layer at scale k (one scalekv_step per layer, or
    the three calls one by one with three_calls=True: the same launches; `select`: the options of a comparison policy,
    through scalekv_step_ex or, with three_calls, scalekv_compress_ex)."""
    wl = inputs.wl
    nk = wl.n_tokens[k]
    O = inputs.O[:, :, :nk, :]
    last = k + 1 == wl.n_scales
    do_compress = not last or compress_last
    wp = kv.window_array(windows[k]) if (do_compress and windows[k] is not None) else None
    for l in range(wl.n_layers):
        Q, K, V = inputs.data[(l, k)]
        if select is not None and not three_calls:
            kv.scalekv_step_ex(l, k, Q, K, V, O, compress=do_compress, window_pos=windows[k], **select)
            continue
        if select is not None:
            kv.scalekv_append(l, k, K, V)
            kv.scalekv_attend(l, Q, O)
            if do_compress:
                kv.scalekv_compress_ex(l, Q, windows[k], qw_is_full_map=True, **select)
            continue
        if not three_calls:
            kv.scalekv_step(l, k, Q, K, V, O, window_pos=wp, whole_map=do_compress and wp is None)
            continue
        kv.scalekv_append(l, k, K, V)
        kv.scalekv_attend(l, Q, O)
        if do_compress:
            if windows[k] is None:
                kv.scalekv_compress(l, Q, None)
            else:
                kv.scalekv_compress(l, Q, windows[k], qw_is_full_map=True)


def run_pass(kv: binding.ScaleKV, inputs: PassInputs, windows, compress_last=False, marks=None, three_calls=False, select=None):
    """One pass: reset, then scale_step for every scale.

    marks: a list that receives CUDA events recorded on stream_main before the reset, after it, and after
    every scale-step (2 + n_scales events), for per-scale-step latencies.
    select: options of scalekv_compress_ex (policy, pool_kernel, n_sink) for the comparison policies; the
    compress of every step then goes through that call.
    """
    def mark():
        if marks is not None:
            ev = torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(kv.stream_main):
                ev.record()
            marks.append(ev)

    mark()
    kv.scalekv_reset()
    mark()
    for k in range(inputs.wl.n_scales):
        scale_step(kv, inputs, windows, k, compress_last=compress_last, three_calls=three_calls, select=select)
        mark()


def pass_work(wl: synth.Workload, budgets, windows, recent=False, one_call_steps=True):
    """Algorithmic work of one pass, from the schedule alone.

    attend_flop       4 n_k L d per slice-step.
    attend_min_bytes  what attend must move: K and V of the L entries once, Q and O, plus - where it also
                      appends - the write of the current map's K/V rows and positions into the pages, and
                      the write of the w x L window logits where it records them (not after the last scale).
                      one_call_steps: the pass is made of scalekv_step calls, whose attend leaves the map in the
                      caller's tensors when the step's compress evicts and after the last scale.
    score_bytes       the score kernel: w x L logits and L positions in, L scores and L keys out (plus K read
                      by the stand-alone logits kernel when attend did not record the logits).
    select_bytes      the select kernel: L keys in, the keep list out.
    compress_bytes    the one-launch compress (score + select + compact of a slice by one CTA): the w x L logits and
                      L positions in, L scores out, the survivors' rows moved; keys and keep list stay on chip.
    compact_bytes     K and V rows (and positions) of the survivors, read and written (upper bound: which
                      rows already sit in place is unknown on the host).
    """
    n = wl.n_tokens
    d = wl.head_dim
    esz = 2 if wl.dtype == "bf16" else 4
    slices = wl.batch * wl.n_heads
    fused = wl.dtype == "bf16" and d == 128
    out = {"attend_flop": 0, "attend_min_bytes": 0, "score_bytes": 0, "compact_bytes": 0, "append_bytes": 0,
           "select_bytes": 0, "attend_launches": 0, "compress_bytes": 0, "compress_launches": 0}
    per_scale_flop = [0] * wl.n_scales
    for l in range(wl.n_layers):
        hist = 0
        for k in range(wl.n_scales):
            L = hist + n[k]
            w = len(windows[k]) if windows[k] is not None else n[k]
            wk = 0 if recent else w          # the positional rules have no window: their budget is the whole cache
            f = 4 * n[k] * L * d * slices
            out["attend_flop"] += f
            per_scale_flop[k] += f
            out["attend_min_bytes"] += (2 * L + 2 * n[k]) * d * esz * slices
            last = k + 1 == wl.n_scales
            evicts = (not last) and budgets[l][k] != binding.KEEP_ALL and budgets[l][k] < L - wk
            if fused:
                if not (one_call_steps and (last or evicts)):
                    out["attend_min_bytes"] += (2 * n[k] * d * esz + 4 * n[k]) * slices
                if not last:
                    out["attend_min_bytes"] += 4 * w * L * slices
            else:
                out["append_bytes"] += 2 * 2 * n[k] * d * esz * slices
            out["attend_launches"] += 1
            if k + 1 == wl.n_scales:
                break
            cand = L - wk
            b = budgets[l][k]
            if b != binding.KEEP_ALL and b < cand:
                if not fused:
                    out["score_bytes"] += L * d * esz * slices
                out["score_bytes"] += (4 * wk * L + 4 * L + 4 * L + 4 * L) * slices
                out["select_bytes"] += (4 * L + 4 * (b + wk)) * slices
                out["compact_bytes"] += (b + wk) * (2 * 2 * d * esz + 8) * slices
                # the one-launch compress: logits and positions in, scores out, the survivors' rows moved
                out["compress_bytes"] += ((4 * wk * L + 4 * L + (0 if recent else 4 * L)) + (b + wk) * (2 * 2 * d * esz + 8)) * slices
                out["compress_launches"] += 1
                hist = b + wk
            else:
                hist = L
    out["per_scale_flop"] = per_scale_flop
    return out
