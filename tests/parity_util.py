"""Shared driver of the GPU-vs-oracle parity tests: steps the CUDA library (through the C ABI)
and the CPU oracle through the same seeded inputs and compares them slice by slice."""
import numpy as np
import torch

from oracle import scalekv_oracle as orc

TOL = {"bf16": 2e-2, "f32": 1e-4}   # max-abs bound on attention outputs
REL = {"bf16": 2.0 ** -7, "f32": 0.0}    # relative part of the bound (see _compare_slice)
TIE_BAND = 1e-3                     # relative score band inside which either choice is accepted


def to64(t):
    return t.detach().to("cpu", torch.float64).numpy()


class ParityRun:
    """Runs `sides` scales of one configuration on both sides.

    inputs_fn(layer, scale) -> (Q, K, V) CPU or CUDA tensors [B, H, n_k, d] in the storage dtype.
    window_fn(scale) -> list of raster indices, or None for "whole current map".
    slices: list of (layer, b, h) that the oracle follows.
    """

    def __init__(self, kv, dtype, sides, budgets, inputs_fn, window_fn, slices, compress_last=False,
                 check_lse=True, max_rows=None, sides_w=None):
        self.kv, self.dtype, self.sides = kv, dtype, list(sides)
        self.budgets, self.inputs_fn, self.window_fn = budgets, inputs_fn, window_fn
        self.slices, self.compress_last, self.check_lse = slices, compress_last, check_lse
        self.max_rows = max_rows      # attention is compared on at most this many evenly spaced query rows per map
        self.n = orc.scale_token_counts(self.sides, sides_w)      # sides = heights when sides_w is given
        self.caches = {s: orc.SliceCache(self.n, kv.head_dim) for s in slices}
        self.resyncs = 0
        self.max_err = 0.0
        self.max_tol = 0.0
        self.max_lse_err = 0.0
        self.evictions = 0

    def run(self):
        kv = self.kv
        layers = sorted({s[0] for s in self.slices}) if kv.n_layers > 1 else [0]
        all_layers = range(kv.n_layers)
        for k, nk in enumerate(self.n):
            wpos = self.window_fn(k)
            for l in all_layers:
                Q, K, V = self.inputs_fn(l, k)
                Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
                lse = torch.empty(kv.batch, kv.n_heads, nk, dtype=torch.float32, device="cuda")
                torch.cuda.synchronize()
                kv.scalekv_append(l, k, Kd, Vd)
                O = kv.scalekv_attend(l, Qd, lse=lse)
                do_compress = (k + 1 < len(self.n)) or self.compress_last
                if do_compress:
                    if wpos is None:
                        kv.scalekv_compress(l, Qd, None)
                    else:
                        # alternate between the two ways of passing the window rows
                        if (k + l) % 2 == 0:
                            kv.scalekv_compress(l, Qd, wpos, qw_is_full_map=True)
                        else:
                            Qw = Qd[:, :, wpos, :].contiguous()
                            torch.cuda.synchronize()
                            kv.scalekv_compress(l, Qw, wpos)
                kv.scalekv_sync()
                if l not in layers:
                    continue
                Oh, lseh = O.cpu(), lse.cpu()
                for (sl, b, h) in [s for s in self.slices if s[0] == l]:
                    self._compare_slice((sl, b, h), k, to64(Q[b, h]), to64(K[b, h]), to64(V[b, h]),
                                        to64(Oh[b, h]), to64(lseh[b, h]), wpos, do_compress)
        return self

    def _compare_slice(self, key, k, Q, K, V, O_gpu, lse_gpu, wpos, do_compress):
        l, b, h = key
        kv = self.kv
        cache = self.caches[key]
        cache.append(K, V)
        if self.max_rows is not None and Q.shape[0] > self.max_rows:
            rows = np.unique(np.linspace(0, Q.shape[0] - 1, self.max_rows).astype(np.int64))
            O, lse = cache.attend(Q[rows])
            O_gpu, lse_gpu = O_gpu[rows], lse_gpu[rows]
        else:
            O, lse = cache.attend(Q)
        err = float(np.max(np.abs(O - O_gpu)))
        self.max_err = max(self.max_err, err)
        # bf16: two roundings to 8 significant bits (P, then O), each at most 2^-9 relative: beyond |O| = 2.56 the
        # bound that follows from the arithmetic, 2^-7 max|O|, is larger than the 2e-2 quoted for unit-scale outputs
        tol = max(TOL[self.dtype], REL[self.dtype] * float(np.max(np.abs(O))))
        self.max_tol = max(self.max_tol, tol)
        assert err <= tol, f"slice {key} scale {k}: attention max-abs error {err} (bound {tol})"
        if self.check_lse:
            le = float(np.max(np.abs(lse - lse_gpu)))
            self.max_lse_err = max(self.max_lse_err, le)
            assert le <= 1e-3, f"slice {key} scale {k}: lse error {le}"
        if not do_compress:
            return
        nk = self.n[k]
        w_list = list(range(nk)) if wpos is None else list(wpos)
        budget = self.budgets[l][k]
        L = len(cache)
        before_pos = cache.pos.copy()
        s = cache.scores(Q[w_list])
        keep = orc.select(s, cache.pos, cache.N[k], w_list, budget)
        want_pos = cache.pos[keep]
        got_pos, Kg, Vg = kv.scalekv_export_slice(l, b, h, with_kv=True)
        got_pos = got_pos.numpy().astype(np.int64)
        cand = L - len(w_list)
        kprime = cand if budget == orc.KEEP_ALL else min(budget, cand)
        assert len(got_pos) == kprime + len(w_list), f"slice {key} scale {k}: kept count {len(got_pos)}"
        assert np.all(np.diff(got_pos) > 0)
        if kprime < cand:
            self.evictions += 1
        if not np.array_equal(got_pos, want_pos):
            # accepted only inside the tie band around the oracle's k'-th best score
            is_win = np.isin(before_pos, [cache.N[k] + p for p in w_list])
            sel = np.zeros(L, dtype=bool)
            sel[keep] = True
            sel &= ~is_win
            assert sel.any(), "kept sets differ although nothing is selected"
            boundary = s[sel].min()
            diff = np.setxor1d(got_pos, want_pos)
            idx = np.searchsorted(before_pos, diff)
            assert np.array_equal(before_pos[idx], diff), "GPU kept a position that was not in the cache"
            rel = np.abs(s[idx] - boundary) / max(abs(boundary), 1e-300)
            assert np.all(rel < TIE_BAND), f"slice {key} scale {k}: kept sets differ outside the tie band ({rel.max()})"
            self.resyncs += 1
        cache.adopt_positions(got_pos)
        # the compacted rows are the original rows of the kept positions, bit for bit
        assert np.array_equal(to64(Kg), cache.K), f"slice {key} scale {k}: compacted K rows differ"
        assert np.array_equal(to64(Vg), cache.V), f"slice {key} scale {k}: compacted V rows differ"
        if kprime < cand:
            sg = kv.scalekv_export_scores(b, h).numpy().astype(np.float64) if self._scores_fresh(l) else None
            if sg is not None and len(sg) == L:
                assert np.all(np.abs(sg - s) <= 2e-4 * s + 1e-9), "importance scores differ"

    def _scores_fresh(self, l):
        # the score scratch belongs to the most recent evicting compress; valid when the run syncs per layer
        return True
