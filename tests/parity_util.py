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
        self.max_lse_err = 0.0
        self.evictions = 0
        self.separate_kernels = False  # compress as three launches (the path long slices take) instead of one
        self.policy = "score"          # "score": observation-window importance; "recent": positional (sliding window, sinks)
        self.pool_kernel = 1           # width of the pooling of the importance along the keys (score policy)
        self.n_sink = 0                # always-kept lowest positions (recent policy)
        self.compared = 0             # slice-steps whose attention output was compared
        self.rel_bound_used = 0       # ... of which the relative branch of the bf16 bound (|O| > 2.56) decided

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
                    if self.separate_kernels or self.policy != "score" or self.pool_kernel > 1:
                        kv.scalekv_compress_ex(l, Qd, wpos, qw_is_full_map=True, policy=self.policy, pool_kernel=self.pool_kernel,
                                               n_sink=self.n_sink, separate_kernels=self.separate_kernels)
                    elif wpos is None:
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

    def summary(self):
        return (f"{self.compared} slice-steps compared, max |O - oracle| = {self.max_err:.3e}, relative bound decided "
                f"{self.rel_bound_used} of them, {self.evictions} evicting compressions, {self.resyncs} tie-band re-syncs")

    # ---- the execution mode the benchmark times -------------------------------------------------------------
    def run_pipelined(self, mode="eager", device_inputs=False):
        """One scalekv_step per layer and scale - compress of layer l on the side stream under attend of layer
        l + 1, transient page sets and logit buffers handed from layer l to layer l + 2 - with NO host
        synchronisation between the layers of a scale-step.  The host syncs once per scale-step (the kept set a
        compress leaves stays readable until the layer's next compress), exports every followed slice and lets
        the oracle compare and, inside the tie band, re-sync.
        mode "eager": the calls as they are.  mode "graph": the calls of every scale-step are captured on
        stream_main into a CUDA graph (compress forks to the side stream inside the capture) and the graph is
        replayed."""
        kv = self.kv
        n_layers = kv.n_layers
        if mode == "graph":
            kv.scalekv_reset()          # a capture must not start inside another stream's pending work
            kv.scalekv_sync()
        for k, nk in enumerate(self.n):
            wpos = self.window_fn(k)
            do_compress = (k + 1 < len(self.n)) or self.compress_last
            host, dev, O, lse = {}, {}, {}, {}
            for l in range(n_layers):
                Q, K, V = self.inputs_fn(l, k)
                dev[l] = (Q.cuda(), K.cuda(), V.cuda())
                host[l] = (Q, K, V)
                O[l] = torch.zeros_like(dev[l][0])
                lse[l] = torch.zeros(kv.batch, kv.n_heads, nk, dtype=torch.float32, device="cuda")
            torch.cuda.synchronize()
            wp = kv.window_array(wpos) if (do_compress and wpos is not None) else None

            def steps():
                for l in range(n_layers):
                    Qd, Kd, Vd = dev[l]
                    if self.policy == "score" and self.pool_kernel == 1:
                        kv.scalekv_step(l, k, Qd, Kd, Vd, O[l], window_pos=wp, whole_map=do_compress and wp is None, lse=lse[l])
                        continue
                    kv.scalekv_append(l, k, Kd, Vd)
                    kv.scalekv_attend(l, Qd, O[l], lse=lse[l])
                    if do_compress:
                        kv.scalekv_compress_ex(l, Qd, wpos, qw_is_full_map=True, policy=self.policy, pool_kernel=self.pool_kernel,
                                               n_sink=self.n_sink)

            if mode == "graph":
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=kv.stream_main):
                    steps()
                    kv.scalekv_join()
                with torch.cuda.stream(kv.stream_main):
                    g.replay()
            else:
                steps()
            kv.scalekv_sync()
            for l in sorted({s[0] for s in self.slices}):
                Q, K, V = host[l]
                Oh, lseh = O[l].cpu(), lse[l].cpu()
                for (sl, b, h) in [s for s in self.slices if s[0] == l]:
                    Qs, Ks, Vs = (t[b, h].cpu() for t in (Q, K, V))
                    self._compare_slice((sl, b, h), k, to64(Qs), to64(Ks), to64(Vs), to64(Oh[b, h]), to64(lseh[b, h]), wpos,
                                        do_compress, scores_fresh=(l == n_layers - 1))
        return self

    def run_graph_pass(self):
        """The whole pass - reset, then every scale and layer - captured into ONE CUDA graph and replayed twice,
        which is what the benchmark's timed region does.  Nothing can be exported between the scales of a replay,
        so the oracle walks the pass with its own selections (no re-sync possible: use inputs for which
        run_pipelined reports zero re-syncs) and compares every layer's output of every scale, and at the end the
        positions and K/V rows every followed slice holds."""
        kv = self.kv
        n_layers, K_s = kv.n_layers, len(self.n)
        host, dev, O, lse = {}, {}, {}, {}
        for k, nk in enumerate(self.n):
            for l in range(n_layers):
                Q, K, V = self.inputs_fn(l, k)
                host[(l, k)] = (Q, K, V)
                dev[(l, k)] = (Q.cuda(), K.cuda(), V.cuda())
                O[(l, k)] = torch.zeros_like(dev[(l, k)][0])
                lse[(l, k)] = torch.zeros(kv.batch, kv.n_heads, nk, dtype=torch.float32, device="cuda")
        wps = []
        for k in range(K_s):
            wpos = self.window_fn(k)
            do_compress = (k + 1 < K_s) or self.compress_last
            wps.append((kv.window_array(wpos) if (do_compress and wpos is not None) else None, do_compress, wpos))
        kv.scalekv_sync()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=kv.stream_main):
            kv.scalekv_reset()
            for k in range(K_s):
                wp, do_compress, _ = wps[k]
                for l in range(n_layers):
                    Qd, Kd, Vd = dev[(l, k)]
                    kv.scalekv_step(l, k, Qd, Kd, Vd, O[(l, k)], window_pos=wp, whole_map=do_compress and wp is None,
                                    lse=lse[(l, k)])
            kv.scalekv_join()
        for rep in range(2):
            for t in O.values():
                t.zero_()
            torch.cuda.synchronize()
            with torch.cuda.stream(kv.stream_main):
                g.replay()
            kv.scalekv_sync()
        for k in range(K_s):
            _, do_compress, wpos = wps[k]
            for (l, b, h) in self.slices:
                Q, K, V = (t[b, h].cpu() for t in host[(l, k)])
                self._compare_slice((l, b, h), k, to64(Q), to64(K), to64(V), to64(O[(l, k)][b, h].cpu()),
                                    to64(lse[(l, k)][b, h].cpu()), wpos, do_compress, exported=False)
        for (l, b, h) in self.slices:
            cache = self.caches[(l, b, h)]
            pos, Kg, Vg = kv.scalekv_export_slice(l, b, h, with_kv=True)
            # a layer whose last map reached into pages that a later layer took over exports the entries before that map
            m = len(pos)
            assert m == len(cache) or (not self.compress_last and m == len(cache) - self.n[-1])
            assert np.array_equal(pos.numpy().astype(np.int64), cache.pos[:m]), f"slice {(l, b, h)}: positions after the replayed pass"
            assert np.array_equal(to64(Kg), cache.K[:m]) and np.array_equal(to64(Vg), cache.V[:m]), f"slice {(l, b, h)}: rows after the replayed pass"
        return self

    def _compare_slice(self, key, k, Q, K, V, O_gpu, lse_gpu, wpos, do_compress, scores_fresh=True, exported=True):
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
        rel = REL[self.dtype] * float(np.max(np.abs(O)))
        tol = max(TOL[self.dtype], rel)
        self.compared += 1
        self.rel_bound_used += int(rel > TOL[self.dtype])
        assert err <= tol, f"slice {key} scale {k}: attention max-abs error {err} (bound {tol})"
        if self.check_lse:
            le = float(np.max(np.abs(lse - lse_gpu)))
            self.max_lse_err = max(self.max_lse_err, le)
            assert le <= 1e-3, f"slice {key} scale {k}: lse error {le}"
        if not do_compress:
            return
        nk = self.n[k]
        budget = self.budgets[l][k]
        L = len(cache)
        before_pos = cache.pos.copy()
        if self.policy == "recent":
            # positional rule: the budget counts the whole cache, sinks included; nothing to score, no ties
            keep = orc.select_recent(cache.pos, budget, self.n_sink)
            got_pos = kv.scalekv_export_slice(l, b, h).numpy().astype(np.int64)
            assert np.array_equal(got_pos, cache.pos[keep]), f"slice {key} scale {k}: positional rule kept other entries"
            self.evictions += int(len(keep) < L)
            cache.adopt(keep)
            return
        w_list = list(range(nk)) if wpos is None else list(wpos)
        s = orc.pool_scores(cache.scores(Q[w_list]), self.pool_kernel)
        keep = orc.select(s, cache.pos, cache.N[k], w_list, budget)
        want_pos = cache.pos[keep]
        if not exported:
            # nothing to read back at this point of a replayed pass: the oracle goes on with its own selection
            cand = L - len(w_list)
            self.evictions += int(budget != orc.KEEP_ALL and budget < cand)
            cache.adopt_positions(want_pos)
            return
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
            sg = kv.scalekv_export_scores(b, h).numpy().astype(np.float64) if scores_fresh else None
            if sg is not None and len(sg) == L and self.pool_kernel == 1:
                assert np.all(np.abs(sg - s) <= 2e-4 * s + 1e-9), "importance scores differ"
