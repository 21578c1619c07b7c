"""scalekv_select_static - the entry point for callers that must not allocate device memory at
the moment they need a top-k (engines whose allocator owns the whole GPU, latency-critical phases
where cudaMalloc's device-wide synchronisation is not acceptable).  Its scratch is a fixed array
inside the library, so this file checks two things through the C ABI: that it selects exactly
what scalekv_compress selects from the same scores, on two calls in a row that reuse the array,
and that it refuses requests larger than the array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import scalekv_oracle as orc
from paper_2505_19602_b200 import binding

pytestmark = pytest.mark.gpu


def test_static_select_matches_compress_on_two_consecutive_calls():
    sides = (4, 8, 12, 16)
    n = [a * a for a in sides]
    N = np.concatenate([[0], np.cumsum(n)])
    B, H, d, budget = 2, 3, 128, 37
    kv = binding.ScaleKV(1, B, H, d, "bf16", sides, sides, [[budget] * len(sides)], max_window=16)
    g = torch.Generator().manual_seed(123)
    calls = 0
    for k in range(len(sides) - 1):
        Q, K, V = (torch.randn(B, H, n[k], d, generator=g).to(torch.bfloat16).cuda() for _ in range(3))
        torch.cuda.synchronize()
        kv.scalekv_append(0, k, K, V)
        kv.scalekv_attend(0, Q)
        kv.scalekv_sync()
        before = [[kv.scalekv_export_slice(0, b, h).numpy().astype(np.int64) for h in range(H)] for b in range(B)]
        L = len(before[0][0])
        wpos = binding.scalekv_window_centroids(sides[k], sides[k], 16)
        kv.scalekv_compress(0, Q, wpos, qw_is_full_map=True)
        kv.scalekv_sync()
        if L - len(wpos) <= budget:
            continue                                   # nothing evicted: no scores were produced
        # the existing entry point's result, and the scores it selected from
        after = [[kv.scalekv_export_slice(0, b, h).numpy().astype(np.int64) for h in range(H)] for b in range(B)]
        scores = [[kv.scalekv_export_scores(b, h) for h in range(H)] for b in range(B)]
        win_abs = np.array([N[k] + p for p in wpos])
        rows, cand_slots = [], []
        for b in range(B):
            for h in range(H):
                cand = np.nonzero(~np.isin(before[b][h], win_abs))[0]
                cand_slots.append(cand)
                rows.append(scores[b][h][torch.from_numpy(cand)])
        dev_scores = torch.stack(rows).cuda()          # [B*H, L - w] candidates only
        idx_out = torch.empty(B * H, budget, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        for rep in range(2):                           # the second call finds the first one's keys in the scratch
            idx_out.fill_(-1)
            binding.scalekv_select_static(dev_scores, budget, idx_out)
            torch.cuda.synchronize()
            idx = idx_out.cpu().numpy()
            for r in range(B * H):
                b, h = divmod(r, H)
                assert np.all(np.diff(idx[r]) > 0)
                chosen = before[b][h][cand_slots[r][idx[r]]]
                got = np.sort(np.concatenate([chosen, win_abs]))
                assert np.array_equal(got, after[b][h]), (k, b, h, rep)
            calls += 1
    assert calls >= 4
    kv.close()


def test_static_select_ties_and_limits():
    # exact ties: lowest indices win; k == len keeps everything
    s = torch.full((3, 50), 0.25, device="cuda")
    s[1, 40] = 0.5
    out = binding.scalekv_select_static(s, 4)
    torch.cuda.synchronize()
    assert out.cpu().tolist() == [[0, 1, 2, 3], [0, 1, 2, 40], [0, 1, 2, 3]]
    out = binding.scalekv_select_static(s[:, :7].contiguous(), 7)
    torch.cuda.synchronize()
    assert out.cpu().tolist() == [list(range(7))] * 3
    # a strided view: row stride larger than the row length
    out = binding.scalekv_select_static(s[:, :20], 2)
    torch.cuda.synchronize()
    assert out.cpu().tolist() == [[0, 1]] * 3
    # beyond the fixed scratch: refused before anything is launched
    big = torch.zeros(2, (1 << 19) + 1, device="cuda")
    with pytest.raises(binding.ScaleKVError) as e:
        binding.scalekv_select_static(big, 5)
    assert e.value.status == 3
    with pytest.raises(binding.ScaleKVError) as e:
        binding.scalekv_select_static(s, 51)
    assert e.value.status == 1
    # a request that exactly fills the array is served
    full = torch.rand(2, 1 << 19, device="cuda")
    out = binding.scalekv_select_static(full, 3)
    torch.cuda.synchronize()
    want = torch.sort(torch.topk(full, 3, dim=1).indices, dim=1).values
    assert torch.equal(out.cpu().long(), want.cpu())


def test_static_select_matches_the_oracle_selection():
    """The same rows through the CPU oracle's selection rule (largest scores, equal scores by lowest index):
    random rows, rows with many repeated values, and a row whose values are all equal."""
    g = torch.Generator().manual_seed(7)
    rows = torch.rand(6, 777, generator=g)
    rows[1] = torch.round(rows[1] * 8) / 8              # heavy ties
    rows[2] = 0.125
    rows[3, 100:300] = rows[3, 5]
    dev = rows.cuda()
    for k in (1, 13, 400, 777):
        for rep in range(2):
            out = binding.scalekv_select_static(dev, k).cpu().numpy()
            for r in range(rows.shape[0]):
                want = orc.select(rows[r].double().numpy(), np.arange(777), 777, [], k)
                assert np.array_equal(out[r], want), (k, r, rep)
