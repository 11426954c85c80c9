"""GPU parity for the pseudo-trajectory path (Sec. 3.1): extraction run at threshold 1, the unmask
rank, and the noisy-sequence builder, against the CPU oracle (integer work: bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import d3_oracle as o
from paper_2601_07568_b200 import binding as d3
from paper_2601_07568_b200 import synth_inputs as si
from gpu_utils import DEV, Ctx

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.tensor(np.asarray(a), dtype=torch.int32, device=DEV).contiguous()


def test_extraction_run_rank_and_noisy_sequences_fp32():
    """Ragged batch of three on the fp32 path: the threshold-1 run unmasks one token per forward, its
    ranks are the oracle's (a permutation of 1..n per sequence), and noisy sequences built from them for
    a sweep of windows and mask ratios equal the oracle's element by element."""
    shape = si.TINY
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("traj", shape, 3, [32, 9, 21], 64, 16, 1.0, 77)
    model = o.model_from_shape(shape, W, np.float64)
    ref = [model.generate(ids[b, :lens[b]], 64, 16, 1.0) for b in range(3)]
    with Ctx(shape, W, block=16, max_batch=3, max_seq=wl.max_seq) as ctx:
        ctx.prefill(ids, lens)
        tok, cs, st = ctx.generate(3, 64, 1.0)
        assert st.denoise_forwards == 3 * 64 and st.forced_commits == 3 * 64
        rank_d = torch.zeros((3, 64), dtype=torch.int32, device=DEV)
        d3.d3_trajectory_rank(ctx.ctx, _dev(cs), rank_d)
        torch.cuda.synchronize()
        rank = rank_d.cpu().numpy()
        for b in range(3):
            assert np.array_equal(tok[b], ref[b]["tokens"])
            assert np.array_equal(rank[b], o.trajectory_rank(ref[b]["commit_step"], 16))
            assert sorted(rank[b].tolist()) == list(range(1, 65))
        # the ground-truth responses the trajectories are combined with: any tokens but the mask id
        rng = np.random.default_rng(12)
        y = rng.integers(0, shape.vocab - 2, size=(3, 64)).astype(np.int32)
        cases = 0
        for s, k in [(0, 16), (0, 64), (16, 32), (37, 11), (48, 16), (64, 0), (5, 0)]:
            for num, den in [(0, 1), (1, 4), (1, 2), (4, 5), (1, 1)]:
                m = o.ceil_ratio(k, num, den)
                s_arr = np.array([s, max(s - 3, 0), s], dtype=np.int32)      # per-sequence windows
                k_arr = np.array([k, k, max(k - 2, 0)], dtype=np.int32)
                m_arr = np.array([m, m, min(m, max(k - 2, 0))], dtype=np.int32)
                out = torch.zeros((3, 64), dtype=torch.int32, device=DEV)
                d3.d3_noisy_sequence(ctx.ctx, _dev(y), rank_d, _dev(s_arr), _dev(k_arr), _dev(m_arr), out)
                torch.cuda.synchronize()
                got = out.cpu().numpy()
                for b in range(3):
                    want = o.noisy_sequence(y[b], rank[b], int(s_arr[b]), int(k_arr[b]), int(m_arr[b]), shape.mask_id)
                    assert np.array_equal(got[b], want), (s, k, num, den, b)
                cases += 1
        assert cases == 35 and ctx.error_word() == 0
        with pytest.raises(d3.D3Error):
            d3.d3_trajectory_rank(ctx.ctx, _dev(cs[:, :60]), rank_d[:, :60].contiguous())


def test_rank_with_several_tokens_per_step_and_long_rows():
    """Ranks of an ordinary run (several tokens per step share a rank) and the builder on rows longer
    than one thread block, several blocks wide, against the oracle."""
    shape = si.TINY
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("traj2", shape, 2, [12, 30], 64, 16, 0.05, 5)
    model = o.model_from_shape(shape, W, np.float64)
    with Ctx(shape, W, block=16, max_batch=2, max_seq=wl.max_seq) as ctx:
        ctx.prefill(ids, lens)
        tok, cs, st = ctx.generate(2, 64, 0.05)
        rank_d = torch.zeros((2, 64), dtype=torch.int32, device=DEV)
        d3.d3_trajectory_rank(ctx.ctx, _dev(cs), rank_d)
        torch.cuda.synchronize()
        for b in range(2):
            ref = model.generate(ids[b, :lens[b]], 64, 16, 0.05)
            assert np.array_equal(cs[b], ref["commit_step"])
            assert np.array_equal(rank_d[b].cpu().numpy(), o.trajectory_rank(ref["commit_step"], 16))
        # synthetic long rows: n = 1000 (four thread blocks per row, ragged tail), random permutation ranks
        rng = np.random.default_rng(9)
        n = 1000
        y = rng.integers(0, shape.vocab - 2, size=(2, n)).astype(np.int32)
        rank = np.stack([rng.permutation(n) + 1 for _ in range(2)]).astype(np.int32)
        s_arr, k_arr = np.array([100, 777], dtype=np.int32), np.array([512, 223], dtype=np.int32)
        m_arr = np.array([o.ceil_ratio(512, 4, 5), o.ceil_ratio(223, 1, 3)], dtype=np.int32)
        out = torch.zeros((2, n), dtype=torch.int32, device=DEV)
        d3.d3_noisy_sequence(ctx.ctx, _dev(y), _dev(rank), _dev(s_arr), _dev(k_arr), _dev(m_arr), out)
        torch.cuda.synchronize()
        for b in range(2):
            want = o.noisy_sequence(y[b], rank[b], int(s_arr[b]), int(k_arr[b]), int(m_arr[b]), shape.mask_id)
            assert np.array_equal(out[b].cpu().numpy(), want)
