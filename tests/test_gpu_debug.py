"""Switches and counters around the decoding path: the give-up path of the bounded device-side waits,
the decision on unusable statistics, the commits-per-decision histogram, and the refusal of a
pipeline depth the column-strip kernel cannot run."""
import numpy as np
import pytest
import torch

from oracle import d3_oracle as o
from paper_2601_07568_b200 import binding as d3
from paper_2601_07568_b200 import synth_inputs as si
from gpu_utils import DEV, Ctx

pytestmark = pytest.mark.gpu


def _small_bf16(name):
    return si.scaled_shape(si.LLADA8B, name=name, n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2,
                           d_ffn=640, vocab=1000, d_head=128)


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """No thread ever completes the barrier the MMA-issuing thread waits on (the probe issues no loads):
    after the shortened limit the kernel returns by itself, the error word carries the time-out bit, the
    call that reads it returns D3_ERR_DEVICE_TIMEOUT, and after clearing the word the same context runs
    a normal forward whose logits equal those from before the probe, bit for bit."""
    shape = _small_bf16("stall")
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("stall", shape, 1, [21], 32, 32, 0.9, 3)
    blk = np.full((1, 32), shape.mask_id, dtype=np.int32)
    with Ctx(shape, W, block=32, max_batch=1, max_seq=wl.max_seq) as ctx:
        ctx.prefill(ids, lens)
        before = ctx.logits(blk)
        assert ctx.error_word() == 0
        with pytest.raises(d3.D3Error):
            d3._check(ctx.ctx, d3.d3_debug_stall_probe(ctx.ctx, 0))  # limit outside 1..2000000
        rc = d3.d3_debug_stall_probe(ctx.ctx, 2000)                 # 2 ms
        assert rc == d3.D3_ERR_DEVICE_TIMEOUT
        assert ctx.error_word() & 1
        # every later status read reports it until the word is cleared
        out = torch.zeros((1, 32), dtype=torch.int32, device=DEV)
        with pytest.raises(d3.D3Error) as ei:
            d3.d3_generate(ctx.ctx, 32, 0.9, out)
        assert ei.value.code == d3.D3_ERR_DEVICE_TIMEOUT
        d3.d3_clear_error_word(ctx.ctx)
        assert ctx.error_word() == 0
        ctx.prefill(ids, lens)
        after = ctx.logits(blk)
        assert np.array_equal(before, after)
        assert ctx.error_word() == 0
    # a float32 context has no tensor-core kernel to probe
    with Ctx(si.TINY, None, block=16, max_batch=1, max_seq=64) as ctx:
        assert d3.d3_debug_stall_probe(ctx.ctx, 1000) == d3.D3_ERR_UNSUPPORTED


def test_unmask_with_unusable_statistics_still_commits_and_raises_the_error_word():
    """Every masked row's confidence is NaN: no row compares as the best, yet the block must lose a
    mask per forward (Sec. 3.2, at-least-one rule).  The lowest masked position is committed and bit 4
    of the error word is raised; unmasked rows are left alone; a block without masks is untouched."""
    with Ctx(si.TINY, None, block=16, max_batch=3, max_seq=64) as ctx:
        B = 16
        conf = torch.full((3, B), float("nan"), device=DEV)
        ent = torch.full((3, B), float("nan"), device=DEV)
        am = torch.arange(3 * B, dtype=torch.int32, device=DEV).reshape(3, B) + 100
        ids = torch.full((3, B), si.TINY.mask_id, dtype=torch.int32, device=DEV)
        mask = torch.ones((3, B), dtype=torch.uint8, device=DEV)
        mask[0, :5] = 0          # sequence 0: positions 0-4 already decided
        ids[0, :5] = 7
        mask[2, :] = 0           # sequence 2: nothing masked
        ids[2, :] = 9
        conf[1, 3] = 0.2         # sequence 1 has one usable row: the ordinary rule applies there
        pos = torch.full((3, B), -1, dtype=torch.int32, device=DEV)
        oid = torch.full((3, B), -1, dtype=torch.int32, device=DEV)
        cnt = torch.zeros(3, dtype=torch.int32, device=DEV)
        d3.d3_op_unmask(ctx.ctx, conf, ent, am, ids, mask, 0.9, pos, oid, cnt)
        torch.cuda.synchronize()
        assert cnt.tolist() == [1, 1, 0]
        assert pos[0, 0].item() == 5 and oid[0, 0].item() == 100 + 5 and mask[0].tolist() == [0] * 6 + [1] * 10
        assert pos[1, 0].item() == 3 and oid[1, 0].item() == 100 + B + 3
        assert mask[2].sum().item() == 0 and (ids[2] == 9).all()
        assert ctx.error_word() == 16
        assert d3.d3_status_of_error_word(16) == d3.D3_ERR_INVALID_ARG
        d3.d3_clear_error_word(ctx.ctx)
        assert ctx.error_word() == 0


def test_commit_histogram_equals_the_oracle_trace():
    """Commits per decision (what tokens per forward averages over): d3_generate on a ragged fp32 batch
    and multi-block decoding, against the histogram of the oracle's per-step commit counts."""
    shape = si.TINY
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("hist", shape, 3, [32, 9, 21], 64, 16, 0.3, 77)
    model = o.model_from_shape(shape, W, np.float64)
    with Ctx(shape, W, block=16, max_batch=12, max_seq=wl.max_seq) as ctx:
        ref = [model.generate(ids[b, :lens[b]], 64, 16, 0.3, record=True) for b in range(3)]
        want = np.zeros(17, dtype=np.int64)
        for r in ref:
            for t in r["trace"]:
                want[int(t["commit"].sum())] += 1
        ctx.prefill(ids, lens)
        tok, _, st = ctx.generate(3, 64, 0.3)
        hist = np.array(d3.d3_commit_histogram(ctx.ctx, 17))
        assert np.array_equal(hist, want)
        assert hist[0] == 0 and hist.sum() == st.denoise_forwards
        assert (hist * np.arange(17)).sum() == st.tokens_committed == 3 * 64
        # multi-block decoding: one entry per (sequence, block, round) decision; Activated blocks may commit nothing
        refm = [model.generate_multiblock(ids[b, :lens[b]], 64, 16, 0.3, 0, max_active=3, record=True) for b in range(3)]
        wantm = np.zeros(17, dtype=np.int64)
        for r in refm:
            for t in r["trace"]:
                for k in range(t["n_win"]):
                    if t["mask_in"][k].any():
                        wantm[int(t["commits"][k].sum())] += 1
        ctx.prefill(ids, lens)
        _, _, stm = ctx.generate_multiblock(3, 64, 0.3, 3)
        histm = np.array(d3.d3_commit_histogram(ctx.ctx, 17))
        assert np.array_equal(histm, wantm)
        assert histm.sum() == stm.denoise_forwards and (histm * np.arange(17)).sum() == 3 * 64
        assert ctx.error_word() == 0


def test_column_strips_refuse_an_odd_pipeline_depth():
    """Two issue pipelines share the stage ring of the column-strip kernel and every stage belongs to one
    of them, which takes an even number of stages: an odd depth asked for by name is refused, an even one
    runs and gives the default schedule's result up to the order of the fp32 sums."""
    shape = _small_bf16("strip-stages")
    with Ctx(shape, None, block=32, max_batch=1, max_seq=64) as ctx:
        g = torch.Generator().manual_seed(5)
        m, n, k = 32, 256, 512
        x = torch.randn((m, k), generator=g).to(torch.bfloat16).to(DEV)
        w = (torch.randn((n, k), generator=g) * 0.05).to(torch.bfloat16).to(DEV)
        packed = torch.empty(d3.d3_packed_weight_elems(n, k), dtype=torch.bfloat16, device=DEV)
        d3.d3_pack_weight(ctx.ctx, w, packed)
        y0 = torch.zeros((m, n), dtype=torch.float32, device=DEV)
        d3.d3_op_linear_packed(ctx.ctx, x, packed, y0, n, 0, -64)
        for stages, ok in [(5, False), (7, False), (4, True), (6, True)]:
            d3.d3_set_tuning(ctx.ctx, strip_stages=stages)
            y = torch.zeros((m, n), dtype=torch.float32, device=DEV)
            if ok:
                d3.d3_op_linear_packed(ctx.ctx, x, packed, y, n, 0, -64)
                torch.cuda.synchronize()
                assert torch.allclose(y, y0, rtol=1e-3, atol=1e-3)
            else:
                with pytest.raises(d3.D3Error) as ei:
                    d3.d3_op_linear_packed(ctx.ctx, x, packed, y, n, 0, -64)
                assert ei.value.code == d3.D3_ERR_UNSUPPORTED
        d3.d3_set_tuning(ctx.ctx)
        with pytest.raises(d3.D3Error):
            d3.d3_set_tuning(ctx.ctx, strip_stages=33)
        assert ctx.error_word() == 0
