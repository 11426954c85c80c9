"""GPU parity for KV-refresh and the cache delay (Sec. 3.2, KV-cache and KV-refresh mechanism) against
the CPU oracle: the explicit call, and both generate loops with a refresh period."""
import numpy as np
import pytest
import torch

from oracle import d3_oracle as o
from paper_2601_07568_b200 import binding as d3
from paper_2601_07568_b200 import synth_inputs as si
from gpu_utils import Ctx, assert_rounding_bounded, record_report
from test_gpu_decode import BF16_STAT_ERR_BOUND, step_locked

pytestmark = pytest.mark.gpu


def _tiny_batch(tau=0.9, seed=77):
    shape = si.TINY
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("refresh", shape, 3, [32, 9, 21], 64, 16, tau, seed)
    return shape, W, wl, ids, lens


def test_explicit_refresh_fp32_logits_equal_the_oracle():
    """Prefill, store two blocks, refresh: the next block's logits are the oracle's after its refresh
    (fp32: 1e-4 of the largest logit), and differ from the logits before the refresh; a refresh of
    prompt-only caches changes nothing."""
    shape, W, wl, ids, lens = _tiny_batch()
    model = o.model_from_shape(shape, W, np.float64)
    rng = np.random.default_rng(3)
    blocks = [rng.integers(0, shape.vocab - 2, size=(3, 16)).astype(np.int32) for _ in range(2)]
    cur = np.full((3, 16), shape.mask_id, dtype=np.int32)
    cur[:, 3] = 5
    with Ctx(shape, W, block=16, max_batch=3, max_seq=wl.max_seq, max_prefill_rows=3 * wl.max_seq) as ctx:
        ctx.prefill(ids, lens)
        base = ctx.logits(cur)
        d3.d3_refresh_cache(ctx.ctx, 3)
        assert np.array_equal(ctx.logits(cur), base)          # nothing stored but the prompt
        for blk in blocks:
            ctx.commit(blk)
        before = ctx.logits(cur)
        d3.d3_refresh_cache(ctx.ctx, 3)
        after = ctx.logits(cur)
        assert np.array_equal(ctx.get_prefix(3), lens + 32) and ctx.error_word() == 0
        for b in range(3):
            st = model.prefill(ids[b, :lens[b]])
            for blk in blocks:
                st = model.finalize_block(st, blk[b])
            lg0, *_ = model.denoise_forward(st, cur[b])
            lg1, *_ = model.denoise_forward(model.refresh(st), cur[b])
            fin = np.isfinite(lg1)
            scale = np.abs(lg1[fin]).max()
            assert np.abs(before[b][fin] - lg0[fin]).max() <= 1e-4 * scale
            assert np.abs(after[b][fin] - lg1[fin]).max() <= 1e-4 * scale
            assert np.abs(after[b][fin] - before[b][fin]).max() > 1e-3 * scale   # the refresh did something


@pytest.mark.parametrize("every", [1, 2])
def test_generate_with_periodic_refresh_fp32_equals_the_oracle(every):
    """Ragged batch of three on the fp32 path: tokens and commit steps bit-equal to the oracle's run with
    the same refresh period; sequences refresh at their own pace (one is flagged while others denoise)."""
    shape, W, wl, ids, lens = _tiny_batch()
    model = o.model_from_shape(shape, W, np.float64)
    ref = [model.generate(ids[b, :lens[b]], 64, 16, 0.9, refresh_every=every) for b in range(3)]
    plain = [model.generate(ids[b, :lens[b]], 64, 16, 0.9) for b in range(3)]
    assert any(not np.array_equal(r["tokens"], p["tokens"]) for r, p in zip(ref, plain)), "the refresh must matter in this case"
    with Ctx(shape, W, block=16, max_batch=3, max_seq=wl.max_seq, max_prefill_rows=3 * wl.max_seq) as ctx:
        d3.d3_set_cache_policy(ctx.ctx, 1, every)
        ctx.prefill(ids, lens)
        tok, cs, st = ctx.generate(3, 64, 0.9)
        for b in range(3):
            assert np.array_equal(tok[b], ref[b]["tokens"]), b
            assert np.array_equal(cs[b], ref[b]["commit_step"]), b
        assert d3.d3_refresh_count(ctx.ctx) == sum(r["n_refresh"] for r in ref)
        assert st.denoise_forwards == sum(r["n_denoise"] for r in ref) and st.finalize_forwards == 12
        assert d3.d3_launch_count_of(ctx.ctx, "refresh_rowmap_kernel") >= 1 and ctx.error_word() == 0
        # policy off again: the plain run
        d3.d3_set_cache_policy(ctx.ctx, 1, 0)
        ctx.prefill(ids, lens)
        tok, _, _ = ctx.generate(3, 64, 0.9)
        for b in range(3):
            assert np.array_equal(tok[b], plain[b]["tokens"])
        assert d3.d3_refresh_count(ctx.ctx) == 0
    # workspaces too small for the refresh forward: an error, not a silent skip
    with Ctx(shape, W, block=16, max_batch=3, max_seq=wl.max_seq, max_prefill_rows=96) as ctx:  # 128 rows of workspace < 3 x 48
        d3.d3_set_cache_policy(ctx.ctx, 1, 1)
        ctx.prefill(ids, lens)
        with pytest.raises(d3.D3Error):
            ctx.generate(3, 64, 0.9)


@pytest.mark.parametrize("delay,every,max_active", [(2, 0, 2), (1, 3, 2), (2, 2, 4), (3, 5, 3)])
def test_multiblock_cache_delay_and_refresh_fp32_equal_the_oracle(delay, every, max_active):
    shape, W, wl, ids, lens = _tiny_batch(tau=0.3)
    model = o.model_from_shape(shape, W, np.float64)
    ref = [model.generate_multiblock(ids[b, :lens[b]], 64, 16, 0.3, 0, max_active=max_active, cache_delay=delay,
                                     refresh_every=every) for b in range(3)]
    with Ctx(shape, W, block=16, max_batch=12, max_seq=wl.max_seq, max_prefill_rows=3 * wl.max_seq) as ctx:
        d3.d3_set_cache_policy(ctx.ctx, delay, every)
        ctx.prefill(ids, lens)
        tok, cr, st = ctx.generate_multiblock(3, 64, 0.3, max_active)
        for b in range(3):
            assert np.array_equal(tok[b], ref[b]["tokens"]), b
            assert np.array_equal(cr[b], ref[b]["commit_round"]), b
        assert st.steps == max(r["rounds"] for r in ref)
        assert st.finalize_forwards == 12 and st.tokens_committed == 3 * 64
        assert d3.d3_refresh_count(ctx.ctx) == sum(r["n_refresh"] for r in ref)
        assert np.array_equal(ctx.get_prefix(3), lens + 64) and ctx.error_word() == 0
        with pytest.raises(d3.D3Error):
            d3.d3_set_cache_policy(ctx.ctx, 0, 0)


def test_refresh_bf16_tensor_core():
    """Through the tensor-core kernels (refresh forwards of 69 to 165 rows, decode forwards of 32): the
    logits after an explicit refresh within 3 % of the largest logit of the oracle with mirrored bf16
    roundings, and generation with a refresh after every block step-locked to the oracle.  The refreshed
    cache must matter: the oracle's run without refresh decodes other tokens."""
    shape = si.scaled_shape(si.LLADA8B, name="refresh-bf16", n_layers=3, d_model=256, n_q_heads=4, n_kv_heads=2,
                            d_ffn=640, vocab=1000, d_head=128)
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("refresh-bf16", shape, 1, [37], 128, 32, 0.9, 29)
    model = o.model_from_shape(shape, W, np.float32, mirror_bf16=True)
    rng = np.random.default_rng(8)
    blk = rng.integers(0, shape.vocab - 2, size=(1, 32)).astype(np.int32)
    cur = np.full((1, 32), shape.mask_id, dtype=np.int32)
    with Ctx(shape, W, block=32, max_batch=1, max_seq=wl.max_seq, max_prefill_rows=wl.max_seq) as ctx:
        ctx.prefill(ids, lens)
        ctx.commit(blk)
        d3.d3_refresh_cache(ctx.ctx, 1)
        got = ctx.logits(cur)[0]
        st = model.refresh(model.finalize_block(model.prefill(ids[0, :lens[0]]), blk[0]))
        lg, *_ = model.denoise_forward(st, cur[0])
        fin = np.isfinite(lg)
        err = np.abs(got[fin] - lg[fin]).max() / np.abs(lg[fin]).max()
        print("bf16 logits after refresh: relative error", err)
        assert err <= 3e-2
        # generation with a refresh after every stored block, the device following the oracle's
        # trajectory step by step: decisions differ only where the oracle's own margin is below 1e-3 or
        # below the two sides' numerical difference
        exact = o.model_from_shape(shape, W, np.float32)
        rep, traces = step_locked(ctx, model, ids, lens, 128, 32, 0.9, logit_tol=3e-2, exact_model=exact, refresh_every=1)
        print("bf16 step-locked with refresh", rep)
        assert traces[0]["n_refresh"] == 3
        record_report("refresh_bf16_step_locked", rep)
        assert rep["max_logit_err"] <= 3e-2
        assert_rounding_bounded(rep, BF16_STAT_ERR_BOUND)
        # free-running through d3_generate: runs to the end with three refreshes (ids may drift after a near-tie)
        d3.d3_set_cache_policy(ctx.ctx, 1, 1)
        ctx.prefill(ids, lens)
        tok, cs, stt = ctx.generate(1, 128, 0.9)
        assert d3.d3_refresh_count(ctx.ctx) == 3 and stt.tokens_committed == 128 and ctx.error_word() == 0
        assert not np.any(tok == shape.mask_id)
        print("free-running equal to the oracle:", np.array_equal(tok[0], traces[0]["tokens"]))
