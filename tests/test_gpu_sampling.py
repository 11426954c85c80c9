"""GPU parity for temperature sampling (Gumbel-max in the LM-head epilogue, Philox-4x32-10 noise)
against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import d3_oracle as o
from paper_2601_07568_b200 import binding as d3
from paper_2601_07568_b200 import synth_inputs as si
from gpu_utils import DEV, Ctx

pytestmark = pytest.mark.gpu


def _perturbed_gap(lg, mask_id, T, noise):
    """Gap between the two largest perturbed logits of every row (float32, as the decision is taken)."""
    pert = lg.astype(np.float32) + np.float32(T) * noise.astype(np.float32)
    pert[:, mask_id] = -np.inf
    top = np.sort(pert, axis=1)[:, -2:]
    return top[:, 1] - top[:, 0]


@pytest.mark.parametrize("T", [0.1, 0.7])
def test_generate_with_temperature_fp32_equals_the_oracle(T):
    """Ragged batch of three on the fp32 path: tokens and commit steps of d3_generate equal the oracle's
    run with the same seed (sequence index = batch index); where a sequence departs, the oracle's two
    best perturbed logits of the first differing step are within 1e-3 (a near-tie), else it is a failure."""
    shape = si.TINY
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("sample", shape, 3, [32, 9, 21], 64, 16, 0.9, 77)
    model = o.model_from_shape(shape, W, np.float64)
    seed = 0x123456789ABCDEF
    ref = [model.generate(ids[b, :lens[b]], 64, 16, 0.9, temperature=T, seed=seed, seq=b, record=True) for b in range(3)]
    greedy = [model.generate(ids[b, :lens[b]], 64, 16, 0.9) for b in range(3)]
    with Ctx(shape, W, block=16, max_batch=3, max_seq=wl.max_seq) as ctx:
        d3.d3_set_sampling(ctx.ctx, T, seed)
        ctx.prefill(ids, lens)
        tok, cs, st = ctx.generate(3, 64, 0.9)
        assert st.tokens_committed == 3 * 64 and ctx.error_word() == 0 and not np.any(tok == shape.mask_id)
        assert d3.d3_launch_count_of(ctx.ctx, "stats_merge_sample_kernel") >= 1
        exact = 0
        for b in range(3):
            if np.array_equal(tok[b], ref[b]["tokens"]) and np.array_equal(cs[b], ref[b]["commit_step"]):
                exact += 1
                continue
            for t in ref[b]["trace"]:     # first step decided differently: must be a near-tie of the perturbed logits
                j, s_ = t["block"], t["step"]
                dev_commit = cs[b, j * 16:(j + 1) * 16] == s_
                if np.array_equal(dev_commit, t["commit"]) and np.array_equal(tok[b, j * 16:(j + 1) * 16][dev_commit], t["tok"][dev_commit]):
                    continue
                state = model.prefill(ids[b, :lens[b]])
                for jj in range(j):
                    state = model.finalize_block(state, ref[b]["tokens"][jj * 16:(jj + 1) * 16])
                lg, *_ = model.denoise_forward(state, t["ids_in"])
                noise = o.gumbel_noise(seed, b, state.prefix_len + np.arange(16), s_, shape.vocab)
                gap = _perturbed_gap(lg, shape.mask_id, T, noise)
                conf_m = np.sort(t["conf"][t["mask_in"]])[::-1]
                near = gap[t["mask_in"]].min() < 1e-3 or np.any(np.abs(conf_m - 0.9) < 1e-3) or (len(conf_m) > 1 and conf_m[0] - conf_m[1] < 1e-3)
                assert near, (b, j, s_)
                break
        print("temperature", T, "sequences bit-equal to the oracle:", exact, "of 3")
        assert exact >= 2
        if T >= 0.5:
            assert any(not np.array_equal(tok[b], greedy[b]["tokens"]) for b in range(3))
        # another seed: other tokens; temperature 0: greedy
        d3.d3_set_sampling(ctx.ctx, T, seed + 1)
        ctx.prefill(ids, lens)
        tok2, _, _ = ctx.generate(3, 64, 0.9)
        assert not np.array_equal(tok2, tok)
        d3.d3_set_sampling(ctx.ctx, 0.0, seed)
        ctx.prefill(ids, lens)
        tok0, _, _ = ctx.generate(3, 64, 0.9)
        for b in range(3):
            assert np.array_equal(tok0[b], greedy[b]["tokens"])
        with pytest.raises(d3.D3Error):
            d3.d3_set_sampling(ctx.ctx, -1.0, 0)


def test_multiblock_with_temperature_fp32_equals_the_oracle():
    """Multi-block decoding with sampling (noise keyed by the round) on a ragged fp32 batch, windows of 2
    and 4 blocks: tokens, commit rounds and round counts equal the oracle's."""
    shape = si.TINY
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("sample-mb", shape, 3, [32, 9, 21], 64, 16, 0.3, 77)
    model = o.model_from_shape(shape, W, np.float64)
    with Ctx(shape, W, block=16, max_batch=12, max_seq=wl.max_seq) as ctx:
        for max_active, T, seed in [(2, 0.5, 99), (4, 0.2, (5 << 32) + 1)]:
            ref = [model.generate_multiblock(ids[b, :lens[b]], 64, 16, 0.3, 0, max_active=max_active, temperature=T, seed=seed, seq=b)
                   for b in range(3)]
            d3.d3_set_sampling(ctx.ctx, T, seed)
            ctx.prefill(ids, lens)
            tok, cr, st = ctx.generate_multiblock(3, 64, 0.3, max_active)
            exact = sum(int(np.array_equal(tok[b], ref[b]["tokens"]) and np.array_equal(cr[b], ref[b]["commit_round"])) for b in range(3))
            print("multi-block sampling, window", max_active, "sequences bit-equal to the oracle:", exact, "of 3")
            assert exact == 3 and st.steps == max(r["rounds"] for r in ref) and ctx.error_word() == 0


def _check_step_against_own_logits(ctx, shape, ids, lens, B, T, seed, n_steps, tol_gap):
    """The explicit step with sampling against the oracle's rule applied to the DEVICE's own fp32 logits of
    the same forward: tokens equal wherever the two best perturbed logits are further apart than
    tol_gap, confidence = softmax probability of the drawn token, entropy untouched by sampling."""
    bs = len(lens)
    ctx.prefill(ids, lens)
    d3.d3_set_sampling(ctx.ctx, T, seed)
    blk = np.full((bs, B), shape.mask_id, dtype=np.int32)
    mask = np.ones((bs, B), dtype=bool)
    compared = differing = 0
    for step in range(1, n_steps + 1):
        lg = ctx.logits(blk)                      # fp32 logits of this forward (no sampling involved)
        got = ctx.step(blk, mask, 0.9)
        for b in range(bs):
            noise = o.gumbel_noise(seed, b, lens[b] + np.arange(B), step, shape.vocab)
            conf, tok, ent = o.sample_stats(lg[b], shape.mask_id, T, noise)
            gap = _perturbed_gap(lg[b], shape.mask_id, T, noise)
            clear = gap > tol_gap
            compared += int(clear.sum())
            differing += int((got["tok"][b] != tok).sum())
            assert np.array_equal(got["tok"][b][clear], tok[clear]), (step, b)
            same = got["tok"][b] == tok
            assert np.allclose(got["conf"][b][same], conf[same], rtol=2e-4, atol=1e-7)
            assert np.allclose(got["ent"][b], ent, rtol=2e-4, atol=1e-5)
        blk, mask = got["ids"], got["mask"]
        if not mask.any():
            break
    return compared, differing


def test_sampling_epilogue_fp32_simt_against_its_own_logits():
    shape = si.TINY
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("sample-step", shape, 3, [32, 9, 21], 64, 16, 0.9, 5)
    with Ctx(shape, W, block=16, max_batch=3, max_seq=wl.max_seq) as ctx:
        compared, differing = _check_step_against_own_logits(ctx, shape, ids, lens, 16, 0.5, 42, 6, 1e-5)
        print("fp32 sampling steps: rows compared", compared, "rows with another token", differing)
        assert compared >= 3 * 16 * 5 and differing <= 2


def test_sampling_epilogue_bf16_tensor_core_against_its_own_logits():
    """The tensor-core LM head (vocabulary of 1000: eight 128-column tiles with a ragged last one; 96
    rows = three sequences of 32) draws the oracle's tokens from its own logits."""
    shape = si.scaled_shape(si.LLADA8B, name="sample-bf16", n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2,
                            d_ffn=640, vocab=1000, d_head=128)
    W = si.gen_weights(shape)
    wl, ids, lens = si.small_workload("sample-bf16", shape, 3, [40, 7, 97], 64, 32, 0.9, 77)
    with Ctx(shape, W, block=32, max_batch=3, max_seq=wl.max_seq) as ctx:
        for T, seed in [(0.1, 3), (1.0, (7 << 32) + 9)]:
            compared, differing = _check_step_against_own_logits(ctx, shape, ids, lens, 32, T, seed, 4, 1e-4)
            print("bf16 sampling T", T, ": rows compared", compared, "rows with another token", differing)
            assert compared >= 3 * 32 * 3 and differing <= 3
        # free-running generation with sampling runs to the end and depends on the seed
        d3.d3_set_sampling(ctx.ctx, 0.7, 11)
        ctx.prefill(ids, lens)
        a, _, st = ctx.generate(3, 64, 0.9)
        ctx.prefill(ids, lens)
        b, _, _ = ctx.generate(3, 64, 0.9)
        d3.d3_set_sampling(ctx.ctx, 0.7, 12)
        ctx.prefill(ids, lens)
        c, _, _ = ctx.generate(3, 64, 0.9)
        assert np.array_equal(a, b) and not np.array_equal(a, c) and st.tokens_committed == 3 * 64 and ctx.error_word() == 0
