"""Parity at the full sizes of the five configurations, in the launch configuration bench.py times.

A whole 8B-shaped forward is out of reach of the CPU oracle inside a test, so the oracle checks
sampled pieces that it can compute one by one from the GPU's own inputs (decoupled checks: an error
anywhere in a sampled piece shows up in that piece, not 30 layers later):

  * sampled layers: the residual rows entering layer L of one denoise forward and the prefix cache
    of that layer are read back; the oracle recomputes the layer in fp32 from them and must reproduce
    the rows leaving the layer and the block's own K/V cache slots;
  * the head: from the rows leaving the last layer the oracle computes logits, softmax statistics
    and the threshold decision, which must match the statistics and the commits of the same GPU step
    (ids bit-exact except oracle near-ties: top-2 probability gap or |confidence - threshold| < 1e-3;
    ids that differ although the gap is larger are tolerated only while the two best logits are closer
    than twice the logit error measured on the same rows, and are counted in the printed report);
  * sampled steps: step 1 of block 1 (all masked), step 2 of block 1 (the partially unmasked block that
    step 1 left) and step 1 of block 2 (the prefix then holds a block the GPU generated and stored); at the
    batch-1 shape also one 64-row forward of two segments (the form d3_generate fuses a finalize forward
    with the next block's first step in) and one 128-row round of four segments (multi-block decoding);
  * prefill as an output: the stored K/V of the first two layers of one long prompt against the oracle's
    forward over the prompt rows;
  * the whole c2 request free-running against the stored decode of the oracle (tests/golden/c2_oracle_trace.json);
  * properties that hold at any size: every generated id is a real token, each sequence commits
    exactly gen_len tokens in at most gen_len forwards, two runs give identical bits.

Tolerances: a layer's update and the cache rows within 3e-2 of their largest magnitude (the bf16
bar of the benchmark spec; the pipeline stores activations in bf16), confidences within 5e-2.
"""
import numpy as np
import pytest
import torch

from oracle import d3_oracle as o
from paper_2601_07568_b200 import binding as d3
from paper_2601_07568_b200 import synth_inputs as si
from gpu_utils import DEV, EPS, Ctx, record_report, top2_gap

pytestmark = pytest.mark.gpu


def _read_kv(ctx, shape, layer, seq, n):
    k = torch.empty((shape.n_kv_heads, n, shape.d_head), dtype=torch.float32, device=DEV)
    v = torch.empty_like(k)
    d3.d3_read_kv(ctx.ctx, layer, seq, 0, n, k, v)
    torch.cuda.synchronize()
    # oracle layout: [positions, kv heads, d_head]
    return k.cpu().numpy().transpose(1, 0, 2).copy(), v.cpu().numpy().transpose(1, 0, 2).copy()


def _denoise_with_tap(ctx, w, layer, tau, ids=None, mask=None):
    bs, B = w.batch, w.block
    d = w.model.d_model
    d3.d3_set_tap(ctx.ctx, layer)
    if ids is None:
        ids = np.full((bs, B), w.model.mask_id, dtype=np.int32)
        mask = np.ones((bs, B), dtype=bool)
    got = ctx.step(ids, mask, tau)
    x_in = torch.empty((bs * B, d), dtype=torch.float32, device=DEV)
    x_out = torch.empty_like(x_in)
    d3.d3_read_tap(ctx.ctx, x_in, x_out, bs * B)
    torch.cuda.synchronize()
    d3.d3_set_tap(ctx.ctx, -1)
    return got, x_in.cpu().numpy().reshape(bs, B, d), x_out.cpu().numpy().reshape(bs, B, d)


def _layer_model(shape, W, layer):
    return o.model_from_shape(shape, {"layers": {layer: W["layers"][layer]}, "lm_head": W["lm_head"],
                                      "tok_emb": W["tok_emb"]}, np.float32)


def _check_step(ctx, w, W, name, tag, layers, seqs, prefix, ids=None, mask=None, report=None):
    """One denoise step of the GPU on the given block state (default: fully masked), checked piecewise
    by the oracle from the GPU's own inputs: the sampled layers (rows leaving the layer, the block's own
    K/V slots) and, at the last layer, logits, statistics and the decision.  ``prefix`` [bs]: cached prefix
    lengths.  Returns the GPU's step result.  Decisions and ids that differ from the oracle's are put in
    classes: excused (oracle margin < 1e-3), rounding (margin at most twice the largest statistic /
    logit error measured on the same rows) or a failure; the rounding classes are counted and bounded."""
    shape = w.model
    B = w.block
    last = shape.n_layers - 1
    bs = w.batch
    if ids is None:
        ids = np.full((bs, B), shape.mask_id, dtype=np.int32)
        mask = np.ones((bs, B), dtype=bool)
    lg_gpu, got_last = None, None
    for layer in layers:
        got, x_in, x_out = _denoise_with_tap(ctx, w, layer, w.threshold, ids, mask)
        got_last = got
        model = _layer_model(shape, W, layer)
        for b in seqs:
            L = int(prefix[b])
            k_all, v_all = _read_kv(ctx, shape, layer, b, L + B)
            pos = L + np.arange(B)
            ref_out, k_rows, v_rows = model.layer_forward(layer, x_in[b].astype(np.float32), pos, k_all[:L], v_all[:L])
            upd_ref, upd_got = ref_out - x_in[b], x_out[b] - x_in[b]
            err = np.max(np.abs(upd_got - upd_ref)) / np.max(np.abs(upd_ref))
            kerr = np.max(np.abs(k_all[L:] - k_rows)) / np.max(np.abs(k_rows))
            verr = np.max(np.abs(v_all[L:] - v_rows)) / np.max(np.abs(v_rows))
            report[f"{tag}:layer{layer}:seq{b}"] = [float(err), float(kerr), float(verr)]
            assert err <= 3e-2, (name, tag, layer, b, err)
            assert kerr <= 3e-2 and verr <= 3e-2, (name, tag, layer, b, kerr, verr)
            if layer != last:
                continue
            # head: logits, statistics and decision of this step from the GPU's final rows
            mk = mask[b]
            lg = model.logits(x_out[b].astype(np.float32))
            p, conf, tok, ent = o.softmax_stats(lg, shape.mask_id)
            part = np.partition(p, -2, axis=-1)
            gap = part[:, -1] - part[:, -2]
            if lg_gpu is None:
                lg_gpu = ctx.logits(ids)
            lerr = float(np.max(np.abs(lg_gpu[b] - lg)))
            assert lerr <= 3e-2 * np.max(np.abs(lg)), (name, tag, b, lerr)
            stat_err = float(np.max(np.abs(got["conf"][b] - conf)))
            assert stat_err <= 5e-2, (name, tag, b, stat_err)
            report[f"{tag}:logit_err:seq{b}"] = lerr / float(np.max(np.abs(lg)))
            report[f"{tag}:stat_err:seq{b}"] = stat_err
            report["max_stat_err"] = max(report.get("max_stat_err", 0.0), stat_err)
            # ids on masked rows: equal, excused (probability gap < 1e-3) or rounding (the two best logits
            # closer than twice the measured logit error)
            top2 = np.partition(np.where(np.arange(shape.vocab)[None, :] == shape.mask_id, -np.inf, lg), -2, axis=-1)
            lgap = top2[:, -1] - top2[:, -2]
            differ = (got["tok"][b] != tok) & mk
            report["rows"] = report.get("rows", 0) + int(mk.sum())
            report["ids_excused"] = report.get("ids_excused", 0) + int((differ & (gap < EPS)).sum())
            report["ids_rounding"] = report.get("ids_rounding", 0) + int((differ & (gap >= EPS) & (lgap <= 2 * lerr)).sum())
            tok_bad = differ & (gap >= EPS) & (lgap > 2 * lerr)
            assert not tok_bad.any(), (name, tag, b, np.flatnonzero(tok_bad))
            # the decision kernel on the GPU's own statistics: bit-exact
            own = o.decide(got["conf"][b], got["ent"][b], mk, np.float32(w.threshold), 0)
            have = np.zeros(B, dtype=bool)
            have[got["pos"][b, :got["count"][b]]] = True
            assert np.array_equal(own, have), (name, tag, b)
            assert np.array_equal(got["ids"][b][have], got["tok"][b][have])
            # against the oracle's decision
            want = o.decide(conf.astype(np.float32), ent.astype(np.float32), mk, np.float32(w.threshold), 0)
            score = np.sort(np.where(mk, conf, -np.inf))[::-1]
            forced_gap = score[0] - score[1] if mk.sum() >= 2 else np.inf
            clears = mk & (conf > w.threshold)
            order0 = int(np.argmax(np.where(mk, conf, -np.inf)))
            for r in np.flatnonzero(want != have):
                margin = abs(conf[r] - w.threshold)
                if not clears.any() or r == order0 or (have[r] and not clears[r]):
                    margin = min(margin, forced_gap)
                if margin < EPS:
                    report["decision_excused"] = report.get("decision_excused", 0) + 1
                elif margin <= 2 * stat_err:  # twice the largest statistic error on this block's rows: a fixed number, not the row's own
                    report["decision_rounding"] = report.get("decision_rounding", 0) + 1
                else:
                    raise AssertionError((name, tag, b, int(r), float(conf[r]), float(got["conf"][b][r]), float(margin)))
    return got_last


def _check_workload(name, layers, seqs, W_full=None):
    w = si.WORKLOADS[name]
    shape = w.model
    ids, lens = si.gen_prompts(w)
    W = W_full if W_full is not None else si.gen_weights(shape)
    report = {}
    B = w.block
    with Ctx(shape, W, block=w.block, max_batch=w.batch, max_seq=w.max_seq,
             max_prefill_rows=w.batch * w.prompt_max) as ctx:
        ctx.prefill(ids, lens)
        # ---- block 1, step 1: all masked
        got = _check_step(ctx, w, W, name, "b1s1", layers, seqs, lens, report=report)
        # ---- block 1, step 2: the GPU's own partially unmasked block (what step 1 left), a middle layer and the head
        mid = shape.n_layers // 2
        got2 = _check_step(ctx, w, W, name, "b1s2", [mid, shape.n_layers - 1], seqs[:1], lens, got["ids"], got["mask"], report=report)
        assert (got["mask"].sum(axis=1) > got2["mask"].sum(axis=1)).all() or not got["mask"].any()
        # ---- finish block 1 on the GPU, store it, and check step 1 of block 2 (the prefix now holds a generated block)
        cur = got2
        for _ in range(B):
            if not cur["mask"].any():
                break
            cur = ctx.step(cur["ids"], cur["mask"], w.threshold)
        assert not cur["mask"].any()
        ctx.commit(cur["ids"])
        assert np.array_equal(ctx.get_prefix(w.batch), lens + B)
        _check_step(ctx, w, W, name, "b2s1", [0, shape.n_layers - 1], seqs[:1], lens + B, report=report)
        assert ctx.error_word() == 0
        # the rounding classes stay a small share of the rows compared (counts are recorded)
        assert report.get("ids_rounding", 0) + report.get("decision_rounding", 0) <= max(2, report["rows"] // 10), report
        # properties at full size: a whole request, twice
        ctx.prefill(ids, lens)
        tok1, cs1, st1 = ctx.generate(w.batch, w.gen_len, w.threshold)
        ctx.prefill(ids, lens)
        tok2, cs2, st2 = ctx.generate(w.batch, w.gen_len, w.threshold)
        assert np.array_equal(tok1, tok2) and np.array_equal(cs1, cs2)
        assert tok1.min() >= 0 and tok1.max() < shape.vocab and not (tok1 == shape.mask_id).any()
        assert st1.tokens_committed == w.batch * w.gen_len
        assert st1.finalize_forwards == w.batch * (w.gen_len // w.block)
        assert w.batch * (w.gen_len // w.block) <= st1.denoise_forwards <= w.batch * w.gen_len
        assert cs1.min() >= 1 and cs1.max() <= w.block
        assert ctx.error_word() == 0
        report["tokens_per_denoise_forward"] = w.batch * w.gen_len / st1.denoise_forwards
        hist = d3.d3_commit_histogram(ctx.ctx, B + 1)
        assert sum(hist) == st1.denoise_forwards and sum(k * h for k, h in enumerate(hist)) == w.batch * w.gen_len
    record_report(f"fullsize_{name}", report)
    print(name, report)
    return report


@pytest.fixture(scope="module")
def llada_weights():
    return si.gen_weights(si.LLADA8B)


def test_c2_full_size(llada_weights):
    _check_workload("c2", layers=[0, 17, 31], seqs=[0], W_full=llada_weights)


def test_c3_full_size_ragged_batch(llada_weights):
    # 32 sequences with prompt lengths in [128, 512]: check the shortest, the longest and one more
    _, lens = si.gen_prompts(si.WORKLOADS["c3"])
    seqs = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 7})
    _check_workload("c3", layers=[0, 31], seqs=seqs, W_full=llada_weights)


def test_c5_full_size_long_prefix(llada_weights):
    _check_workload("c5", layers=[0, 31], seqs=[0, 3], W_full=llada_weights)


def test_c4_full_size_gqa():
    _check_workload("c4", layers=[0, 27], seqs=[0, 5])


def test_c2_full_size_sampling_refresh_and_multiblock(llada_weights):
    """The widened decoding features at the full 8B shape (batch 1, 32-row forwards, 126464-token head):
    the tokens the sampling epilogue draws are the oracle's Gumbel-max rule applied to the device's own
    fp32 logits of the same forward (all 988 vocabulary tiles, ragged last tile); a KV-refresh of a
    prompt-only cache changes no bit of the next logits, and after a stored block it does; multi-block
    decoding with four blocks in flight commits every token in fewer rounds than block-by-block
    decoding takes forwards, reproducibly."""
    w = si.WORKLOADS["c2"]
    shape = w.model
    ids, lens = si.gen_prompts(w)
    B = w.block
    with Ctx(shape, llada_weights, block=B, max_batch=w.batch, max_seq=w.max_seq, max_prefill_rows=w.batch * w.max_seq) as ctx:
        # ---- sampling against the device's own logits
        ctx.prefill(ids, lens)
        blk = np.full((1, B), shape.mask_id, dtype=np.int32)
        mask = np.ones((1, B), dtype=bool)
        lg = ctx.logits(blk)[0]
        greedy = np.argmax(np.where(np.arange(shape.vocab)[None, :] == shape.mask_id, -np.inf, lg), axis=1)
        away = 0
        for T, seed in [(0.1, 20260107), (4.0, (9 << 32) + 5)]:     # the paper's setting, and one that does move tokens
            ctx.prefill(ids, lens)                                   # the step counter of the explicit calls starts again
            d3.d3_set_sampling(ctx.ctx, T, seed)
            got = ctx.step(blk, mask, w.threshold)
            d3.d3_set_sampling(ctx.ctx, 0.0, 0)
            noise = o.gumbel_noise(seed, 0, lens[0] + np.arange(B), 1, shape.vocab)
            conf, tok, ent = o.sample_stats(lg, shape.mask_id, T, noise)
            pert = lg.astype(np.float32) + np.float32(T) * noise
            pert[:, shape.mask_id] = -np.inf
            top = np.sort(pert, axis=1)[:, -2:]
            clear = (top[:, 1] - top[:, 0]) > 1e-3       # the two paths' logits differ by their K-split order
            assert clear.sum() >= B - 2
            assert np.array_equal(got["tok"][0][clear], tok[clear])
            same = got["tok"][0] == tok
            assert np.allclose(got["conf"][0][same], conf[same], rtol=1e-3, atol=1e-7)
            assert np.allclose(got["ent"][0], ent, rtol=1e-3, atol=1e-4)
            away += int((tok != greedy).sum())
            print("c2 sampling T", T, ": rows compared", int(clear.sum()), "rows drawn away from the arg max", int((tok != greedy).sum()))
        assert away > 0
        # ---- KV-refresh
        ctx.prefill(ids, lens)
        base = ctx.logits(blk)
        d3.d3_refresh_cache(ctx.ctx, 1)
        assert np.array_equal(ctx.logits(blk), base)
        stored = np.random.default_rng(1).integers(0, shape.vocab - 2, size=(1, B)).astype(np.int32)
        ctx.commit(stored)
        before = ctx.logits(blk)
        d3.d3_refresh_cache(ctx.ctx, 1)
        after = ctx.logits(blk)
        assert np.isfinite(after[:, :, :shape.mask_id]).all() and np.abs(after - before)[:, :, :shape.mask_id].max() > 0
        assert np.array_equal(ctx.get_prefix(1), lens + B) and ctx.error_word() == 0
        # ---- multi-block decoding, four blocks in flight (128-row rounds)
        ctx.prefill(ids, lens)
        tok1, _, st1 = ctx.generate(1, w.gen_len, w.threshold)
        ctx.prefill(ids, lens)
        mb1, cr1, sm1 = ctx.generate_multiblock(1, w.gen_len, w.threshold, 4)
        ctx.prefill(ids, lens)
        mb2, cr2, sm2 = ctx.generate_multiblock(1, w.gen_len, w.threshold, 4)
        assert np.array_equal(mb1, mb2) and np.array_equal(cr1, cr2)
        assert sm1.tokens_committed == w.gen_len and not (mb1 == shape.mask_id).any() and mb1.min() >= 0 and mb1.max() < shape.vocab
        assert sm1.steps < st1.denoise_forwards + st1.finalize_forwards and cr1.min() >= 1 and cr1.max() <= sm1.steps
        assert ctx.error_word() == 0
        print("c2 multi-block: rounds", sm1.steps, "against", st1.denoise_forwards + st1.finalize_forwards, "forwards block by block")


def test_c2_full_size_windows_of_two_and_four_blocks(llada_weights):
    """The 64-row forward of two segments (the form in which d3_generate runs a block's finalize forward
    together with the next block's first step) and the 128-row round of four segments (multi-block
    decoding) at the full 8B shape: a tapped layer is recomputed by the oracle segment by segment from
    the GPU's own inputs (segment k sees the prefix and segments 0..k-1 as the same forward wrote them),
    and the statistics of the last layer's rows are compared with the oracle's."""
    w = si.WORKLOADS["c2"]
    shape = w.model
    ids, lens = si.gen_prompts(w)
    B, d = w.block, shape.d_model
    L = int(lens[0])
    report = {}
    rng = np.random.default_rng(11)
    with Ctx(shape, llada_weights, block=B, max_batch=4, max_seq=w.max_seq, max_prefill_rows=w.prompt_max) as ctx:
        for n_win in (2, 4):
            # segment 0 complete (random real tokens), later segments progressively more masked
            blocks = []
            for k in range(n_win):
                keep = rng.random(B) < (1.0 if k == 0 else 0.6 - 0.2 * k)
                blocks.append(np.where(keep, rng.integers(0, shape.vocab - 2, size=B), shape.mask_id).astype(np.int32))
            win = torch.tensor(np.concatenate(blocks)[None, :], device=DEV)
            R = n_win * B
            for layer in (1, shape.n_layers - 1):
                ctx.prefill(ids, lens)
                d3.d3_set_tap(ctx.ctx, layer)
                conf = torch.empty(R, dtype=torch.float32, device=DEV)
                ent = torch.empty_like(conf)
                am = torch.empty(R, dtype=torch.int32, device=DEV)
                d3.d3_denoise_window(ctx.ctx, win, n_win, conf, ent, am)
                x_in = torch.empty((R, d), dtype=torch.float32, device=DEV)
                x_out = torch.empty_like(x_in)
                d3.d3_read_tap(ctx.ctx, x_in, x_out, R)
                torch.cuda.synchronize()
                d3.d3_set_tap(ctx.ctx, -1)
                x_in, x_out = x_in.cpu().numpy(), x_out.cpu().numpy()
                k_all, v_all = _read_kv(ctx, shape, layer, 0, L + R)
                model = _layer_model(shape, llada_weights, layer)
                for k in range(n_win):
                    rows = slice(k * B, (k + 1) * B)
                    seen = L + k * B   # the prefix and the earlier segments
                    ref_out, k_rows, v_rows = model.layer_forward(layer, x_in[rows].astype(np.float32), seen + np.arange(B),
                                                                  k_all[:seen], v_all[:seen])
                    upd_ref, upd_got = ref_out - x_in[rows], x_out[rows] - x_in[rows]
                    err = float(np.max(np.abs(upd_got - upd_ref)) / np.max(np.abs(upd_ref)))
                    kerr = float(np.max(np.abs(k_all[seen:seen + B] - k_rows)) / np.max(np.abs(k_rows)))
                    verr = float(np.max(np.abs(v_all[seen:seen + B] - v_rows)) / np.max(np.abs(v_rows)))
                    report[f"win{n_win}:layer{layer}:seg{k}"] = [err, kerr, verr]
                    assert err <= 3e-2 and kerr <= 3e-2 and verr <= 3e-2, (n_win, layer, k, err, kerr, verr)
                    if layer == shape.n_layers - 1:
                        lg = model.logits(x_out[rows].astype(np.float32))
                        _, o_conf, o_tok, _ = o.softmax_stats(lg, shape.mask_id)
                        gap = top2_gap(lg, shape.mask_id)
                        g_conf, g_tok = conf.cpu().numpy()[rows], am.cpu().numpy()[rows]
                        serr = float(np.max(np.abs(g_conf - o_conf)))
                        report[f"win{n_win}:stat_err:seg{k}"] = serr
                        assert serr <= 5e-2
                        assert not ((g_tok != o_tok) & (gap > 2 * serr + EPS)).any()
            assert ctx.error_word() == 0
        # which kernels ran: the 64-row forward as a chain launch, the 128-row one on the per-matmul kernels
        assert d3.d3_launch_count_of(ctx.ctx, "chain_kernel") > 0
    record_report("fullsize_c2_windows", report)


def test_c5_prefill_cache_rows_against_the_oracle(llada_weights):
    """Prefill as an output at the long-prompt shape (4 x 4096 prompt rows: the 256-column-tile matmuls
    and the prefill attention): the stored K/V of layers 0 and 1 of one sequence against the oracle's
    forward over the prompt rows (layer 0 from the embeddings, layer 1 from the oracle's own layer-0
    output, so layer 1 also checks the GPU's layer-0 attention, O-proj and FFN over 4096 keys)."""
    w = si.WORKLOADS["c5"]
    shape = w.model
    ids, lens = si.gen_prompts(w)
    seq = 1
    P = int(lens[seq])
    with Ctx(shape, llada_weights, block=w.block, max_batch=w.batch, max_seq=w.max_seq,
             max_prefill_rows=w.batch * w.prompt_max) as ctx:
        ctx.prefill(ids, lens)
        got = [_read_kv(ctx, shape, layer, seq, P) for layer in (0, 1)]
        assert ctx.error_word() == 0
    model = o.model_from_shape(shape, {"layers": {0: llada_weights["layers"][0], 1: llada_weights["layers"][1]},
                                       "lm_head": llada_weights["lm_head"], "tok_emb": llada_weights["tok_emb"]}, np.float32)
    x = model.embed(ids[seq, :P])
    pos = np.arange(P)
    report = {}
    for layer in (0, 1):
        x, k_rows, v_rows = model.layer_forward(layer, x, pos, None, None)
        k_got, v_got = got[layer]
        kerr = float(np.max(np.abs(k_got - k_rows)) / np.max(np.abs(k_rows)))
        verr = float(np.max(np.abs(v_got - v_rows)) / np.max(np.abs(v_rows)))
        report[f"layer{layer}"] = [kerr, verr]
        assert kerr <= 3e-2 and verr <= 3e-2, (layer, kerr, verr)
    record_report("fullsize_c5_prefill_cache", report)


def test_c2_full_request_free_running_against_the_stored_oracle_decode(llada_weights):
    """The whole c2 request, free-running, against the oracle's own decode of it (stored: it takes the
    oracle tens of minutes; tests/golden/make_c2_oracle_trace.py writes it from oracle/ alone).  Tokens and
    commit steps are compared block by block; at the first block that differs, the earliest step at which
    the two sides decided differently must be a near-tie of the oracle -- margin below 1e-3, or at most
    twice the largest end-to-end confidence error between the two sides, which is measured here: at every
    (re)synchronisation both sides are in the same state, and the GPU's statistics of the fully masked
    block are compared with the stored ones of the oracle (32 layers of bf16 roundings apart) -- and the
    GPU is re-synchronised from the oracle's tokens at the next block.  The counts are recorded.

    What this test can and cannot show.  Over a whole 32-layer forward the bf16 roundings of the
    activations (the same storage points on both sides, but different outcomes wherever the fp32 sums
    differ in their last bits) add up to a few per cent of the largest logit, end to end, and a logit
    difference of one unit moves a confidence by up to 0.25: measured here, confidences of the same state
    differ by up to 0.3-0.4 between the GPU and the oracle, and as much between two GPU schedules.  Token
    sequences of the 8B-shaped random model therefore part early and legitimately; bit-level parity at
    this size is carried by the decoupled checks above (sampled layers, head, decisions from the GPU's own
    inputs).  What is asserted here: every first difference lies inside the measured end-to-end
    difference, the arg-max tokens of the same state agree on most rows, the end-to-end difference stays
    below 0.5, and both sides need a similar number of forwards."""
    import json
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "c2_oracle_trace.json")
    if not os.path.exists(path):
        pytest.skip("no stored oracle decode of c2")
    with open(path) as f:
        ref = json.load(f)
    w = si.WORKLOADS["c2"]
    assert ref["workload"] == "c2" and ref["gen_len"] == w.gen_len and ref["block"] == w.block
    shape = w.model
    ids, lens = si.gen_prompts(w)
    B, tau = w.block, w.threshold
    want_tok = np.array(ref["tokens"], dtype=np.int32)
    want_cs = np.array(ref["commit_step"], dtype=np.int32)
    n_blocks = w.gen_len // B
    report = dict(blocks=n_blocks, resyncs=0, excused=0, rounding=0, margins=[], oracle_denoise_forwards=ref["n_denoise"])
    stat_err = 0.0
    agree = []
    with Ctx(shape, llada_weights, block=B, max_batch=1, max_seq=w.max_seq, max_prefill_rows=w.prompt_max) as ctx:
        j0 = 0
        first_forwards = None
        while j0 < n_blocks:
            ctx.prefill(ids, lens)
            for jj in range(j0):
                ctx.commit(want_tok[None, jj * B:(jj + 1) * B])
            # same state on both sides: the end-to-end statistic error of a whole forward
            t1 = next(t for t in ref["steps"] if t["block"] == j0 and t["step"] == 1)
            got = ctx.step(np.full((1, B), shape.mask_id, dtype=np.int32), np.ones((1, B), dtype=bool), tau)
            stat_err = max(stat_err, float(np.max(np.abs(got["conf"][0] - np.array(t1["conf"])))))
            assert stat_err <= 0.5, stat_err
            agree.append(float(np.mean(got["tok"][0] == np.array(t1["tok"]))))
            tok, cs, st = ctx.generate(1, w.gen_len - j0 * B, tau)
            if first_forwards is None:
                first_forwards = int(st.denoise_forwards)
            tok, cs = tok[0], cs[0]
            bad = None
            for j in range(n_blocks - j0):
                sl = slice(j * B, (j + 1) * B)
                gl = slice((j0 + j) * B, (j0 + j + 1) * B)
                if not (np.array_equal(tok[sl], want_tok[gl]) and np.array_equal(cs[sl], want_cs[gl])):
                    bad = j
                    break
            if bad is None:
                break
            jb = j0 + bad
            sl = slice(bad * B, (bad + 1) * B)
            gl = slice(jb * B, (jb + 1) * B)
            differ = (tok[sl] != want_tok[gl]) | (cs[sl] != want_cs[gl])
            s_star = int(np.minimum(cs[sl], want_cs[gl])[differ].min())
            t = next(t for t in ref["steps"] if t["block"] == jb and t["step"] == s_star)
            mk = np.array(t["mask_in"], dtype=bool)
            conf, gap = np.array(t["conf"]), np.array(t["gap"])
            ora_commit = np.zeros(B, dtype=bool)
            ora_commit[t["commit"]] = True
            gpu_commit = mk & (cs[sl] == s_star)
            score = np.where(mk, conf, -np.inf)
            order = np.argsort(-score, kind="stable")
            forced_gap = score[order[0]] - score[order[1]] if mk.sum() >= 2 else np.inf
            clears = mk & (conf > tau)
            margins = []
            for r in np.flatnonzero(gpu_commit != ora_commit):
                m = abs(conf[r] - tau)
                if not clears.any() or r == order[0] or (gpu_commit[r] and not clears[r]):
                    m = min(m, forced_gap)
                margins.append(float(m))
            both = gpu_commit & ora_commit
            margins.extend(float(gap[r]) for r in np.flatnonzero(both & (tok[sl] != want_tok[gl])))
            assert margins, ("block differs but not at its first differing step", jb, s_star)
            worst = max(margins)
            assert worst <= max(2 * stat_err, EPS), ("divergence that no near-tie explains", jb, s_star, margins, stat_err)
            report["excused" if worst < EPS else "rounding"] += 1
            report["margins"].append(round(worst, 6))
            report["resyncs"] += 1
            j0 = jb + 1
        report["gpu_denoise_forwards_first_run"] = first_forwards
        report["end_to_end_stat_err"] = stat_err
        report["argmax_agreement_at_sync_points"] = [round(a, 3) for a in agree]
        assert ctx.error_word() == 0
    record_report("fullsize_c2_free_running_vs_stored_oracle", report)
    assert report["resyncs"] <= n_blocks
    assert np.mean(agree) >= 0.7, agree
    assert 0.6 * ref["n_denoise"] <= first_forwards <= 1.6 * ref["n_denoise"], (first_forwards, ref["n_denoise"])
