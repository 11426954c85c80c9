"""Pins for the oracle's decoding path: brute force, special cases, an independent torch forward."""
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import d3_oracle as o
from paper_2601_07568_b200 import synth_inputs as si

HERE = os.path.dirname(os.path.abspath(__file__))


def paper_facts():
    facts = {}
    for line in open(os.path.join(HERE, "golden", "paper_facts.txt")):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            facts[k.strip()] = float(v)
    return facts


def micro_model(seed=3, n_layers=2, d=32, hq=4, hkv=2, dh=8, f=48, V=40, scale=4.0, std=0.3):
    """A tiny GQA model with larger weights so that confidences spread over (0,1)."""
    rng = np.random.default_rng(seed)
    lay = {}
    for l in range(n_layers):
        lay[l] = dict(wq=rng.normal(0, std, (hq * dh, d)), wk=rng.normal(0, std, (hkv * dh, d)),
                      wv=rng.normal(0, std, (hkv * dh, d)), wo=rng.normal(0, std, (d, hq * dh)),
                      w_gate=rng.normal(0, std, (f, d)), w_up=rng.normal(0, std, (f, d)),
                      w_down=rng.normal(0, std, (d, f)))
    W = dict(tok_emb=rng.normal(0, 1.0, (V, d)), lm_head=rng.normal(0, std / 4, (V, d)), layers=lay)
    return o.OracleModel(n_layers=n_layers, d_model=d, n_q_heads=hq, n_kv_heads=hkv, d_head=dh, d_ffn=f,
                         vocab=V, mask_id=V - 1, weights=W, logit_scale=scale, dtype=np.float64)


@pytest.fixture(scope="module")
def c1():
    w = si.WORKLOADS["c1"]
    W = si.gen_weights(w.model)
    ids, lens = si.gen_prompts(w)
    return w, o.model_from_shape(w.model, W, np.float64), ids[0, :lens[0]]


# ----------------------------------------------------------------------------- independent forward
def torch_forward(m: o.OracleModel, ids, visible=None):
    """The same architecture written with torch CPU ops (float64), whole sequence, no cache."""
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    n = len(ids)
    x = t(m.w["tok_emb"])[torch.tensor(np.asarray(ids), dtype=torch.long)]
    half = m.d_head // 2
    inv = torch.pow(torch.tensor(m.rope_theta, dtype=torch.float64),
                    -torch.arange(0, m.d_head, 2, dtype=torch.float64) / m.d_head)
    ang = torch.arange(n, dtype=torch.float64)[:, None] * inv[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)  # e^{i angle}

    def rope(z):  # z: [n, h, dh]
        zc = torch.complex(z[..., :half], z[..., half:]) * rot[:, None, :]
        return torch.cat([zc.real, zc.imag], -1)

    am = None if visible is None else torch.tensor(visible)
    for l in range(m.n_layers):
        W = m.w["layers"][l]
        xn = F.rms_norm(x, (m.d_model,), None, m.rms_eps)
        q = rope(F.linear(xn, t(W["wq"])).view(n, m.n_q_heads, m.d_head)).transpose(0, 1)
        k = rope(F.linear(xn, t(W["wk"])).view(n, m.n_kv_heads, m.d_head)).transpose(0, 1)
        v = F.linear(xn, t(W["wv"])).view(n, m.n_kv_heads, m.d_head).transpose(0, 1)
        a = F.scaled_dot_product_attention(q[None], k[None], v[None], attn_mask=am, enable_gqa=True)[0]
        x = x + F.linear(a.transpose(0, 1).reshape(n, -1), t(W["wo"]))
        xn = F.rms_norm(x, (m.d_model,), None, m.rms_eps)
        x = x + F.linear(F.silu(F.linear(xn, t(W["w_gate"]))) * F.linear(xn, t(W["w_up"])), t(W["w_down"]))
    xn = F.rms_norm(x, (m.d_model,), None, m.rms_eps)
    return (F.linear(xn, t(m.w["lm_head"])) * m.logit_scale).numpy()


def test_forward_matches_independent_torch_model_c1(c1):
    w, m, prompt = c1
    ids = np.concatenate([prompt, np.full(w.block, m.mask_id)])
    x, _, _ = m.forward_rows(ids, np.arange(len(ids)), None)
    assert np.allclose(m.logits(x), torch_forward(m, ids), rtol=1e-9, atol=1e-9)


def test_forward_matches_independent_torch_model_gqa_with_segments():
    m = micro_model()
    rng = np.random.default_rng(0)
    ids = rng.integers(0, 38, size=14)
    seg = np.array([0] * 6 + [1] * 4 + [2] * 4)
    vis = seg[None, :] <= seg[:, None]
    x, _, _ = m.forward_rows(ids, np.arange(14), None, vis)
    assert np.allclose(m.logits(x), torch_forward(m, ids, vis), rtol=1e-9, atol=1e-9)


# ----------------------------------------------------------------------------- cache == brute force
@pytest.mark.parametrize("P", [0, 1, 5])
def test_cached_prefix_equals_full_recompute(P):
    m = micro_model()
    rng = np.random.default_rng(P)
    B = 4
    prompt = rng.integers(0, 38, size=P)
    state = m.prefill(prompt)
    done = []
    for j in range(3):
        cur = np.full(B, m.mask_id)
        cur[rng.integers(0, B)] = rng.integers(0, 38)  # a partly unmasked block
        lg_c, conf_c, tok_c, ent_c = m.denoise_forward(state, cur)
        lg_b, conf_b, tok_b, ent_b = m.brute_force_block(prompt, done, cur)
        assert np.allclose(lg_c, lg_b, rtol=1e-11, atol=1e-11)
        assert np.allclose(conf_c, conf_b, atol=1e-12) and np.array_equal(tok_c, tok_b)
        final = rng.integers(0, 38, size=B)
        state = m.finalize_block(state, final)
        done.append(final)
    assert state.prefix_len == P + 3 * B


def test_cache_must_hold_final_tokens_not_masked_ones():
    # If the cached K/V came from the last denoise forward (which still saw mask tokens), the next
    # block would differ from the full recompute: the finalize forward is what makes the cache exact.
    m = micro_model()
    prompt = np.array([1, 2, 3])
    state = m.prefill(prompt)
    final = np.array([4, 5, 6, 7])
    good = m.finalize_block(state, final)
    stale = m.finalize_block(state, np.array([4, 5, m.mask_id, 7]))
    cur = np.full(4, m.mask_id)
    ref = m.brute_force_block(prompt, [final], cur)[0]
    assert np.allclose(m.denoise_forward(good, cur)[0], ref, atol=1e-11)
    assert not np.allclose(m.denoise_forward(stale, cur)[0], ref, atol=1e-3)


def test_fully_unmasked_block_is_dense_bidirectional_attention():
    # one segment only (no prompt): every row sees every row -> identical to the plain torch model
    m = micro_model()
    ids = np.array([3, 9, 1, 30, 22, 17])
    lg = m.denoise_forward(m.empty_state(), ids)[0]
    assert np.allclose(lg, torch_forward(m, ids), rtol=1e-9, atol=1e-9)
    # and bidirectional: changing the LAST token changes the FIRST row's logits
    ids2 = ids.copy()
    ids2[-1] = 5
    assert not np.allclose(m.denoise_forward(m.empty_state(), ids2)[0][0], lg[0], atol=1e-6)


def test_later_segments_do_not_influence_earlier_ones():
    m = micro_model()
    prompt = np.array([1, 2, 3, 4])
    a = m.brute_force_block(prompt, [], np.array([5, 6, 7]))[0]
    x, _, _ = m.forward_rows(np.concatenate([prompt, [5, 6, 7], [8, 9, 10]]), np.arange(10), None,
                             (np.array([0] * 4 + [1] * 3 + [2] * 3)[None, :]
                              <= np.array([0] * 4 + [1] * 3 + [2] * 3)[:, None]))
    assert np.allclose(m.logits(x[4:7]), a, atol=1e-11)


# ----------------------------------------------------------------------------- decision rule
def brute_decide(conf, ent, mask, tau, mode):
    B = len(mask)
    out = [False] * B
    best = None
    for r in range(B):
        if not mask[r]:
            continue
        s = conf[r] if mode == 0 else -ent[r]
        if (mode == 0 and conf[r] > tau) or (mode == 1 and ent[r] < tau):
            out[r] = True
        if best is None or s > best[0]:
            best = (s, r)
    if best is not None:
        out[best[1]] = True
    return np.array(out)


def test_decide_matches_brute_force_on_all_small_cases():
    rng = np.random.default_rng(1)
    grid = [0.1, 0.5, 0.5, 0.9]  # repeated value -> ties
    for mask in itertools.product([False, True], repeat=4):
        for _ in range(8):
            conf = rng.choice(grid, size=4)
            ent = rng.choice(grid, size=4)
            for tau in (0.05, 0.5, 0.7, 1.0):
                for mode in (0, 1):
                    got = o.decide(conf, ent, np.array(mask), tau, mode)
                    assert np.array_equal(got, brute_decide(conf, ent, mask, tau, mode))
                    assert not np.any(got & ~np.array(mask))
                    assert got.any() == any(mask)


def test_decide_strict_threshold_and_forced_commit():
    conf = np.array([0.9, 0.95, 0.2, 0.9])
    ent = np.zeros(4)
    m = np.ones(4, bool)
    assert list(o.decide(conf, ent, m, 0.9, 0)) == [False, True, False, False]  # 0.9 is not > 0.9
    assert list(o.decide(conf, ent, m, 0.99, 0)) == [False, True, False, False]  # forced top-1
    assert list(o.decide(conf, ent, np.array([1, 0, 1, 1], bool), 0.99, 0)) == [True, False, False, False]
    assert list(o.decide(conf, ent, m, 0.1, 0)) == [True] * 4


def test_commit_set_shrinks_as_threshold_rises(c1):
    w, m, prompt = c1
    mm = micro_model()
    state = mm.prefill(np.array([1, 2, 3]))
    ids = np.full(8, mm.mask_id)
    _, conf, tok, ent = mm.denoise_forward(state, ids)
    prev = None
    for tau in np.linspace(0.0, 1.0, 21):
        c = o.decide(conf, ent, np.ones(8, bool), tau, 0)
        assert c.sum() >= 1
        if prev is not None:
            assert not np.any(c & ~prev)
        prev = c


# ----------------------------------------------------------------------------- whole loop
def test_threshold_one_is_sequential_most_confident_first():
    facts = paper_facts()
    m = micro_model()
    prompt = np.array([7, 8, 9, 10, 11])
    r = m.generate(prompt, 16, 4, 1.0, record=True)
    tok, order = m.sequential_decode(prompt, 16, 4)
    assert np.array_equal(r["tokens"], tok)
    assert all(t["commit"].sum() == facts["min_tokens_per_forward"] for t in r["trace"])
    assert r["n_denoise"] == 16 and r["tpf_denoise"] == facts["tpf_one_token_per_step"]
    got_order = [t["block"] * 4 + int(np.argmax(t["commit"])) for t in r["trace"]]
    assert got_order == list(order)


def test_threshold_one_c1_equals_sequential(c1):
    w, m, prompt = c1
    r = m.generate(prompt, w.gen_len, w.block, 1.0)
    tok, _ = m.sequential_decode(prompt, w.gen_len, w.block)
    assert np.array_equal(r["tokens"], tok)


def test_tiny_threshold_commits_whole_block_in_one_step():
    m = micro_model()
    r = m.generate(np.array([1, 2, 3]), 12, 4, 1.0 / m.vocab - 1e-9)
    assert r["n_denoise"] == 3 and r["tpf_denoise"] == 4.0 and r["n_finalize"] == 3


def test_progress_and_step_bounds():
    m = micro_model(seed=5)
    for tau in (0.2, 0.5, 0.9):
        r = m.generate(np.array([4, 4, 4, 4]), 24, 8, tau, record=True)
        for t in r["trace"]:
            assert t["mask_out"].sum() < t["mask_in"].sum()
            assert t["step"] <= 8
            assert np.array_equal(t["ids_out"][~t["mask_in"]], t["ids_in"][~t["mask_in"]])
        assert np.all(r["tokens"] != m.mask_id) and np.all(r["commit_step"] >= 1)
        assert r["n_finalize"] == 3


def test_entropy_mode_runs_and_orders_by_entropy():
    m = micro_model(seed=6)
    r = m.generate(np.array([1, 2]), 8, 4, 0.45, mode=o.MODE_ENTROPY, record=True)
    for t in r["trace"]:
        masked = np.flatnonzero(t["mask_in"])
        best = masked[np.argmin(t["ent"][masked])]
        assert t["commit"][best]
        assert np.array_equal(t["commit"][masked] & (masked != best), (t["ent"][masked] < 0.45) & (masked != best))


def test_paper_block_arithmetic():
    f = paper_facts()
    assert f["max_generation_length"] / f["block_size"] == f["blocks_per_generation"]
    w = si.WORKLOADS["c2"]
    assert w.block == f["block_size"] and w.gen_len == f["max_generation_length"]


def test_batch_elements_are_independent_and_deterministic(c1):
    w, m, prompt = c1
    a = m.generate(prompt, 32, 16, 0.3)
    b = m.generate(prompt, 32, 16, 0.3)
    assert np.array_equal(a["tokens"], b["tokens"]) and a["n_denoise"] == b["n_denoise"]


def test_mirror_mode_stays_close_to_exact():
    w = si.WORKLOADS["c1"]
    shape = si.scaled_shape(si.LLADA8B, name="s", n_layers=2, d_model=128, n_q_heads=2, n_kv_heads=2,
                            d_ffn=256, vocab=300, d_head=64)
    W = si.gen_weights(shape)
    ids = np.arange(20) % 290
    a = o.model_from_shape(shape, W, np.float64)
    b = o.model_from_shape(shape, W, np.float32, mirror_bf16=True)
    la = a.denoise_forward(a.prefill(ids[:12]), ids[12:])[0]
    lb = b.denoise_forward(b.prefill(ids[:12]), ids[12:])[0]
    assert np.max(np.abs(la - lb)) < 3e-2 * np.max(np.abs(la))


def test_eos_early_stop_is_a_prefix_of_the_run_without_it():
    """Early stopping on EOS (Sec. 3.2): with the EOS id set to a token that the free run first commits
    at step k of block j, decoding makes exactly the same commits up to and including that step, then
    stops: no later forward, every undecoded position still the mask id, j finalize forwards."""
    w = si.WORKLOADS["c1"]
    W = si.gen_weights(w.model)
    ids, lens = si.gen_prompts(w)
    model = o.model_from_shape(w.model, W, np.float64)
    prompt = ids[0, :lens[0]]
    free = model.generate(prompt, w.gen_len, w.block, 0.3, record=True)
    assert not free["stopped_early"] and free["n_finalize"] == w.gen_len // w.block
    trace = free["trace"]
    # the last step (not the very first) that commits a token no earlier step has committed
    seen = set()
    pick = None
    for n, t in enumerate(trace):
        toks = [int(x) for x in t["ids_out"][t["commit"]]]
        fresh = [x for x in toks if x not in seen]
        if n >= 1 and fresh:
            pick = (n, fresh[0])
        seen.update(toks)
    assert pick is not None and trace[pick[0]]["block"] >= 1
    n_stop, eos = pick
    got = model.generate(prompt, w.gen_len, w.block, 0.3, eos_id=eos)
    t = trace[n_stop]
    assert got["stopped_early"]
    assert got["n_denoise"] == n_stop + 1 and got["n_finalize"] == t["block"]
    want = np.full(w.gen_len, w.model.mask_id, dtype=np.int32)
    B = w.block
    want[:t["block"] * B] = free["tokens"][:t["block"] * B]
    want[t["block"] * B:(t["block"] + 1) * B] = np.where(t["mask_out"], w.model.mask_id, t["ids_out"])
    assert np.array_equal(got["tokens"], want)
    assert np.any(got["tokens"] == eos) and np.any(got["tokens"] == w.model.mask_id)
    assert got["n_denoise"] < free["n_denoise"]
    # an id that never comes up changes nothing
    never = next(x for x in range(w.model.vocab) if x not in seen and x != w.model.mask_id)
    same = model.generate(prompt, w.gen_len, w.block, 0.3, eos_id=never)
    assert not same["stopped_early"] and np.array_equal(same["tokens"], free["tokens"])


# ----------------------------------------------------------------------------- multi-block decoding
def _c1_model():
    w = si.WORKLOADS["c1"]
    W = si.gen_weights(w.model)
    ids, lens = si.gen_prompts(w)
    return w, o.model_from_shape(w.model, W, np.float64), ids[0, :lens[0]]


@pytest.mark.parametrize("tau,mode", [(0.9, o.MODE_CONFIDENCE), (0.3, o.MODE_CONFIDENCE), (2.42, o.MODE_ENTROPY)])
def test_multiblock_with_one_block_in_flight_is_single_block_decoding(tau, mode):
    """Multi-block decoding (Sec. 3.2) bounded to one block in flight has nothing to run in parallel: the
    same tokens in the same order as block-by-block decoding, one round per denoise or finalize forward."""
    w, model, prompt = _c1_model()
    one = model.generate(prompt, w.gen_len, w.block, tau, mode, record=True)
    mb = model.generate_multiblock(prompt, w.gen_len, w.block, tau, mode, max_active=1)
    assert np.array_equal(mb["tokens"], one["tokens"])
    assert mb["rounds"] == one["n_denoise"] + one["n_finalize"]
    assert all(r == w.block for r in mb["rows"])
    # commit order: rounds of the multi-block run count the finalize forwards of earlier blocks too
    B = w.block
    for j in range(w.gen_len // B):
        steps = one["commit_step"][j * B:(j + 1) * B]
        rounds = mb["commit_round"][j * B:(j + 1) * B]
        assert np.array_equal(rounds - rounds.min(), steps - steps.min())
    for a, b in zip(mb["state"].k, one["state"].k):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("tau,mode,max_active", [(0.3, o.MODE_CONFIDENCE, 2), (2.42, o.MODE_ENTROPY, 3), (0.9, o.MODE_CONFIDENCE, 4)])
def test_multiblock_rounds_follow_the_state_rules_and_the_joint_forward_is_block_causal(tau, mode, max_active):
    """Each round against what the paper fixes: a block is created only once its predecessor is 10 %
    complete, an Activated block (predecessor below 95 %) commits nothing but what clears the threshold,
    a Fully-Activated one at least one token, a complete block commits nothing and enters the cache
    after one more forward, in order.  And the statistics a block in flight gets are those of a
    forward without any cache over prompt + earlier blocks (as they stand) + the block, under
    segment visibility: evaluating the blocks in flight one after the other is the joint forward."""
    w, model, prompt = _c1_model()
    B, n_blocks = w.block, w.gen_len // w.block
    res = model.generate_multiblock(prompt, w.gen_len, B, tau, mode, max_active=max_active, record=True)
    tr = res["trace"]
    assert res["rounds"] == len(tr) and np.all(res["commit_round"] >= 1) and not np.any(res["tokens"] == w.model.mask_id)
    single = model.generate(prompt, w.gen_len, B, tau, mode)
    assert res["rounds"] <= single["n_denoise"] + single["n_finalize"]
    cached: list = []
    checked_joint = 0
    for n, t in enumerate(tr):
        assert 1 <= t["n_win"] <= max_active and res["rows"][n] == t["n_win"] * B
        assert t["lo"] == len(cached)
        for k in range(t["n_win"]):
            m_in, commit = t["mask_in"][k], t["commits"][k]
            conf, tok, ent = t["stats"][k]
            unm_prev = B if k == 0 else int(B - t["mask_in"][k - 1].sum())
            fully = k == 0 or 100 * unm_prev >= 95 * B
            assert fully == t["fully"][k]
            clears = m_in & ((conf > tau) if mode == o.MODE_CONFIDENCE else (ent < tau))
            if not m_in.any():
                assert not commit.any() and t["complete_before"][k]
            elif fully:
                assert commit.sum() >= 1 and np.array_equal(commit | clears, commit) and (commit & ~m_in).sum() == 0
                assert (commit & ~clears).sum() <= 1
            else:
                assert np.array_equal(commit, clears)
            if t["n_win"] >= 2 and k >= 1 and checked_joint < 3:
                lg, c2, t2, e2 = model.brute_force_block(prompt, cached + [t["ids_in"][q] for q in range(k)], t["ids_in"][k])
                assert np.allclose(c2, conf, rtol=1e-9, atol=1e-12) and np.array_equal(t2, tok)
                checked_joint += 1
        # a block appears only when its predecessor is 10 % complete (or nothing was in flight)
        if n + 1 < len(tr):
            nxt = tr[n + 1]
            popped = nxt["lo"] - t["lo"]
            for q in range(popped):
                assert t["complete_before"][q]
                cached.append(t["ids_out"][q])
            if nxt["n_win"] > t["n_win"] - popped:
                assert nxt["n_win"] == t["n_win"] - popped + 1
                if t["n_win"] - popped > 0:
                    assert 100 * int(B - t["mask_out"][-1].sum()) >= 10 * B
                assert nxt["mask_in"][-1].all()
    assert checked_joint >= 1
    assert np.array_equal(np.concatenate(cached + [x for x in tr[-1]["ids_out"]])[:w.gen_len], res["tokens"])


def test_multiblock_eos_stop_is_a_prefix_of_the_free_run_and_window_one_is_single_block():
    """Early stop in multi-block decoding: with the EOS id set to a token first committed in round k (k > 1)
    of the free run, the run makes the same commits up to and including round k and then halts: the
    blocks in flight go out as they stood after that round, nothing later is decoded.  With one block in
    flight it is the early stop of block-by-block decoding."""
    w, model, prompt = _c1_model()
    B = w.block
    free = model.generate_multiblock(prompt, w.gen_len, B, 0.3, o.MODE_CONFIDENCE, max_active=3, record=True)
    seen, pick = set(), None
    for t in free["trace"]:
        toks = [int(x) for k in range(t["n_win"]) for x in t["ids_out"][k][t["commits"][k]]]
        fresh = [x for x in toks if x not in seen]
        if t["round"] >= 2 and fresh and t["round"] < free["rounds"] - 1:
            pick = (t, fresh[0])
        seen.update(toks)
    assert pick is not None
    t, eos = pick
    got = model.generate_multiblock(prompt, w.gen_len, B, 0.3, o.MODE_CONFIDENCE, max_active=3, eos_id=eos)
    assert got["stopped_early"] and got["rounds"] == t["round"] < free["rounds"]
    want = np.full(w.gen_len, w.model.mask_id, dtype=np.int32)
    want[:t["lo"] * B] = free["tokens"][:t["lo"] * B]
    for k in range(t["n_win"]):
        want[(t["lo"] + k) * B:(t["lo"] + k + 1) * B] = np.where(t["mask_out"][k], w.model.mask_id, t["ids_out"][k])
    assert np.array_equal(got["tokens"], want) and np.any(got["tokens"] == eos)
    assert np.array_equal(got["commit_round"][got["tokens"] != w.model.mask_id] <= t["round"], np.ones(int((got["tokens"] != w.model.mask_id).sum()), bool))
    assert got["state"].prefix_len == len(prompt) + t["lo"] * B        # nothing in flight was stored
    # one block in flight: the same tokens as the single-block early stop
    one = model.generate(prompt, w.gen_len, B, 0.3, eos_id=eos)
    mb1 = model.generate_multiblock(prompt, w.gen_len, B, 0.3, o.MODE_CONFIDENCE, max_active=1, eos_id=eos)
    assert one["stopped_early"] and mb1["stopped_early"] and np.array_equal(one["tokens"], mb1["tokens"])


def test_multiblock_sampling_with_one_block_in_flight_draws_per_round():
    """Sampling in multi-block decoding keys the noise by the round; the run is reproducible, depends on
    the seed, and at temperature 0 is the greedy run."""
    w, model, prompt = _c1_model()
    B = w.block
    greedy = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=2)
    zero = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=2, temperature=0.0, seed=5)
    assert np.array_equal(greedy["tokens"], zero["tokens"])
    a = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=2, temperature=0.6, seed=5, record=True)
    b = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=2, temperature=0.6, seed=5)
    c = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=2, temperature=0.6, seed=6)
    assert np.array_equal(a["tokens"], b["tokens"]) and not np.array_equal(a["tokens"], c["tokens"])
    assert not np.array_equal(a["tokens"], greedy["tokens"])
    # the recorded tokens of a round are the Gumbel-max draws for (seed, position, round) from that round's logits
    t = a["trace"][0]
    st = model.prefill(prompt)
    lg, *_ = model.denoise_forward(st, t["ids_in"][0])
    noise = o.gumbel_noise(5, 0, len(prompt) + np.arange(B), 1, w.model.vocab)
    _, tok, _ = o.sample_stats(lg, w.model.mask_id, 0.6, noise)
    assert np.array_equal(tok, t["stats"][0][1])
