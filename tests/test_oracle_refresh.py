"""Pins for the oracle's KV-refresh and cache delay (Sec. 3.2, KV-cache and KV-refresh mechanism).

The refresh is checked against cache-free forwards under an explicit visibility matrix (a path that
never touches the cache code), against what the arithmetic fixes (layer-0 keys and values depend on a
position's own token only) and against the runs without refresh where the two must coincide."""
import numpy as np
import pytest

from oracle import d3_oracle as o
from paper_2601_07568_b200 import synth_inputs as si
from test_oracle_decoding import micro_model


def _c1_model():
    w = si.WORKLOADS["c1"]
    model = o.model_from_shape(w.model, si.gen_weights(w.model), dtype=np.float64)
    ids, lens = si.gen_prompts(w)
    return w, model, ids[0, :lens[0]]


def _state_after(model, prompt, blocks):
    st = model.prefill(prompt)
    for b in blocks:
        st = model.finalize_block(st, b)
    return st


def test_refresh_keeps_layer0_and_changes_deeper_layers():
    """Layer-0 K and V are functions of a position's own token and position, so a refresh cannot change
    them; from layer 1 on the prompt rows have now seen the stored blocks, so they must change."""
    m = micro_model(n_layers=3)
    rng = np.random.default_rng(5)
    prompt = rng.integers(0, 38, size=6)
    blocks = [rng.integers(0, 38, size=4) for _ in range(2)]
    st = _state_after(m, prompt, blocks)
    rf = m.refresh(st)
    assert rf.prefix_len == st.prefix_len == 14 and np.array_equal(rf.ids, np.concatenate([prompt] + blocks))
    assert np.allclose(rf.k[0], st.k[0], rtol=0, atol=1e-12) and np.allclose(rf.v[0], st.v[0], rtol=0, atol=1e-12)
    for l in (1, 2):
        assert np.abs(rf.k[l][:6] - st.k[l][:6]).max() > 1e-6      # prompt rows now see the blocks
        # the last stored block saw everything before the refresh already: unchanged only in what it
        # reads from itself; its inputs from earlier rows changed, so it changes as well
        assert np.abs(rf.v[l][:10] - st.v[l][:10]).max() > 1e-6


def test_refresh_of_a_prompt_only_cache_is_the_identity():
    m = micro_model()
    prompt = np.arange(7) % 38
    st = m.prefill(prompt)
    rf = m.refresh(st)
    for a, b in zip(st.k + st.v, rf.k + rf.v):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("n_done", [1, 3])
def test_block_forward_after_refresh_is_a_cache_free_forward_over_one_merged_segment(n_done):
    """After a refresh the stored prefix behaves as one bidirectional segment: the next block's
    statistics equal those of a forward without any cache in which prompt and stored blocks form
    segment 0 and the block segment 1."""
    m = micro_model(n_layers=2)
    rng = np.random.default_rng(11)
    prompt = rng.integers(0, 38, size=5)
    blocks = [rng.integers(0, 38, size=4) for _ in range(n_done)]
    cur = np.array([m.mask_id, 3, m.mask_id, 9])
    st = m.refresh(_state_after(m, prompt, blocks))
    _, conf, tok, ent = m.denoise_forward(st, cur)
    _, c2, t2, e2 = m.brute_force_block(np.concatenate([prompt] + blocks), [], cur)
    assert np.allclose(conf, c2, rtol=1e-10, atol=1e-13) and np.array_equal(tok, t2) and np.allclose(ent, e2, rtol=1e-9, atol=1e-12)
    # and it differs from the block-causal cache (otherwise the refresh would be vacuous)
    _, c3, _, _ = m.denoise_forward(_state_after(m, prompt, blocks), cur)
    assert np.abs(c3 - conf).max() > 1e-9


@pytest.mark.parametrize("every", [1, 2])
def test_generate_with_refresh_matches_cache_free_forwards_segment_by_segment(every):
    """Every denoise step of a run with periodic refresh against a forward without cache: what was
    stored at the last refresh is one segment, each block stored since is a segment of its own."""
    w, model, prompt = _c1_model()
    B, n_blocks = w.block, w.gen_len // w.block
    res = model.generate(prompt, w.gen_len, B, 0.9, record=True, refresh_every=every)
    assert res["n_refresh"] == (n_blocks - 1) // every
    toks = res["tokens"]
    checked = 0
    for t in res["trace"]:
        j = t["block"]
        if t["step"] != 1 and not (j == n_blocks - 1 and t["step"] == 2):
            continue
        merged = (j // every) * every                      # blocks inside the refreshed segment
        base = np.concatenate([prompt] + [toks[q * B:(q + 1) * B] for q in range(merged)])
        later = [toks[q * B:(q + 1) * B] for q in range(merged, j)]
        _, c2, t2, _ = model.brute_force_block(base, later, t["ids_in"])
        assert np.allclose(t["conf"], c2, rtol=1e-9, atol=1e-12) and np.array_equal(t["tok"], t2)
        checked += 1
    assert checked >= n_blocks


def test_refresh_period_beyond_the_request_changes_nothing():
    w, model, prompt = _c1_model()
    a = model.generate(prompt, w.gen_len, w.block, 0.9)
    b = model.generate(prompt, w.gen_len, w.block, 0.9, refresh_every=w.gen_len // w.block)
    assert b["n_refresh"] == 0 and np.array_equal(a["tokens"], b["tokens"]) and np.array_equal(a["commit_step"], b["commit_step"])
    c = model.generate_multiblock(prompt, w.gen_len, w.block, 0.9, o.MODE_CONFIDENCE, max_active=2)
    d = model.generate_multiblock(prompt, w.gen_len, w.block, 0.9, o.MODE_CONFIDENCE, max_active=2, refresh_every=10 ** 6)
    assert d["n_refresh"] == 0 and np.array_equal(c["tokens"], d["tokens"]) and c["rounds"] == d["rounds"]


def test_refresh_changes_later_blocks_only():
    """Tokens decoded before the first refresh are those of the run without refresh."""
    w, model, prompt = _c1_model()
    B = w.block
    a = model.generate(prompt, w.gen_len, B, 0.9)
    b = model.generate(prompt, w.gen_len, B, 0.9, refresh_every=2)
    assert np.array_equal(a["tokens"][:2 * B], b["tokens"][:2 * B])
    assert b["n_refresh"] >= 1 and not np.any(b["tokens"] == w.model.mask_id)


@pytest.mark.parametrize("delay", [1, 2, 3])
def test_cache_delay_counts_stabilizing_rounds(delay):
    """A complete block leaves the window after exactly `delay` forwards in which it was complete, in
    order; with one block in flight every block then costs delay - 1 rounds more than with delay 1,
    and the tokens are the same (a complete block's K/V do not depend on how often they are recomputed)."""
    w, model, prompt = _c1_model()
    B, n_blocks = w.block, w.gen_len // w.block
    base = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=1)
    res = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=1, cache_delay=delay)
    assert np.array_equal(res["tokens"], base["tokens"])
    assert res["rounds"] == base["rounds"] + (delay - 1) * n_blocks
    for a, b in zip(res["state"].k, base["state"].k):
        assert np.array_equal(a, b)
    # several blocks in flight: count the complete-before rounds of every block from the trace
    res = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=3, cache_delay=delay, record=True)
    seen = np.zeros(n_blocks, dtype=int)
    last_lo = 0
    for t in res["trace"]:
        assert t["lo"] >= last_lo
        for q in range(last_lo, t["lo"]):
            assert seen[q] == delay                     # stored exactly after `delay` stabilizing forwards
        last_lo = t["lo"]
        for k in range(t["n_win"]):
            if t["complete_before"][k]:
                seen[t["lo"] + k] += 1
                assert seen[t["lo"] + k] <= delay
    assert np.all(seen[last_lo:] == delay) and not np.any(res["tokens"] == w.model.mask_id)


def test_multiblock_refresh_rounds_and_equivalence_with_manual_refresh():
    """refresh_every = r refreshes after rounds r, 2r, ... while blocks are in flight and something is
    stored; replaying the trace by hand (refreshing a separately built cache at those rounds) gives
    the statistics the run recorded."""
    w, model, prompt = _c1_model()
    B = w.block
    r = 3
    res = model.generate_multiblock(prompt, w.gen_len, B, 0.9, o.MODE_CONFIDENCE, max_active=2, refresh_every=r, record=True)
    tr = res["trace"]
    assert res["n_refresh"] == sum(1 for t in tr[:-1] if t["round"] % r == 0)   # the prompt is always stored; none after the last round
    st = model.prefill(prompt)
    stored = 0
    for t in tr:
        while stored < t["lo"]:
            st = model.finalize_block(st, res["tokens"][stored * B:(stored + 1) * B])
            stored += 1
        if t["round"] > 1 and (t["round"] - 1) % r == 0:
            st = model.refresh(st)
        _, conf, tok, _ = model.denoise_forward(st, t["ids_in"][0])
        assert np.allclose(conf, t["stats"][0][0], rtol=1e-10, atol=1e-13) and np.array_equal(tok, t["stats"][0][1])
