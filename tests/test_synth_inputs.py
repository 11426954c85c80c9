"""The seeded input generators: determinism, partial regeneration, value distribution."""
import numpy as np
import torch

from paper_2601_07568_b200 import synth_inputs as si


def test_tensor_is_deterministic_and_row_ranges_match():
    shape = si.scaled_shape(si.LLADA8B, name="s", n_layers=2, d_model=1024, n_q_heads=8, n_kv_heads=8,
                            d_ffn=5000, vocab=9001)
    full = si.gen_tensor(shape, "w_gate", 1)
    assert full.dtype == np.uint16 and full.shape == (5000, 1024)
    assert np.array_equal(full, si.gen_tensor(shape, "w_gate", 1))
    part = si.gen_tensor(shape, "w_gate", 1, rows=(4090, 4200))  # crosses a chunk boundary
    assert np.array_equal(part, full[4090:4200])
    assert not np.array_equal(full[:10], si.gen_tensor(shape, "w_up", 1)[:10])
    assert not np.array_equal(full[:10], si.gen_tensor(shape, "w_gate", 0)[:10])


def test_weight_distribution_and_bf16_rounding():
    x = si.gen_tensor(si.TINY, "w_gate", 0)
    assert x.dtype == np.float32 and abs(x.std() - 0.02) < 5e-4 and abs(x.mean()) < 5e-4
    t = torch.randn(4096)
    bits = si.f32_to_bf16_bits(t.numpy())
    assert np.array_equal(bits, t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(si.bf16_bits_to_f32(bits), t.to(torch.bfloat16).float().numpy())


def test_prompts():
    for name, w in si.WORKLOADS.items():
        ids, lens = si.gen_prompts(w)
        assert ids.shape == (w.batch, w.prompt_max) and ids.dtype == np.int32
        assert lens.min() >= w.prompt_min and lens.max() <= w.prompt_max
        for b in range(w.batch):
            assert np.all(ids[b, :lens[b]] < w.model.vocab - 2) and np.all(ids[b, :lens[b]] >= 0)
            assert np.all(ids[b, lens[b]:] == w.model.pad_id)
    ids, lens = si.gen_prompts(si.WORKLOADS["c3"])
    assert len(set(lens.tolist())) > 8  # ragged


def test_param_counts():
    assert si.LLADA8B.params_per_layer() == 218_103_808
    assert si.QWEN7B.params_per_layer() == 233_046_016
    assert si.TINY.params_per_layer() == 262_144
