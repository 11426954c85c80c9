"""d3_lm_head_stats_static: the LM-head statistics for callers that may not allocate device memory
(allocator frozen, fixed memory budget, real-time loop).  Its scratch is a fixed array inside the
library image instead of a cudaMalloc'd workspace, so the test checks these things through the C ABI:
the results equal those of the context-based d3_op_lm_head_stats on the same inputs, and the CPU
oracle's softmax statistics of the same logits; a second call right after the first (smaller problem,
so stale entries of the first remain in the array) is still right; the free device memory is the same
before and after a call; a problem beyond the array's capacity, and tensors whose sizes do not fit
together, are refused.  The file name sorts last so that a run stopping at the first failure has
already been through every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import d3_oracle as o
from paper_2601_07568_b200 import binding as d3
from paper_2601_07568_b200 import synth_inputs as si
from gpu_utils import DEV, Ctx

pytestmark = pytest.mark.gpu

SHAPE = si.scaled_shape(si.TINY, name="static-stats", n_layers=1, d_model=128, n_q_heads=4, n_kv_heads=4,
                        d_ffn=128, vocab=1000)


def _both(ctx, m, V, k, mask_id, scale, seed, dtype):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn((m, k), generator=g).to(dtype).to(DEV)
    w = (torch.randn((V, k), generator=g) * 0.05).to(dtype).to(DEV)
    outs = []
    for _ in range(2):
        outs.append((torch.full((m,), -1.0, device=DEV), torch.full((m,), -1.0, device=DEV),
                     torch.full((m,), -1, dtype=torch.int32, device=DEV)))
    d3.d3_op_lm_head_stats(ctx.ctx, x, w, scale, mask_id, *outs[0])
    torch.cuda.synchronize()
    d3.d3_lm_head_stats_static(x, w, scale, mask_id, *outs[1])  # a first use may still load kernel code
    torch.cuda.synchronize()
    for t in outs[1]:
        t.fill_(-1)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    d3.d3_lm_head_stats_static(x, w, scale, mask_id, *outs[1])
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0  # the call took no device memory
    (c0, e0, a0), (c1, e1, a1) = [[t.cpu().numpy() for t in out] for out in outs]
    # the oracle's statistics of the same logits (the operands as the kernels see them, product in fp64)
    logits = scale * (x.cpu().to(torch.float64).numpy() @ w.cpu().to(torch.float64).numpy().T)
    _, conf, tok, ent = o.softmax_stats(logits, mask_id)
    return c0, e0, a0, c1, e1, a1, conf, tok, ent


@pytest.mark.parametrize("dtype,impl", [(torch.float32, d3.D3_GEMM_AUTO), (torch.bfloat16, d3.D3_GEMM_SIMT),
                                        (torch.bfloat16, d3.D3_GEMM_AUTO)])
def test_static_stats_match_context_entry_point_twice_in_a_row(dtype, impl):
    shape = SHAPE if dtype == torch.float32 else si.scaled_shape(SHAPE, name="static-stats-bf16", n_layers=1,
                                                                 d_model=128, n_q_heads=4, n_kv_heads=4,
                                                                 d_ffn=128, vocab=1000, dtype="bf16")
    with Ctx(shape, None, block=32, max_batch=2, max_seq=64, gemm_impl=impl) as ctx:
        # first call: 40 rows x 1000 columns (8 tiles); second: fewer rows, fewer tiles, other mask id
        for m, V, k, mask_id, scale, seed in [(40, 1000, 128, 999, 20.0, 1), (7, 300, 64, 130, 3.0, 2)]:
            c0, e0, a0, c1, e1, a1, conf, tok, ent = _both(ctx, m, V, k, mask_id, scale, seed, dtype)
            # against the oracle: fp32 accumulation of exact products of the stored operands
            assert np.max(np.abs(c1 - conf)) <= 1e-4 and np.max(np.abs(e1 - ent)) <= 1e-3
            differ_o = a1 != tok
            assert not (differ_o & (conf > 0.6)).any()  # another token only where the two best are close
            same_kernels = dtype == torch.float32 or impl == d3.D3_GEMM_SIMT
            if same_kernels:  # both entry points run the same SIMT kernels: identical bits
                assert np.array_equal(c0, c1) and np.array_equal(e0, e1) and np.array_equal(a0, a1)
            else:  # context path on the tensor cores: tolerance of tests/test_gpu_ops.py for bf16 statistics
                assert np.max(np.abs(c0 - c1)) <= 3e-3 and np.max(np.abs(e0 - e1)) <= 9e-3
                differ = a0 != a1
                assert not (differ & (np.minimum(c0, c1) > 0.6)).any()  # only near-ties may pick another token
            assert np.all(a1 != mask_id) and np.all((a1 >= 0) & (a1 < V))
            assert np.all((c1 > 0) & (c1 <= 1.0 + 1e-6)) and np.all(e1 >= 0)
        assert ctx.error_word() == 0


def test_static_stats_refuses_sizes_beyond_the_array():
    x = torch.zeros((8, 8), device=DEV)
    c = torch.zeros(8, device=DEV)
    a = torch.zeros(8, dtype=torch.int32, device=DEV)
    L = d3.lib()
    m = d3.D3_STATIC_MAX_PARTIALS // 2 + 1  # two tiles per row -> one entry too many
    rc = L.d3_lm_head_stats_static(C.c_void_p(x.data_ptr()), C.c_void_p(x.data_ptr()), C.c_int32(d3.D3_DTYPE_F32),
                                   C.c_int32(m), C.c_int32(256), C.c_int32(8), C.c_float(1.0), C.c_int32(0),
                                   C.c_void_p(c.data_ptr()), C.c_void_p(c.data_ptr()), C.c_void_p(a.data_ptr()),
                                   C.c_void_p(0))
    assert rc == d3.D3_ERR_SHAPE
    rc = L.d3_lm_head_stats_static(None, None, C.c_int32(0), C.c_int32(1), C.c_int32(1), C.c_int32(1), C.c_float(1.0),
                                   C.c_int32(0), None, None, None, C.c_void_p(0))
    assert rc == d3.D3_ERR_INVALID_ARG
    with pytest.raises(d3.D3Error):
        d3.d3_lm_head_stats_static(torch.zeros((m, 8), device=DEV), torch.zeros((256, 8), device=DEV), 1.0, 0,
                                   torch.zeros(m, device=DEV), torch.zeros(m, device=DEV),
                                   torch.zeros(m, dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()


def test_static_stats_binding_refuses_tensors_that_do_not_fit_together():
    """The C ABI sees pointers only, so the binding is where mismatched sizes are caught: one case per
    check, none of which reaches the library."""
    x = torch.zeros((8, 16), device=DEV)
    w = torch.zeros((64, 16), device=DEV)
    f = lambda n: torch.zeros(n, device=DEV)
    i = lambda n: torch.zeros(n, dtype=torch.int32, device=DEV)
    bad = [
        (x.reshape(-1), w, f(8), f(8), i(8)),          # x not 2-D
        (x, w.reshape(4, 16, 16), f(8), f(8), i(8)),   # w not 2-D
        (x, torch.zeros((64, 8), device=DEV), f(8), f(8), i(8)),  # inner sizes differ
        (x, w, f(7), f(8), i(8)),                      # conf too short
        (x, w, f(8), f(7), i(8)),                      # entropy too short
        (x, w, f(8), f(8), i(7)),                      # argmax too short
    ]
    for args in bad:
        with pytest.raises(ValueError):
            d3.d3_lm_head_stats_static(args[0], args[1], 1.0, 0, *args[2:])
    d3.d3_lm_head_stats_static(x, w, 1.0, 0, f(8), f(8), i(8))  # the well-formed call goes through
    torch.cuda.synchronize()
