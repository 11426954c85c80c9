"""ctypes binding of libd3.so: argument marshalling only.

Every function here has the name of the C entry point it calls (see include/d3.h) and does nothing
but turn torch tensors into raw pointers and check the returned status.  All arithmetic of the
decoding path runs in the CUDA kernels of the library; there is no CPU fallback: if the library
cannot be loaded, or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libd3.so")

D3_OK = 0
D3_ERR_INVALID_ARG, D3_ERR_SHAPE, D3_ERR_OOM, D3_ERR_CUDA = -1, -2, -3, -4
D3_ERR_DEVICE_TIMEOUT, D3_ERR_STATE, D3_ERR_UNSUPPORTED = -5, -6, -7
D3_DTYPE_F32, D3_DTYPE_BF16 = 0, 1
D3_DECIDE_CONFIDENCE, D3_DECIDE_ENTROPY = 0, 1
D3_GEMM_AUTO, D3_GEMM_SIMT = 0, 1

EXPORTS = [
    "d3_create", "d3_destroy", "d3_load_weights", "d3_prefill", "d3_denoise_step", "d3_commit_block",
    "d3_generate", "d3_get_step_stats", "d3_forward_logits", "d3_set_tap", "d3_read_tap", "d3_read_kv",
    "d3_get_state", "d3_set_state", "d3_op_linear", "d3_packed_weight_elems", "d3_pack_weight", "d3_op_linear_packed", "d3_op_lm_head_stats", "d3_op_attention",
    "d3_op_write_kv", "d3_op_unmask", "d3_lm_head_stats_static", "d3_set_overlap", "d3_profile_enable", "d3_profile_read", "d3_get_error_word", "d3_launch_count", "d3_launch_count_of", "d3_set_eos", "d3_early_stops", "d3_generate_multiblock", "d3_refresh_cache", "d3_set_cache_policy", "d3_refresh_count", "d3_trajectory_rank", "d3_noisy_sequence", "d3_set_sampling", "d3_device_bytes",
    "d3_denoise_window", "d3_commit_histogram",
    "d3_strerror", "d3_last_error", "d3_version",
]
# measurement and test switches (include/d3_debug.h)
DEBUG_EXPORTS = ["d3_tuning_defaults", "d3_set_tuning", "d3_set_fused_finalize", "d3_debug_stall_probe",
                 "d3_clear_error_word", "d3_status_of_error_word"]


class d3_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "d_head", "d_ffn",
                                          "vocab", "mask_id")] + \
               [(n, C.c_float) for n in ("rope_theta", "rms_eps", "logit_scale")] + \
               [(n, C.c_int32) for n in ("dtype", "block", "max_batch", "max_seq", "max_prefill_rows",
                                          "decide_mode", "gemm_impl")]


class d3_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tok_emb", "lm_head", "final_norm")] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate",
                                                     "w_up", "w_down")]


class d3_stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("denoise_forwards", "finalize_forwards", "tokens_committed",
                                          "forced_commits", "steps", "kernel_launches")] + \
               [("prefill_ms", C.c_float), ("decode_ms", C.c_float)]


class D3Error(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"d3 error {code}: {msg}")
        self.code = code


_lib = None


def lib() -> C.CDLL:
    """Load libd3.so (built in-tree by build.py).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2601_07568_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        L.d3_strerror.restype = C.c_char_p
        L.d3_last_error.restype = C.c_char_p
        L.d3_last_error.argtypes = [C.c_void_p]
        L.d3_version.restype = C.c_char_p
        L.d3_launch_count.restype = C.c_int64
        L.d3_launch_count.argtypes = [C.c_void_p]
        L.d3_launch_count_of.restype = C.c_int64
        L.d3_launch_count_of.argtypes = [C.c_void_p, C.c_char_p]
        L.d3_early_stops.restype = C.c_int64
        L.d3_early_stops.argtypes = [C.c_void_p]
        L.d3_refresh_count.restype = C.c_int64
        L.d3_refresh_count.argtypes = [C.c_void_p]
        L.d3_device_bytes.restype = C.c_int64
        L.d3_device_bytes.argtypes = [C.c_void_p]
        L.d3_destroy.restype = None
        L.d3_destroy.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return C.c_void_p(t.data_ptr())


def _dev(t: torch.Tensor, dtype=None) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t


def _check(ctx, rc: int) -> None:
    if rc != D3_OK:
        L = lib()
        detail = L.d3_last_error(ctx).decode() if ctx else ""
        raise D3Error(rc, f"{L.d3_strerror(rc).decode()}: {detail}")


# ----------------------------------------------------------------------------- C entry points
def d3_create(cfg: d3_config, stream: Optional[torch.cuda.Stream] = None) -> C.c_void_p:
    if not torch.cuda.is_available():
        raise RuntimeError("d3 needs a CUDA device (no CPU fallback)")
    ctx = C.c_void_p(0)
    s = C.c_void_p(stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream)
    rc = lib().d3_create(C.byref(cfg), s, C.byref(ctx))
    if rc != D3_OK:
        raise D3Error(rc, lib().d3_strerror(rc).decode())
    return ctx


def d3_destroy(ctx) -> None:
    lib().d3_destroy(ctx)


def d3_load_weights(ctx, tensors: Dict[str, object], n_layers: int) -> None:
    """tensors: {"tok_emb", "lm_head", optional "final_norm", "layers": [ {wq, wk, wv, wo, w_gate, w_up,
    w_down, optional attn_norm, ffn_norm} ]}; all on the host or all on the device."""
    first = tensors["tok_emb"]
    on_dev = bool(first.is_cuda)
    keep = []

    def p(t):
        if t is None:
            return None
        if bool(t.is_cuda) != on_dev:
            raise ValueError("all weights must live on the same side (host or device)")
        t = t.contiguous()
        keep.append(t)
        return t.data_ptr()

    w = d3_weights()
    w.tok_emb, w.lm_head, w.final_norm = p(tensors["tok_emb"]), p(tensors["lm_head"]), p(tensors.get("final_norm"))
    layers = tensors["layers"]
    arrays = {}
    for name in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down"):
        arr = (C.c_void_p * n_layers)()
        for l in range(n_layers):
            arr[l] = p(layers[l].get(name))
        arrays[name] = arr
        setattr(w, name, C.cast(arr, C.POINTER(C.c_void_p)))
    _check(ctx, lib().d3_load_weights(ctx, C.byref(w), C.c_int(1 if on_dev else 0)))


def d3_prefill(ctx, prompt_ids: torch.Tensor, prompt_lens: torch.Tensor) -> None:
    bs, p_max = prompt_ids.shape
    _check(ctx, lib().d3_prefill(ctx, _ptr(_dev(prompt_ids, torch.int32)), _ptr(_dev(prompt_lens, torch.int32)),
                                 C.c_int32(bs), C.c_int32(p_max)))


def d3_denoise_step(ctx, block_ids: torch.Tensor, mask: torch.Tensor, threshold: float, out_pos: torch.Tensor,
                    out_ids: torch.Tensor, out_count: torch.Tensor) -> None:
    bs = block_ids.shape[0]
    _check(ctx, lib().d3_denoise_step(ctx, _ptr(_dev(block_ids, torch.int32)), _ptr(_dev(mask, torch.uint8)),
                                      C.c_float(threshold), C.c_int32(bs), _ptr(_dev(out_pos, torch.int32)),
                                      _ptr(_dev(out_ids, torch.int32)), _ptr(_dev(out_count, torch.int32))))


def d3_commit_block(ctx, block_ids: torch.Tensor) -> None:
    _check(ctx, lib().d3_commit_block(ctx, _ptr(_dev(block_ids, torch.int32)), C.c_int32(block_ids.shape[0])))


def d3_generate(ctx, gen_len: int, threshold: float, out_ids: torch.Tensor,
                commit_step: Optional[torch.Tensor] = None) -> d3_stats:
    st = d3_stats()
    bs = out_ids.shape[0]
    _check(ctx, lib().d3_generate(ctx, C.c_int32(gen_len), C.c_float(threshold), C.c_int32(bs),
                                  _ptr(_dev(out_ids, torch.int32)),
                                  _ptr(_dev(commit_step, torch.int32)) if commit_step is not None else C.c_void_p(0),
                                  C.byref(st)))
    return st


def d3_generate_multiblock(ctx, gen_len: int, threshold: float, out_ids: torch.Tensor, max_active: int,
                           commit_round: Optional[torch.Tensor] = None) -> d3_stats:
    st = d3_stats()
    bs = out_ids.shape[0]
    _check(ctx, lib().d3_generate_multiblock(ctx, C.c_int32(gen_len), C.c_float(threshold), C.c_int32(bs),
                                             C.c_int32(max_active), _ptr(_dev(out_ids, torch.int32)),
                                             _ptr(_dev(commit_round, torch.int32)) if commit_round is not None else C.c_void_p(0),
                                             C.byref(st)))
    return st


def d3_get_step_stats(ctx, conf: torch.Tensor, entropy: torch.Tensor, argmax: torch.Tensor, bs: int) -> None:
    _check(ctx, lib().d3_get_step_stats(ctx, _ptr(_dev(conf, torch.float32)), _ptr(_dev(entropy, torch.float32)),
                                        _ptr(_dev(argmax, torch.int32)), C.c_int32(bs)))


def d3_forward_logits(ctx, block_ids: torch.Tensor, logits: torch.Tensor) -> None:
    _check(ctx, lib().d3_forward_logits(ctx, _ptr(_dev(block_ids, torch.int32)), C.c_int32(block_ids.shape[0]),
                                        _ptr(_dev(logits, torch.float32))))


def d3_denoise_window(ctx, window_ids: torch.Tensor, n_win: int, conf: torch.Tensor, entropy: torch.Tensor,
                      argmax: torch.Tensor) -> None:
    bs = window_ids.shape[0]
    _check(ctx, lib().d3_denoise_window(ctx, _ptr(_dev(window_ids, torch.int32)), C.c_int32(bs), C.c_int32(n_win),
                                        _ptr(_dev(conf, torch.float32)), _ptr(_dev(entropy, torch.float32)),
                                        _ptr(_dev(argmax, torch.int32))))


def d3_commit_histogram(ctx, n: int):
    """hist[k] = decisions of the latest generate call that committed exactly k tokens, k < n."""
    h = (C.c_int64 * n)()
    _check(ctx, lib().d3_commit_histogram(ctx, h, C.c_int32(n)))
    return [int(v) for v in h]


def d3_set_tap(ctx, layer: int) -> None:
    _check(ctx, lib().d3_set_tap(ctx, C.c_int32(layer)))


def d3_read_tap(ctx, resid_in: torch.Tensor, resid_out: torch.Tensor, rows: int) -> None:
    _check(ctx, lib().d3_read_tap(ctx, _ptr(_dev(resid_in, torch.float32)), _ptr(_dev(resid_out, torch.float32)),
                                  C.c_int32(rows)))


def d3_read_kv(ctx, layer: int, seq: int, pos0: int, n: int, k_out: torch.Tensor, v_out: torch.Tensor) -> None:
    _check(ctx, lib().d3_read_kv(ctx, C.c_int32(layer), C.c_int32(seq), C.c_int32(pos0), C.c_int32(n),
                                 _ptr(_dev(k_out, torch.float32)), _ptr(_dev(v_out, torch.float32))))


def d3_get_state(ctx, prefix_len: torch.Tensor) -> None:
    _check(ctx, lib().d3_get_state(ctx, _ptr(_dev(prefix_len, torch.int32)), C.c_int32(prefix_len.numel())))


def d3_set_state(ctx, prefix_len: torch.Tensor) -> None:
    _check(ctx, lib().d3_set_state(ctx, _ptr(_dev(prefix_len, torch.int32)), C.c_int32(prefix_len.numel())))


def d3_op_linear(ctx, x: torch.Tensor, w: torch.Tensor, y: torch.Tensor, epilogue: int, splits: int = 0) -> None:
    m, k = x.shape
    n = w.shape[0]
    _check(ctx, lib().d3_op_linear(ctx, _ptr(_dev(x)), _ptr(_dev(w)), _ptr(_dev(y)), C.c_int32(m), C.c_int32(n),
                                   C.c_int32(k), C.c_int32(epilogue), C.c_int32(splits)))


def d3_packed_weight_elems(n: int, k: int) -> int:
    f = lib().d3_packed_weight_elems
    f.restype = C.c_int64
    return int(f(C.c_int32(n), C.c_int32(k)))


def d3_pack_weight(ctx, w: torch.Tensor, packed: torch.Tensor) -> None:
    n, k = w.shape
    if packed.numel() < d3_packed_weight_elems(n, k):
        raise ValueError("packed buffer too small")
    _check(ctx, lib().d3_pack_weight(ctx, _ptr(_dev(w, torch.bfloat16)), C.c_int32(n), C.c_int32(k),
                                     _ptr(_dev(packed, torch.bfloat16))))


def d3_op_linear_packed(ctx, x: torch.Tensor, w_packed: torch.Tensor, y: torch.Tensor, n: int, epilogue: int,
                        splits: int = 0) -> None:
    m, k = x.shape
    _check(ctx, lib().d3_op_linear_packed(ctx, _ptr(_dev(x)), _ptr(_dev(w_packed)), _ptr(_dev(y)), C.c_int32(m),
                                          C.c_int32(n), C.c_int32(k), C.c_int32(epilogue), C.c_int32(splits)))


def _check_head_shapes(x, w, conf, entropy, argmax) -> None:
    """The C ABI sees pointers only: sizes that would make a kernel read or write past a tensor are
    refused here."""
    if x.dim() != 2 or w.dim() != 2:
        raise ValueError("x and w must be 2-D")
    if w.shape[1] != x.shape[1]:
        raise ValueError(f"w has {w.shape[1]} columns, x has {x.shape[1]}")
    m = x.shape[0]
    for name, t in (("conf", conf), ("entropy", entropy), ("argmax", argmax)):
        if t.numel() < m:
            raise ValueError(f"{name} holds {t.numel()} elements, {m} rows need as many")


def d3_op_lm_head_stats(ctx, x: torch.Tensor, w: torch.Tensor, scale: float, mask_id: int, conf: torch.Tensor,
                        entropy: torch.Tensor, argmax: torch.Tensor) -> None:
    _dev(x), _dev(w, x.dtype)
    _check_head_shapes(x, w, conf, entropy, argmax)
    m, k = x.shape
    _check(ctx, lib().d3_op_lm_head_stats(ctx, _ptr(_dev(x)), _ptr(_dev(w)), C.c_int32(m), C.c_int32(w.shape[0]),
                                          C.c_int32(k), C.c_float(scale), C.c_int32(mask_id),
                                          _ptr(_dev(conf, torch.float32)), _ptr(_dev(entropy, torch.float32)),
                                          _ptr(_dev(argmax, torch.int32))))


def d3_op_attention(ctx, q: torch.Tensor, layer: int, bs: int, rows: int, kv_len: torch.Tensor,
                    out: torch.Tensor) -> None:
    _check(ctx, lib().d3_op_attention(ctx, _ptr(_dev(q)), C.c_int32(layer), C.c_int32(bs), C.c_int32(rows),
                                      _ptr(_dev(kv_len, torch.int32)), _ptr(_dev(out))))


def d3_op_write_kv(ctx, layer: int, seq: int, pos0: int, k: torch.Tensor, v: torch.Tensor) -> None:
    n = k.shape[1]
    _check(ctx, lib().d3_op_write_kv(ctx, C.c_int32(layer), C.c_int32(seq), C.c_int32(pos0), C.c_int32(n),
                                     _ptr(_dev(k, torch.float32)), _ptr(_dev(v, torch.float32))))


def d3_op_unmask(ctx, conf: torch.Tensor, entropy: torch.Tensor, argmax: torch.Tensor, block_ids: torch.Tensor,
                 mask: torch.Tensor, threshold: float, out_pos: torch.Tensor, out_ids: torch.Tensor,
                 out_count: torch.Tensor) -> None:
    _check(ctx, lib().d3_op_unmask(ctx, _ptr(_dev(conf, torch.float32)), _ptr(_dev(entropy, torch.float32)),
                                   _ptr(_dev(argmax, torch.int32)), _ptr(_dev(block_ids, torch.int32)),
                                   _ptr(_dev(mask, torch.uint8)), C.c_float(threshold),
                                   C.c_int32(block_ids.shape[0]), _ptr(_dev(out_pos, torch.int32)),
                                   _ptr(_dev(out_ids, torch.int32)), _ptr(_dev(out_count, torch.int32))))


D3_STATIC_MAX_PARTIALS = 65536


def d3_lm_head_stats_static(x: torch.Tensor, w: torch.Tensor, scale: float, mask_id: int, conf: torch.Tensor,
                            entropy: torch.Tensor, argmax: torch.Tensor,
                            stream: Optional[torch.cuda.Stream] = None) -> None:
    """Context-free LM-head statistics that allocate nothing on the device (for callers that may not
    allocate: frozen-allocator regions, fixed memory budgets, real-time loops).  x [m, k] and w [vocab, k]
    are float32 or bfloat16 CUDA tensors of the same type; the outputs are written on ``stream`` (default:
    torch's current stream).  Raises D3Error(D3_ERR_SHAPE) when m * ceil(vocab/128) exceeds
    D3_STATIC_MAX_PARTIALS.  Calls that may overlap on the GPU race on the shared scratch array."""
    _dev(x), _dev(w, x.dtype)
    if x.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("x and w must be float32 or bfloat16")
    _check_head_shapes(x, w, conf, entropy, argmax)
    m, k = x.shape
    s = C.c_void_p(stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream)
    rc = lib().d3_lm_head_stats_static(_ptr(x), _ptr(w), C.c_int32(D3_DTYPE_BF16 if x.dtype == torch.bfloat16 else D3_DTYPE_F32),
                                       C.c_int32(m), C.c_int32(w.shape[0]), C.c_int32(k), C.c_float(scale),
                                       C.c_int32(mask_id), _ptr(_dev(conf, torch.float32)),
                                       _ptr(_dev(entropy, torch.float32)), _ptr(_dev(argmax, torch.int32)), s)
    if rc != D3_OK:
        raise D3Error(rc, lib().d3_strerror(rc).decode())


PROF_CLASSES = ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_head", "gemm_other", "attention",
                "rmsnorm", "other", "chain")


def d3_set_overlap(ctx, on: bool) -> None:
    _check(ctx, lib().d3_set_overlap(ctx, C.c_int(1 if on else 0)))


class d3_tuning(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("ring_kb", "ctas_per_sm", "producers", "tile_columns", "attn_key_tiles",
                                          "cluster_k_split", "row_tile_pairs", "round_robin", "column_strips",
                                          "strip_stages", "chain", "chain_clusters", "chain_l2_ahead", "weights_as_rows", "attention_tmem", "cta_pairs")]


def d3_tuning_defaults() -> d3_tuning:
    t = d3_tuning()
    lib().d3_tuning_defaults(C.byref(t))
    return t


def d3_set_tuning(ctx, tuning: Optional[d3_tuning] = None, **fields) -> None:
    """Scheduling overrides (include/d3_debug.h).  ``tuning`` or the defaults, with ``fields`` set by name."""
    t = tuning if tuning is not None else d3_tuning_defaults()
    for k, v in fields.items():
        if not hasattr(t, k):
            raise ValueError(f"d3_tuning has no field {k}")
        setattr(t, k, v)
    _check(ctx, lib().d3_set_tuning(ctx, C.byref(t)))


def d3_set_fused_finalize(ctx, on: bool) -> None:
    _check(ctx, lib().d3_set_fused_finalize(ctx, C.c_int(1 if on else 0)))


def d3_debug_stall_probe(ctx, limit_us: int) -> int:
    """Returns the status code of the probe (D3_ERR_DEVICE_TIMEOUT is the expected outcome)."""
    return int(lib().d3_debug_stall_probe(ctx, C.c_int32(limit_us)))


def d3_clear_error_word(ctx) -> None:
    _check(ctx, lib().d3_clear_error_word(ctx))


def d3_status_of_error_word(word: int) -> int:
    return int(lib().d3_status_of_error_word(C.c_uint32(word)))


def d3_profile_enable(ctx, on: bool) -> None:
    _check(ctx, lib().d3_profile_enable(ctx, C.c_int(1 if on else 0)))


def d3_profile_read(ctx) -> Dict[str, Dict[str, float]]:
    n = len(PROF_CLASSES)
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    _check(ctx, lib().d3_profile_read(ctx, ms, cnt))
    return {name: {"ms": float(ms[i]), "launches": int(cnt[i])} for i, name in enumerate(PROF_CLASSES)}


def d3_get_error_word(ctx) -> int:
    w = C.c_uint32(0)
    _check(ctx, lib().d3_get_error_word(ctx, C.byref(w)))
    return int(w.value)


def d3_launch_count(ctx) -> int:
    return int(lib().d3_launch_count(ctx))


def d3_launch_count_of(ctx, kernel: str) -> int:
    return int(lib().d3_launch_count_of(ctx, kernel.encode()))


def d3_set_eos(ctx, eos_id: int) -> None:
    _check(ctx, lib().d3_set_eos(ctx, C.c_int32(eos_id)))


def d3_early_stops(ctx) -> int:
    return int(lib().d3_early_stops(ctx))


def d3_trajectory_rank(ctx, commit_step: torch.Tensor, rank: torch.Tensor) -> None:
    bs, gen_len = commit_step.shape
    _check(ctx, lib().d3_trajectory_rank(ctx, _ptr(_dev(commit_step, torch.int32)), C.c_int32(bs), C.c_int32(gen_len),
                                         _ptr(_dev(rank, torch.int32))))


def d3_noisy_sequence(ctx, y: torch.Tensor, rank: torch.Tensor, s: torch.Tensor, k: torch.Tensor, m: torch.Tensor,
                      out: torch.Tensor) -> None:
    bs, n = y.shape
    _check(ctx, lib().d3_noisy_sequence(ctx, _ptr(_dev(y, torch.int32)), _ptr(_dev(rank, torch.int32)),
                                        _ptr(_dev(s, torch.int32)), _ptr(_dev(k, torch.int32)), _ptr(_dev(m, torch.int32)),
                                        C.c_int32(bs), C.c_int32(n), _ptr(_dev(out, torch.int32))))


def d3_set_sampling(ctx, temperature: float = 0.0, seed: int = 0) -> None:
    _check(ctx, lib().d3_set_sampling(ctx, C.c_float(temperature), C.c_uint64(seed)))


def d3_refresh_cache(ctx, bs: int) -> None:
    _check(ctx, lib().d3_refresh_cache(ctx, C.c_int32(bs)))


def d3_set_cache_policy(ctx, cache_delay: int = 1, refresh_every: int = 0) -> None:
    _check(ctx, lib().d3_set_cache_policy(ctx, C.c_int32(cache_delay), C.c_int32(refresh_every)))


def d3_refresh_count(ctx) -> int:
    return int(lib().d3_refresh_count(ctx))


def d3_device_bytes(ctx) -> int:
    return int(lib().d3_device_bytes(ctx))


def d3_version() -> str:
    return lib().d3_version().decode()


def d3_strerror(code: int) -> str:
    return lib().d3_strerror(C.c_int(code)).decode()


def d3_last_error(ctx) -> str:
    return lib().d3_last_error(ctx).decode()


# ----------------------------------------------------------------------------- convenience
def make_config(shape, *, block: int, max_batch: int, max_seq: int, max_prefill_rows: int = 0,
                decide_mode: int = D3_DECIDE_CONFIDENCE, gemm_impl: int = D3_GEMM_AUTO) -> d3_config:
    """d3_config from any object with the usual model-shape attributes."""
    cfg = d3_config()
    cfg.n_layers, cfg.d_model = shape.n_layers, shape.d_model
    cfg.n_q_heads, cfg.n_kv_heads, cfg.d_head = shape.n_q_heads, shape.n_kv_heads, shape.d_head
    cfg.d_ffn, cfg.vocab, cfg.mask_id = shape.d_ffn, shape.vocab, shape.mask_id
    cfg.rope_theta, cfg.rms_eps, cfg.logit_scale = shape.rope_theta, shape.rms_eps, shape.logit_scale
    cfg.dtype = D3_DTYPE_BF16 if shape.dtype == "bf16" else D3_DTYPE_F32
    cfg.block, cfg.max_batch, cfg.max_seq = block, max_batch, max_seq
    cfg.max_prefill_rows = max_prefill_rows
    cfg.decide_mode, cfg.gemm_impl = decide_mode, gemm_impl
    return cfg


def weights_from_numpy(shape, weights: Dict[str, object], pin: bool = False) -> Dict[str, object]:
    """Wrap generator output (fp32 arrays or bf16 bit patterns) as host torch tensors, without copies."""
    import numpy as np

    def t(a):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
        return torch.from_numpy(a)

    out = {"tok_emb": t(weights["tok_emb"]), "lm_head": t(weights["lm_head"]),
           "layers": [{k: t(v) for k, v in weights["layers"][l].items()} for l in range(shape.n_layers)]}
    if weights.get("final_norm") is not None:
        out["final_norm"] = t(weights["final_norm"])
    return out
