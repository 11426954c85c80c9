"""Seeded synthetic inputs: model shapes, random-init weights and random prompts.

This module serves both the CUDA path and the CPU oracle's tests.  It holds
none of the decoding method's arithmetic: it only draws i.i.d. numbers and
lays them out.  It imports neither the CUDA binding nor the oracle.

Recipe
------
* Every weight matrix is i.i.d. N(0, 0.02^2).  A tensor is drawn in flat
  chunks of ``CHUNK`` elements; chunk ``c`` of tensor ``tid`` uses numpy's
  Philox bit generator keyed by ``(seed << 32 | tid, c)``, so any tensor (or
  any chunk of it) can be regenerated on its own and in parallel.
* fp32 models keep the fp32 draw; bf16 models keep its round-to-nearest-even
  bf16 bit pattern in a ``uint16`` array.
* Norm gains are 1 (not drawn).
* Prompts are uniform ids in ``[0, vocab-2)``, i.e. never ``pad_id`` (V-2) nor
  ``mask_id`` (V-1); ragged batches are right-padded with ``pad_id``.

The workloads stand in for the paper's evaluation setting (generation length
256, block size 32, batch 1 or 4, prompts from a few hundred to ~1000 tokens;
Appendix "More Implementation Details" and the SGLang table); no benchmark
item is reproduced anywhere.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Iterable, List, Optional, Tuple

import numpy as np

CHUNK = 1 << 22  # elements per independently keyed chunk
WEIGHT_STD = 0.02

# tensor ids inside one model
TID_TOK_EMB = 0
TID_LM_HEAD = 1
_LAYER_BASE = 16
_LAYER_STRIDE = 8
LAYER_TENSORS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


@dataclasses.dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    d_head: int
    d_ffn: int
    vocab: int
    dtype: str  # "fp32" or "bf16"
    rope_theta: float = 1.0e4
    rms_eps: float = 1.0e-5
    logit_scale: float = 20.0
    weight_seed: int = 0

    @property
    def mask_id(self) -> int:
        return self.vocab - 1

    @property
    def pad_id(self) -> int:
        return self.vocab - 2

    def tensor_shape(self, name: str) -> Tuple[int, int]:
        d, f = self.d_model, self.d_ffn
        qd, kd = self.n_q_heads * self.d_head, self.n_kv_heads * self.d_head
        return {
            "tok_emb": (self.vocab, d),
            "lm_head": (self.vocab, d),
            "wq": (qd, d),
            "wk": (kd, d),
            "wv": (kd, d),
            "wo": (d, qd),
            "w_gate": (f, d),
            "w_up": (f, d),
            "w_down": (d, f),
        }[name]

    def params_per_layer(self) -> int:
        return sum(int(np.prod(self.tensor_shape(n))) for n in LAYER_TENSORS)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    model: ModelShape
    batch: int
    prompt_min: int
    prompt_max: int
    gen_len: int
    block: int
    threshold: float
    prompt_seed: int
    length_seed: int = 0

    @property
    def max_seq(self) -> int:
        return self.prompt_max + self.gen_len


TINY = ModelShape("tiny-fp32", 2, 128, 4, 4, 32, 512, 512, "fp32")
LLADA8B = ModelShape("llada8b-shaped-bf16", 32, 4096, 32, 32, 128, 12288, 126464, "bf16")
QWEN7B = ModelShape("qwen2.5-7b-shaped-bf16", 28, 3584, 28, 4, 128, 18944, 152064, "bf16")

WORKLOADS: Dict[str, Workload] = {
    "c1": Workload("c1", TINY, 1, 32, 32, 64, 16, 0.9, 1001),
    "c2": Workload("c2", LLADA8B, 1, 256, 256, 256, 32, 0.9, 1002),
    "c3": Workload("c3", LLADA8B, 32, 128, 512, 256, 32, 0.9, 1003, 2003),
    "c4": Workload("c4", QWEN7B, 8, 512, 512, 512, 32, 0.9, 1004),
    "c5": Workload("c5", LLADA8B, 4, 4096, 4096, 1024, 64, 0.8, 1005),
}


def scaled_shape(base: ModelShape, *, name: str, n_layers: int, d_model: int, n_q_heads: int,
                 n_kv_heads: int, d_ffn: int, vocab: int, d_head: Optional[int] = None,
                 dtype: Optional[str] = None) -> ModelShape:
    """A smaller model of the same family (same dtype, RoPE, eps, scale) for parity cases."""
    return dataclasses.replace(base, name=name, n_layers=n_layers, d_model=d_model,
                               n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                               d_head=d_head or base.d_head, d_ffn=d_ffn, vocab=vocab,
                               dtype=dtype or base.dtype)


# ----------------------------------------------------------------------------- bf16 bit patterns
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even bf16 bit pattern (uint16) of an fp32 array (no NaN inputs expected)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------- weights
def tensor_id(name: str, layer: Optional[int] = None) -> int:
    if name == "tok_emb":
        return TID_TOK_EMB
    if name == "lm_head":
        return TID_LM_HEAD
    return _LAYER_BASE + _LAYER_STRIDE * int(layer) + LAYER_TENSORS.index(name)


def _draw_chunk(seed: int, tid: int, c: int, n: int, as_bf16: bool) -> np.ndarray:
    g = np.random.Generator(np.random.Philox(key=[(int(seed) << 32) | int(tid), int(c)]))
    x = g.standard_normal(n, dtype=np.float32)
    x *= np.float32(WEIGHT_STD)
    return f32_to_bf16_bits(x) if as_bf16 else x


def _threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def gen_tensor(shape: ModelShape, name: str, layer: Optional[int] = None,
               rows: Optional[Tuple[int, int]] = None, pool: Optional[ThreadPoolExecutor] = None
               ) -> np.ndarray:
    """One weight matrix ``[out, in]`` (fp32, or bf16 bits as uint16).

    ``rows=(r0, r1)`` returns only that row range (still chunk-exact)."""
    n_out, n_in = shape.tensor_shape(name)
    tid = tensor_id(name, layer)
    as_bf16 = shape.dtype == "bf16"
    r0, r1 = (0, n_out) if rows is None else rows
    lo, hi = r0 * n_in, r1 * n_in
    c0, c1 = lo // CHUNK, (hi + CHUNK - 1) // CHUNK
    total = n_out * n_in
    out = np.empty(hi - lo, dtype=np.uint16 if as_bf16 else np.float32)

    def work(c: int) -> None:
        beg, end = c * CHUNK, min((c + 1) * CHUNK, total)
        buf = _draw_chunk(shape.weight_seed, tid, c, end - beg, as_bf16)
        a, b = max(beg, lo), min(end, hi)
        out[a - lo:b - lo] = buf[a - beg:b - beg]

    cs = range(c0, c1)
    if pool is not None and len(cs) > 1:
        list(pool.map(work, cs))
    else:
        for c in cs:
            work(c)
    return out.reshape(r1 - r0, n_in)


def gen_layer(shape: ModelShape, layer: int, pool: Optional[ThreadPoolExecutor] = None
              ) -> Dict[str, np.ndarray]:
    return {n: gen_tensor(shape, n, layer, pool=pool) for n in LAYER_TENSORS}


def gen_weights(shape: ModelShape, layers: Optional[Iterable[int]] = None, with_embed: bool = True,
                with_head: bool = True) -> Dict[str, object]:
    """All (or selected) tensors: {"tok_emb", "lm_head", "layers": {l: {...}}}."""
    sel: List[int] = list(range(shape.n_layers)) if layers is None else list(layers)
    out: Dict[str, object] = {"layers": {}}
    with ThreadPoolExecutor(_threads()) as pool:
        if with_embed:
            out["tok_emb"] = gen_tensor(shape, "tok_emb", pool=pool)
        if with_head:
            out["lm_head"] = gen_tensor(shape, "lm_head", pool=pool)
        for l in sel:
            out["layers"][l] = gen_layer(shape, l, pool=pool)
    return out


# ----------------------------------------------------------------------------- prompts
def gen_prompts(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    """Right-padded prompt ids ``[batch, prompt_max]`` int32 and lengths ``[batch]`` int32."""
    shape = w.model
    if w.prompt_min == w.prompt_max:
        lens = np.full(w.batch, w.prompt_max, dtype=np.int32)
    else:
        gl = np.random.Generator(np.random.Philox(key=[w.length_seed, 0]))
        lens = gl.integers(w.prompt_min, w.prompt_max + 1, size=w.batch).astype(np.int32)
    gi = np.random.Generator(np.random.Philox(key=[w.prompt_seed, 0]))
    ids = gi.integers(0, shape.vocab - 2, size=(w.batch, w.prompt_max)).astype(np.int32)
    for b in range(w.batch):
        ids[b, lens[b]:] = shape.pad_id
    return ids, lens


def small_workload(name: str, model: ModelShape, batch: int, prompt_lens: Iterable[int], gen_len: int,
                   block: int, threshold: float, prompt_seed: int) -> Tuple[Workload, np.ndarray, np.ndarray]:
    """A parity-sized workload with explicit (possibly ragged) prompt lengths."""
    lens = np.asarray(list(prompt_lens), dtype=np.int32)
    assert lens.shape == (batch,)
    pmax = int(lens.max()) if batch else 0
    w = Workload(name, model, batch, int(lens.min()) if batch else 0, pmax, gen_len, block, threshold,
                 prompt_seed)
    gi = np.random.Generator(np.random.Philox(key=[prompt_seed, 0]))
    ids = gi.integers(0, model.vocab - 2, size=(batch, max(pmax, 1))).astype(np.int32)[:, :pmax]
    for b in range(batch):
        ids[b, lens[b]:] = model.pad_id
    return w, np.ascontiguousarray(ids), lens
