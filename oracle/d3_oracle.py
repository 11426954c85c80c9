"""CPU oracle for threshold-based masked-block diffusion decoding.

TEST INFRASTRUCTURE ONLY.  Plain NumPy, written from the paper's description
of the decoding loop; it shares no code with the CUDA path and must never be
imported by the product package.  Only tests, the smoke check and the
benchmark's CPU-baseline leg use it.

What the paper fixes (cited per function) and what it leaves open
-----------------------------------------------------------------
* A diffusion LLM predicts every masked position of a block at once with a
  bidirectional (non-causal) transformer (Sec. 1; Appendix "Combined with
  SGLang", item (i)).
* Generation proceeds block by block with a fixed block size (Appendix "More
  Implementation Details", inference settings).
* Each forward pass is followed by a decision: tokens whose confidence clears
  a threshold are decoded in parallel (Sec. 2, the threshold paragraph), or,
  in the entropy variant, tokens whose predictive entropy is below the
  threshold, lower entropy first (Sec. 3.2, first paragraph).
* At least one token is decoded per forward pass regardless of the threshold
  (Sec. 3.2, the Fully-Activated state).
* A finished block's key/value states enter the cache only after a further
  forward pass over its final tokens (Sec. 3.2, "Completed but Stabilizing";
  KV-cache paragraph: a short delay before caching).
* Unmasking exactly one token per step is the teacher-trajectory mode
  (Sec. 3.1; Appendix, pseudo-trajectory extraction).
* Multi-block decoding (Sec. 3.2, "Entropy-Based Multi-Block Parallel
  Decoding"): the current and future blocks are decoded in one forward pass.  A
  new block is created (Activated) when its predecessor is 10 % complete and
  decodes only tokens that clear the threshold; when the predecessor is 95 %
  complete it is Fully-Activated and decodes at least one token per forward; a
  block whose tokens are all unmasked goes through one more forward
  (Completed but Stabilizing) before its key/value states are stored
  (Completed).  Readings taken here: blocks in flight see the cache, earlier
  blocks in flight and themselves, never later ones (the same block-causal
  visibility as everywhere else, so a stabilizing forward shared with other
  blocks equals one of its own); states are read from the masks as they stand
  before a forward; completion is compared in integers (100 u >= 10 B, 100 u >=
  95 B for u unmasked of B tokens); the number of blocks in flight is bounded
  by a parameter; blocks enter the cache in order, one stabilizing round each.
* Decoding halts as soon as the end-of-sequence token has been generated
  (Sec. 3.2, "Early Stopping on EOS Token"): the generated tokens are checked
  after every decoding step.  Reading taken here: the sequence stops after the
  step that commits the EOS id anywhere in the current block; positions that
  are still masked (in this block and all later ones) are returned as the
  mask id, and the unfinished block gets no finalize forward.
* KV-refresh (Sec. 3.2, "KV-Cache and KV-Refresh Mechanism"; abstract: all
  previously cached states are recomputed periodically) and the cache delay
  (Appendix, inference settings: 1-2 iterations).  Readings taken here: a
  refresh is one forward over the tokens of the stored prefix (prompt and
  stored blocks) in which every position sees every other one, and it
  replaces the stored K and V; blocks in flight take no part and the next
  forwards read the refreshed cache.  Block-by-block decoding refreshes each
  time the number of stored blocks reaches a multiple of the period while
  blocks remain; multi-block decoding refreshes after every period-th round
  while blocks are in flight.  The cache delay is the number of stabilizing
  rounds (forwards in which the block was already complete) before a block's
  K and V are stored.

* Pseudo-trajectory (Sec. 3.1): the teacher unmasks exactly one token per
  step and decodes past EOS to the full length; only the order is kept.  The
  noisy sequence keeps y_i up to the window start s and wherever trajectory
  state T_{s+ceil(kt)} is unmasked, and masks everything after the window
  and wherever that state is masked.  Readings: the extraction run is
  ``generate`` at threshold 1 (no probability exceeds 1, so every step commits
  only the forced, most confident token) without EOS stop; in the overlap of
  the equation's cases i <= s wins, then i > s+k, then the trajectory; the
  tokens y must not contain the mask id.

* Temperature (Appendix, inference settings: 0.0 or 0.1).  Readings: at
  temperature T > 0 a row's token is drawn from softmax(l / T) by the
  Gumbel-max rule, arg max_v (l_v + T g_v) compared in float32, with the mask
  token excluded; the confidence that meets the threshold is softmax(l) of the
  drawn token and the entropy is that of softmax(l); the noise comes from
  Philox-4x32-10 keyed by the seed with counter (v // 4, absolute position,
  step within the block, sequence index), uniform = top 23 bits centred in
  their bucket, g = -ln(-ln u) in float32.

Readings taken where the paper is silent are listed in the repository's
design notes; in short: block-causal visibility between segments (prompt =
segment 0, generation block j = segment j), which makes the prefix cache
exact; confidence = softmax probability of the arg-max token with the mask
token excluded; strict comparisons (conf > tau, entropy < tau, nats); forced
commit = most confident masked position, lowest index on ties; one finalize
forward per block; rotate-half RoPE; RMSNorm with eps inside the root.

Parity status: the decoding loop, decision rule, cache and every layer
primitive are pinned by tests/test_oracle_*.py (closed forms, library
routines, brute force).  The numeric values of the logits for the synthetic
configurations are "parity unpinned" by the paper, which prints no per-step
values; they are pinned only through those invariants and an independent
torch-CPU forward.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

MODE_CONFIDENCE = 0  # commit if max-prob > tau
MODE_ENTROPY = 1     # commit if entropy (nats) < tau


# ----------------------------------------------------------------------------- number formats
def bf16_bits_to_float(bits: np.ndarray, dtype=np.float32) -> np.ndarray:
    """uint16 bf16 bit patterns -> floating point (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(dtype, copy=False)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bf16 value (ties to even), result in x's dtype."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(x.dtype, copy=False)


# ----------------------------------------------------------------------------- layer primitives
def rms_norm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope_tables(positions: np.ndarray, d_head: int, theta: float) -> Tuple[np.ndarray, np.ndarray]:
    """cos/sin of position * theta^(-2k/d_head), k = 0..d_head/2-1, in float64: [n, d_head/2]."""
    k = np.arange(d_head // 2, dtype=np.float64)
    inv_freq = np.power(np.float64(theta), -2.0 * k / d_head)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang), np.sin(ang)


def apply_rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotate-half RoPE.  x: [n, heads, d_head]; pairs are (k, k + d_head/2)."""
    half = x.shape[-1] // 2
    x1, x2 = x[..., :half], x[..., half:]
    c, s = cos[:, None, :].astype(x.dtype), sin[:, None, :].astype(x.dtype)
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def softmax_rows(s: np.ndarray) -> np.ndarray:
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray,
              visible: Optional[np.ndarray] = None, round_probs_bf16: bool = False) -> np.ndarray:
    """softmax(q k^T / sqrt(d_head)) v per head, no causal mask.

    q: [n, hq, dh]; k, v: [L, hkv, dh]; query head h reads kv head h // (hq/hkv).
    visible: optional bool [n, L]; False entries get probability 0."""
    n, hq, dh = q.shape
    hkv = k.shape[1]
    group = hq // hkv
    out = np.empty_like(q)
    scale = 1.0 / np.sqrt(np.float64(dh))
    for h in range(hq):
        g = h // group
        s = (q[:, h, :] @ k[:, g, :].T) * q.dtype.type(scale)
        if visible is not None:
            s = np.where(visible, s, -np.inf)
        p = softmax_rows(s)
        if round_probs_bf16:
            p = round_to_bf16(p)
        out[:, h, :] = p @ v[:, g, :]
    return out


def softmax_stats(logits: np.ndarray, mask_id: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Per row: probabilities with the mask token excluded, confidence = max prob,
    token = arg max (lowest index on ties), entropy in nats.  Computed in float64."""
    l = np.array(logits, dtype=np.float64, copy=True)
    l[:, mask_id] = -np.inf
    p = softmax_rows(l)
    tok = np.argmax(l, axis=-1).astype(np.int32)  # first occurrence = lowest index
    conf = p[np.arange(p.shape[0]), tok]
    with np.errstate(divide="ignore", invalid="ignore"):
        plogp = np.where(p > 0.0, p * np.log(p), 0.0)
    ent = -np.sum(plogp, axis=-1)
    return p, conf, tok, ent


# ----------------------------------------------------------------------------- sampling noise
def philox4x32_10(counter: np.ndarray, key: Tuple[int, int]) -> np.ndarray:
    """Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
    1, 2, 3", SC'11): counter [..., 4] uint32, key two 32-bit words; returns [..., 4] uint32.
    One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 as 64-bit products;
    c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); the key is bumped by the Weyl constants
    between rounds."""
    M0, M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
    W0, W1 = 0x9E3779B9, 0xBB67AE85
    c = np.asarray(counter, dtype=np.uint64) & np.uint64(0xFFFFFFFF)
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    lo32, sh = np.uint64(0xFFFFFFFF), np.uint64(32)
    for r in range(10):
        p0, p1 = M0 * c0, M1 * c2
        hi0, lo0, hi1, lo1 = p0 >> sh, p0 & lo32, p1 >> sh, p1 & lo32
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
        k0, k1 = (k0 + W0) & 0xFFFFFFFF, (k1 + W1) & 0xFFFFFFFF
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def uniform_from_bits(x: np.ndarray) -> np.ndarray:
    """float32 in (0, 1) from a 32-bit word: the top 23 bits, centred in their bucket (k + 1/2 with
    k < 2^23 is exact in float32, so neither end point is reached)."""
    return ((np.asarray(x, dtype=np.uint32) >> np.uint32(9)).astype(np.float32) + np.float32(0.5)) * np.float32(2.0 ** -23)


def gumbel_noise(seed: int, seq: int, positions: np.ndarray, step: int, vocab: int) -> np.ndarray:
    """Standard Gumbel noise g = -ln(-ln u) (float32) for every (row, vocabulary index): one
    Philox call per four consecutive vocabulary indices with counter (v // 4, absolute position of
    the row, decoding step within the block, sequence index) and key = the two halves of the
    seed; index v takes output word v % 4."""
    positions = np.asarray(positions, dtype=np.uint32)
    nq = (vocab + 3) // 4
    ctr = np.zeros((len(positions), nq, 4), dtype=np.uint32)
    ctr[..., 0] = np.arange(nq, dtype=np.uint32)[None, :]
    ctr[..., 1] = positions[:, None]
    ctr[..., 2] = np.uint32(step)
    ctr[..., 3] = np.uint32(seq)
    bits = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)).reshape(len(positions), nq * 4)[:, :vocab]
    u = uniform_from_bits(bits)
    return -np.log(-np.log(u))  # float32 throughout


def sample_stats(logits: np.ndarray, mask_id: int, temperature: float, noise: np.ndarray
                 ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Temperature sampling by the Gumbel-max rule (Appendix, inference settings: temperature 0
    or 0.1): the token of a row is arg max_v (l_v + T g_v), which is a draw from
    softmax(l / T); the mask token is excluded.  The comparison is made in float32 (the
    precision the logits exist in on the device).  Confidence is the model's probability of
    the drawn token, softmax(l)[token]; the entropy is that of softmax(l), as without
    sampling.  Returns (conf, tok, entropy)."""
    _, _, _, ent = softmax_stats(logits, mask_id)
    l = np.array(logits, dtype=np.float64, copy=True)
    l[:, mask_id] = -np.inf
    p = softmax_rows(l)
    pert = l.astype(np.float32) + np.float32(temperature) * np.asarray(noise, dtype=np.float32)
    pert[:, mask_id] = -np.inf
    tok = np.argmax(pert, axis=-1).astype(np.int32)
    conf = p[np.arange(p.shape[0]), tok]
    return conf, tok, ent


def decide(conf: np.ndarray, ent: np.ndarray, mask: np.ndarray, tau: float, mode: int = MODE_CONFIDENCE
           ) -> np.ndarray:
    """Which masked positions of one block are committed this step (bool [B]).

    Every masked position clearing the threshold, plus always the single most confident
    masked position (highest max-prob, or lowest entropy in entropy mode; lowest index on
    ties).  A block without masked positions commits nothing."""
    mask = np.asarray(mask, dtype=bool)
    commit = np.zeros(mask.shape, dtype=bool)
    if not mask.any():
        return commit
    if mode == MODE_CONFIDENCE:
        commit = mask & (conf > tau)
        score = np.where(mask, conf, -np.inf)
        forced = int(np.argmax(score))
    else:
        commit = mask & (ent < tau)
        score = np.where(mask, ent, np.inf)
        forced = int(np.argmin(score))
    commit[forced] = True
    return commit


# ----------------------------------------------------------------------------- model
@dataclass
class SeqState:
    """Per-sequence cache: post-RoPE K and V of the committed prefix, per layer [L, hkv, dh],
    and the token ids of that prefix (needed to recompute the cache, see ``refresh``)."""
    k: List[np.ndarray]
    v: List[np.ndarray]
    ids: np.ndarray = field(default_factory=lambda: np.zeros(0, dtype=np.int32))

    @property
    def prefix_len(self) -> int:
        return int(self.k[0].shape[0])

    def copy(self) -> "SeqState":
        return SeqState([a.copy() for a in self.k], [a.copy() for a in self.v], self.ids.copy())


class OracleModel:
    """Pre-norm transformer without causal mask: RMSNorm, RoPE attention (MHA/GQA), SwiGLU FFN,
    untied LM head, logits multiplied by ``logit_scale``.  No biases; norm gains default to 1.

    ``weights``: {"tok_emb": [V,d], "lm_head": [V,d], "layers": {l: {"wq","wk","wv","wo",
    "w_gate","w_up","w_down"}}}, each matrix [out, in], floating point or bf16 bits (uint16).
    ``dtype`` is the arithmetic type.  ``mirror_bf16`` additionally rounds activations to bf16
    where a bf16 pipeline stores them (normed input, q/k/v after RoPE, attention output, FFN
    hidden) so that rounding can be told from errors; the residual stream is never rounded.
    """

    def __init__(self, *, n_layers: int, d_model: int, n_q_heads: int, n_kv_heads: int, d_head: int,
                 d_ffn: int, vocab: int, mask_id: int, weights: Dict[str, object],
                 rope_theta: float = 1.0e4, rms_eps: float = 1.0e-5, logit_scale: float = 20.0,
                 dtype=np.float64, mirror_bf16: bool = False, gains: Optional[Dict[str, object]] = None):
        self.n_layers, self.d_model = n_layers, d_model
        self.n_q_heads, self.n_kv_heads, self.d_head = n_q_heads, n_kv_heads, d_head
        self.d_ffn, self.vocab, self.mask_id = d_ffn, vocab, mask_id
        self.rope_theta, self.rms_eps, self.logit_scale = rope_theta, rms_eps, logit_scale
        self.dtype = np.dtype(dtype)
        self.mirror = mirror_bf16
        self.w = weights
        self.gains = gains or {}

    # -- helpers
    def _mat(self, a: np.ndarray) -> np.ndarray:
        if a.dtype == np.uint16:
            return bf16_bits_to_float(a, self.dtype)
        return a.astype(self.dtype, copy=False)

    def _gain(self, name: str, layer: Optional[int] = None) -> np.ndarray:
        g = self.gains.get((name, layer)) if layer is not None else self.gains.get(name)
        if g is None:
            return np.ones(self.d_model, dtype=self.dtype)
        return np.asarray(g, dtype=self.dtype)

    def _r(self, x: np.ndarray) -> np.ndarray:
        return round_to_bf16(x) if self.mirror else x

    def embed(self, ids: np.ndarray) -> np.ndarray:
        return self._mat(np.asarray(self.w["tok_emb"])[np.asarray(ids, dtype=np.int64)])

    # -- one layer
    def layer_forward(self, layer: int, x: np.ndarray, positions: np.ndarray,
                      k_prefix: Optional[np.ndarray], v_prefix: Optional[np.ndarray],
                      visible: Optional[np.ndarray] = None
                      ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """x: [n, d] rows at absolute ``positions``; keys/values = prefix cache followed by
        these rows' own K/V.  Returns (x_out, k_rows, v_rows) with k_rows post-RoPE."""
        W = self.w["layers"][layer]
        n = x.shape[0]
        hq, hkv, dh = self.n_q_heads, self.n_kv_heads, self.d_head
        xn = self._r(rms_norm(x, self._gain("attn_norm", layer), self.rms_eps))
        q = (xn @ self._mat(W["wq"]).T).reshape(n, hq, dh)
        k = (xn @ self._mat(W["wk"]).T).reshape(n, hkv, dh)
        v = (xn @ self._mat(W["wv"]).T).reshape(n, hkv, dh)
        cos, sin = rope_tables(positions, dh, self.rope_theta)
        q = self._r(apply_rope(q, cos, sin))
        k = self._r(apply_rope(k, cos, sin))
        v = self._r(v)
        if k_prefix is not None and k_prefix.shape[0] > 0:
            k_all = np.concatenate([k_prefix.astype(self.dtype, copy=False), k], axis=0)
            v_all = np.concatenate([v_prefix.astype(self.dtype, copy=False), v], axis=0)
        else:
            k_all, v_all = k, v
        o = self._r(attention(q, k_all, v_all, visible, round_probs_bf16=False))
        x = x + o.reshape(n, hq * dh) @ self._mat(W["wo"]).T
        xn = self._r(rms_norm(x, self._gain("ffn_norm", layer), self.rms_eps))
        gate = xn @ self._mat(W["w_gate"]).T
        up = xn @ self._mat(W["w_up"]).T
        h = self._r(silu(gate) * up)
        x = x + h @ self._mat(W["w_down"]).T
        return x, k, v

    def forward_rows(self, ids: np.ndarray, positions: np.ndarray, state: Optional[SeqState],
                     visible: Optional[np.ndarray] = None
                     ) -> Tuple[np.ndarray, List[np.ndarray], List[np.ndarray]]:
        """All layers over the given rows against ``state``'s cache.  Returns the residual
        stream after the last layer and the rows' per-layer K/V."""
        x = self.embed(ids)
        ks, vs = [], []
        for l in range(self.n_layers):
            kp = state.k[l] if state is not None else None
            vp = state.v[l] if state is not None else None
            x, k, v = self.layer_forward(l, x, positions, kp, vp, visible)
            ks.append(k)
            vs.append(v)
        return x, ks, vs

    def logits(self, x: np.ndarray) -> np.ndarray:
        xn = self._r(rms_norm(x, self._gain("final_norm"), self.rms_eps))
        return (xn @ self._mat(np.asarray(self.w["lm_head"])).T) * self.dtype.type(self.logit_scale)

    # -- decoding path
    def empty_state(self) -> SeqState:
        z = lambda: np.zeros((0, self.n_kv_heads, self.d_head), dtype=self.dtype)
        return SeqState([z() for _ in range(self.n_layers)], [z() for _ in range(self.n_layers)])

    def prefill(self, prompt: np.ndarray) -> SeqState:
        """Forward over the prompt alone (bidirectional within it); keep post-RoPE K and V."""
        prompt = np.asarray(prompt)
        if prompt.shape[0] == 0:
            return self.empty_state()
        _, ks, vs = self.forward_rows(prompt, np.arange(prompt.shape[0]), None)
        return SeqState(ks, vs, prompt.astype(np.int32))

    def refresh(self, state: SeqState) -> SeqState:
        """KV-refresh (Sec. 3.2, KV-cache and KV-refresh mechanism): all previously cached
        states are recomputed by a full forward pass.  Reading taken here: one forward over
        the tokens of the whole stored prefix (prompt and stored blocks), every position
        seeing every other one, replaces the stored K and V; blocks in flight take no part."""
        return self.prefill(state.ids)

    def denoise_forward(self, state: SeqState, block_ids: np.ndarray, sampler: Optional[Dict[str, object]] = None):
        """One forward of the block's rows (masked rows hold mask_id) against the prefix cache.
        Returns (logits [B, V], conf, tok, entropy).  ``sampler`` = dict(temperature, seed, seq,
        step) draws the tokens at that temperature (``sample_stats``) instead of taking the
        arg max."""
        B = len(block_ids)
        pos = state.prefix_len + np.arange(B)
        x, _, _ = self.forward_rows(np.asarray(block_ids), pos, state)
        lg = self.logits(x)
        if sampler is not None and sampler["temperature"] > 0:
            noise = gumbel_noise(sampler["seed"], sampler["seq"], pos, sampler["step"], self.vocab)
            conf, tok, ent = sample_stats(lg, self.mask_id, sampler["temperature"], noise)
        else:
            _, conf, tok, ent = softmax_stats(lg, self.mask_id)
        return lg, conf, tok, ent

    def denoise_step(self, state: SeqState, block_ids: np.ndarray, mask: np.ndarray, tau: float,
                     mode: int = MODE_CONFIDENCE, sampler: Optional[Dict[str, object]] = None):
        """Forward + decision.  Returns (new_ids, new_mask, commit[bool B], conf, tok, entropy)."""
        block_ids = np.array(block_ids, dtype=np.int32, copy=True)
        mask = np.array(mask, dtype=bool, copy=True)
        _, conf, tok, ent = self.denoise_forward(state, block_ids, sampler)
        commit = decide(conf, ent, mask, tau, mode)
        block_ids[commit] = tok[commit]
        mask[commit] = False
        return block_ids, mask, commit, conf, tok, ent

    def finalize_block(self, state: SeqState, block_ids: np.ndarray) -> SeqState:
        """Forward of the fully unmasked block; its K/V are appended to the cache."""
        B = len(block_ids)
        pos = state.prefix_len + np.arange(B)
        _, ks, vs = self.forward_rows(np.asarray(block_ids), pos, state)
        return SeqState([np.concatenate([a, b], axis=0) for a, b in zip(state.k, ks)],
                        [np.concatenate([a, b], axis=0) for a, b in zip(state.v, vs)],
                        np.concatenate([state.ids, np.asarray(block_ids, dtype=np.int32)]))

    def generate(self, prompt: np.ndarray, gen_len: int, block: int, tau: float,
                 mode: int = MODE_CONFIDENCE, record: bool = False,
                 eos_id: Optional[int] = None, refresh_every: int = 0,
                 temperature: float = 0.0, seed: int = 0, seq: int = 0) -> Dict[str, object]:
        """Block-by-block threshold decoding of one sequence.

        Returns tokens [gen_len], the step index (within its block, from 1) at which each
        position was committed, forward counts, and optionally a per-step trace.  With
        ``eos_id`` decoding halts after the step that commits that id (Sec. 3.2, early
        stopping on EOS); undecoded positions stay ``mask_id``.  With ``refresh_every`` = r > 0
        the cache is refreshed (``refresh``) each time the number of stored blocks reaches a
        multiple of r while blocks remain to be decoded (periodic KV-refresh, Sec. 3.2).
        ``temperature`` > 0 samples the tokens (``sample_stats``); the noise of a forward is
        keyed by (seed; sequence index ``seq``, absolute position, step within the block)."""
        assert gen_len % block == 0
        state = self.prefill(prompt)
        n_refresh = 0
        out = np.full(gen_len, self.mask_id, dtype=np.int32)
        commit_step = np.zeros(gen_len, dtype=np.int32)
        n_denoise = n_finalize = 0
        stopped = False
        trace: List[Dict[str, object]] = []
        for j in range(gen_len // block):
            ids = np.full(block, self.mask_id, dtype=np.int32)
            mask = np.ones(block, dtype=bool)
            step = 0
            while mask.any():
                step += 1
                assert step <= block, "each step must remove at least one mask"
                ids_in, mask_in = ids.copy(), mask.copy()
                sampler = dict(temperature=temperature, seed=seed, seq=seq, step=step) if temperature > 0 else None
                ids, mask, commit, conf, tok, ent = self.denoise_step(state, ids, mask, tau, mode, sampler)
                n_denoise += 1
                commit_step[j * block:(j + 1) * block][commit] = step
                if record:
                    trace.append(dict(block=j, step=step, prefix_len=state.prefix_len, ids_in=ids_in,
                                      mask_in=mask_in, conf=conf, tok=tok, ent=ent, commit=commit,
                                      ids_out=ids.copy(), mask_out=mask.copy()))
                if eos_id is not None and np.any(ids[commit] == eos_id):
                    stopped = True
                    break
            if stopped:
                out[j * block:(j + 1) * block] = np.where(mask, self.mask_id, ids)
                break
            state = self.finalize_block(state, ids)
            n_finalize += 1
            out[j * block:(j + 1) * block] = ids
            if refresh_every > 0 and (j + 1) % refresh_every == 0 and j + 1 < gen_len // block:
                state = self.refresh(state)
                n_refresh += 1
        res = dict(tokens=out, commit_step=commit_step, n_denoise=n_denoise, n_finalize=n_finalize,
                   stopped_early=stopped, n_refresh=n_refresh,
                   tpf_denoise=gen_len / max(n_denoise, 1),
                   tpf_all=gen_len / max(n_denoise + n_finalize, 1), state=state)
        if record:
            res["trace"] = trace
        return res

    def generate_multiblock(self, prompt: np.ndarray, gen_len: int, block: int, tau: float,
                            mode: int = MODE_ENTROPY, max_active: int = 2, record: bool = False,
                            cache_delay: int = 1, refresh_every: int = 0, eos_id: Optional[int] = None,
                            temperature: float = 0.0, seed: int = 0, seq: int = 0) -> Dict[str, object]:
        """Multi-block decoding of one sequence (Sec. 3.2, multi-block decoding strategy).

        Every round is one forward over the blocks in flight (oldest first), each seeing the
        cache, the earlier blocks in flight as they stand (masked rows included) and itself.
        Returns tokens [gen_len], the round (from 1) in which each position was committed, the
        number of rounds, the rows each round covered, and optionally a per-round trace.
        ``cache_delay``: stabilizing rounds a complete block goes through before its K/V are
        stored (1 or 2 in the paper's settings).  ``refresh_every`` = r > 0: after every r-th
        round the stored cache is refreshed (``refresh``) while blocks are still in flight.
        ``eos_id``: decoding halts after the round that commits that id in any block in flight;
        the blocks in flight go out as they stand (masked positions as ``mask_id``) and are not
        stored.  ``temperature`` > 0 samples the tokens; the noise of a round is keyed by (seed;
        ``seq``, absolute position, round)."""
        assert gen_len % block == 0 and max_active >= 1 and cache_delay >= 1
        n_blocks = gen_len // block
        state = self.prefill(prompt)
        out = np.full(gen_len, self.mask_id, dtype=np.int32)
        commit_round = np.zeros(gen_len, dtype=np.int32)
        lo = 0                                   # first block in flight
        win_ids: List[np.ndarray] = [np.full(block, self.mask_id, dtype=np.int32)]
        win_mask: List[np.ndarray] = [np.ones(block, dtype=bool)]
        win_stab: List[int] = [0]                # stabilizing forwards each block in flight has had
        rounds = 0
        n_refresh = 0
        stopped = False
        rows: List[int] = []
        trace: List[Dict[str, object]] = []
        while win_ids:
            rounds += 1
            assert rounds <= n_blocks * (block + cache_delay) + 1, "every round must make progress"
            n_win = len(win_ids)
            rows.append(n_win * block)
            # states as the masks stand before the forward
            unmasked = [int(block - m.sum()) for m in win_mask]
            complete_before = [u == block for u in unmasked]
            fully = [True if w == 0 else 100 * unmasked[w - 1] >= 95 * block for w in range(n_win)]
            ids_in = [a.copy() for a in win_ids]
            mask_in = [a.copy() for a in win_mask]
            # the forward: block w sees the cache and blocks 0..w-1 of the window
            tmp = state
            stats = []
            sampler = dict(temperature=temperature, seed=seed, seq=seq, step=rounds) if temperature > 0 else None
            for w in range(n_win):
                _, conf, tok, ent = self.denoise_forward(tmp, win_ids[w], sampler)
                stats.append((conf, tok, ent))
                if w + 1 < n_win:
                    tmp = self.finalize_block(tmp, win_ids[w])
            # decisions
            commits = []
            for w in range(n_win):
                conf, tok, ent = stats[w]
                m = win_mask[w]
                if complete_before[w]:
                    commit = np.zeros(block, dtype=bool)
                elif fully[w]:
                    commit = decide(conf, ent, m, tau, mode)
                else:  # Activated: only what clears the threshold
                    commit = m & ((conf > tau) if mode == MODE_CONFIDENCE else (ent < tau))
                win_ids[w] = win_ids[w].copy()
                win_ids[w][commit] = tok[commit]
                win_mask[w] = m & ~commit
                commit_round[(lo + w) * block:(lo + w + 1) * block][commit] = rounds
                commits.append(commit)
            if record:
                trace.append(dict(round=rounds, lo=lo, n_win=n_win, fully=list(fully), ids_in=ids_in, mask_in=mask_in,
                                  complete_before=list(complete_before), stats=stats, commits=commits,
                                  ids_out=[a.copy() for a in win_ids], mask_out=[a.copy() for a in win_mask]))
            if eos_id is not None and any(np.any(win_ids[w][commits[w]] == eos_id) for w in range(n_win)):
                for w in range(n_win):   # early stop: everything in flight goes out as it stands
                    out[(lo + w) * block:(lo + w + 1) * block] = np.where(win_mask[w], self.mask_id, win_ids[w])
                stopped = True
                break
            # blocks that were complete before this forward have had a stabilizing round: the
            # oldest ones enter the cache, in order, once they have had cache_delay of them
            for w in range(n_win):
                if complete_before[w]:
                    win_stab[w] += 1
            while win_ids and win_stab[0] >= cache_delay:
                state = self.finalize_block(state, win_ids[0])
                out[lo * block:(lo + 1) * block] = win_ids[0]
                win_ids.pop(0); win_mask.pop(0); win_stab.pop(0)
                lo += 1
            # a new block: when the newest one is 10 % complete (or nothing is in flight)
            nxt = lo + len(win_ids)
            if nxt < n_blocks and len(win_ids) < max_active:
                if not win_ids or 100 * int(block - win_mask[-1].sum()) >= 10 * block:
                    win_ids.append(np.full(block, self.mask_id, dtype=np.int32))
                    win_mask.append(np.ones(block, dtype=bool))
                    win_stab.append(0)
            if refresh_every > 0 and rounds % refresh_every == 0 and win_ids and state.prefix_len > 0:
                state = self.refresh(state)
                n_refresh += 1
        res = dict(tokens=out, commit_round=commit_round, rounds=rounds, rows=rows, state=state,
                   n_refresh=n_refresh, stopped_early=stopped,
                   tokens_per_round=gen_len / max(rounds, 1))
        if record:
            res["trace"] = trace
        return res

    # -- independent references used to pin the path above
    def brute_force_block(self, prompt: np.ndarray, done_blocks: Sequence[np.ndarray],
                          cur_block: np.ndarray):
        """The same block forward with no cache: the whole sequence (prompt, finished blocks,
        current block) goes through the stack under segment visibility seg(key) <= seg(query).
        Returns (logits of the current block's rows, conf, tok, entropy)."""
        segs = [np.asarray(prompt)] + [np.asarray(b) for b in done_blocks] + [np.asarray(cur_block)]
        ids = np.concatenate(segs)
        seg_id = np.concatenate([np.full(len(s), i) for i, s in enumerate(segs)])
        visible = seg_id[None, :] <= seg_id[:, None]
        x, _, _ = self.forward_rows(ids, np.arange(len(ids)), None, visible)
        lg = self.logits(x[-len(cur_block):])
        _, conf, tok, ent = softmax_stats(lg, self.mask_id)
        return lg, conf, tok, ent

    def sequential_decode(self, prompt: np.ndarray, gen_len: int, block: int) -> Tuple[np.ndarray, np.ndarray]:
        """One token per forward pass: in each block, repeatedly run the block forward and unmask
        only the masked position whose prediction is most probable.  Written separately from
        ``generate``/``decide``.  Returns (tokens, order) where order[t] is the global position
        unmasked at step t."""
        state = self.prefill(prompt)
        tokens = np.full(gen_len, self.mask_id, dtype=np.int32)
        order = []
        for j in range(gen_len // block):
            ids = np.full(block, self.mask_id, dtype=np.int32)
            for _ in range(block):
                _, conf, tok, _ = self.denoise_forward(state, ids)
                best, best_r = -1.0, -1
                for r in range(block):
                    if ids[r] == self.mask_id and conf[r] > best:
                        best, best_r = conf[r], r
                ids[best_r] = tok[best_r]
                order.append(j * block + best_r)
            state = self.finalize_block(state, ids)
            tokens[j * block:(j + 1) * block] = ids
        return tokens, np.asarray(order, dtype=np.int32)


# ----------------------------------------------------------------------------- pseudo-trajectory
def trajectory_rank(commit_step: np.ndarray, block: int) -> np.ndarray:
    """Decoding step (1-based, counted over the whole response) at which each position was unmasked,
    from the per-block step indices ``generate`` records: blocks are decoded one after the other,
    so a block's steps follow all steps of the blocks before it (Sec. 3.1: the recorded decoding
    trajectory T_1..T_n; with exactly one token per step the ranks are a permutation of 1..n)."""
    commit_step = np.asarray(commit_step)
    n = commit_step.shape[0]
    assert n % block == 0
    rank = np.zeros(n, dtype=np.int64)
    done = 0
    for j in range(n // block):
        cs = commit_step[j * block:(j + 1) * block]
        rank[j * block:(j + 1) * block] = done + cs
        done += int(cs.max())
    return rank


def trajectory_states(y: np.ndarray, rank: np.ndarray, mask_id: int) -> np.ndarray:
    """The trajectory written out: row j (0..n_steps) is the response after j decoding steps, the
    positions unmasked so far holding y's tokens and the rest ``mask_id`` (Sec. 3.1, T_j)."""
    y = np.asarray(y)
    n_steps = int(np.max(rank)) if len(rank) else 0
    T = np.full((n_steps + 1, len(y)), mask_id, dtype=np.int64)
    for j in range(n_steps + 1):
        for i in range(len(y)):
            if rank[i] <= j:
                T[j, i] = y[i]
    return T


def ceil_ratio(k: int, t_num: int, t_den: int) -> int:
    """ceil(k * t) for the mask ratio t = t_num / t_den in integers."""
    assert t_den > 0 and 0 <= t_num <= t_den and k >= 0
    return -((-k * t_num) // t_den)


def noisy_sequence(y: np.ndarray, rank: np.ndarray, s: int, k: int, m: int, mask_id: int) -> np.ndarray:
    """The noisy training sequence of Sec. 3.1 (the displayed equation): with positions counted
    from 1, window w = {s, .., s+k} and m = ceil(k t), position i keeps y_i if i <= s or it is
    unmasked in trajectory state T_{s+m}, and is the mask token if i > s+k or it is still masked
    in T_{s+m}.  Reading taken where the two cases overlap: i <= s keeps the token, i > s+k is
    masked, and only in between does the trajectory decide.  A step index beyond the recorded
    trajectory means its last state."""
    y = np.asarray(y)
    T = trajectory_states(y, rank, mask_id)
    step = min(s + m, T.shape[0] - 1)
    out = np.empty(len(y), dtype=np.int64)
    for i in range(1, len(y) + 1):
        if i <= s:
            out[i - 1] = y[i - 1]
        elif i > s + k:
            out[i - 1] = mask_id
        else:
            out[i - 1] = y[i - 1] if T[step, i - 1] != mask_id else mask_id
    return out


def model_from_shape(shape, weights: Dict[str, object], dtype=np.float64, mirror_bf16: bool = False
                     ) -> OracleModel:
    """Build an OracleModel from any object with the usual shape attributes."""
    return OracleModel(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                       n_kv_heads=shape.n_kv_heads, d_head=shape.d_head, d_ffn=shape.d_ffn,
                       vocab=shape.vocab, mask_id=shape.mask_id, weights=weights,
                       rope_theta=shape.rope_theta, rms_eps=shape.rms_eps,
                       logit_scale=shape.logit_scale, dtype=dtype, mirror_bf16=mirror_bf16)
