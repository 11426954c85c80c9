"""Helpers shared by the GPU parity tests: context construction and oracle-side bookkeeping."""
import numpy as np
import torch

from oracle import d3_oracle as o
from paper_2601_07568_b200 import binding as d3
from paper_2601_07568_b200 import synth_inputs as si

DEV = "cuda:0"


class Ctx:
    """A d3 context with its weights loaded; frees itself on close()."""

    def __init__(self, shape, weights, *, block, max_batch, max_seq, max_prefill_rows=0,
                 decide_mode=d3.D3_DECIDE_CONFIDENCE, gemm_impl=d3.D3_GEMM_AUTO):
        self.shape, self.block = shape, block
        torch.cuda.set_device(0)
        self.cfg = d3.make_config(shape, block=block, max_batch=max_batch, max_seq=max_seq,
                                  max_prefill_rows=max_prefill_rows, decide_mode=decide_mode, gemm_impl=gemm_impl)
        self.ctx = d3.d3_create(self.cfg)
        if weights is not None:
            d3.d3_load_weights(self.ctx, d3.weights_from_numpy(shape, weights), shape.n_layers)

    def close(self):
        if self.ctx is not None:
            d3.d3_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # -- thin wrappers returning host arrays
    def prefill(self, ids: np.ndarray, lens: np.ndarray):
        d3.d3_prefill(self.ctx, torch.tensor(ids, dtype=torch.int32, device=DEV).contiguous(),
                      torch.tensor(lens, dtype=torch.int32, device=DEV))

    def logits(self, block_ids: np.ndarray) -> np.ndarray:
        bs, B = block_ids.shape
        out = torch.empty(bs * B, self.shape.vocab, dtype=torch.float32, device=DEV)
        d3.d3_forward_logits(self.ctx, torch.tensor(block_ids, dtype=torch.int32, device=DEV), out)
        torch.cuda.synchronize()
        return out.cpu().numpy().reshape(bs, B, -1)

    def step(self, block_ids: np.ndarray, mask: np.ndarray, tau: float):
        bs, B = block_ids.shape
        ids = torch.tensor(block_ids, dtype=torch.int32, device=DEV)
        m = torch.tensor(mask.astype(np.uint8), dtype=torch.uint8, device=DEV)
        pos = torch.full((bs, B), -1, dtype=torch.int32, device=DEV)
        oid = torch.full((bs, B), -1, dtype=torch.int32, device=DEV)
        cnt = torch.zeros(bs, dtype=torch.int32, device=DEV)
        d3.d3_denoise_step(self.ctx, ids, m, tau, pos, oid, cnt)
        conf = torch.empty(bs * B, dtype=torch.float32, device=DEV)
        ent = torch.empty(bs * B, dtype=torch.float32, device=DEV)
        am = torch.empty(bs * B, dtype=torch.int32, device=DEV)
        d3.d3_get_step_stats(self.ctx, conf, ent, am, bs)
        torch.cuda.synchronize()
        return dict(ids=ids.cpu().numpy(), mask=m.cpu().numpy().astype(bool), pos=pos.cpu().numpy(),
                    out_ids=oid.cpu().numpy(), count=cnt.cpu().numpy(), conf=conf.cpu().numpy().reshape(bs, B),
                    ent=ent.cpu().numpy().reshape(bs, B), tok=am.cpu().numpy().reshape(bs, B))

    def commit(self, block_ids: np.ndarray):
        d3.d3_commit_block(self.ctx, torch.tensor(block_ids, dtype=torch.int32, device=DEV))

    def generate(self, bs: int, gen_len: int, tau: float):
        out = torch.full((bs, gen_len), -1, dtype=torch.int32, device=DEV)
        cs = torch.zeros((bs, gen_len), dtype=torch.int32, device=DEV)
        st = d3.d3_generate(self.ctx, gen_len, tau, out, cs)
        return out.cpu().numpy(), cs.cpu().numpy(), st

    def generate_multiblock(self, bs: int, gen_len: int, tau: float, max_active: int):
        out = torch.full((bs, gen_len), -1, dtype=torch.int32, device=DEV)
        cr = torch.zeros((bs, gen_len), dtype=torch.int32, device=DEV)
        st = d3.d3_generate_multiblock(self.ctx, gen_len, tau, out, max_active, cr)
        return out.cpu().numpy(), cr.cpu().numpy(), st

    def set_prefix(self, lens):
        d3.d3_set_state(self.ctx, torch.tensor(lens, dtype=torch.int32, device=DEV))

    def get_prefix(self, bs):
        t = torch.zeros(bs, dtype=torch.int32, device=DEV)
        d3.d3_get_state(self.ctx, t)
        torch.cuda.synchronize()
        return t.cpu().numpy()

    def error_word(self) -> int:
        return d3.d3_get_error_word(self.ctx)


def oracle_near_tie(conf: np.ndarray, probs_top2_gap: np.ndarray, mask: np.ndarray, tau: float, eps=1e-3):
    """Positions excused from bit-exact commit comparison: oracle confidence within eps of the
    threshold or top-2 probability gap below eps (token near-tie); and whether the forced choice
    is a near-tie between the two best masked positions."""
    near = (np.abs(conf - tau) < eps) | (probs_top2_gap < eps)
    cm = np.where(mask, conf, -np.inf)
    srt = np.sort(cm)[::-1]
    forced_tie = bool(mask.sum() >= 2 and (srt[0] - srt[1]) < eps)
    return near, forced_tie


def top2_gap(logits: np.ndarray, mask_id: int) -> np.ndarray:
    p, conf, tok, ent = o.softmax_stats(logits, mask_id)
    part = np.partition(p, -2, axis=-1)
    return part[:, -1] - part[:, -2]
