"""Helpers shared by the GPU parity tests: context construction, oracle-side bookkeeping, the record
of parity counts and the free-running comparison protocol."""
import json
import os

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


# ----------------------------------------------------------------------------- parity record
EPS = 1e-3                 # the near-tie bound of the parity rule
# At most this share of the compared (step, masked position) pairs may fall into the "rounding" class.
# Measured on the small random-init bf16 models of these tests: 2-5.5 % (the SIMT bf16 path as much as the
# tensor-core path: with confidences in error by 1-3e-2, which the 3e-2 logit bar allows, every decision
# whose oracle margin is below that error can fall either way, and a random model spreads its
# confidences evenly over (0, 1)).  The counts of every run are written by record_report().
ROUNDING_SHARE_MAX = 0.08
_REPORTS = {}


def record_report(name: str, report: dict) -> None:
    """Keep the counts of a parity comparison and write all of them to $D3_REPORT_DIR/parity_reports.json
    (default: a parity_reports folder beside the tests), so that the number of excused and
    rounding-class positions behind a green run is on record."""
    clean = {}
    for k, v in report.items():
        if isinstance(v, (np.floating, np.integer)):
            v = v.item()
        if isinstance(v, (int, float, str, bool)) or v is None:
            clean[str(k)] = v
        elif isinstance(v, (list, tuple)) and all(isinstance(x, (int, float, str, bool)) for x in v):
            clean[str(k)] = list(v)
        else:
            clean[str(k)] = str(v)
    _REPORTS[name] = clean
    out_dir = os.environ.get("D3_REPORT_DIR") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "parity_reports")
    try:
        os.makedirs(out_dir, exist_ok=True)
        path = os.path.join(out_dir, "parity_reports.json")
        merged = {}
        if os.path.exists(path):
            try:
                with open(path) as f:
                    merged = json.load(f)
            except ValueError:
                merged = {}
        merged.update(_REPORTS)
        with open(path, "w") as f:
            json.dump(merged, f, indent=1, sort_keys=True)
    except OSError:
        pass


def assert_rounding_bounded(report: dict, stat_err_bound: float) -> None:
    """The bar for a bf16 step-locked comparison: nothing unexplained, the rounding class (oracle margin
    between 1e-3 and twice the largest statistic error of the run) is a small share of the positions,
    and that largest statistic error itself stays below ``stat_err_bound``."""
    assert report["self_diff"] == 0 and report["unexplained"] == 0, report
    assert report["max_stat_err"] <= stat_err_bound, report
    assert report["rounding"] <= max(1, int(ROUNDING_SHARE_MAX * report["positions"])), report


def free_running_p2(ctx, model, prompt: np.ndarray, gen_len: int, block: int, tau: float, noise: float,
                    generate=None):
    """Free-running comparison of d3_generate with the oracle on one sequence (batch 1).

    Both sides decode on their own.  Tokens and commit steps are compared block by block; at the first
    block that differs, the earliest step of that block at which the two sides took different decisions
    is located (up to it both sides were in the same state), and the oracle's margin at that step -- the
    distance of the differing position's confidence from the threshold, the gap between the two best
    masked positions when the forced commit differs, the top-2 probability gap when the token differs --
    must be below 1e-3 (``excused``) or at most ``noise`` (``rounding``: below the two sides' own
    numerical difference as measured by the step-locked run of the same model); anything else fails.
    The GPU is then re-synchronised from the oracle: prefill, the oracle's blocks up to and including
    the differing one committed with d3_commit_block, and decoding continues from there.  Returns the
    counts."""
    from oracle import d3_oracle as o
    if generate is None:
        generate = lambda n: ctx.generate(1, n, tau)  # noqa: E731
    ref = model.generate(prompt, gen_len, block, tau, record=True)
    n_blocks = gen_len // block
    ids = prompt[None, :].astype(np.int32)
    lens = np.array([len(prompt)], dtype=np.int32)
    report = dict(blocks=n_blocks, resyncs=0, excused=0, rounding=0, margins=[])
    j0 = 0
    while j0 < n_blocks:
        ctx.prefill(ids, lens)
        for jj in range(j0):
            ctx.commit(ref["tokens"][None, jj * block:(jj + 1) * block].astype(np.int32))
        tok, cs, _ = generate(gen_len - j0 * block)
        tok, cs = tok[0], cs[0]
        want_tok, want_cs = ref["tokens"][j0 * block:], ref["commit_step"][j0 * block:]
        bad = None
        for j in range(n_blocks - j0):
            sl = slice(j * block, (j + 1) * block)
            if not (np.array_equal(tok[sl], want_tok[sl]) and np.array_equal(cs[sl], want_cs[sl])):
                bad = j
                break
        if bad is None:
            break
        jb = j0 + bad
        sl = slice(bad * block, (bad + 1) * block)
        differ = (tok[sl] != want_tok[sl]) | (cs[sl] != want_cs[sl])
        s_star = int(np.minimum(cs[sl], want_cs[sl])[differ].min())
        t = next(t for t in ref["trace"] if t["block"] == jb and t["step"] == s_star)
        mk = t["mask_in"]
        conf = t["conf"]
        gpu_commit = mk & (cs[sl] == s_star)
        ora_commit = t["commit"]
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
        tok_diff = np.flatnonzero(both & (tok[sl] != want_tok[sl]))
        if len(tok_diff):
            st = model.prefill(prompt)
            for jj in range(jb):
                st = model.finalize_block(st, ref["tokens"][jj * block:(jj + 1) * block])
            gap = top2_gap(model.denoise_forward(st, t["ids_in"])[0], model.mask_id)
            margins.extend(float(gap[r]) for r in tok_diff)
        assert margins, ("the two sides differ in block %d but not at its first differing step" % jb, s_star)
        worst = max(margins)
        assert worst <= max(noise, EPS), ("divergence that no near-tie explains", jb, s_star, margins, noise)
        report["excused" if worst < EPS else "rounding"] += 1
        report["margins"].append(round(worst, 6))
        report["resyncs"] += 1
        j0 = jb + 1
    return report
