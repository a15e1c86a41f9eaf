"""Token streams: Zipf-distributed ids with copy-spans that repeat earlier text.

A stream is what a sequence's token history looks like to the drafter: mostly frequent tokens, with
stretches that re-quote earlier context (the locality the cache table exploits).  All draws come from
the counter-based hash, keyed by (seed, sequence index).
"""
from functools import lru_cache
import math
import numpy as np

from .rng import uniform_f64
from .configs import CbConfig

# tensor ids used by the stream generator (distinct from those in tensors.py)
_TID_ZIPF, _TID_START, _TID_LEN, _TID_SRC, _TID_FRAC = 101, 102, 103, 104, 105
_SEQ_STRIDE = 1 << 24   # flat index = b * _SEQ_STRIDE + position


@lru_cache(maxsize=8)
def _zipf_cdf(vocab: int, s: float) -> np.ndarray:
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    return c / c[-1]


def _rank_to_id(rank: np.ndarray, vocab: int) -> np.ndarray:
    """Fixed multiplicative permutation of [0, vocab): frequent ranks are scattered over the id space."""
    a = 2654435761 % vocab
    while math.gcd(a, vocab) != 1:
        a += 1
    return ((rank.astype(np.int64) * a + 12345) % vocab).astype(np.int32)


def _zipf_tokens(cfg: CbConfig, b: int, n: int) -> np.ndarray:
    u = uniform_f64(cfg.seed, _TID_ZIPF, b * _SEQ_STRIDE + np.arange(n))
    rank = np.minimum(np.searchsorted(_zipf_cdf(cfg.vocab, cfg.zipf_s), u, side="right"), cfg.vocab - 1)
    return _rank_to_id(rank, cfg.vocab)


def _fill_spans(out: np.ndarray, lo: int, hi: int, frac: float, span_range, src_hi_fn, cfg: CbConfig, b: int):
    """Overwrite parts of out[lo:hi] with copies of earlier text so that about ``frac`` of the positions
    fall inside copy spans. src_hi_fn(pos) is the exclusive upper bound of positions a span may copy from."""
    if frac <= 0.0:
        return
    smin, smax = span_range
    mean_len = 0.5 * (smin + smax)
    q = frac / (mean_len * (1.0 - frac) + frac)          # per-position start probability outside spans
    pos_idx = b * _SEQ_STRIDE + np.arange(lo, hi)
    starts = np.nonzero(uniform_f64(cfg.seed, _TID_START, pos_idx) < q)[0] + lo
    u_len = uniform_f64(cfg.seed, _TID_LEN, b * _SEQ_STRIDE + starts)
    u_src = uniform_f64(cfg.seed, _TID_SRC, b * _SEQ_STRIDE + starts)
    busy_until = lo
    for k, p in enumerate(starts.tolist()):
        if p < busy_until:
            continue
        length = min(smin + int(u_len[k] * (smax - smin + 1)), hi - p)
        src_hi = src_hi_fn(p)
        if src_hi < 1:
            continue                                     # no history yet: keep the Zipf draw
        src = int(u_src[k] * src_hi)
        if src + length <= p:
            out[p:p + length] = out[src:src + length]
        else:                                            # the span runs into itself: token by token
            for j in range(length):
                out[p + j] = out[src + j]
        busy_until = p + length


def make_stream(cfg: CbConfig, b: int, length: int) -> np.ndarray:
    """int32 token stream of ``length`` ids for sequence ``b``."""
    out = _zipf_tokens(cfg, b, length).copy()
    if cfg.turns <= 1:
        _fill_spans(out, 0, length, cfg.copy_frac, cfg.span_range, lambda p: p, cfg, b)
    else:
        turn = length // cfg.turns
        fr = uniform_f64(cfg.seed, _TID_FRAC, b * 64 + np.arange(cfg.turns))
        for t in range(1, cfg.turns):
            lo, hi = t * turn, (length if t == cfg.turns - 1 else (t + 1) * turn)
            frac = 0.2 + 0.4 * float(fr[t])
            smax = cfg.span_range[1]
            _fill_spans(out, lo, hi, frac, cfg.span_range, lambda p, lo=lo, smax=smax: max(0, lo - smax), cfg, b)
    return out


def stream_length(cfg: CbConfig, ctx_b: int) -> int:
    return cfg.stream_len if cfg.stream_len > 0 else ctx_b + 512


def make_streams(cfg: CbConfig, ctx: np.ndarray):
    """Streams of the whole batch, right-padded with -1 to a common row length.
    Returns (tokens int32 [B, max_len], lengths int32 [B])."""
    lens = np.array([stream_length(cfg, int(c)) for c in ctx], dtype=np.int32)
    toks = np.full((cfg.batch, int(lens.max())), -1, dtype=np.int32)
    for b in range(cfg.batch):
        toks[b, : lens[b]] = make_stream(cfg, b, int(lens[b]))
    return toks, lens
