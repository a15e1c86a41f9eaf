"""The five synthetic workload shapes plus shrunk-capacity eviction-stress variants.

Shapes (batch, heads, head_dim, context, tree size, table parameters, vocabulary, stream statistics) are
those of the benchmark definition; crt (= max_nodes / 4) and the depth cap of config 3 are choices made
here because the definition leaves them open.
"""
from dataclasses import dataclass, replace
from typing import Tuple


@dataclass(frozen=True)
class CbConfig:
    name: str
    batch: int
    LL: int
    FL: int
    LC: int
    FC: int
    max_nodes: int          # tree-size cap, root included (the paper's total draft length)
    max_depth: int
    crt: int                # nodes reserved for query level >= 2
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ctx_range: Tuple[int, int]   # inclusive; equal ends = fixed context
    vocab: int
    zipf_s: float
    copy_frac: float        # target fraction of positions inside copy spans
    span_range: Tuple[int, int]
    stream_len: int         # 0 = ctx_b + 512
    turns: int = 1          # >1: multi-turn stream (config 4)
    page_size: int = 16
    seed: int = 0

    @property
    def max_ctx(self) -> int:
        return self.ctx_range[1]

    @property
    def gqa(self) -> int:
        return self.n_q_heads // self.n_kv_heads


CONFIGS = {
    "c1_tiny": CbConfig("c1_tiny", 1, 2, 3, 4096, 4, 16, 5, 4, 8, 8, 64, (512, 512), 32000, 1.1, 0.30,
                        (4, 32), 2048),
    "c2_7b": CbConfig("c2_7b", 1, 2, 4, 16384, 4, 64, 8, 16, 32, 32, 128, (4096, 4096), 32000, 1.1, 0.40,
                      (4, 32), 8192),
    "c3_8b_gqa": CbConfig("c3_8b_gqa", 32, 3, 4, 16384, 4, 64, 8, 16, 32, 8, 128, (1024, 8192), 128256, 1.05,
                          0.35, (4, 32), 0),
    "c4_13b_turns": CbConfig("c4_13b_turns", 64, 2, 3, 8192, 6, 32, 6, 8, 40, 40, 128, (2048, 2048), 32000,
                             1.1, 0.0, (8, 64), 4096, turns=4),
    "c5_70b_long": CbConfig("c5_70b_long", 128, 3, 5, 65536, 8, 128, 10, 32, 64, 8, 128, (32768, 32768),
                            128256, 1.05, 0.25, (4, 32), 0),
}
# Eviction stress: the five shapes never evict a leader (LC >= 2x stream length), so shrink LC.
CONFIGS["c1_evict256"] = replace(CONFIGS["c1_tiny"], name="c1_evict256", LC=256)
CONFIGS["c1_evict1024"] = replace(CONFIGS["c1_tiny"], name="c1_evict1024", LC=1024)
CONFIGS["c3_evict256"] = replace(CONFIGS["c3_8b_gqa"], name="c3_evict256", LC=256, batch=4)
CONFIGS["c3_evict1024"] = replace(CONFIGS["c3_8b_gqa"], name="c3_evict1024", LC=1024, batch=4)
# The paper's tuned table regime (Section 4: LL = 1, LC = 2^20, FL = 3, FC = 128, TDL = 96, CRT = 16) on config 2's model
# shape; the depth cap (8 followers deep) is a choice made here.  The second variant shrinks the capacities so that both
# LRU domains evict, with a follower capacity that is not a multiple of the warp width.
CONFIGS["p_tuned"] = replace(CONFIGS["c2_7b"], name="p_tuned", LL=1, FL=3, LC=1 << 20, FC=128, max_nodes=96, crt=16,
                             max_depth=24)
CONFIGS["p_fc40_evict"] = replace(CONFIGS["p_tuned"], name="p_fc40_evict", LC=512, FC=40)


# The 70B shape on a batch small enough for a profiler capture (keys and values of 8 sequences: 1.1 GB).
CONFIGS["c5_70b_b8"] = replace(CONFIGS["c5_70b_long"], name="c5_70b_b8", batch=8)


def get_config(name: str) -> CbConfig:
    return CONFIGS[name]
