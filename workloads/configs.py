"""The five benchmark configurations as concrete shapes.

Index 0..4 follow the order of the benchmark description: tiny, 7B-shaped
single layer, GQA ragged batch, long context, full 32-layer step.
"""
from dataclasses import dataclass, replace


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    B: int            # sequences
    Hq: int           # query heads
    Hkv: int          # KV heads
    d: int            # head dim
    L: int            # layers that share one tree / mask
    S_lo: int         # prefix length range (inclusive)
    S_hi: int
    Scap: int         # cache capacity per sequence (rows)
    N: int            # tree nodes including the root (= Nmax)
    D: int            # max depth (edges from the root)
    V: int            # vocabulary (0: config has no logits)
    tree: str         # "uniform" | "topk" | "spine" | "chains"
    topk: int
    P: int            # candidate-path rows (0: one row per leaf, capacity = N)
    std: float        # std of Q/K/V entries
    plant: str        # "none" | "full" | "geometric"

    def scaled(self, **kw):
        return replace(self, **kw)


CONFIGS = [
    VerifyConfig("tiny", B=1, Hq=4, Hkv=2, d=64, L=1, S_lo=128, S_hi=128, Scap=256,
                 N=15, D=4, V=1024, tree="uniform", topk=0, P=0, std=1.0, plant="none"),
    VerifyConfig("llama7b_layer", B=1, Hq=32, Hkv=32, d=128, L=1, S_lo=2048, S_hi=2048, Scap=2304,
                 N=60, D=6, V=32000, tree="topk", topk=10, P=0, std=128 ** -0.5, plant="none"),
    VerifyConfig("gqa8b_ragged", B=8, Hq=32, Hkv=8, d=128, L=1, S_lo=1024, S_hi=8192, Scap=8448,
                 N=64, D=7, V=128256, tree="topk", topk=8, P=0, std=128 ** -0.5, plant="full"),
    VerifyConfig("long_context", B=4, Hq=32, Hkv=8, d=128, L=1, S_lo=32768, S_hi=32768, Scap=33024,
                 N=128, D=8, V=0, tree="topk", topk=8, P=0, std=128 ** -0.5, plant="none"),
    VerifyConfig("full_step_32l", B=16, Hq=32, Hkv=8, d=128, L=32, S_lo=512, S_hi=4096, Scap=4224,
                 N=60, D=6, V=153600, tree="topk", topk=10, P=10, std=128 ** -0.5, plant="geometric"),
]


def get_config(i_or_name) -> VerifyConfig:
    if isinstance(i_or_name, int):
        return CONFIGS[i_or_name]
    for c in CONFIGS:
        if c.name == i_or_name:
            return c
    raise KeyError(i_or_name)
