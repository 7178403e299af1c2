"""Workload shapes: a tiny case plus head/vocabulary geometries of the model families the paper
evaluates (7B MHA, 8B GQA, 70B GQA) with its tree budget (depth 6, 10 per expansion, 60 draft tokens;
Appendix A)."""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class Config:
    name: str
    B: int  # independent sequences
    V: int  # vocabulary
    k: int  # children per node and frontier size
    D: int  # tree depth
    m: int  # rerank budget (draft tokens sent to verification)
    n_layers: int
    Hq: int
    Hkv: int
    d: int
    kv_len: int  # committed tokens per sequence (fixed-length configs)
    kv_len_range: tuple | None = None  # (lo, hi): log-uniform ragged lengths instead of kv_len
    temperature: float = 0.0
    p_easy: float | None = 0.5  # None: one p_easy ~ U(0,1) per sequence

    @property
    def N(self) -> int:  # candidate nodes per tree
        return self.k + (self.D - 1) * self.k * self.k

    @property
    def R(self) -> int:  # draft-logit rows per cycle
        return 1 + (self.D - 1) * self.k

    @property
    def g(self) -> int:
        return self.Hq // self.Hkv

    def with_(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    "tiny": Config("tiny", 1, 1000, 4, 3, 16, 1, 4, 4, 64, 128, temperature=0.0),
    "vicuna7b": Config("vicuna7b", 1, 32000, 10, 6, 60, 32, 32, 32, 128, 1024, temperature=0.0),
    "llama3_8b": Config("llama3_8b", 1, 128256, 10, 6, 60, 32, 32, 8, 128, 4096, temperature=1.0),
    "llama2_70b": Config("llama2_70b", 1, 32000, 10, 6, 60, 80, 64, 8, 128, 8192, temperature=0.0),
    "llama3_8b_batched": Config("llama3_8b_batched", 32, 128256, 10, 6, 60, 32, 32, 8, 128, 4096,
                                kv_len_range=(512, 16384), temperature=1.0, p_easy=None),
}


def get_config(name: str, **overrides) -> Config:
    cfg = CONFIGS[name]
    return cfg.with_(**overrides) if overrides else cfg
