"""Shapes of the five synthetic workloads (paper notation in the field names).

H query heads, H_G key/value heads, d head dim, d_c compressed dim (d' in the
paper), l_I initial tokens, l_L local tokens, l_C chunk length, k selected
middle tokens, eps proximity distance (Eq. 8).  The head counts and d' of
configs 2, 3 and 5 are the paper's Section 4.1 parameters (H=32, d_H=4096,
d'=128, 8 GQA heads, l_I=128); eps=3 is the value whose ablation column
matches the paper's main tables.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class EsaShape:
    name: str
    H: int
    H_G: int
    d: int
    d_c: int
    l_C: int
    l_I: int
    l_L: int
    k: int
    eps: int
    S: int            # prefill length (tokens already cached before decode)
    B: int = 1        # independent sequences
    n_decode: int = 0  # decode steps after the prefill
    seed: int = 0
    n_layers: int = 1
    kind: str = "normal"  # "normal" | "headscale" | "gmm_needles"

    @property
    def d_H(self) -> int:
        return self.H * self.d

    @property
    def d_G(self) -> int:
        return self.H_G * self.d

    @property
    def max_tokens(self) -> int:
        return self.S + self.n_decode

    def with_(self, **kw) -> "EsaShape":
        return replace(self, **kw)


CONFIGS = {
    # single layer, tiny: full chunked prefill + 16 decode steps
    "c1": EsaShape("c1", H=8, H_G=2, d=64, d_c=32, l_C=128, l_I=4, l_L=512, k=256,
                   eps=3, S=4096, B=1, n_decode=16, seed=0),
    # Llama-3-8B attention shape, 32k prefill in chunks of 512
    "c2": EsaShape("c2", H=32, H_G=8, d=128, d_c=128, l_C=512, l_I=128, l_L=2048,
                   k=4096, eps=3, S=32768, seed=1, kind="headscale"),
    # Llama-3-8B shape, decode: 8 sequences with 131072 cached tokens, 256 steps
    "c3": EsaShape("c3", H=32, H_G=8, d=128, d_c=128, l_C=1, l_I=128, l_L=2048,
                   k=4096, eps=3, S=131072, B=8, n_decode=256, seed=2),
    # 7B / 32k-native shape: 256k prefill in chunks of 1024
    "c4": EsaShape("c4", H=28, H_G=4, d=128, d_c=128, l_C=1024, l_I=128, l_L=4096,
                   k=8192, eps=3, S=262144, seed=3),
    # 32-layer Llama-3-8B stack, 128k prefill, mixture keys with planted needles
    "c5": EsaShape("c5", H=32, H_G=8, d=128, d_c=128, l_C=512, l_I=128, l_L=2048,
                   k=4096, eps=3, S=131072, seed=4, n_layers=32, kind="gmm_needles"),
}


def get_config(name: str) -> EsaShape:
    return CONFIGS[name]
