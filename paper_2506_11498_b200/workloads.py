"""Seeded synthetic inputs shaped like the paper's long-context post-training workload.

Shared by the CUDA path's tests/benchmark and by the oracle's tests.  Holds no arithmetic of
the method: only shapes, seeds and value distributions.  The paper (Section 4.1) trains
Qwen2.5-1.5B at 32K context with lag L = 1024 and retention r = 0.5, and every evaluated row of
Table 1 uses L = context / 32; its datasets and weights are not available here, so these
tensors stand in for the projected Q/K/V of one attention layer.

Recipe (all on the CPU, one ``torch.Generator`` per workload, seeded with ``seed``):
draw fp32 standard normals in the order Q, K, V, dO, batch element by batch element; apply the
workload's value structure to K in fp32; round to bf16 (round-to-nearest-even).
  * ``normal``          : nothing added.
  * ``channel_offset``  : K[b,h,:,c] += o[h,c], o ~ N(0, std 2), drawn right after K's normals
                          of batch element 0 and reused for every batch element (outlier channels).
  * ``salient``         : per (b, kv head) each token position is marked with probability 0.01
                          (uniform draw right after that batch element's K normals); marked K rows
                          are multiplied by 8.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    N: int
    d: int
    L: int      # lag window = query chunk
    K: int      # kept tokens per window
    S: int      # sink tokens
    seed: int = 0
    values: str = "normal"   # normal | channel_offset | salient

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


CFG1 = Workload("cfg1_4k_mha_d64", 1, 8, 8, 4096, 64, 512, 128, 16, seed=0, values="normal")
CFG2 = Workload("cfg2_32k_gqa7_d128", 1, 28, 4, 32768, 128, 1024, 256, 4, seed=1, values="channel_offset")
CFG3 = Workload("cfg3_64k_gqa7_d128", 1, 28, 4, 65536, 128, 2048, 512, 4, seed=2, values="channel_offset")
CFG4 = Workload("cfg4_128k_b2_gqa4_d128", 2, 32, 8, 131072, 128, 4096, 1024, 4, seed=3, values="salient")
CONFIGS = {w.name: w for w in (CFG1, CFG2, CFG3, CFG4)}


def sweep_points():
    """Config 5: lag window x retention ratio sweep on the 32K GQA layer (one tensor set)."""
    base = Workload("cfg5_sweep", 1, 28, 4, 32768, 128, 1024, 256, 4, seed=4, values="normal")
    pts = []
    for L in (256, 512, 1024, 2048, 4096):
        for den in (16, 8, 4, 2):
            pts.append(base.with_(name=f"cfg5_L{L}_r1/{den}", L=L, K=L // den))
    return pts


def generate(w: Workload, tensors=("Q", "K", "V", "dO")) -> dict:
    """CPU bf16 tensors [B, H, N, d].  Tensors not requested are still drawn (and dropped) so
    that a requested tensor has the same values whichever subset is asked for."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    out = {k: torch.empty((w.B, w.Hq if k in ("Q", "dO") else w.Hkv, w.N, w.d), dtype=torch.bfloat16)
           for k in tensors}
    offset = None
    for b in range(w.B):
        for name in ("Q", "K", "V", "dO"):
            H = w.Hq if name in ("Q", "dO") else w.Hkv
            x = torch.randn((H, w.N, w.d), generator=g, dtype=torch.float32)
            if name == "K":
                if w.values == "channel_offset":
                    if offset is None:
                        offset = 2.0 * torch.randn((H, 1, w.d), generator=g, dtype=torch.float32)
                    x += offset
                elif w.values == "salient":
                    mark = torch.rand((H, w.N, 1), generator=g) < 0.01
                    x = torch.where(mark, x * 8.0, x)
            if name in out:
                out[name][b].copy_(x)
            del x
    return out
