"""The five seeded workloads (shapes, planted structure, budgets, seeds).

`skip_scale` (the paper's Delta in the length-adaptive threshold ln(Delta/N),
Eq. 5) is frozen per workload so that every consumer passes the same number.  The
values were calibrated once with the fp64 oracle on a fixed sample of query blocks
of each seeded workload, so that the threshold alone (no cap) computes about 0.9x
the Stage-2 budget; the paper's own Delta = 2000 belongs to real Qwen3-8B
activations, whose logit gaps are far wider than this generator's.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

from .generator import Structure, make_qkv


@dataclass(frozen=True)
class Workload:
    name: str
    hq: int
    hkv: int
    n: int
    d: int = 128
    block: int = 128
    kap_budget: float = 0.25        # Stage-1 fraction of causal candidates kept
    osk_budget: float = 0.10        # Stage-2 ("tightened") fraction, cap on computed blocks
    stride: int = 8                 # KAP sampling stride s
    skip_scale: float = 2000.0      # Delta
    seed: int = 0
    structure: Structure = field(default_factory=Structure)
    layers: int = 1

    @property
    def n_blocks(self) -> int:
        return self.n // self.block

    def make(self, layer: int = 0, threads: int = 8):
        st = self.structure
        if self.layers > 1:                       # layer-varying needle density 8..128
            st = replace(st, needles=8 * 2 ** (layer % 5))
        return make_qkv(self.seed + layer, self.hq, self.hkv, self.n, self.d, self.block, st, threads)


WORKLOADS = {
    # small case: the CPU oracle finishes it in seconds
    "gqa4_4k": Workload("gqa4_4k", hq=4, hkv=1, n=4096, kap_budget=0.25, osk_budget=0.10,
                        skip_scale=3500.0, seed=1001, structure=Structure(band=2, needles=3)),
    "qwen3_32k": Workload("qwen3_32k", hq=32, hkv=8, n=32768, kap_budget=0.20, osk_budget=0.08,
                          skip_scale=20000.0, seed=2001, structure=Structure(band=4, needles=16)),
    "qwen3_128k": Workload("qwen3_128k", hq=32, hkv=8, n=131072, kap_budget=0.10, osk_budget=0.04,
                           skip_scale=90000.0, seed=3001, structure=Structure(band=4, needles=64)),
    "llama31_64k_sweep": Workload("llama31_64k_sweep", hq=32, hkv=8, n=65536, kap_budget=0.25,
                                  osk_budget=0.125, skip_scale=14500.0, seed=4001,
                                  structure=Structure(band=4, needles=32)),
    "qwen3_128k_x36": Workload("qwen3_128k_x36", hq=32, hkv=8, n=131072, kap_budget=0.10,
                               osk_budget=0.04, skip_scale=90000.0, seed=5000,
                               structure=Structure(band=4, needles=64), layers=36),
}

# the budget grid of the sweep workload: Stage-1 budget x (Stage-2 as a multiple of Stage-1)
SWEEP_STAGE1 = (0.5, 0.25, 0.125)
SWEEP_STAGE2_MULT = (1.0, 0.5, 0.25)


def tiny(seed: int = 7, hq: int = 2, hkv: int = 1, n: int = 1024, needles: int = 2, band: int = 2):
    """A test-sized workload with the same structure."""
    return Workload(f"tiny_{hq}x{hkv}x{n}", hq=hq, hkv=hkv, n=n, seed=seed,
                    structure=Structure(band=band, needles=needles))
