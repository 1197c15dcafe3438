"""Named workloads: model shape, prefix, draft count, generation length, n-gram recipe.

Hyper-parameters are the paper's (Appendix B: alpha = 0.54, tau = 0.06 and interpolation
weights [0.01, 0.04, 0.15, 0.18, 0.12] for n = 2..6; Appendix C: alpha = 0.55, tau = 0.1 when
only n = 2..4 are used).  The paper gives no value for the penalty delta of Eq. 7; 0.01 is this
recipe's choice.  Prefix 15 tokens / drafts of 10 tokens follow Section 4.1.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

from .model import SHAPES, ModelShape

LAMBDA_2_TO_6: Tuple[float, ...] = (0.01, 0.04, 0.15, 0.18, 0.12)


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    prefix_kind: str
    prefix_len: int
    k: int
    gen_tokens: int               # tokens per draft: 1 from the first timestep + (gen_tokens - 1) steps
    orders: Tuple[int, ...]
    retain: int                   # n-grams kept per order (most frequent first)
    stream_len: int
    zipf_s: float
    alpha: float
    tau: float
    delta: float = 0.01
    max_pos: int = 4096
    kv_dtype: str = "bf16"
    lam: Tuple[float, ...] = field(default=LAMBDA_2_TO_6)

    def lambdas(self) -> List[float]:
        """lambda indexed by n - 2, eight entries."""
        out = [0.0] * 8
        for n in self.orders:
            out[n - 2] = self.lam[n - 2]
        return out


WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", SHAPES["tiny"], "uniform", 16, 3, 9, (2, 3, 4), 20_000, 200_000, 1.1,
                     0.55, 0.1, max_pos=256),
    "7b_k3": Workload("7b_k3", SHAPES["7b"], "zipf", 15, 3, 10, (2, 3, 4, 5, 6), 10_000_000,
                      200_000_000, 1.1, 0.54, 0.06),
    "7b_sweep": Workload("7b_sweep", SHAPES["7b"], "zipf", 15, 3, 32, (2, 3, 4, 5, 6), 10_000_000,
                         200_000_000, 1.1, 0.54, 0.06),
    "7b_long": Workload("7b_long", SHAPES["7b"], "zipf", 2048, 3, 128, (2, 3, 4, 5, 6), 10_000_000,
                        200_000_000, 1.1, 0.54, 0.06),
    "13b_k5": Workload("13b_k5", SHAPES["13b"], "zipf", 64, 5, 64, (2, 3, 4, 5, 6), 100_000_000,
                       200_000_000, 1.05, 0.54, 0.06),
}


def get_workload(name: str) -> Workload:
    return WORKLOADS[name]
