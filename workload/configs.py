"""The five synthetic workloads (sizes, length distributions, seeds, multipliers).

Pure description of inputs: no scheduling arithmetic lives here.  Every number
is an input to the method (request-table shape, client count, caps, the
integer-microsecond cost coefficients, the Q16.16 multipliers to sweep).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

from .gen import LengthDist, batch_lengths, estimated_outputs

# (prefill_fixed_us, prefill_per_token_us, decode_fixed_us, decode_per_seq_us,
#  decode_kv_div, est_per_prompt_token, est_per_output_token)
COST_MODEL: Tuple[int, ...] = (20000, 40, 15000, 300, 16, 40, 350)

SHORT_P = LengthDist(120.0, 0.4, 16, 512)
SHORT_O = LengthDist(130.0, 0.5, 8, 512)
LONG_P = LengthDist(300.0, 0.6, 16, 4096)
LONG_O = LengthDist(250.0, 0.7, 8, 2048)

LAMBDA_ONE = 1 << 16            # 1.0 in Q16.16
LAMBDA_PREFILL_FIRST = 0xFFFFFFFF
LAMBDA_NEVER_PREEMPT = 0


@dataclass(frozen=True)
class Workload:
    name: str
    seeds: Tuple[int, ...]
    n_req: int
    n_clients: int
    batch_cap: int
    kv_budget: int
    dist_p: LengthDist
    dist_o: LengthDist
    lambdas_q16: Tuple[int, ...] = (LAMBDA_ONE,)
    ls_rounds: int = 0
    cost_model: Tuple[int, ...] = COST_MODEL
    est_sigma: float = -1.0          # >= 0: the scheduler sees noisy output-length estimates
    kv_reserve: int = 0              # > 0: KV tokens reserved per request (needed with estimates)

    @property
    def n_inst(self) -> int:
        return len(self.seeds)

    def subset(self, first: int, count: int) -> "Workload":
        """The same workload restricted to instances [first, first+count)."""
        return Workload(self.name, self.seeds[first:first + count], self.n_req, self.n_clients,
                        self.batch_cap, self.kv_budget, self.dist_p, self.dist_o,
                        self.lambdas_q16, self.ls_rounds, self.cost_model, self.est_sigma, self.kv_reserve)

    def estimates(self):
        """uint32 table [n_inst][n_req] of estimated output lengths, or None when lengths are exact."""
        if self.est_sigma < 0:
            return None
        _, o = self.lengths()
        return np.stack([estimated_outputs(int(s), o[k], self.est_sigma, self.dist_o.lo, self.dist_o.hi)
                         for k, s in enumerate(self.seeds)])

    def lengths(self):
        """uint32 tables p, o of shape [n_inst][n_req]."""
        return batch_lengths(self.seeds, self.n_req, self.dist_p, self.dist_o)


def workload(name: str) -> Workload:
    if name == "c0":      # one small instance
        return Workload("c0", (0,), 200, 4, 16, 32768, SHORT_P, SHORT_O)
    if name == "c1":      # one math-QA-batch-shaped instance
        return Workload("c1", (1,), 1300, 8, 32, 65536, SHORT_P, SHORT_O)
    if name == "c2":      # 100-case study
        return Workload("c2", tuple(range(100, 200)), 1300, 8, 32, 65536, SHORT_P, SHORT_O)
    if name == "c3":      # multiplier sweep, 64 values k/16, 20 local-search rounds
        return Workload("c3", tuple(range(100, 200)), 1300, 8, 32, 65536, SHORT_P, SHORT_O,
                        tuple(k * 4096 for k in range(1, 65)), 20)
    if name == "c4":      # scale-out stress
        return Workload("c4", tuple(range(1000, 2024)), 20000, 64, 128, 262144, LONG_P, LONG_O,
                        (LAMBDA_ONE,), 100)
    if name == "c1e":     # c1 with output lengths known only up to a log-normal error (sigma 0.3);
        # every request reserves the largest prompt + the largest output
        return Workload("c1e", (1,), 1300, 8, 32, 65536, SHORT_P, SHORT_O, est_sigma=0.3, kv_reserve=1024)
    if name == "c2e":     # the 100-case study under the same uncertainty
        return Workload("c2e", tuple(range(100, 200)), 1300, 8, 32, 65536, SHORT_P, SHORT_O,
                        est_sigma=0.3, kv_reserve=1024)
    if name == "paper":   # shaped like the paper's own experiment (Table "Experiment settings")
        return paper_shaped()
    raise KeyError(name)


# Lengths with the paper's moments: input 68.43 +- 25.04 tokens, output 344.83 +- 187.99 capped at
# 512 (log-normals with those means and deviations before clipping).
PAPER_P = LengthDist(64.26, 0.3545, 4, 512)
PAPER_O = LengthDist(302.8, 0.5101, 1, 512)
# 0.13 ms per prompt token + 25 ms as a level table (Eq. 5-7), 0.21 ms per running request + 29 ms
# per decode round, no KV term; estimates count output tokens only.
PAPER_LEVELS = tuple((cap, 25000 + 130 * cap) for cap in (512, 1024, 2048, 4096, 8192, 16384))
PAPER_COST = (25000, 130, 29000, 210, 0x7FFFFFFF, 0, 71000, PAPER_LEVELS)


def paper_shaped(n_inst: int = 100, first_seed: int = 5000) -> Workload:
    """One client = the paper's whole system: 200 concurrent requests (1024 KV blocks of 128 tokens,
    five blocks per request), 1,319 requests per instance, lambda = 1.0."""
    return Workload("paper", tuple(range(first_seed, first_seed + n_inst)), 1319, 1, 200, 1024 * 128,
                    PAPER_P, PAPER_O, (LAMBDA_ONE,), 0, PAPER_COST)


def shard(n_units: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous block [first, first+count) of n_units owned by this rank (sizes differ by <= 1)."""
    base, extra = divmod(n_units, world_size)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)
