from .gen import LengthDist, batch_lengths, instance_lengths, philox4x32_10  # noqa: F401
from .configs import (COST_MODEL, LAMBDA_NEVER_PREEMPT, LAMBDA_ONE, LAMBDA_PREFILL_FIRST,  # noqa: F401
                      Workload, paper_shaped, shard, workload)
