"""Worker of the world_size-2 gloo test: exercises the replica plumbing on CPU."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import numpy as np

from paper_2609_40093_b200 import inputs
from paper_2609_40093_b200.replicas import Replicas

rep = Replicas(backend="gloo")
cfg = inputs.shard_config(inputs.CONFIGS["C1"], rep.rank)
idx = inputs.make_topk_idx(cfg)
rep.barrier()
slow = rep.max_over_ranks(1.0 + rep.rank)                 # rank r "took" 1+r seconds
rate = rep.whole_job_rate(units_per_rank=64, seconds_this_rank=1.0 + rep.rank)
rep.barrier()
print(json.dumps({"rank": rep.rank, "world": rep.world, "slow": slow, "rate": rate,
                  "idx_sum": int(idx.sum()), "idx_head": idx[:4].ravel().tolist()}))
rep.close()
