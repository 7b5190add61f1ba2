"""Worker of the two-process CPU test: what bench.py does around its timed region, with the gloo backend."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2511_15927_b200 import dist_util as D  # noqa: E402

rank, local_rank, world = D.env_ranks()
D.init("gloo", local_rank)
D.barrier()
ms = 10.0 * (rank + 1)                       # rank r "measured" 10 (r+1) ms for 4 steps
ms_max = D.max_over_ranks(ms)
value = D.whole_job_value(1000, 4, ms_max)   # 1000 tokens per rank and step
out = {"rank": rank, "world": world, "ms_max": ms_max, "value": value}
D.barrier()
if rank == 0:
    print(json.dumps(out), flush=True)       # one line, rank 0 only
D.shutdown()
