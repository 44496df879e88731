"""Worker of test_multirank_cpu.py: one rank of a gloo job on CPU.  Prints one JSON line."""
import hashlib
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402
import torch.distributed as dist  # noqa: E402

from oracle import direct  # noqa: E402
from paper_2208_00763_b200 import inputs, ranks  # noqa: E402


def main():
    world, rank, _ = ranks.rank_info()
    joined = ranks.init("gloo")
    case = inputs.c2_cases(1 << 12)[18]                     # a 4-bit case of the sweep, short signal
    f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"],
                              ranks.rank_seed(case["seed"], rank))
    y = direct.conv1d_full(f, g)                            # this rank's shard of the job, no exchange
    digest = hashlib.sha256(np.ascontiguousarray(f).tobytes()).hexdigest()
    ranks.barrier()
    my_ms = 10.0 + 5.0 * rank                               # stand-in for the device time of this rank
    job_ms = ranks.max_over_ranks(my_ms)
    macs = float(y.size) * case["K"]
    digests = [None] * world
    if joined:
        dist.all_gather_object(digests, digest)
    else:
        digests = [digest]
    out = {"rank": rank, "world": world, "joined": joined, "job_ms": job_ms, "digests": digests,
           "value": ranks.whole_job_rate(macs, 1, job_ms, world), "macs": macs, "checksum": int(y.sum())}
    ranks.shutdown()
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
