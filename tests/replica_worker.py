"""Worker of test_replicas_gloo.py: one rank of a CPU (gloo) run of the replica bookkeeping."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2510_26577_b200 import replicas, workloads as wl  # noqa: E402


def main():
    r = replicas.init("gloo")
    w = replicas.workload_for_rank(wl.CONFIGS["c1_tiny"], r.rank)
    root = int(wl.root_tokens(w)[0])
    replicas.barrier(r)
    # rank k pretends to have processed 16 + k tokens in 1 + k milliseconds
    tokens, ms = replicas.aggregate(r, 16 + r.rank, 1.0 + r.rank)
    replicas.barrier(r)
    out = {"rank": r.rank, "world": r.world, "seed": w.seed, "root": root, "tokens": tokens, "ms": ms,
           "is_root": r.is_root}
    with open(os.path.join(sys.argv[1], f"rank{r.rank}.json"), "w") as f:
        json.dump(out, f)
    replicas.shutdown(r)


if __name__ == "__main__":
    main()
