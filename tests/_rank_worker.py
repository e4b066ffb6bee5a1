"""Child process of tests/test_multi_rank.py: one gloo rank that reports made-up per-rank figures."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2005_06728_b200 import benchutil  # noqa: E402


def main():
    dist = benchutil.init_process_group("gloo")
    r = benchutil.rank_info()
    benchutil.barrier()
    # rank r pretends to have taken (10 + 5 r) ms for (r + 1) * 1000 bytes
    agg = benchutil.aggregate(10.0 + 5.0 * r["rank"], 1000.0 * (r["rank"] + 1))
    benchutil.barrier()
    if r["rank"] == 0:
        print(json.dumps(agg), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
